// CUDA-core cross-check evaluation of  y_t = W0 x_t + U_B (sB_k .* (M (sA_k .* (V_A^T x_t))))
// (Algorithm 1, line 7, without materialising the candidate's weight).  fp32 throughout, including the
// rank-r intermediate, so it is slightly more accurate than the tensor-core path.  Not used by
// essa_apply_projection.
#include "common.cuh"

namespace essa {
namespace {

// One CTA per token: p = V_A^T x_t (threads stride over d_in, shared-memory tree per rank coordinate),
// then u = sB .* (M (sA .* p)) written as fp32 [T][64].
__global__ void __launch_bounds__(256) simt_rank_kernel(const __nv_bfloat16* __restrict__ x, int n, int r,
                                                        const __nv_bfloat16* __restrict__ V_A,
                                                        const float* __restrict__ M, const int32_t* __restrict__ off,
                                                        int P, const float* __restrict__ sigma, int ld_sigma,
                                                        int sA_col, int sB_col, float* __restrict__ u_out) {
  __shared__ float part[8][kRankPadMax];
  __shared__ float q[kRankPadMax];
  const int t = blockIdx.x;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // each warp handles a strided set of input features; each lane a strided set of rank coordinates
  float acc[2] = {0.f, 0.f};  // coordinates lane and lane+32
  for (int c = warp; c < n; c += 8) {
    const float xv = __bfloat162float(x[(size_t)t * n + c]);
    if (lane < r) acc[0] = fmaf(__bfloat162float(V_A[(size_t)c * r + lane]), xv, acc[0]);
    if (lane + 32 < r) acc[1] = fmaf(__bfloat162float(V_A[(size_t)c * r + lane + 32]), xv, acc[1]);
  }
  part[warp][lane] = acc[0];
  part[warp][lane + 32] = acc[1];
  __syncthreads();
  const int k = find_candidate(off, P, t);
  if (threadIdx.x < kRankPadMax) {
    const int i = threadIdx.x;
    float p = 0.f;
    for (int w = 0; w < 8; ++w) p += part[w][i];
    q[i] = (i < r) ? sigma[(size_t)k * ld_sigma + sA_col + i] * p : 0.f;
  }
  __syncthreads();
  if (threadIdx.x < kRankPadMax) {
    const int j = threadIdx.x;
    float v = 0.f;
    for (int i = 0; i < r; ++i) v = fmaf(M[j * kRankPadMax + i], q[i], v);
    u_out[(size_t)t * kRankPadMax + j] = (j < r) ? sigma[(size_t)k * ld_sigma + sB_col + j] * v : 0.f;
  }
}

// 64 x 64 output tile per CTA, 16-wide K chunks, 4 x 4 outputs per thread.
// kQ: 0 = bf16 W0, 1 = INT8 codes with a per-channel scale, 2 = INT4 codes (two per byte) with per-group scales.
template <int kQ>
__global__ void __launch_bounds__(256) simt_gemm_kernel(const __nv_bfloat16* __restrict__ x, int T, int n, int m, int r,
                                                        const void* __restrict__ W0v, const __half* __restrict__ scale,
                                                        const __nv_bfloat16* __restrict__ U_B,
                                                        const float* __restrict__ u, __nv_bfloat16* __restrict__ y) {
  __shared__ float xs[16][65];
  __shared__ float ws[16][65];
  const int t0 = blockIdx.y * 64, o0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;  // tx -> channels, ty -> tokens
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; ++a)
#pragma unroll
    for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;

  auto tile_pass = [&](auto load_x, auto load_w, int kdim) {
    for (int c0 = 0; c0 < kdim; c0 += 16) {
      for (int idx = threadIdx.x; idx < 64 * 16; idx += 256) {
        const int row = idx >> 4, c = idx & 15;
        xs[c][row] = (t0 + row < T && c0 + c < kdim) ? load_x(t0 + row, c0 + c) : 0.f;
        ws[c][row] = (o0 + row < m && c0 + c < kdim) ? load_w(o0 + row, c0 + c) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        float xv[4], wv[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) xv[a] = xs[c][ty * 4 + a];
#pragma unroll
        for (int b = 0; b < 4; ++b) wv[b] = ws[c][tx * 4 + b];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xv[a], wv[b], acc[a][b]);
      }
      __syncthreads();
    }
  };

  // base contraction W0 x
  tile_pass([&](int t, int c) { return __bfloat162float(x[(size_t)t * n + c]); },
            [&](int o, int c) {
              if constexpr (kQ == 1) {
                return (float)reinterpret_cast<const int8_t*>(W0v)[(size_t)o * n + c];
              } else if constexpr (kQ == 2) {
                const uint32_t byte = reinterpret_cast<const uint8_t*>(W0v)[((size_t)o * n + c) >> 1];
                const int nib = (c & 1) ? (int)(byte >> 4) : (int)(byte & 15u);
                return (float)((nib ^ 8) - 8) * __half2float(scale[(size_t)o * (n / 128) + c / 128]);
              } else {
                return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(W0v)[(size_t)o * n + c]);
              }
            },
            n);
  if constexpr (kQ == 1) {
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int o = o0 + tx * 4 + b;
      const float s = (o < m) ? __half2float(scale[o]) : 0.f;
#pragma unroll
      for (int a = 0; a < 4; ++a) acc[a][b] *= s;
    }
  }
  // up-projection U_B u
  tile_pass([&](int t, int j) { return u[(size_t)t * kRankPadMax + j]; },
            [&](int o, int j) { return __bfloat162float(U_B[(size_t)o * r + j]); }, r);

#pragma unroll
  for (int a = 0; a < 4; ++a) {
    const int t = t0 + ty * 4 + a;
    if (t >= T) continue;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
      const int o = o0 + tx * 4 + b;
      if (o < m) y[(size_t)t * m + o] = __float2bfloat16(acc[a][b]);
    }
  }
}

}  // namespace

int32_t launch_projection_simt(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, cudaStream_t stream) {
  if (g.T == 0) return ESSA_OK;
  int32_t st = ensure_scratch(ctx, ctx->simt_buf, (size_t)g.T * kRankPadMax * sizeof(float), false, stream);
  if (st != ESSA_OK) return st;
  float* u = static_cast<float*>(ctx->simt_buf.ptr);
  simt_rank_kernel<<<(unsigned)g.T, 256, 0, stream>>>(g.x, a->d_in, a->rank, a->V_A, a->M, g.seg_offsets, g.P, g.sigma,
                                                      g.ld_sigma, g.sA_col, g.sB_col, u);
  dim3 grid((a->d_out + 63) / 64, (unsigned)((g.T + 63) / 64));
  if (a->w0_dtype == ESSA_W0_INT8_PERCHANNEL)
    simt_gemm_kernel<1><<<grid, 256, 0, stream>>>(g.x, (int)g.T, a->d_in, a->d_out, a->rank, a->W0q, a->w0_scale, a->U_B, u, g.y);
  else if (a->w0_dtype == ESSA_W0_INT4_GROUP128)
    simt_gemm_kernel<2><<<grid, 256, 0, stream>>>(g.x, (int)g.T, a->d_in, a->d_out, a->rank, a->W0q, a->w0_gscale, a->U_B, u, g.y);
  else
    simt_gemm_kernel<0><<<grid, 256, 0, stream>>>(g.x, (int)g.T, a->d_in, a->d_out, a->rank, a->W0, nullptr, a->U_B, u, g.y);
  ctx->launches += 2;
  return check_cuda(ctx, cudaGetLastError(), "simt projection launch");
}

}  // namespace essa
