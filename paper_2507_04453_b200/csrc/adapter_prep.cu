// One-time re-layout of an adapter's frozen bases (Section 3, "LoRA + SVD parameterization") into the
// operand formats the projection kernels consume, and the r x r core M = V_B^T U_A.
#include "common.cuh"

namespace essa {
namespace {

// VAt[j][c] = V_A[c][j] for j < r, 0 for r <= j < 64.   (K-major B operand of p = V_A^T x)
__global__ void build_vat_kernel(const __nv_bfloat16* __restrict__ V_A, int n, int r, __nv_bfloat16* __restrict__ VAt) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n) return;
  for (int j = 0; j < kRankPadMax; ++j) VAt[(size_t)j * n + c] = (j < r) ? V_A[(size_t)c * r + j] : __float2bfloat16(0.f);
}

// UBp[e][o][j]: bf16 W0 -> one slab, U_B[o][j] zero-padded to 64 columns.
// INT8 W0 -> two slabs holding g = U_B[o][j] / scale[o] split as hi = bf16(g), lo = bf16(g - hi), because the
// kernel multiplies the whole accumulator (base + rank term) by scale[o] once at the end.
__global__ void build_ubp_kernel(const __nv_bfloat16* __restrict__ U_B, const __half* __restrict__ scale, int m, int r,
                                 int ext, __nv_bfloat16* __restrict__ UBp) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= m * kRankPadMax) return;
  const int o = idx / kRankPadMax, j = idx % kRankPadMax;
  float g = (j < r) ? __bfloat162float(U_B[(size_t)o * r + j]) : 0.f;
  if (ext == 1) {
    UBp[idx] = __float2bfloat16(g);
  } else {
    const float s = __half2float(scale[o]);
    g = (s != 0.f) ? g / s : 0.f;
    const __nv_bfloat16 hi = __float2bfloat16(g);
    UBp[idx] = hi;
    UBp[(size_t)m * kRankPadMax + idx] = __float2bfloat16(g - __bfloat162float(hi));
  }
}

// M[j][i] = sum_l V_B[l][j] * U_A[l][i]  (fp32), zero-padded to 64 x 64.
__global__ void build_core_kernel(const __nv_bfloat16* __restrict__ U_A, const __nv_bfloat16* __restrict__ V_B, int r,
                                  float* __restrict__ M) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= kRankPadMax * kRankPadMax) return;
  const int j = idx / kRankPadMax, i = idx % kRankPadMax;
  float acc = 0.f;
  if (j < r && i < r)
    for (int l = 0; l < r; ++l) acc = fmaf(__bfloat162float(V_B[l * r + j]), __bfloat162float(U_A[l * r + i]), acc);
  M[idx] = acc;
}

// INT8 codes -> bf16 (exact).  A block takes 8192 consecutive codes in four rounds; per round a thread widens eight
// codes, so a warp's loads (256 B) and stores (512 B) are each one contiguous run.  count is a multiple of 64 (d_in is).
constexpr int kWidenPerBlock = 8192;
__global__ void __launch_bounds__(256) widen_int8_kernel(const int8_t* __restrict__ q, __nv_bfloat16* __restrict__ out, size_t count) {
  const size_t base = (size_t)blockIdx.x * kWidenPerBlock + (size_t)threadIdx.x * 8;
  uint2 w[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const size_t i = base + (size_t)k * 2048;
    w[k] = i < count ? __ldg(reinterpret_cast<const uint2*>(q + i)) : make_uint2(0u, 0u);
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const size_t i = base + (size_t)k * 2048;
    uint4 o;
    int8x4_to_bf16x4(w[k].x, o.x, o.y);
    int8x4_to_bf16x4(w[k].y, o.z, o.w);
    if (i < count) *reinterpret_cast<uint4*>(out + i) = o;
  }
}

// INT4 group-wise codes -> bf16 weights (code * group scale, rounded once); same tiling: per round a thread widens the
// eight codes of four packed bytes, which share a group (groups are 128 wide and d_in is a multiple of 128).
__global__ void __launch_bounds__(256) widen_int4_kernel(const uint8_t* __restrict__ packed, const __half* __restrict__ gscale,
                                                         __nv_bfloat16* __restrict__ out, int d_in, size_t count) {
  const size_t base = (size_t)blockIdx.x * kWidenPerBlock + (size_t)threadIdx.x * 8;  // first weight of this thread
  const int groups = d_in / 128;
  uint32_t w[4];
  float s[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const size_t i = base + (size_t)k * 2048;
    const bool in = i < count;
    const size_t o = i / d_in, c = i % d_in;
    w[k] = in ? __ldg(reinterpret_cast<const uint32_t*>(packed + i / 2)) : 0u;
    s[k] = in ? __half2float(gscale[o * groups + c / 128]) : 0.f;
  }
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const size_t i = base + (size_t)k * 2048;
    uint32_t v[4];
    int4x8_to_bf16x8(w[k], s[k], v);
    if (i < count) *reinterpret_cast<uint4*>(out + i) = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

// Candidate reconstruction (Algorithm 1, line 7: A' = U_A diag(sA_k) V_A^T, B' = U_B diag(sB_k) V_B^T), for export to
// an engine that wants the dense LoRA factors.  CUDA cores: 2 r^2 (n + m) FLOP per candidate against 2 r (n + m)
// bytes written, i.e. r FLOP per byte; RP = rank rounded up to 16 keeps the per-thread vectors in registers.
// A'[i][c] = sum_j U_A[i][j] sA[j] V_A[c][j]: one thread per input feature c, blockIdx.y = candidate; a thread scales
// its row of V_A once and takes the r dot products with the rows of U_A (shared memory, broadcast reads); the stores
// of a warp are consecutive in c.
template <int RP>
__global__ void __launch_bounds__(128) export_a_kernel(const __nv_bfloat16* __restrict__ U_A, const __nv_bfloat16* __restrict__ V_A,
                                                      int n, int r, const float* __restrict__ sigma, int ld_sigma, int sA_col,
                                                      int k_begin, __nv_bfloat16* __restrict__ A_out) {
  __shared__ __align__(16) float ua[RP * RP];
  __shared__ float sa[RP];
  const int kk = blockIdx.y;
  for (int idx = threadIdx.x; idx < RP * RP; idx += blockDim.x) {
    const int i = idx / RP, j = idx % RP;
    ua[idx] = (i < r && j < r) ? __bfloat162float(U_A[i * r + j]) : 0.f;
  }
  if (threadIdx.x < RP) sa[threadIdx.x] = threadIdx.x < r ? sigma[(size_t)(k_begin + kk) * ld_sigma + sA_col + threadIdx.x] : 0.f;
  __syncthreads();
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= n) return;
  float w[RP];
#pragma unroll
  for (int j = 0; j < RP; ++j) w[j] = j < r ? sa[j] * __bfloat162float(V_A[(size_t)c * r + j]) : 0.f;
  __nv_bfloat16* out = A_out + (size_t)kk * r * n + c;
  for (int i = 0; i < r; ++i) {
    float acc = 0.f;
#pragma unroll
    for (int j = 0; j < RP; j += 4) {  // one 16-byte broadcast read per four multiply-adds
      const float4 u4 = *reinterpret_cast<const float4*>(ua + i * RP + j);
      acc = fmaf(u4.x, w[j], acc);
      acc = fmaf(u4.y, w[j + 1], acc);
      acc = fmaf(u4.z, w[j + 2], acc);
      acc = fmaf(u4.w, w[j + 3], acc);
    }
    out[(size_t)i * n] = __float2bfloat16(acc);
  }
}

// B'[o][j] = sum_i U_B[o][i] sB[i] V_B[j][i]: one thread per output channel o, blockIdx.y = candidate.  The 128 rows
// of a block are one contiguous piece of the output: they are staged in shared memory and stored 16 bytes at a time.
template <int RP>
__global__ void __launch_bounds__(128) export_b_kernel(const __nv_bfloat16* __restrict__ U_B, const __nv_bfloat16* __restrict__ V_B,
                                                      int m, int r, const float* __restrict__ sigma, int ld_sigma, int sB_col,
                                                      int k_begin, __nv_bfloat16* __restrict__ B_out) {
  __shared__ __align__(16) float vb[RP * RP];
  __shared__ float sb[RP];
  __shared__ __align__(16) __nv_bfloat16 tile[128 * RP];  // [row][r], packed
  const int kk = blockIdx.y;
  for (int idx = threadIdx.x; idx < RP * RP; idx += blockDim.x) {
    const int j = idx / RP, i = idx % RP;
    vb[idx] = (i < r && j < r) ? __bfloat162float(V_B[j * r + i]) : 0.f;
  }
  if (threadIdx.x < RP) sb[threadIdx.x] = threadIdx.x < r ? sigma[(size_t)(k_begin + kk) * ld_sigma + sB_col + threadIdx.x] : 0.f;
  __syncthreads();
  const int o0 = blockIdx.x * 128;
  const int o = o0 + threadIdx.x;
  if (o < m) {
    float w[RP];
#pragma unroll
    for (int i = 0; i < RP; ++i) w[i] = i < r ? sb[i] * __bfloat162float(U_B[(size_t)o * r + i]) : 0.f;
    for (int j = 0; j < r; ++j) {
      float acc = 0.f;
#pragma unroll
      for (int i = 0; i < RP; i += 4) {
        const float4 v4 = *reinterpret_cast<const float4*>(vb + j * RP + i);
        acc = fmaf(v4.x, w[i], acc);
        acc = fmaf(v4.y, w[i + 1], acc);
        acc = fmaf(v4.z, w[i + 2], acc);
        acc = fmaf(v4.w, w[i + 3], acc);
      }
      tile[threadIdx.x * r + j] = __float2bfloat16(acc);
    }
  }
  __syncthreads();
  const int rows = min(128, m - o0);
  const size_t bytes = (size_t)rows * r * 2;  // m is a multiple of 8: a multiple of 16 bytes, and the piece starts 16-byte aligned
  uint4* dst = reinterpret_cast<uint4*>(B_out + ((size_t)kk * m + o0) * r);
  const uint4* src = reinterpret_cast<const uint4*>(tile);
  for (size_t v = threadIdx.x; v < bytes / 16; v += blockDim.x) dst[v] = src[v];
}

}  // namespace

int32_t launch_export_candidates(essa_ctx* ctx, const essa_adapter* a, const float* sigma, int32_t ld_sigma, int32_t sA_col,
                                 int32_t sB_col, int32_t k_begin, int32_t k_count, __nv_bfloat16* A_out, __nv_bfloat16* B_out,
                                 cudaStream_t stream) {
  if (k_count == 0) return ESSA_OK;
  if (A_out) {
    dim3 grid((unsigned)((a->d_in + 127) / 128), (unsigned)k_count);
    switch (a->r_pad) {
      case 16: export_a_kernel<16><<<grid, 128, 0, stream>>>(a->U_A, a->V_A, a->d_in, a->rank, sigma, ld_sigma, sA_col, k_begin, A_out); break;
      case 32: export_a_kernel<32><<<grid, 128, 0, stream>>>(a->U_A, a->V_A, a->d_in, a->rank, sigma, ld_sigma, sA_col, k_begin, A_out); break;
      case 48: export_a_kernel<48><<<grid, 128, 0, stream>>>(a->U_A, a->V_A, a->d_in, a->rank, sigma, ld_sigma, sA_col, k_begin, A_out); break;
      default: export_a_kernel<64><<<grid, 128, 0, stream>>>(a->U_A, a->V_A, a->d_in, a->rank, sigma, ld_sigma, sA_col, k_begin, A_out); break;
    }
    ctx->launches += 1;
  }
  if (B_out) {
    dim3 grid((unsigned)((a->d_out + 127) / 128), (unsigned)k_count);
    switch (a->r_pad) {
      case 16: export_b_kernel<16><<<grid, 128, 0, stream>>>(a->U_B, a->V_B, a->d_out, a->rank, sigma, ld_sigma, sB_col, k_begin, B_out); break;
      case 32: export_b_kernel<32><<<grid, 128, 0, stream>>>(a->U_B, a->V_B, a->d_out, a->rank, sigma, ld_sigma, sB_col, k_begin, B_out); break;
      case 48: export_b_kernel<48><<<grid, 128, 0, stream>>>(a->U_B, a->V_B, a->d_out, a->rank, sigma, ld_sigma, sB_col, k_begin, B_out); break;
      default: export_b_kernel<64><<<grid, 128, 0, stream>>>(a->U_B, a->V_B, a->d_out, a->rank, sigma, ld_sigma, sB_col, k_begin, B_out); break;
    }
    ctx->launches += 1;
  }
  return check_cuda(ctx, cudaGetLastError(), "export_candidates launch");
}

int32_t launch_widen_int4(essa_ctx* ctx, const uint8_t* packed, const __half* gscale, __nv_bfloat16* out, int d_out, int d_in,
                          cudaStream_t stream) {
  const size_t count = (size_t)d_out * d_in;
  if (count == 0) return ESSA_OK;
  widen_int4_kernel<<<(unsigned)((count + kWidenPerBlock - 1) / kWidenPerBlock), 256, 0, stream>>>(packed, gscale, out, d_in, count);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "widen_int4 launch");
}

int32_t launch_widen_int8(essa_ctx* ctx, const int8_t* q, __nv_bfloat16* out, size_t count, cudaStream_t stream) {
  if (count == 0) return ESSA_OK;
  widen_int8_kernel<<<(unsigned)((count + kWidenPerBlock - 1) / kWidenPerBlock), 256, 0, stream>>>(q, out, count);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "widen_int8 launch");
}

int32_t launch_adapter_prep(essa_ctx* ctx, essa_adapter* a, const __nv_bfloat16* U_A, const __nv_bfloat16* V_B,
                            cudaStream_t stream) {
  build_vat_kernel<<<(a->d_in + 127) / 128, 128, 0, stream>>>(a->V_A, a->d_in, a->rank, a->VAt);
  const int tot = a->d_out * kRankPadMax;
  build_ubp_kernel<<<(tot + 255) / 256, 256, 0, stream>>>(a->U_B, a->w0_scale, a->d_out, a->rank, a->ext_blocks, a->UBp);
  build_core_kernel<<<(kRankPadMax * kRankPadMax + 255) / 256, 256, 0, stream>>>(U_A, V_B, a->rank, a->M);
  ctx->launches += 3;
  return check_cuda(ctx, cudaGetLastError(), "adapter prep launch");
}

}  // namespace essa
