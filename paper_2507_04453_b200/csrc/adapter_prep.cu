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

// INT8 codes -> bf16 (exact), 16 codes per thread.  count is a multiple of 64 (d_in is).
__global__ void widen_int8_kernel(const int8_t* __restrict__ q, __nv_bfloat16* __restrict__ out, size_t count) {
  const size_t i = (blockIdx.x * (size_t)blockDim.x + threadIdx.x) * 16;
  if (i >= count) return;
  const uint4 w = *reinterpret_cast<const uint4*>(q + i);
  uint4 o0, o1;
  int8x4_to_bf16x4(w.x, o0.x, o0.y);
  int8x4_to_bf16x4(w.y, o0.z, o0.w);
  int8x4_to_bf16x4(w.z, o1.x, o1.y);
  int8x4_to_bf16x4(w.w, o1.z, o1.w);
  reinterpret_cast<uint4*>(out + i)[0] = o0;
  reinterpret_cast<uint4*>(out + i)[1] = o1;
}

}  // namespace

int32_t launch_widen_int8(essa_ctx* ctx, const int8_t* q, __nv_bfloat16* out, size_t count, cudaStream_t stream) {
  const size_t threads = (count + 15) / 16;
  widen_int8_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(q, out, count);
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
