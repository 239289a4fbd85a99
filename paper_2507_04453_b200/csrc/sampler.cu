// Candidate sampling: sigma_k = mean + step * Bfactor (Dvec .* z_k), z_k from a counter-based stream
// (Section 3, "Evolutionary optimization": x^(k) ~ N(m_t, sigma_t^2 C_t), regenerable from a seed;
//  Algorithm 1, line 5).  Philox4x32-10 (Salmon et al., SC'11) + Box-Muller, all in this file.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u, kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kWeyl0 = 0x9E3779B9u, kWeyl1 = 0xBB67AE85u;

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint2 k) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(kPhiloxM0, c.x), lo0 = kPhiloxM0 * c.x;
    const uint32_t hi1 = __umulhi(kPhiloxM1, c.z), lo1 = kPhiloxM1 * c.z;
    c = make_uint4(hi1 ^ c.y ^ k.x, lo1, hi0 ^ c.w ^ k.y, lo0);
    k.x += kWeyl0;
    k.y += kWeyl1;
  }
  return c;
}

// Word -> uniform strictly inside (0,1): (2*(w>>9)+1) * 2^-24 (exact).
__device__ __forceinline__ double uniform_open01(uint32_t w) { return static_cast<double>(2u * (w >> 9) + 1u) * 0x1p-24; }

// The transform and the covariance product run in fp64 and the result is rounded to fp32 once, so the table
// matches a double-precision evaluation to fp32 rounding for any step size (the work is tiny: P*d normals).
__device__ __forceinline__ void box_muller(uint32_t w_radius, uint32_t w_angle, double& z0, double& z1) {
  const double rho = sqrt(-2.0 * log(uniform_open01(w_radius)));
  double s, c;
  sincospi(2.0 * uniform_open01(w_angle), &s, &c);  // angle = 2*pi*u
  z0 = rho * c;
  z1 = rho * s;
}

// Four standard normals: coordinates 4j..4j+3 of candidate k.
__device__ __forceinline__ void normals_block(uint2 key, uint32_t j, uint32_t k, double (&z)[4]) {
  const uint4 w = philox4x32_10(make_uint4(j, k, 0u, 0u), key);
  box_muller(w.x, w.y, z[0], z[1]);
  box_muller(w.z, w.w, z[2], z[3]);
}

// Completion count for a consumer that runs concurrently (the decode kernel of a fused draw + block call): every
// block adds one, after its rows of the table are visible device-wide.
__device__ __forceinline__ void block_done(uint32_t* done) {
  if (done == nullptr) return;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) red_release_add_u32(done, 1u);
}

// Identity covariance factor: sigma[k][i] = mean[i] + step * Dvec[i] * z_k[i].  One thread per (k, block j).
__global__ void sample_diag_kernel(const float* __restrict__ mean, float step, const float* __restrict__ Dvec, int d,
                                   uint2 key, int k_begin, int k_count, const int32_t* __restrict__ index, int ld_out,
                                   float* __restrict__ sigma_out, uint32_t* done, const float* __restrict__ step_ptr) {
  grid_dep_launch();  // a dependent launch of the next kernel may begin its set-up; it reads sigma after its own wait
  if (step_ptr != nullptr) step = *step_ptr;  // step size kept in device memory (search-distribution state)
  const int nb = (d + 3) >> 2;
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx < (long long)k_count * nb) {
    const int kk = (int)(idx / nb), j = (int)(idx % nb);
    double zz[4];
    normals_block(key, (uint32_t)j, (uint32_t)(k_begin + kk), zz);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int i = 4 * j + e;
      if (i < d) {
        const double w = Dvec ? (double)Dvec[i] * zz[e] : zz[e];
        const int col = index ? index[i] : i;  // top-alpha: coordinate i of the optimised vector sits in column index[i]
        if (col >= 0 && col < ld_out) sigma_out[(size_t)kk * ld_out + col] = (float)((double)mean[i] + (double)step * w);
      }
    }
  }
  block_done(done);
}

// Full covariance factor.  blockIdx.x = group of kCand candidates, blockIdx.y = tile of kRows rows of Bfactor.
// Phase 1: w[c][j] = Dvec[j] * z_c[j] into shared memory (every block regenerates its candidates' normals).
// Phase 2: a warp owns eight rows at once: lane = 4 * row + quarter, each quarter of a row's lanes strides over
// the columns (16-byte loads when the rows are 16-byte aligned), so a row's sum is finished by two shuffle steps
// and all eight rows' loads are in flight together; the quarter-0 lane writes mean[i] + step * acc.
constexpr int kCand = 4, kRows = 64, kSamplerThreads = 256;

template <bool VEC>
__global__ void __launch_bounds__(kSamplerThreads) sample_full_kernel(const float* __restrict__ mean, float step,
                                                                      const float* __restrict__ Bfactor,
                                                                      const float* __restrict__ Dvec, int d, uint2 key,
                                                                      int k_begin, int k_count,
                                                                      const int32_t* __restrict__ index, int ld_out,
                                                                      float* __restrict__ sigma_out, uint32_t* done,
                                                                      const float* __restrict__ step_ptr) {
  extern __shared__ __align__(16) double w_smem[];  // [kCand][d4], d4 = 4*ceil(d/4)
  grid_dep_launch();  // a dependent launch of the next kernel may begin its set-up; it reads sigma after its own wait
  if (step_ptr != nullptr) step = *step_ptr;  // step size kept in device memory (search-distribution state)
  const int nb = (d + 3) >> 2, d4 = nb * 4;
  const int kk0 = blockIdx.x * kCand;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, q = lane & 3;
  const int i = blockIdx.y * kRows + warp * 8 + r;
  const bool live = i < d;
  const float* brow = Bfactor + (size_t)(live ? i : d - 1) * d;  // idle lanes re-read the last row and drop the sum
  // the first 128 columns of the row are requested before the normals are generated, so the loads' latency
  // hides behind the transform
  constexpr int kPrefetch = 8;
  float4 pre[kPrefetch];
  if (VEC) {
#pragma unroll
    for (int u = 0; u < kPrefetch; ++u) {
      const int j0 = 4 * q + 16 * u;
      pre[u] = (j0 < d) ? __ldg(reinterpret_cast<const float4*>(brow + j0)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }
  // one thread per Box-Muller pair: coordinates 4j + 2h, 4j + 2h + 1 of candidate c (both halves of a block
  // recompute the block's four words, which costs far less than the transform)
  for (int idx = threadIdx.x; idx < kCand * nb * 2; idx += blockDim.x) {
    const int c = idx / (nb * 2), jh = idx % (nb * 2), j = jh >> 1, h = jh & 1;
    double z0 = 0.0, z1 = 0.0;
    if (kk0 + c < k_count) {
      const uint4 w = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)(k_begin + kk0 + c), 0u, 0u), key);
      box_muller(h ? w.z : w.x, h ? w.w : w.y, z0, z1);
    }
    const int i0 = 4 * j + 2 * h;
    w_smem[c * d4 + i0] = (i0 < d) ? (Dvec ? (double)Dvec[i0] * z0 : z0) : 0.0;
    w_smem[c * d4 + i0 + 1] = (i0 + 1 < d) ? (Dvec ? (double)Dvec[i0 + 1] * z1 : z1) : 0.0;
  }
  __syncthreads();
  double acc[kCand];
#pragma unroll
  for (int c = 0; c < kCand; ++c) acc[c] = 0.0;
  if (VEC) {  // d % 4 == 0 and Bfactor 16-byte aligned
    auto consume = [&](const float4& b4, int j0) {
      const double b[4] = {(double)b4.x, (double)b4.y, (double)b4.z, (double)b4.w};
#pragma unroll
      for (int c = 0; c < kCand; ++c) {
        const double2 w01 = *reinterpret_cast<const double2*>(w_smem + c * d4 + j0);
        const double2 w23 = *reinterpret_cast<const double2*>(w_smem + c * d4 + j0 + 2);
        acc[c] = fma(b[0], w01.x, acc[c]);
        acc[c] = fma(b[1], w01.y, acc[c]);
        acc[c] = fma(b[2], w23.x, acc[c]);
        acc[c] = fma(b[3], w23.y, acc[c]);
      }
    };
#pragma unroll
    for (int u = 0; u < kPrefetch; ++u) {
      const int j0 = 4 * q + 16 * u;
      if (j0 < d) consume(pre[u], j0);
    }
#pragma unroll 8
    for (int j0 = 4 * q + 16 * kPrefetch; j0 < d; j0 += 16)
      consume(__ldg(reinterpret_cast<const float4*>(brow + j0)), j0);
  } else {
#pragma unroll 4
    for (int j = q; j < d; j += 4) {
      const double b = (double)__ldg(brow + j);
#pragma unroll
      for (int c = 0; c < kCand; ++c) acc[c] = fma(b, w_smem[c * d4 + j], acc[c]);
    }
  }
#pragma unroll
  for (int c = 0; c < kCand; ++c) {
    acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 1);
    acc[c] += __shfl_xor_sync(0xffffffffu, acc[c], 2);
  }
  if (live && q == 0) {
    const double mi = (double)mean[i];
    const int col = index ? index[i] : i;
    if (col >= 0 && col < ld_out) {
#pragma unroll
      for (int c = 0; c < kCand; ++c)
        if (kk0 + c < k_count) sigma_out[(size_t)(kk0 + c) * ld_out + col] = (float)(mi + (double)step * acc[c]);
    }
  }
  block_done(done);
}

__global__ void stream_words_kernel(uint2 key, int k_begin, int k_count, int n_blocks, uint32_t* __restrict__ out) {
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx >= (long long)k_count * n_blocks) return;
  const int kk = (int)(idx / n_blocks), j = (int)(idx % n_blocks);
  const uint4 w = philox4x32_10(make_uint4((uint32_t)j, (uint32_t)(k_begin + kk), 0u, 0u), key);
  reinterpret_cast<uint4*>(out)[idx] = w;
}

__global__ void philox_once_kernel(uint4 ctr, uint2 key, uint32_t* out) {
  const uint4 w = philox4x32_10(ctr, key);
  out[0] = w.x; out[1] = w.y; out[2] = w.z; out[3] = w.w;
}

__global__ void segment_map_kernel(const int32_t* __restrict__ off, int P, int T, int32_t* __restrict__ cand) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < T) cand[t] = find_candidate(off, P, t);
}

inline uint2 key_of(uint64_t seed) { return make_uint2((uint32_t)(seed & 0xffffffffull), (uint32_t)(seed >> 32)); }

// Rows of the table = frozen values everywhere (top-alpha: the coordinates the optimiser does not see).
__global__ void fill_rows_kernel(const float* __restrict__ frozen, int d, int k_count, float* __restrict__ sigma_out) {
  const long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (idx < (long long)k_count * d) sigma_out[idx] = frozen[idx % d];
}

}  // namespace

int32_t launch_fill_rows(essa_ctx* ctx, const float* frozen, int32_t d, int32_t k_count, float* sigma_out, cudaStream_t stream) {
  const long long total = (long long)k_count * d;
  if (total == 0) return ESSA_OK;
  fill_rows_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(frozen, d, k_count, sigma_out);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "fill_rows launch");
}

// index != NULL: coordinate i of the sampled vector is written to column index[i] of rows of ld_out floats.
// done != NULL: every block of the launch adds one to *done when its part of the table is visible; *blocks_out
// receives the number of blocks launched (0 when nothing was launched).  step_dev != NULL: the step size is read
// from device memory instead of `step`.
int32_t launch_sampler(essa_ctx* ctx, const float* mean, float step, const float* Bfactor, const float* Dvec, int32_t d,
                       uint64_t seed, int32_t k_begin, int32_t k_count, const int32_t* index, int32_t ld_out, float* sigma_out,
                       cudaStream_t stream, uint32_t* done, uint32_t* blocks_out, const float* step_dev) {
  if (blocks_out) *blocks_out = 0;
  if (k_count == 0 || d == 0) return ESSA_OK;
  const int nb = (d + 3) / 4;
  if (Bfactor == nullptr) {
    const long long total = (long long)k_count * nb;
    const int threads = 256;
    const long long blocks = (total + threads - 1) / threads;
    if (blocks > 0x7fffffffLL) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "sample_population: P*d too large");
    sample_diag_kernel<<<(unsigned)blocks, threads, 0, stream>>>(mean, step, Dvec, d, key_of(seed), k_begin, k_count, index,
                                                                 ld_out, sigma_out, done, step_dev);
    if (blocks_out) *blocks_out = (uint32_t)blocks;
  } else {
    if (d > 4096) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "sample_population: d > 4096 with a full covariance factor");
    const size_t smem = (size_t)kCand * nb * 4 * sizeof(double);
    const bool vec = (d % 4 == 0) && (reinterpret_cast<uintptr_t>(Bfactor) % 16 == 0);
    auto kernel = vec ? sample_full_kernel<true> : sample_full_kernel<false>;
    if (smem > 48 * 1024) {
      cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
      if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(sample_full_kernel)");
    }
    dim3 grid((k_count + kCand - 1) / kCand, (d + kRows - 1) / kRows);
    kernel<<<grid, kSamplerThreads, smem, stream>>>(mean, step, Bfactor, Dvec, d, key_of(seed), k_begin, k_count, index, ld_out,
                                                    sigma_out, done, step_dev);
    if (blocks_out) *blocks_out = grid.x * grid.y;
  }
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "sampler launch");
}

int32_t launch_stream_words(essa_ctx* ctx, uint64_t seed, int32_t k_begin, int32_t k_count, int32_t n_blocks,
                            uint32_t* words_out, cudaStream_t stream) {
  const long long total = (long long)k_count * n_blocks;
  if (total == 0) return ESSA_OK;
  stream_words_kernel<<<(unsigned)((total + 255) / 256), 256, 0, stream>>>(key_of(seed), k_begin, k_count, n_blocks,
                                                                           words_out);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "stream_words launch");
}

int32_t launch_philox_once(essa_ctx* ctx, const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t* d_out = nullptr;
  cudaError_t e = cudaMalloc(&d_out, 16);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMalloc");
  philox_once_kernel<<<1, 1>>>(make_uint4(ctr[0], ctr[1], ctr[2], ctr[3]), make_uint2(key[0], key[1]), d_out);
  ctx->launches += 1;
  e = cudaMemcpy(out, d_out, 16, cudaMemcpyDeviceToHost);
  cudaFree(d_out);
  return check_cuda(ctx, e, "philox_once");
}

int32_t launch_segment_map(essa_ctx* ctx, const int32_t* seg_offsets, int32_t P, int64_t T, int32_t* cand_out,
                           cudaStream_t stream) {
  if (T == 0) return ESSA_OK;
  segment_map_kernel<<<(unsigned)((T + 255) / 256), 256, 0, stream>>>(seg_offsets, P, (int)T, cand_out);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "segment_map launch");
}

}  // namespace essa
