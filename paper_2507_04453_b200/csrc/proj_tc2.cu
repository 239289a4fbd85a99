// CTA-pair version of the prefill base + up launch (Algorithm 1, line 7, for all candidates at once):
//   y_t = W0 x_t + U_B u_t   on 256-token x 256-channel tiles, one tile per pair of CTAs (cta_group::2).
//
// Each CTA of a pair loads 128 token rows of x (its half of the UMMA M side) and 128 rows of W0 (its half of the
// N side); the leader CTA issues one tcgen05.mma of M = 256, N = 256 per 16-wide K step for both, and each CTA
// finds its 128 token rows of the result in its own TMEM.  Per K block a CTA therefore brings in 32 KB instead of the
// 48 KB of the single-CTA kernel, which buys six pipeline stages instead of four: a TMA tile load takes ~2500
// cycles, a K block 512 cycles of tensor-core time, and four stages cannot cover that.
// The rank-r up-projection is one more K slab (two for INT8 storage), as in the single-CTA kernel; u comes from
// the rank-down launch.
//
// Warp roles per CTA (192 threads): warp 0 = TMA producer, warp 1 = TMEM allocator (+ MMA issuer in the leader),
// warps 2..5 = epilogue.  Barriers: `full` lives in the leader (one arrive.expect_tx for the bytes of both CTAs;
// the peer's copies count on it through its cluster address); `empty` and `tmem_full` exist in both CTAs and are
// signalled by multicast commits; `tmem_empty` lives in the leader and collects the eight epilogue warps of the
// pair.  All waits are bounded; every thread of the pair meets at a cluster barrier before leaving.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int P2_M = 128;        // token rows per CTA (256 per pair)
constexpr int P2_NH = 128;       // W0 rows per CTA (256 channels per pair)
constexpr int P2_N = 256;
constexpr int P2_K = 64;
constexpr int P2_THREADS = 192;
constexpr int P2_A_BYTES = P2_M * P2_K * 2, P2_B_BYTES = P2_NH * P2_K * 2, P2_STAGE = P2_A_BYTES + P2_B_BYTES;  // 32 KB
constexpr int P2_STAGES = 6;
constexpr int P2_SMEM = 1024 + P2_STAGES * P2_STAGE + 1024;
constexpr uint32_t P2_TMEM_COLS = 512;  // two 256-column accumulators

struct P2Params {
  int T, n_out;
  int main_kb, ext_kb, ext_ksteps;
  int m_tiles, n_tiles;  // pair tiles: ceil(T / 256) x ceil(d_out / 256)
  __nv_bfloat16* y;
  int ldy;
  const __half* scale;
  int32_t* status;
};

__global__ void __launch_bounds__(P2_THREADS, 1)
essa_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2a,
                const __grid_constant__ CUtensorMap tmB2b, const P2Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + P2_STAGES * P2_A_BYTES;
  uint8_t* aux = smem + P2_STAGES * P2_STAGE;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], tmem_full[2], tmem_empty[2], drain
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * P2_STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * P2_STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * P2_STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int total_kb = p.main_kb + p.ext_kb;
  const int tiles = p.m_tiles * p.n_tiles;
  // the leader's copies of the barriers the peer signals
  const uint32_t full_leader = map_to_cta(bar_full, 0);
  const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < P2_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 8); }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), P2_TMEM_COLS);  // all 512 columns: the same base address in both CTAs
    tmem_relinquish();
  }
  tc_fence_before();
  cluster_sync_all();  // both CTAs' barriers are initialised before either touches the other's
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (each CTA: its halves)
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int w = pair; ok && w < tiles; w += n_pairs) {
        const int m_tile = w / p.n_tiles, n_tile = w - m_tile * p.n_tiles;
        const int row_a = m_tile * 2 * P2_M + (int)rank * P2_M;     // tokens of this CTA
        const int row_b = n_tile * P2_N + (int)rank * P2_NH;        // channels of this CTA
        for (int kb = 0; kb < total_kb; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          if (leader) mbar_expect_tx(bar_full + 8 * stage, 2u * P2_STAGE);  // the bytes of both CTAs
          const uint32_t fb = full_leader + 8 * stage;
          const uint32_t da = smem_u32(smem_a + stage * P2_A_BYTES), db = smem_u32(smem_b + stage * P2_B_BYTES);
          if (kb < p.main_kb) {
            tma_load_2d_pair(da, &tmA, kb * P2_K, row_a, fb);
            tma_load_2d_pair(db, &tmB, kb * P2_K, row_b, fb);
          } else {
            tma_load_2d_pair(da, &tmA2, 0, row_a, fb);
            tma_load_2d_pair(db, (kb - p.main_kb) == 0 ? &tmB2a : &tmB2b, 0, row_b, fb);
          }
          ++issued;
          if (++stage == P2_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok && issued > 0) {
        // giving up with copies in flight: their completion is counted in the leader, which this CTA may not be,
        // so simply give them time to land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (lane == 0 && leader) {
      constexpr uint32_t idesc = make_idesc(2 * P2_M, P2_N);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int w = pair; ok && w < tiles; w += n_pairs, ++it) {
        const int buf = it & 1;
        const uint32_t use = (uint32_t)(it >> 1);
        if (!mbar_wait(bar_tempty + 8 * buf, (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * P2_N);
        for (int kb = 0; kb < total_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(smem_a + stage * P2_A_BYTES));
          const uint64_t b_desc = make_smem_desc(smem_u32(smem_b + stage * P2_B_BYTES));
          const int nk = (kb < p.main_kb) ? (P2_K / 16) : p.ext_ksteps;
          for (int k = 0; k < nk; ++k) umma_bf16_2cta(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          umma_commit_2cta(bar_empty + 8 * stage, 3);  // the stage is free in both CTAs
          if (++stage == P2_STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit_2cta(bar_tfull + 8 * buf, 3);  // the accumulator is complete in both CTAs
      }
      if (!ok) {
        umma_commit(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (each CTA: its 128 tokens)
    const int quad = warp & 3;
    const int row_in_tile = quad * 32 + lane;
    int it = 0;
    for (int w = pair; w < tiles; w += n_pairs, ++it) {
      const int m_tile = w / p.n_tiles, n_tile = w - m_tile * p.n_tiles;
      const int buf = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      int got = 1;
      if (lane == 0) got = mbar_wait(bar_tfull + 8 * buf, use & 1, abort_flag, p.status) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      while (!mbar_try_wait(bar_tfull + 8 * buf, use & 1)) {}  // complete: acquire for every lane
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * P2_N);
      const int t = m_tile * 2 * P2_M + (int)rank * P2_M + row_in_tile;
      const bool row_ok = t < p.T;
      const int col_base = n_tile * P2_N;
#pragma unroll 1
      for (int c = 0; c < P2_N / 16; ++c) {
        const int col0 = col_base + c * 16;
        if (col0 >= p.n_out) break;
        float v[16];
        tmem_ld16(t_addr + c * 16, v);
        if (row_ok) {
          if (p.scale != nullptr) {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] *= (col0 + i < p.n_out) ? __half2float(__ldg(p.scale + col0 + i)) : 0.f;
          }
          __nv_bfloat16* dst = p.y + (size_t)t * p.ldy + col0;
#pragma unroll
          for (int g = 0; g < 2; ++g) {
            if (col0 + 8 * g < p.n_out) {  // d_out is a multiple of 8: a group of 8 is all in or all out
              uint4 o;
              o.x = pack_bf16x2(v[8 * g + 0], v[8 * g + 1]);
              o.y = pack_bf16x2(v[8 * g + 2], v[8 * g + 3]);
              o.z = pack_bf16x2(v[8 * g + 4], v[8 * g + 5]);
              o.w = pack_bf16x2(v[8 * g + 6], v[8 * g + 7]);
              *reinterpret_cast<uint4*>(dst + 8 * g) = o;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);  // 8 warps of the pair release the accumulator
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();  // no CTA leaves while its partner may still signal it or read its shared memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, P2_TMEM_COLS);
  }
}

}  // namespace

// Pair-tile launch of the base + up step; the caller has checked that the shape suits it.
int32_t launch_base_up_pair(essa_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmA2,
                            const CUtensorMap& tmB2a, const CUtensorMap& tmB2b, int T, int d_out, int main_kb, int ext_kb,
                            int ext_ksteps, __nv_bfloat16* y, const __half* scale, cudaStream_t stream) {
  P2Params p{};
  p.T = T;
  p.n_out = d_out;
  p.main_kb = main_kb;
  p.ext_kb = ext_kb;
  p.ext_ksteps = ext_ksteps;
  p.m_tiles = (T + 2 * P2_M - 1) / (2 * P2_M);
  p.n_tiles = (d_out + P2_N - 1) / P2_N;
  p.y = y;
  p.ldy = d_out;
  p.scale = scale;
  p.status = ctx->d_status;
  const cudaError_t ea = cudaFuncSetAttribute(essa_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, P2_SMEM);
  if (ea != cudaSuccess) return check_cuda(ctx, ea, "cudaFuncSetAttribute(essa_tc2_kernel)");
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  const int pairs = (int)(tiles < sm / 2 ? tiles : sm / 2);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(P2_THREADS, 1, 1);
  cfg.dynamicSmemBytes = P2_SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ctx->launches += 1;
  return check_cuda(ctx, cudaLaunchKernelEx(&cfg, essa_tc2_kernel, tmA, tmB, tmA2, tmB2a, tmB2b, p), "essa_tc2_kernel launch");
}

}  // namespace essa
