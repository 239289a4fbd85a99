// Wide CTA-pair version of the prefill base + up launch (Algorithm 1, line 7, for all candidates at once):
//   y_t = W0 x_t + U_B u_t   on 512-token x 256-channel tiles, one tile per pair of CTAs (cta_group::2), for up to
//   four projections that share the token count (the q, k, v, o of a block) in ONE persistent launch.
//
// Why this shape.  Measured on B200 with operands streamed by TMA exactly as here: a K block (64 wide) of a
// 256 x 256 pair tile -- four MMAs of M = 256, N = 256 into one accumulator, then the commit that frees the stage --
// takes ~670 cycles although the four MMAs need 512; the same loop without any loads takes the same 670, so the
// issue side bounds it, not the data.  Eight MMAs per stage that fill two accumulators in turn (four into the
// first, four into the second, both against the same W0 slab) run at 1030 cycles per stage, i.e. at the tensor
// cores' rate, and bring in 48 KB instead of 64 KB per CTA for the same arithmetic.  So a pair owns TWO 256-token
// accumulators (all 512 TMEM columns of each CTA): per K block each CTA loads two 128-row boxes of x (its halves
// of the two M = 256 operands) and one 128-row box of W0 (its half of the N side), four stages of 48 KB.
// With both accumulators busy the epilogue cannot overlap the next tile's main loop; eight epilogue warps (four per
// accumulator) drain them side by side, and the issuer starts the next tile's first accumulator as soon as that
// one is drained.
//
// The rank-r up-projection is one more K slab (two for INT8 storage: hi and lo of U_B / scale) whose x-side
// operand is u from the rank-down launch.  Work list of a pair: tile w, w + n_pairs, ... of the concatenated tile
// lists of the jobs; inside a job the channel tile runs fastest, so W0 stays in L2 while x streams.
//
// Warp roles per CTA (352 threads): warp 0 = TMA producer for x / u, warp 1 = TMEM allocator (+ MMA issuer in the
// leader), warps 2..5 = epilogue of accumulator 0, warps 6..9 = epilogue of accumulator 1, warp 10 = TMA producer
// for W0 / U_B.  Barriers: `full` lives in the leader (one arrive.expect_tx for the bytes of both CTAs; the
// peer's copies count on it through its cluster address); `empty` and `tmem_full` exist in both CTAs and are
// signalled by multicast commits; `tmem_empty` lives in the leader and collects the eight warps of the pair that
// drain that accumulator.  All waits are bounded; every thread of the pair meets at a cluster barrier before leaving.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int W_BOX = 128 * 64 * 2;   // one 128-row x 64-column bf16 box: 16 KB
constexpr int W_A_BYTES = 2 * W_BOX;  // two x boxes per CTA and stage
constexpr int W_B_BYTES = W_BOX;
constexpr int W_STAGE = W_A_BYTES + W_B_BYTES;  // 48 KB
constexpr int W_STAGES = 4;
constexpr int W_THREADS = 352;
constexpr int W_OUT_BOX = 32 * 64 * 2;  // store staging per epilogue warp: one box of 32 token rows x 64 channels (4 KB, 128-byte swizzle)
constexpr int W_SMEM = 1024 + W_STAGES * W_STAGE + 8 * W_OUT_BOX + 1024;
constexpr uint32_t W_TMEM_COLS = 512;  // two 256-column accumulators
constexpr int W_TILE_M = 512, W_TILE_N = 256;

struct WMaps {
  // per job: x, W0, u, U_B slab 0, U_B slab 1 (boxes of 128 rows x 64 columns), y (store boxes of 32 rows x 64 columns)
  CUtensorMap m[kWideMaxJobs][6];
};

struct WJobDev {
  int n_out, main_kb, ext_kb, ext_ksteps, n_tiles, tile_begin;
  int keep_tiles;  // channel tiles (from 0) whose W0 rows are loaded with the evict-last L2 policy
  const __half* scale;
};

struct WParams {
  int T, m_tiles, n_jobs, tiles;
  int l2_hints;  // bit 0: W0 / U_B loads evict-last, bit 1: x / u loads evict-first, bit 2: y stores evict-first, bit 3: K walks back on odd tiles
  WJobDev job[kWideMaxJobs];
  int32_t* status;
};

__global__ void __launch_bounds__(W_THREADS, 1) essa_tcw_kernel(const __grid_constant__ WMaps maps, const WParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* stg_all = smem + W_STAGES * W_STAGE;  // 8 x 4 KB, 1024-byte aligned
  uint8_t* aux = stg_all + 8 * W_OUT_BOX;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], tmem_full[2], tmem_empty[2], drain
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * W_STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * W_STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * W_STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const uint32_t full_leader = map_to_cta(bar_full, 0);
  const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);

  // tile w of the concatenated lists -> (job, token tile, channel tile)
  auto tile_of = [&](int w, int& j, int& m_tile, int& n_tile) {
    j = 0;
    while (j + 1 < p.n_jobs && w >= p.job[j + 1].tile_begin) ++j;
    const int w2 = w - p.job[j].tile_begin;
    m_tile = w2 / p.job[j].n_tiles;
    n_tile = w2 - m_tile * p.job[j].n_tiles;
  };

  if (threadIdx.x == 0) {
    for (int j = 0; j < p.n_jobs; ++j) {
      tma_prefetch_desc(&maps.m[j][0]);
      tma_prefetch_desc(&maps.m[j][1]);
    }
    for (int s = 0; s < W_STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 8); }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), W_TMEM_COLS);  // all 512 columns: the same base address in both CTAs
    tmem_relinquish();
  }
  tc_fence_before();
  cluster_sync_all();  // both CTAs' barriers are initialised before either touches the other's
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == 10) {
    // ------------------------------------------------------------------ TMA producers (each CTA: its halves)
    const bool prod_a = warp == 0;
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      // W0 is read again by every later round of the grid and should stay in L2 while x and y stream past it
      const uint64_t pol_w = l2_policy_evict_last(), pol_x = l2_policy_evict_first();
      const bool hint_w = (p.l2_hints & 1) != 0, hint_x = (p.l2_hints & 2) != 0;
      int it = 0;
      for (int w = pair; ok && w < p.tiles; w += n_pairs, ++it) {
        int j, m_tile, n_tile;
        tile_of(w, j, m_tile, n_tile);
        const WJobDev& jb = p.job[j];
        const int total_kb = jb.main_kb + jb.ext_kb;
        // Every other tile of a pair walks K backwards.  All pairs run in step, so a round of the grid streams the
        // same K slabs of W0 (and of the token tiles it shares with the round before) in the same order; the rounds'
        // footprint (config 4: 91 MB) exceeds what L2 keeps, and with every round walking K forwards a slab is always
        // gone when its turn comes again.  Walking back, a round starts with the slabs the round before used last.
        const bool k_back = (p.l2_hints & 8) != 0 && (it & 1) != 0;
        const int row_a = m_tile * W_TILE_M + (int)rank * 128;  // + 256 for the second accumulator's box
        const int row_b = n_tile * W_TILE_N + (int)rank * 128;  // channels of this CTA
        for (int kb = 0; kb < total_kb; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          if (leader && prod_a) mbar_expect_tx(bar_full + 8 * stage, 2u * W_STAGE);  // the bytes of both CTAs
          const uint32_t fb = full_leader + 8 * stage;
          const uint32_t da = smem_u32(smem + stage * W_STAGE), db = da + W_A_BYTES;
          if (prod_a) {
            const CUtensorMap* tm = kb < jb.main_kb ? &maps.m[j][0] : &maps.m[j][2];
            const int col = kb < jb.main_kb ? (k_back ? jb.main_kb - 1 - kb : kb) * 64 : 0;
            if (hint_x) {
              tma_load_2d_pair_hint(da, tm, col, row_a, fb, pol_x);
              tma_load_2d_pair_hint(da + W_BOX, tm, col, row_a + 256, fb, pol_x);
            } else {
              tma_load_2d_pair(da, tm, col, row_a, fb);
              tma_load_2d_pair(da + W_BOX, tm, col, row_a + 256, fb);
            }
          } else {
            const CUtensorMap* tm = kb < jb.main_kb ? &maps.m[j][1] : (kb == jb.main_kb ? &maps.m[j][3] : &maps.m[j][4]);
            const int col = kb < jb.main_kb ? (k_back ? jb.main_kb - 1 - kb : kb) * 64 : 0;
            if (hint_w && n_tile < jb.keep_tiles) tma_load_2d_pair_hint(db, tm, col, row_b, fb, pol_w);
            else tma_load_2d_pair(db, tm, col, row_b, fb);
          }
          ++issued;
          if (++stage == W_STAGES) { stage = 0; phase ^= 1; }
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
      constexpr uint32_t idesc = make_idesc(256, W_TILE_N);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int w = pair; ok && w < p.tiles; w += n_pairs, ++it) {
        int j, m_tile, n_tile;
        tile_of(w, j, m_tile, n_tile);
        const WJobDev& jb = p.job[j];
        const int total_kb = jb.main_kb + jb.ext_kb;
        for (int kb = 0; ok && kb < total_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * W_STAGE);
          const uint64_t b_desc = make_smem_desc(sa + W_A_BYTES);
          const uint64_t a_desc0 = make_smem_desc(sa), a_desc1 = make_smem_desc(sa + W_BOX);
          const uint32_t d0 = tmem_base, d1 = tmem_base + (uint32_t)W_TILE_N;
          if (kb > 0 && kb < jb.main_kb) {
            // the hot path, straight-line: four MMAs into the first accumulator, four into the second, one W0 slab
            // (the issuing thread's own instructions between two MMAs count: with a loop and a predicate per MMA
            // this K block measured 1435 cycles instead of 1030)
            umma_bf16_2cta(d0, a_desc0, b_desc, idesc, 1u);
            umma_bf16_2cta(d0, a_desc0 + 2, b_desc + 2, idesc, 1u);
            umma_bf16_2cta(d0, a_desc0 + 4, b_desc + 4, idesc, 1u);
            umma_bf16_2cta(d0, a_desc0 + 6, b_desc + 6, idesc, 1u);
            umma_bf16_2cta(d1, a_desc1, b_desc, idesc, 1u);
            umma_bf16_2cta(d1, a_desc1 + 2, b_desc + 2, idesc, 1u);
            umma_bf16_2cta(d1, a_desc1 + 4, b_desc + 4, idesc, 1u);
            umma_bf16_2cta(d1, a_desc1 + 6, b_desc + 6, idesc, 1u);
          } else {
            // first K block of a tile (waits for the accumulators, starts them) and the rank slabs (end them)
            const int nk = (kb < jb.main_kb) ? 4 : jb.ext_ksteps;
#pragma unroll 1
            for (int b = 0; b < 2; ++b) {
              if (kb == 0) {
                // the epilogue warps of the previous tile must have drained this accumulator
                if (!mbar_wait(bar_tempty + 8 * b, (uint32_t)((it & 1) ^ 1), abort_flag, p.status)) { ok = false; break; }
                tc_fence_after();
              }
              const uint64_t a_desc = b == 0 ? a_desc0 : a_desc1;
              const uint32_t d_tmem = b == 0 ? d0 : d1;
              for (int k = 0; k < nk; ++k) umma_bf16_2cta(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
              if (kb == total_kb - 1) umma_commit_2cta(bar_tfull + 8 * b, 3);  // this accumulator is complete in both CTAs
            }
          }
          if (!ok) break;
          umma_commit_2cta(bar_empty + 8 * stage, 3);  // the stage is free in both CTAs
          if (++stage == W_STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        umma_commit(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (each CTA: its 2 x 128 tokens)
    const int acc = (warp - 2) >> 2;  // which accumulator this warp drains
    const int quad = warp & 3;        // the TMEM lanes this warp may read
    const uint32_t stg = smem_u32(stg_all + (warp - 2) * W_OUT_BOX);
    const uint64_t pol_y = l2_policy_evict_first();
    int it = 0;
    for (int w = pair; w < p.tiles; w += n_pairs, ++it) {
      int j, m_tile, n_tile;
      tile_of(w, j, m_tile, n_tile);
      const WJobDev& jb = p.job[j];
      int got = 1;
      if (lane == 0) got = mbar_wait(bar_tfull + 8 * acc, (uint32_t)(it & 1), abort_flag, p.status) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      while (!mbar_try_wait(bar_tfull + 8 * acc, (uint32_t)(it & 1))) {}  // complete: acquire for every lane
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(acc * W_TILE_N);
      const int row0 = m_tile * W_TILE_M + acc * 256 + (int)rank * 128 + quad * 32;  // first token row of this warp
      const int col_base = n_tile * W_TILE_N;
      // 32 channels at a time: TMEM -> registers (scale, round to bf16) -> this warp's staging box in shared memory
      // (128-byte-swizzled rows of 64 channels); every second chunk completes the box -> one TMA store, which clips
      // rows >= T and channels >= n_out.  (Storing straight from the row-per-thread registers made every 16-byte store
      // instruction touch 32 different lines and took 16 k cycles per tile.)  The next chunk's TMEM load is in flight
      // while a chunk is packed and staged; a box is refilled once the store before has read it.
      uint32_t ra[32], rb[32];
      tmem_ld32_issue(t_addr, ra);
      auto chunk = [&](int c, const uint32_t (&r)[32]) {
        const int col0 = col_base + c * 32;
        uint32_t pk[16];
        if (jb.scale != nullptr) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            const float s0 = (col0 + 2 * i < jb.n_out) ? __half2float(__ldg(jb.scale + col0 + 2 * i)) : 0.f;
            const float s1 = (col0 + 2 * i + 1 < jb.n_out) ? __half2float(__ldg(jb.scale + col0 + 2 * i + 1)) : 0.f;
            pk[i] = pack_bf16x2(__uint_as_float(r[2 * i]) * s0, __uint_as_float(r[2 * i + 1]) * s1);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1]));
        }
        const int half = c & 1;
        if (half == 0) {
          if (lane == 0) bulk_wait_group_read0();  // the store before has read the box
          __syncwarp();
        }
#pragma unroll
        for (int j4 = 0; j4 < 4; ++j4)
          sts_v4(stg + (uint32_t)(lane * 128 + (((half * 4 + j4) ^ (lane & 7)) << 4)), make_uint4(pk[4 * j4], pk[4 * j4 + 1], pk[4 * j4 + 2], pk[4 * j4 + 3]));
        if (half == 1) {
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0 && row0 < p.T && col0 - 32 < jb.n_out) {
            if (p.l2_hints & 4) tma_store_2d_hint(&maps.m[j][5], stg, col0 - 32, row0, pol_y);
            else tma_store_2d(&maps.m[j][5], stg, col0 - 32, row0);
            bulk_commit_group();
          }
        }
      };
#pragma unroll 1
      for (int c = 0; c < W_TILE_N / 32; c += 2) {
        tmem_ld_wait();
        tmem_ld32_issue(t_addr + (c + 1) * 32, rb);
        chunk(c, ra);
        tmem_ld_wait();
        if (c + 2 < W_TILE_N / 32) {
          tmem_ld32_issue(t_addr + (c + 2) * 32, ra);
        } else {
          // every TMEM read of this tile is done: the issuer may start the next tile in this accumulator
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * acc);  // 8 warps of the pair release the accumulator
        }
        chunk(c + 1, rb);
      }
    }
    if (lane == 0) bulk_wait_group0();  // the last stores have left shared memory and are written
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();  // no CTA leaves while its partner may still signal it or read its shared memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, W_TMEM_COLS);
  }
}

}  // namespace

// Estimated cycles of a projection's base + up step on 256-token pair tiles and on these 512-token ones (measured
// K-block costs; whole rounds of the persistent grid), used to pick the tile shape.
bool wide_tiles_pay(int64_t T, int d_out, int total_kb, int sm_count) {
  const int pairs = (sm_count > 0 ? sm_count : 148) / 2;
  const long long n_tiles = (d_out + 255) / 256;
  const long long t2 = ((T + 255) / 256) * n_tiles, tw = ((T + 511) / 512) * n_tiles;
  const double c2 = (double)((t2 + pairs - 1) / pairs) * (total_kb * 880.0 + 1500.0);
  const double cw = (double)((tw + pairs - 1) / pairs) * (total_kb * 1040.0 + 6000.0);
  return cw < c2;
}

// One launch for the base + up step of n_jobs projections that share T.
int32_t launch_base_up_wide(essa_ctx* ctx, const WideJob* jobs, int n_jobs, int T, cudaStream_t stream) {
  if (n_jobs < 1 || n_jobs > kWideMaxJobs) return fail(ctx, ESSA_ERR_INVALID_ARG, "launch_base_up_wide: bad job count");
  WMaps maps;
  WParams p{};
  p.T = T;
  p.m_tiles = (T + W_TILE_M - 1) / W_TILE_M;
  p.n_jobs = n_jobs;
  p.status = ctx->d_status;
  p.l2_hints = ctx->l2_hints & 15;
  long long tiles = 0;
  for (int j = 0; j < n_jobs; ++j) {
    const WideJob& s = jobs[j];
    WJobDev& d = p.job[j];
    d.n_out = s.d_out;
    d.main_kb = s.main_kb;
    d.ext_kb = s.ext_kb;
    d.ext_ksteps = s.ext_ksteps;
    d.n_tiles = (s.d_out + W_TILE_N - 1) / W_TILE_N;
    d.tile_begin = (int)tiles;
    // Evict-last protects about 21 MB of L2 on this part: config 4's q projection (W0 = 52 MB, re-read from HBM by
    // every round of the grid) read 1324 MB without hints, 1170 / 1057 / 1196 / 1316 MB with the first 4 / 8 / 12 / 16
    // channel tiles (10 / 21 / 31 / 42 MB) marked, 1320 MB with all 20.  So mark as many leading tiles as fit 21 MB.
    const int forced = ctx->l2_hints >> 8;
    const long long tile_bytes = 256LL * s.main_kb * 64 * 2;
    d.keep_tiles = forced > 0 ? forced : (int)(tile_bytes > 0 ? (21LL << 20) / tile_bytes : 0);
    if (d.keep_tiles < 1) d.keep_tiles = 1;
    d.scale = s.scale;
    tiles += (long long)p.m_tiles * d.n_tiles;
    if (tiles > 0x7fffffffLL) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "launch_base_up_wide: too many tiles");
    maps.m[j][0] = *s.tmA;
    maps.m[j][1] = *s.tmB;
    maps.m[j][2] = *s.tmA2;
    maps.m[j][3] = *s.tmB2a;
    maps.m[j][4] = *s.tmB2b;
    const int32_t ms = make_tensor_map_2d(ctx, &maps.m[j][5], 0, s.y, (uint64_t)T, (uint64_t)s.d_out, (uint64_t)s.d_out * 2, 32, 64, 128);
    if (ms != ESSA_OK) return ms;
  }
  for (int j = n_jobs; j < kWideMaxJobs; ++j)
    for (int i = 0; i < 6; ++i) maps.m[j][i] = maps.m[0][i];
  p.tiles = (int)tiles;
  static bool attr_done[64] = {};  // the attribute is per device
  bool& done = attr_done[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0];
  if (!done) {
    const cudaError_t ea = cudaFuncSetAttribute(essa_tcw_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, W_SMEM);
    if (ea != cudaSuccess) return check_cuda(ctx, ea, "cudaFuncSetAttribute(essa_tcw_kernel)");
    done = true;
  }
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const int pairs = (int)(tiles < sm / 2 ? tiles : sm / 2);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(W_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)W_SMEM;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ctx->launches += 1;
  void* args[] = {(void*)&maps, (void*)&p};
  return check_cuda(ctx, cudaLaunchKernelExC(&cfg, (const void*)essa_tcw_kernel, args), "essa_tcw_kernel launch");
}

}  // namespace essa
