// Rank-down launch of prefill-sized calls on CTA pairs (Algorithm 1, candidate reconstruction folded into the forward):
//   u_t = sB_k .* (M (sA_k .* (V_A^T x_t))),  k = cand(t),  for every token of up to four projections (same T) in ONE launch.
//
// The launch reads x once and is bound by HBM, so what matters is that every SM streams the same number of bytes and
// that neither the tensor core nor the threads that issue the copies hold the stream back.  (a) Balance: the token rows
// of all jobs form one list of 64-row units; pair p of the persistent grid owns units [p U / n_pairs, (p + 1) U / n_pairs)
// and walks them in tiles of up to eight units (512 rows: two halves of M = 256 across the pair, each CTA holding up to
// two units of either half) where it has at least twelve units, of up to four otherwise (one half; the ring is then
// twice as deep); boxes beyond a pair's range are not loaded.  The 128-row tiles of the single-CTA kernel
// left the grid's last round a quarter idle (257 tiles on 148 SMs).  (b) Tensor time: one tcgen05.mma.cta_group::2
// covers 256 token rows, half the MMAs per byte of x of the M = 128 kernel, whose narrow MMAs (N = r_pad) cost ~150
// cycles each whatever N is; and a K block's eight MMAs fill the two halves' accumulators in turn before one commit,
// which the tensor core takes at twice the rate of four MMAs into one accumulator + commit (rank-down launch of four
// 3584-wide inputs at 16384 tokens: 102 -> 96 us; of four 5120-wide ones at 35462 tokens: 302 -> 270 us; with fewer
// than twelve units per pair the 256-row tiles measured faster: 63 against 73 us at 8192 tokens).
// (c) Several threads issue the copies, the K blocks in turn.
//
// Per K block (64 wide) a CTA loads its units of x (per half one 128-row box, or one 64-row box at the end of its
// range) and its half of the V_A^T tile (r_pad / 2 rows); the leader issues per half four MMAs of M = 256, N = r_pad
// into that half's accumulator of one of two buffers, so the epilogue of a tile (per token row in registers: sA, the
// r x r core M, sB; u stored as bf16) overlaps the next tile's K loop.
//
// Warp roles per CTA (320 threads): warps 0 and 6..9 = TMA producers, warp 1 = TMEM allocator (+ MMA issuer in the
// leader), warps 2..5 = epilogue.  Barriers as in the other pair kernels: `full` in the leader (bytes of both CTAs),
// `empty` / `tmem_full` in both CTAs by multicast commits, `tmem_empty` in the leader collecting the pair's eight
// epilogue warps.  All waits are bounded; every thread meets at a cluster barrier before leaving.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int D_UNIT_ROWS = 64;
constexpr int D_UNIT_BYTES = D_UNIT_ROWS * 64 * 2;  // 8 KB: 64 rows x 64 bf16
constexpr int D_HALF_BYTES = 2 * D_UNIT_BYTES;      // a CTA's two units of one half of the tile (one 128-row operand)
constexpr int D_A_BYTES = 2 * D_HALF_BYTES;         // both halves
constexpr int D_THREADS = 320;
constexpr int D_PRODUCERS = 5;
constexpr uint32_t D_TMEM_COLS = 256;  // two buffers x two halves, accumulators of up to 64 columns
__host__ __device__ constexpr int d_v_bytes(int rp) { return rp * 64; }  // rp / 2 rows x 128 B
// ring depth for stages that hold one half (tiles of up to four units) or both; the shared memory is the same either way
constexpr int D_MAX_STAGES = 12;
__host__ __device__ constexpr int d_stages(int rp, int a_bytes) {
  return (227 * 1024 - 2048) / (a_bytes + d_v_bytes(rp)) > D_MAX_STAGES ? D_MAX_STAGES : (227 * 1024 - 2048) / (a_bytes + d_v_bytes(rp));
}
constexpr int d_smem() { return 227 * 1024; }

struct DnMaps {
  CUtensorMap x[kWideMaxJobs];   // boxes of 64 rows x 64 columns
  CUtensorMap x2[kWideMaxJobs];  // boxes of 128 rows x 64 columns (a CTA's two units in one copy)
  CUtensorMap v[kWideMaxJobs];   // V_A^T, boxes of r_pad / 2 rows x 64 columns
};

struct DnJob {
  int main_kb, r, sA_col, sB_col;
  const float* M;      // [64][64] fp32
  __nv_bfloat16* u;    // [T][64]
};

struct DnParams {
  int T, units_per_job, n_jobs, n_producers, max_units;
  long long total_units;
  DnJob job[kWideMaxJobs];
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma;
  int32_t* status;
};

template <int RP>
__global__ void __launch_bounds__(D_THREADS, 1) essa_down_kernel(const __grid_constant__ DnMaps maps, const DnParams p) {
  constexpr int V_BYTES = d_v_bytes(RP);
  const int A_BYTES = p.max_units > 4 ? D_A_BYTES : D_HALF_BYTES;  // a stage's x part: both halves of a tile, or one
  const int STAGES = d_stages(RP, A_BYTES);
  const int STAGE = A_BYTES + V_BYTES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* aux = smem + STAGES * STAGE;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], tmem_full[2], tmem_empty[2], drain
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const uint32_t full_leader = map_to_cta(bar_full, 0);
  const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);

  // this pair's units of the global list, walked in tiles: (job, first row, units in the tile <= 4)
  const long long u_begin = p.total_units * pair / n_pairs, u_end = p.total_units * (pair + 1) / n_pairs;
  auto tile_at = [&](long long g, int& j, int& row0, int& n_units) {
    j = (int)(g / p.units_per_job);
    const int ju = (int)(g - (long long)j * p.units_per_job);
    long long n = u_end - g;
    if (n > p.max_units) n = p.max_units;
    if (n > p.units_per_job - ju) n = p.units_per_job - ju;
    n_units = (int)n;
    row0 = ju * D_UNIT_ROWS;
  };

  if (threadIdx.x == 0) {
    for (int j = 0; j < p.n_jobs; ++j) {
      tma_prefetch_desc(&maps.x2[j]);
      tma_prefetch_desc(&maps.v[j]);
    }
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 8); }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), D_TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  cluster_sync_all();  // both CTAs' barriers are initialised before either touches the other's
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp >= 6) {
    // ------------------------------------------------------------------ TMA producers (each CTA: its units, its half of V_A^T)
    // The producer threads take the K blocks in turn (thread i: blocks i, i + n, ...): issuing a copy occupies its
    // thread for a few hundred cycles.
    const int pi = warp == 0 ? 0 : warp - 5;  // 0 .. 4
    if (lane == 0 && pi < p.n_producers) {
      long long seq = 0;  // K blocks of this pair so far
      int issued = 0;
      bool ok = true;
      for (long long g = u_begin; ok && g < u_end;) {
        int j, row0, n_units;
        tile_at(g, j, row0, n_units);
        g += n_units;
        const int main_kb = p.job[j].main_kb;
        // units of this CTA: tile units 2 rank, 2 rank + 1 (first half of the tile) and 4 + 2 rank, 5 + 2 rank (second half)
        const int mine0 = n_units - 2 * (int)rank, mine1 = n_units - 4 - 2 * (int)rank;
        const int row_mine = row0 + 2 * (int)rank * D_UNIT_ROWS;
        for (int kb = 0; kb < main_kb; ++kb, ++seq) {
          if ((int)(seq % p.n_producers) != pi) continue;
          const int stage = (int)(seq % STAGES);
          const uint32_t phase = (uint32_t)((seq / STAGES) & 1);
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          if (leader) mbar_expect_tx(bar_full + 8 * stage, (uint32_t)(n_units * D_UNIT_BYTES + 2 * V_BYTES));
          const uint32_t fb = full_leader + 8 * stage;
          const uint32_t da = smem_u32(smem + stage * STAGE);
          if (mine0 > 1) tma_load_2d_pair(da, &maps.x2[j], kb * 64, row_mine, fb);
          else if (mine0 > 0) tma_load_2d_pair(da, &maps.x[j], kb * 64, row_mine, fb);
          if (mine1 > 1) tma_load_2d_pair(da + D_HALF_BYTES, &maps.x2[j], kb * 64, row_mine + 4 * D_UNIT_ROWS, fb);
          else if (mine1 > 0) tma_load_2d_pair(da + D_HALF_BYTES, &maps.x[j], kb * 64, row_mine + 4 * D_UNIT_ROWS, fb);
          tma_load_2d_pair(da + A_BYTES, &maps.v[j], kb * 64, (int)rank * (RP / 2), fb);
          ++issued;
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
      constexpr uint32_t idesc = make_idesc(256, RP);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (long long g = u_begin; ok && g < u_end; ++it) {
        int j, row0, n_units;
        tile_at(g, j, row0, n_units);
        g += n_units;
        const int main_kb = p.job[j].main_kb;
        const int buf = it & 1;
        if (!mbar_wait(bar_tempty + 8 * buf, (uint32_t)(((it >> 1) & 1) ^ 1), abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d0 = tmem_base + (uint32_t)(buf * 128), d1 = d0 + 64u;  // the tile's two halves
        const bool two = n_units > 4;
        for (int kb = 0; kb < main_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + stage * STAGE);
          // a CTA's two units of a half are consecutive 64-row boxes: one 128-row K-major operand per half
          const uint64_t a0 = make_smem_desc(sa), a1 = make_smem_desc(sa + D_HALF_BYTES), v_desc = make_smem_desc(sa + A_BYTES);
          const uint32_t acc = kb > 0 ? 1u : 0u;
          // straight-line (the issuing thread's own instructions between two MMAs count); four MMAs into the first half's
          // accumulator, then four into the second's: filling two accumulators in turn before the commit runs at the
          // tensor cores' rate, four MMAs into one accumulator + commit do not (~840 cycles instead of 512)
          umma_bf16_2cta(d0, a0, v_desc, idesc, acc);
          umma_bf16_2cta(d0, a0 + 2, v_desc + 2, idesc, 1u);
          umma_bf16_2cta(d0, a0 + 4, v_desc + 4, idesc, 1u);
          umma_bf16_2cta(d0, a0 + 6, v_desc + 6, idesc, 1u);
          if (two) {
            umma_bf16_2cta(d1, a1, v_desc, idesc, acc);
            umma_bf16_2cta(d1, a1 + 2, v_desc + 2, idesc, 1u);
            umma_bf16_2cta(d1, a1 + 4, v_desc + 4, idesc, 1u);
            umma_bf16_2cta(d1, a1 + 6, v_desc + 6, idesc, 1u);
          }
          umma_commit_2cta(bar_empty + 8 * stage, 3);  // the stage is free in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
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
    // ------------------------------------------------------------------ epilogue warps (each CTA: its 128 token rows)
    const int quad = warp & 3;
    const int row_in_cta = quad * 32 + lane;  // 0 .. 127: unit row_in_cta / 64 of this CTA
    int it = 0;
    for (long long g = u_begin; g < u_end; ++it) {
      int j, row0, n_units;
      tile_at(g, j, row0, n_units);
      g += n_units;
      const DnJob& jb = p.job[j];
      const int buf = it & 1;
      int got = 1;
      if (lane == 0) got = mbar_wait(bar_tfull + 8 * buf, (uint32_t)((it >> 1) & 1), abort_flag, p.status) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (!got) break;
      while (!mbar_try_wait(bar_tfull + 8 * buf, (uint32_t)((it >> 1) & 1))) {}  // complete: acquire for every lane
      tc_fence_after();
      const int halves = n_units > 4 ? 2 : 1;
#pragma unroll 1
      for (int hf = 0; hf < halves; ++hf) {
        const uint32_t p_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * 128 + hf * 64);
        float q[RP];
#pragma unroll
        for (int c = 0; c < RP / 16; ++c) {
          float v[16];
          tmem_ld16(p_addr + c * 16, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) q[c * 16 + i] = v[i];
        }
        if (hf == halves - 1) {
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(tempty_leader + 8 * buf);  // the buffer may take the tile after next
        }
        const int unit_in_tile = 4 * hf + 2 * (int)rank + row_in_cta / D_UNIT_ROWS;
        const int t = row0 + hf * 256 + (int)rank * 128 + row_in_cta;
        if (unit_in_tile < n_units && t < p.T) {
          const int k = find_candidate(p.seg, p.P, t);
          const float* srow = p.sigma + (size_t)k * p.ld_sigma;
#pragma unroll
          for (int i = 0; i < RP; ++i) q[i] = (i < jb.r) ? q[i] * __ldg(srow + jb.sA_col + i) : 0.f;
          uint32_t packed[kRankPadMax / 2];
#pragma unroll
          for (int j2 = 0; j2 < RP / 2; ++j2) {
            float uu[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int jj = 2 * j2 + h;
              float acc = 0.f;
#pragma unroll
              for (int i4 = 0; i4 < RP / 4; ++i4) {
                const float4 mm = __ldg(reinterpret_cast<const float4*>(jb.M + jj * kRankPadMax) + i4);  // same address in every lane
                acc = fmaf(mm.x, q[4 * i4], acc);
                acc = fmaf(mm.y, q[4 * i4 + 1], acc);
                acc = fmaf(mm.z, q[4 * i4 + 2], acc);
                acc = fmaf(mm.w, q[4 * i4 + 3], acc);
              }
              uu[h] = (jj < jb.r) ? acc * __ldg(srow + jb.sB_col + jj) : 0.f;
            }
            packed[j2] = pack_bf16x2(uu[0], uu[1]);
          }
#pragma unroll
          for (int j2 = RP / 2; j2 < kRankPadMax / 2; ++j2) packed[j2] = 0u;
          uint4* dst = reinterpret_cast<uint4*>(jb.u + (size_t)t * kRankPadMax);
#pragma unroll
          for (int gq = 0; gq < kRankPadMax / 8; ++gq)
            dst[gq] = make_uint4(packed[4 * gq], packed[4 * gq + 1], packed[4 * gq + 2], packed[4 * gq + 3]);
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncwarp();
  cluster_sync_all();  // no CTA leaves while its partner may still signal it or read its shared memory
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, D_TMEM_COLS);
  }
}

template <int RP>
int32_t launch_down(essa_ctx* ctx, const DnMaps& maps, const DnParams& p, int pairs, cudaStream_t stream) {
  static bool attr_done[64] = {};  // the attribute is per device
  bool& done = attr_done[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0];
  if (!done) {
    const cudaError_t ea = cudaFuncSetAttribute(essa_down_kernel<RP>, cudaFuncAttributeMaxDynamicSharedMemorySize, d_smem());
    if (ea != cudaSuccess) return check_cuda(ctx, ea, "cudaFuncSetAttribute(essa_down_kernel)");
    done = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(D_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)d_smem();
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
  return check_cuda(ctx, cudaLaunchKernelExC(&cfg, (const void*)essa_down_kernel<RP>, args), "essa_down_kernel launch");
}

}  // namespace

// Whether the pair kernel takes a rank-down step of n_jobs projections over T tokens: every pair of the grid should get
// at least a few units, and all jobs must share the padded rank (one kernel instance per launch).
bool down_pairs_suit(const essa_ctx* ctx, const DownJob* jobs, int n_jobs, int64_t T) {
  if (ctx->down_pairs <= 0 || n_jobs < 1 || n_jobs > kWideMaxJobs || T < 512) return false;
  // (measured: config 2, r = 16, four projections: 125 -> 102 us; config 4, r = 32: 319 -> 259 us; config 5b, r = 64, one
  // projection: 186 -> 205 us, so ranks padded beyond 32 stay on the single-CTA kernel)
  if (jobs[0].a->r_pad > 32) return false;
  for (int j = 1; j < n_jobs; ++j)
    if (jobs[j].a->r_pad != jobs[0].a->r_pad) return false;
  const int pairs = (ctx->sm_count > 0 ? ctx->sm_count : 148) / 2;
  const long long units = (long long)n_jobs * ((T + D_UNIT_ROWS - 1) / D_UNIT_ROWS);
  return units >= 4LL * pairs;
}

int32_t launch_rank_down_pairs(essa_ctx* ctx, const DownJob* jobs, int n_jobs, int64_t T, const int32_t* seg, int32_t P,
                               const float* sigma, int32_t ld_sigma, cudaStream_t stream) {
  DnMaps maps;
  DnParams p{};
  p.T = (int)T;
  p.units_per_job = (int)((T + D_UNIT_ROWS - 1) / D_UNIT_ROWS);
  p.n_jobs = n_jobs;
  p.n_producers = ctx->down_pairs > D_PRODUCERS ? D_PRODUCERS : ctx->down_pairs;
  p.total_units = (long long)n_jobs * p.units_per_job;
  {
    const int pairs_dev = (ctx->sm_count > 0 ? ctx->sm_count : 148) / 2;
    p.max_units = ctx->down_tile_units > 0 ? ctx->down_tile_units : (p.total_units >= 12LL * pairs_dev ? 8 : 4);
  }
  p.seg = seg;
  p.P = P;
  p.sigma = sigma;
  p.ld_sigma = ld_sigma;
  p.status = ctx->d_status;
  for (int j = 0; j < n_jobs; ++j) {
    const essa_adapter* a = jobs[j].a;
    p.job[j].main_kb = a->d_in / 64;
    p.job[j].r = a->rank;
    p.job[j].sA_col = jobs[j].sA_col;
    p.job[j].sB_col = jobs[j].sB_col;
    p.job[j].M = a->M;
    p.job[j].u = jobs[j].u;
    int32_t st = make_tensor_map_2d(ctx, &maps.x[j], 0, jobs[j].x, (uint64_t)T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                                    D_UNIT_ROWS, 64, 128);
    if (st != ESSA_OK) return st;
    st = make_tensor_map_2d(ctx, &maps.x2[j], 0, jobs[j].x, (uint64_t)T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                            2 * D_UNIT_ROWS, 64, 128);
    if (st != ESSA_OK) return st;
    maps.v[j] = a->tm_VAtH;
  }
  for (int j = n_jobs; j < kWideMaxJobs; ++j) {
    maps.x[j] = maps.x[0];
    maps.x2[j] = maps.x2[0];
    maps.v[j] = maps.v[0];
  }
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const int pairs = sm / 2;
  switch (jobs[0].a->r_pad) {
    case 16: return launch_down<16>(ctx, maps, p, pairs, stream);
    case 32: return launch_down<32>(ctx, maps, p, pairs, stream);
    case 48: return launch_down<48>(ctx, maps, p, pairs, stream);
    case 64: return launch_down<64>(ctx, maps, p, pairs, stream);
    default: return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "rank-down: bad padded rank");
  }
}

}  // namespace essa
