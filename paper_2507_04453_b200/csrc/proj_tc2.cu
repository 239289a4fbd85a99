// CTA-pair version of the prefill base + up launch (Algorithm 1, line 7, for all candidates at once):
//   y_t = W0 x_t + U_B u_t   on 256-token x 256-channel tiles, one tile per pair of CTAs (cta_group::2).
//
// Each CTA of a pair loads 128 token rows of x (its half of the UMMA M side) and 128 rows of W0 (its half of the
// N side); the leader CTA issues one tcgen05.mma of M = 256, N = 256 per 16-wide K step for both, and each CTA
// finds its 128 token rows of the result in its own TMEM.  Per K block a CTA therefore brings in 32 KB instead of the
// 48 KB of the single-CTA kernel, which buys six pipeline stages instead of four: a TMA tile load takes ~2500
// cycles, a K block 512 cycles of tensor-core time, and four stages cannot cover that.
// The rank-r up-projection is one more K slab (two for INT8 storage), as in the single-CTA kernel.  u comes from
// the rank-down launch (RP = 0) or, fused (RP = padded rank), from this kernel itself: the tiles of channel
// column 0 come first in every pair's work list, and while a pair runs the K loop of such a tile it also
// accumulates  P = x V_A  for its 256 tokens (one more MMA of N = RP per K step against an RP/2-row tile of V_A^T
// per CTA, into the accumulator buffer the tile does not use).  The epilogue warps then form
// u = sB_k .* (M (sA_k .* p)) for their token rows, store it (bf16) and release-increment a per-(token tile, CTA
// rank) counter; every producer thread acquires that counter (bounded) before it loads a tile's u slab.  Tiles of
// the first column wait only for themselves, all other tiles only for first-column tiles, which precede them in
// every pair's list, so the waits end.  This removes the separate rank-down launch.
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
constexpr int P2_THREADS = 224;  // warps 0..5 as below, warp 6 = second TMA producer (the W0 / U_B halves)
constexpr int P2_A_BYTES = P2_M * P2_K * 2, P2_B_BYTES = P2_NH * P2_K * 2, P2_STAGE = P2_A_BYTES + P2_B_BYTES;  // 32 KB
constexpr int P2_STAGES = 6;
__host__ __device__ constexpr int p2_stages(int rp) { return rp > 48 ? 5 : P2_STAGES; }
__host__ __device__ constexpr int p2_v_bytes(int rp) { return rp * 64; }  // RP/2 rows of V_A^T x 128 B per CTA and stage
__host__ __device__ constexpr int p2_smem(int rp) { return 1024 + p2_stages(rp) * (P2_STAGE + p2_v_bytes(rp)) + 1024; }
constexpr uint32_t P2_TMEM_COLS = 512;  // two 256-column accumulators

struct P2Params {
  int T, n_out;
  int main_kb, ext_kb, ext_ksteps;
  int m_tiles, n_tiles;  // pair tiles: ceil(T / 256) x ceil(d_out / 256)
  __nv_bfloat16* y;
  int ldy;
  const __half* scale;
  int32_t* status;
  // fused down-projection (RP > 0)
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma, sA_col, sB_col, r;
  const float* M;        // [64][64] fp32
  __nv_bfloat16* u;      // [T][64]
  uint32_t* u_ready;     // [m_tiles][2]: epoch of the last call that published u for (token tile, CTA rank)
  uint32_t u_target;     // this call's epoch (epochs grow from call to call on a context)
};

template <int RP>
__global__ void __launch_bounds__(P2_THREADS, 1)
essa_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2a,
                const __grid_constant__ CUtensorMap tmB2b, const __grid_constant__ CUtensorMap tmV, const P2Params p) {
  constexpr int STAGES = p2_stages(RP);
  constexpr int V_BYTES = p2_v_bytes(RP);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * P2_A_BYTES;
  uint8_t* smem_v = smem + STAGES * P2_STAGE;  // RP > 0: per stage, this CTA's RP/2 rows of the V_A^T tile
  uint8_t* aux = smem + STAGES * (P2_STAGE + V_BYTES);
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[S], empty[S], tmem_full[2], tmem_empty[2], drain, p_full, p_free
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * STAGES + 7));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* down_count = reinterpret_cast<volatile int*>(tmem_slot + 2);  // epilogue warps that have stored their u rows

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;
  const uint32_t bar_pfull = bar_drain + 8, bar_pfree = bar_pfull + 8;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();  // 0 = leader of the pair
  const bool leader = rank == 0;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int total_kb = p.main_kb + p.ext_kb;
  const int tiles = p.m_tiles * p.n_tiles;
  // the leader's copies of the barriers the peer signals
  const uint32_t full_leader = map_to_cta(bar_full, 0);
  const uint32_t tempty_leader = map_to_cta(bar_tempty, 0);
  const uint32_t pfree_leader = map_to_cta(bar_pfree, 0);
  // Work list of a pair: item w, w + n_pairs, ...  Fused: the tiles of channel column 0 (which also produce u for
  // their token rows) are items 0 .. m_tiles - 1, the others follow row by row.
  auto tile_of = [&](int w, int& m_tile, int& n_tile) {
    if (RP == 0) {
      m_tile = w / p.n_tiles;
      n_tile = w - m_tile * p.n_tiles;
    } else if (w < p.m_tiles) {
      m_tile = w;
      n_tile = 0;
    } else {
      const int w2 = w - p.m_tiles;
      m_tile = w2 / (p.n_tiles - 1);
      n_tile = 1 + (w2 - m_tile * (p.n_tiles - 1));
    }
  };

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 8); }
    mbar_init(bar_drain, 1);
    mbar_init(bar_pfull, 1);
    mbar_init(bar_pfree, 8);
    *abort_flag = 0;
    *down_count = 0;
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

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------------ TMA producers (each CTA: its halves).  Warp 0
    // brings in the activation rows (and the V_A^T rows of a fused first-column tile), warp 6 the W0 / U_B rows: a
    // thread that has just issued a 16 KB box does not get back to the next free slot in time to keep both operand
    // streams full (measured on the decode kernel: one issuing thread was 1.4 times slower per K block than two).
    // Both walk the same stages and wait for the same `empty` phases; the leader's warp 0 posts the byte count.
    const bool prod_a = warp == 0;
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int w = pair; ok && w < tiles; w += n_pairs) {
        int m_tile, n_tile;
        tile_of(w, m_tile, n_tile);
        const bool down = RP > 0 && n_tile == 0;                    // this tile also accumulates P = x V_A
        const int row_a = m_tile * 2 * P2_M + (int)rank * P2_M;     // tokens of this CTA
        const int row_b = n_tile * P2_N + (int)rank * P2_NH;        // channels of this CTA
        for (int kb = 0; kb < total_kb; ++kb) {
          if (RP > 0 && kb == p.main_kb && prod_a) {
            // the u slab of this CTA's token rows: published by the first-column tile of this token tile
            const uint32_t* flag = p.u_ready + 2 * m_tile + (int)rank;
            const long long t0 = clock64();
            while ((int32_t)(ld_acquire_u32(flag) - p.u_target) < 0) {
              if (*abort_flag || clock64() - t0 > kWaitLimitCycles) {
                *abort_flag = 1;
                atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
                ok = false;
                break;
              }
            }
            if (!ok) break;
            fence_proxy_async_global();  // the async-proxy read of u comes after the acquire
          }
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          const bool with_v = down && kb < p.main_kb;
          if (leader && prod_a) mbar_expect_tx(bar_full + 8 * stage, 2u * (P2_STAGE + (with_v ? V_BYTES : 0)));  // the bytes of both CTAs
          const uint32_t fb = full_leader + 8 * stage;
          const uint32_t da = smem_u32(smem_a + stage * P2_A_BYTES), db = smem_u32(smem_b + stage * P2_B_BYTES);
          if (kb < p.main_kb) {
            if (prod_a) {
              tma_load_2d_pair(da, &tmA, kb * P2_K, row_a, fb);
              if (with_v) tma_load_2d_pair(smem_u32(smem_v + stage * V_BYTES), &tmV, kb * P2_K, (int)rank * (RP / 2), fb);
            } else {
              tma_load_2d_pair(db, &tmB, kb * P2_K, row_b, fb);
            }
          } else if (prod_a) {
            tma_load_2d_pair(da, &tmA2, 0, row_a, fb);
          } else {
            tma_load_2d_pair(db, (kb - p.main_kb) == 0 ? &tmB2a : &tmB2b, 0, row_b, fb);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
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
      int n_down = 0;          // first-column tiles so far
      bool prev_down = false;  // the previous tile kept P in the buffer this tile accumulates into
      for (int w = pair; ok && w < tiles; w += n_pairs, ++it) {
        int m_tile, n_tile;
        tile_of(w, m_tile, n_tile);
        const bool down = RP > 0 && n_tile == 0;
        const int buf = it & 1;
        const uint32_t use = (uint32_t)(it >> 1);
        if (!mbar_wait(bar_tempty + 8 * buf, (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
        // P of the previous first-column tile sat in this buffer: its epilogue must have read it
        if (prev_down && !mbar_wait(bar_pfree, (uint32_t)((n_down - 1) & 1), abort_flag, p.status)) { ok = false; break; }
        // P of this tile goes to the other buffer: the previous tile's epilogue must have drained it
        if (down && it > 0 && !mbar_wait(bar_tempty + 8 * (buf ^ 1), (uint32_t)(((it - 1) >> 1) & 1), abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * P2_N);
        const uint32_t p_tmem = tmem_base + (uint32_t)((buf ^ 1) * P2_N);
        for (int kb = 0; kb < total_kb; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(smem_a + stage * P2_A_BYTES));
          const uint64_t b_desc = make_smem_desc(smem_u32(smem_b + stage * P2_B_BYTES));
          if (kb > 0 && kb < p.main_kb) {
            // the hot path as straight-line code: the issuing thread's own instructions between two MMAs (a loop
            // counter, a predicate) show up in the K block's time
            umma_bf16_2cta(d_tmem, a_desc, b_desc, idesc, 1u);
            umma_bf16_2cta(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
            umma_bf16_2cta(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
            umma_bf16_2cta(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
          } else {
            const int nk = (kb < p.main_kb) ? (P2_K / 16) : p.ext_ksteps;
            for (int k = 0; k < nk; ++k) umma_bf16_2cta(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > 0 || k > 0) ? 1u : 0u);
          }
          if (down && kb < p.main_kb) {
            constexpr uint32_t idesc_p = make_idesc(2 * P2_M, RP > 0 ? RP : 16);
            const uint64_t v_desc = make_smem_desc(smem_u32(smem_v + stage * V_BYTES));
            for (int k = 0; k < P2_K / 16; ++k) umma_bf16_2cta(p_tmem, a_desc + 2 * k, v_desc + 2 * k, idesc_p, (kb > 0 || k > 0) ? 1u : 0u);
            if (kb == p.main_kb - 1) umma_commit_2cta(bar_pfull, 3);  // P is complete in both CTAs
          }
          umma_commit_2cta(bar_empty + 8 * stage, 3);  // the stage is free in both CTAs
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (down) ++n_down;
        prev_down = down;
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
    int n_down = 0;
    for (int w = pair; w < tiles; w += n_pairs, ++it) {
      int m_tile, n_tile;
      tile_of(w, m_tile, n_tile);
      const int buf = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      if (RP > 0 && n_tile == 0) {
        // ---- first-column tile: P = x V_A of this thread's token row is in the other accumulator buffer;
        //      u = sB_k .* (M (sA_k .* p)), one token per thread, then publish
        constexpr int R = RP > 0 ? RP : 16;
        int gotp = 1;
        if (lane == 0) gotp = mbar_wait(bar_pfull, (uint32_t)(n_down & 1), abort_flag, p.status) ? 1 : 0;
        gotp = __shfl_sync(0xffffffffu, gotp, 0);
        if (!gotp) break;
        while (!mbar_try_wait(bar_pfull, (uint32_t)(n_down & 1))) {}  // complete: acquire for every lane
        tc_fence_after();
        const uint32_t p_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)((buf ^ 1) * P2_N);
        float q[R];
#pragma unroll
        for (int c = 0; c < R / 16; ++c) {
          float v[16];
          tmem_ld16(p_addr + c * 16, v);
#pragma unroll
          for (int i = 0; i < 16; ++i) q[c * 16 + i] = v[i];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(pfree_leader);  // the buffer may take the next tile's accumulator
        const int t = m_tile * 2 * P2_M + (int)rank * P2_M + row_in_tile;
        if (t < p.T) {
          const int k = find_candidate(p.seg, p.P, t);
          const float* srow = p.sigma + (size_t)k * p.ld_sigma;
#pragma unroll
          for (int i = 0; i < R; ++i) q[i] = (i < p.r) ? q[i] * __ldg(srow + p.sA_col + i) : 0.f;
          uint32_t packed[kRankPadMax / 2];
#pragma unroll
          for (int j2 = 0; j2 < R / 2; ++j2) {
            float uu[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
              const int j = 2 * j2 + h;
              float acc = 0.f;
#pragma unroll
              for (int i4 = 0; i4 < R / 4; ++i4) {
                const float4 mm = __ldg(reinterpret_cast<const float4*>(p.M + j * kRankPadMax) + i4);  // same address in every lane
                acc = fmaf(mm.x, q[4 * i4], acc);
                acc = fmaf(mm.y, q[4 * i4 + 1], acc);
                acc = fmaf(mm.z, q[4 * i4 + 2], acc);
                acc = fmaf(mm.w, q[4 * i4 + 3], acc);
              }
              uu[h] = (j < p.r) ? acc * __ldg(srow + p.sB_col + j) : 0.f;
            }
            packed[j2] = pack_bf16x2(uu[0], uu[1]);
          }
#pragma unroll
          for (int j2 = R / 2; j2 < kRankPadMax / 2; ++j2) packed[j2] = 0u;
          uint4* dst = reinterpret_cast<uint4*>(p.u + (size_t)t * kRankPadMax);
#pragma unroll
          for (int g = 0; g < kRankPadMax / 8; ++g)
            dst[g] = make_uint4(packed[4 * g], packed[4 * g + 1], packed[4 * g + 2], packed[4 * g + 3]);
        }
        // publish: the last of this CTA's four epilogue warps to get here (a counter in shared memory, no barrier
        // that a warp which gave up could leave the others waiting at) stores the call's epoch with release
        __threadfence();
        __syncwarp();
        if (lane == 0) {
          const int arrived = atomicAdd(const_cast<int*>(down_count), 1);
          if ((arrived & 3) == 3) {  // the counter only grows: four arrivals per first-column tile
            __threadfence();
            st_release_u32(p.u_ready + 2 * m_tile + (int)rank, p.u_target);
          }
        }
        ++n_down;
      }
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
                            int ext_ksteps, __nv_bfloat16* y, const __half* scale, const PairDown* down, cudaStream_t stream) {
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
  int rp = 0;
  if (down != nullptr) {
    rp = down->r_pad;
    p.seg = down->seg;
    p.P = down->P;
    p.sigma = down->sigma;
    p.ld_sigma = down->ld_sigma;
    p.sA_col = down->sA_col;
    p.sB_col = down->sB_col;
    p.r = down->r;
    p.M = down->M;
    p.u = down->u;
    p.u_ready = down->u_ready;
    p.u_target = down->u_target;
  }
  const void* kernel = rp == 0    ? (const void*)essa_tc2_kernel<0>
                       : rp == 16 ? (const void*)essa_tc2_kernel<16>
                       : rp == 32 ? (const void*)essa_tc2_kernel<32>
                       : rp == 48 ? (const void*)essa_tc2_kernel<48>
                                  : (const void*)essa_tc2_kernel<64>;
  const int smem = p2_smem(rp);
  static bool attr_done[64][5] = {};  // the attribute is per device and kernel instance
  bool& done = attr_done[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0][rp / 16];
  if (!done) {
    const cudaError_t ea = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (ea != cudaSuccess) return check_cuda(ctx, ea, "cudaFuncSetAttribute(essa_tc2_kernel)");
    done = true;
  }
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
  const long long tiles = (long long)p.m_tiles * p.n_tiles;
  int pairs = (int)(tiles < sm / 2 ? tiles : sm / 2);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
  cfg.blockDim = dim3(P2_THREADS, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (down != nullptr) {
    // tiles wait for u published by other pairs: every pair of the grid must be resident at once
    static int resident[64][5] = {};  // per device and padded rank
    int* cached = &resident[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0][rp / 16];
    if (*cached == 0) {
      int n_clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &cfg) != cudaSuccess || n_clusters <= 0) {
        cudaGetLastError();
        n_clusters = 1;
      }
      *cached = n_clusters;
    }
    if (pairs > *cached) {
      pairs = *cached;
      cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    }
  }
  ctx->launches += 1;
  const CUtensorMap& tmV = down != nullptr ? *down->tmV : tmB2a;  // unused when not fused
  void* args[] = {(void*)&tmA, (void*)&tmB, (void*)&tmA2, (void*)&tmB2a, (void*)&tmB2b, (void*)&tmV, (void*)&p};
  return check_cuda(ctx, cudaLaunchKernelExC(&cfg, kernel, args), "essa_tc2_kernel launch");
}

}  // namespace essa
