// Tensor-core path of the population-batched adapted projection (Algorithm 1, line 7, for all candidates
// at once):   y_t = W0 x_t + U_B u_t,   u_t = sB_k .* (M (sA_k .* (V_A^T x_t))),   k = cand(t),  M = V_B^T U_A.
//
// Two launches of one warp-specialised kernel template, both TMA -> shared memory -> tcgen05.mma -> TMEM:
//   1. rank-down : D[128 tokens][r_pad] = x_tile . V_A^T over K = d_in; the epilogue owns one token per thread
//                  (TMEM lane), looks up the token's candidate in the segment offsets, applies sA_k, the r x r
//                  core M (shared memory) and sB_k in registers, and writes u_t as bf16 (64 columns, zero padded).
//   2. base + up : D[128 tokens][BLOCK_N channels] = [x | u] . [W0 | U_B]^T : the base contraction over
//                  K = d_in streams W0 once for the whole population, and the rank-r up-projection is one
//                  more K-slab (two for INT8 W0) of the same accumulation.  Epilogue: fp32 -> (x scale[o]) -> bf16.
// No per-candidate weight is ever formed; per-candidate state is the 2r singular values read in step 1.
//
// Small token counts (decode) use split-K over CTAs: partial tiles are added into an fp32 workspace with
// vector reductions and the last CTA to arrive for a tile (atomic counter, no spinning) runs the epilogue
// and re-zeroes the workspace.
//
// Warp roles (192 threads): warp 0 = TMA producer (one lane), warp 1 = TMEM allocator + MMA issuer (one lane),
// warps 2..5 = epilogue (warp w may access TMEM lanes 32*(w%4)..+31).  Two TMEM accumulators let the epilogue
// of one tile overlap the main loop of the next.  Every mbarrier wait is bounded: on expiry the CTA records
// ESSA_ERR_DEVICE_TIMEOUT in the status word, drains its outstanding copies, frees its TMEM and exits.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int BLOCK_M = 128;  // tokens per tile (UMMA M)
constexpr int BLOCK_K = 64;   // 64 bf16 = one 128-byte swizzle row
constexpr int UMMA_K = 16;
constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kSmemBudget = 227 * 1024;

enum { EPI_STORE = 0, EPI_RANK = 1 };

struct KParams {
  int T;           // rows of the activation operand
  int n_out;       // valid accumulator columns: d_out (EPI_STORE) or r_pad (EPI_RANK)
  int main_kb;     // d_in / 64
  int ext_kb;      // rank-path K-slabs appended after the main ones (EPI_STORE only)
  int ext_ksteps;  // r_pad / 16: UMMA K-steps that matter in a rank-path slab
  int m_tiles, n_tiles, splits;
  // EPI_STORE
  __nv_bfloat16* y;
  int ldy;
  const __half* scale;  // per-output-channel scale (INT8 W0) or nullptr
  // EPI_RANK
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma, sA_col, sB_col, r;
  const float* M;  // [64][64] fp32
  __nv_bfloat16* u;  // [T][64]
  // split-K
  float* ws;
  int* cnt;
  int32_t* status;
};

template <int BLOCK_N, int EPI>
struct Cfg {
  static constexpr int A_BYTES = BLOCK_M * BLOCK_K * 2;
  static constexpr int B_BYTES = BLOCK_N * BLOCK_K * 2;
  static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
  static constexpr int M_SMEM_BYTES = (EPI == EPI_RANK) ? BLOCK_N * BLOCK_N * 4 : 0;
  static constexpr int AUX_BYTES = 1024;  // barriers, TMEM slot, flags
  static constexpr int STAGES_RAW = (kSmemBudget - 1024 /*alignment slack*/ - AUX_BYTES - M_SMEM_BYTES) / STAGE_BYTES;
  static constexpr int STAGES = STAGES_RAW > 8 ? 8 : STAGES_RAW;
  static constexpr int SMEM_BYTES = 1024 + STAGES * STAGE_BYTES + M_SMEM_BYTES + AUX_BYTES;
  // two accumulators, each starting at a power-of-two column offset
  static constexpr int ACC_STRIDE = BLOCK_N <= 32 ? 32 : BLOCK_N <= 64 ? 64 : BLOCK_N <= 128 ? 128 : 256;
  static constexpr int TMEM_COLS = 2 * ACC_STRIDE;
  static_assert(BLOCK_N % 16 == 0 && BLOCK_N >= 16 && BLOCK_N <= 256, "UMMA N for M = 128");
  static_assert(STAGES >= 2, "pipeline too shallow");
};

// ------------------------------------------------------------------------------------------------ the kernel
template <int BLOCK_N, int EPI>
__global__ void __launch_bounds__(kThreads, 1)
essa_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2a,
               const __grid_constant__ CUtensorMap tmB2b, const KParams p) {
  using C = Cfg<BLOCK_N, EPI>;
  constexpr int STAGES = C::STAGES;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * C::A_BYTES;
  float* smem_m = reinterpret_cast<float*>(smem + STAGES * C::STAGE_BYTES);
  uint8_t* aux = smem + STAGES * C::STAGE_BYTES + C::M_SMEM_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);  // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * STAGES + 5));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* last_flag = reinterpret_cast<volatile int*>(tmem_slot + 2);
  volatile int* epi_abort = reinterpret_cast<volatile int*>(tmem_slot + 3);

  const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8 * STAGES;
  const uint32_t bar_tfull = bar_empty + 8 * STAGES, bar_tempty = bar_tfull + 16, bar_drain = bar_tempty + 16;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int total_kb = p.main_kb + p.ext_kb;
  const int tiles = p.m_tiles * p.n_tiles;
  const int items = tiles * p.splits;

  if (threadIdx.x == 0) {
    tma_prefetch_desc(&tmA);
    tma_prefetch_desc(&tmB);
    if (p.ext_kb > 0) { tma_prefetch_desc(&tmA2); tma_prefetch_desc(&tmB2a); }
    for (int s = 0; s < STAGES; ++s) { mbar_init(bar_full + 8 * s, 1); mbar_init(bar_empty + 8 * s, 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(bar_tfull + 8 * b, 1); mbar_init(bar_tempty + 8 * b, 4); }
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    *last_flag = 0;
    *epi_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), C::TMEM_COLS);
    tmem_relinquish();
  }
  if (EPI == EPI_RANK && warp >= 2) {
    // core matrix M (zero-padded, row stride 64 in global) -> shared [BLOCK_N][BLOCK_N]
    for (int idx = threadIdx.x - 64; idx < BLOCK_N * BLOCK_N; idx += kEpiThreads)
      smem_m[idx] = p.M[(idx / BLOCK_N) * kRankPadMax + (idx % BLOCK_N)];
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  // work item w -> (tile, split); tile -> (m_tile, n_tile) with n fastest; split s covers K-blocks [kb0, kb1)
  auto item_range = [&](int w, int& m_tile, int& n_tile, int& kb0, int& kb1, int& tile) {
    tile = w / p.splits;
    const int s = w - tile * p.splits;
    m_tile = tile / p.n_tiles;
    n_tile = tile - m_tile * p.n_tiles;
    const int base = total_kb / p.splits, rem = total_kb % p.splits;
    kb0 = s * base + min(s, rem);
    kb1 = kb0 + base + (s < rem ? 1 : 0);
  };

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < items; w += gridDim.x) {
        int m_tile, n_tile, kb0, kb1, tile;
        item_range(w, m_tile, n_tile, kb0, kb1, tile);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(bar_empty + 8 * stage, phase ^ 1, abort_flag, p.status)) { ok = false; break; }
          const uint32_t fb = bar_full + 8 * stage;
          mbar_expect_tx(fb, C::STAGE_BYTES);
          const uint32_t da = smem_u32(smem_a + stage * C::A_BYTES), db = smem_u32(smem_b + stage * C::B_BYTES);
          if (kb < p.main_kb) {
            tma_load_2d(da, &tmA, kb * BLOCK_K, m_tile * BLOCK_M, fb);
            tma_load_2d(db, &tmB, kb * BLOCK_K, n_tile * BLOCK_N, fb);
          } else {
            tma_load_2d(da, &tmA2, 0, m_tile * BLOCK_M, fb);
            tma_load_2d(db, (kb - p.main_kb) == 0 ? &tmB2a : &tmB2b, 0, n_tile * BLOCK_N, fb);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
      }
      if (!ok) {
        // Aborting: let the copies already issued land before the CTA's shared memory is released.
        const int outstanding = issued < STAGES ? issued : STAGES;
        int s = stage;
        uint32_t ph = phase;
        for (int i = 0; i < outstanding; ++i) {
          if (--s < 0) { s = STAGES - 1; ph ^= 1; }
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_full + 8 * s, ph) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = make_idesc(BLOCK_M, BLOCK_N);
      int stage = 0;
      uint32_t phase = 0;
      int it = 0;
      bool ok = true;
      for (int w = blockIdx.x; ok && w < items; w += gridDim.x, ++it) {
        int m_tile, n_tile, kb0, kb1, tile;
        item_range(w, m_tile, n_tile, kb0, kb1, tile);
        const int buf = it & 1;
        const uint32_t use = (uint32_t)(it >> 1);
        if (!mbar_wait(bar_tempty + 8 * buf, (use & 1) ^ 1, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(buf * C::ACC_STRIDE);
        for (int kb = kb0; kb < kb1; ++kb) {
          if (!mbar_wait(bar_full + 8 * stage, phase, abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_desc = make_smem_desc(smem_u32(smem_a + stage * C::A_BYTES));
          const uint64_t b_desc = make_smem_desc(smem_u32(smem_b + stage * C::B_BYTES));
          // advancing K by 16 bf16 inside the swizzled row = +32 bytes = +2 in the (addr >> 4) field
          if (kb > kb0 && kb < p.main_kb) {
            // the hot path as straight-line code: the issuing thread's own instructions between two MMAs (a loop
            // counter, a predicate) show up in the K block's time
            umma_bf16(d_tmem, a_desc, b_desc, idesc, 1u);
            umma_bf16(d_tmem, a_desc + 2, b_desc + 2, idesc, 1u);
            umma_bf16(d_tmem, a_desc + 4, b_desc + 4, idesc, 1u);
            umma_bf16(d_tmem, a_desc + 6, b_desc + 6, idesc, 1u);
          } else {
            const int nk = (kb < p.main_kb) ? (BLOCK_K / UMMA_K) : p.ext_ksteps;
            for (int k = 0; k < nk; ++k) umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
          }
          umma_commit(bar_empty + 8 * stage);
          if (++stage == STAGES) { stage = 0; phase ^= 1; }
        }
        if (ok) umma_commit(bar_tfull + 8 * buf);
      }
      if (!ok) {
        // make sure no MMA is still writing TMEM / reading shared memory when the CTA tears down
        umma_commit(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quad = warp & 3;                   // TMEM lane quadrant this warp may access
    const int row_in_tile = quad * 32 + lane;    // accumulator row (token within the tile) owned by this thread
    const int epi_tid = threadIdx.x - 64;
    int it = 0;
    bool ok = true;
    for (int w = blockIdx.x; ok && w < items; w += gridDim.x, ++it) {
      int m_tile, n_tile, kb0, kb1, tile;
      item_range(w, m_tile, n_tile, kb0, kb1, tile);
      const int buf = it & 1;
      const uint32_t use = (uint32_t)(it >> 1);
      // lane 0 polls (bounded); the warp then takes one common decision
      int got = 1;
      if (lane == 0) got = mbar_wait(bar_tfull + 8 * buf, use & 1, abort_flag, p.status) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (p.splits > 1) {
        // the four epilogue warps meet at named barriers below, so they must also agree on aborting
        epi_bar_sync();
        if (epi_tid == 0) *epi_abort = *abort_flag;
        epi_bar_sync();
        if (*epi_abort) got = 0;
      }
      if (!got) { ok = false; break; }
      while (!mbar_try_wait(bar_tfull + 8 * buf, use & 1)) {}  // already complete: returns at once (acquire for every lane)
      tc_fence_after();
      const uint32_t t_addr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * C::ACC_STRIDE);
      const int t = m_tile * BLOCK_M + row_in_tile;
      const bool row_ok = t < p.T;
      const int col_base = n_tile * BLOCK_N;
      float* ws_tile = p.ws + (size_t)tile * BLOCK_M * BLOCK_N;  // [BLOCK_N/4][128 rows][4]

      if (p.splits > 1) {
        // partial tile -> fp32 workspace (coalesced: consecutive rows are 16 bytes apart)
#pragma unroll 1
        for (int c = 0; c < BLOCK_N / 16; ++c) {
          if (col_base + c * 16 >= p.n_out) break;
          float v[16];
          tmem_ld16(t_addr + c * 16, v);
          if (row_ok) {
#pragma unroll
            for (int g = 0; g < 4; ++g)
              red_add_v4(ws_tile + ((size_t)(c * 4 + g) * BLOCK_M + row_in_tile) * 4, v[4 * g], v[4 * g + 1], v[4 * g + 2],
                         v[4 * g + 3]);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
        __threadfence();
        epi_bar_sync();
        if (epi_tid == 0) {
          const int prev = atomicAdd(p.cnt + tile, 1);
          const int last = (prev == p.splits - 1);
          if (last) p.cnt[tile] = 0;  // all arrivals are in; leave the counter clean for the next call
          *last_flag = last;
        }
        epi_bar_sync();
        const bool last = *last_flag != 0;
        epi_bar_sync();  // everyone has read the flag before a later item overwrites it
        if (!last) continue;
        __threadfence();
      }

      if constexpr (EPI == EPI_STORE) {
#pragma unroll 1
        for (int c = 0; c < BLOCK_N / 16; ++c) {
          const int col0 = col_base + c * 16;
          if (col0 >= p.n_out) break;
          float v[16] = {};
          if (p.splits > 1) {
            if (row_ok) {
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                float* a = ws_tile + ((size_t)(c * 4 + g) * BLOCK_M + row_in_tile) * 4;
                const float4 f = ld_cg_v4(a);
                st_cg_zero_v4(a);
                v[4 * g] = f.x; v[4 * g + 1] = f.y; v[4 * g + 2] = f.z; v[4 * g + 3] = f.w;
              }
            }
          } else {
            tmem_ld16(t_addr + c * 16, v);
          }
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
      } else {
        // rank path, one token per thread:  q = sA_k .* p ;  v = M q ;  u = sB_k .* v
        constexpr int R = BLOCK_N;
        float q[R];
#pragma unroll
        for (int c = 0; c < R / 16; ++c) {
          float v[16] = {};
          if (p.splits > 1) {
            if (row_ok) {
#pragma unroll
              for (int g = 0; g < 4; ++g) {
                float* a = ws_tile + ((size_t)(c * 4 + g) * BLOCK_M + row_in_tile) * 4;
                const float4 f = ld_cg_v4(a);
                st_cg_zero_v4(a);
                v[4 * g] = f.x; v[4 * g + 1] = f.y; v[4 * g + 2] = f.z; v[4 * g + 3] = f.w;
              }
            }
          } else {
            tmem_ld16(t_addr + c * 16, v);
          }
#pragma unroll
          for (int i = 0; i < 16; ++i) q[c * 16 + i] = v[i];
        }
        if (row_ok) {
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
                const float4 mm = *reinterpret_cast<const float4*>(smem_m + j * R + 4 * i4);
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
      }
      if (p.splits == 1) {
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_tempty + 8 * buf);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, C::TMEM_COLS);
  }
}

// ------------------------------------------------------------------------------------------------ host side
template <int BLOCK_N, int EPI>
int32_t launch_one(essa_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmA2,
                   const CUtensorMap& tmB2a, const CUtensorMap& tmB2b, const KParams& p, int grid, cudaStream_t stream) {
  using C = Cfg<BLOCK_N, EPI>;
  static bool attr_done_dev[64] = {};  // the attribute is per device
  bool& attr_done = attr_done_dev[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0];
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(essa_tc_kernel<BLOCK_N, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         C::SMEM_BYTES);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(essa_tc_kernel)");
    attr_done = true;
  }
  essa_tc_kernel<BLOCK_N, EPI><<<grid, kThreads, C::SMEM_BYTES, stream>>>(tmA, tmB, tmA2, tmB2a, tmB2b, p);
  ctx->launches += 1;
  return check_cuda(ctx, cudaGetLastError(), "essa_tc_kernel launch");
}

int stages_for(int block_n, bool rank_epi) {
  const int stage_bytes = BLOCK_M * BLOCK_K * 2 + block_n * BLOCK_K * 2;
  const int m_bytes = rank_epi ? block_n * block_n * 4 : 0;
  int s = (kSmemBudget - 1024 - 1024 - m_bytes) / stage_bytes;
  return s > 8 ? 8 : s;
}

// Relative cost (in SM cycles) of running `tiles` output tiles of width bn with a given split-K factor.
double schedule_cost(int tiles, int bn, int total_kb, int splits, int sm) {
  const double load = 2.0 * (BLOCK_M + bn);  // cycles to bring one K-block of A and B from L2 at ~64 B/clk
  const double mma = 2.0 * bn;               // 4 UMMAs of 128 x bn x 16
  const double per_kb = load > mma ? load : mma;
  const int kb_per_item = (total_kb + splits - 1) / splits;
  const double epilogue = 10.0 * bn * (splits > 1 ? 3.0 : 1.0);
  const double fixed = 3000.0;  // prologue, pipeline fill, teardown
  const long long items = (long long)tiles * splits;
  const double waves = (double)((items + sm - 1) / sm);
  return waves * (kb_per_item * per_kb + epilogue) + fixed;
}

}  // namespace

// Schedule of the two prefill launches (rank-down, base + up).
static void plan_prefill(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count,
                         essa_plan* out) {
  *out = essa_plan{};
  const int sm = sm_count > 0 ? sm_count : 148;
  const int m_tiles = (int)((T + BLOCK_M - 1) / BLOCK_M);
  const int main_kb = d_in / BLOCK_K;
  const int ext = (w0_dtype == ESSA_W0_INT8_PERCHANNEL) ? 2 : 1;
  const int total_kb = main_kb + ext;
  const int r_pad = ((rank + 15) / 16) * 16;
  int best_bn = 256, best_splits = 1;
  double best = 1e300;
  const int bns[3] = {256, 128, 64};
  for (int bi = 0; bi < 3; ++bi) {
    const int bn = bns[bi];
    const int n_tiles = (d_out + bn - 1) / bn;
    const long long tiles = (long long)m_tiles * n_tiles;
    if (tiles == 0) continue;
    const int max_splits = tiles >= sm ? 1 : (int)((sm + tiles - 1) / tiles);
    for (int s = 1; s <= max_splits && s <= total_kb; ++s) {
      // padded-channel waste counts as extra work
      const double waste = (double)(n_tiles * bn) / (double)d_out;
      const double c = schedule_cost((int)(tiles > 0x7fffffff ? 0x7fffffff : tiles), bn, total_kb, s, sm) * (tiles >= sm ? waste : 1.0);
      if (c < best) { best = c; best_bn = bn; best_splits = s; }
    }
  }
  out->block_m = BLOCK_M;
  out->block_n = best_bn;
  out->block_k = BLOCK_K;
  out->stages = stages_for(best_bn, false);
  out->k_blocks = total_kb;
  out->splits = best_splits;
  const int n_tiles = (d_out + best_bn - 1) / best_bn;
  out->tiles = m_tiles * n_tiles;
  const long long items = (long long)out->tiles * best_splits;
  out->grid = (int)(items < sm ? items : sm);
  // rank-down kernel: one tile per 128 tokens, N = r_pad; split K until the SMs are covered
  // (with at least one tile per SM the K range stays whole: splitting it to even out the persistent grid's last round
  // measured SLOWER at every split -- config 4, four launches: 301 us unsplit, 325 / 458 / 715 us split 2 / 4 / 8 ways --
  // because the partial sums go through fp32 atomics in a workspace)
  int ds = 1;
  if (m_tiles > 0 && m_tiles < sm) {
    ds = sm / m_tiles;
    if (ds > main_kb) ds = main_kb;
    if (ds < 1) ds = 1;
  }
  out->down_splits = ds;
  const long long ditems = (long long)m_tiles * ds;
  out->down_grid = (int)(ditems < sm ? ditems : sm);
  int64_t scratch = T * kRankPadMax * 2;
  if (best_splits > 1) scratch += (int64_t)out->tiles * BLOCK_M * best_bn * 4 + (int64_t)out->tiles * 4;
  if (ds > 1) scratch += (int64_t)m_tiles * BLOCK_M * r_pad * 4 + (int64_t)m_tiles * 4;
  out->scratch_bytes = scratch;
}

void plan_projection(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count,
                     essa_plan* out) {
  *out = essa_plan{};
  if (plan_decode(d_in, d_out, rank, w0_dtype, T, sm_count, out)) return;
  plan_prefill(d_in, d_out, rank, w0_dtype, T, sm_count, out);
}

// ESSA_OPT_DOWN_SPLITS: a given K split of the rank-down launch instead of the planner's.
static void override_down_splits(const essa_ctx* ctx, essa_plan* pl, int m_tiles, int main_kb) {
  if (ctx->down_splits <= 0) return;
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;
  int ds = ctx->down_splits < main_kb ? ctx->down_splits : main_kb;
  if (ds < 1) ds = 1;
  pl->down_splits = ds;
  const long long items = (long long)m_tiles * ds;
  pl->down_grid = (int)(items < sm ? items : sm);
}

// Rank-down launch of a prefill call: u_t = sB_k .* (M (sA_k .* (V_A^T x_t))) for all tokens, bf16, [T][64].
static int32_t launch_rank_down(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, int down_splits, int down_grid,
                                const CUtensorMap& tm_x, __nv_bfloat16* u, cudaStream_t stream) {
  KParams kp{};
  kp.T = (int)g.T;
  kp.n_out = a->r_pad;
  kp.main_kb = a->d_in / BLOCK_K;
  kp.ext_kb = 0;
  kp.ext_ksteps = 0;
  kp.m_tiles = (int)((g.T + BLOCK_M - 1) / BLOCK_M);
  kp.n_tiles = 1;
  kp.splits = down_splits;
  kp.seg = g.seg_offsets;
  kp.P = g.P;
  kp.sigma = g.sigma;
  kp.ld_sigma = g.ld_sigma;
  kp.sA_col = g.sA_col;
  kp.sB_col = g.sB_col;
  kp.r = a->rank;
  kp.M = a->M;
  kp.u = u;
  kp.ws = static_cast<float*>(ctx->splitk_ws.ptr);
  kp.cnt = static_cast<int*>(ctx->splitk_cnt.ptr);
  kp.status = ctx->d_status;
  switch (a->r_pad) {
    case 16: return launch_one<16, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream);
    case 32: return launch_one<32, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream);
    case 48: return launch_one<48, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream);
    case 64: return launch_one<64, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream);
    default: return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: bad padded rank");
  }
}

int32_t launch_projection_tc(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, cudaStream_t stream) {
  if (g.T == 0) return ESSA_OK;
  if (g.T > 0x7fffffffLL - BLOCK_M) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: T too large");
  essa_plan pl;
  plan_projection(a->d_in, a->d_out, a->rank, a->w0_dtype, g.T, ctx->sm_count, &pl);
  if (pl.decode) {
    cudaEvent_t* dev = nullptr;
    if (ctx->prof_on) {
      if ((size_t)(ctx->prof_calls + 1) * 3 <= ctx->prof_events.size()) dev = &ctx->prof_events[(size_t)ctx->prof_calls++ * 3];
      else ++ctx->prof_dropped;
    }
    if (dev) { cudaEventRecord(dev[0], stream); cudaEventRecord(dev[1], stream); }
    const int32_t dst = launch_projection_decode(ctx, a, g, pl, stream);
    if (dev) cudaEventRecord(dev[2], stream);
    return dst;
  }
  const int m_tiles = (int)((g.T + BLOCK_M - 1) / BLOCK_M);
  override_down_splits(ctx, &pl, m_tiles, a->d_in / BLOCK_K);

  int32_t st = ensure_scratch(ctx, ctx->u_buf, (size_t)g.T * kRankPadMax * 2, false, stream);
  if (st != ESSA_OK) return st;
  size_t ws_need = 0, cnt_need = 0;
  if (pl.splits > 1) { ws_need = (size_t)pl.tiles * BLOCK_M * pl.block_n * 4; cnt_need = (size_t)pl.tiles * 4; }
  if (pl.down_splits > 1) {
    ws_need = ws_need > (size_t)m_tiles * BLOCK_M * a->r_pad * 4 ? ws_need : (size_t)m_tiles * BLOCK_M * a->r_pad * 4;
    cnt_need = cnt_need > (size_t)m_tiles * 4 ? cnt_need : (size_t)m_tiles * 4;
  }
  if (ws_need) {
    st = ensure_scratch(ctx, ctx->splitk_ws, ws_need, true, stream);
    if (st != ESSA_OK) return st;
    st = ensure_scratch(ctx, ctx->splitk_cnt, cnt_need, true, stream);
    if (st != ESSA_OK) return st;
  }
  __nv_bfloat16* u = static_cast<__nv_bfloat16*>(ctx->u_buf.ptr);

  CUtensorMap tm_x, tm_u;
  st = make_tensor_map_2d(ctx, &tm_x, 0, g.x, (uint64_t)g.T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2, BLOCK_M, BLOCK_K, 128);
  if (st != ESSA_OK) return st;
  st = make_tensor_map_2d(ctx, &tm_u, 0, u, (uint64_t)g.T, kRankPadMax, kRankPadMax * 2, BLOCK_M, BLOCK_K, 128);
  if (st != ESSA_OK) return st;

  cudaEvent_t* ev = nullptr;
  if (ctx->prof_on) {
    if ((size_t)(ctx->prof_calls + 1) * 3 <= ctx->prof_events.size()) ev = &ctx->prof_events[(size_t)ctx->prof_calls++ * 3];
    else ++ctx->prof_dropped;
  }
  if (ev) cudaEventRecord(ev[0], stream);
  // large prefill calls run base + up on 256 x 256 CTA-pair tiles
  const bool use_pairs = ctx->pair_tiles && pl.block_n == 256 && pl.splits == 1 && g.T >= 512;

  // ---- INT8 storage: dequantise the codes (unscaled, exact) into the context's scratch for this call's GEMM
  CUtensorMap tm_wdeq;
  if (a->w0_dtype != ESSA_W0_BF16) {
    const size_t cnt = (size_t)a->d_out * a->d_in;
    st = ensure_scratch(ctx, ctx->w_deq, cnt * 2, false, stream);
    if (st != ESSA_OK) return st;
    st = a->w0_dtype == ESSA_W0_INT8_PERCHANNEL
             ? launch_widen_int8(ctx, a->W0q, static_cast<__nv_bfloat16*>(ctx->w_deq.ptr), cnt, stream)
             : launch_widen_int4(ctx, reinterpret_cast<const uint8_t*>(a->W0q), a->w0_gscale, static_cast<__nv_bfloat16*>(ctx->w_deq.ptr),
                                 a->d_out, a->d_in, stream);
    if (st != ESSA_OK) return st;
    st = make_tensor_map_2d(ctx, &tm_wdeq, 0, ctx->w_deq.ptr, (uint64_t)a->d_out, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                            (uint32_t)(use_pairs ? 128 : pl.block_n), BLOCK_K, 128);
    if (st != ESSA_OK) return st;
  }

  // ---- fused: the pair-tile launch computes u itself (no rank-down launch)
  // (measured: it pays when the first-column tiles, one per 256 tokens, keep most pairs busy in the first round and
  // no pair takes two of them: with fewer token tiles the other pairs idle until u appears, with more the
  // first-column tiles, which cannot overlap their epilogue with the next tile, cost more than the launch saved)
  const int n_pairs_dev = (ctx->sm_count > 0 ? ctx->sm_count : 148) / 2;
  const int64_t pair_rows = (g.T + 255) / 256;
  const bool fused = use_pairs && (ctx->fuse_down == 2 ||
                                   (ctx->fuse_down == 1 && pair_rows <= n_pairs_dev && 4 * pair_rows >= 3 * n_pairs_dev));
  PairDown pd{};
  if (fused) {
    const int pair_m_tiles = (int)((g.T + 255) / 256);
    void* before = ctx->pair_ready.ptr;
    st = ensure_scratch(ctx, ctx->pair_ready, (size_t)pair_m_tiles * 2 * sizeof(uint32_t), true, stream);
    if (st != ESSA_OK) return st;
    if (ctx->pair_ready.ptr != before) ctx->pair_epoch = 0;  // a new (zeroed) counter array
    ctx->pair_epoch += 1;
    pd.r_pad = a->r_pad;
    pd.r = a->rank;
    pd.tmV = &a->tm_VAtH;
    pd.seg = g.seg_offsets;
    pd.P = g.P;
    pd.sigma = g.sigma;
    pd.ld_sigma = g.ld_sigma;
    pd.sA_col = g.sA_col;
    pd.sB_col = g.sB_col;
    pd.M = a->M;
    pd.u = u;
    pd.u_ready = static_cast<uint32_t*>(ctx->pair_ready.ptr);
    pd.u_target = ctx->pair_epoch;
  }

  // ---- launch 1: rank-down
  if (!fused) {
    const DownJob dj{a, g.x, g.sA_col, g.sB_col, u};
    if (down_pairs_suit(ctx, &dj, 1, g.T))
      st = launch_rank_down_pairs(ctx, &dj, 1, g.T, g.seg_offsets, g.P, g.sigma, g.ld_sigma, stream);
    else
      st = launch_rank_down(ctx, a, g, pl.down_splits, pl.down_grid, tm_x, u, stream);
    if (st != ESSA_OK) return st;
  }
  if (ev) cudaEventRecord(ev[1], stream);

  // ---- launch 2: base contraction + up-projection
  KParams mp{};
  mp.T = (int)g.T;
  mp.n_out = a->d_out;
  mp.main_kb = a->d_in / BLOCK_K;
  mp.ext_kb = a->ext_blocks;
  mp.ext_ksteps = a->r_pad / UMMA_K;
  mp.m_tiles = m_tiles;
  mp.n_tiles = (a->d_out + pl.block_n - 1) / pl.block_n;
  mp.splits = pl.splits;
  mp.y = g.y;
  mp.ldy = a->d_out;
  mp.scale = (a->w0_dtype == ESSA_W0_INT8_PERCHANNEL) ? a->w0_scale : nullptr;
  mp.ws = static_cast<float*>(ctx->splitk_ws.ptr);
  mp.cnt = static_cast<int*>(ctx->splitk_cnt.ptr);
  mp.status = ctx->d_status;
  if (use_pairs && !fused &&
      (ctx->wide_tiles == 2 || (ctx->wide_tiles == 1 && wide_tiles_pay(g.T, a->d_out, a->d_in / BLOCK_K + a->ext_blocks, ctx->sm_count)))) {
    WideJob job{};
    job.tmA = &tm_x;
    job.tmB = (a->w0_dtype != ESSA_W0_BF16) ? &tm_wdeq : &a->tm_W0[1];
    job.tmA2 = &tm_u;
    job.tmB2a = &a->tm_UBp[1][0];
    job.tmB2b = &a->tm_UBp[1][a->ext_blocks > 1 ? 1 : 0];
    job.d_out = a->d_out;
    job.main_kb = a->d_in / BLOCK_K;
    job.ext_kb = a->ext_blocks;
    job.ext_ksteps = a->r_pad / UMMA_K;
    job.y = g.y;
    job.scale = mp.scale;
    st = launch_base_up_wide(ctx, &job, 1, (int)g.T, stream);
    if (ev) cudaEventRecord(ev[2], stream);
    return st;
  }
  if (use_pairs) {
    const CUtensorMap& tmW128 = (a->w0_dtype != ESSA_W0_BF16) ? tm_wdeq : a->tm_W0[1];
    st = launch_base_up_pair(ctx, tm_x, tmW128, tm_u, a->tm_UBp[1][0], a->tm_UBp[1][a->ext_blocks > 1 ? 1 : 0], (int)g.T,
                             a->d_out, a->d_in / BLOCK_K, a->ext_blocks, a->r_pad / UMMA_K, g.y, mp.scale, fused ? &pd : nullptr,
                             stream);
    if (st != ESSA_OK && fused) ctx->pair_epoch -= 1;  // nothing was enqueued: the device never reaches this epoch
    if (ev) cudaEventRecord(ev[2], stream);
    return st;
  }
  const int bi = pl.block_n == 64 ? 0 : pl.block_n == 128 ? 1 : 2;
  const CUtensorMap& tmW = (a->w0_dtype != ESSA_W0_BF16) ? tm_wdeq : a->tm_W0[bi];
  const CUtensorMap& tmU0 = a->tm_UBp[bi][0];
  const CUtensorMap& tmU1 = a->tm_UBp[bi][a->ext_blocks > 1 ? 1 : 0];
  switch (pl.block_n) {
    case 64: st = launch_one<64, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, pl.grid, stream); break;
    case 128: st = launch_one<128, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, pl.grid, stream); break;
    default: st = launch_one<256, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, pl.grid, stream); break;
  }
  if (ev) cudaEventRecord(ev[2], stream);
  return st;
}

// The base + up steps of a block's projections (same tokens, segments and table) in ONE wide-tile launch after
// their rank-down launches: the concatenated tile list fills the persistent grid's rounds far better than four
// lists of their own (config 4: 3120 tiles on 74 pairs = 42.2 rounds, against 17.6 + 3.5 + 3.5 + 17.6 rounded up to
// 19 + 4 + 4 + 19).  Returns kBlockNotFused when the block does not suit it (quantised storage, small shapes, options).
int32_t launch_block_prefill(essa_ctx* ctx, const BlockItem* items, int n, int64_t T, const int32_t* seg, int32_t P,
                             const float* sigma, int32_t ld_sigma, cudaStream_t stream) {
  if (n < 2 || n > kWideMaxJobs || T < 512 || T > 0x7fffffffLL - 512) return kBlockNotFused;
  if (!ctx->pair_tiles || ctx->wide_tiles == 0 || ctx->fuse_down != 0) return kBlockNotFused;
  essa_plan pl[kWideMaxJobs];
  const int pairs = (ctx->sm_count > 0 ? ctx->sm_count : 148) / 2;
  long long tiles_w = 0;
  double cost_pair = 0.0, work_w = 0.0, longest_w = 0.0;
  for (int i = 0; i < n; ++i) {
    const essa_adapter* a = items[i].a;
    if (a->w0_dtype != ESSA_W0_BF16) return kBlockNotFused;  // the dequantisation scratch holds one W0 at a time
    plan_projection(a->d_in, a->d_out, a->rank, a->w0_dtype, T, ctx->sm_count, &pl[i]);
    if (pl[i].decode || pl[i].block_n != 256 || pl[i].splits != 1) return kBlockNotFused;
    const int kb = a->d_in / BLOCK_K + a->ext_blocks;
    const long long nt = (a->d_out + 255) / 256;
    const long long t2 = ((T + 255) / 256) * nt, tw = ((T + 511) / 512) * nt;
    cost_pair += (double)((t2 + pairs - 1) / pairs) * (kb * 880.0 + 1500.0);
    work_w += (double)tw * (kb * 1040.0 + 6000.0);
    longest_w = longest_w > kb * 1040.0 + 6000.0 ? longest_w : kb * 1040.0 + 6000.0;
    tiles_w += tw;
  }
  // whole rounds of the persistent grid for the concatenated list (the last, partial round costs one tile)
  const double cost_w = tiles_w <= pairs ? longest_w : work_w / pairs + longest_w * (tiles_w % pairs ? 0.5 : 0.0);
  if (ctx->wide_tiles == 1 && cost_w >= cost_pair) return kBlockNotFused;

  const int m_tiles = (int)((T + BLOCK_M - 1) / BLOCK_M);
  for (int i = 0; i < n; ++i) override_down_splits(ctx, &pl[i], m_tiles, items[i].a->d_in / BLOCK_K);
  const size_t u_stride = (((size_t)T * kRankPadMax * 2 + 255) / 256) * 256;
  int32_t st = ensure_scratch(ctx, ctx->u_buf, (size_t)n * u_stride, false, stream);
  if (st != ESSA_OK) return st;
  size_t ws_need = 0, cnt_need = 0;
  for (int i = 0; i < n; ++i)
    if (pl[i].down_splits > 1) {
      const size_t w = (size_t)m_tiles * BLOCK_M * items[i].a->r_pad * 4;
      ws_need = ws_need > w ? ws_need : w;
      cnt_need = (size_t)m_tiles * 4;
    }
  if (ws_need) {
    st = ensure_scratch(ctx, ctx->splitk_ws, ws_need, true, stream);
    if (st != ESSA_OK) return st;
    st = ensure_scratch(ctx, ctx->splitk_cnt, cnt_need, true, stream);
    if (st != ESSA_OK) return st;
  }
  CUtensorMap tm_x[kWideMaxJobs], tm_u[kWideMaxJobs];
  WideJob jobs[kWideMaxJobs];
  for (int i = 0; i < n; ++i) {
    const essa_adapter* a = items[i].a;
    __nv_bfloat16* u = reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(ctx->u_buf.ptr) + (size_t)i * u_stride);
    st = make_tensor_map_2d(ctx, &tm_x[i], 0, items[i].x, (uint64_t)T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2, BLOCK_M, BLOCK_K, 128);
    if (st != ESSA_OK) return st;
    st = make_tensor_map_2d(ctx, &tm_u[i], 0, u, (uint64_t)T, kRankPadMax, kRankPadMax * 2, BLOCK_M, BLOCK_K, 128);
    if (st != ESSA_OK) return st;
    jobs[i].tmA = &tm_x[i];
    jobs[i].tmB = &a->tm_W0[1];
    jobs[i].tmA2 = &tm_u[i];
    jobs[i].tmB2a = &a->tm_UBp[1][0];
    jobs[i].tmB2b = &a->tm_UBp[1][a->ext_blocks > 1 ? 1 : 0];
    jobs[i].d_out = a->d_out;
    jobs[i].main_kb = a->d_in / BLOCK_K;
    jobs[i].ext_kb = a->ext_blocks;
    jobs[i].ext_ksteps = a->r_pad / UMMA_K;
    jobs[i].y = items[i].y;
    jobs[i].scale = nullptr;
  }
  cudaEvent_t* ev = nullptr;
  if (ctx->prof_on) {
    if ((size_t)(ctx->prof_calls + 1) * 3 <= ctx->prof_events.size()) ev = &ctx->prof_events[(size_t)ctx->prof_calls++ * 3];
    else ++ctx->prof_dropped;
  }
  if (ev) cudaEventRecord(ev[0], stream);
  DownJob dj[kWideMaxJobs];
  for (int i = 0; i < n; ++i)
    dj[i] = DownJob{items[i].a, items[i].x, items[i].sA_col, items[i].sB_col,
                    reinterpret_cast<__nv_bfloat16*>(static_cast<uint8_t*>(ctx->u_buf.ptr) + (size_t)i * u_stride)};
  if (down_pairs_suit(ctx, dj, n, T)) {  // one launch for the rank-down step of all projections
    st = launch_rank_down_pairs(ctx, dj, n, T, seg, P, sigma, ld_sigma, stream);
    if (st != ESSA_OK) return st;
  } else {
    for (int i = 0; i < n; ++i) {
      const ProjArgs g{items[i].x, T, seg, P, sigma, ld_sigma, items[i].sA_col, items[i].sB_col, items[i].y};
      st = launch_rank_down(ctx, items[i].a, g, pl[i].down_splits, pl[i].down_grid, tm_x[i], dj[i].u, stream);
      if (st != ESSA_OK) return st;
    }
  }
  if (ev) cudaEventRecord(ev[1], stream);
  st = launch_base_up_wide(ctx, jobs, n, (int)T, stream);
  if (ev) cudaEventRecord(ev[2], stream);
  return st;
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant (essa_apply_projection_static).
//
// Some callers may not allocate device memory at the moment they need a projection: code that runs inside a
// memory-pool-managed region where every cudaMalloc would fragment or synchronise the pool, a latency-critical
// serving loop that must never hit an implicit device synchronisation, or a process that has handed the whole
// GPU memory budget to another allocator.  For them the rank-path vector u (the only scratch the two launches
// need when split-K is off) lives in this file-scope device array instead of context-owned cudaMalloc memory.
// Every GPU that loads the library holds these kStaticMaxTokens * 128 bytes (512 KB) until the process exits.
//
// In host code the name g_static_u is only a host-side stand-in for the symbol: passing it to a kernel would
// hand the device a host address.  The device address is obtained once per device with cudaGetSymbolAddress,
// with that device current, and it is that pointer the kernels (and the TMA tensor map) receive.
constexpr int kStaticMaxTokens = ESSA_STATIC_MAX_TOKENS;
static __device__ __align__(256) unsigned char g_static_u[(size_t)kStaticMaxTokens * kRankPadMax * 2];

constexpr int kMaxDevices = 64;
static void* g_static_u_addr[kMaxDevices] = {};  // device address of g_static_u, per device, set on first use

int32_t launch_projection_tc_static(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, cudaStream_t stream) {
  if (g.T == 0) return ESSA_OK;
  if (g.T > kStaticMaxTokens)
    return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE,
                "apply_projection_static: T exceeds ESSA_STATIC_MAX_TOKENS (the fixed scratch holds 4096 tokens); "
                "use essa_apply_projection");
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess || cur != ctx->device || cur < 0 || cur >= kMaxDevices)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection_static: the context's device must be the current device");
  if (g_static_u_addr[cur] == nullptr) {
    // One-time set-up on this device (not capturable: do the first call before any stream capture).
    void* p = nullptr;
    const cudaError_t e = cudaGetSymbolAddress(&p, g_static_u);
    if (e != cudaSuccess || p == nullptr) return check_cuda(ctx, e == cudaSuccess ? cudaErrorInvalidSymbol : e, "cudaGetSymbolAddress(g_static_u)");
    g_static_u_addr[cur] = p;
  }
  __nv_bfloat16* u = static_cast<__nv_bfloat16*>(g_static_u_addr[cur]);
  // INT8 / INT4 storage: the call dequantises W0 into the context's scratch, which this entry point will not grow.
  const bool int8 = a->w0_dtype != ESSA_W0_BF16;  // (any quantised storage)
  if (int8 && ctx->w_deq.bytes < (size_t)a->d_out * a->d_in * 2)
    return fail(ctx, ESSA_ERR_ALLOC,
                "apply_projection_static: quantised weights need the context's dequantisation scratch, which is not large "
                "enough yet; size it once with essa_reserve_dequant (this entry point does not allocate)");

  // Same two launches as essa_apply_projection, with split-K off so that u is the only scratch.  Nothing in u has
  // to start at zero: the rank-down launch writes all 64 columns of every row < T and rows >= T are never read
  // (the tensor map over u has exactly T rows), so the previous call's contents are simply overwritten.
  essa_plan pl;
  plan_prefill(a->d_in, a->d_out, a->rank, a->w0_dtype, g.T, ctx->sm_count, &pl);
  const int m_tiles = (int)((g.T + BLOCK_M - 1) / BLOCK_M);
  const int n_tiles = (a->d_out + pl.block_n - 1) / pl.block_n;
  const int sm = ctx->sm_count > 0 ? ctx->sm_count : 148;

  CUtensorMap tm_x, tm_u;
  int32_t st = make_tensor_map_2d(ctx, &tm_x, 0, g.x, (uint64_t)g.T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2, BLOCK_M, BLOCK_K, 128);
  if (st != ESSA_OK) return st;
  st = make_tensor_map_2d(ctx, &tm_u, 0, u, (uint64_t)g.T, kRankPadMax, kRankPadMax * 2, BLOCK_M, BLOCK_K, 128);
  if (st != ESSA_OK) return st;

  KParams kp{};
  kp.T = (int)g.T;
  kp.n_out = a->r_pad;
  kp.main_kb = a->d_in / BLOCK_K;
  kp.m_tiles = m_tiles;
  kp.n_tiles = 1;
  kp.splits = 1;
  kp.seg = g.seg_offsets;
  kp.P = g.P;
  kp.sigma = g.sigma;
  kp.ld_sigma = g.ld_sigma;
  kp.sA_col = g.sA_col;
  kp.sB_col = g.sB_col;
  kp.r = a->rank;
  kp.M = a->M;
  kp.u = u;
  kp.status = ctx->d_status;
  const int down_grid = m_tiles < sm ? m_tiles : sm;
  switch (a->r_pad) {
    case 16: st = launch_one<16, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream); break;
    case 32: st = launch_one<32, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream); break;
    case 48: st = launch_one<48, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream); break;
    case 64: st = launch_one<64, EPI_RANK>(ctx, tm_x, a->tm_VAt, tm_x, a->tm_VAt, a->tm_VAt, kp, down_grid, stream); break;
    default: return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection_static: bad padded rank");
  }
  if (st != ESSA_OK) return st;

  KParams mp{};
  mp.T = (int)g.T;
  mp.n_out = a->d_out;
  mp.main_kb = a->d_in / BLOCK_K;
  mp.ext_kb = a->ext_blocks;
  mp.ext_ksteps = a->r_pad / UMMA_K;
  mp.m_tiles = m_tiles;
  mp.n_tiles = n_tiles;
  mp.splits = 1;
  mp.y = g.y;
  mp.ldy = a->d_out;
  mp.scale = (a->w0_dtype == ESSA_W0_INT8_PERCHANNEL) ? a->w0_scale : nullptr;
  mp.status = ctx->d_status;
  const long long tiles = (long long)m_tiles * n_tiles;
  const int grid = (int)(tiles < sm ? tiles : sm);
  const int bi = pl.block_n == 64 ? 0 : pl.block_n == 128 ? 1 : 2;
  CUtensorMap tm_wdeq;
  if (int8) {
    st = a->w0_dtype == ESSA_W0_INT8_PERCHANNEL
             ? launch_widen_int8(ctx, a->W0q, static_cast<__nv_bfloat16*>(ctx->w_deq.ptr), (size_t)a->d_out * a->d_in, stream)
             : launch_widen_int4(ctx, reinterpret_cast<const uint8_t*>(a->W0q), a->w0_gscale, static_cast<__nv_bfloat16*>(ctx->w_deq.ptr),
                                 a->d_out, a->d_in, stream);
    if (st != ESSA_OK) return st;
    st = make_tensor_map_2d(ctx, &tm_wdeq, 0, ctx->w_deq.ptr, (uint64_t)a->d_out, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                            (uint32_t)pl.block_n, BLOCK_K, 128);
    if (st != ESSA_OK) return st;
  }
  const CUtensorMap& tmW = int8 ? tm_wdeq : a->tm_W0[bi];
  const CUtensorMap& tmU0 = a->tm_UBp[bi][0];
  const CUtensorMap& tmU1 = a->tm_UBp[bi][a->ext_blocks > 1 ? 1 : 0];
  switch (pl.block_n) {
    case 64: return launch_one<64, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, grid, stream);
    case 128: return launch_one<128, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, grid, stream);
    default: return launch_one<256, EPI_STORE>(ctx, tm_x, tmW, tm_u, tmU0, tmU1, mp, grid, stream);
  }
}

}  // namespace essa
