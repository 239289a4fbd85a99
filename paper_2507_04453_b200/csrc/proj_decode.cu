// Decode-regime schedule of the population-batched adapted projection (Algorithm 1, line 7, for all
// candidates at once):   y_t = W0 x_t + U_B (sB_k .* (M (sA_k .* (V_A^T x_t)))),   k = cand(t).
//
// With at most a few hundred tokens in the whole population the call is bound by streaming W0 from HBM
// once, so the roles of the operands are swapped with respect to the prefill kernel: 128 rows of W0 (output
// channels) are the UMMA M side, all tokens are the N side, and the reduction over d_in is split over the
// CTAs of a thread-block cluster so that every SM streams a disjoint slice of W0.  One launch does the
// whole call; there is no global scratch:
//
//   K loop (TMA -> shared -> tcgen05.mma -> TMEM), per 64-wide K block of this CTA's slice:
//       D_main[128 ch][tokens] += W0_tile . x_tile^T            (base contraction)
//       D_p[tokens][r_pad]     += x_tile  . V_A_tile            (partial down-projection, same x tile)
//     W0 tiles come from HBM and need a deep ring (HBM latency x bandwidth), x / V_A tiles are L2 hits and get
//     a shallow ring of their own, so that most of shared memory holds W0 bytes in flight.
//   rank core, one token per thread:  u = sB_k .* (M (sA_k .* p))  -> bf16 -> shared, in the swizzled
//       K-major operand layout.  The map p -> u is linear, so applying it to this CTA's partial p and
//       summing over the cluster gives the same rank term as applying it to the full p.
//   up-projection:  D_main += U_B_tile . u^T  (one more UMMA K slab; two for INT8 storage)
//   cluster reduction: after a cluster barrier (all MMAs of the cluster done, operand buffers dead) every
//       CTA pushes the s-th slice of tokens of its fp32 partial tile into CTA s's shared memory (distributed
//       shared memory stores); after a second barrier CTA s sums the slots in fixed rank order (results are
//       deterministic), applies the INT8 per-channel scale, rounds to bf16 once and stores y.
//
// Warp roles (224 threads): warp 0 = W0 / U_B producer, warp 1 = TMEM allocator + MMA issuer, warps 2..5 =
// rank core + epilogue, warp 6 = x / V_A producer.  All mbarrier waits are bounded; a CTA that gives up
// records ESSA_ERR_DEVICE_TIMEOUT, still joins both cluster barriers, frees its TMEM and exits.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int DEC_M = 128;       // W0 rows per CTA (UMMA M)
constexpr int DEC_K = 64;        // 64 bf16 = one 128-byte swizzle row
constexpr int DEC_TOK = 256;     // tokens per tile (UMMA N limit)
constexpr int kDecThreads = 224;
constexpr int kDecSmemBudget = 227 * 1024;
constexpr int W_TILE_BYTES = DEC_M * DEC_K * 2;  // 16 KB
constexpr int kMaxWStages = 10, kMaxXStages = 4;
constexpr int RECV_PAD = 4;      // floats of padding per receive-buffer row (bank-conflict-free 16-byte accesses)

struct DParams {
  int T;          // tokens in the call
  int tn;         // UMMA N of a token tile: multiple of 16, <= 256
  int xrows;      // rows reserved per x stage (128 or 256): the down-projection reads 128-row halves
  int d_out;
  int main_kb;    // d_in / 64
  int m_tiles, tok_tiles, splits;
  int w_stages, x_stages;
  int ext;        // U_B slabs: 1 (bf16 W0) or 2 (INT8 W0: hi + lo of U_B / scale)
  __nv_bfloat16* y;
  int ldy;
  const __half* scale;
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma, sA_col, sB_col, r;
  const float* M;  // [64][64] fp32
  int32_t* status;
};

__host__ __device__ inline int dec_x_stage_bytes(int xrows, int r_pad) { return xrows * 128 + r_pad * 128; }
// tokens of the receive buffer each CTA of a cluster of `splits` owns: a multiple of 16 so that a 16-token
// accumulator chunk never straddles two owners
__host__ __device__ inline int dec_rows_per_owner(int tn, int splits) { return (((tn + splits - 1) / splits) + 15) / 16 * 16; }
__host__ __device__ inline int dec_recv_bytes(int tn, int splits) {
  return splits * DEC_M * (dec_rows_per_owner(tn, splits) + RECV_PAD) * 4;
}

// Candidate that owns token t.  Equal-length segments (the usual decode and prefill batches) are found by
// one proportional guess checked against the offsets; anything else falls back to the binary search.
__device__ __forceinline__ int find_candidate_guess(const int32_t* __restrict__ off, int P, int T, int t) {
  const int g = min(P - 1, (int)(((long long)t * P) / T));
  if (__ldg(off + g) <= t && t < __ldg(off + g + 1)) return g;
  return find_candidate(off, P, t);
}

template <int R_PAD>
__global__ void __launch_bounds__(kDecThreads, 1)
essa_decode_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmX,
                   const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmUB0,
                   const __grid_constant__ CUtensorMap tmUB1, const DParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int SW = p.w_stages, SX = p.x_stages;
  const int x_bytes = p.xrows * 128;
  const int xs_bytes = dec_x_stage_bytes(p.xrows, R_PAD);
  uint8_t* smem_w = smem;                       // W0 ring (the U_B slabs are its last items)
  uint8_t* smem_x = smem + SW * W_TILE_BYTES;   // x / V_A ring
  uint8_t* smem_u = smem_x;                     // u tile: overlays x stage 0 once the K loop is done
  float* smem_m = reinterpret_cast<float*>(smem_x + SX * xs_bytes);
  uint8_t* aux = reinterpret_cast<uint8_t*>(smem_m + R_PAD * R_PAD);
  // receive buffer of the cluster reduction, [splits][128 ch][per + pad] fp32: overlays both rings, which are
  // dead once every MMA of the cluster has completed
  float* recv = reinterpret_cast<float*>(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * kMaxWStages + 2 * kMaxXStages + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const uint32_t bar_wfull = smem_u32(bars), bar_wempty = bar_wfull + 8 * kMaxWStages;
  const uint32_t bar_xfull = bar_wempty + 8 * kMaxWStages, bar_xempty = bar_xfull + 8 * kMaxXStages;
  const uint32_t bar_p = bar_xempty + 8 * kMaxXStages, bar_u = bar_p + 8, bar_d = bar_u + 8, bar_drain = bar_d + 8;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = (int)cluster_ctarank();
  const int item = blockIdx.x / p.splits;
  const int m_tile = item % p.m_tiles;
  const int tok_tile = item / p.m_tiles;
  // this CTA's K blocks [kb0, kb1)
  const int kbase = p.main_kb / p.splits, krem = p.main_kb % p.splits;
  const int kb0 = split * kbase + min(split, krem);
  const int kb1 = kb0 + kbase + (split < krem ? 1 : 0);
  const int nkb = kb1 - kb0;
  const int n_w = nkb + p.ext;  // items of the W0 ring: the K blocks, then the U_B slabs
  const int halves = p.tn > 128 ? 2 : 1;
  const int per = dec_rows_per_owner(p.tn, p.splits);
  const int recv_ld = per + RECV_PAD;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t P_COL = 256;  // D_p halves at columns 256 and 320
  const uint32_t x_tx = (uint32_t)(p.tn * 128 + R_PAD * 128);

  auto load_w = [&](int i) {  // item i of the W0 ring
    const int s = i % SW;
    const uint32_t fb = bar_wfull + 8 * s;
    mbar_expect_tx(fb, (uint32_t)W_TILE_BYTES);
    const uint32_t dst = smem_u32(smem_w + s * W_TILE_BYTES);
    if (i < nkb) tma_load_2d(dst, &tmW, (kb0 + i) * DEC_K, m_tile * DEC_M, fb);
    else tma_load_2d(dst, (i - nkb) == 0 ? &tmUB0 : &tmUB1, 0, m_tile * DEC_M, fb);
  };
  auto load_x = [&](int i) {  // K block i of the x / V_A ring
    const int s = i % SX;
    const uint32_t fb = bar_xfull + 8 * s;
    uint8_t* st = smem_x + s * xs_bytes;
    mbar_expect_tx(fb, x_tx);
    tma_load_2d(smem_u32(st), &tmX, (kb0 + i) * DEC_K, tok_tile * DEC_TOK, fb);
    tma_load_2d(smem_u32(st + x_bytes), &tmV, (kb0 + i) * DEC_K, 0, fb);
  };

  const int first_w = n_w < SW ? n_w : SW;  // both rings start empty: their first fills need no wait
  const int first_x = nkb < SX ? nkb : SX;
  if (threadIdx.x == 0) {
    for (int s = 0; s < SW; ++s) { mbar_init(bar_wfull + 8 * s, 1); mbar_init(bar_wempty + 8 * s, 1); }
    for (int s = 0; s < SX; ++s) { mbar_init(bar_xfull + 8 * s, 1); mbar_init(bar_xempty + 8 * s, 1); }
    mbar_init(bar_p, 1);
    mbar_init(bar_u, 128);
    mbar_init(bar_d, 1);
    mbar_init(bar_drain, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    // start streaming at once
    for (int i = 0; i < first_w; ++i) {
      load_w(i);
      if (i < first_x) load_x(i);
    }
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 || warp == 6) {
    // ------------------------------------------------------------------ TMA producers (W0 ring / x ring)
    if (lane == 0) {
      const bool is_w = warp == 0;
      const int S = is_w ? SW : SX;
      const int n = is_w ? n_w : nkb;
      const uint32_t bar_e = is_w ? bar_wempty : bar_xempty, bar_f = is_w ? bar_wfull : bar_xfull;
      int issued = is_w ? first_w : first_x;
      bool ok = true;
      for (int i = issued; i < n; ++i) {
        if (!mbar_wait(bar_e + 8 * (i % S), (uint32_t)(((i / S) & 1) ^ 1), abort_flag, p.status)) { ok = false; break; }
        if (is_w) load_w(i); else load_x(i);
        ++issued;
      }
      if (!ok || *abort_flag) {
        // giving up: let the copies already issued land before the CTA's shared memory is released
        const int outstanding = issued < S ? issued : S;
        for (int j = 0; j < outstanding; ++j) {
          const int i = issued - 1 - j;
          const long long t0 = clock64();
          while (!mbar_try_wait(bar_f + 8 * (i % S), (uint32_t)((i / S) & 1)) && clock64() - t0 < kWaitLimitCycles) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_main = make_idesc(DEC_M, p.tn);
      constexpr uint32_t idesc_p = make_idesc(128, R_PAD);
      bool ok = true;
      for (int i = 0; i < nkb; ++i) {
        const int sw = i % SW, sx = i % SX;
        if (!mbar_wait(bar_xfull + 8 * sx, (uint32_t)((i / SX) & 1), abort_flag, p.status) ||
            !mbar_wait(bar_wfull + 8 * sw, (uint32_t)((i / SW) & 1), abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        uint8_t* xs = smem_x + sx * xs_bytes;
        const uint64_t dw = make_smem_desc(smem_u32(smem_w + sw * W_TILE_BYTES));
        const uint64_t dx = make_smem_desc(smem_u32(xs));
        const uint64_t dv = make_smem_desc(smem_u32(xs + x_bytes));
        const uint32_t acc0 = i > 0 ? 1u : 0u;
#pragma unroll
        for (int k = 0; k < DEC_K / 16; ++k) umma_bf16(tmem_base, dw + 2 * k, dx + 2 * k, idesc_main, (acc0 | (uint32_t)k) ? 1u : 0u);
        umma_commit(bar_wempty + 8 * sw);
        for (int h = 0; h < halves; ++h) {
          // rows h*128 .. h*128+127 of the x tile as the M side: +16 KB = +1024 in the (address >> 4) field
#pragma unroll
          for (int k = 0; k < DEC_K / 16; ++k)
            umma_bf16(tmem_base + P_COL + 64 * h, dx + 1024 * h + 2 * k, dv + 2 * k, idesc_p, (acc0 | (uint32_t)k) ? 1u : 0u);
        }
        umma_commit(bar_xempty + 8 * sx);
      }
      if (ok) {
        umma_commit(bar_p);
        ok = mbar_wait(bar_u, 0, abort_flag, p.status);
      }
      for (int e = 0; ok && e < p.ext; ++e) {
        const int i = nkb + e;
        if (!mbar_wait(bar_wfull + 8 * (i % SW), (uint32_t)((i / SW) & 1), abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        const uint64_t dub = make_smem_desc(smem_u32(smem_w + (i % SW) * W_TILE_BYTES));
        const uint64_t du = make_smem_desc(smem_u32(smem_u));
#pragma unroll
        for (int k = 0; k < R_PAD / 16; ++k) umma_bf16(tmem_base, dub + 2 * k, du + 2 * k, idesc_main, 1u);
      }
      if (ok) {
        umma_commit(bar_d);
      } else {
        umma_commit(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  }

  // ------------------------------------------------------------------ warps 2..5: rank core, then the epilogue
  const int quad = warp & 3;
  const int row = quad * 32 + lane;  // TMEM lane owned by this thread (warps 2..5 only)
  const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
  const bool epi = warp >= 2 && warp <= 5;
  int got = 0;
  if (epi) {
    // While the K loop streams: core matrix -> shared, this thread's candidates and their singular values.
    constexpr int PRE = (R_PAD <= 32) ? 2 : 1;  // halves whose singular values are fetched ahead of the wait
    for (int idx = threadIdx.x - 64; idx < R_PAD * R_PAD / 4; idx += 128) {
      const int r = idx / (R_PAD / 4), c4 = idx % (R_PAD / 4);
      reinterpret_cast<float4*>(smem_m)[idx] = __ldg(reinterpret_cast<const float4*>(p.M + r * kRankPadMax) + c4);
    }
    int cand[2];
    float sa[PRE][R_PAD], sb[PRE][R_PAD];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int tl = h * 128 + row, t = tok_tile * DEC_TOK + tl;
      cand[h] = (h < halves && tl < p.tn && t < p.T) ? find_candidate_guess(p.seg, p.P, p.T, t) : -1;
    }
    auto load_sigma = [&](int k, float (&a)[R_PAD], float (&b)[R_PAD]) {
      const float* srow = p.sigma + (size_t)(k < 0 ? 0 : k) * p.ld_sigma;
#pragma unroll
      for (int i = 0; i < R_PAD; ++i) {
        a[i] = (k >= 0 && i < p.r) ? __ldg(srow + p.sA_col + i) : 0.f;
        b[i] = (k >= 0 && i < p.r) ? __ldg(srow + p.sB_col + i) : 0.f;
      }
    };
#pragma unroll
    for (int h = 0; h < PRE; ++h) load_sigma(cand[h], sa[h], sb[h]);
    epi_bar_sync();  // core matrix is in shared memory

    got = 1;
    if (lane == 0) got = mbar_wait(bar_p, 0, abort_flag, p.status) ? 1 : 0;
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got) {
      while (!mbar_try_wait(bar_p, 0)) {}  // complete: returns at once (acquire for every lane)
      tc_fence_after();
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        if (h < halves) {
          const int tl = h * 128 + row;  // token within the tile
          if (h >= PRE) load_sigma(cand[h], sa[0], sb[0]);
          float (&a)[R_PAD] = sa[h < PRE ? h : 0];
          float (&b)[R_PAD] = sb[h < PRE ? h : 0];
          float q[R_PAD];
#pragma unroll
          for (int c = 0; c < R_PAD / 16; ++c) {
            float v[16];
            tmem_ld16(t_lane + P_COL + 64 * h + c * 16, v);
#pragma unroll
            for (int i = 0; i < 16; ++i) q[c * 16 + i] = v[i] * a[c * 16 + i];  // sA_k .* p (zero for padding / no token)
          }
          if (tl < p.tn) {
            uint32_t packed[R_PAD / 2];
#pragma unroll
            for (int j2 = 0; j2 < R_PAD / 2; ++j2) {
              float uu[2];
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {
                const int j = 2 * j2 + hh;
                float acc = 0.f;
#pragma unroll
                for (int i4 = 0; i4 < R_PAD / 4; ++i4) {
                  const float4 mm = *reinterpret_cast<const float4*>(smem_m + j * R_PAD + 4 * i4);
                  acc = fmaf(mm.x, q[4 * i4], acc);
                  acc = fmaf(mm.y, q[4 * i4 + 1], acc);
                  acc = fmaf(mm.z, q[4 * i4 + 2], acc);
                  acc = fmaf(mm.w, q[4 * i4 + 3], acc);
                }
                uu[hh] = acc * b[j];  // sB_k .* (M q)
              }
              packed[j2] = pack_bf16x2(uu[0], uu[1]);
            }
            // row tl of the K-major operand: 128 bytes, 16-byte chunk c stored at position c ^ (tl & 7)
            uint8_t* urow = smem_u + (size_t)tl * 128;
#pragma unroll
            for (int c = 0; c < R_PAD / 8; ++c)
              *reinterpret_cast<uint4*>(urow + ((c ^ (tl & 7)) << 4)) =
                  make_uint4(packed[4 * c], packed[4 * c + 1], packed[4 * c + 2], packed[4 * c + 3]);
          }
        }
      }
      fence_proxy_async_smem();
      tc_fence_before();
      mbar_arrive(bar_u);
      // ---- wait for the accumulator (base + rank term of this K slice)
      if (lane == 0) got = mbar_wait(bar_d, 0, abort_flag, p.status) ? 1 : 0;
      got = __shfl_sync(0xffffffffu, got, 0);
      if (got) {
        while (!mbar_try_wait(bar_d, 0)) {}
        tc_fence_after();
      }
    }
  }

  // ------------------------------------------------------------------ cluster reduction and store
  // Every CTA of the cluster has finished its MMAs (or given up): the rings are dead and may be overwritten by
  // the peers' partial sums.
  __syncwarp();
  cluster_sync_all();
  if (epi && got) {
    // push: token chunk c (16 tokens) of this thread's channel goes to slot `split` of the chunk's owner,
    // token-contiguous so that four tokens travel per store
    const uint32_t recv_addr = smem_u32(recv);
#pragma unroll 1
    for (int c = 0; c < p.tn / 16; ++c) {
      float v[16];
      tmem_ld16(t_lane + c * 16, v);
      const int owner = (c * 16) / per;
      const int j = c * 16 - owner * per;  // first token of the chunk within the owner's slice
      const uint32_t dst = map_to_cta(recv_addr + (uint32_t)(((split * DEC_M + row) * recv_ld + j) * 4), (uint32_t)owner);
#pragma unroll
      for (int i = 0; i < 4; ++i) st_dsmem_v4(dst + 16 * i, v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    }
    tc_fence_before();
  }
  __syncwarp();
  cluster_sync_all();  // all partial sums have arrived; nobody touches a peer's shared memory after this point
  if (epi) {
    // thread = channel: sum the slots in rank order, scale, round, store (a warp writes 64 contiguous bytes per token)
    const int ch = m_tile * DEC_M + row;
    const int j_end = min(per, p.tn - split * per);  // tokens of this CTA's slice inside the tile
    const int t0 = tok_tile * DEC_TOK + split * per;  // first token of the slice
    const int j_lim = min(j_end, p.T - t0);           // ... and inside the call
    if (ch < p.d_out) {
      const float sc = p.scale != nullptr ? __half2float(__ldg(p.scale + ch)) : 1.f;
      const float* mine = recv + (size_t)row * recv_ld;
      __nv_bfloat16* ycol = p.y + (size_t)t0 * p.ldy + ch;
      for (int j = 0; j < j_lim; j += 4) {
        float4 acc = *reinterpret_cast<const float4*>(mine + j);
        for (int r = 1; r < p.splits; ++r) {
          const float4 v = *reinterpret_cast<const float4*>(mine + (size_t)r * DEC_M * recv_ld + j);
          acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        const float o[4] = {acc.x * sc, acc.y * sc, acc.z * sc, acc.w * sc};
#pragma unroll
        for (int i = 0; i < 4; ++i)
          if (j + i < j_lim) ycol[(size_t)(j + i) * p.ldy] = __float2bfloat16(o[i]);
      }
    }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

inline int dec_smem_bytes(int w_stages, int x_stages, int xrows, int r_pad) {
  return 1024 + w_stages * W_TILE_BYTES + x_stages * dec_x_stage_bytes(xrows, r_pad) + r_pad * r_pad * 4 + 1024;
}

template <int R_PAD>
int32_t launch_decode(essa_ctx* ctx, const CUtensorMap& tmW, const CUtensorMap& tmX, const CUtensorMap& tmV,
                      const CUtensorMap& tmUB0, const CUtensorMap& tmUB1, const DParams& p, int smem_bytes,
                      cudaStream_t stream) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(essa_decode_kernel<R_PAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBudget);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(essa_decode_kernel)");
    attr_done = true;
  }
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)(p.m_tiles * p.tok_tiles * p.splits), 1, 1);
  cfg.blockDim = dim3(kDecThreads, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)p.splits;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ctx->launches += 1;
  return check_cuda(ctx, cudaLaunchKernelEx(&cfg, essa_decode_kernel<R_PAD>, tmW, tmX, tmV, tmUB0, tmUB1, p),
                    "essa_decode_kernel launch");
}

}  // namespace

// Schedule of the decode kernel for T tokens; returns false when the call should use the prefill kernels.
bool plan_decode(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count, essa_plan* out) {
  if (T <= 0 || T > kDecodeMaxTokens) return false;
  const int sm = sm_count > 0 ? sm_count : 148;
  const int r_pad = ((rank + 15) / 16) * 16;
  const int ext = (w0_dtype == ESSA_W0_INT8_PERCHANNEL) ? 2 : 1;
  const int tn = T <= DEC_TOK ? (int)((T + 15) / 16) * 16 : DEC_TOK;
  const int tok_tiles = (int)((T + DEC_TOK - 1) / DEC_TOK);
  const int xrows = tn <= 128 ? 128 : 256;
  const int m_tiles = (d_out + DEC_M - 1) / DEC_M;
  const int main_kb = d_in / DEC_K;
  const int items = m_tiles * tok_tiles;
  // cluster size: a power of two (packs into a GPC's SMs without stragglers), at most 8 (portable limit)
  int splits = 1;
  while (splits * 2 <= 8 && items * splits * 2 <= sm && splits * 2 <= main_kb) splits *= 2;
  const int kb_per = (main_kb + splits - 1) / splits;
  // x / V_A tiles are L2 hits: two stages (three when they are small); the rest of shared memory holds W0 in flight
  const int xs = dec_x_stage_bytes(xrows, r_pad);
  int x_stages = xs <= 24 * 1024 ? 3 : 2;
  if (x_stages > kb_per) x_stages = kb_per;
  int w_stages = (kDecSmemBudget - dec_smem_bytes(0, x_stages, xrows, r_pad)) / W_TILE_BYTES;
  if (w_stages > kMaxWStages) w_stages = kMaxWStages;
  if (w_stages > kb_per + ext) w_stages = kb_per + ext;
  if (w_stages < 1) return false;
  // the receive buffer of the cluster reduction overlays both rings
  while (w_stages * W_TILE_BYTES + x_stages * xs < dec_recv_bytes(tn, splits)) ++w_stages;
  if (w_stages > kMaxWStages || dec_smem_bytes(w_stages, x_stages, xrows, r_pad) > kDecSmemBudget) return false;
  out->block_m = DEC_M;
  out->block_n = tn;
  out->block_k = DEC_K;
  out->stages = w_stages;
  out->x_stages = x_stages;
  out->k_blocks = main_kb + ext;
  out->splits = splits;
  out->tiles = items;
  out->grid = items * splits;
  out->down_splits = 0;
  out->down_grid = 0;
  out->scratch_bytes = 0;
  out->decode = 1;
  return true;
}

int32_t launch_projection_decode(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, const essa_plan& pl,
                                 cudaStream_t stream) {
  DParams p{};
  p.T = (int)g.T;
  p.tn = pl.block_n;
  p.xrows = p.tn <= 128 ? 128 : 256;
  p.d_out = a->d_out;
  p.main_kb = a->d_in / DEC_K;
  p.m_tiles = (a->d_out + DEC_M - 1) / DEC_M;
  p.tok_tiles = (int)((g.T + DEC_TOK - 1) / DEC_TOK);
  p.splits = pl.splits;
  p.w_stages = pl.stages;
  p.x_stages = pl.x_stages;
  p.ext = a->ext_blocks;
  p.y = g.y;
  p.ldy = a->d_out;
  p.scale = (a->w0_dtype == ESSA_W0_INT8_PERCHANNEL) ? a->w0_scale : nullptr;
  p.seg = g.seg_offsets;
  p.P = g.P;
  p.sigma = g.sigma;
  p.ld_sigma = g.ld_sigma;
  p.sA_col = g.sA_col;
  p.sB_col = g.sB_col;
  p.r = a->rank;
  p.M = a->M;
  p.status = ctx->d_status;

  CUtensorMap tm_x;
  int32_t st = make_tensor_map_2d(ctx, &tm_x, 0, g.x, (uint64_t)g.T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                                  (uint32_t)p.tn, DEC_K, 128);
  if (st != ESSA_OK) return st;
  const int smem_bytes = dec_smem_bytes(p.w_stages, p.x_stages, p.xrows, a->r_pad);
  if (smem_bytes > kDecSmemBudget || p.w_stages > kMaxWStages || p.x_stages > kMaxXStages)
    return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: decode schedule exceeds shared memory");
  const CUtensorMap& tmW = a->tm_W0[1];  // 128-row boxes
  const CUtensorMap& tmU0 = a->tm_UBp[1][0];
  const CUtensorMap& tmU1 = a->tm_UBp[1][a->ext_blocks > 1 ? 1 : 0];
  switch (a->r_pad) {
    case 16: return launch_decode<16>(ctx, tmW, tm_x, a->tm_VAt, tmU0, tmU1, p, smem_bytes, stream);
    case 32: return launch_decode<32>(ctx, tmW, tm_x, a->tm_VAt, tmU0, tmU1, p, smem_bytes, stream);
    case 48: return launch_decode<48>(ctx, tmW, tm_x, a->tm_VAt, tmU0, tmU1, p, smem_bytes, stream);
    case 64: return launch_decode<64>(ctx, tmW, tm_x, a->tm_VAt, tmU0, tmU1, p, smem_bytes, stream);
    default: return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: bad padded rank");
  }
}

}  // namespace essa
