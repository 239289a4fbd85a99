// Decode-regime schedule of the population-batched adapted projection (Algorithm 1, line 7, for all
// candidates at once):   y_t = W0 x_t + U_B (sB_k .* (M (sA_k .* (V_A^T x_t)))),   k = cand(t).
//
// With at most a few hundred tokens in the whole population the call is bound by streaming W0 from HBM
// once, so the roles of the operands are swapped with respect to the prefill kernel: 128 rows of W0 (output
// channels) are the UMMA M side, all tokens are the N side, and the reduction over d_in is split over the
// CTAs of a thread-block cluster so that every SM streams a disjoint slice of W0.  One launch does the
// whole call:
//
//   base contraction (TMA -> shared -> tcgen05.mma -> TMEM), per 64-wide K block of this CTA's slice:
//       D[128 ch][tokens] += W0_tile . x_tile^T
//     A tcgen05.mma of 128 rows costs about the same whatever its width, and a TMA load takes ~2500 cycles even
//     when it hits L2, so the loop issues only the four wide MMAs per K block and keeps all of shared memory
//     full of loads in flight (a ring of W0 tiles from HBM, a ring of x tiles from L2).
//   rank path.  Down-projection p = V_A^T x on the tensor core, as a by-product of the loop: the x tiles are in
//     shared memory anyway, so for a few K blocks (a "slice") a CTA also loads the matching 64-column tile of
//     V_A^T and issues a second MMA with the same x descriptor into a second accumulator,
//     P[rank row][token] += V_A^T_tile . x_tile^T.  The slices of a projection are spread over its CTAs (each
//     CTA starts its K loop at its own slice, so the slices finish within the first few K blocks); an owner's
//     epilogue warps copy the fp32 partial to a per-slice slot in global memory and count an arrival.
//     Finishing step, on the CUDA cores of the epilogue warps (idle during the loop): the first CTAs of the
//     grid each take groups of 8 tokens, wait (bounded) for all slices, sum the slots in slice order,
//     u = sB_k .* (M (sA_k .* p)) in fp32, and publish u_t (bf16) to a small global buffer followed by a
//     release-increment of a counter.
//   up-projection: the CTAs of K split 0 wait (bounded) until the counter shows all T rows, TMA-load u as one
//     more K slab and add  U_B_tile . u^T  (two slabs for INT8 storage) to their accumulator.
//   cluster reduction: after a cluster barrier (all MMAs of the cluster done, operand buffers dead) every
//     CTA pushes the s-th slice of tokens of its fp32 partial tile into CTA s's shared memory (distributed
//     shared memory stores); after a second barrier CTA s sums the slots in fixed rank order (results are
//     deterministic), applies the INT8 per-channel scale, rounds to bf16 once and stores y.
//
// Slice owners never wait for another CTA before they deliver, the finishing CTAs wait only for the owners, and
// both are low-numbered CTAs of the first wave, so every wait ends; all are bounded all the same.  Warp roles: warp 0 = TMA
// producer of the frozen operands (W0 ring, V_A^T tiles), warp 1 = TMEM allocator + MMA issuer, warps 2..5 = rank
// path + epilogue, one more warp (6, or 10 for INT8 storage) = TMA producer of the activations (x ring, u tile);
// INT8 storage adds warps 6..9, which turn the streamed codes into bf16 operand tiles in shared memory.  A CTA that gives up
// on a wait records ESSA_ERR_DEVICE_TIMEOUT, still joins both cluster barriers, frees its TMEM and exits.
#include "common.cuh"
#include "tc_ptx.cuh"

namespace essa {
namespace {

constexpr int DEC_M = 128;       // W0 rows per CTA (UMMA M)
constexpr int DEC_K = 64;        // 64 bf16 = one 128-byte swizzle row
constexpr int kDecThreads = 224;             // warps 0..5 and the activation producer (warp 6)
constexpr int kDecSmemBudget = 227 * 1024;
constexpr int W_TILE_BYTES = DEC_M * DEC_K * 2;  // 16 KB
constexpr int kMaxWStages = 16, kMaxXStages = 6, kMaxCStages = 8;
constexpr int kInt8ConvStages = 4;  // converted tiles between the converting warps and the tensor core
constexpr int kDecThreadsInt8 = 352;         // warps 0..5, INT8 -> bf16 converters (6..9), activation producer (10)
constexpr int RAW_TILE_BYTES = DEC_M * DEC_K;    // 8 KB: one W0 tile as stored INT8 codes
// Storage / conversion modes of the kernel.  kModeBf16: W0 tiles are the MMA operand as stored.  kModeInt8Smem: four
// warps turn tiles of INT8 codes into bf16 operand tiles in shared memory (any token count).  kModeInt8Tmem (at
// most 128 tokens, so that tensor memory has room): the four warps write the converted tile straight into TENSOR
// memory (tcgen05.st, thread = row of the tile) and the MMA takes its A operand from there, which removes the
// write and the read of the converted tile from the shared-memory traffic that bounds the other INT8 mode.
// kModeInt4Tmem: the same for INT4 group-wise storage (4 KB tiles of packed codes, the group scale folded into the
// bf16 value by the converting thread).
constexpr int kModeBf16 = 0, kModeInt8Smem = 1, kModeInt8Tmem = 2, kModeInt4Tmem = 3;
constexpr int RAW4_TILE_BYTES = DEC_M * DEC_K / 2;  // 4 KB: one W0 tile as packed INT4 codes
constexpr int kTmemAStages = 8;                  // converted tiles in tensor memory (32 columns each)
constexpr int kUbSlots = 2;                      // kModeInt8Tmem: the U_B slabs have shared-memory slots of their own
constexpr int kFinishTokens = 8;   // tokens of one finishing unit of the rank path (two threads x four tokens per rank row)
static_assert(kFinishTokens == 8, "finish_unit loads four tokens per thread as one float4");
constexpr int kMaxPSlices = 32;    // slots of partial down-projections per projection
// Ring of V_A^T tiles (used only during a CTA's slice): 16 KB cut into slots of r_pad rows x 128 bytes, so a rank-16
// adapter has eight tiles in flight and a rank-64 adapter two.  (A projection with few row tiles has long slices,
// seven K blocks at the 512-channel k / v projections of the 7B shape: with two slots their V_A^T loads, one L2 round
// trip each, ran one after the other and the whole rank path of the launch waited for them.)
constexpr int kVatStages = 8;      // most slots (barriers are laid out for this many)
constexpr int VAT_RING_BYTES = 2 * kRankPadMax * DEC_K * 2;  // 16 KB
__host__ __device__ inline int vat_stages(int r_pad) { const int s = VAT_RING_BYTES / (r_pad * 128); return s > kVatStages ? kVatStages : s; }
constexpr int DEC_AUX_BYTES = 8 * 1024;  // barriers, flags, finishing-step buffers
constexpr uint32_t TMEM_P_COL = 256;     // the down-projection accumulator sits behind the main one

struct DParams {
  int T;          // tokens in the call (<= 256)
  int tn;         // UMMA N: T rounded up to a multiple of 16
  int xbox;       // rows per TMA box of the x tile (divides tn)
  int d_in, d_out;
  int main_kb;    // d_in / 64
  int m_tiles, splits;
  int w_stages, x_stages;
  int c_stages;   // INT8 storage: depth of the ring of converted (bf16) W0 tiles; 0 for bf16 storage
  int ext;        // U_B slabs: 1 (bf16 W0) or 2 (INT8 W0: hi + lo of U_B / scale)
  __nv_bfloat16* y;
  int ldy;
  const __half* scale;
  const __half* gscale;      // INT4 storage: [d_out][d_in / 128] group scales (folded into the converted values)
  // rank path
  int r_pad;                 // rank rows of a V_A^T tile (the TMA box): 16 / 32 / 48 / 64
  int p_c;                   // K blocks per slice: CTA (m_tile j, split s) owns local K blocks [j p_c, (j+1) p_c)
  int p_per_split;           // slots reserved per split (slot = split * p_per_split + j)
  int rank_groups;           // finishing units: groups of kFinishTokens tokens
  float* p_part;             // [kMaxPSlices][64 rank rows][256 tokens] fp32: partial down-projections, one slot per slice
  uint32_t* p_count;         // slices delivered so far (monotonic across calls)
  uint32_t p_target;         // value of *p_count once this call's slices are all in
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma, sA_col, sB_col, r;
  const float* M;            // [64][64] fp32
  __nv_bfloat16* u;          // [256][64] bf16, rows published by the workers
  uint32_t* u_count;         // rows published so far (monotonic across calls)
  uint32_t u_target;         // value of *u_count once this call's T rows are in
  int32_t* status;
};

// A launch covers up to kMaxBlockProj projections that share the tokens, segments and singular-value table (the
// q, k, v, o of an attention block): each has its own parameter set and tensor maps; CTAs
// cta_begin[i] .. cta_begin[i+1]-1 stream projection i's W0, rank-path units unit_begin[i] .. belong to it.
constexpr int kMaxBlockProj = ESSA_MAX_BLOCK_ITEMS;
struct DBlock {
  int n_proj;
  int cta_begin[kMaxBlockProj + 1];   // multiples of the cluster size; cta_begin[n_proj] = W0-streaming CTAs
  int unit_begin[kMaxBlockProj + 1];  // rank-path units (token group x K slice) per projection
  int rank_ctas;                      // CTAs 0 .. rank_ctas-1 (all in the first wave) take units w, w + rank_ctas, ...
  // Down-projection CTAs.  When the wave has CTAs to spare beyond the W0-streaming ones (n_down > 0: CTAs
  // cta_begin[n_proj] .. + n_down - 1), THEY compute p = V_A^T x: CTA c of them takes K blocks
  // [c KB / n_down, (c + 1) KB / n_down) of every projection (x and V_A^T tiles from L2, one accumulator per
  // projection, delivered to slot c) and the W0-streaming CTAs carry no slices at all.  Otherwise (n_down = 0)
  // the slices ride on the K loops of the first row tiles as described at the top of the file.  (Measured at the
  // 7B decode shape: the 512-channel k / v projections have four row tiles per K split, so their CTAs carried
  // seven-block slices, finished 4 k cycles after everybody else and delivered so late that the up-projection of
  // every projection waited for them.)
  int n_down;
  // Fused draw + block call: the singular-value table is being written by the population-draw kernel launched just
  // before this one; that kernel counts its finished blocks in *sigma_ready.  The launch then does not wait for the
  // draw as a whole (it streams W0 and x beside it) and only the rank path waits for the count (bounded).
  const uint32_t* sigma_ready;
  uint32_t sigma_target;
  // Multi-layer call: blocks of consecutive layers overlap (a CTA of the next block starts as soon as an SM is free),
  // so a later block may not wait for the one before it.  layer_mode 1 (first block): after its own wait for earlier
  // work it publishes layers_epoch in *layers_flag; 2 (later blocks): no wait for the previous kernel, but the
  // activations and the table are touched only once *layers_flag has reached layers_epoch (bounded wait).
  int layer_mode;
  uint32_t* layers_flag;
  uint32_t layers_epoch;
  // Every CTA adds one to *set_done when it is through with the scratch set of its launch.  A later block of a
  // multi-layer call starts only once the earlier launches on ITS set have finished (set_wait_target CTAs), and its
  // CTA 0 leaves only once the launches on the OTHER set issued before it have (other_wait_target), so that the
  // launches of a context complete in the order they were issued although they do not wait for one another.
  long long wait_limit;  // cycles a wait on another thread block's counter may last
  uint32_t* set_done;
  uint32_t set_wait_target;
  const uint32_t* other_done;
  uint32_t other_wait_target;
  DParams proj[kMaxBlockProj];
};
struct DMaps {
  CUtensorMap tm[kMaxBlockProj][6];   // per projection: W0, x, u, U_B slab 0, U_B slab 1, V_A^T
};

// tokens of the receive buffer each CTA of a cluster of `splits` owns: a multiple of 16 so that a 16-token
// accumulator chunk never straddles two owners
__host__ __device__ inline int dec_rows_per_owner(int tn, int splits) { return (((tn + splits - 1) / splits) + 15) / 16 * 16; }
__host__ __device__ inline int dec_recv_bytes(int tn, int splits) {
  return splits * dec_rows_per_owner(tn, splits) * DEC_M * 4;
}

// One finishing unit of the rank path, by the 128 epilogue threads of one CTA: tokens t0 .. t0 + 7 of a projection.
// Thread (h, j) = (etid / 64, etid % 64) owns rank coordinate j of the tokens t0 + 4h .. t0 + 4h + 3: it sums the
// slices' partial p_j (one 16-byte load per slice: the slots are stored [rank row][token]) in slice order
// (deterministic), forms q = sA_k .* p; after a barrier v_j = (M q)_j with its
// row of the core matrix, u_j = sB_k,j v_j, stored as bf16; then the group's tokens are added to the published-row
// count.  Everything that does not depend on the slices (candidate lookup, singular values, the row of M) is
// requested before the wait for them.  Returns false when the wait gave up.
__device__ __forceinline__ bool finish_unit(const DParams& p, int n_down, int grp, float* qbuf /*[kFinishTokens][64]*/, volatile int* flag,
                                            volatile int* abort_flag, int etid) {
  constexpr int TPT = kFinishTokens / 2;  // tokens per thread
  const int j = etid & 63, h = etid >> 6;
  const int t0 = grp * kFinishTokens;
  const int g_n = min(kFinishTokens, p.T - t0);
  // equal-length segments are found by one proportional guess, checked against its two offsets
  float s_a[TPT], s_b[TPT];
#pragma unroll
  for (int g = 0; g < TPT; ++g) {
    s_a[g] = 0.f; s_b[g] = 0.f;
    const int tl = TPT * h + g;
    if (tl < g_n && j < p.r) {
      const int t = t0 + tl;
      const int guess = min(p.P - 1, (int)(((long long)t * p.P) / p.T));
      const int lo = __ldg(p.seg + guess), hi = __ldg(p.seg + guess + 1);
      const int k = (lo <= t && t < hi) ? guess : find_candidate(p.seg, p.P, t);
      const float* srow = p.sigma + (size_t)k * p.ld_sigma;
      s_a[g] = __ldg(srow + p.sA_col + j);
      s_b[g] = __ldg(srow + p.sB_col + j);
    }
  }
  float4 mreg[kRankPadMax / 4];  // row j of M (zero beyond the rank)
#pragma unroll
  for (int i4 = 0; i4 < kRankPadMax / 4; ++i4) mreg[i4] = __ldg(reinterpret_cast<const float4*>(p.M + j * kRankPadMax) + i4);
  // all slices delivered?
  if (etid == 0) {
    int ok = 1;
    const long long w0 = clock64();
    while ((int32_t)(ld_acquire_u32(p.p_count) - p.p_target) < 0) {
      if (*abort_flag || clock64() - w0 > kWaitLimitCycles) { ok = 0; break; }
    }
    if (!ok) {
      *abort_flag = 1;
      atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
    }
    *flag = ok;
  }
  epi_bar_sync();
  const bool ok = *flag != 0;
  if (ok) {
    float pj[TPT];
#pragma unroll
    for (int g = 0; g < TPT; ++g) pj[g] = 0.f;
    // With a padded rank of 16 or 32 only a quarter or half of the 64 rank lanes carry a coordinate: the lanes
    // beyond help with the loads.  Lane j = G jj-lanes: group sg = j / RPp sums the slots sg, sg + G, ... of
    // coordinate jj = j % RPp (eight 16-byte loads in flight), the groups' sums meet in shared memory and are
    // added in group order (still one fixed order: results stay bit-identical run to run).
    const int RPp = p.r_pad <= 16 ? 16 : p.r_pad <= 32 ? 32 : 64;
    const int G = 64 / RPp, jj = j % RPp, sg = j / RPp;
    float4* pbuf = reinterpret_cast<float4*>(qbuf + kFinishTokens * kRankPadMax);  // [2][G][RPp] float4, 2 KB
    if (jj < p.r) {
      // slot sp * p_per_split + sl exists when slice sl of split sp does
      const int kbase = p.main_kb / p.splits, krem = p.main_kb % p.splits;
      const int n_flat = n_down > 0 ? n_down : p.splits * p.p_per_split;
      const float* base = p.p_part + (size_t)jj * kDecodeMaxTokens + t0 + TPT * h;
      for (int i0 = sg; i0 < n_flat; i0 += 8 * G) {
        float4 v4[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int idx = i0 + u * G;
          const int sp = idx / p.p_per_split, sl = idx - sp * p.p_per_split;
          // (down-projection CTAs: slot idx exists when CTA idx got at least one K block of this projection)
          const bool valid = idx < n_flat && (n_down > 0 ? ((long long)(idx + 1) * p.main_kb) / n_down > ((long long)idx * p.main_kb) / n_down
                                                         : sl * p.p_c < kbase + (sp < krem ? 1 : 0));
          v4[u] = valid ? ld_cg_f32x4(base + (size_t)idx * kRankPadMax * kDecodeMaxTokens) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) { pj[0] += v4[u].x; pj[1] += v4[u].y; pj[2] += v4[u].z; pj[3] += v4[u].w; }
      }
    }
    if (G > 1) {
      pbuf[(h * G + sg) * RPp + jj] = make_float4(pj[0], pj[1], pj[2], pj[3]);
      epi_bar_sync();
      if (sg == 0) {
        for (int q = 1; q < G; ++q) {
          const float4 o = pbuf[(h * G + q) * RPp + jj];
          pj[0] += o.x; pj[1] += o.y; pj[2] += o.z; pj[3] += o.w;
        }
      } else {
        pj[0] = pj[1] = pj[2] = pj[3] = 0.f;  // lanes beyond the padded rank carry no coordinate
      }
    }
#pragma unroll
    for (int g = 0; g < TPT; ++g) qbuf[(TPT * h + g) * kRankPadMax + j] = pj[g] * s_a[g];  // sA_k .* p  (zero beyond the rank)
    epi_bar_sync();
    float v[TPT];
#pragma unroll
    for (int g = 0; g < TPT; ++g) v[g] = 0.f;
#pragma unroll
    for (int i4 = 0; i4 < kRankPadMax / 4; ++i4) {
      const float4 mm = mreg[i4];
#pragma unroll
      for (int g = 0; g < TPT; ++g) {
        const float4 qq = *reinterpret_cast<const float4*>(qbuf + (TPT * h + g) * kRankPadMax + 4 * i4);
        v[g] = fmaf(mm.x, qq.x, v[g]);
        v[g] = fmaf(mm.y, qq.y, v[g]);
        v[g] = fmaf(mm.z, qq.z, v[g]);
        v[g] = fmaf(mm.w, qq.w, v[g]);
      }
    }
#pragma unroll
    for (int g = 0; g < TPT; ++g)
      if (TPT * h + g < g_n) p.u[(size_t)(t0 + TPT * h + g) * kRankPadMax + j] = __float2bfloat16(v[g] * s_b[g]);  // sB_k .* (M q)
    // publish: every writer's rows are visible device-wide before the count moves
    __threadfence();
    epi_bar_sync();
    if (etid == 0) red_release_add_u32(p.u_count, (uint32_t)g_n);
  }
  epi_bar_sync();  // qbuf / flag may be reused
  return ok;
}

// Sum token rows j0, j0 + 4, ... < j_end of this CTA's slice over the NS receive slots (cluster rank order:
// deterministic), scale, round to bf16, store; four tokens per pass so that their loads overlap.
// recv layout: [slot][per][128 channels] fp32; each thread owns 4 consecutive channels.
template <int NS>
__device__ __forceinline__ void sum_store(uint32_t mine /*shared-space address*/, int per, int j0, int j_end, const float (&sc)[4],
                                          __nv_bfloat16* yrow0, int ldy) {
  for (int j = j0; j < j_end; j += 16) {
    float4 acc[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int jj = min(j + 4 * u, j_end - 1);  // clamped rows are loaded twice and stored once
      acc[u] = lds_v4f(mine + (uint32_t)(jj * DEC_M * 4));
#pragma unroll
      for (int r = 1; r < NS; ++r) {
        const float4 v = lds_v4f(mine + (uint32_t)((r * per + jj) * DEC_M * 4));
        acc[u].x += v.x; acc[u].y += v.y; acc[u].z += v.z; acc[u].w += v.w;
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int jj = j + 4 * u;
      if (jj < j_end) {
        uint2 o;
        o.x = pack_bf16x2(acc[u].x * sc[0], acc[u].y * sc[1]);
        o.y = pack_bf16x2(acc[u].z * sc[2], acc[u].w * sc[3]);
        *reinterpret_cast<uint2*>(yrow0 + (size_t)jj * ldy) = o;
      }
    }
  }
}

__host__ __device__ constexpr uint32_t tmem_a_col(int stage) { return stage < 4 ? 128u + 32u * stage : 384u + 32u * (stage - 4); }

// PAIR: two CTAs with neighbouring cluster ranks (two W0 row tiles of the same K split) act as one 256-row tcgen05
// CTA pair (cta_group::2).  Each streams (and, for quantised storage, converts) its own W0 tile but only its HALF of
// the token rows of x; the leader (even rank) issues MMAs of M = 256 that read both CTAs' operands and write both
// CTAs' accumulators.  Measured on B200: a cta_group::1 MMA of 128 rows costs ~150 cycles whatever its width, a
// cta_group::2 MMA of 256 x N x 16 runs at the nominal rate (N / 2 cycles), so a pair spends a quarter (128 tokens)
// to a half (256 tokens) of the tensor-core time per W0 tile, and a CTA brings in half the x bytes.
// "full" barriers of rings the pair's MMA reads live in the leader, which posts the bytes of both CTAs; the peer's
// copies complete on them through their cluster address; "empty" barriers exist in both CTAs (multicast commits).
template <int MODE, bool PAIR>
__global__ void __launch_bounds__(MODE != kModeBf16 ? kDecThreadsInt8 : kDecThreads, 1)
essa_decode_kernel(const __grid_constant__ DMaps maps, const __grid_constant__ DBlock blk) {
  static_assert(!(PAIR && MODE == kModeInt8Smem), "the shared-memory conversion mode has no CTA-pair variant");
  constexpr bool INT8 = MODE == kModeInt8Smem;   // codes converted through shared memory
  constexpr bool TS = MODE >= kModeInt8Tmem;     // codes converted into tensor memory (A operand from TMEM)
  constexpr bool I4 = MODE == kModeInt4Tmem;     // ... from packed INT4 codes with group-wise scales
  constexpr bool QUANT = MODE != kModeBf16;
  // which projection this CTA streams (CTAs past the last one only take rank-path units)
  int pi = 0;
  while (pi + 1 < blk.n_proj && (int)blockIdx.x >= blk.cta_begin[pi + 1]) ++pi;
  const DParams& p = blk.proj[pi];
  const CUtensorMap& tmW = maps.tm[pi][0];
  const CUtensorMap& tmX = maps.tm[pi][1];
  const CUtensorMap& tmU = maps.tm[pi][2];
  const CUtensorMap& tmUB0 = maps.tm[pi][3];
  const CUtensorMap& tmUB1 = maps.tm[pi][4];
  const CUtensorMap& tmV = maps.tm[pi][5];
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int SW = p.w_stages, SX = p.x_stages;
  const int hn = PAIR ? p.tn / 2 : p.tn;  // token rows of an x tile held by this CTA
  const int x_bytes = hn * 128;
  constexpr int W_SLOT = I4 ? RAW4_TILE_BYTES : QUANT ? RAW_TILE_BYTES : W_TILE_BYTES;
  const int SC = INT8 ? p.c_stages : (TS ? kUbSlots : 0);   // 16 KB slots behind the W0 ring
  const int SA = TS ? p.c_stages : 1;                       // kModeInt8Tmem: converted tiles in tensor memory
  // V_A^T tiles first: their MMA descriptor spans 128 rows, of which only the r_pad rows of the TMA box are data
  // (the accumulator rows beyond are never read), so the 16 KB it covers must lie inside the allocation
  uint8_t* smem_v = smem;
  const int SV = vat_stages(p.r_pad), v_slot = p.r_pad * 128;
  uint8_t* smem_w = smem_v + VAT_RING_BYTES;  // W0 ring as stored (bf16: the U_B slabs are its last items)
  uint8_t* smem_c = smem_w + SW * W_SLOT;      // INT8: ring of converted bf16 tiles (the U_B slabs are its last items)
  uint8_t* smem_x = smem_c + SC * W_TILE_BYTES;  // x ring (the u tile is its last item)
  uint8_t* aux = smem_x + SX * x_bytes;
  // receive buffer of the cluster reduction, [splits][per tokens][128 ch] fp32: overlays both rings, which are
  // dead once every MMA of the cluster has completed
  float* recv = reinterpret_cast<float*>(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(aux + 8 * (2 * kMaxWStages + 2 * kMaxXStages + 2 * kMaxCStages + 2 + 2 * kVatStages + 1 + kUbSlots + 4));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  float* qbuf = reinterpret_cast<float*>(aux + 1024);      // [kFinishTokens][64]

  const uint32_t bar_wfull = smem_u32(bars), bar_wempty = bar_wfull + 8 * kMaxWStages;
  const uint32_t bar_xfull = bar_wempty + 8 * kMaxWStages, bar_xempty = bar_xfull + 8 * kMaxXStages;
  const uint32_t bar_cfull = bar_xempty + 8 * kMaxXStages, bar_cempty = bar_cfull + 8 * kMaxCStages;
  const uint32_t bar_d = bar_cempty + 8 * kMaxCStages, bar_drain = bar_d + 8;
  const uint32_t bar_vfull = bar_drain + 8, bar_vempty = bar_vfull + 8 * kVatStages, bar_p = bar_vempty + 8 * kVatStages;
  const uint32_t bar_ub = bar_p + 8;  // kModeInt8Tmem: one per U_B slab
  const uint32_t bar_pr = bar_ub + 8 * kUbSlots, bar_pfree = bar_pr + 16;  // down-projection CTAs: accumulator ready / read out (two each)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int crank = (int)cluster_ctarank();
  const int half = PAIR ? (crank & 1) : 0;        // which W0 tile / which half of the tokens of the pair
  const int split = PAIR ? (crank >> 1) : crank;  // K split
  const bool leader = half == 0;
  const uint32_t leader_rank = (uint32_t)(crank & ~1);
  const uint16_t pair_mask = (uint16_t)(3u << leader_rank);
  const bool is_main = (int)blockIdx.x < blk.cta_begin[blk.n_proj];  // later CTAs of the grid only take rank-path units
  const int m_tile = PAIR ? (((int)blockIdx.x - blk.cta_begin[pi]) / (2 * p.splits)) * 2 + half
                          : ((int)blockIdx.x - blk.cta_begin[pi]) / p.splits;
  const int owner_idx = PAIR ? (m_tile >> 1) : m_tile;  // which slice of the down-projection (a pair's leader owns it)
  // this CTA's K blocks [kb0, kb1)
  const int kbase = p.main_kb / p.splits, krem = p.main_kb % p.splits;
  const int kb0 = split * kbase + min(split, krem);
  const int kb1 = kb0 + kbase + (split < krem ? 1 : 0);
  const int nkb = is_main ? kb1 - kb0 : 0;
  const int n_ext = (is_main && split == 0) ? p.ext : 0;  // K split 0 adds the rank term
  const int n_w = QUANT ? nkb : nkb + n_ext;  // items of the W0 ring: the K blocks (bf16: then the U_B slabs)
  const int n_x = nkb + (n_ext ? 1 : 0);     // items of the x ring: the K blocks, then the u tile
  const int per = dec_rows_per_owner(p.tn, p.splits);
  constexpr uint32_t TMEM_COLS = 512;  // main accumulator (up to 256 tokens) + down-projection accumulator
  // The K loop starts at this CTA's slice of the down-projection and wraps around: item i is local K block
  // (r0 + i) mod nkb, and the first c_own items also feed the second accumulator.
  const int r0 = nkb > 0 ? (owner_idx * p.p_c) % nkb : 0;  // (the same in both CTAs of a pair)
  const int c_own = (blk.n_down == 0 && is_main && leader && owner_idx * p.p_c < nkb) ? min(p.p_c, nkb - owner_idx * p.p_c) : 0;
  const int dcta = (int)blockIdx.x - blk.cta_begin[blk.n_proj];  // index among the down-projection CTAs
  const bool is_down = !is_main && dcta < blk.n_down;
  auto kcol = [&](int i) { const int l = r0 + i; return (kb0 + (l >= nkb ? l - nkb : l)) * DEC_K; };

  // a copy whose completion the pair's MMA waits for: counted on the leader's barrier
  auto tma_pair = [&](uint32_t dst, const CUtensorMap* tm, int c_inner, int c_outer, uint32_t fb) {
    if (PAIR) tma_load_2d_pair(dst, tm, c_inner, c_outer, map_to_cta(fb, leader_rank));
    else tma_load_2d(dst, tm, c_inner, c_outer, fb);
  };
  auto load_w = [&](int i) {  // item i of the W0 ring
    const int s = i % SW;
    const uint32_t fb = bar_wfull + 8 * s;
    const uint32_t dst = smem_u32(smem_w + s * W_SLOT);
    if (QUANT) {  // 128 rows of 64 codes (unswizzled; tensor-memory modes: swizzled); read by this CTA's converters only
      mbar_expect_tx(fb, (uint32_t)W_SLOT);
      tma_load_2d(dst, &tmW, I4 ? kcol(i) / 2 : kcol(i), m_tile * DEC_M, fb);
    } else {     // one 128-row box, an operand of the (pair's) MMA
      if (leader) mbar_expect_tx(fb, (uint32_t)(PAIR ? 2 * W_SLOT : W_SLOT));
      const CUtensorMap* tm = i < nkb ? &tmW : ((i - nkb) == 0 ? &tmUB0 : &tmUB1);
      tma_pair(dst, tm, i < nkb ? kcol(i) : 0, m_tile * DEC_M, fb);
    }
  };
  auto load_ub = [&](int e) {  // INT8: U_B slab e goes straight into item nkb + e of the converted ring
    const int s = (nkb + e) % (SC > 0 ? SC : 1);
    const uint32_t fb = bar_cfull + 8 * s;
    mbar_expect_tx(fb, (uint32_t)W_TILE_BYTES);
    const uint32_t dst = smem_u32(smem_c + s * W_TILE_BYTES);
    const CUtensorMap* tm = e == 0 ? &tmUB0 : &tmUB1;
    tma_load_2d(dst, tm, 0, m_tile * DEC_M, fb);
  };
  auto load_ub_slot = [&](int e) {  // tensor-memory modes: U_B slab e into its own slot
    const uint32_t fb = bar_ub + 8 * e;
    if (leader) mbar_expect_tx(fb, (uint32_t)(PAIR ? 2 * W_TILE_BYTES : W_TILE_BYTES));
    tma_pair(smem_u32(smem_c + e * W_TILE_BYTES), e == 0 ? &tmUB0 : &tmUB1, 0, m_tile * DEC_M, fb);
  };
  auto load_x = [&](int i) {  // item i of the x ring
    const int s = i % SX;
    const uint32_t fb = bar_xfull + 8 * s;
    const uint32_t dst = smem_u32(smem_x + s * x_bytes);
    if (leader) mbar_expect_tx(fb, (uint32_t)(PAIR ? 2 * x_bytes : x_bytes));
    const CUtensorMap* tm = i < nkb ? &tmX : &tmU;
    const int col = i < nkb ? kcol(i) : 0;
    for (int r = 0; r < hn; r += p.xbox) tma_pair(dst + (uint32_t)(r * 128), tm, col, half * hn + r, fb);
  };
  auto load_v = [&](int i) {  // V_A^T tile of item i < c_own: r_pad rank rows x 64 input features
    const int s = i % SV;
    const uint32_t fb = bar_vfull + 8 * s;
    mbar_expect_tx(fb, (uint32_t)v_slot);
    tma_load_2d(smem_u32(smem_v + s * v_slot), &tmV, kcol(i), 0, fb);
  };

  // the ring starts empty: its first fill needs no wait (a pair's peer whose copies count on the leader's barriers
  // starts after the cluster barrier below, once those barriers exist)
  const int first_w = (PAIR && !QUANT && !leader) ? 0 : (n_w < SW ? n_w : SW);
  if (threadIdx.x == 0) {
    // kModeInt8Tmem: a tile of codes is read, and its converted tile written, by four warps (one arrival each)
    for (int s = 0; s < SW; ++s) { mbar_init(bar_wfull + 8 * s, 1); mbar_init(bar_wempty + 8 * s, TS ? 4 : 1); }
    for (int s = 0; s < SX; ++s) { mbar_init(bar_xfull + 8 * s, 1); mbar_init(bar_xempty + 8 * s, 1); }
    if (TS) {
      // (a pair's leader collects the converting warps of both CTAs)
      for (int s = 0; s < SA; ++s) { mbar_init(bar_cfull + 8 * s, PAIR ? 8 : 4); mbar_init(bar_cempty + 8 * s, 1); }
      for (int e = 0; e < kUbSlots; ++e) mbar_init(bar_ub + 8 * e, 1);
    } else {
      for (int s = 0; s < SC; ++s) { mbar_init(bar_cfull + 8 * s, 1); mbar_init(bar_cempty + 8 * s, 1); }
    }
    mbar_init(bar_d, 1);
    mbar_init(bar_drain, 1);
    for (int s = 0; s < kVatStages; ++s) { mbar_init(bar_vfull + 8 * s, 1); mbar_init(bar_vempty + 8 * s, 1); }
    mbar_init(bar_p, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(bar_pr + 8 * b, 1); mbar_init(bar_pfree + 8 * b, 1); }
    *abort_flag = 0;
    *reinterpret_cast<volatile int*>(tmem_slot + 3) = 0;  // conversion ticket
    *reinterpret_cast<volatile int*>(tmem_slot + 4) = 0;  // ... and whose turn it is to claim a slot
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < first_w; ++i) load_w(i);  // the frozen weights depend on nothing: stream at once
  }
  if (warp == 1 && (is_main || is_down)) {
    tmem_alloc(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  if (PAIR) cluster_sync_all(); else __syncthreads();  // PAIR: both CTAs' barriers exist before either uses the other's
  tc_fence_after();
  const uint32_t tmem_base = (is_main || is_down) ? *tmem_slot : 0u;  // PAIR: the same address in both CTAs (an SM's only allocation)
  // Everything up to here (barriers, TMEM, the first tiles of the frozen W0) depends on no earlier kernel and, with
  // a programmatic dependent launch, overlaps the kernel before this one in the stream (typically the population
  // draw); x, the singular values, the scratch buffers and y are touched only after this point.  In a fused draw +
  // block call the kernel before is known to be the draw, which writes nothing but the table: no wait here, the
  // rank path waits for the table instead.
  grid_dep_launch();  // the next launch may start its CTAs wherever an SM is free (it waits, or not, on its own terms)
  if (blk.sigma_ready == nullptr && blk.layer_mode != 2) grid_dep_wait();
  if (blk.layer_mode == 1 && blockIdx.x == 0 && threadIdx.x == 0) st_release_u32(blk.layers_flag, blk.layers_epoch);
  auto wait_count = [&](const uint32_t* counter, uint32_t target) -> bool {  // bounded; by one thread
    const long long w0 = clock64();
    while ((int32_t)(ld_acquire_u32(counter) - target) < 0) {
      if (*abort_flag || clock64() - w0 > blk.wait_limit) {
        *abort_flag = 1;
        atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
        return false;
      }
    }
    return true;
  };
  auto wait_layers_flag = [&]() -> bool { return wait_count(blk.layers_flag, blk.layers_epoch); };
  if (blk.layer_mode == 2) {  // the scratch set must be free of the launch two blocks back
    if (threadIdx.x == 0) wait_count(blk.set_done, blk.set_wait_target);
    __syncthreads();
  }

  // ------------------------------------------------------------------ TMA producers: warp 0 streams the frozen
  // operands (the W0 ring and, during this CTA's slice, the V_A^T tiles), warp kXWarp the activations (the x ring,
  // then the u tile).  One issuing thread for both rings measured 1.4 times slower per K block than two (a thread
  // that has just issued a 32 KB box does not get to the other ring's free slot in time).  Each ring is filled in
  // its own order with a bounded wait for the slot; a thread that gives up waits for its copies in flight.
  constexpr int kXWarp = QUANT ? 10 : 6;
  auto drain = [&](int issued, int S, uint32_t bar_f) {
    const int outstanding = issued < S ? issued : S;
    for (int j = 0; j < outstanding; ++j) {
      const int i = issued - 1 - j;
      const long long t0 = clock64();
      while (!mbar_try_wait(bar_f + 8 * (i % S), (uint32_t)((i / S) & 1)) && clock64() - t0 < kWaitLimitCycles) {}
    }
  };
  // a pair's peer cannot see the completion of copies that are counted on the leader's barrier: it gives them time
  auto drain_remote = [&]() {
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000LL) {}
  };
  // ------------------------------------------------------------------ down-projection CTA (see DBlock::n_down)
  // Its units are (projection, K block) in projection order; unit u uses slot u mod depth of the x ring (x tiles of
  // whichever projection, tn rows each) and of a ring of eight 8 KB V_A^T slots at the start of shared memory (this
  // CTA has no W0 ring).  Projection q (counting the ones it has K blocks of) accumulates in TMEM columns 256 (q & 1).
  constexpr int RV = 8, RV_SLOT = 8192;
  auto down_range = [&](int pj, int& a, int& b) {
    const int KB = blk.proj[pj].main_kb;
    a = (int)(((long long)dcta * KB) / blk.n_down);
    b = (int)(((long long)(dcta + 1) * KB) / blk.n_down);
  };
  if (is_down && warp == 0) {
    if (lane == 0) {
      int u = 0;
      bool ok = true;
      for (int pj = 0; ok && pj < blk.n_proj; ++pj) {
        int a, b;
        down_range(pj, a, b);
        for (int kb = a; ok && kb < b; ++kb, ++u) {
          const int sv = u % RV;
          if (u >= RV) ok = mbar_wait(bar_vempty + 8 * sv, (uint32_t)(((u / RV) & 1) ^ 1), abort_flag, p.status);
          if (!ok) break;
          mbar_expect_tx(bar_vfull + 8 * sv, (uint32_t)(blk.proj[pj].r_pad * 128));
          tma_load_2d(smem_u32(smem + sv * RV_SLOT), &maps.tm[pj][5], kb * DEC_K, 0, bar_vfull + 8 * sv);
        }
      }
      if (!ok || *abort_flag) drain(u, RV, bar_vfull);
    }
  } else if (is_down && warp == kXWarp) {
    if (lane == 0) {
      int u = 0;
      bool ok = true;
      if (blk.layer_mode == 2) {
        ok = wait_layers_flag();
        if (ok) fence_proxy_async_global();
      }
      for (int pj = 0; ok && pj < blk.n_proj; ++pj) {
        int a, b;
        down_range(pj, a, b);
        for (int kb = a; ok && kb < b; ++kb, ++u) {
          const int sx = u % SX;
          if (u >= SX) ok = mbar_wait(bar_xempty + 8 * sx, (uint32_t)(((u / SX) & 1) ^ 1), abort_flag, p.status);
          if (!ok) break;
          mbar_expect_tx(bar_xfull + 8 * sx, (uint32_t)x_bytes);
          tma_load_2d(smem_u32(smem_x + sx * x_bytes), &maps.tm[pj][1], kb * DEC_K, 0, bar_xfull + 8 * sx);
        }
      }
      if (!ok || *abort_flag) drain(u, SX, bar_xfull);
    }
  } else if (is_down && warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = make_idesc(DEC_M, p.tn);
      int u = 0, q = 0;
      bool ok = true;
      for (int pj = 0; ok && pj < blk.n_proj; ++pj) {
        int a, b;
        down_range(pj, a, b);
        if (b <= a) continue;
        const int acc = q & 1;
        // the accumulator was last used two projections ago: its slot must have been read out
        if (q >= 2 && !mbar_wait(bar_pfree + 8 * acc, (uint32_t)(((q >> 1) - 1) & 1), abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        for (int kb = a; kb < b; ++kb, ++u) {
          const int sx = u % SX, sv = u % RV;
          if (!mbar_wait(bar_xfull + 8 * sx, (uint32_t)((u / SX) & 1), abort_flag, p.status) ||
              !mbar_wait(bar_vfull + 8 * sv, (uint32_t)((u / RV) & 1), abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t dv = make_smem_desc(smem_u32(smem + sv * RV_SLOT));
          const uint64_t dx = make_smem_desc(smem_u32(smem_x + sx * x_bytes));
#pragma unroll
          for (int k = 0; k < DEC_K / 16; ++k) umma_bf16(tmem_base + (uint32_t)(acc * 256), dv + 2 * k, dx + 2 * k, idesc, (kb > a || k > 0) ? 1u : 0u);
          umma_commit(bar_xempty + 8 * sx);
          umma_commit(bar_vempty + 8 * sv);
        }
        if (!ok) break;
        umma_commit(bar_pr + 8 * acc);
        ++q;
      }
      if (!ok) {
        umma_commit(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  } else if (warp == 0) {
    if (lane == 0) {
      int iw = first_w, iv = 0;
      bool ok = true;
      if (TS) for (int e = 0; e < n_ext; ++e) load_ub_slot(e);
      while (ok && (iw < n_w || iv < c_own)) {
        // The V_A^T tile of item iv goes out no later than the W0 tile of the same item, as soon as its slot is free;
        // the thread only blocks for the slot when nothing else is left to issue or when the W0 slot it would wait
        // for next is held by an MMA that itself needs this tile.
        if (iv < c_own && iv <= iw) {
          const uint32_t vb = bar_vempty + 8 * (iv % SV), vph = (uint32_t)(((iv / SV) & 1) ^ 1);
          bool slot_free = iv < SV || mbar_test_wait(vb, vph);
          if (!slot_free && (iw >= n_w || iw - SW >= iv)) slot_free = ok = mbar_wait(vb, vph, abort_flag, p.status);
          if (slot_free) {
            load_v(iv++);
            continue;
          }
          if (!ok) break;
        }
        if (iw < n_w) {
          if (iw >= SW) ok = mbar_wait(bar_wempty + 8 * (iw % SW), (uint32_t)(((iw / SW) & 1) ^ 1), abort_flag, p.status);
          if (ok) load_w(iw++);
        }
      }
      if (!ok || *abort_flag) {
        if (PAIR && !QUANT && !leader) drain_remote(); else drain(iw, SW, bar_wfull);
        drain(iv, SV, bar_vfull);
      }
    }
  } else if (warp == kXWarp) {
    if (lane == 0) {
      int ix = 0;
      bool ok = true;
      if (blk.layer_mode == 2) {  // the activations may only just have been written by the work before the call
        ok = wait_layers_flag();
        if (ok) fence_proxy_async_global();
      }
      while (ok && ix < n_x) {
        if (ix >= SX) ok = mbar_wait(bar_xempty + 8 * (ix % SX), (uint32_t)(((ix / SX) & 1) ^ 1), abort_flag, p.status);
        if (ok && ix == nkb) {
          // the u tile also needs every row published: acquire the count (bounded), then order the async-proxy
          // read after it
          const long long t0 = clock64();
          while ((int32_t)(ld_acquire_u32(p.u_count) - p.u_target) < 0) {
            if (*abort_flag || clock64() - t0 > blk.wait_limit) {
              *abort_flag = 1;
              atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
              ok = false;
              break;
            }
          }
          if (ok) fence_proxy_async_global();
        }
        if (ok) load_x(ix++);
      }
      if (!ok || *abort_flag) { if (PAIR && !leader) drain_remote(); else drain(ix, SX, bar_xfull); }
    }
  } else if (warp == 1 && is_main) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0 && leader) {
      const uint32_t idesc = make_idesc(PAIR ? 2 * DEC_M : DEC_M, p.tn);
      auto mma = [&](uint32_t d, uint64_t da, uint64_t db, uint32_t acc) {
        if (PAIR) umma_bf16_2cta(d, da, db, idesc, acc); else umma_bf16(d, da, db, idesc, acc);
      };
      auto mma_ts = [&](uint32_t d, uint32_t ta, uint64_t db, uint32_t acc) {
        if (PAIR) umma_bf16_ts_2cta(d, ta, db, idesc, acc); else umma_bf16_ts(d, ta, db, idesc, acc);
      };
      auto commit = [&](uint32_t bar) {  // PAIR: to the barrier at this offset in both CTAs
        if (PAIR) umma_commit_2cta(bar, pair_mask); else umma_commit(bar);
      };
      auto commit_own = [&](uint32_t bar) {  // to this CTA's barrier only
        if (PAIR) umma_commit_2cta(bar, (uint16_t)(1u << crank)); else umma_commit(bar);
      };
      bool ok = true;
      // The loop is bound by what this thread itself executes between two MMAs (the K block's four MMAs need ~685
      // cycles of tensor time at 256 tokens, the block took ~1080 with operands always ready), so the ring positions,
      // phases and descriptors advance by increments: no division by the runtime ring depths, no address arithmetic.
      const int SWm = INT8 ? SC : TS ? SA : SW;  // depth of the ring the MMA's weight operand comes from
      int sw = 0, sx = 0;
      uint32_t wph = 0, xph = 0;
      const uint32_t wf0 = (INT8 || TS) ? bar_cfull : bar_wfull;
      const uint64_t dw0 = make_smem_desc(smem_u32(INT8 ? smem_c : smem_w)), dx0 = make_smem_desc(smem_u32(smem_x));
      const uint64_t dw_step = (uint64_t)(W_TILE_BYTES >> 4), dx_step = (uint64_t)(x_bytes >> 4);  // descriptors hold address >> 4
      uint64_t dw = dw0, dx = dx0;
      for (int i = 0; i < nkb; ++i) {
        if (!mbar_wait(bar_xfull + 8 * sx, xph, abort_flag, p.status) ||
            !mbar_wait(wf0 + 8 * sw, wph, abort_flag, p.status)) { ok = false; break; }
        tc_fence_after();
        if (TS) {  // A operand: the converted tile in tensor memory, 8 columns (16 bf16) per K step
          const uint32_t ta = tmem_base + tmem_a_col(sw);
#pragma unroll
          for (int k = 0; k < DEC_K / 16; ++k) mma_ts(tmem_base, ta + 8 * k, dx + 2 * k, (i > 0 || k > 0) ? 1u : 0u);
        } else {
#pragma unroll
          for (int k = 0; k < DEC_K / 16; ++k) mma(tmem_base, dw + 2 * k, dx + 2 * k, (i > 0 || k > 0) ? 1u : 0u);
        }
        if (i < c_own) {
          // this CTA's slice of the down-projection: V_A^T tile against the same x tile, second accumulator
          const int sv = i % SV;
          if (!mbar_wait(bar_vfull + 8 * sv, (uint32_t)((i / SV) & 1), abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t dv = make_smem_desc(smem_u32(smem_v + sv * v_slot));
#pragma unroll
          // (PAIR: the peer's rows of this accumulator come from whatever its shared memory holds there; never read)
          for (int k = 0; k < DEC_K / 16; ++k) mma(tmem_base + TMEM_P_COL, dv + 2 * k, dx + 2 * k, (i > 0 || k > 0) ? 1u : 0u);
          commit_own(bar_vempty + 8 * sv);
          if (i == c_own - 1) commit_own(bar_p);  // the slice is complete
        }
        commit(((INT8 || TS) ? bar_cempty : bar_wempty) + 8 * sw);
        commit(bar_xempty + 8 * sx);
        if (++sw == SWm) { sw = 0; wph ^= 1u; dw = dw0; } else { dw += dw_step; }
        if (++sx == SX) { sx = 0; xph ^= 1u; dx = dx0; } else { dx += dx_step; }
      }
      if (ok && n_ext > 0) {
        // rank term: u tile (x ring item nkb) against the U_B slabs (W0 ring items nkb ..)
        ok = mbar_wait(bar_xfull + 8 * (nkb % SX), (uint32_t)((nkb / SX) & 1), abort_flag, p.status);
        const uint64_t du = make_smem_desc(smem_u32(smem_x + (nkb % SX) * x_bytes));
        const int ksteps = (p.r + 15) / 16;
        for (int e = 0; ok && e < n_ext; ++e) {
          const int i = nkb + e;
          const int su = INT8 ? i % SC : TS ? e : i % SW;
          const uint32_t ubar = INT8 ? bar_cfull + 8 * su : TS ? bar_ub + 8 * e : bar_wfull + 8 * su;
          if (!mbar_wait(ubar, TS ? 0u : (uint32_t)((INT8 ? i / SC : i / SW) & 1), abort_flag, p.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t dub = make_smem_desc(smem_u32(((INT8 || TS) ? smem_c : smem_w) + su * W_TILE_BYTES));
          for (int k = 0; k < ksteps; ++k) mma(tmem_base, dub + 2 * k, du + 2 * k, 1u);
        }
      }
      if (ok) {
        commit(bar_d);
      } else {
        commit_own(bar_drain);
        const long long t0 = clock64();
        while (!mbar_try_wait(bar_drain, 0) && clock64() - t0 < kWaitLimitCycles) {}
      }
    }
  }

  // ------------------------------------------------------------------ INT8 -> bf16 conversion (INT8 storage only)
  // Items of the converted ring are handed out to warps 6..9 by a ticket counter in shared memory, so the
  // warps work on different tiles at once.  A warp converts a whole tile:
  // raw tile = 128 rows of 64 codes, row r at byte 64 r; converted tile = the K-major 128-byte-swizzled operand
  // layout, row r at byte 128 r, 16-byte chunk c at position c ^ (r & 7).  Lane l takes the 16-code chunks
  // l, l + 32, ... (conflict-free 16-byte reads), two at a time for instruction-level parallelism.  Tickets
  // nkb .. are the U_B slabs, which arrive ready-made by TMA into the same ring (its slots are reused in item
  // order, which the ticket order preserves).
  volatile int* ticket = reinterpret_cast<volatile int*>(tmem_slot + 3);
  volatile int* turn = reinterpret_cast<volatile int*>(tmem_slot + 4);
  auto convert_loop = [&]() {
    const int SCd = SC > 0 ? SC : 1;
    for (;;) {
      int i = 0;
      if (lane == 0) i = atomicAdd(const_cast<int*>(ticket), 1);
      i = __shfl_sync(0xffffffffu, i, 0);
      if (i >= nkb + n_ext) break;
      const int sc = i % SCd;
      int got_c = 1;
      if (lane == 0) {
        // Slots are claimed strictly in ticket order: a parity wait is only meaningful for the oldest waiter (a
        // warp further ahead than the ring is deep would see the parity of an older phase), so each ticket
        // holder first waits for its turn, then for its slot, then passes the turn on.
        const long long t0 = clock64();
        while (*turn != i) {
          if (*abort_flag || clock64() - t0 > kWaitLimitCycles) { got_c = 0; break; }
        }
        if (got_c) {
          got_c = (i < SCd || mbar_wait(bar_cempty + 8 * sc, (uint32_t)(((i / SCd) & 1) ^ 1), abort_flag, p.status)) ? 1 : 0;
          __threadfence_block();
          *turn = i + 1;
        }
        if (!got_c) {
          *abort_flag = 1;
          atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
        }
        if (got_c && i >= nkb) {
          load_ub(i - nkb);
          if (*abort_flag) {
            const long long t0 = clock64();
            while (!mbar_try_wait(bar_cfull + 8 * sc, (uint32_t)((i / SCd) & 1)) && clock64() - t0 < kWaitLimitCycles) {}
          }
        }
        if (got_c && i < nkb) got_c = mbar_wait(bar_wfull + 8 * (i % SW), (uint32_t)((i / SW) & 1), abort_flag, p.status) ? 1 : 0;
      }
      got_c = __shfl_sync(0xffffffffu, got_c, 0);
      if (!got_c) break;
      if (i >= nkb) continue;
      const int sr = i % SW;
      // (lane 0 has observed the phase and the shuffle orders the other lanes after it: a barrier probe by all 32 lanes
      // costs ~200 cycles even when the phase is complete)
      const uint32_t raw = smem_u32(smem_w + sr * RAW_TILE_BYTES);
      const uint32_t out = smem_u32(smem_c + sc * W_TILE_BYTES);
#pragma unroll 2
      for (int c0 = 0; c0 < RAW_TILE_BYTES / 16; c0 += 64) {
        uint4 w[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) w[h] = lds_v4(raw + (uint32_t)((c0 + 32 * h + lane) * 16));
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int chunk = c0 + 32 * h + lane;
          const int r = chunk >> 2, part = chunk & 3;
          uint4 o0, o1;
          int8x4_to_bf16x4(w[h].x, o0.x, o0.y);
          int8x4_to_bf16x4(w[h].y, o0.z, o0.w);
          int8x4_to_bf16x4(w[h].z, o1.x, o1.y);
          int8x4_to_bf16x4(w[h].w, o1.z, o1.w);
          const uint32_t orow = out + (uint32_t)(r * 128);
          sts_v4(orow + (uint32_t)(((2 * part) ^ (r & 7)) << 4), o0);
          sts_v4(orow + (uint32_t)(((2 * part + 1) ^ (r & 7)) << 4), o1);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();  // the whole tile is written (and the raw tile read)
      if (lane == 0) {
        mbar_arrive(bar_cfull + 8 * sc);
        mbar_arrive(bar_wempty + 8 * sr);
      }
    }
  };
  if (INT8 && warp >= 6 && warp <= 9) convert_loop();
  // kModeInt8Tmem.  Warp w of the four converting warps owns rows (= tensor-memory lanes) 32 (w mod 4) .. + 31 of
  // EVERY tile, a thread one row: it reads the row's 64 codes (four 16-byte chunks; the tile was loaded with the
  // 64-byte swizzle, chunk c of row r at position c ^ ((r >> 1) & 3), so the eight rows a quarter-warp reads at once
  // fall into eight different bank groups), converts them exactly and stores the 32 packed bf16 pairs into the
  // 32 columns of the tile's stage with one tcgen05.st.  The stage is handed to the MMA warp when all four warps
  // have arrived; the slot of codes goes back to the TMA producer the same way.
  if (TS && warp >= 6 && warp <= 9) {
    const int band = warp & 3;
    const int r = band * 32 + lane;
    // one row of tile i: codes from the ring slot -> 32 packed bf16 pairs
    auto convert_row = [&](int i, int sr /* = i mod SW */, uint32_t (&v)[32]) {
      if (I4) {
        // a row of the tile is 32 bytes = two 16-byte chunks, loaded with the 32-byte swizzle (chunk c of row r at
        // position c ^ ((r >> 2) & 1): again eight different bank groups per quarter-warp); the 64 codes of the row
        // lie in one group of 128 input features and share its scale
        const uint32_t raw = smem_u32(smem_w + sr * W_SLOT) + (uint32_t)(r * 32);
        const int ch = m_tile * DEC_M + r;
        const float gs = ch < p.d_out ? __half2float(__ldg(p.gscale + (size_t)ch * (p.d_in >> 7) + (kcol(i) >> 7))) : 0.f;
        uint4 w[2];
#pragma unroll
        for (int c = 0; c < 2; ++c) w[c] = lds_v4(raw + (uint32_t)((c ^ ((r >> 2) & 1)) << 4));
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const uint32_t ws[4] = {w[c].x, w[c].y, w[c].z, w[c].w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            uint32_t o4[4];
            int4x8_to_bf16x8(ws[k], gs, o4);
#pragma unroll
            for (int e = 0; e < 4; ++e) v[16 * c + 4 * k + e] = o4[e];
          }
        }
      } else {
        const uint32_t raw = smem_u32(smem_w + sr * W_SLOT) + (uint32_t)(r * 64);
        uint4 w[4];
#pragma unroll
        for (int c = 0; c < 4; ++c) w[c] = lds_v4(raw + (uint32_t)((c ^ ((r >> 1) & 3)) << 4));
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int8x4_to_bf16x4(w[c].x, v[8 * c + 0], v[8 * c + 1]);
          int8x4_to_bf16x4(w[c].y, v[8 * c + 2], v[8 * c + 3]);
          int8x4_to_bf16x4(w[c].z, v[8 * c + 4], v[8 * c + 5]);
          int8x4_to_bf16x4(w[c].w, v[8 * c + 6], v[8 * c + 7]);
        }
      }
    };
    // lane 0 observes the barriers of tile i (its stage of tensor memory is free, its codes have landed)
    auto tile_ready = [&](int i) -> bool {
      const int sa = i % SA, sr = i % SW;
      if (i >= SA && !mbar_wait(bar_cempty + 8 * sa, (uint32_t)(((i / SA) & 1) ^ 1), abort_flag, p.status)) return false;
      return mbar_wait(bar_wfull + 8 * sr, (uint32_t)((i / SW) & 1), abort_flag, p.status);
    };
    auto publish = [&](int i) {  // by lane 0, after the tile's store has completed
      const int sa = i % SA, sr = i % SW;
      if (PAIR) mbar_arrive_cluster(map_to_cta(bar_cfull + 8 * sa, leader_rank)); else mbar_arrive(bar_cfull + 8 * sa);
      mbar_arrive(bar_wempty + 8 * sr);
    };
    // Two tiles at a time: their loads, arithmetic and stores interleave (a warp alone on a tile spent most of its
    // ~590 cycles waiting for its own shared-memory loads and dependent arithmetic), and the barrier round trips
    // are shared.
    int i = 0;
    const bool two = SW >= 2 && SA >= 2;  // (tile i + 1 must not need the slot or the stage tile i still holds)
    // Ring positions and phases of tiles i and i + 1 advance by increments: the divisions by the runtime ring depths
    // they replace (sixteen per round, in every lane) cost more than the barrier observation itself.
    int sr0 = 0, sr1 = SW > 1 ? 1 : 0, sa0 = 0, sa1 = SA > 1 ? 1 : 0;
    uint32_t rph0 = 0, rph1 = 0, aph0 = 0, aph1 = 0;  // (i / SW) & 1, (i / SA) & 1 of the two tiles
    for (; two && i + 1 < nkb; i += 2) {
      // lanes 0..3 observe the four barriers of the two tiles side by side (free stages of tensor memory, landed codes:
      // one lane taking them in turn spent ~100 cycles on each although they were complete); the vote orders the other
      // lanes' reads of the tiles after that.  (Probing the barriers with all 32 lanes cost ~420 cycles per tile.)
      int got_c = 1;
      if (lane < 4) {
        const bool second = (lane & 1) != 0;
        const bool stage_free = lane >= 2;  // lanes 2, 3: the tile's stage of tensor memory; lanes 0, 1: its codes
        const uint32_t bar = stage_free ? bar_cempty + 8 * (second ? sa1 : sa0) : bar_wfull + 8 * (second ? sr1 : sr0);
        const uint32_t par = stage_free ? ((second ? aph1 : aph0) ^ 1u) : (second ? rph1 : rph0);
        if (!stage_free || i + (second ? 1 : 0) >= SA) got_c = mbar_wait(bar, par, abort_flag, p.status) ? 1 : 0;
      }
      got_c = __all_sync(0xffffffffu, got_c);
      if (!got_c) break;
      tc_fence_after();  // the MMAs that read these stages have completed (their commit released them)
      uint32_t va[32], vb[32];
      convert_row(i, sr0, va);
      convert_row(i + 1, sr1, vb);
      tmem_st32_issue(tmem_base + ((uint32_t)(band * 32) << 16) + tmem_a_col(sa0), va);
      tmem_st32_issue(tmem_base + ((uint32_t)(band * 32) << 16) + tmem_a_col(sa1), vb);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        if (PAIR) {
          mbar_arrive_cluster(map_to_cta(bar_cfull + 8 * sa0, leader_rank));
          mbar_arrive_cluster(map_to_cta(bar_cfull + 8 * sa1, leader_rank));
        } else {
          mbar_arrive(bar_cfull + 8 * sa0);
          mbar_arrive(bar_cfull + 8 * sa1);
        }
        mbar_arrive(bar_wempty + 8 * sr0);
        mbar_arrive(bar_wempty + 8 * sr1);
      }
      sr0 += 2; if (sr0 >= SW) { sr0 -= SW; rph0 ^= 1u; }
      sr1 += 2; if (sr1 >= SW) { sr1 -= SW; rph1 ^= 1u; }
      sa0 += 2; if (sa0 >= SA) { sa0 -= SA; aph0 ^= 1u; }
      sa1 += 2; if (sa1 >= SA) { sa1 -= SA; aph1 ^= 1u; }
    }
    for (; i < nkb; ++i) {  // an odd last tile (or every tile, with a ring of one)
      int got_c = 1;
      if (lane == 0) got_c = tile_ready(i) ? 1 : 0;
      got_c = __shfl_sync(0xffffffffu, got_c, 0);
      if (!got_c) break;
      tc_fence_after();
      uint32_t va[32];
      convert_row(i, i % SW, va);
      tmem_st32(tmem_base + ((uint32_t)(band * 32) << 16) + tmem_a_col(i % SA), va);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) publish(i);
    }
  }

  // ------------------------------------------------------------------ warps 2..5: rank path, then the epilogue
  const int quad = warp & 3;
  const int row = quad * 32 + lane;  // TMEM lane (output channel of the tile) owned by this thread
  const uint32_t t_lane = tmem_base + ((uint32_t)(quad * 32) << 16);
  const bool epi = warp >= 2 && warp <= 5;
  int got = 0;
  if (epi) {
    const int etid = threadIdx.x - 64;
    volatile int* flag = reinterpret_cast<volatile int*>(tmem_slot + 2);
    if (is_down) {
      int q = 0;
      bool fine = true;
      for (int pj = 0; fine && pj < blk.n_proj; ++pj) {
        int a, b;
        down_range(pj, a, b);
        if (b <= a) continue;
        const DParams& pp = blk.proj[pj];
        const int acc = q & 1;
        int have = 0;
        if (lane == 0) have = mbar_wait(bar_pr + 8 * acc, (uint32_t)((q >> 1) & 1), abort_flag, p.status) ? 1 : 0;
        have = __shfl_sync(0xffffffffu, have, 0);
        if (!have) { fine = false; break; }
        while (!mbar_try_wait(bar_pr + 8 * acc, (uint32_t)((q >> 1) & 1))) {}  // complete: acquire for every lane
        tc_fence_after();
        if (quad * 32 < pp.r_pad) {
          float* slot = pp.p_part + (size_t)dcta * kDecodeMaxTokens * kRankPadMax;
#pragma unroll 1
          for (int c = 0; c < pp.tn / 16; ++c) {
            float v[16];
            tmem_ld16(t_lane + (uint32_t)(acc * 256) + c * 16, v);
            if (row < pp.r_pad) {
              float4* dst = reinterpret_cast<float4*>(slot + (size_t)row * kDecodeMaxTokens + c * 16);
#pragma unroll
              for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
          }
        }
        tc_fence_before();
        __threadfence();
        epi_bar_sync();
        if (etid == 0) {
          red_release_add_u32(pp.p_count, 1u);
          mbar_arrive(bar_pfree + 8 * acc);
        }
        ++q;
      }
    }
    if (c_own > 0) {
      // this CTA's slice of the down-projection: accumulator rows (rank index) x columns (token) -> its slot
      int have = 0;
      if (lane == 0) have = mbar_wait(bar_p, 0, abort_flag, p.status) ? 1 : 0;
      have = __shfl_sync(0xffffffffu, have, 0);
      if (have) {
        while (!mbar_try_wait(bar_p, 0)) {}  // complete: returns at once (acquire for every lane)
        tc_fence_after();
        if (quad * 32 < p.r_pad) {
          float* slot = p.p_part + (size_t)(split * p.p_per_split + owner_idx) * kDecodeMaxTokens * kRankPadMax;
#pragma unroll 1
          for (int c = 0; c < p.tn / 16; ++c) {
            float v[16];
            tmem_ld16(t_lane + TMEM_P_COL + c * 16, v);
            if (row < p.r_pad) {  // [rank row][token]; columns of tokens beyond T are zero (their x rows are)
              float4* dst = reinterpret_cast<float4*>(slot + (size_t)row * kDecodeMaxTokens + c * 16);
#pragma unroll
              for (int i = 0; i < 4; ++i) dst[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
            }
          }
          tc_fence_before();
        }
        __threadfence();
        epi_bar_sync();
        if (etid == 0) red_release_add_u32(p.p_count, 1u);
      }
    }
    if ((int)blockIdx.x < blk.rank_ctas) {
      // this CTA's finishing units of the rank path (of any projection of the block), while its K loop streams
      bool fine = true;
      if (blk.layer_mode == 2 && (int)blockIdx.x < blk.unit_begin[blk.n_proj]) {
        if (etid == 0) *flag = wait_layers_flag() ? 1 : 0;
        epi_bar_sync();
        fine = *flag != 0;
        epi_bar_sync();  // flag may be reused
      }
      if (fine && blk.sigma_ready != nullptr && (int)blockIdx.x < blk.unit_begin[blk.n_proj]) {
        // the table must be complete before its rows are read
        if (etid == 0) {
          int ok = 1;
          const long long w0 = clock64();
          while ((int32_t)(ld_acquire_u32(blk.sigma_ready) - blk.sigma_target) < 0) {
            if (*abort_flag || clock64() - w0 > kWaitLimitCycles) { ok = 0; break; }
          }
          if (!ok) {
            *abort_flag = 1;
            atomicCAS(p.status, 0, ESSA_ERR_DEVICE_TIMEOUT);
          }
          *flag = ok;
        }
        epi_bar_sync();
        fine = *flag != 0;
        epi_bar_sync();  // flag may be reused
      }
      for (int unit = blockIdx.x; fine && unit < blk.unit_begin[blk.n_proj]; unit += blk.rank_ctas) {
        int pj = 0;
        while (pj + 1 < blk.n_proj && unit >= blk.unit_begin[pj + 1]) ++pj;
        fine = finish_unit(blk.proj[pj], blk.n_down, unit - blk.unit_begin[pj], qbuf, flag, abort_flag, etid);
      }
    }
    got = is_main ? 1 : 0;
    if (is_main && lane == 0) got = mbar_wait(bar_d, 0, abort_flag, p.status) ? 1 : 0;
    got = __shfl_sync(0xffffffffu, got, 0);
    if (got) {
      while (!mbar_try_wait(bar_d, 0)) {}  // complete: returns at once (acquire for every lane)
      tc_fence_after();
    }
  }

  // ------------------------------------------------------------------ cluster reduction and store
  // Every CTA of the cluster has finished its MMAs (or given up): the rings are dead and may be overwritten by
  // the peers' partial sums.
  __syncwarp();
  cluster_sync_all();
  if (epi && got) {
    // push: token chunk c (16 tokens) of this thread's channel goes to slot `split` of the chunk's owner;
    // a warp writes 128 contiguous bytes (32 channels of one token) per store
    const uint32_t recv_addr = smem_u32(recv);
#pragma unroll 1
    for (int c = 0; c < p.tn / 16; ++c) {
      float v[16];
      tmem_ld16(t_lane + c * 16, v);
      const int owner = (c * 16) / per;
      const int j = c * 16 - owner * per;  // first token of the chunk within the owner's slice
      const uint32_t dst = map_to_cta(recv_addr + (uint32_t)((((split * per + j) * DEC_M) + row) * 4),
                                      (uint32_t)(PAIR ? 2 * owner + half : owner));
#pragma unroll
      for (int i = 0; i < 16; ++i) st_dsmem_f32(dst + (uint32_t)(i * DEC_M * 4), v[i]);
    }
    tc_fence_before();
  }
  __syncwarp();
  cluster_sync_all();  // all partial sums have arrived; nobody touches a peer's shared memory after this point
  if (epi && is_main) {
    // each thread owns 4 consecutive channels; warp ew takes tokens ew, ew + 4, ... of this CTA's slice
    const int ew = warp - 2;
    const int t0 = split * per;                             // first token of the slice
    const int j_lim = min(min(per, p.tn - t0), p.T - t0);    // tokens of the slice inside the call
    const int ch0 = m_tile * DEC_M + 4 * lane;
    if (ch0 < p.d_out) {  // d_out is a multiple of 8: a group of 4 channels is all in or all out
      float sc[4] = {1.f, 1.f, 1.f, 1.f};
      if (p.scale != nullptr) {
#pragma unroll
        for (int i = 0; i < 4; ++i) sc[i] = __half2float(__ldg(p.scale + ch0 + i));
      }
      const uint32_t mine = smem_u32(recv + 4 * lane);
      __nv_bfloat16* yrow0 = p.y + (size_t)t0 * p.ldy + ch0;
      const int ldy = p.ldy;
      switch (p.splits) {
        case 1: sum_store<1>(mine, per, ew, j_lim, sc, yrow0, ldy); break;
        case 2: sum_store<2>(mine, per, ew, j_lim, sc, yrow0, ldy); break;
        case 4: sum_store<4>(mine, per, ew, j_lim, sc, yrow0, ldy); break;
        default: sum_store<8>(mine, per, ew, j_lim, sc, yrow0, ldy); break;
      }
    }
  }
  __syncthreads();
  if (warp == 1 && (is_main || is_down)) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (threadIdx.x == 0) {
    if (blk.layer_mode == 2 && blockIdx.x == 0) wait_count(blk.other_done, blk.other_wait_target);
    red_release_add_u32(blk.set_done, 1u);
  }
}

// Shared-memory rings: V_A^T tiles, the W0 ring (16 KB bf16 tiles, or 8 KB tiles of codes), the 16 KB slots behind it
// (kModeInt8Smem: c_stages converted tiles; kModeInt8Tmem: the U_B slabs), the x ring.
inline int dec_w_slot(int mode) { return mode == kModeBf16 ? W_TILE_BYTES : mode == kModeInt4Tmem ? RAW4_TILE_BYTES : RAW_TILE_BYTES; }
// (x_rows: token rows of an x tile held by one CTA: all of them, or half when the CTAs work in pairs)
inline int dec_ring_bytes(int mode, int w_stages, int c_stages, int x_stages, int x_rows) {
  const int slots16k = mode == kModeInt8Smem ? c_stages : mode >= kModeInt8Tmem ? kUbSlots : 0;
  return VAT_RING_BYTES + w_stages * dec_w_slot(mode) + slots16k * W_TILE_BYTES + x_stages * x_rows * 128;
}
inline int dec_smem_bytes(int mode, int w_stages, int c_stages, int x_stages, int x_rows) {
  return 1024 + dec_ring_bytes(mode, w_stages, c_stages, x_stages, x_rows) + DEC_AUX_BYTES;
}
// INT8 storage converts into tensor memory whenever the accumulators leave room for the converted tiles there.
// INT4 storage has the tensor-memory mode only: larger calls take the prefill kernels (negative: no decode schedule).
inline int dec_mode(int w0_dtype, int tn) {
  if (w0_dtype == ESSA_W0_BF16) return kModeBf16;
  if (w0_dtype == ESSA_W0_INT4_GROUP128) return tn <= 128 ? kModeInt4Tmem : -1;
  return tn <= 128 ? kModeInt8Tmem : kModeInt8Smem;
}

}  // namespace

// Schedule shared by the projections of one decode launch (n of them, sizes d_in[i] -> d_out[i], same storage type):
// cluster size, ring depths.  Returns false when the launch would not fit one wave of the GPU.
// *pair_out: the CTAs work as tcgen05 pairs (allow_pair, a token count that halves into multiples of 16, a mode that
// has the pair variant, and no fewer CTAs streaming than without).
static bool plan_decode_block(int n, const int* d_in, const int* d_out, int w0_dtype, int64_t T, int sm_count, bool allow_pair,
                              int* splits_out, int* w_stages_out, int* x_stages_out, int* m_tiles_total_out,
                              int* c_stages_out = nullptr, bool* pair_out = nullptr) {
  if (T <= 0 || T > kDecodeMaxTokens || n < 1 || n > kMaxBlockProj) return false;
  const int sm = sm_count > 0 ? sm_count : 148;
  const int tn = (int)((T + 15) / 16) * 16;
  int m_total = 0, m_pairs = 0, min_kb = 1 << 30;
  for (int i = 0; i < n; ++i) {
    const int m = (d_out[i] + DEC_M - 1) / DEC_M;
    m_total += m;
    m_pairs += (m + 1) / 2;  // an odd last tile is paired with an empty one
    if (d_in[i] / DEC_K < min_kb) min_kb = d_in[i] / DEC_K;
  }
  // cluster size: a power of two (packs into a GPC's SMs without stragglers), at most 8 (portable limit).
  // All clusters must be resident at once (the CTAs that add the rank term wait for rows other CTAs publish, and
  // a second wave would double the time anyway).  With one CTA per SM, clusters of 4 fill about 132 of 148 SMs
  // and clusters of 8 about 120 (they may not straddle GPCs).
  auto resident = [&](int c) { return c >= 8 ? sm * 120 / 148 : c >= 4 ? sm * 132 / 148 : sm; };
  if (n > 1 && m_total > resident(1)) return false;
  int splits = 1;
  while (splits * 2 <= 8 && m_total * splits * 2 <= resident(splits * 2) && splits * 2 <= min_kb) splits *= 2;
  const int mode = dec_mode(w0_dtype, tn);
  if (mode < 0) return false;
  // pairs: a cluster is 2 x splits CTAs
  bool pair = false;
  if (allow_pair && mode != kModeInt8Smem && tn % 32 == 0 && tn >= 64 && 2 * m_pairs <= resident(2)) {
    int ps = 1;
    while (ps * 4 <= 8 && 2 * m_pairs * ps * 2 <= resident(ps * 4) && ps * 2 <= min_kb) ps *= 2;
    if (2 * m_pairs * ps >= m_total * splits) {
      pair = true;
      splits = ps;
      m_total = 2 * m_pairs;
    }
  }
  // Ring depths.  Per K block the tensor core needs ~560 cycles; a tile load takes ~2500 (L2) to ~4000 (HBM)
  // cycles, so both rings want several tiles in flight: equal depth first, what is left goes to W0.
  // INT8 storage: W0 tiles travel as 8 KB of codes; a ring of converted bf16 tiles (which also takes the U_B slabs,
  // loaded into it directly) sits between the converting warps and the tensor core.
  const int c_stages = mode == kModeInt8Smem ? kInt8ConvStages : mode >= kModeInt8Tmem ? kTmemAStages : 0;
  const int w_slot = dec_w_slot(mode);
  const int x_rows = pair ? tn / 2 : tn;  // token rows of an x tile per CTA
  const int xb = x_rows * 128;
  const int budget = kDecSmemBudget - dec_smem_bytes(mode, 0, c_stages, 0, 0);
  int x_stages = budget / (w_slot + xb);
  if (x_stages > kMaxXStages) x_stages = kMaxXStages;
  if (x_stages < 1) return false;
  int w_stages = (budget - x_stages * xb) / w_slot;
  if (w_stages > kMaxWStages) w_stages = kMaxWStages;
  if (w_stages < 1) return false;
  // the receive buffer of the cluster reduction overlays the rings
  if (dec_ring_bytes(mode, w_stages, c_stages, x_stages, x_rows) < dec_recv_bytes(tn, splits)) return false;
  if (c_stages_out) *c_stages_out = c_stages;
  if (pair_out) *pair_out = pair;
  *splits_out = splits;
  *w_stages_out = w_stages;
  *x_stages_out = x_stages;
  *m_tiles_total_out = m_total;
  return true;
}

// Schedule of the decode kernel for one projection of T tokens; returns false when the call should use the prefill kernels.
bool plan_decode(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count, essa_plan* out) {
  (void)rank;
  const bool int8 = w0_dtype == ESSA_W0_INT8_PERCHANNEL;
  int splits, w_stages, x_stages, m_tiles;
  const int di = d_in, dout = d_out;
  bool pair = false;
  if (!plan_decode_block(1, &di, &dout, w0_dtype, T, sm_count, false, &splits, &w_stages, &x_stages, &m_tiles, nullptr, &pair)) return false;
  out->block_m = pair ? 2 * DEC_M : DEC_M;  // rows of W0 per MMA: one CTA's tile, or a pair's two
  out->block_n = (int)((T + 15) / 16) * 16;
  out->block_k = DEC_K;
  out->stages = w_stages;
  out->x_stages = x_stages;
  out->k_blocks = d_in / DEC_K + (int8 ? 2 : 1);
  out->splits = splits;
  out->tiles = m_tiles;
  out->grid = m_tiles * splits;
  out->down_splits = 0;
  out->down_grid = 0;
  out->scratch_bytes = 0;
  out->decode = 1;
  return true;
}

// One launch for n projections that share tokens, segments and the singular-value table.  Returns ESSA_OK, an
// error, or kBlockNotFused (> 0) when the block does not fit the one-wave decode schedule and the caller should
// issue the projections one by one.
int32_t launch_block_decode(essa_ctx* ctx, const BlockItem* items, int n, int64_t T, const int32_t* seg, int32_t P,
                            const float* sigma, int32_t ld_sigma, cudaStream_t stream, const uint32_t* sigma_ready,
                            uint32_t sigma_target, int set, int layer_mode) {
  if (n < 1 || n > kMaxBlockProj || T <= 0 || T > kDecodeMaxTokens) return kBlockNotFused;
  const int w0_dtype = items[0].a->w0_dtype;
  const bool int8 = w0_dtype == ESSA_W0_INT8_PERCHANNEL;
  int d_in[kMaxBlockProj], d_out[kMaxBlockProj];
  for (int i = 0; i < n; ++i) {
    if (items[i].a->w0_dtype != w0_dtype) return kBlockNotFused;
    d_in[i] = items[i].a->d_in;
    d_out[i] = items[i].a->d_out;
  }
  int splits, w_stages, x_stages, m_total, c_stages;
  bool pair = false;
  if (!plan_decode_block(n, d_in, d_out, w0_dtype, T, ctx->sm_count, ctx->decode_pairs, &splits, &w_stages, &x_stages, &m_total,
                         &c_stages, &pair)) {
    if (n > 1) return kBlockNotFused;
    return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: no decode schedule fits shared memory");
  }
  const int tn = (int)((T + 15) / 16) * 16;
  const int mode = dec_mode(w0_dtype, tn);
  if (mode < 0) return kBlockNotFused;
  const int csize = pair ? 2 * splits : splits;  // CTAs per cluster
  const int x_rows = pair ? tn / 2 : tn;         // token rows of an x tile per CTA

  // only CTAs of the first wave may be producers of u: ask the runtime how many clusters fit at once
  static int resident_caches[64][8][9] = {};  // per device, kernel instance, cluster size
  const int inst = mode * 2 + (pair ? 1 : 0);
  int* resident_cache = resident_caches[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0][inst];
  const void* kernel = mode == kModeBf16      ? (pair ? (const void*)essa_decode_kernel<kModeBf16, true> : (const void*)essa_decode_kernel<kModeBf16, false>)
                       : mode == kModeInt8Smem ? (const void*)essa_decode_kernel<kModeInt8Smem, false>
                       : mode == kModeInt8Tmem ? (pair ? (const void*)essa_decode_kernel<kModeInt8Tmem, true> : (const void*)essa_decode_kernel<kModeInt8Tmem, false>)
                                               : (pair ? (const void*)essa_decode_kernel<kModeInt4Tmem, true> : (const void*)essa_decode_kernel<kModeInt4Tmem, false>);
  const int threads = mode != kModeBf16 ? kDecThreadsInt8 : kDecThreads;
  {
    static bool attr_done[64][8] = {};  // the attribute is per device and kernel instance
    bool& done = attr_done[(ctx->device >= 0 && ctx->device < 64) ? ctx->device : 0][inst];
    if (!done) {
      const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kDecSmemBudget);
      if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(essa_decode_kernel)");
      done = true;
    }
  }
  if (resident_cache[csize] == 0) {
    cudaLaunchConfig_t q{};
    q.gridDim = dim3((unsigned)(148 * csize), 1, 1);
    q.blockDim = dim3((unsigned)threads, 1, 1);
    q.dynamicSmemBytes = (size_t)kDecSmemBudget;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = (unsigned)csize;
    qa[0].val.clusterDim.y = 1;
    qa[0].val.clusterDim.z = 1;
    q.attrs = qa;
    q.numAttrs = 1;
    int n_clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&n_clusters, kernel, &q) != cudaSuccess || n_clusters <= 0) {
      cudaGetLastError();
      n_clusters = 1;  // unknown: only the first cluster is certainly in the first wave
    }
    resident_cache[csize] = n_clusters;
  }
  const int resident_ctas = resident_cache[csize] * csize;
  const int main_ctas = m_total * splits;
  if (n > 1 && main_ctas > resident_ctas) return kBlockNotFused;
  // Launch a full wave: the CTAs beyond the W0-streaming ones only take finishing units of the rank path (groups
  // of 8 tokens).
  const int grid_total = main_ctas > resident_ctas ? main_ctas : resident_ctas;

  DBlock blk{};
  DMaps maps{};
  blk.n_proj = n;
  blk.sigma_ready = sigma_ready;
  blk.sigma_target = sigma_target;
  blk.layer_mode = layer_mode;
  blk.layers_flag = ctx->layers_flag;
  blk.layers_epoch = ctx->layers_epoch;
  blk.wait_limit = (long long)ctx->wait_limit_mcycles * 1000000LL;
  blk.set_done = ctx->dec_set_done + (set & 1);
  blk.set_wait_target = ctx->dec_set_issued[set & 1];
  blk.other_done = ctx->dec_set_done + ((set & 1) ^ 1);
  blk.other_wait_target = ctx->dec_set_issued[(set & 1) ^ 1];
  const int s0 = (set & 1) * kMaxBlockProj;  // first scratch slot of this launch
  blk.rank_ctas = grid_total < resident_ctas ? grid_total : resident_ctas;
  // CTAs of the wave beyond the W0-streaming ones take over the down-projection when there are at least four of them
  // (no CTA pairs: their x tiles are halves), at most one slot each, and their V_A^T ring fits below the x ring.
  {
    const int spare = grid_total - main_ctas;
    const int below_x = VAT_RING_BYTES + w_stages * dec_w_slot(mode) + (mode == kModeInt8Smem ? c_stages : mode >= kModeInt8Tmem ? kUbSlots : 0) * W_TILE_BYTES;
    blk.n_down = (!pair && spare >= 4 && below_x >= 8 * 8192 + W_TILE_BYTES && ctx->down_ctas) ? (spare < kMaxPSlices ? spare : kMaxPSlices) : 0;
  }
  int cta = 0, unit = 0;
  // The counters' next values are committed to the context only once the launch has been accepted: after a failed
  // call the device never reaches them, and a later call must not wait for rows nobody publishes.
  uint32_t next_pepoch[kMaxBlockProj] = {}, next_epoch[kMaxBlockProj] = {};
  for (int i = 0; i < n; ++i) {
    const essa_adapter* a = items[i].a;
    DParams& p = blk.proj[i];
    p.T = (int)T;
    p.tn = tn;
    p.xbox = x_rows;  // one box per tile (at most 256 rows)
    p.d_in = a->d_in;
    p.d_out = a->d_out;
    p.main_kb = a->d_in / DEC_K;
    p.m_tiles = (a->d_out + DEC_M - 1) / DEC_M;
    if (pair) p.m_tiles = (p.m_tiles + 1) / 2 * 2;  // CTAs come in pairs; a tile past d_out loads zeros and stores nothing
    p.splits = splits;
    p.w_stages = w_stages;
    p.x_stages = x_stages;
    p.c_stages = c_stages;
    p.ext = a->ext_blocks;
    p.y = items[i].y;
    p.ldy = a->d_out;
    p.scale = int8 ? a->w0_scale : nullptr;
    p.gscale = a->w0_gscale;
    p.r_pad = a->r_pad;
    p.rank_groups = ((int)T + kFinishTokens - 1) / kFinishTokens;
    // slices of the down-projection: the K blocks of a split are dealt to the first row tiles, p_c each, at most
    // kMaxPSlices slots per projection
    {
      const int nkb_max = (p.main_kb + splits - 1) / splits;
      int owners = kMaxPSlices / splits;  // per split
      const int owner_ctas = pair ? p.m_tiles / 2 : p.m_tiles;  // per split: a pair's leader owns a slice
      if (owners > owner_ctas) owners = owner_ctas;
      if (owners > 16) owners = 16;
      if (owners < 1) owners = 1;
      p.p_c = (nkb_max + owners - 1) / owners;
      p.p_per_split = (nkb_max + p.p_c - 1) / p.p_c;
      int delivered = 0;
      if (blk.n_down > 0) {  // one slot per down-projection CTA that gets a K block of this projection
        for (int c = 0; c < blk.n_down; ++c)
          delivered += ((long long)(c + 1) * p.main_kb) / blk.n_down > ((long long)c * p.main_kb) / blk.n_down ? 1 : 0;
      } else
      for (int sp = 0; sp < splits; ++sp) {
        const int nkb_s = p.main_kb / splits + (sp < p.main_kb % splits ? 1 : 0);
        delivered += (nkb_s + p.p_c - 1) / p.p_c;
      }
      p.p_count = ctx->dec_pcnt + s0 + i;
      next_pepoch[i] = ctx->dec_pepoch[s0 + i] + (uint32_t)delivered;
      p.p_target = next_pepoch[i];
    }
    p.p_part = static_cast<float*>(ctx->dec_ppart) + (size_t)(s0 + i) * kMaxPSlices * kDecodeMaxTokens * kRankPadMax;
    p.seg = seg;
    p.P = P;
    p.sigma = sigma;
    p.ld_sigma = ld_sigma;
    p.sA_col = items[i].sA_col;
    p.sB_col = items[i].sB_col;
    p.r = a->rank;
    p.M = a->M;
    p.u = static_cast<__nv_bfloat16*>(ctx->dec_u) + (size_t)(s0 + i) * kDecodeMaxTokens * kRankPadMax;
    p.u_count = ctx->dec_cnt + s0 + i;
    next_epoch[i] = ctx->dec_epoch[s0 + i] + (uint32_t)T;
    p.u_target = next_epoch[i] + (ctx->debug_stall_rank_rows ? 1u : 0u);  // (testing: a row nobody publishes)
    p.status = ctx->d_status;
    blk.cta_begin[i] = cta;
    blk.unit_begin[i] = unit;
    cta += p.m_tiles * splits;
    unit += p.rank_groups;

    maps.tm[i][0] = mode == kModeInt4Tmem ? a->tm_W0q4 : mode == kModeInt8Tmem ? a->tm_W0q64 : int8 ? a->tm_W0q : a->tm_W0[1];  // 128-row boxes of bf16 W0 / of codes
    // activation map: looked up by (pointer, tokens, features, box); u map: one per (projection slot, box)
    {
      essa_ctx::XMapEntry* hit = nullptr;
      for (auto& e : ctx->xmap_cache)
        if (e.ptr == items[i].x && e.T == T && e.d_in == a->d_in && e.box == (uint32_t)p.xbox) { hit = &e; break; }
      if (!hit) {
        essa_ctx::XMapEntry fresh;
        const int32_t st = make_tensor_map_2d(ctx, &fresh.tm, 0, items[i].x, (uint64_t)T, (uint64_t)a->d_in, (uint64_t)a->d_in * 2,
                                              (uint32_t)p.xbox, DEC_K, 128);
        if (st != ESSA_OK) return st;
        fresh.ptr = items[i].x; fresh.T = T; fresh.d_in = a->d_in; fresh.box = (uint32_t)p.xbox;
        hit = &ctx->xmap_cache[ctx->xmap_next];
        ctx->xmap_next = (ctx->xmap_next + 1) % 16;
        *hit = fresh;
      }
      maps.tm[i][1] = hit->tm;
      if (ctx->dec_u_map_box[s0 + i] != (uint32_t)p.xbox) {
        const int32_t st = make_tensor_map_2d(ctx, &ctx->dec_u_map[s0 + i], 0, p.u, (uint64_t)kDecodeMaxTokens, kRankPadMax,
                                              kRankPadMax * 2, (uint32_t)p.xbox, DEC_K, 128);
        if (st != ESSA_OK) return st;
        ctx->dec_u_map_box[s0 + i] = (uint32_t)p.xbox;
      }
      maps.tm[i][2] = ctx->dec_u_map[s0 + i];
    }
    maps.tm[i][3] = a->tm_UBp[1][0];  // 128-row boxes of the U_B slabs
    maps.tm[i][4] = a->tm_UBp[1][a->ext_blocks > 1 ? 1 : 0];
    maps.tm[i][5] = a->tm_VAt;
  }
  for (int i = n; i <= kMaxBlockProj; ++i) { blk.cta_begin[i] = cta; blk.unit_begin[i] = unit; }

  const int smem_bytes = dec_smem_bytes(mode, w_stages, c_stages, x_stages, x_rows);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)grid_total, 1, 1);
  cfg.blockDim = dim3((unsigned)threads, 1, 1);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)csize;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // see grid_dep_wait in the kernel
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  void* kargs[] = {(void*)&maps, (void*)&blk};
  const cudaError_t e = cudaLaunchKernelExC(&cfg, kernel, kargs);
  if (e != cudaSuccess) return check_cuda(ctx, e, "essa_decode_kernel launch");
  ctx->launches += 1;
  ctx->dec_set_issued[set & 1] += (uint32_t)grid_total;
  for (int i = 0; i < n; ++i) {
    ctx->dec_pepoch[s0 + i] = next_pepoch[i];
    ctx->dec_epoch[s0 + i] = next_epoch[i];
  }
  return ESSA_OK;
}

int32_t launch_projection_decode(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& g, const essa_plan& pl,
                                 cudaStream_t stream) {
  (void)pl;
  const BlockItem item{a, g.x, g.sA_col, g.sB_col, g.y};
  const int32_t st = launch_block_decode(ctx, &item, 1, g.T, g.seg_offsets, g.P, g.sigma, g.ld_sigma, stream);
  return st == kBlockNotFused ? fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "apply_projection: no decode schedule for this call") : st;
}

}  // namespace essa
