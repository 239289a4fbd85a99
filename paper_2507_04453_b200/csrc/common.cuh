// Internal declarations shared by the translation units of libessa.so (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <vector>

#include "essa.h"

namespace essa {

constexpr int kRankPadMax = 64;
constexpr int kDecSets = 2;  // decode scratch sets: consecutive blocks of a multi-layer call alternate between them
constexpr int kDecSlots = kDecSets * ESSA_MAX_BLOCK_ITEMS;
constexpr int kDecodeMaxTokens = 256;  // calls with at most this many tokens use the decode schedule (proj_decode.cu)  // rank-path operands are stored 64 columns wide (one 128-byte swizzle row)

// Device status word values are the ESSA_ERR_* codes; 0 = nothing recorded.
struct Scratch {
  void* ptr = nullptr;
  size_t bytes = 0;
};

}  // namespace essa

struct essa_ctx {
  int device = -1;
  int sm_count = 0;
  std::string last_error;
  int32_t* d_status = nullptr;  // device status word
  int64_t launches = 0;         // kernels of this library enqueued through this context
  int wait_limit_mcycles = 3000;  // ESSA_OPT_WAIT_LIMIT_MCYCLES
  bool debug_stall_rank_rows = false;  // ESSA_OPT_DEBUG_STALL_RANK_ROWS
  bool decode_pairs = false;  // ESSA_OPT_DECODE_PAIRS
  bool down_ctas = true;      // ESSA_OPT_DECODE_DOWN_CTAS
  bool pair_tiles = true;       // prefill base + up on 256 x 256 CTA-pair tiles (essa_set_option)
  int down_tile_units = 0;      // most 64-row units per tile of that kernel: 0 = automatic, 1..8 (essa_set_option)
  int down_pairs = 5;           // prefill rank-down step on CTA pairs: 0 = off, 1..5 = TMA-issuing threads per CTA (essa_set_option)
  int l2_hints = 13;            // L2 eviction hints of the wide prefill kernel's TMA copies (essa_set_option)
  int down_splits = 0;          // K split of the prefill rank-down launch: 0 = the planner's choice (essa_set_option)
  int wide_tiles = 1;           // ... on 512 x 256 pair tiles: 0 never, 1 where the planner's estimate favours them, 2 always
  int fuse_down = 0;            // ... which also compute the down-projection (no rank-down launch): 0 never (default),
                                // 1 in the token range where it measured faster, 2 whenever pair tiles are used
  essa::Scratch pair_ready;     // [token tiles][2] uint32: epoch of the last call that published u for (token tile, CTA rank)
  uint32_t pair_epoch = 0;      // epoch of the latest fused call (grows by one per call)
  // decode schedule: rank-path vector u of one call, [kDecodeMaxTokens][64] bf16, and the count of rows
  // published so far (monotonic across calls; dec_epoch is the host's copy of where the next call starts)
  void* dec_u = nullptr;
  uint32_t* dec_cnt = nullptr;
  uint32_t dec_epoch[essa::kDecSlots] = {};  // (one buffer / counter set per scratch set and projection of a block launch)
  void* dec_ppart = nullptr;    // [32][kDecodeMaxTokens][64] fp32 per projection: per-slice partial down-projections
  uint32_t* dec_pcnt = nullptr; // slices delivered so far, per projection (monotonic; dec_pepoch is the host's copy)
  uint32_t dec_pepoch[essa::kDecSlots] = {};
  uint32_t* dec_set_done = nullptr;  // [kDecSets] CTAs of decode launches on each scratch set that have finished (monotonic)
  uint32_t dec_set_issued[essa::kDecSets] = {};  // ... and how many have been launched (host count)
  uint32_t* layers_flag = nullptr;  // multi-layer calls: epoch of the latest call whose first block has seen its inputs complete
  uint32_t layers_epoch = 0;
  uint32_t* samp_cnt = nullptr; // blocks of fused population draws finished so far (monotonic; samp_epoch is the host's copy)
  uint32_t samp_epoch = 0;
  // Scratch owned by the context (grown on demand, never shrunk).
  essa::Scratch u_buf;        // [T_cap][64] bf16: rank-path vector u_t, zero-padded to 64 columns
  essa::Scratch splitk_ws;    // fp32 partial tiles for split-K (kept all-zero between calls)
  essa::Scratch splitk_cnt;   // int32 arrival counters, one per output tile (kept zero between calls)
  essa::Scratch simt_buf;     // [T_cap][64] fp32: rank-path vector of the CUDA-core cross-check path
  essa::Scratch stage_x, stage_y, stage_off, stage_sigma;  // device staging of the host-buffer entry point
  essa::Scratch w_deq;        // [d_out][d_in] bf16: INT8 W0 of the current prefill call, dequantised (unscaled) per call
  // host-buffer entry point: copy streams and per-chunk events of its three-stage pipeline (created on first use)
  cudaStream_t host_h2d = nullptr, host_d2h = nullptr;
  std::vector<cudaEvent_t> host_events;
  void* encode_tiled = nullptr;  // cuTensorMapEncodeTiled, resolved through the runtime
  // Calls that use the context's scratch buffers and counters are ordered on the device: when a call arrives on
  // another stream than the previous one, the new stream first waits for an event recorded on the old one.
  cudaStream_t last_stream = nullptr;
  bool last_stream_valid = false;
  cudaEvent_t order_event = nullptr;
  // decode launches: tensor maps of recently used activation buffers (encoding one costs about a microsecond and a
  // decode step is tens of microseconds), keyed by (pointer, tokens, features, box rows); round-robin replacement
  struct XMapEntry { const void* ptr = nullptr; int64_t T = 0; int32_t d_in = 0; uint32_t box = 0; CUtensorMap tm; };
  XMapEntry xmap_cache[16];
  int xmap_next = 0;
  CUtensorMap dec_u_map[essa::kDecSlots];           // maps of the decode u buffers (one box of tn rows)
  uint32_t dec_u_map_box[essa::kDecSlots] = {};
  // essa_profile_begin/end: three events per recorded call
  bool prof_on = false;
  int prof_calls = 0, prof_dropped = 0;
  std::vector<cudaEvent_t> prof_events;
};

struct essa_adapter {
  int d_in = 0, d_out = 0, rank = 0, r_pad = 0, w0_dtype = 0;
  void* W0 = nullptr;            // [d_out][d_in] bf16 (bf16 storage only)
  int8_t* W0q = nullptr;         // [d_out][d_in] int8 codes as given (INT8 storage only)
  __half* w0_scale = nullptr;    // [d_out] fp16 (INT8)
  __half* w0_gscale = nullptr;   // [d_out][d_in / 128] fp16 (INT4; W0q then holds two codes per byte, [d_out][d_in / 2])
  __nv_bfloat16* VAt = nullptr;  // [64][d_in]: V_A^T, rows >= rank are zero (K-major operand of the down-projection)
  __nv_bfloat16* UBp = nullptr;  // [ext][d_out][64]: U_B zero-padded to 64 columns; INT8: (U_B/scale) split hi, lo
  __nv_bfloat16* U_B = nullptr;  // [d_out][rank] as given (CUDA-core path)
  __nv_bfloat16* V_A = nullptr;  // [d_in][rank] as given (CUDA-core path)
  __nv_bfloat16* U_A = nullptr;  // [rank][rank] as given (candidate export)
  __nv_bfloat16* V_B = nullptr;  // [rank][rank] as given (candidate export)
  float* M = nullptr;            // [64][64] fp32: M = V_B^T U_A zero-padded
  int ext_blocks = 1;            // rank-path K-slabs appended to the base contraction (1 bf16, 2 INT8)
  CUtensorMap tm_W0[3];          // box rows 64 / 128 / 256 (bf16 storage only)
  CUtensorMap tm_UBp[3][2];
  CUtensorMap tm_VAt;
  CUtensorMap tm_VAtH;           // the same with boxes of r_pad / 2 rows (one CTA's half in the pair kernel)
  CUtensorMap tm_W0q;            // INT8 storage: the codes, 128-row x 64-byte boxes, unswizzled
  CUtensorMap tm_W0q64;          // ... the same boxes with the 64-byte swizzle (row-per-thread readers)
  CUtensorMap tm_W0q4;           // INT4 storage: the packed codes, 128-row x 32-byte boxes, 32-byte swizzle
};

namespace essa {

int32_t fail(essa_ctx* ctx, int32_t code, const std::string& msg);
int32_t check_cuda(essa_ctx* ctx, cudaError_t e, const char* what);
int32_t ensure_scratch(essa_ctx* ctx, Scratch& s, size_t bytes, bool zero, cudaStream_t stream);
void order_stream(essa_ctx* ctx, cudaStream_t stream);

// kind: 0 = bf16, 1 = uint8/int8.  rows x cols (cols contiguous), box = box_rows x box_cols, swizzle bytes in {0,32,64,128}.
int32_t make_tensor_map_2d(essa_ctx* ctx, CUtensorMap* out, int kind, const void* base, uint64_t rows, uint64_t cols,
                           uint64_t row_stride_bytes, uint32_t box_rows, uint32_t box_cols, int swizzle_bytes);

// sampler.cu
int32_t launch_sampler(essa_ctx* ctx, const float* mean, float step, const float* Bfactor, const float* Dvec, int32_t d,
                       uint64_t seed, int32_t k_begin, int32_t k_count, const int32_t* index, int32_t ld_out, float* sigma_out,
                       cudaStream_t stream, uint32_t* done = nullptr, uint32_t* blocks_out = nullptr,
                       const float* step_dev = nullptr);
int32_t launch_fill_rows(essa_ctx* ctx, const float* frozen, int32_t d, int32_t k_count, float* sigma_out, cudaStream_t stream);
int32_t launch_stream_words(essa_ctx* ctx, uint64_t seed, int32_t k_begin, int32_t k_count, int32_t n_blocks,
                            uint32_t* words_out, cudaStream_t stream);
int32_t launch_philox_once(essa_ctx* ctx, const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
int32_t launch_segment_map(essa_ctx* ctx, const int32_t* seg_offsets, int32_t P, int64_t T, int32_t* cand_out,
                           cudaStream_t stream);

// adapter_prep.cu
int32_t launch_widen_int8(essa_ctx* ctx, const int8_t* q, __nv_bfloat16* out, size_t count, cudaStream_t stream);
// INT4 group-wise storage -> bf16 weights (code * group scale, one rounding): out [d_out][d_in].
int32_t launch_widen_int4(essa_ctx* ctx, const uint8_t* packed, const __half* gscale, __nv_bfloat16* out, int d_out, int d_in,
                          cudaStream_t stream);
int32_t launch_adapter_prep(essa_ctx* ctx, essa_adapter* a, const __nv_bfloat16* U_A, const __nv_bfloat16* V_B,
                            cudaStream_t stream);
// Reconstructed factors of candidates k_begin .. k_begin + k_count - 1: A_out [k][rank][d_in], B_out [k][d_out][rank] bf16.
int32_t launch_export_candidates(essa_ctx* ctx, const essa_adapter* a, const float* sigma, int32_t ld_sigma, int32_t sA_col,
                                 int32_t sB_col, int32_t k_begin, int32_t k_count, __nv_bfloat16* A_out, __nv_bfloat16* B_out,
                                 cudaStream_t stream);

struct ProjArgs {
  const __nv_bfloat16* x;
  int64_t T;
  const int32_t* seg_offsets;
  int32_t P;
  const float* sigma;
  int32_t ld_sigma, sA_col, sB_col;
  __nv_bfloat16* y;
};

// proj_simt.cu / proj_tc.cu
int32_t launch_projection_simt(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& args, cudaStream_t stream);
int32_t launch_projection_tc(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& args, cudaStream_t stream);
int32_t launch_projection_tc_static(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& args, cudaStream_t stream);
void plan_projection(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count,
                     essa_plan* out);
// proj_tc2.cu
// `down` != nullptr: the launch also computes u (fused down-projection) instead of reading the rank-down launch's.
struct PairDown {
  int r_pad, r;
  const CUtensorMap* tmV;  // V_A^T with boxes of r_pad / 2 rows x 64 columns
  const int32_t* seg;
  int P;
  const float* sigma;
  int ld_sigma, sA_col, sB_col;
  const float* M;
  __nv_bfloat16* u;
  uint32_t* u_ready;
  uint32_t u_target;
};
int32_t launch_base_up_pair(essa_ctx* ctx, const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmA2,
                            const CUtensorMap& tmB2a, const CUtensorMap& tmB2b, int T, int d_out, int main_kb, int ext_kb,
                            int ext_ksteps, __nv_bfloat16* y, const __half* scale, const PairDown* down, cudaStream_t stream);
// proj_tc3.cu: base + up on 512-token x 256-channel pair tiles, up to kWideMaxJobs projections (same T) per launch
constexpr int kWideMaxJobs = 4;
struct WideJob {
  const CUtensorMap *tmA, *tmB, *tmA2, *tmB2a, *tmB2b;  // x, W0, u, U_B slab 0 / 1: boxes of 128 rows x 64 columns
  int d_out, main_kb, ext_kb, ext_ksteps;
  __nv_bfloat16* y;
  const __half* scale;
};
bool wide_tiles_pay(int64_t T, int d_out, int total_kb, int sm_count);
int32_t launch_base_up_wide(essa_ctx* ctx, const WideJob* jobs, int n_jobs, int T, cudaStream_t stream);
// proj_down.cu: the rank-down step of up to kWideMaxJobs projections (same T, same padded rank) in one CTA-pair launch
struct DownJob {
  const essa_adapter* a;
  const __nv_bfloat16* x;
  int32_t sA_col, sB_col;
  __nv_bfloat16* u;  // [T][64]
};
bool down_pairs_suit(const essa_ctx* ctx, const DownJob* jobs, int n_jobs, int64_t T);
int32_t launch_rank_down_pairs(essa_ctx* ctx, const DownJob* jobs, int n_jobs, int64_t T, const int32_t* seg, int32_t P,
                               const float* sigma, int32_t ld_sigma, cudaStream_t stream);
// proj_decode.cu
struct BlockItem {
  const essa_adapter* a;
  const __nv_bfloat16* x;
  int32_t sA_col, sB_col;
  __nv_bfloat16* y;
};
constexpr int32_t kBlockNotFused = 1;  // launch_block_decode: the block does not fit the one-wave decode schedule
// sigma_ready != NULL: the table is being written by the kernel launched just before on the same stream, which
// counts its finished blocks in *sigma_ready; the launch does not wait for that kernel as a whole, only (bounded)
// for the count to reach sigma_target before it reads the table.
// set: which of the context's decode scratch sets the launch uses.  layer_mode: 0 = a call of its own; 1 = first block
// of a multi-layer call (after its own wait for earlier work it publishes layers_epoch in the context's flag);
// 2 = later block of a multi-layer call (does not wait for the block before it, which it overlaps; waits, bounded,
// for that flag before it touches the activations and the table).
int32_t launch_block_decode(essa_ctx* ctx, const BlockItem* items, int n, int64_t T, const int32_t* seg, int32_t P,
                            const float* sigma, int32_t ld_sigma, cudaStream_t stream, const uint32_t* sigma_ready = nullptr,
                            uint32_t sigma_target = 0, int set = 0, int layer_mode = 0);
// proj_tc.cu: prefill-sized block: the projections' rank-down launches, then one wide-tile launch for all of them
// (kBlockNotFused if the block does not suit it).
int32_t launch_block_prefill(essa_ctx* ctx, const BlockItem* items, int n, int64_t T, const int32_t* seg, int32_t P,
                             const float* sigma, int32_t ld_sigma, cudaStream_t stream);
bool plan_decode(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count, essa_plan* out);
int32_t launch_projection_decode(essa_ctx* ctx, const essa_adapter* a, const ProjArgs& args, const essa_plan& plan,
                                 cudaStream_t stream);

#ifdef __CUDACC__
// Four INT8 codes (one 32-bit word) -> four bf16 values, exactly and without leaving the 16-bit lanes: for a code
// byte b, 0x4300 | (b & 0x7f) is the bf16 number 128 + low7(b) and 0x4300 | (b & 0x80) is 128 (b >= 0) or 256
// (b < 0); their difference low7(b) - 128 sign(b) is the code, and all three numbers fit bf16's eight significant
// bits, so the packed subtraction is exact.
__device__ __forceinline__ void int8x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
  const uint32_t s0 = __byte_perm(w, 0u, 0x4140);  // [b0, 0, b1, 0]
  const uint32_t s1 = __byte_perm(w, 0u, 0x4342);  // [b2, 0, b3, 0]
  const uint32_t p0 = (s0 & 0x007f007fu) | 0x43004300u, d0 = (s0 & 0x00800080u) | 0x43004300u;
  const uint32_t p1 = (s1 & 0x007f007fu) | 0x43004300u, d1 = (s1 & 0x00800080u) | 0x43004300u;
  const __nv_bfloat162 q0 = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&p0), *reinterpret_cast<const __nv_bfloat162*>(&d0));
  const __nv_bfloat162 q1 = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&p1), *reinterpret_cast<const __nv_bfloat162*>(&d1));
  lo = *reinterpret_cast<const uint32_t*>(&q0);
  hi = *reinterpret_cast<const uint32_t*>(&q1);
}

// Four packed INT4 bytes (eight codes, memory order: low nibble first) -> eight bf16 values = code * s, one rounding
// each.  A nibble n is the two's-complement code (n ^ 8) - 8.  The nibbles are biased four at a time with two wide
// masks; one byte permute then drops a biased nibble into the mantissa of 2^23 (0x4B000000 | (n ^ 8) is the fp32
// number 8388608 + (n ^ 8)), and subtracting 8388616 leaves the code exactly.  Its product with the fp16 group scale is
// exact in fp32 and rounded once when the pair is packed.  (Eleven integer-pipe instructions per eight codes; the
// first version, which built bf16 pairs with shifts and masks per byte and unpacked them again, took about twice as
// many: config 6a 103 -> 97 us per step.)
__device__ __forceinline__ void int4x8_to_bf16x8(uint32_t w, float s, uint32_t (&out)[4]) {
  const uint32_t lo8 = (w & 0x0f0f0f0fu) ^ 0x08080808u, hi8 = ((w >> 4) & 0x0f0f0f0fu) ^ 0x08080808u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float lo = __uint_as_float(__byte_perm(lo8, 0x4B000000u, 0x7440u | (uint32_t)j)) - 8388616.f;
    const float hi = __uint_as_float(__byte_perm(hi8, 0x4B000000u, 0x7440u | (uint32_t)j)) - 8388616.f;
    const __nv_bfloat162 r = __floats2bfloat162_rn(lo * s, hi * s);
    out[j] = *reinterpret_cast<const uint32_t*>(&r);
  }
}

// Largest k in [0, P-1] with off[k] <= t (candidate that owns token t; empty segments own nothing).
// Never reads outside off[0..P]; for offsets that are not monotone the result is some k in range.
__device__ __forceinline__ int find_candidate(const int32_t* __restrict__ off, int P, int t) {
  int lo = 0, hi = P;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (__ldg(off + mid) <= t) lo = mid; else hi = mid;
  }
  return lo;
}
#endif

}  // namespace essa
