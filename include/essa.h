/*
 * essa.h -- C ABI of the B200 (sm_100a) ESSA population-projection library.
 *
 * The library computes, for a whole CMA-ES population at once, the forward of the
 * SVD-reparameterised LoRA attention projections of ESSA (arXiv 2507.04453):
 *
 *   Section 3, "LoRA + SVD parameterization":  W0 in R^{m x n} frozen, update B A with
 *       A = U_A Sigma_A V_A^T (r x n),  B = U_B Sigma_B V_B^T (m x r), bases frozen;
 *   Algorithm 1, line 7:  candidate k uses  W'_k = W0 + U_B diag(sB_k) V_B^T U_A diag(sA_k) V_A^T;
 *   Section 3, "Evolutionary optimization" / Algorithm 1, line 5:  candidates are drawn from
 *       N(m, step^2 C) out of one shared random stream and are regenerable from a seed.
 *
 * The GPU path never materialises A'_k, B'_k or W'_k: with M = V_B^T U_A (r x r, computed once
 * per adapter) it evaluates   y_t = W0 x_t + U_B (sB_k .* (M (sA_k .* (V_A^T x_t)))),  k = cand(t).
 *
 * Conventions
 *   - C linkage, plain pointers and sizes.  "dev" = device pointer on the context's GPU,
 *     "host" = host pointer.  All matrices are row-major and dense unless a leading dimension
 *     is given.  bf16 = upper 16 bits of an IEEE fp32; fp16 = IEEE binary16.
 *   - Every call returns an int32 status: ESSA_OK (0) or a negative ESSA_ERR_* code; the text of
 *     the most recent error on a context is available from essa_last_error().
 *   - Work is enqueued on the caller's stream (a cudaStream_t passed as void*; NULL = the
 *     legacy default stream).  Calls do not synchronise unless stated.  The projection calls of
 *     one context share its scratch buffers and counters, so the library keeps them ordered on
 *     the device: a call that arrives on another stream than the context's previous projection
 *     call first makes its stream wait (an event) for that previous call.  Use one context per
 *     stream for calls that should overlap.
 *   - Ownership: the caller owns every pointer it passes.  essa_load_adapter copies what it
 *     needs into library-owned device memory (released by essa_free_adapter).  Device buffers
 *     passed to asynchronous calls must stay valid until the stream has executed the call.
 *   - Host-side validation happens before anything is launched.  Conditions only visible on
 *     the device (a bounded wait that expired) are recorded in a device status word that
 *     essa_get_status() reads; kernels never trap.
 *   - There is no CPU fallback: without a usable sm_100 device essa_create fails with
 *     ESSA_ERR_NO_DEVICE and nothing else can be called.
 */
#ifndef ESSA_H_
#define ESSA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ESSA_OK 0
#define ESSA_ERR_INVALID_ARG (-1)       /* null pointer, negative size, bad offsets, bad columns   */
#define ESSA_ERR_UNSUPPORTED_SHAPE (-2) /* a size outside what the kernels are built for           */
#define ESSA_ERR_ALLOC (-3)             /* device or host allocation failed                        */
#define ESSA_ERR_CUDA (-4)              /* a CUDA runtime/driver call returned an error            */
#define ESSA_ERR_DEVICE_TIMEOUT (-5)    /* a bounded device-side wait expired (see essa_get_status) */
#define ESSA_ERR_NO_DEVICE (-6)         /* no CUDA device, or not compute capability 10.x          */

#define ESSA_W0_BF16 0            /* W0 stored as bf16                                               */
#define ESSA_W0_INT8_PERCHANNEL 1 /* W0[o][i] = q[o][i] * scale[o], q int8, scale fp16 per out-channel */
#define ESSA_W0_INT4_GROUP128 2   /* W0[o][i] = q[o][i] * scale[o][i / 128], q a 4-bit two's-complement code in [-8, 7]:
                                     byte j of a row packs the codes of features 2j (low nibble) and 2j+1 (high
                                     nibble); scale fp16 per (out-channel, group of 128 input features).  The paper
                                     names the precision only (Section 5, precision study; the 72B runs); this
                                     storage scheme is the library's reading.  d_in must be a multiple of 128. */

#define ESSA_MAX_RANK 64
#define ESSA_MAX_BLOCK_ITEMS 4 /* projections one essa_apply_block call takes (q, k, v, o of an attention block) */
#define ESSA_STATIC_MAX_TOKENS 4096 /* largest T essa_apply_projection_static accepts */

typedef struct essa_ctx essa_ctx;         /* one per (process, device); not thread-safe */
typedef struct essa_adapter essa_adapter; /* one per adapted projection matrix          */

/* Library version (major*10000 + minor*100 + patch). Needs no device. */
int32_t essa_version(void);
/* Static description of a status code. Needs no device. */
const char* essa_status_string(int32_t status);

/* Create a context on CUDA device `device` (makes it current for the calling thread).
 * Fails with ESSA_ERR_NO_DEVICE if there is no such device or it is not sm_100-class. */
int32_t essa_create(essa_ctx** out, int32_t device);
/* Release the context's scratch memory. Adapters must have been freed before. Synchronises the device. */
int32_t essa_destroy(essa_ctx* ctx);
/* Text of the last error recorded on ctx (never NULL; "" if none). Valid until the next call on ctx. */
const char* essa_last_error(essa_ctx* ctx);
/* Synchronise the device, then read (and clear) the device status word: 0, or the ESSA_ERR_* code a
 * kernel recorded (ESSA_ERR_DEVICE_TIMEOUT if a bounded wait ran out; the affected output is undefined). */
int32_t essa_get_status(essa_ctx* ctx, int32_t* device_status);
/* Scheduling options of a context.
 *   ESSA_OPT_PAIR_TILES (0 / 1): run the base + up step of prefill-sized calls (T >= 512, 256-channel tiles) on
 *   256-token x 256-channel tiles shared by pairs of CTAs (tcgen05 cta_group::2) instead of 128 x 256 tiles per CTA.
 *   ESSA_OPT_FUSE_DOWN (0 / 1 / 2): on those pair tiles also compute the down-projection and the rank core inside
 *   the same launch (the tiles of the first channel column produce u for their token rows, the others wait for it),
 *   instead of a separate rank-down launch: 0 never (the default: the two-launch
 *   schedule measured within 0-3 % of it and has no waits between CTAs), 1 when the token count is in the range
 *   where it measured faster (about 14 K to 19 K tokens on 148 SMs), 2 whenever pair tiles are used.
 *   ESSA_OPT_PAIR_TILES defaults to 1. */
#define ESSA_OPT_PAIR_TILES 1
#define ESSA_OPT_FUSE_DOWN 2
/*   ESSA_OPT_WAIT_LIMIT_MCYCLES (1 .. 100000, default 3000): how long, in millions of SM cycles, the decode kernel's
 *   waits on counters that other thread blocks advance may last before the kernel gives up and records
 *   ESSA_ERR_DEVICE_TIMEOUT (the waits on its own copies and MMAs keep their fixed limit and end at once when a
 *   thread of the block has given up).
 *   ESSA_OPT_DEBUG_STALL_RANK_ROWS (0 / 1; for testing the give-up path without a fault): while set, a decode launch
 *   waits for one more row of the rank-path vector than the call publishes, so its up-projection never becomes
 *   ready, the wait runs out, the output is undefined and essa_get_status reports ESSA_ERR_DEVICE_TIMEOUT. */
#define ESSA_OPT_WAIT_LIMIT_MCYCLES 3
#define ESSA_OPT_DEBUG_STALL_RANK_ROWS 4
/*   ESSA_OPT_DECODE_PAIRS (0 / 1, default 0): run the decode kernel's CTAs as tcgen05 CTA pairs (two W0 row tiles per
 *   MMA of 256 rows, each CTA loading half of the token rows of x) when the token count is a multiple of 32.  The MMAs
 *   themselves are two to four times cheaper that way, but the pair's leader waits for both CTAs' operands before every
 *   K block and the launch measured 15 - 50 % SLOWER on B200 (config 3: 37 -> 44 us per step, config 5a: 129 -> 197 us),
 *   so it is off unless asked for. */
#define ESSA_OPT_DECODE_PAIRS 5
/*   ESSA_OPT_DECODE_DOWN_CTAS (0 / 1, default 1): when a decode launch has at least four thread blocks of its wave left
 *   over beyond the ones that stream W0, those compute the down-projection V_A^T x for the whole launch (x and V_A^T
 *   come from L2) instead of the first row tiles carrying slices of it on their K loops.  0 restores the slices. */
#define ESSA_OPT_DECODE_DOWN_CTAS 6
/*   ESSA_OPT_WIDE_TILES (0 / 1 / 2, default 1): prefill base + up launches use 512-token x 256-channel CTA-pair tiles
 *   (two accumulators per pair; the tensor cores run at their rate on that loop) where the planner's estimate puts
 *   them ahead of the 256 x 256 pair tiles (1), wherever the pair tiles would run (2), or never (0).  Both tile
 *   shapes add the K blocks in the same order in fp32. */
#define ESSA_OPT_WIDE_TILES 7
/*   ESSA_OPT_DOWN_SPLITS (0 .. 64, default 0): split of the K range of a prefill call's rank-down launch (each token
 *   tile's down-projection is shared by that many thread blocks, which add their fp32 partial sums in a workspace);
 *   0 leaves the choice to the planner, which balances the persistent grid's rounds. */
#define ESSA_OPT_DOWN_SPLITS 8
/*   ESSA_OPT_L2_HINTS (default 13): how the wide prefill kernel treats L2.  Bits 0-3:
 *   bit 0 = the W0 rows of a projection's leading channel tiles are loaded evict-last (as many tiles as fit ~21 MB: more
 *   than that thrashes), bit 1 = x / u loads evict-first (measured harmful: the pairs that share a token tile lose it),
 *   bit 2 = y stores evict-first, bit 3 = every other tile of a CTA pair walks K backwards, so that a round of the
 *   persistent grid starts with the K slabs the round before used last (the result's fp32 summation order then
 *   differs between tiles; it is the same from call to call).  Config 4's q projection reads 1404 MB from HBM with 0,
 *   990 with 8, 832 with 9, 797 with 13 (x and W0 are 415 MB).  Bits 8-15, if non-zero: the number of leading channel
 *   tiles to mark, instead of the 21 MB rule (for measurements). */
#define ESSA_OPT_L2_HINTS 9
/*   ESSA_OPT_DOWN_PAIRS (0 .. 5, default 5): the rank-down step of prefill-sized calls runs on CTA pairs (one launch for all
 *   projections of a block, token rows dealt to the pairs in 64-row units) where every pair gets at least four units and
 *   the rank is at most 32 (beyond that the single-CTA kernel measured faster);
 *   the value is the number of threads per CTA that issue its TMA copies in turn.  0 keeps one single-CTA launch of
 *   128-token tiles per projection. */
#define ESSA_OPT_DOWN_PAIRS 10
/*   ESSA_OPT_DOWN_TILE_UNITS (0 .. 8, default 0): the most 64-row units a tile of the CTA-pair rank-down kernel takes
 *   (up to 4: one accumulator per tile; 5 .. 8: two).  0 picks 8 where every pair gets at least twelve units and 4
 *   otherwise (for measurements). */
#define ESSA_OPT_DOWN_TILE_UNITS 11
int32_t essa_set_option(essa_ctx* ctx, int32_t option, int32_t value);
/* Number of kernels of this library enqueued through ctx since it was created (host counter). */
int32_t essa_get_launch_count(essa_ctx* ctx, int64_t* launches);
/* Pre-size the context's scratch memory (rank-path buffer, split-K workspace, host-call staging) for
 * up to max_tokens tokens and max_d_out output channels so that later calls do not allocate. */
int32_t essa_reserve(essa_ctx* ctx, int64_t max_tokens, int32_t max_d_in, int32_t max_d_out);

/* Pre-size the context's dequantisation scratch (d_in * d_out bf16) that prefill-sized calls on INT8-stored
 * adapters use, so that those calls do not allocate.  Needed before essa_apply_projection_static on such adapters. */
int32_t essa_reserve_dequant(essa_ctx* ctx, int32_t max_d_in, int32_t max_d_out);

/* Frozen data of one adapted projection (Section 3, "LoRA + SVD parameterization"). */
typedef struct essa_adapter_desc {
  int32_t d_in;     /* n: input features.  Must be a multiple of 64.                           */
  int32_t d_out;    /* m: output features. Must be a multiple of 8.                            */
  int32_t rank;     /* r: LoRA rank, 1..ESSA_MAX_RANK                                          */
  int32_t w0_dtype; /* ESSA_W0_BF16, ESSA_W0_INT8_PERCHANNEL or ESSA_W0_INT4_GROUP128          */
  const void* W0;       /* [d_out][d_in] bf16 or int8; INT4: [d_out][d_in / 2] bytes           */
  const void* w0_scale; /* INT8: [d_out] fp16; INT4: [d_out][d_in / 128] fp16; NULL for bf16   */
  const void* U_A;      /* [r][r]      bf16: left singular vectors of A                        */
  const void* V_A;      /* [d_in][r]   bf16: right singular vectors of A                       */
  const void* U_B;      /* [d_out][r]  bf16: left singular vectors of B                        */
  const void* V_B;      /* [r][r]      bf16: right singular vectors of B                       */
  int32_t on_device;    /* 0: the six pointers are host pointers; 1: device pointers           */
} essa_adapter_desc;

/* Copy and re-lay-out an adapter into library-owned device memory and precompute M = V_B^T U_A.
 * The bases are used as given (orthonormality is not assumed).  Asynchronous on `stream` when the
 * sources are device pointers (they must stay valid until the stream has passed the call); with host
 * pointers the call returns after the copies have completed.  INT8 storage: every scale must be
 * positive and finite (a zero scale would drop that channel's rank term together with its W0 row). */
int32_t essa_load_adapter(essa_ctx* ctx, const essa_adapter_desc* desc, essa_adapter** out, void* stream);
/* Free an adapter. Synchronises the device first. */
int32_t essa_free_adapter(essa_ctx* ctx, essa_adapter* adapter);

/* Draw a population (Section 3: x^(k) ~ N(m_t, sigma_t^2 C_t); Algorithm 1 line 5).
 *   sigma_out[k][i] = mean[i] + step * sum_j Bfactor[i][j] * Dvec[j] * z_k[j],   k = 0..P-1,
 * a sample of N(mean, step^2 * Bfactor diag(Dvec)^2 Bfactor^T).  z_k is a standard-normal vector
 * taken from the shared stream: Philox4x32-10 with key = (seed low word, seed high word) and counter
 * (j, k, 0, 0) yields four 32-bit words per block j; word w maps to u = (2*(w>>9)+1)*2^-24 and the
 * word pairs (0,1) and (2,3) give coordinates 4j..4j+3 by Box-Muller
 * (sqrt(-2 ln u0) * {cos, sin}(2 pi u1)).  A candidate therefore depends on <seed, k> only.
 * The transform and the sum run in fp64 on the device; each entry is rounded to fp32 once.
 *   mean    [d] fp32 dev;  Bfactor [d][d] fp32 dev, row-major, or NULL for identity;
 *   Dvec    [d] fp32 dev or NULL for ones;  sigma_out [P][d] fp32 dev (written).
 * d >= 1; with a non-NULL Bfactor d <= 4096.  P = 0 is a legal no-op. */
int32_t essa_sample_population(essa_ctx* ctx, const float* mean, float step, const float* Bfactor,
                               const float* Dvec, int32_t d, uint64_t seed, int32_t P, float* sigma_out,
                               void* stream);
/* Same, for candidates k_begin .. k_begin+k_count-1 only (row 0 of sigma_out is candidate k_begin):
 * what one worker of a candidate-sharded job regenerates locally. */
int32_t essa_sample_population_range(essa_ctx* ctx, const float* mean, float step, const float* Bfactor,
                                     const float* Dvec, int32_t d, uint64_t seed, int32_t k_begin,
                                     int32_t k_count, float* sigma_out, void* stream);

/* Search-distribution state and its update (Section 3, "Evolutionary optimization": CMA-ES samples the population from
 * N(m_t, sigma_t^2 C_t) and, once every candidate's reward is known, updates (m, sigma, C) from the reward ranking;
 * Algorithm 1: the common state (m_0, sigma_0, C_0) of its initialisation line and the CMA-ES update every worker
 * performs after the <seed, reward> exchange).  The paper prints no update formulas; the library implements the
 * (mu/mu_w, lambda)-CMA-ES of Hansen's tutorial with its default strategy parameters for (d, lambda), non-negative
 * recombination weights (mu = floor(lambda / 2)), c_m = 1, and a fresh decomposition C = B diag(D^2) B^T on every
 * update.  Rewards are MAXIMISED; ties keep population order; a NaN reward ranks last.
 * The state lives in device memory (fp64; the sampler reads fp32 copies of m, sigma, B, D), so
 * ask -> evaluate -> tell -> ask needs no host round trip.  d <= 1024, 2 <= lambda <= 65536. */
typedef struct essa_cma essa_cma;
/* m_0 = mean0 [d] fp32 HOST, sigma_0 = step0 > 0, C_0 = I, both evolution paths zero.  Synchronous. */
int32_t essa_cma_create(essa_ctx* ctx, int32_t d, int32_t lambda, const float* mean0_host, float step0, essa_cma** out);
/* Synchronises the device, then frees the state. */
int32_t essa_cma_destroy(essa_ctx* ctx, essa_cma* state);
/* essa_sample_population_range from the state: rows k_begin .. k_begin + k_count - 1 of the population
 * m + sigma B (D .* z_k), sigma_out [k_count][d] fp32 dev.  Asynchronous on `stream`. */
int32_t essa_cma_ask(essa_ctx* ctx, essa_cma* state, uint64_t seed, int32_t k_begin, int32_t k_count, float* sigma_out,
                     void* stream);
/* One update from a whole population: population [lambda][ld] fp32 dev (row k = candidate k as it was evaluated,
 * ld >= d), rewards [lambda] fp32 dev.  Steps, in the tutorial's order: rank; y_i = (x_i:lambda - m) / sigma for the mu
 * best; m += sigma sum w_i y_i; p_sigma with C^{-1/2} = B D^{-1} B^T; sigma; the stall indicator h_sigma; p_c; rank-one
 * and rank-mu update of C; decomposition (one-sided Jacobi rotations, at most 30 sweeps, eigenvalues ascending).
 * Asynchronous on `stream`: the launches are enqueued and the call returns (the number of Jacobi sweeps enqueued adapts to
 * convergence reports that arrive without blocking).  Calls on one state must be ordered by the caller (one stream). */
int32_t essa_tell(essa_ctx* ctx, essa_cma* state, const float* population, int32_t ld, const float* rewards, void* stream);
/* Overwrite parts of the state from HOST fp64 arrays (NULL = keep): mean [d], step [1], C [d][d] symmetric positive
 * definite (the decomposition is recomputed), p_sigma [d], p_c [d]; generation >= 0 sets the update counter.
 * Synchronises `stream` first. */
int32_t essa_cma_set(essa_ctx* ctx, essa_cma* state, const double* mean, const double* step, const double* C,
                     const double* p_sigma, const double* p_c, int32_t generation, void* stream);
/* Copy the state to HOST fp64 arrays (NULL = skip): mean [d], step [1], C [d][d], B [d][d] row-major (column j =
 * eigenvector j), D [d] ascending, p_sigma [d], p_c [d]; *generation = updates done; *sweeps = Jacobi sweeps the last
 * decomposition ran.  Synchronises the device. */
int32_t essa_cma_get(essa_ctx* ctx, essa_cma* state, double* mean, double* step, double* C, double* B, double* D,
                     double* p_sigma, double* p_c, int32_t* generation, int32_t* sweeps);
/* Strategy parameters in use: out9 = {mu, mu_eff, c_sigma, d_sigma, c_c, c_1, c_mu, c_m, E|N(0,I)|}.  Needs no device. */
int32_t essa_cma_params(essa_cma* state, double* out9);

/* Candidate reconstruction for hand-off to an external inference engine (Algorithm 1, line 7, as the paper's
 * workers do it: A'_k = U_A diag(sA_k) V_A^T, B'_k = U_B diag(sB_k) V_B^T, the engine then runs W0 + B'_k A'_k).
 * The projection entry points above never form these matrices; this call does, for candidates
 * k_begin .. k_begin + k_count - 1 of the table (row k of sigma is candidate k):
 *   A_out [k_count][rank][d_in] bf16 dev, B_out [k_count][d_out][rank] bf16 dev (either may be NULL to skip it);
 *   sigma [>= k_begin + k_count][ld_sigma] fp32 dev; sA_col / sB_col as in essa_apply_projection.
 * fp32 accumulation, one rounding to bf16.  k_count <= 65535 per call. */
int32_t essa_export_candidates(essa_ctx* ctx, const essa_adapter* adapter, const float* sigma, int32_t ld_sigma,
                               int32_t sA_col, int32_t sB_col, int32_t k_begin, int32_t k_count, void* A_out, void* B_out,
                               void* stream);

/* Top-alpha selection (Section 3, "LoRA + SVD parameterization": only the top-alpha fraction of the singular
 * values of each factor is exposed to the optimizer; the sensitivity study's caption fixes the rounding:
 * rank 8 with alpha = 0.1 rounds down to zero trainable values).  With alpha = alpha_num / alpha_den and a table
 * whose n_factors slices of `rank` columns follow one another, writes the columns of the
 * floor(alpha * rank) leading entries of every slice to index_out (host, ascending; may be NULL to ask for the
 * count only) and their number to *count_out.  Integer arithmetic: no rounding of alpha itself. */
int32_t essa_top_alpha_index(int32_t n_factors, int32_t rank, int32_t alpha_num, int32_t alpha_den, int32_t* index_out,
                             int32_t* count_out);
/* Draw a population when only d_t of the d coordinates are optimised (top-alpha selection):
 *   sigma_out[k][c] = frozen[c] for every column c, then for i < d_t
 *   sigma_out[k][index[i]] = mean_t[i] + step * sum_j Bfactor_t[i][j] * Dvec_t[j] * z_k[j],
 * with z_k the d_t-dimensional standard-normal vector of candidate k_begin + k from the shared stream (blocks of
 * four coordinates of the OPTIMISED vector, as in essa_sample_population).  d_t = 0 gives k_count copies of frozen.
 *   frozen [d] fp32 dev (the values the other coordinates keep, e.g. the singular values after SFT);
 *   index [d_t] int32 dev, distinct columns in [0, d) (entries outside the range are skipped);
 *   mean_t [d_t], Bfactor_t [d_t][d_t] or NULL, Dvec_t [d_t] or NULL: the search distribution over the optimised
 *   coordinates; sigma_out [k_count][d] fp32 dev (written). */
int32_t essa_sample_population_masked(essa_ctx* ctx, const float* frozen, const int32_t* index, const float* mean_t,
                                      float step, const float* Bfactor_t, const float* Dvec_t, int32_t d, int32_t d_t,
                                      uint64_t seed, int32_t k_begin, int32_t k_count, float* sigma_out, void* stream);

/* Population-batched adapted projection (Algorithm 1 line 7 applied to every candidate's tokens).
 *   x           [T][d_in] bf16 dev: all candidates' tokens stacked; token t belongs to the candidate
 *               k with seg_offsets[k] <= t < seg_offsets[k+1];
 *   seg_offsets [P+1] int32 dev, 0 = o[0] <= o[1] <= ... <= o[P] = T (empty segments allowed);
 *   sigma       [P][ld_sigma] fp32 dev: candidate k reads sA_k = sigma[k][sA_col .. sA_col+r) and
 *               sB_k = sigma[k][sB_col .. sB_col+r);
 *   y           [T][d_out] bf16 dev (written): y_t = W0 x_t + U_B (sB_k .* (M (sA_k .* (V_A^T x_t)))).
 * Accumulation is fp32 with one rounding to bf16 at the end; the rank-r intermediate is rounded to
 * bf16 once before the up-projection.  T = 0 is a legal no-op.  The offsets are read on the device
 * only: out-of-order offsets cannot cause out-of-bounds accesses but give unspecified candidates.
 * May grow the context's scratch memory (a synchronising allocation) unless essa_reserve covered it. */
int32_t essa_apply_projection(essa_ctx* ctx, const essa_adapter* adapter, const void* x, int64_t T,
                              const int32_t* seg_offsets, int32_t P, const float* sigma, int32_t ld_sigma,
                              int32_t sA_col, int32_t sB_col, void* y, void* stream);

/* Several adapted projections over the SAME tokens, segments and singular-value table in one call: the q, k, v, o
 * projections of an attention block ("Slice n" of Figure 1: one contiguous block of the table per LoRA matrix).
 * The result is what n_items calls of essa_apply_projection give (item i reads x_i, writes y_i, uses columns
 * sA_col_i / sB_col_i of the table).  At decode sizes (T <= 256, all items stored alike, W0 row tiles of the
 * whole block within one wave of the GPU) the block runs as ONE kernel launch, which is where the time of such
 * small calls goes; otherwise the items are issued one after the other.  1 <= n_items <= ESSA_MAX_BLOCK_ITEMS. */
typedef struct essa_block_item {
  const essa_adapter* adapter;
  const void* x;           /* [T][d_in] bf16 dev (items may share one x)  */
  int32_t sA_col, sB_col;  /* columns of this projection's sA / sB in the table */
  void* y;                 /* [T][d_out] bf16 dev (written)               */
} essa_block_item;
int32_t essa_apply_block(essa_ctx* ctx, const essa_block_item* items, int32_t n_items, int64_t T,
                         const int32_t* seg_offsets, int32_t P, const float* sigma, int32_t ld_sigma, void* stream);

/* The blocks of several layers in one call ("Slice n" of Figure 1: the table holds one contiguous slice of singular
 * values per LoRA matrix of every layer; the appendix's bookkeeping counts layers x 4 matrices x 2 r coordinates).
 * items holds n_layers x n_items entries, layer-major: items[l * n_items + i] is projection i of layer l with its own
 * adapter, activations x, output y and table columns; tokens, segments and the table are shared by all of them.  The
 * result is what n_layers calls of essa_apply_block give.  Every layer's activations are the caller's (whatever runs
 * between the projections of consecutive layers is outside this library), so they must all be final when the call is
 * made.  At decode sizes (T <= 256) each layer is one launch and the launches are chained WITHOUT waiting for one
 * another: a layer's thread blocks start wherever the layer before has released an SM, so launch gaps and the tail of
 * one layer overlap the weight streaming of the next; the launches still complete in order.  Larger calls, and layers
 * that do not fit the one-launch schedule, are issued like essa_apply_block. */
int32_t essa_apply_layers(essa_ctx* ctx, const essa_block_item* items, int32_t n_layers, int32_t n_items, int64_t T,
                          const int32_t* seg_offsets, int32_t P, const float* sigma, int32_t ld_sigma, void* stream);

/* Population draw and block projections in one call (Algorithm 1, lines 5 and 7, for the candidates this worker
 * evaluates): exactly essa_sample_population_range(mean, step, Bfactor, Dvec, d, seed, k_begin, P, sigma_out)
 * followed by essa_apply_block(items, n_items, T, seg_offsets, P, sigma_out, ld_sigma = d).  Because the library
 * itself enqueues the two kernels back to back, at decode sizes the block kernel does not wait for the draw to
 * finish: it streams W0 and the activations beside it, and only its rank path waits (bounded) until the draw
 * reports the table complete.  The activations, segment offsets and adapters must therefore be final when the call
 * is made (they may not be produced by work enqueued after it); sigma_out [P][d] is written and may be read by later
 * work on the stream as usual.  Results are identical to the two separate calls. */
int32_t essa_sample_apply_block(essa_ctx* ctx, const float* mean, float step, const float* Bfactor, const float* Dvec,
                                int32_t d, uint64_t seed, int32_t k_begin, int32_t P, float* sigma_out,
                                const essa_block_item* items, int32_t n_items, int64_t T, const int32_t* seg_offsets,
                                void* stream);

/* The same operation with HOST buffers: x, seg_offsets, sigma are copied to the device, the
 * projection runs, y is copied back, and the call returns after `stream` has been synchronised.
 * seg_offsets are validated on the host (ESSA_ERR_INVALID_ARG if not monotone from 0 to T).
 * Calls of 4096 tokens or more are cut into up to eight chunks of whole candidates (candidates are independent)
 * that run as a three-stage pipeline: copies in on one internal stream, projections on `stream`, copies out on
 * another, so both copy directions and the compute overlap.  Pinned host memory is what makes the copies
 * asynchronous; pageable memory works, serially. */
int32_t essa_apply_projection_host(essa_ctx* ctx, const essa_adapter* adapter, const void* x_host, int64_t T,
                                   const int32_t* seg_offsets_host, int32_t P, const float* sigma_host,
                                   int32_t ld_sigma, int32_t sA_col, int32_t sB_col, void* y_host,
                                   void* stream);
/* essa_apply_block with HOST buffers (Algorithm 1, line 7, for the projections of a block): items_host[i].x and
 * .y are host pointers, everything else as in essa_apply_projection_host.  At decode sizes the whole block is
 * copied in, runs as one essa_apply_block call and is copied out; larger blocks run the three-stage pipeline over
 * all (projection, chunk) units, so one projection's copy-out overlaps the next one's copy-in. */
int32_t essa_apply_block_host(essa_ctx* ctx, const essa_block_item* items_host, int32_t n_items, int64_t T,
                              const int32_t* seg_offsets_host, int32_t P, const float* sigma_host, int32_t ld_sigma,
                              void* stream);

/* (No counterpart in the paper: an engineering variant of essa_apply_projection.)
 * The same operation, same arguments and same result as essa_apply_projection, for callers that must not
 * allocate device memory when they call: code running while another allocator owns the GPU's memory budget,
 * or a latency-critical loop that cannot afford the implicit synchronisation of cudaMalloc / cudaFree.  This
 * entry point calls no cudaMalloc, cudaFree or any other allocating routine: its only scratch (the rank-path
 * vector u, 128 bytes per token) is a fixed array compiled into the library, ESSA_STATIC_MAX_TOKENS * 128 bytes
 * = 512 KB, which every GPU that loads the library holds until the process exits.  Split-K is off on this path,
 * so small token counts run on fewer SMs than essa_apply_projection would use.
 *   - T > ESSA_STATIC_MAX_TOKENS is rejected with ESSA_ERR_UNSUPPORTED_SHAPE (and a message in
 *     essa_last_error); use essa_apply_projection for larger batches.
 *   - The context's device must be the current device, else ESSA_ERR_INVALID_ARG.
 *   - Adapters stored as INT8 are dequantised per call into the context's dequantisation scratch; this entry
 *     point does not grow it and returns ESSA_ERR_ALLOC unless essa_reserve_dequant (or an earlier
 *     essa_apply_projection on an adapter at least as large) has sized it.
 *   - The first call on a device looks up the array's device address (cudaGetSymbolAddress); make that first
 *     call before any stream capture.
 *   - All calls, from every context and stream on that GPU, share the one array and it keeps the last call's
 *     contents.  Nothing in it needs clearing (each call overwrites every entry it later reads), but two calls
 *     that overlap on the GPU race on it: keep calls to this entry point ordered (one stream, or events). */
int32_t essa_apply_projection_static(essa_ctx* ctx, const essa_adapter* adapter, const void* x, int64_t T,
                                     const int32_t* seg_offsets, int32_t P, const float* sigma,
                                     int32_t ld_sigma, int32_t sA_col, int32_t sB_col, void* y, void* stream);

/* Straightforward CUDA-core (no tensor core, fp32 rank path) evaluation of the same formula, same
 * arguments as essa_apply_projection.  A cross-check for the tensor-core path at sizes the CPU
 * oracle cannot cover; never used by essa_apply_projection. */
int32_t essa_apply_projection_simt(essa_ctx* ctx, const essa_adapter* adapter, const void* x, int64_t T,
                                   const int32_t* seg_offsets, int32_t P, const float* sigma,
                                   int32_t ld_sigma, int32_t sA_col, int32_t sB_col, void* y, void* stream);

/* How essa_apply_projection would schedule a call (host-only arithmetic; needs no device). */
typedef struct essa_plan {
  int32_t block_m;       /* tokens per tile                                          */
  int32_t block_n;       /* output channels per tile                                 */
  int32_t block_k;       /* reduction elements per pipeline stage                    */
  int32_t stages;        /* shared-memory pipeline depth                             */
  int32_t k_blocks;      /* stages' worth of K per tile, including the rank-path slab */
  int32_t splits;        /* split-K factor (1 = none)                                */
  int32_t tiles;         /* output tiles (token tiles x channel tiles)               */
  int32_t grid;          /* CTAs launched by the main kernel                         */
  int32_t down_splits;   /* split-K factor of the rank-path down-projection kernel   */
  int32_t down_grid;     /* CTAs launched by the down-projection kernel              */
  int64_t scratch_bytes; /* device scratch the call needs                            */
  int32_t decode;        /* 1: decode schedule (one launch; block_m = W0 rows per CTA, block_n = tokens
                            per tile, stages = depth of the W0 ring, splits = CTAs of a cluster sharing
                            the reduction over d_in); 0: prefill */
  int32_t x_stages;      /* decode schedule: depth of the activation ring; 0 otherwise */
} essa_plan;
int32_t essa_plan_projection(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T,
                             int32_t sm_count, essa_plan* out);

/* Per-kernel device time of essa_apply_projection calls, for roofline reporting.  Between
 * essa_profile_begin and essa_profile_end every essa_apply_projection call records CUDA events on its
 * stream before, between and after its two kernel launches (up to max_calls calls; later ones are not
 * recorded).  essa_profile_end synchronises the device and sums the elapsed times per kernel. */
typedef struct essa_profile {
  double rank_down_ms;        /* total time of the rank-down kernel launches            */
  double base_up_ms;          /* total time of the base-contraction + up-projection launches */
  int32_t calls;              /* recorded calls (each = one launch of either kernel)    */
  int32_t dropped;            /* calls made while profiling that did not fit max_calls  */
} essa_profile;
int32_t essa_profile_begin(essa_ctx* ctx, int32_t max_calls);
int32_t essa_profile_end(essa_ctx* ctx, essa_profile* out);

/* Host-side check of segment offsets: 0 = o[0] <= ... <= o[P] = T. Needs no device. */
int32_t essa_validate_segments(const int32_t* seg_offsets_host, int32_t P, int64_t T);

/* Diagnostics for parity tests (all outputs are device buffers, asynchronous on `stream`). */
/* words_out[k_count][n_blocks][4] uint32: the raw Philox words of candidates k_begin.. (bit-exact check). */
int32_t essa_debug_stream_words(essa_ctx* ctx, uint64_t seed, int32_t k_begin, int32_t k_count,
                                int32_t n_blocks, uint32_t* words_out, void* stream);
/* One Philox4x32-10 block for an arbitrary counter and key (host in, host out; synchronous). */
int32_t essa_debug_philox(essa_ctx* ctx, const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);
/* cand_out[t] = candidate index the projection kernels derive for token t (device binary search). */
int32_t essa_debug_segment_map(essa_ctx* ctx, const int32_t* seg_offsets, int32_t P, int64_t T,
                               int32_t* cand_out, void* stream);
/* The adapter's precomputed core M = V_B^T U_A, copied to host as [r][r] fp32 (synchronous). */
int32_t essa_debug_core_matrix(essa_ctx* ctx, const essa_adapter* adapter, float* M_host);

#ifdef __cplusplus
}
#endif
#endif /* ESSA_H_ */
