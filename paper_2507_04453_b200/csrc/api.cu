// C ABI of libessa.so: contexts, adapters, argument validation, scratch memory, host-buffer entry point.
// The operations themselves live in sampler.cu (Section 3, "Evolutionary optimization"), proj_tc.cu and
// proj_simt.cu (Algorithm 1, line 7).
#include <cstdio>
#include <cstring>
#include <new>

#include "common.cuh"

namespace essa {

int32_t fail(essa_ctx* ctx, int32_t code, const std::string& msg) {
  if (ctx) ctx->last_error = msg;
  return code;
}

int32_t check_cuda(essa_ctx* ctx, cudaError_t e, const char* what) {
  if (e == cudaSuccess) return ESSA_OK;
  return fail(ctx, ESSA_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

int32_t ensure_scratch(essa_ctx* ctx, Scratch& s, size_t bytes, bool zero, cudaStream_t stream) {
  if (bytes <= s.bytes) return ESSA_OK;
  // Growing replaces the buffer: earlier work that may still use the old one must have finished.
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaDeviceSynchronize (scratch growth)");
  if (s.ptr) cudaFree(s.ptr);
  s.ptr = nullptr;
  s.bytes = 0;
  size_t cap = bytes + bytes / 4;
  cap = (cap + 255) & ~size_t(255);
  e = cudaMalloc(&s.ptr, cap);
  if (e != cudaSuccess) {
    cudaGetLastError();
    return fail(ctx, ESSA_ERR_ALLOC, std::string("cudaMalloc of scratch failed: ") + cudaGetErrorString(e));
  }
  s.bytes = cap;
  if (zero) {
    e = cudaMemsetAsync(s.ptr, 0, cap, stream);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemsetAsync (scratch)");
  }
  return ESSA_OK;
}

// Device-side ordering of calls that share the context's scratch: see essa_ctx::last_stream.
void order_stream(essa_ctx* ctx, cudaStream_t stream) {
  if (ctx->last_stream_valid && ctx->last_stream != stream) {
    if (!ctx->order_event && cudaEventCreateWithFlags(&ctx->order_event, cudaEventDisableTiming) != cudaSuccess) {
      cudaGetLastError();
      ctx->order_event = nullptr;
    }
    // (a stream the caller has destroyed in the meantime has no work left to wait for: errors are dropped)
    if (ctx->order_event && cudaEventRecord(ctx->order_event, ctx->last_stream) == cudaSuccess)
      cudaStreamWaitEvent(stream, ctx->order_event, 0);
    cudaGetLastError();
  }
  ctx->last_stream = stream;
  ctx->last_stream_valid = true;
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int32_t make_tensor_map_2d(essa_ctx* ctx, CUtensorMap* out, int kind, const void* base, uint64_t rows, uint64_t cols,
                           uint64_t row_stride_bytes, uint32_t box_rows, uint32_t box_cols, int swizzle_bytes) {
  if (!ctx->encode_tiled) return fail(ctx, ESSA_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  if ((reinterpret_cast<uintptr_t>(base) & 15) != 0 || (row_stride_bytes & 15) != 0)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "tensor base and row pitch must be 16-byte aligned");
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {row_stride_bytes};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                                : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                : swizzle_bytes == 32 ? CU_TENSOR_MAP_SWIZZLE_32B
                                                      : CU_TENSOR_MAP_SWIZZLE_NONE;
  const CUtensorMapDataType dt = kind == 0 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_UINT8;
  const CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled)(
      out, dt, 2, const_cast<void*>(base), gdim, gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw,
      CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    char buf[160];
    snprintf(buf, sizeof buf, "cuTensorMapEncodeTiled failed (CUresult %d) rows=%llu cols=%llu box=%ux%u", (int)r,
             (unsigned long long)rows, (unsigned long long)cols, box_rows, box_cols);
    return fail(ctx, ESSA_ERR_CUDA, buf);
  }
  return ESSA_OK;
}

namespace {

int32_t validate_projection_args(essa_ctx* ctx, const essa_adapter* a, const void* x, int64_t T, const int32_t* seg,
                                 int32_t P, const float* sigma, int32_t ld_sigma, int32_t sA_col, int32_t sB_col,
                                 const void* y) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!a) return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: adapter is NULL");
  if (T < 0 || P < 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: negative T or P");
  if (T == 0) return ESSA_OK;
  if (P == 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: T > 0 needs at least one candidate");
  if (!x || !seg || !sigma || !y) return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: NULL buffer");
  if (sA_col < 0 || sB_col < 0 || sA_col + a->rank > ld_sigma || sB_col + a->rank > ld_sigma)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: sigma columns outside the row (ld_sigma)");
  if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(y) & 15))
    return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_projection: x and y must be 16-byte aligned");
  return ESSA_OK;
}

void free_scratch(essa::Scratch& s) {
  if (s.ptr) cudaFree(s.ptr);
  s.ptr = nullptr;
  s.bytes = 0;
}

}  // namespace
}  // namespace essa

using namespace essa;

extern "C" {

int32_t essa_version(void) { return 100; }

const char* essa_status_string(int32_t status) {
  switch (status) {
    case ESSA_OK: return "ok";
    case ESSA_ERR_INVALID_ARG: return "invalid argument";
    case ESSA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case ESSA_ERR_ALLOC: return "allocation failed";
    case ESSA_ERR_CUDA: return "CUDA error";
    case ESSA_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case ESSA_ERR_NO_DEVICE: return "no usable sm_100 CUDA device";
    default: return "unknown status";
  }
}

int32_t essa_create(essa_ctx** out, int32_t device) {
  if (!out) return ESSA_ERR_INVALID_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || count <= 0 || device < 0 || device >= count) {
    cudaGetLastError();
    return ESSA_ERR_NO_DEVICE;
  }
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess || prop.major != 10) {
    cudaGetLastError();
    return ESSA_ERR_NO_DEVICE;
  }
  if (cudaSetDevice(device) != cudaSuccess) { cudaGetLastError(); return ESSA_ERR_NO_DEVICE; }
  essa_ctx* ctx = new (std::nothrow) essa_ctx();
  if (!ctx) return ESSA_ERR_ALLOC;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    ctx->encode_tiled = fn;
  else
    cudaGetLastError();
  if (cudaMalloc(&ctx->d_status, sizeof(int32_t)) != cudaSuccess || cudaMemset(ctx->d_status, 0, sizeof(int32_t)) != cudaSuccess ||
      cudaMalloc(&ctx->dec_u, (size_t)kDecSlots * kDecodeMaxTokens * kRankPadMax * 2) != cudaSuccess ||
      cudaMemset(ctx->dec_u, 0, (size_t)kDecSlots * kDecodeMaxTokens * kRankPadMax * 2) != cudaSuccess ||
      cudaMalloc(&ctx->dec_cnt, kDecSlots * sizeof(uint32_t)) != cudaSuccess ||
      cudaMemset(ctx->dec_cnt, 0, kDecSlots * sizeof(uint32_t)) != cudaSuccess ||
      cudaMalloc(&ctx->dec_ppart, (size_t)kDecSlots * 32 * kDecodeMaxTokens * kRankPadMax * 4) != cudaSuccess ||
      cudaMalloc(&ctx->dec_pcnt, kDecSlots * sizeof(uint32_t)) != cudaSuccess ||
      cudaMemset(ctx->dec_pcnt, 0, kDecSlots * sizeof(uint32_t)) != cudaSuccess ||
      cudaMalloc(&ctx->dec_set_done, kDecSets * sizeof(uint32_t)) != cudaSuccess ||
      cudaMemset(ctx->dec_set_done, 0, kDecSets * sizeof(uint32_t)) != cudaSuccess ||
      cudaMalloc(&ctx->layers_flag, sizeof(uint32_t)) != cudaSuccess || cudaMemset(ctx->layers_flag, 0, sizeof(uint32_t)) != cudaSuccess ||
      cudaMalloc(&ctx->samp_cnt, sizeof(uint32_t)) != cudaSuccess || cudaMemset(ctx->samp_cnt, 0, sizeof(uint32_t)) != cudaSuccess) {
    if (ctx->samp_cnt) cudaFree(ctx->samp_cnt);
    if (ctx->layers_flag) cudaFree(ctx->layers_flag);
    if (ctx->dec_set_done) cudaFree(ctx->dec_set_done);
    if (ctx->dec_ppart) cudaFree(ctx->dec_ppart);
    if (ctx->dec_pcnt) cudaFree(ctx->dec_pcnt);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->dec_u) cudaFree(ctx->dec_u);
    if (ctx->dec_cnt) cudaFree(ctx->dec_cnt);
    cudaGetLastError();
    delete ctx;
    return ESSA_ERR_ALLOC;
  }
  *out = ctx;
  return ESSA_OK;
}

int32_t essa_destroy(essa_ctx* ctx) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  cudaDeviceSynchronize();
  free_scratch(ctx->u_buf);
  free_scratch(ctx->splitk_ws);
  free_scratch(ctx->splitk_cnt);
  free_scratch(ctx->simt_buf);
  free_scratch(ctx->stage_x);
  free_scratch(ctx->stage_y);
  free_scratch(ctx->stage_off);
  free_scratch(ctx->stage_sigma);
  free_scratch(ctx->w_deq);
  free_scratch(ctx->pair_ready);
  for (cudaEvent_t e : ctx->prof_events) cudaEventDestroy(e);
  if (ctx->order_event) cudaEventDestroy(ctx->order_event);
  for (cudaEvent_t e : ctx->host_events) cudaEventDestroy(e);
  if (ctx->host_h2d) cudaStreamDestroy(ctx->host_h2d);
  if (ctx->host_d2h) cudaStreamDestroy(ctx->host_d2h);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->dec_u) cudaFree(ctx->dec_u);
  if (ctx->dec_cnt) cudaFree(ctx->dec_cnt);
  if (ctx->dec_ppart) cudaFree(ctx->dec_ppart);
  if (ctx->dec_pcnt) cudaFree(ctx->dec_pcnt);
  if (ctx->samp_cnt) cudaFree(ctx->samp_cnt);
  if (ctx->layers_flag) cudaFree(ctx->layers_flag);
  if (ctx->dec_set_done) cudaFree(ctx->dec_set_done);
  delete ctx;
  return ESSA_OK;
}

const char* essa_last_error(essa_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "context is NULL"; }

int32_t essa_get_status(essa_ctx* ctx, int32_t* device_status) {
  if (!ctx || !device_status) return ESSA_ERR_INVALID_ARG;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaDeviceSynchronize");
  e = cudaMemcpy(device_status, ctx->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpy(status)");
  if (*device_status != 0) {
    // A kernel gave up part-way: restore the invariants later calls rely on (zeroed split-K scratch).
    cudaMemset(ctx->d_status, 0, sizeof(int32_t));
    if (ctx->splitk_ws.ptr) cudaMemset(ctx->splitk_ws.ptr, 0, ctx->splitk_ws.bytes);
    if (ctx->splitk_cnt.ptr) cudaMemset(ctx->splitk_cnt.ptr, 0, ctx->splitk_cnt.bytes);
    cudaMemset(ctx->dec_cnt, 0, kDecSlots * sizeof(uint32_t));
    cudaMemset(ctx->dec_pcnt, 0, kDecSlots * sizeof(uint32_t));
    cudaMemset(ctx->layers_flag, 0, sizeof(uint32_t));
    cudaMemset(ctx->dec_set_done, 0, kDecSets * sizeof(uint32_t));
    for (uint32_t& e : ctx->dec_set_issued) e = 0;
    ctx->layers_epoch = 0;
    for (uint32_t& e : ctx->dec_epoch) e = 0;
    for (uint32_t& e : ctx->dec_pepoch) e = 0;
    cudaMemset(ctx->samp_cnt, 0, sizeof(uint32_t));
    ctx->samp_epoch = 0;
    if (ctx->pair_ready.ptr) cudaMemset(ctx->pair_ready.ptr, 0, ctx->pair_ready.bytes);
    ctx->pair_epoch = 0;
  }
  return ESSA_OK;
}

int32_t essa_set_option(essa_ctx* ctx, int32_t option, int32_t value) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  switch (option) {
    case ESSA_OPT_PAIR_TILES: ctx->pair_tiles = value != 0; return ESSA_OK;
    case ESSA_OPT_FUSE_DOWN:
      if (value < 0 || value > 2) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_FUSE_DOWN takes 0, 1 or 2");
      ctx->fuse_down = value;
      return ESSA_OK;
    case ESSA_OPT_WAIT_LIMIT_MCYCLES:
      if (value < 1 || value > 100000) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_WAIT_LIMIT_MCYCLES takes 1 .. 100000");
      ctx->wait_limit_mcycles = value;
      return ESSA_OK;
    case ESSA_OPT_DEBUG_STALL_RANK_ROWS: ctx->debug_stall_rank_rows = value != 0; return ESSA_OK;
    case ESSA_OPT_DECODE_PAIRS: ctx->decode_pairs = value != 0; return ESSA_OK;
    case ESSA_OPT_DECODE_DOWN_CTAS: ctx->down_ctas = value != 0; return ESSA_OK;
    case ESSA_OPT_DOWN_SPLITS:
      if (value < 0 || value > 64) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_DOWN_SPLITS takes 0 .. 64");
      ctx->down_splits = value;
      return ESSA_OK;
    case ESSA_OPT_DOWN_PAIRS:
      if (value < 0 || value > 5) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_DOWN_PAIRS takes 0 .. 5");
      ctx->down_pairs = value;
      return ESSA_OK;
    case ESSA_OPT_DOWN_TILE_UNITS:
      if (value < 0 || value > 8) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_DOWN_TILE_UNITS takes 0 .. 8");
      ctx->down_tile_units = value;
      return ESSA_OK;
    case ESSA_OPT_L2_HINTS:
      if (value < 0 || value > 0xffff) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_L2_HINTS takes 0 .. 65535");
      ctx->l2_hints = value;
      return ESSA_OK;
    case ESSA_OPT_WIDE_TILES:
      if (value < 0 || value > 2) return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: ESSA_OPT_WIDE_TILES takes 0, 1 or 2");
      ctx->wide_tiles = value;
      return ESSA_OK;
    default: return fail(ctx, ESSA_ERR_INVALID_ARG, "set_option: unknown option");
  }
}

int32_t essa_get_launch_count(essa_ctx* ctx, int64_t* launches) {
  if (!ctx || !launches) return ESSA_ERR_INVALID_ARG;
  *launches = ctx->launches;
  return ESSA_OK;
}

int32_t essa_reserve(essa_ctx* ctx, int64_t max_tokens, int32_t max_d_in, int32_t max_d_out) {
  if (!ctx || max_tokens < 0 || max_d_in < 0 || max_d_out < 0) return ESSA_ERR_INVALID_ARG;
  // one rank-path vector per projection of a block (a prefill-sized block call keeps all of them at once)
  int32_t st = ensure_scratch(ctx, ctx->u_buf, (size_t)ESSA_MAX_BLOCK_ITEMS * ((size_t)max_tokens * kRankPadMax * 2 + 256), false, nullptr);
  if (st != ESSA_OK) return st;
  // split-K is only used while there are fewer tiles than SMs: at most sm_count tiles of 128 x 256 fp32
  // ... and by the rank-down launch, whose K range may be split at any token count: 128 x 64 fp32 per token tile
  const size_t m_tiles = (size_t)((max_tokens + 127) / 128);
  const size_t ws_tc = (size_t)ctx->sm_count * 128 * 256 * 4, ws_down = m_tiles * 128 * kRankPadMax * 4;
  st = ensure_scratch(ctx, ctx->splitk_ws, ws_tc > ws_down ? ws_tc : ws_down, true, nullptr);
  if (st != ESSA_OK) return st;
  const size_t cnt_tc = (size_t)ctx->sm_count * 4 * 4, cnt_down = m_tiles * 4;
  st = ensure_scratch(ctx, ctx->splitk_cnt, cnt_tc > cnt_down ? cnt_tc : cnt_down, true, nullptr);
  if (st != ESSA_OK) return st;
  st = ensure_scratch(ctx, ctx->stage_x, (size_t)max_tokens * max_d_in * 2, false, nullptr);
  if (st != ESSA_OK) return st;
  st = ensure_scratch(ctx, ctx->stage_y, (size_t)max_tokens * max_d_out * 2, false, nullptr);
  if (st != ESSA_OK) return st;
  return check_cuda(ctx, cudaDeviceSynchronize(), "cudaDeviceSynchronize");
}

int32_t essa_reserve_dequant(essa_ctx* ctx, int32_t max_d_in, int32_t max_d_out) {
  if (!ctx || max_d_in < 0 || max_d_out < 0) return ESSA_ERR_INVALID_ARG;
  const int32_t st = ensure_scratch(ctx, ctx->w_deq, (size_t)max_d_in * max_d_out * 2, false, nullptr);
  if (st != ESSA_OK) return st;
  return check_cuda(ctx, cudaDeviceSynchronize(), "cudaDeviceSynchronize");
}

int32_t essa_load_adapter(essa_ctx* ctx, const essa_adapter_desc* d, essa_adapter** out, void* stream_v) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!d || !out) return fail(ctx, ESSA_ERR_INVALID_ARG, "load_adapter: NULL descriptor or output");
  *out = nullptr;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  if (d->d_in <= 0 || d->d_out <= 0 || d->rank <= 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "load_adapter: sizes must be positive");
  if (d->rank > ESSA_MAX_RANK) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "load_adapter: rank > 64");
  if (d->d_in % 64 != 0) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "load_adapter: d_in must be a multiple of 64");
  if (d->d_out % 8 != 0) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "load_adapter: d_out must be a multiple of 8");
  if (d->w0_dtype != ESSA_W0_BF16 && d->w0_dtype != ESSA_W0_INT8_PERCHANNEL && d->w0_dtype != ESSA_W0_INT4_GROUP128)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "load_adapter: unknown w0_dtype");
  if (!d->W0 || !d->U_A || !d->V_A || !d->U_B || !d->V_B) return fail(ctx, ESSA_ERR_INVALID_ARG, "load_adapter: NULL matrix");
  const bool int8 = d->w0_dtype == ESSA_W0_INT8_PERCHANNEL;
  const bool int4 = d->w0_dtype == ESSA_W0_INT4_GROUP128;
  if ((int8 || int4) && !d->w0_scale) return fail(ctx, ESSA_ERR_INVALID_ARG, "load_adapter: quantised W0 needs w0_scale");
  if (int4 && d->d_in % 128 != 0) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "load_adapter: INT4 storage needs d_in to be a multiple of 128");

  essa_adapter* a = new (std::nothrow) essa_adapter();
  if (!a) return fail(ctx, ESSA_ERR_ALLOC, "load_adapter: host allocation failed");
  a->d_in = d->d_in; a->d_out = d->d_out; a->rank = d->rank; a->w0_dtype = d->w0_dtype;
  a->r_pad = ((d->rank + 15) / 16) * 16;
  a->ext_blocks = int8 ? 2 : 1;
  const size_t n = d->d_in, m = d->d_out, r = d->rank;
  // INT8 weights stay stored as codes (1 byte per weight).  The decode kernel converts them to bf16 in shared
  // memory; a prefill call dequantises them once into the context's scratch before its GEMM.  Either way the fp16
  // per-channel scale is applied to the fp32 accumulator, so the dequantisation is exact.
  const size_t w0_bytes = m * n * 2;
  cudaError_t e = cudaSuccess;
  auto alloc = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
  if (!int8 && !int4) alloc(&a->W0, w0_bytes);
  if (int8) { alloc((void**)&a->w0_scale, m * 2); alloc((void**)&a->W0q, m * n); }
  if (int4) { alloc((void**)&a->w0_gscale, m * (n / 128) * 2); alloc((void**)&a->W0q, m * n / 2); }
  alloc((void**)&a->VAt, (size_t)kRankPadMax * n * 2);
  alloc((void**)&a->UBp, (size_t)a->ext_blocks * m * kRankPadMax * 2);
  alloc((void**)&a->U_B, m * r * 2);
  alloc((void**)&a->V_A, n * r * 2);
  alloc((void**)&a->M, (size_t)kRankPadMax * kRankPadMax * 4);
  alloc((void**)&a->U_A, r * r * 2);
  alloc((void**)&a->V_B, r * r * 2);
  int32_t st = ESSA_OK;
  if (e != cudaSuccess) {
    cudaGetLastError();
    st = fail(ctx, ESSA_ERR_ALLOC, std::string("load_adapter: cudaMalloc failed: ") + cudaGetErrorString(e));
  }
  const cudaMemcpyKind kind = d->on_device ? cudaMemcpyDeviceToDevice : cudaMemcpyHostToDevice;
  auto copy = [&](void* dst, const void* src, size_t bytes) {
    if (st == ESSA_OK) st = check_cuda(ctx, cudaMemcpyAsync(dst, src, bytes, kind, stream), "load_adapter: copy");
  };
  copy((int8 || int4) ? (void*)a->W0q : a->W0, d->W0, int8 ? m * n : int4 ? m * n / 2 : w0_bytes);
  if (int8) copy(a->w0_scale, d->w0_scale, m * 2);
  if (int4) copy(a->w0_gscale, d->w0_scale, m * (n / 128) * 2);
  copy(a->U_B, d->U_B, m * r * 2);
  copy(a->V_A, d->V_A, n * r * 2);
  copy(a->U_A, d->U_A, r * r * 2);
  copy(a->V_B, d->V_B, r * r * 2);
  if (st == ESSA_OK) st = launch_adapter_prep(ctx, a, a->U_A, a->V_B, stream);
  if (st == ESSA_OK) {
    const uint32_t rows[3] = {64, 128, 256};
    for (int i = 0; i < 3 && st == ESSA_OK; ++i) {
      if (!int8 && !int4) st = make_tensor_map_2d(ctx, &a->tm_W0[i], 0, a->W0, m, n, n * 2, rows[i], 64, 128);
      for (int e2 = 0; e2 < a->ext_blocks && st == ESSA_OK; ++e2)
        st = make_tensor_map_2d(ctx, &a->tm_UBp[i][e2], 0, a->UBp + (size_t)e2 * m * kRankPadMax, m, kRankPadMax,
                                kRankPadMax * 2, rows[i], 64, 128);
    }
    if (st == ESSA_OK && int8) st = make_tensor_map_2d(ctx, &a->tm_W0q, 1, a->W0q, m, n, n, 128, 64, 0);
    if (st == ESSA_OK && int8) st = make_tensor_map_2d(ctx, &a->tm_W0q64, 1, a->W0q, m, n, n, 128, 64, 64);
    if (st == ESSA_OK && int4) st = make_tensor_map_2d(ctx, &a->tm_W0q4, 1, a->W0q, m, n / 2, n / 2, 128, 32, 32);
    if (st == ESSA_OK) st = make_tensor_map_2d(ctx, &a->tm_VAt, 0, a->VAt, kRankPadMax, n, n * 2, a->r_pad, 64, 128);
    if (st == ESSA_OK) st = make_tensor_map_2d(ctx, &a->tm_VAtH, 0, a->VAt, kRankPadMax, n, n * 2, a->r_pad / 2, 64, 128);
  }
  // With host sources the caller's buffers are only needed until the copies have run; device sources stay
  // asynchronous (the caller keeps them valid until the stream has passed this call).
  if (!d->on_device && cudaStreamSynchronize(stream) != cudaSuccess && st == ESSA_OK)
    st = check_cuda(ctx, cudaGetLastError(), "load_adapter: sync");
  if (st != ESSA_OK) {
    essa_free_adapter(ctx, a);
    return st;
  }
  *out = a;
  return ESSA_OK;
}

int32_t essa_free_adapter(essa_ctx* ctx, essa_adapter* a) {
  if (!ctx || !a) return ESSA_ERR_INVALID_ARG;
  cudaDeviceSynchronize();
  void* ptrs[] = {a->W0, a->W0q, a->w0_scale, a->w0_gscale, a->VAt, a->UBp, a->U_B, a->V_A, a->U_A, a->V_B, a->M};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  delete a;
  return ESSA_OK;
}

static int32_t validate_sampler(essa_ctx* ctx, const float* mean, int32_t d, int32_t k_begin, int32_t k_count,
                                const float* sigma_out) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (d <= 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population: d must be positive");
  if (k_count < 0 || k_begin < 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population: negative candidate range");
  if ((int64_t)k_begin + k_count > 0x7fffffffLL) return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population: candidate index overflow");
  if (k_count > 0 && (!mean || !sigma_out)) return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population: NULL buffer");
  return ESSA_OK;
}

int32_t essa_sample_population(essa_ctx* ctx, const float* mean, float step, const float* Bfactor, const float* Dvec,
                               int32_t d, uint64_t seed, int32_t P, float* sigma_out, void* stream) {
  const int32_t st = validate_sampler(ctx, mean, d, 0, P, sigma_out);
  if (st != ESSA_OK) return st;
  return launch_sampler(ctx, mean, step, Bfactor, Dvec, d, seed, 0, P, nullptr, d, sigma_out, static_cast<cudaStream_t>(stream));
}

int32_t essa_sample_population_range(essa_ctx* ctx, const float* mean, float step, const float* Bfactor,
                                     const float* Dvec, int32_t d, uint64_t seed, int32_t k_begin, int32_t k_count,
                                     float* sigma_out, void* stream) {
  const int32_t st = validate_sampler(ctx, mean, d, k_begin, k_count, sigma_out);
  if (st != ESSA_OK) return st;
  return launch_sampler(ctx, mean, step, Bfactor, Dvec, d, seed, k_begin, k_count, nullptr, d, sigma_out,
                        static_cast<cudaStream_t>(stream));
}

int32_t essa_export_candidates(essa_ctx* ctx, const essa_adapter* a, const float* sigma, int32_t ld_sigma, int32_t sA_col,
                               int32_t sB_col, int32_t k_begin, int32_t k_count, void* A_out, void* B_out, void* stream) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!a) return fail(ctx, ESSA_ERR_INVALID_ARG, "export_candidates: adapter is NULL");
  if (k_begin < 0 || k_count < 0) return fail(ctx, ESSA_ERR_INVALID_ARG, "export_candidates: negative candidate range");
  if (k_count == 0) return ESSA_OK;
  if (!sigma || (!A_out && !B_out)) return fail(ctx, ESSA_ERR_INVALID_ARG, "export_candidates: NULL buffer");
  if (sA_col < 0 || sB_col < 0 || sA_col + a->rank > ld_sigma || sB_col + a->rank > ld_sigma)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "export_candidates: sigma columns outside the row");
  if (k_count > 65535) return fail(ctx, ESSA_ERR_UNSUPPORTED_SHAPE, "export_candidates: more than 65535 candidates in one call");
  return launch_export_candidates(ctx, a, sigma, ld_sigma, sA_col, sB_col, k_begin, k_count, static_cast<__nv_bfloat16*>(A_out),
                                  static_cast<__nv_bfloat16*>(B_out), static_cast<cudaStream_t>(stream));
}

int32_t essa_top_alpha_index(int32_t n_factors, int32_t rank, int32_t alpha_num, int32_t alpha_den, int32_t* index_out,
                             int32_t* count_out) {
  if (n_factors < 0 || rank < 1 || alpha_den < 1 || alpha_num < 0 || alpha_num > alpha_den || !count_out) return ESSA_ERR_INVALID_ARG;
  const int32_t per = (int32_t)(((int64_t)alpha_num * rank) / alpha_den);  // floor(alpha * rank), exactly
  *count_out = n_factors * per;
  if (index_out)
    for (int32_t f = 0; f < n_factors; ++f)
      for (int32_t j = 0; j < per; ++j) index_out[(size_t)f * per + j] = f * rank + j;
  return ESSA_OK;
}

int32_t essa_sample_population_masked(essa_ctx* ctx, const float* frozen, const int32_t* index, const float* mean_t, float step,
                                      const float* Bfactor_t, const float* Dvec_t, int32_t d, int32_t d_t, uint64_t seed,
                                      int32_t k_begin, int32_t k_count, float* sigma_out, void* stream_v) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (d < 1 || d_t < 0 || d_t > d || k_begin < 0 || k_count < 0)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population_masked: need 0 <= d_t <= d, d >= 1, k_begin >= 0, k_count >= 0");
  if (k_count == 0) return ESSA_OK;
  if (!frozen || !sigma_out || (d_t > 0 && (!index || !mean_t)))
    return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_population_masked: NULL buffer");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  const int32_t st = launch_fill_rows(ctx, frozen, d, k_count, sigma_out, stream);
  if (st != ESSA_OK || d_t == 0) return st;
  return launch_sampler(ctx, mean_t, step, Bfactor_t, Dvec_t, d_t, seed, k_begin, k_count, index, d, sigma_out, stream);
}

int32_t essa_apply_projection(essa_ctx* ctx, const essa_adapter* a, const void* x, int64_t T, const int32_t* seg,
                              int32_t P, const float* sigma, int32_t ld_sigma, int32_t sA_col, int32_t sB_col, void* y,
                              void* stream) {
  const int32_t st = validate_projection_args(ctx, a, x, T, seg, P, sigma, ld_sigma, sA_col, sB_col, y);
  if (st != ESSA_OK || T == 0) return st;
  ProjArgs g{static_cast<const __nv_bfloat16*>(x), T, seg, P, sigma, ld_sigma, sA_col, sB_col, static_cast<__nv_bfloat16*>(y)};
  order_stream(ctx, static_cast<cudaStream_t>(stream));
  return launch_projection_tc(ctx, a, g, static_cast<cudaStream_t>(stream));
}

// essa_apply_block, optionally right behind a population draw that is still running (sigma_ready: see
// launch_block_decode; honoured only by the one-launch decode schedule, the other schedules are ordered behind the
// draw by the stream).
static int32_t apply_block_impl(essa_ctx* ctx, const essa_block_item* items, int32_t n_items, int64_t T, const int32_t* seg,
                                int32_t P, const float* sigma, int32_t ld_sigma, void* stream_v, const uint32_t* sigma_ready,
                                uint32_t sigma_target) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!items || n_items < 1 || n_items > ESSA_MAX_BLOCK_ITEMS)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_block: 1 .. ESSA_MAX_BLOCK_ITEMS items expected");
  for (int32_t i = 0; i < n_items; ++i) {
    const int32_t st = validate_projection_args(ctx, items[i].adapter, items[i].x, T, seg, P, sigma, ld_sigma,
                                                items[i].sA_col, items[i].sB_col, items[i].y);
    if (st != ESSA_OK) return st;
  }
  if (T == 0) return ESSA_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  order_stream(ctx, stream);
  if (T <= kDecodeMaxTokens) {
    BlockItem bi[ESSA_MAX_BLOCK_ITEMS];
    for (int32_t i = 0; i < n_items; ++i)
      bi[i] = BlockItem{items[i].adapter, static_cast<const __nv_bfloat16*>(items[i].x), items[i].sA_col, items[i].sB_col,
                        static_cast<__nv_bfloat16*>(items[i].y)};
    cudaEvent_t* ev = nullptr;
    if (ctx->prof_on) {
      if ((size_t)(ctx->prof_calls + 1) * 3 <= ctx->prof_events.size()) ev = &ctx->prof_events[(size_t)ctx->prof_calls * 3];
      else ++ctx->prof_dropped;
    }
    if (ev) { cudaEventRecord(ev[0], stream); cudaEventRecord(ev[1], stream); }
    const int32_t st = launch_block_decode(ctx, bi, n_items, T, seg, P, sigma, ld_sigma, stream, sigma_ready, sigma_target);
    if (st != kBlockNotFused) {
      if (ev) { cudaEventRecord(ev[2], stream); ++ctx->prof_calls; }
      return st;
    }
  }
  {
    BlockItem bi[ESSA_MAX_BLOCK_ITEMS];
    for (int32_t i = 0; i < n_items; ++i)
      bi[i] = BlockItem{items[i].adapter, static_cast<const __nv_bfloat16*>(items[i].x), items[i].sA_col, items[i].sB_col,
                        static_cast<__nv_bfloat16*>(items[i].y)};
    const int32_t st = launch_block_prefill(ctx, bi, n_items, T, seg, P, sigma, ld_sigma, stream);
    if (st != kBlockNotFused) return st;
  }
  for (int32_t i = 0; i < n_items; ++i) {
    ProjArgs g{static_cast<const __nv_bfloat16*>(items[i].x), T, seg, P, sigma, ld_sigma, items[i].sA_col, items[i].sB_col,
               static_cast<__nv_bfloat16*>(items[i].y)};
    const int32_t st = launch_projection_tc(ctx, items[i].adapter, g, stream);
    if (st != ESSA_OK) return st;
  }
  return ESSA_OK;
}

int32_t essa_apply_block(essa_ctx* ctx, const essa_block_item* items, int32_t n_items, int64_t T, const int32_t* seg,
                         int32_t P, const float* sigma, int32_t ld_sigma, void* stream_v) {
  return apply_block_impl(ctx, items, n_items, T, seg, P, sigma, ld_sigma, stream_v, nullptr, 0);
}

int32_t essa_apply_layers(essa_ctx* ctx, const essa_block_item* items, int32_t n_layers, int32_t n_items, int64_t T,
                          const int32_t* seg, int32_t P, const float* sigma, int32_t ld_sigma, void* stream_v) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!items || n_layers < 1 || n_items < 1 || n_items > ESSA_MAX_BLOCK_ITEMS)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "apply_layers: need n_layers >= 1 and 1 .. ESSA_MAX_BLOCK_ITEMS items per layer");
  for (int64_t j = 0; j < (int64_t)n_layers * n_items; ++j) {
    const int32_t st = validate_projection_args(ctx, items[j].adapter, items[j].x, T, seg, P, sigma, ld_sigma, items[j].sA_col,
                                                items[j].sB_col, items[j].y);
    if (st != ESSA_OK) return st;
  }
  if (T == 0) return ESSA_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  order_stream(ctx, stream);
  // Decode sizes: one launch per layer; consecutive launches alternate between the context's two scratch sets and do
  // not wait for one another, so a layer's CTAs start wherever the layer before has freed an SM.  A layer that does
  // not fit the one-launch schedule (and every layer of a larger call) is issued like essa_apply_block.
  bool chain = T <= kDecodeMaxTokens && n_layers > 1;
  if (chain) ctx->layers_epoch += 1;
  for (int32_t l = 0; l < n_layers; ++l) {
    const essa_block_item* it = items + (size_t)l * n_items;
    int32_t st = kBlockNotFused;
    if (T <= kDecodeMaxTokens) {
      BlockItem bi[ESSA_MAX_BLOCK_ITEMS];
      for (int32_t i = 0; i < n_items; ++i)
        bi[i] = BlockItem{it[i].adapter, static_cast<const __nv_bfloat16*>(it[i].x), it[i].sA_col, it[i].sB_col,
                          static_cast<__nv_bfloat16*>(it[i].y)};
      st = launch_block_decode(ctx, bi, n_items, T, seg, P, sigma, ld_sigma, stream, nullptr, 0, l & 1,
                               !chain ? 0 : l == 0 ? 1 : 2);
      if (st == kBlockNotFused && l == 0) chain = false;  // nobody would publish the flag the later layers wait for
    }
    if (st == kBlockNotFused) st = apply_block_impl(ctx, it, n_items, T, seg, P, sigma, ld_sigma, stream_v, nullptr, 0);
    if (st != ESSA_OK) return st;
  }
  return ESSA_OK;
}

int32_t essa_sample_apply_block(essa_ctx* ctx, const float* mean, float step, const float* Bfactor, const float* Dvec, int32_t d,
                                uint64_t seed, int32_t k_begin, int32_t P, float* sigma_out, const essa_block_item* items,
                                int32_t n_items, int64_t T, const int32_t* seg, void* stream_v) {
  int32_t st = validate_sampler(ctx, mean, d, k_begin, P, sigma_out);
  if (st != ESSA_OK) return st;
  if (!items || n_items < 1 || n_items > ESSA_MAX_BLOCK_ITEMS)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "sample_apply_block: 1 .. ESSA_MAX_BLOCK_ITEMS items expected");
  // validate the block before anything is enqueued, so that a bad argument leaves no half-done call behind
  for (int32_t i = 0; i < n_items; ++i) {
    st = validate_projection_args(ctx, items[i].adapter, items[i].x, T, seg, P, sigma_out, d, items[i].sA_col, items[i].sB_col,
                                  items[i].y);
    if (st != ESSA_OK) return st;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  uint32_t blocks = 0;
  st = launch_sampler(ctx, mean, step, Bfactor, Dvec, d, seed, k_begin, P, nullptr, d, sigma_out, stream, ctx->samp_cnt, &blocks);
  if (st != ESSA_OK) return st;
  ctx->samp_epoch += blocks;  // the draw is enqueued: its blocks will be counted
  if (T == 0) return ESSA_OK;
  return apply_block_impl(ctx, items, n_items, T, seg, P, sigma_out, d, stream_v, blocks > 0 ? ctx->samp_cnt : nullptr,
                          ctx->samp_epoch);
}

// Allocation-free variant: see the comment above g_static_u in proj_tc.cu.
int32_t essa_apply_projection_static(essa_ctx* ctx, const essa_adapter* a, const void* x, int64_t T, const int32_t* seg,
                                     int32_t P, const float* sigma, int32_t ld_sigma, int32_t sA_col, int32_t sB_col,
                                     void* y, void* stream) {
  const int32_t st = validate_projection_args(ctx, a, x, T, seg, P, sigma, ld_sigma, sA_col, sB_col, y);
  if (st != ESSA_OK || T == 0) return st;
  ProjArgs g{static_cast<const __nv_bfloat16*>(x), T, seg, P, sigma, ld_sigma, sA_col, sB_col, static_cast<__nv_bfloat16*>(y)};
  order_stream(ctx, static_cast<cudaStream_t>(stream));
  return launch_projection_tc_static(ctx, a, g, static_cast<cudaStream_t>(stream));
}

int32_t essa_apply_projection_simt(essa_ctx* ctx, const essa_adapter* a, const void* x, int64_t T, const int32_t* seg,
                                   int32_t P, const float* sigma, int32_t ld_sigma, int32_t sA_col, int32_t sB_col,
                                   void* y, void* stream) {
  const int32_t st = validate_projection_args(ctx, a, x, T, seg, P, sigma, ld_sigma, sA_col, sB_col, y);
  if (st != ESSA_OK || T == 0) return st;
  ProjArgs g{static_cast<const __nv_bfloat16*>(x), T, seg, P, sigma, ld_sigma, sA_col, sB_col, static_cast<__nv_bfloat16*>(y)};
  order_stream(ctx, static_cast<cudaStream_t>(stream));
  return launch_projection_simt(ctx, a, g, static_cast<cudaStream_t>(stream));
}

// Host-buffer calls: n projections over the same tokens, segments and table; items[i].x / .y are HOST pointers.
static int32_t host_pipeline(essa_ctx* ctx, const essa_block_item* items, int32_t n, int64_t T, const int32_t* seg_host,
                             int32_t P, const float* sigma_host, int32_t ld_sigma, void* stream_v, const char* who) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (!items || n < 1 || n > ESSA_MAX_BLOCK_ITEMS) return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": 1 .. ESSA_MAX_BLOCK_ITEMS items expected");
  if (T < 0 || P < 0) return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": negative T or P");
  for (int32_t i = 0; i < n; ++i)
    if (!items[i].adapter) return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": adapter is NULL");
  if (T == 0) return ESSA_OK;
  if (!seg_host || !sigma_host || P == 0) return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": NULL buffer or no candidates");
  for (int32_t i = 0; i < n; ++i)
    if (!items[i].x || !items[i].y) return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": NULL buffer or no candidates");
  if (essa_validate_segments(seg_host, P, T) != ESSA_OK)
    return fail(ctx, ESSA_ERR_INVALID_ARG, std::string(who) + ": seg_offsets must rise from 0 to T");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
  // staging: the items' x (and y) one after the other, each 256-byte aligned.  Items that pass the SAME host
  // activations (the q, k, v projections of a block read one x) share one staged copy: x_src[i] is the first item
  // with that pointer and width, and only such first items are copied in.
  size_t x_off[ESSA_MAX_BLOCK_ITEMS + 1] = {0}, y_off[ESSA_MAX_BLOCK_ITEMS + 1] = {0};
  int x_src[ESSA_MAX_BLOCK_ITEMS];
  size_t x_at[ESSA_MAX_BLOCK_ITEMS];
  for (int32_t i = 0; i < n; ++i) {
    x_src[i] = i;
    for (int32_t j = 0; j < i; ++j)
      if (items[j].x == items[i].x && items[j].adapter->d_in == items[i].adapter->d_in) { x_src[i] = x_src[j]; break; }
    x_at[i] = x_src[i] == i ? x_off[i] : x_at[x_src[i]];
    x_off[i + 1] = x_off[i] + (x_src[i] == i ? (((size_t)T * items[i].adapter->d_in * 2 + 255) & ~(size_t)255) : 0);
    y_off[i + 1] = y_off[i] + (((size_t)T * items[i].adapter->d_out * 2 + 255) & ~(size_t)255);
  }
  const size_t ob = (size_t)(P + 1) * 4, sb = (size_t)P * ld_sigma * 4;
  int32_t st;
  if ((st = ensure_scratch(ctx, ctx->stage_x, x_off[n], false, stream)) != ESSA_OK) return st;
  if ((st = ensure_scratch(ctx, ctx->stage_y, y_off[n], false, stream)) != ESSA_OK) return st;
  if ((st = ensure_scratch(ctx, ctx->stage_sigma, sb, false, stream)) != ESSA_OK) return st;

  // Chunks of whole candidates, at least kMinChunkTokens tokens each and at most kMaxChunks of them: candidates are
  // independent, so a chunk is a call of its own on a slice of x, y, the offsets and the table.
  constexpr int64_t kMinChunkTokens = 2048;
  constexpr int kMaxChunks = 8;
  std::vector<int32_t> first;  // first candidate of each chunk, then P
  first.push_back(0);
  if (T >= 2 * kMinChunkTokens) {
    int64_t target = T / kMaxChunks;
    if (target < kMinChunkTokens) target = kMinChunkTokens;
    for (int32_t k = 1; k < P; ++k)
      if ((int64_t)seg_host[k] - seg_host[first.back()] >= target && T - seg_host[k] >= kMinChunkTokens) first.push_back(k);
  }
  first.push_back(P);
  const int n_chunks = (int)first.size() - 1;
  if ((st = ensure_scratch(ctx, ctx->stage_off, ob + (size_t)n_chunks * 4, false, stream)) != ESSA_OK) return st;
  uint8_t* xd = static_cast<uint8_t*>(ctx->stage_x.ptr);
  uint8_t* yd = static_cast<uint8_t*>(ctx->stage_y.ptr);

  if (n_chunks == 1) {
    // small call (decode sizes among them): everything in, one device call for the block, everything out
    cudaError_t e = cudaMemcpyAsync(ctx->stage_off.ptr, seg_host, ob, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage_sigma.ptr, sigma_host, sb, cudaMemcpyHostToDevice, stream);
    essa_block_item dev[ESSA_MAX_BLOCK_ITEMS];
    for (int32_t i = 0; i < n && e == cudaSuccess; ++i) {
      if (x_src[i] == i)
        e = cudaMemcpyAsync(xd + x_at[i], items[i].x, (size_t)T * items[i].adapter->d_in * 2, cudaMemcpyHostToDevice, stream);
      dev[i] = essa_block_item{items[i].adapter, xd + x_at[i], items[i].sA_col, items[i].sB_col, yd + y_off[i]};
    }
    if (e != cudaSuccess) return check_cuda(ctx, e, "host call: H2D");
    st = essa_apply_block(ctx, dev, n, T, static_cast<const int32_t*>(ctx->stage_off.ptr), P,
                          static_cast<const float*>(ctx->stage_sigma.ptr), ld_sigma, stream_v);
    if (st != ESSA_OK) return st;
    for (int32_t i = 0; i < n && e == cudaSuccess; ++i)
      e = cudaMemcpyAsync(items[i].y, yd + y_off[i], (size_t)T * items[i].adapter->d_out * 2, cudaMemcpyDeviceToHost, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    return check_cuda(ctx, e, "host call: D2H");
  }

  // Three-stage pipeline over (projection, chunk) units: host -> device copies on one stream, the projections on
  // `stream`, device -> host copies on a third, chained by events, so that a unit's copies overlap its neighbours'
  // compute and the two copy directions overlap each other (with pinned host memory).
  if (!ctx->host_h2d && cudaStreamCreateWithFlags(&ctx->host_h2d, cudaStreamNonBlocking) != cudaSuccess)
    return check_cuda(ctx, cudaGetLastError(), "host call: cudaStreamCreate");
  if (!ctx->host_d2h && cudaStreamCreateWithFlags(&ctx->host_d2h, cudaStreamNonBlocking) != cudaSuccess)
    return check_cuda(ctx, cudaGetLastError(), "host call: cudaStreamCreate");
  const size_t n_events = (size_t)2 * kMaxChunks * ESSA_MAX_BLOCK_ITEMS + 1;
  while (ctx->host_events.size() < n_events) {
    cudaEvent_t ev;
    if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) != cudaSuccess)
      return check_cuda(ctx, cudaGetLastError(), "host call: cudaEventCreate");
    ctx->host_events.push_back(ev);
  }
  // per-chunk offsets, rebased to start at 0: chunk c occupies entries [first[c] + c, first[c + 1] + c] of one array
  std::vector<int32_t> off((size_t)P + n_chunks);
  for (int c = 0; c < n_chunks; ++c)
    for (int32_t k = first[c]; k <= first[c + 1]; ++k) off[(size_t)k + c] = seg_host[k] - seg_host[first[c]];
  cudaError_t e = cudaEventRecord(ctx->host_events[n_events - 1], stream);  // earlier work on `stream` may still read the staging buffers
  if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->host_h2d, ctx->host_events[n_events - 1], 0);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage_off.ptr, off.data(), off.size() * 4, cudaMemcpyHostToDevice, ctx->host_h2d);
  if (e == cudaSuccess) e = cudaMemcpyAsync(ctx->stage_sigma.ptr, sigma_host, sb, cudaMemcpyHostToDevice, ctx->host_h2d);
  if (e != cudaSuccess) return check_cuda(ctx, e, "host call: H2D");
  auto drain = [&]() {
    cudaStreamSynchronize(ctx->host_h2d);
    cudaStreamSynchronize(stream);
    cudaStreamSynchronize(ctx->host_d2h);
  };
  int unit = 0;
  for (int32_t i = 0; i < n; ++i) {
    const essa_adapter* a = items[i].adapter;
    const uint8_t* xh = static_cast<const uint8_t*>(items[i].x);
    uint8_t* yh = static_cast<uint8_t*>(items[i].y);
    for (int c = 0; c < n_chunks; ++c, ++unit) {
      const int64_t t0 = seg_host[first[c]], t1 = seg_host[first[c + 1]];
      const size_t xo = (size_t)t0 * a->d_in * 2, yo = (size_t)t0 * a->d_out * 2;
      e = cudaSuccess;
      if (x_src[i] == i)  // (a shared x was copied by an earlier item; copies and events on host_h2d are in order)
        e = cudaMemcpyAsync(xd + x_at[i] + xo, xh + xo, (size_t)(t1 - t0) * a->d_in * 2, cudaMemcpyHostToDevice, ctx->host_h2d);
      if (e == cudaSuccess) e = cudaEventRecord(ctx->host_events[2 * unit], ctx->host_h2d);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(stream, ctx->host_events[2 * unit], 0);
      if (e != cudaSuccess) { drain(); return check_cuda(ctx, e, "host call: H2D"); }
      if (t1 > t0) {
        st = essa_apply_projection(ctx, a, xd + x_at[i] + xo, t1 - t0, static_cast<const int32_t*>(ctx->stage_off.ptr) + first[c] + c,
                                   first[c + 1] - first[c], static_cast<const float*>(ctx->stage_sigma.ptr) + (size_t)first[c] * ld_sigma,
                                   ld_sigma, items[i].sA_col, items[i].sB_col, yd + y_off[i] + yo, stream_v);
        if (st != ESSA_OK) { drain(); return st; }
      }
      e = cudaEventRecord(ctx->host_events[2 * unit + 1], stream);
      if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->host_d2h, ctx->host_events[2 * unit + 1], 0);
      if (e == cudaSuccess) e = cudaMemcpyAsync(yh + yo, yd + y_off[i] + yo, (size_t)(t1 - t0) * a->d_out * 2, cudaMemcpyDeviceToHost, ctx->host_d2h);
      if (e != cudaSuccess) { drain(); return check_cuda(ctx, e, "host call: D2H"); }
    }
  }
  e = cudaStreamSynchronize(ctx->host_d2h);
  if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(ctx->host_h2d);
  return check_cuda(ctx, e, "host call: D2H");
}

int32_t essa_apply_projection_host(essa_ctx* ctx, const essa_adapter* a, const void* x_host, int64_t T,
                                   const int32_t* seg_host, int32_t P, const float* sigma_host, int32_t ld_sigma,
                                   int32_t sA_col, int32_t sB_col, void* y_host, void* stream_v) {
  const essa_block_item item{a, x_host, sA_col, sB_col, y_host};
  return host_pipeline(ctx, &item, 1, T, seg_host, P, sigma_host, ld_sigma, stream_v, "apply_projection_host");
}

int32_t essa_apply_block_host(essa_ctx* ctx, const essa_block_item* items_host, int32_t n_items, int64_t T,
                              const int32_t* seg_host, int32_t P, const float* sigma_host, int32_t ld_sigma, void* stream_v) {
  return host_pipeline(ctx, items_host, n_items, T, seg_host, P, sigma_host, ld_sigma, stream_v, "apply_block_host");
}

int32_t essa_plan_projection(int32_t d_in, int32_t d_out, int32_t rank, int32_t w0_dtype, int64_t T, int32_t sm_count,
                             essa_plan* out) {
  if (!out || d_in <= 0 || d_out <= 0 || rank <= 0 || T < 0) return ESSA_ERR_INVALID_ARG;
  if (rank > ESSA_MAX_RANK || d_in % 64 != 0 || d_out % 8 != 0) return ESSA_ERR_UNSUPPORTED_SHAPE;
  if (w0_dtype != ESSA_W0_BF16 && w0_dtype != ESSA_W0_INT8_PERCHANNEL && w0_dtype != ESSA_W0_INT4_GROUP128) return ESSA_ERR_INVALID_ARG;
  plan_projection(d_in, d_out, rank, w0_dtype, T, sm_count, out);
  return ESSA_OK;
}

int32_t essa_profile_begin(essa_ctx* ctx, int32_t max_calls) {
  if (!ctx || max_calls < 0) return ESSA_ERR_INVALID_ARG;
  while (ctx->prof_events.size() < (size_t)max_calls * 3) {
    cudaEvent_t e;
    if (cudaEventCreate(&e) != cudaSuccess) return check_cuda(ctx, cudaGetLastError(), "cudaEventCreate");
    ctx->prof_events.push_back(e);
  }
  ctx->prof_calls = 0;
  ctx->prof_dropped = 0;
  ctx->prof_on = true;
  return ESSA_OK;
}

int32_t essa_profile_end(essa_ctx* ctx, essa_profile* out) {
  if (!ctx || !out) return ESSA_ERR_INVALID_ARG;
  ctx->prof_on = false;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return check_cuda(ctx, e, "cudaDeviceSynchronize");
  out->rank_down_ms = out->base_up_ms = 0.0;
  out->calls = ctx->prof_calls;
  out->dropped = ctx->prof_dropped;
  for (int c = 0; c < ctx->prof_calls; ++c) {
    float a = 0.f, b = 0.f;
    cudaEvent_t* ev = &ctx->prof_events[(size_t)c * 3];
    if (cudaEventElapsedTime(&a, ev[0], ev[1]) != cudaSuccess || cudaEventElapsedTime(&b, ev[1], ev[2]) != cudaSuccess)
      return check_cuda(ctx, cudaGetLastError(), "cudaEventElapsedTime");
    out->rank_down_ms += a;
    out->base_up_ms += b;
  }
  return ESSA_OK;
}

int32_t essa_validate_segments(const int32_t* seg, int32_t P, int64_t T) {
  if (!seg || P < 0 || T < 0) return ESSA_ERR_INVALID_ARG;
  if (seg[0] != 0) return ESSA_ERR_INVALID_ARG;
  for (int32_t k = 0; k < P; ++k)
    if (seg[k + 1] < seg[k]) return ESSA_ERR_INVALID_ARG;
  return seg[P] == T ? ESSA_OK : ESSA_ERR_INVALID_ARG;
}

int32_t essa_debug_stream_words(essa_ctx* ctx, uint64_t seed, int32_t k_begin, int32_t k_count, int32_t n_blocks,
                                uint32_t* words_out, void* stream) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (k_begin < 0 || k_count < 0 || n_blocks < 0 || ((int64_t)k_count * n_blocks > 0 && !words_out))
    return fail(ctx, ESSA_ERR_INVALID_ARG, "debug_stream_words: bad arguments");
  return launch_stream_words(ctx, seed, k_begin, k_count, n_blocks, words_out, static_cast<cudaStream_t>(stream));
}

int32_t essa_debug_philox(essa_ctx* ctx, const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  if (!ctx || !ctr || !key || !out) return ESSA_ERR_INVALID_ARG;
  return launch_philox_once(ctx, ctr, key, out);
}

int32_t essa_debug_segment_map(essa_ctx* ctx, const int32_t* seg, int32_t P, int64_t T, int32_t* cand_out, void* stream) {
  if (!ctx) return ESSA_ERR_INVALID_ARG;
  if (T < 0 || P < 0 || (T > 0 && (P == 0 || !seg || !cand_out)) || T > 0x7fffffffLL)
    return fail(ctx, ESSA_ERR_INVALID_ARG, "debug_segment_map: bad arguments");
  return launch_segment_map(ctx, seg, P, T, cand_out, static_cast<cudaStream_t>(stream));
}

int32_t essa_debug_core_matrix(essa_ctx* ctx, const essa_adapter* a, float* M_host) {
  if (!ctx || !a || !M_host) return ESSA_ERR_INVALID_ARG;
  float full[kRankPadMax * kRankPadMax];
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(full, a->M, sizeof full, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return check_cuda(ctx, e, "debug_core_matrix");
  for (int j = 0; j < a->rank; ++j)
    for (int i = 0; i < a->rank; ++i) M_host[j * a->rank + i] = full[j * kRankPadMax + i];
  return ESSA_OK;
}

}  // extern "C"
