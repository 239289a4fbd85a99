"""ctypes binding of libessa.so: argument marshalling only.

Every function here forwards to the C entry point of the same name (``essa_`` prefix dropped on the
methods of :class:`Context`); all arithmetic runs in the library's CUDA kernels.  torch supplies device
memory (``tensor.data_ptr()``) and streams, nothing else.  There is no fallback: if the library has not
been built, or no sm_100 GPU is present, the calls raise.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libessa.so")

ESSA_OK = 0
ESSA_ERR_INVALID_ARG = -1
ESSA_ERR_UNSUPPORTED_SHAPE = -2
ESSA_ERR_ALLOC = -3
ESSA_ERR_CUDA = -4
ESSA_ERR_DEVICE_TIMEOUT = -5
ESSA_ERR_NO_DEVICE = -6
ESSA_W0_BF16 = 0
ESSA_W0_INT8_PERCHANNEL = 1
ESSA_W0_INT4_GROUP128 = 2
ESSA_OPT_PAIR_TILES = 1
ESSA_OPT_FUSE_DOWN = 2
ESSA_OPT_WAIT_LIMIT_MCYCLES = 3
ESSA_OPT_DEBUG_STALL_RANK_ROWS = 4
ESSA_OPT_DECODE_PAIRS = 5
ESSA_OPT_DECODE_DOWN_CTAS = 6
ESSA_OPT_WIDE_TILES = 7
ESSA_OPT_DOWN_SPLITS = 8
ESSA_OPT_L2_HINTS = 9
ESSA_OPT_DOWN_PAIRS = 10
ESSA_OPT_DOWN_TILE_UNITS = 11

EXPORTED_SYMBOLS = (
    "essa_version", "essa_status_string", "essa_create", "essa_destroy", "essa_last_error", "essa_get_status",
    "essa_reserve", "essa_load_adapter", "essa_free_adapter", "essa_sample_population",
    "essa_sample_population_range", "essa_apply_projection", "essa_apply_projection_host",
    "essa_apply_projection_simt", "essa_plan_projection", "essa_validate_segments", "essa_debug_stream_words",
    "essa_debug_philox", "essa_debug_segment_map", "essa_debug_core_matrix", "essa_profile_begin", "essa_profile_end",
    "essa_apply_projection_static", "essa_get_launch_count", "essa_reserve_dequant", "essa_apply_block", "essa_apply_block_host", "essa_set_option",
    "essa_top_alpha_index", "essa_sample_population_masked", "essa_export_candidates", "essa_sample_apply_block",
    "essa_apply_layers", "essa_cma_create", "essa_cma_destroy", "essa_cma_ask", "essa_tell", "essa_cma_set", "essa_cma_get", "essa_cma_params",
)


def top_alpha_index(n_factors: int, rank: int, alpha) -> list:
    """essa_top_alpha_index: columns of the floor(alpha * rank) leading entries of each of n_factors slices of `rank`
    columns.  alpha may be a float, a string or a Fraction; it is turned into an exact ratio of integers first."""
    from fractions import Fraction
    fr = alpha if isinstance(alpha, Fraction) else Fraction(str(alpha))
    lib = load_library()
    cnt = C.c_int32(0)
    st = lib.essa_top_alpha_index(n_factors, rank, fr.numerator, fr.denominator, None, C.byref(cnt))
    if st != ESSA_OK:
        raise EssaError(st, "top_alpha_index: bad arguments")
    out = (C.c_int32 * max(cnt.value, 1))()
    st = lib.essa_top_alpha_index(n_factors, rank, fr.numerator, fr.denominator, out, C.byref(cnt))
    if st != ESSA_OK:
        raise EssaError(st, "top_alpha_index: bad arguments")
    return [int(out[i]) for i in range(cnt.value)]


class EssaError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"essa status {status}: {message}")
        self.status = status


class AdapterDesc(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("d_out", C.c_int32), ("rank", C.c_int32), ("w0_dtype", C.c_int32),
                ("W0", C.c_void_p), ("w0_scale", C.c_void_p), ("U_A", C.c_void_p), ("V_A", C.c_void_p),
                ("U_B", C.c_void_p), ("V_B", C.c_void_p), ("on_device", C.c_int32)]


class BlockItem(C.Structure):
    _fields_ = [("adapter", C.c_void_p), ("x", C.c_void_p), ("sA_col", C.c_int32), ("sB_col", C.c_int32), ("y", C.c_void_p)]


class Plan(C.Structure):
    _fields_ = [("block_m", C.c_int32), ("block_n", C.c_int32), ("block_k", C.c_int32), ("stages", C.c_int32),
                ("k_blocks", C.c_int32), ("splits", C.c_int32), ("tiles", C.c_int32), ("grid", C.c_int32),
                ("down_splits", C.c_int32), ("down_grid", C.c_int32), ("scratch_bytes", C.c_int64),
                ("decode", C.c_int32), ("x_stages", C.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class Profile(C.Structure):
    _fields_ = [("rank_down_ms", C.c_double), ("base_up_ms", C.c_double), ("calls", C.c_int32), ("dropped", C.c_int32)]


_lib = None


def load_library() -> C.CDLL:
    """dlopen libessa.so (built by ``python -m paper_2507_04453_b200.build``) and declare signatures."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(f"{LIB_PATH} not built: run `python -m paper_2507_04453_b200.build` (or __graft_entry__.build())")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, u64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint64, C.c_float
    sig = {
        "essa_version": (i32, []),
        "essa_status_string": (C.c_char_p, [i32]),
        "essa_create": (i32, [C.POINTER(vp), i32]),
        "essa_destroy": (i32, [vp]),
        "essa_last_error": (C.c_char_p, [vp]),
        "essa_get_status": (i32, [vp, C.POINTER(i32)]),
        "essa_reserve": (i32, [vp, i64, i32, i32]),
        "essa_get_launch_count": (i32, [vp, C.POINTER(i64)]),
        "essa_reserve_dequant": (i32, [vp, i32, i32]),
        "essa_set_option": (i32, [vp, i32, i32]),
        "essa_apply_block": (i32, [vp, C.POINTER(BlockItem), i32, i64, vp, i32, vp, i32, vp]),
        "essa_apply_block_host": (i32, [vp, C.POINTER(BlockItem), i32, i64, vp, i32, vp, i32, vp]),
        "essa_apply_layers": (i32, [vp, C.POINTER(BlockItem), i32, i32, i64, vp, i32, vp, i32, vp]),
        "essa_sample_apply_block": (i32, [vp, vp, f32, vp, vp, i32, u64, i32, i32, vp, C.POINTER(BlockItem), i32, i64, vp, vp]),
        "essa_cma_create": (i32, [vp, i32, i32, vp, f32, C.POINTER(vp)]),
        "essa_cma_destroy": (i32, [vp, vp]),
        "essa_cma_ask": (i32, [vp, vp, u64, i32, i32, vp, vp]),
        "essa_tell": (i32, [vp, vp, vp, i32, vp, vp]),
        "essa_cma_set": (i32, [vp, vp, vp, vp, vp, vp, vp, i32, vp]),
        "essa_cma_get": (i32, [vp, vp, vp, vp, vp, vp, vp, vp, vp, C.POINTER(i32), C.POINTER(i32)]),
        "essa_cma_params": (i32, [vp, vp]),
        "essa_load_adapter": (i32, [vp, C.POINTER(AdapterDesc), C.POINTER(vp), vp]),
        "essa_free_adapter": (i32, [vp, vp]),
        "essa_sample_population": (i32, [vp, vp, f32, vp, vp, i32, u64, i32, vp, vp]),
        "essa_sample_population_range": (i32, [vp, vp, f32, vp, vp, i32, u64, i32, i32, vp, vp]),
        "essa_top_alpha_index": (i32, [i32, i32, i32, i32, vp, vp]),
        "essa_export_candidates": (i32, [vp, vp, vp, i32, i32, i32, i32, i32, vp, vp, vp]),
        "essa_sample_population_masked": (i32, [vp, vp, vp, vp, f32, vp, vp, i32, i32, u64, i32, i32, vp, vp]),
        "essa_apply_projection": (i32, [vp, vp, vp, i64, vp, i32, vp, i32, i32, i32, vp, vp]),
        "essa_apply_projection_host": (i32, [vp, vp, vp, i64, vp, i32, vp, i32, i32, i32, vp, vp]),
        "essa_apply_projection_simt": (i32, [vp, vp, vp, i64, vp, i32, vp, i32, i32, i32, vp, vp]),
        "essa_apply_projection_static": (i32, [vp, vp, vp, i64, vp, i32, vp, i32, i32, i32, vp, vp]),
        "essa_plan_projection": (i32, [i32, i32, i32, i32, i64, i32, C.POINTER(Plan)]),
        "essa_validate_segments": (i32, [vp, i32, i64]),
        "essa_debug_stream_words": (i32, [vp, u64, i32, i32, i32, vp, vp]),
        "essa_debug_philox": (i32, [vp, C.POINTER(C.c_uint32), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]),
        "essa_debug_segment_map": (i32, [vp, vp, i32, i64, vp, vp]),
        "essa_debug_core_matrix": (i32, [vp, vp, vp]),
        "essa_profile_begin": (i32, [vp, i32]),
        "essa_profile_end": (i32, [vp, C.POINTER(Profile)]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype = res
        fn.argtypes = args
    _lib = lib
    return lib


def plan_projection(d_in: int, d_out: int, rank: int, w0_dtype: int, T: int, sm_count: int = 148) -> dict:
    """essa_plan_projection: the schedule a call would use (host arithmetic, no device needed)."""
    lib = load_library()
    p = Plan()
    st = lib.essa_plan_projection(d_in, d_out, rank, w0_dtype, T, sm_count, C.byref(p))
    if st != ESSA_OK:
        raise EssaError(st, lib.essa_status_string(st).decode())
    return p.as_dict()


def validate_segments(seg_offsets, T: int) -> int:
    """essa_validate_segments on a host int32 array; returns the status code."""
    lib = load_library()
    seg = np.ascontiguousarray(seg_offsets, dtype=np.int32)
    return lib.essa_validate_segments(seg.ctypes.data_as(C.c_void_p), len(seg) - 1, T)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream(stream) -> Optional[int]:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


class AdapterHandle:
    def __init__(self, ctx: "Context", handle: int, d_in: int, d_out: int, rank: int, w0_dtype: int):
        self.ctx, self.handle = ctx, handle
        self.d_in, self.d_out, self.rank, self.w0_dtype = d_in, d_out, rank, w0_dtype

    def free(self):
        if self.handle:
            self.ctx._check(self.ctx.lib.essa_free_adapter(self.ctx.handle, self.handle))
            self.handle = None


class PreparedBlock:
    """essa_apply_block with its arguments marshalled ahead of time (see Context.prepare_block)."""

    def __init__(self, ctx, adapters, xs, seg_offsets, sigma, cols, outs):
        n = len(adapters)
        T = xs[0].shape[0]
        self.keep = (list(adapters), list(xs), seg_offsets, sigma, list(outs))
        self.arr = (BlockItem * n)()
        for i in range(n):
            self.arr[i] = BlockItem(adapters[i].handle, xs[i].data_ptr() if T else None, cols[i][0], cols[i][1],
                                    outs[i].data_ptr() if T else None)
        self.ctx = ctx
        self.fn = ctx.lib.essa_apply_block
        self.args = (ctx.handle, self.arr, n, T, seg_offsets.data_ptr(), seg_offsets.numel() - 1, sigma.data_ptr(),
                     sigma.stride(0) if sigma.dim() == 2 else sigma.numel())

    def run(self, stream_handle):
        """stream_handle: the integer cudaStream_t (torch's ``stream.cuda_stream``; 0 / None = default stream)."""
        st = self.fn(*self.args, stream_handle or None)
        if st != ESSA_OK:
            self.ctx._check(st)


class PreparedLayers:
    """essa_apply_layers with its arguments marshalled ahead of time (see Context.prepare_layers)."""

    def __init__(self, ctx, layers, seg_offsets, sigma):
        n_layers, n_items = len(layers), len(layers[0])
        T = layers[0][0][1].shape[0]
        self.keep = (layers, seg_offsets, sigma)
        self.arr = (BlockItem * (n_layers * n_items))()
        for l, layer in enumerate(layers):
            assert len(layer) == n_items
            for i, (ad, x, cols, y) in enumerate(layer):
                self.arr[l * n_items + i] = BlockItem(ad.handle, x.data_ptr() if T else None, cols[0], cols[1],
                                                      y.data_ptr() if T else None)
        self.ctx = ctx
        self.fn = ctx.lib.essa_apply_layers
        self.args = (ctx.handle, self.arr, n_layers, n_items, T, seg_offsets.data_ptr(), seg_offsets.numel() - 1,
                     sigma.data_ptr(), sigma.stride(0) if sigma.dim() == 2 else sigma.numel())

    def run(self, stream_handle):
        st = self.fn(*self.args, stream_handle or None)
        if st != ESSA_OK:
            self.ctx._check(st)


class PreparedSampleBlock:
    """essa_sample_apply_block with its arguments marshalled ahead of time (see Context.prepare_sample_block)."""

    def __init__(self, ctx, mean, step, Bfactor, Dvec, seed, P, sigma_out, adapters, xs, seg_offsets, cols, outs, k_begin):
        n = len(adapters)
        T = xs[0].shape[0]
        self.keep = (mean, Bfactor, Dvec, sigma_out, list(adapters), list(xs), seg_offsets, list(outs))
        self.arr = (BlockItem * n)()
        for i in range(n):
            self.arr[i] = BlockItem(adapters[i].handle, xs[i].data_ptr() if T else None, cols[i][0], cols[i][1],
                                    outs[i].data_ptr() if T else None)
        self.ctx = ctx
        self.fn = ctx.lib.essa_sample_apply_block
        self.args = (ctx.handle, mean.data_ptr(), step, _ptr(Bfactor), _ptr(Dvec), mean.numel(), seed, k_begin, P,
                     sigma_out.data_ptr(), self.arr, n, T, seg_offsets.data_ptr())

    def run(self, stream_handle):
        st = self.fn(*self.args, stream_handle or None)
        if st != ESSA_OK:
            self.ctx._check(st)


class PreparedSample:
    """essa_sample_population(_range) with its arguments marshalled ahead of time (see Context.prepare_sample)."""

    def __init__(self, ctx, mean, step, Bfactor, Dvec, seed, P, out, k_begin):
        self.keep = (mean, Bfactor, Dvec, out)
        self.ctx = ctx
        d = mean.numel()
        if k_begin == 0:
            self.fn = ctx.lib.essa_sample_population
            self.args = (ctx.handle, mean.data_ptr(), step, _ptr(Bfactor), _ptr(Dvec), d, seed, P, out.data_ptr())
        else:
            self.fn = ctx.lib.essa_sample_population_range
            self.args = (ctx.handle, mean.data_ptr(), step, _ptr(Bfactor), _ptr(Dvec), d, seed, k_begin, P, out.data_ptr())

    def run(self, stream_handle):
        st = self.fn(*self.args, stream_handle or None)
        if st != ESSA_OK:
            self.ctx._check(st)


class CmaState:
    """Device-resident search-distribution state (essa_cma_*): argument marshalling only."""

    def __init__(self, ctx, d: int, lam: int, mean0, step0: float):
        self.ctx, self.d, self.lam = ctx, d, lam
        m = np.ascontiguousarray(mean0, dtype=np.float32)
        h = C.c_void_p()
        ctx._check(ctx.lib.essa_cma_create(ctx.handle, d, lam, m.ctypes.data_as(C.c_void_p), float(step0), C.byref(h)))
        self.handle = h.value

    def close(self):
        if self.handle:
            self.ctx.lib.essa_cma_destroy(self.ctx.handle, self.handle)
            self.handle = None

    def ask(self, seed: int, P=None, out=None, k_begin: int = 0, stream=None):
        """essa_cma_ask: candidates k_begin .. k_begin + P - 1 of the population, [P, d] fp32 on the device."""
        torch = self.ctx.torch
        P = self.lam if P is None else P
        if out is None:
            out = torch.empty((P, self.d), dtype=torch.float32, device=self.ctx.device)
        self.ctx._check(self.ctx.lib.essa_cma_ask(self.ctx.handle, self.handle, seed, k_begin, P, out.data_ptr(), _stream(stream)))
        return out

    def tell(self, population, rewards, stream=None):
        """essa_tell: population [lambda, ld] fp32 and rewards [lambda] fp32, both on the device."""
        self.ctx._check(self.ctx.lib.essa_tell(self.ctx.handle, self.handle, population.data_ptr(), population.stride(0),
                                               rewards.data_ptr(), _stream(stream)))

    def set(self, mean=None, step=None, C_=None, p_sigma=None, p_c=None, generation: int = -1, stream=None):
        """essa_cma_set from host fp64 arrays (None = keep)."""
        keep = []

        def ptr(a, shape):
            if a is None:
                return None
            a = np.ascontiguousarray(np.asarray(a, dtype=np.float64).reshape(shape))
            keep.append(a)
            return a.ctypes.data_as(C.c_void_p)
        d = self.d
        self.ctx._check(self.ctx.lib.essa_cma_set(self.ctx.handle, self.handle, ptr(mean, (d,)), ptr(step, (1,)), ptr(C_, (d, d)),
                                                  ptr(p_sigma, (d,)), ptr(p_c, (d,)), generation, _stream(stream)))

    def get(self) -> dict:
        """essa_cma_get: the whole state as host fp64 arrays."""
        d = self.d
        out = {"mean": np.empty(d), "step": np.empty(1), "C": np.empty((d, d)), "B": np.empty((d, d)), "D": np.empty(d),
               "p_sigma": np.empty(d), "p_c": np.empty(d)}
        gen, sweeps = C.c_int32(0), C.c_int32(0)
        p = lambda k: out[k].ctypes.data_as(C.c_void_p)
        self.ctx._check(self.ctx.lib.essa_cma_get(self.ctx.handle, self.handle, p("mean"), p("step"), p("C"), p("B"), p("D"),
                                                  p("p_sigma"), p("p_c"), C.byref(gen), C.byref(sweeps)))
        out["step"] = float(out["step"][0])
        out["generation"], out["sweeps"] = gen.value, sweeps.value
        return out

    def params(self) -> dict:
        """essa_cma_params: the strategy parameters in use."""
        v = np.empty(9)
        self.ctx._check(self.ctx.lib.essa_cma_params(self.handle, v.ctypes.data_as(C.c_void_p)))
        names = ("mu", "mu_eff", "c_sigma", "d_sigma", "c_c", "c_1", "c_mu", "c_m", "chi_n")
        return dict(zip(names, (float(x) for x in v)))


class Context:
    """Owns one essa_ctx on a CUDA device."""

    def __init__(self, device: int = 0):
        import torch
        self.lib = load_library()
        self.torch = torch
        self.device = torch.device("cuda", device)
        h = C.c_void_p()
        st = self.lib.essa_create(C.byref(h), device)
        if st != ESSA_OK:
            raise EssaError(st, self.lib.essa_status_string(st).decode())
        self.handle = h.value

    # -- plumbing
    def _check(self, st: int):
        if st != ESSA_OK:
            raise EssaError(st, self.lib.essa_last_error(self.handle).decode() or self.lib.essa_status_string(st).decode())

    def close(self):
        if self.handle:
            self.lib.essa_destroy(self.handle)
            self.handle = None

    @property
    def gpu_launches(self) -> int:
        """essa_get_launch_count: kernels of this library enqueued through this context so far."""
        v = C.c_int64(0)
        self._check(self.lib.essa_get_launch_count(self.handle, C.byref(v)))
        return v.value

    def get_status(self) -> int:
        v = C.c_int32(0)
        self._check(self.lib.essa_get_status(self.handle, C.byref(v)))
        return v.value

    def reserve(self, max_tokens: int, max_d_in: int, max_d_out: int):
        self._check(self.lib.essa_reserve(self.handle, max_tokens, max_d_in, max_d_out))

    def set_option(self, option: int, value: int):
        """essa_set_option (ESSA_OPT_PAIR_TILES = 1, ESSA_OPT_FUSE_DOWN = 2)."""
        self._check(self.lib.essa_set_option(self.handle, option, value))

    def reserve_dequant(self, max_d_in: int, max_d_out: int):
        """essa_reserve_dequant: pre-size the scratch that prefill calls on INT8-stored adapters dequantise into."""
        self._check(self.lib.essa_reserve_dequant(self.handle, max_d_in, max_d_out))

    # -- adapters
    def load_adapter(self, ad) -> AdapterHandle:
        """essa_load_adapter from a workloads.Adapter (host arrays; values already bf16/fp16/int8 exact)."""
        torch = self.torch
        bf = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(torch.bfloat16).contiguous()
        keep = {k: bf(getattr(ad, k)) for k in ("U_A", "V_A", "U_B", "V_B")}
        if ad.w0_dtype == "bf16":
            keep["W0"] = bf(ad.W0)
            dtype, scale_ptr = ESSA_W0_BF16, None
        elif ad.w0_dtype == "int4":  # two 4-bit codes per byte, fp16 scale per (channel, group of 128 features)
            keep["W0"] = torch.from_numpy(np.ascontiguousarray(ad.W0_q, dtype=np.uint8))
            keep["scale"] = torch.from_numpy(np.ascontiguousarray(ad.W0_scale, dtype=np.float16))
            dtype, scale_ptr = ESSA_W0_INT4_GROUP128, keep["scale"].data_ptr()
        else:
            keep["W0"] = torch.from_numpy(np.ascontiguousarray(ad.W0_q, dtype=np.int8))
            keep["scale"] = torch.from_numpy(np.ascontiguousarray(ad.W0_scale, dtype=np.float16))
            dtype, scale_ptr = ESSA_W0_INT8_PERCHANNEL, keep["scale"].data_ptr()
        desc = AdapterDesc(ad.d_in, ad.d_out, ad.rank, dtype, keep["W0"].data_ptr(), scale_ptr, keep["U_A"].data_ptr(),
                           keep["V_A"].data_ptr(), keep["U_B"].data_ptr(), keep["V_B"].data_ptr(), 0)
        h = C.c_void_p()
        self._check(self.lib.essa_load_adapter(self.handle, C.byref(desc), C.byref(h), _stream(None)))
        return AdapterHandle(self, h.value, ad.d_in, ad.d_out, ad.rank, dtype)

    def load_adapter_device(self, d_in, d_out, rank, W0, U_A, V_A, U_B, V_B, w0_scale=None) -> AdapterHandle:
        """essa_load_adapter from device tensors (bf16 bases; W0 bf16, or int8 with fp16 w0_scale)."""
        dtype = ESSA_W0_BF16 if w0_scale is None else ESSA_W0_INT8_PERCHANNEL
        desc = AdapterDesc(d_in, d_out, rank, dtype, W0.data_ptr(), _ptr(w0_scale), U_A.data_ptr(), V_A.data_ptr(),
                           U_B.data_ptr(), V_B.data_ptr(), 1)
        h = C.c_void_p()
        self._check(self.lib.essa_load_adapter(self.handle, C.byref(desc), C.byref(h), _stream(None)))
        return AdapterHandle(self, h.value, d_in, d_out, rank, dtype)

    def cma_state(self, d: int, lam: int, mean0, step0: float) -> "CmaState":
        """essa_cma_create: search-distribution state (m_0 = mean0 host array, sigma_0 = step0, C_0 = I) on the device."""
        return CmaState(self, d, lam, mean0, step0)

    # -- sampling
    def sample_population(self, mean, step: float, Bfactor, Dvec, seed: int, P: int, out=None, k_begin: int = 0,
                          stream=None):
        """essa_sample_population(_range): sigma[P, d] fp32 on the device."""
        torch = self.torch
        d = mean.numel()
        if out is None:
            out = torch.empty((P, d), dtype=torch.float32, device=self.device)
        if k_begin == 0:
            st = self.lib.essa_sample_population(self.handle, mean.data_ptr(), step, _ptr(Bfactor), _ptr(Dvec), d,
                                                 seed, P, out.data_ptr(), _stream(stream))
        else:
            st = self.lib.essa_sample_population_range(self.handle, mean.data_ptr(), step, _ptr(Bfactor), _ptr(Dvec),
                                                       d, seed, k_begin, P, out.data_ptr(), _stream(stream))
        self._check(st)
        return out

    def sample_population_masked(self, frozen, index, mean_t, step: float, Bfactor_t, Dvec_t, seed: int, P: int,
                                 out=None, k_begin: int = 0, stream=None):
        """essa_sample_population_masked: sigma[P, d] with the columns `index` (int32, device) drawn around mean_t
        and every other column equal to frozen."""
        torch = self.torch
        d = frozen.numel()
        d_t = 0 if index is None else index.numel()
        if out is None:
            out = torch.empty((P, d), dtype=torch.float32, device=self.device)
        st = self.lib.essa_sample_population_masked(self.handle, frozen.data_ptr(), _ptr(index) if d_t else None,
                                                    _ptr(mean_t) if d_t else None, step, _ptr(Bfactor_t), _ptr(Dvec_t),
                                                    d, d_t, seed, k_begin, P, out.data_ptr(), _stream(stream))
        self._check(st)
        return out

    def export_candidates(self, adapter, sigma, sA_col: int, sB_col: int, k_begin: int, k_count: int, want_a=True,
                          want_b=True, stream=None):
        """essa_export_candidates: (A'[k_count, rank, d_in], B'[k_count, d_out, rank]) bf16 on the device."""
        torch = self.torch
        A = torch.empty((k_count, adapter.rank, adapter.d_in), dtype=torch.bfloat16, device=self.device) if want_a else None
        B = torch.empty((k_count, adapter.d_out, adapter.rank), dtype=torch.bfloat16, device=self.device) if want_b else None
        st = self.lib.essa_export_candidates(self.handle, adapter.handle, sigma.data_ptr(), sigma.stride(0), sA_col, sB_col,
                                             k_begin, k_count, _ptr(A) if k_count else None, _ptr(B) if k_count else None,
                                             _stream(stream))
        self._check(st)
        return A, B

    # -- projection
    def _proj(self, fn, adapter, x, seg_offsets, sigma, sA_col, sB_col, out, stream):
        torch = self.torch
        T = x.shape[0]
        P = seg_offsets.numel() - 1
        if out is None:
            out = torch.empty((T, adapter.d_out), dtype=torch.bfloat16, device=self.device)
        st = fn(self.handle, adapter.handle, x.data_ptr() if T else None, T, seg_offsets.data_ptr(), P, sigma.data_ptr(),
                sigma.stride(0) if sigma.dim() == 2 else sigma.numel(), sA_col, sB_col, out.data_ptr() if T else None,
                _stream(stream))
        self._check(st)
        return out

    def apply_projection(self, adapter, x, seg_offsets, sigma, sA_col: int, sB_col: int, out=None, stream=None):
        """essa_apply_projection: y[T, d_out] bf16 (one launch at decode sizes, else rank-down then base + up)."""
        y = self._proj(self.lib.essa_apply_projection, adapter, x, seg_offsets, sigma, sA_col, sB_col, out, stream)
        return y

    def apply_block(self, adapters, xs, seg_offsets, sigma, cols, outs=None, stream=None):
        """essa_apply_block: several projections over the same tokens / segments / sigma table in one call.

        adapters, xs, cols (pairs (sA_col, sB_col)) and outs are parallel sequences; returns the list of outputs."""
        torch = self.torch
        T = xs[0].shape[0]
        P = seg_offsets.numel() - 1
        n = len(adapters)
        if outs is None:
            outs = [torch.empty((T, a.d_out), dtype=torch.bfloat16, device=self.device) for a in adapters]
        arr = (BlockItem * n)()
        for i in range(n):
            arr[i] = BlockItem(adapters[i].handle, xs[i].data_ptr() if T else None, cols[i][0], cols[i][1],
                               outs[i].data_ptr() if T else None)
        st = self.lib.essa_apply_block(self.handle, arr, n, T, seg_offsets.data_ptr(), P, sigma.data_ptr(),
                                       sigma.stride(0) if sigma.dim() == 2 else sigma.numel(), _stream(stream))
        self._check(st)
        return outs

    def prepare_block(self, adapters, xs, seg_offsets, sigma, cols, outs):
        """The arguments of one essa_apply_block call marshalled once; ``run(stream)`` then issues the call with a
        single foreign-function call (at decode sizes the Python-side marshalling of a step is otherwise comparable
        to the step's device time).  The tensors must stay alive and in place while the object is used."""
        return PreparedBlock(self, adapters, xs, seg_offsets, sigma, cols, outs)

    def prepare_layers(self, layers, seg_offsets, sigma):
        """The arguments of one essa_apply_layers call marshalled once.  layers: a list (one entry per layer) of lists
        of (adapter, x, (sA_col, sB_col), y) tuples; ``run(stream)`` issues the call."""
        return PreparedLayers(self, layers, seg_offsets, sigma)

    def apply_layers(self, layers, seg_offsets, sigma, stream=None):
        """essa_apply_layers: the blocks of several layers in one call (see prepare_layers for the argument layout)."""
        PreparedLayers(self, layers, seg_offsets, sigma).run(_stream(stream))

    def prepare_sample_block(self, mean, step: float, Bfactor, Dvec, seed: int, P: int, sigma_out, adapters, xs, seg_offsets,
                             cols, outs, k_begin: int = 0):
        """The arguments of one essa_sample_apply_block call (population draw + the block's projections) marshalled
        once; ``run(stream)`` issues it."""
        return PreparedSampleBlock(self, mean, step, Bfactor, Dvec, seed, P, sigma_out, adapters, xs, seg_offsets, cols, outs,
                                   k_begin)

    def sample_apply_block(self, mean, step: float, Bfactor, Dvec, seed: int, P: int, adapters, xs, seg_offsets, cols,
                           sigma_out=None, outs=None, k_begin: int = 0, stream=None):
        """essa_sample_apply_block: draw the population into sigma_out[P, d] and run the block's projections on it.
        Returns (sigma_out, outs)."""
        torch = self.torch
        d = mean.numel()
        T = xs[0].shape[0]
        if sigma_out is None:
            sigma_out = torch.empty((P, d), dtype=torch.float32, device=self.device)
        if outs is None:
            outs = [torch.empty((T, a.d_out), dtype=torch.bfloat16, device=self.device) for a in adapters]
        prep = PreparedSampleBlock(self, mean, step, Bfactor, Dvec, seed, P, sigma_out, adapters, xs, seg_offsets, cols, outs,
                                   k_begin)
        prep.run(_stream(stream))
        return sigma_out, outs

    def prepare_sample(self, mean, step: float, Bfactor, Dvec, seed: int, P: int, out, k_begin: int = 0):
        """The arguments of one essa_sample_population(_range) call marshalled once; ``run(stream)`` issues it."""
        return PreparedSample(self, mean, step, Bfactor, Dvec, seed, P, out, k_begin)

    def apply_projection_static(self, adapter, x, seg_offsets, sigma, sA_col: int, sB_col: int, out, stream=None):
        """essa_apply_projection_static: same result as apply_projection without any device allocation.

        For callers that cannot allocate when they call (another allocator owns the GPU memory, or no implicit
        synchronisation is tolerable): the library's fixed 512 KB array is the only scratch, so T is limited to
        ESSA_STATIC_MAX_TOKENS (4096) and `out` must be supplied by the caller (this wrapper allocates nothing).
        Calls share that array: keep them ordered on the GPU.
        """
        if out is None:
            raise ValueError("apply_projection_static needs a caller-provided output tensor")
        y = self._proj(self.lib.essa_apply_projection_static, adapter, x, seg_offsets, sigma, sA_col, sB_col, out, stream)
        return y

    def apply_projection_simt(self, adapter, x, seg_offsets, sigma, sA_col: int, sB_col: int, out=None, stream=None):
        """essa_apply_projection_simt: CUDA-core cross-check of the same formula."""
        y = self._proj(self.lib.essa_apply_projection_simt, adapter, x, seg_offsets, sigma, sA_col, sB_col, out, stream)
        return y

    def apply_projection_host(self, adapter, x_host, seg_offsets_host, sigma_host, sA_col: int, sB_col: int, y_host,
                              stream=None):
        """essa_apply_projection_host: host tensors in (bf16 x, int32 offsets, fp32 sigma), host bf16 y out."""
        T = x_host.shape[0]
        P = seg_offsets_host.numel() - 1
        st = self.lib.essa_apply_projection_host(self.handle, adapter.handle, x_host.data_ptr(), T,
                                                 seg_offsets_host.data_ptr(), P, sigma_host.data_ptr(),
                                                 sigma_host.stride(0), sA_col, sB_col, y_host.data_ptr(), _stream(stream))
        self._check(st)
        return y_host

    def apply_block_host(self, adapters, xs_host, seg_offsets_host, sigma_host, cols, ys_host, stream=None):
        """essa_apply_block_host: apply_block with host tensors (bf16 x per projection, int32 offsets, fp32 sigma) and
        host bf16 outputs."""
        T = xs_host[0].shape[0]
        P = seg_offsets_host.numel() - 1
        n = len(adapters)
        arr = (BlockItem * n)()
        for i in range(n):
            arr[i] = BlockItem(adapters[i].handle, xs_host[i].data_ptr() if T else None, cols[i][0], cols[i][1],
                               ys_host[i].data_ptr() if T else None)
        st = self.lib.essa_apply_block_host(self.handle, arr, n, T, seg_offsets_host.data_ptr(), P, sigma_host.data_ptr(),
                                            sigma_host.stride(0), _stream(stream))
        self._check(st)
        return ys_host

    def profile_begin(self, max_calls: int):
        """essa_profile_begin: record per-kernel CUDA events inside the following apply_projection calls."""
        self._check(self.lib.essa_profile_begin(self.handle, max_calls))

    def profile_end(self) -> dict:
        """essa_profile_end: {rank_down_ms, base_up_ms, calls, dropped} summed over the recorded calls."""
        p = Profile()
        self._check(self.lib.essa_profile_end(self.handle, C.byref(p)))
        return {"rank_down_ms": p.rank_down_ms, "base_up_ms": p.base_up_ms, "calls": p.calls, "dropped": p.dropped}

    # -- diagnostics
    def debug_philox(self, ctr, key):
        c = (C.c_uint32 * 4)(*[int(v) for v in ctr])
        k = (C.c_uint32 * 2)(*[int(v) for v in key])
        o = (C.c_uint32 * 4)()
        self._check(self.lib.essa_debug_philox(self.handle, c, k, o))
        return [int(v) for v in o]

    def debug_stream_words(self, seed: int, k_begin: int, k_count: int, n_blocks: int):
        torch = self.torch
        out = torch.empty((k_count, n_blocks, 4), dtype=torch.int32, device=self.device)
        self._check(self.lib.essa_debug_stream_words(self.handle, seed, k_begin, k_count, n_blocks, out.data_ptr(), _stream(None)))
        return out

    def debug_segment_map(self, seg_offsets, T: int):
        torch = self.torch
        out = torch.empty((T,), dtype=torch.int32, device=self.device)
        self._check(self.lib.essa_debug_segment_map(self.handle, seg_offsets.data_ptr(), seg_offsets.numel() - 1, T,
                                                    out.data_ptr() if T else None, _stream(None)))
        return out

    def debug_core_matrix(self, adapter) -> np.ndarray:
        M = np.empty((adapter.rank, adapter.rank), dtype=np.float32)
        self._check(self.lib.essa_debug_core_matrix(self.handle, adapter.handle, M.ctypes.data_as(C.c_void_p)))
        return M
