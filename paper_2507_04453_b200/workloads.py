"""Seeded synthetic inputs for the ESSA population-projection path.

This module only *draws inputs*: token activations, frozen base weights,
frozen singular-vector bases, base singular values, segment lengths and the
CMA-ES search-distribution state.  It contains none of the method's
arithmetic (no Philox, no Box-Muller, no projection maths) so that both the
CUDA path and the CPU oracle can be fed from it without sharing any code of
the method itself.

Shapes follow the Qwen2.5 attention projections (q/o: d_model -> d_model,
k/v: d_model -> d_kv) the paper's backbones have (Section 4, "Models");
values are synthetic: the paper's checkpoints and datasets are not used.

All floating-point arrays returned here hold values that are exactly
representable in the storage type the GPU sees (bf16 for activations, weights
and bases; fp16 for INT8 scales; fp32 for the CMA-ES state), carried in
float32 numpy arrays, so that widening them to fp64 on the oracle side is
exact and both sides consume identical numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

PROJ_NAMES = ("q", "k", "v", "o")


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    if np.any(bits & np.uint32(0xFFFF)):
        raise ValueError("value is not representable in bf16")
    return (bits >> np.uint32(16)).astype(np.uint16).reshape(a.shape)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).reshape(b.shape)


@dataclass(frozen=True)
class WorkloadConfig:
    """One of the five benchmark configurations."""

    cfg_id: int
    name: str
    projections: Tuple[Tuple[str, int, int], ...]  # (name, d_in, d_out)
    rank: int
    P: int
    seg_kind: str  # "fixed" | "uniform" | "mixed"
    seg_len: int  # fixed length, or the upper end of U{1..seg_len}
    w0_dtype: str  # "bf16" | "int8" | "int4"
    step: float
    full_B: bool
    random_D: bool
    philox_seed: int

    @property
    def d(self) -> int:
        """CMA-ES dimension: one sA and one sB vector of length r per projection."""
        return len(self.projections) * 2 * self.rank

    def sigma_cols(self, proj_idx: int) -> Tuple[int, int]:
        """Columns of the sigma table holding (sA, sB) of projection proj_idx.

        A row is laid out as one contiguous slice per LoRA matrix:
        [q: sA(r) sB(r)] [k: ...] [v: ...] [o: ...].
        """
        base = proj_idx * 2 * self.rank
        return base, base + self.rank


def _qkvo(d_model: int, d_kv: int):
    return (("q", d_model, d_model), ("k", d_model, d_kv), ("v", d_model, d_kv), ("o", d_model, d_model))


CONFIGS: Dict[str, WorkloadConfig] = {
    "1": WorkloadConfig(1, "tiny-896-r8-P4x16", (("p", 896, 896),), 8, 4, "fixed", 16, "bf16", 0.1, False, False, 0),
    "2": WorkloadConfig(2, "qwen2.5-7b-prefill-r16-P32x512", _qkvo(3584, 512), 16, 32, "fixed", 512, "bf16", 0.05, False, True, 2),
    "3": WorkloadConfig(3, "qwen2.5-7b-decode-r16-P256x1", _qkvo(3584, 512), 16, 256, "fixed", 1, "bf16", 0.05, True, True, 3),
    "4": WorkloadConfig(4, "qwen2.5-32b-ragged-r32-P64", _qkvo(5120, 1024), 32, 64, "uniform", 1024, "bf16", 0.05, False, False, 4),
    "5a": WorkloadConfig(5, "qwen2.5-72b-int8-decode-r64-P128x1", _qkvo(8192, 1024), 64, 128, "fixed", 1, "int8", 0.05, False, False, 5),
    "5b": WorkloadConfig(5, "qwen2.5-72b-int8-prefill-r64-P128x256", _qkvo(8192, 1024), 64, 128, "fixed", 256, "int8", 0.05, False, False, 5),
    "5c": WorkloadConfig(5, "qwen2.5-72b-int8-mixed-r64-P128", _qkvo(8192, 1024), 64, 128, "mixed", 256, "int8", 0.05, False, False, 5),
    # the 72B-shaped block with INT4 group-wise weights (the paper's 72B runs are INT4, one candidate per GPU)
    "6a": WorkloadConfig(6, "qwen2.5-72b-int4-decode-r64-P128x1", _qkvo(8192, 1024), 64, 128, "fixed", 1, "int4", 0.05, False, False, 6),
    "6b": WorkloadConfig(6, "qwen2.5-72b-int4-prefill-r64-P128x256", _qkvo(8192, 1024), 64, 128, "fixed", 256, "int4", 0.05, False, False, 6),
}


def scaled_config(base: str, *, d_model: int, d_kv: int, rank: Optional[int] = None, P: Optional[int] = None,
                  seg_len: Optional[int] = None) -> WorkloadConfig:
    """A reduced-size copy of a configuration (same structure, smaller shapes) for tests."""
    c = CONFIGS[base]
    projs = (("p", d_model, d_model),) if len(c.projections) == 1 else _qkvo(d_model, d_kv)
    return WorkloadConfig(c.cfg_id, c.name + "-scaled", projs, rank or c.rank, P or c.P, c.seg_kind,
                          seg_len or c.seg_len, c.w0_dtype, c.step, c.full_B, c.random_D, c.philox_seed)


def _rng(cfg: WorkloadConfig, stream: int) -> np.random.Generator:
    """Generator for (config, stream); projection i uses stream i, shared state uses 900+."""
    return np.random.default_rng([1000 * cfg.cfg_id + stream, 0x2507_04453])


def _orthonormal(rng: np.random.Generator, rows: int, cols: int) -> np.ndarray:
    """Q factor (rows x cols, orthonormal columns) of a Gaussian matrix, sign-fixed, rounded to bf16."""
    g = rng.standard_normal((rows, cols))
    q, rr = np.linalg.qr(g)
    q = q * np.sign(np.diag(rr))[None, :]
    return round_to_bf16(q.astype(np.float32))


@dataclass
class Adapter:
    """Frozen per-projection data: base weight and the four singular-vector bases."""

    name: str
    d_in: int
    d_out: int
    rank: int
    w0_dtype: str
    W0: Optional[np.ndarray]  # [d_out, d_in] float32 (bf16-exact) when w0_dtype == "bf16"
    W0_q: Optional[np.ndarray]  # [d_out, d_in] int8 when w0_dtype == "int8"; [d_out, d_in/2] uint8 (two codes per byte) for "int4"
    W0_scale: Optional[np.ndarray]  # [d_out] float16 for "int8"; [d_out, d_in/128] float16 for "int4"
    U_A: np.ndarray  # [r, r]
    V_A: np.ndarray  # [d_in, r]
    U_B: np.ndarray  # [d_out, r]
    V_B: np.ndarray  # [r, r]
    sigma0_A: np.ndarray  # [r] float32, descending
    sigma0_B: np.ndarray  # [r] float32, descending


def quantize_int8_per_channel(W: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Symmetric per-output-channel INT8 storage of a float weight: (q int8, scale fp16).

    scale[o] = max_i |W[o,i]| / 127 rounded to fp16; q = clip(rint(W / scale), -127, 127).
    This is how the synthetic INT8 checkpoint is *produced*; both the CUDA path and the
    oracle consume the stored (q, scale) pair, so the quantisation error itself is not
    part of any comparison.
    """
    W = np.asarray(W, dtype=np.float32)
    amax = np.maximum(np.abs(W).max(axis=1), 1e-12)
    scale = (amax / 127.0).astype(np.float16)
    q = np.clip(np.rint(W / scale.astype(np.float32)[:, None]), -127, 127).astype(np.int8)
    return q, scale


INT4_GROUP = 128


def quantize_int4_groupwise(W: np.ndarray, group: int = INT4_GROUP) -> Tuple[np.ndarray, np.ndarray]:
    """Symmetric group-wise INT4 storage of a float weight: (packed uint8 [m, n/2], scale fp16 [m, n/group]).

    scale[o,g] = max |W[o, g*group:(g+1)*group]| / 7 rounded to fp16; q = clip(rint(W / scale), -7, 7); byte j of a row
    packs the codes of features 2j (low nibble) and 2j+1 (high nibble) as 4-bit two's complement.  As with INT8 this is
    how the synthetic checkpoint is *produced*; both sides consume the stored (packed, scale) pair."""
    W = np.asarray(W, dtype=np.float32)
    m, n = W.shape
    g = W.reshape(m, n // group, group)
    amax = np.maximum(np.abs(g).max(axis=2), 1e-12)
    scale = (amax / 7.0).astype(np.float16)
    q = np.clip(np.rint(g / scale.astype(np.float32)[:, :, None]), -7, 7).astype(np.int8).reshape(m, n)
    u = (q.astype(np.int16) & 0x0F).astype(np.uint8)
    packed = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    return np.ascontiguousarray(packed), np.ascontiguousarray(scale)


def make_adapter(cfg: WorkloadConfig, proj_idx: int) -> Adapter:
    name, n, m = cfg.projections[proj_idx]
    r = cfg.rank
    rng = _rng(cfg, proj_idx)
    w = (rng.standard_normal((m, n), dtype=np.float32) / np.float32(np.sqrt(n)))
    W0 = W0_q = W0_scale = None
    if cfg.w0_dtype == "bf16":
        W0 = round_to_bf16(w)
    elif cfg.w0_dtype == "int4":
        W0_q, W0_scale = quantize_int4_groupwise(w)
    else:
        W0_q, W0_scale = quantize_int8_per_channel(w)
    del w
    U_A = _orthonormal(rng, r, r)
    V_A = _orthonormal(rng, n, r)
    U_B = _orthonormal(rng, m, r)
    V_B = _orthonormal(rng, r, r)
    s0A = np.sort(rng.uniform(0.01, 1.0, r))[::-1].astype(np.float32)
    s0B = np.sort(rng.uniform(0.01, 1.0, r))[::-1].astype(np.float32)
    return Adapter(name, n, m, r, cfg.w0_dtype, W0, W0_q, W0_scale, U_A, V_A, U_B, V_B,
                   np.ascontiguousarray(s0A), np.ascontiguousarray(s0B))


def make_segments(cfg: WorkloadConfig) -> np.ndarray:
    """Segment offsets int32[P+1]: candidate k owns tokens [off[k], off[k+1])."""
    rng = _rng(cfg, 900)
    if cfg.seg_kind == "fixed":
        lens = np.full(cfg.P, cfg.seg_len, dtype=np.int64)
    elif cfg.seg_kind == "uniform":
        lens = rng.integers(1, cfg.seg_len + 1, size=cfg.P)
    elif cfg.seg_kind == "mixed":  # decode candidates interleaved with prefill candidates
        lens = np.where(np.arange(cfg.P) % 2 == 0, 1, cfg.seg_len).astype(np.int64)
    else:
        raise ValueError(cfg.seg_kind)
    off = np.zeros(cfg.P + 1, dtype=np.int64)
    np.cumsum(lens, out=off[1:])
    return off.astype(np.int32)


def make_tokens(cfg: WorkloadConfig, proj_idx: int, T: int) -> np.ndarray:
    """Activations x[T, d_in] ~ N(0,1), bf16-exact float32. Each projection call has its own x."""
    n = cfg.projections[proj_idx][1]
    rng = _rng(cfg, 100 + proj_idx)
    return round_to_bf16(rng.standard_normal((T, n), dtype=np.float32))


@dataclass
class CmaState:
    """Search-distribution state N(mean, step^2 * B diag(D)^2 B^T) and the population seed."""

    mean: np.ndarray  # [d] float32
    step: float
    Bfactor: Optional[np.ndarray]  # [d, d] float32 row-major or None (identity)
    Dvec: Optional[np.ndarray]  # [d] float32 or None (ones)
    seed: int
    d: int = field(init=False)

    def __post_init__(self):
        self.d = int(self.mean.shape[0])


def make_cma_state(cfg: WorkloadConfig, adapters: List[Adapter]) -> CmaState:
    """mean = the adapters' base singular values in table order; B, D per the configuration."""
    mean = np.concatenate([np.concatenate([a.sigma0_A, a.sigma0_B]) for a in adapters]).astype(np.float32)
    d = mean.shape[0]
    assert d == cfg.d
    rng = _rng(cfg, 901)
    Dvec = rng.uniform(0.5, 1.5, d).astype(np.float32) if cfg.random_D else None
    Bf = None
    if cfg.full_B:
        g = rng.standard_normal((d, d))
        q, rr = np.linalg.qr(g)
        Bf = np.ascontiguousarray((q * np.sign(np.diag(rr))[None, :]).astype(np.float32))
    return CmaState(np.ascontiguousarray(mean), float(np.float32(cfg.step)), Bf, Dvec, int(cfg.philox_seed))


def tile_straddling_candidates(offsets: np.ndarray, tile: int = 128, limit: int = 8) -> List[int]:
    """Candidates whose token range crosses a multiple of `tile` (interesting for tiled kernels)."""
    out = []
    for k in range(len(offsets) - 1):
        a, b = int(offsets[k]), int(offsets[k + 1])
        if b > a and (a // tile) != ((b - 1) // tile):
            out.append(k)
            if len(out) >= limit:
                break
    return out


def stratified_candidates(cfg: WorkloadConfig, offsets: np.ndarray, extra: int = 4) -> List[int]:
    """A fixed subset of candidates for oracle checks at sizes the oracle cannot cover in full."""
    lens = np.diff(offsets.astype(np.int64))
    P = len(lens)
    pick = {0, P - 1, int(np.argmin(lens)), int(np.argmax(lens))}
    pick.update(tile_straddling_candidates(offsets))
    rng = _rng(cfg, 902)
    pick.update(int(v) for v in rng.integers(0, P, size=extra))
    return sorted(pick)
