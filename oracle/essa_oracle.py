"""CPU oracle for the ESSA population-projection path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 statement of what the path computes, written from the paper:

* sampling   -- a population of candidate singular-value vectors drawn from
                N(m, step^2 * C) out of one shared, seed-addressable random stream
                (Section 3, "Evolutionary optimization"; Algorithm 1, line 5);
* projection -- every candidate's adapted attention projection
                W' = W0 + B'A',  A' = U_A diag(sA) V_A^T,  B' = U_B diag(sB) V_B^T
                (Section 3, "LoRA + SVD parameterization"; Algorithm 1, line 7),
                applied to that candidate's own tokens.

The projection oracle materialises the dense per-candidate update exactly as
Algorithm 1 line 7 writes it; there is no blocking, fusion or reordering.

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
module.  It shares no code with the CUDA library and imports nothing from it.

Pins (tests/test_oracle_pins.py): Philox known-answer vectors published with the
generator; closed-form uniforms; Box-Muller radius identity, moments and a KS
test against the normal CDF; identity/orthogonal covariance special cases and the
empirical covariance; SVD round trip (sigma = singular values of the LoRA factors
reproduces B.A); the M = I special case checked with a library SVD; zero sigma
reproduces W0.x exactly; bilinearity in (sA, sB); brute-force scalar loops on tiny
shapes; linear-scan segment map vs a library search; INT4 dequantisation against
scalar loops, against the nibble table written out, and against the INT8 path when
the codes fit four bits and a row's groups share one scale.

Parity unpinned: the paper prints no worked numeric example for either function,
so both are pinned by identities, special cases, library routines and brute force
only.  The random-stream layout (which Philox counter feeds which coordinate) is
this build's own convention -- the paper only requires that any population member
be regenerable from a seed -- and is pinned by determinism/regenerability checks.
"""
from __future__ import annotations

from typing import Iterable, Optional

import numpy as np

# ---------------------------------------------------------------------------
# Shared random stream: Philox4x32-10 (Salmon, Moraes, Dror, Shaw, SC'11).
# ---------------------------------------------------------------------------
_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = 0x9E3779B9
_PHILOX_W1 = 0xBB67AE85
_MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(ctr: np.ndarray, key: np.ndarray) -> np.ndarray:
    """Ten Philox-4x32 rounds.  ctr: uint32[..., 4]; key: uint32[..., 2] -> uint32[..., 4]."""
    ctr = np.asarray(ctr, dtype=np.uint32)
    key = np.asarray(key, dtype=np.uint32)
    c0, c1, c2, c3 = (ctr[..., i].astype(np.uint64) for i in range(4))
    k0 = key[..., 0].astype(np.uint64)
    k1 = key[..., 1].astype(np.uint64)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0  # 32x32 -> 64-bit product
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> np.uint64(32), p0 & _MASK32
        hi1, lo1 = p1 >> np.uint64(32), p1 & _MASK32
        c0, c1, c2, c3 = (hi1 ^ c1 ^ k0), lo1, (hi0 ^ c3 ^ k1), lo0
        k0 = (k0 + np.uint64(_PHILOX_W0)) & _MASK32
        k1 = (k1 + np.uint64(_PHILOX_W1)) & _MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def uniform_open01(words: np.ndarray) -> np.ndarray:
    """Map 32-bit words to (0,1): u = (2*(w >> 9) + 1) * 2^-24.  Exact in fp32 and fp64."""
    w = np.asarray(words, dtype=np.uint32).astype(np.uint64)
    return (2.0 * (w >> np.uint64(9)).astype(np.float64) + 1.0) * (2.0 ** -24)


def box_muller(w_radius: np.ndarray, w_angle: np.ndarray):
    """Two standard normals from two 32-bit words (both branches of Box-Muller)."""
    rho = np.sqrt(-2.0 * np.log(uniform_open01(w_radius)))
    phi = 2.0 * np.pi * uniform_open01(w_angle)
    return rho * np.cos(phi), rho * np.sin(phi)


def candidate_stream_words(seed: int, k: np.ndarray, n_blocks: int) -> np.ndarray:
    """Philox words of candidates k: uint32[len(k), n_blocks, 4].

    Stream layout: key = (low, high) 32-bit halves of the 64-bit seed; the counter of
    block j of candidate k is (j, k, 0, 0).  Any candidate is therefore regenerable
    from <seed, k> alone, which is what lets workers exchange only seeds and rewards
    (Section 3, "Evolutionary optimization").
    """
    k = np.asarray(k, dtype=np.uint32).reshape(-1)
    ctr = np.zeros((k.shape[0], n_blocks, 4), dtype=np.uint32)
    ctr[..., 0] = np.arange(n_blocks, dtype=np.uint32)[None, :]
    ctr[..., 1] = k[:, None]
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    return philox4x32_10(ctr, np.broadcast_to(key, ctr.shape[:-1] + (2,)))


def standard_normals(seed: int, k: np.ndarray, d: int) -> np.ndarray:
    """z[len(k), d] in fp64: block j gives coordinates 4j..4j+3 = (z0,z1 from words 0,1; z2,z3 from words 2,3)."""
    nb = (d + 3) // 4
    w = candidate_stream_words(seed, k, nb)
    z = np.empty(w.shape[:2] + (4,), dtype=np.float64)
    z[..., 0], z[..., 1] = box_muller(w[..., 0], w[..., 1])
    z[..., 2], z[..., 3] = box_muller(w[..., 2], w[..., 3])
    return z.reshape(w.shape[0], nb * 4)[:, :d]


def sample_population(mean, step: float, Bfactor, Dvec, seed: int, P: int, k_begin: int = 0) -> np.ndarray:
    """sigma[P, d] (fp64): candidate k = mean + step * Bfactor @ (Dvec * z_k), i.e. a draw from
    N(mean, step^2 * C) with C = Bfactor diag(Dvec)^2 Bfactor^T (Section 3: N(m_t, sigma_t^2 C_t)).
    Bfactor None means identity, Dvec None means ones.
    """
    mean = np.asarray(mean, dtype=np.float64)
    d = mean.shape[0]
    z = standard_normals(seed, np.arange(k_begin, k_begin + P), d)
    w = z if Dvec is None else z * np.asarray(Dvec, dtype=np.float64)[None, :]
    if Bfactor is not None:
        w = w @ np.asarray(Bfactor, dtype=np.float64).T
    return mean[None, :] + float(step) * w


def top_alpha_index(n_factors: int, rank: int, alpha) -> np.ndarray:
    """Columns of the optimised singular values when only the top-alpha fraction of each factor's `rank` values is
    exposed to the optimizer (Section 3, "LoRA + SVD parameterization"); the count per factor is alpha * rank
    rounded DOWN (the caption of the rank / population / alpha sensitivity figure: rank 8 with alpha = 0.1 leaves
    zero trainable values).  The table holds the factors' slices one after the other, leading values first."""
    from fractions import Fraction
    per = int(Fraction(str(alpha)) * rank // 1)
    return np.array([f * rank + j for f in range(n_factors) for j in range(per)], dtype=np.int64)


def sample_population_masked(frozen, index, mean_t, step: float, Bfactor_t, Dvec_t, seed: int, P: int,
                             k_begin: int = 0) -> np.ndarray:
    """sigma[P, d] (fp64) when only the coordinates `index` are optimised: those columns are a draw from
    N(mean_t, step^2 C_t) taken from the shared stream in the optimised vector's own numbering, every other column
    keeps its frozen value (Section 3: the rest of the singular values stay as they were after SFT)."""
    frozen = np.asarray(frozen, dtype=np.float64)
    sigma = np.tile(frozen[None, :], (P, 1))
    index = np.asarray(index, dtype=np.int64)
    if index.size:
        sigma[:, index] = sample_population(mean_t, step, Bfactor_t, Dvec_t, seed, P, k_begin)
    return sigma


# ---------------------------------------------------------------------------
# Projection.
# ---------------------------------------------------------------------------
def candidate_of_token(offsets, T: int) -> np.ndarray:
    """cand[t] = k with offsets[k] <= t < offsets[k+1], by linear scan (empty segments own nothing)."""
    offsets = np.asarray(offsets, dtype=np.int64)
    cand = np.full(T, -1, dtype=np.int64)
    for k in range(offsets.shape[0] - 1):
        cand[offsets[k]:offsets[k + 1]] = k
    return cand


def dequantize_int8(q, scale) -> np.ndarray:
    """W0[o,i] = q[o,i] * scale[o] in fp64 (weight-only INT8 storage of the frozen base)."""
    return np.asarray(q).astype(np.float64) * np.asarray(scale).astype(np.float64)[:, None]


def dequantize_int4(packed, scale, group: int = 128) -> np.ndarray:
    """W0[o,i] = q[o,i] * scale[o, i // group] in fp64 (weight-only INT4 storage of the frozen base, group-wise scales).

    packed is uint8 [m, n/2]: byte j of a row holds the codes of input features 2j (low nibble) and 2j+1 (high nibble),
    each a 4-bit two's-complement integer in [-8, 7]; scale is fp16 [m, n/group].  The paper only names the precision
    ("INT4", Section 5 precision study); this storage scheme is the build's reading of it."""
    packed = np.asarray(packed, dtype=np.uint8)
    m, half = packed.shape
    codes = np.empty((m, 2 * half), dtype=np.int64)
    codes[:, 0::2] = packed & 0x0F
    codes[:, 1::2] = packed >> 4
    codes = np.where(codes >= 8, codes - 16, codes)
    sc = np.asarray(scale).astype(np.float64)
    return codes.astype(np.float64) * np.repeat(sc, group, axis=1)


def reconstruct_factors(U_A, V_A, U_B, V_B, sA, sB):
    """The two LoRA factors of one candidate, as Algorithm 1 line 7 writes them:
    A' = U_A diag(sA) V_A^T (r x n), B' = U_B diag(sB) V_B^T (m x r)."""
    U_A, V_A, U_B, V_B = (np.asarray(a, dtype=np.float64) for a in (U_A, V_A, U_B, V_B))
    A_prime = U_A @ np.diag(np.asarray(sA, dtype=np.float64)) @ V_A.T
    B_prime = U_B @ np.diag(np.asarray(sB, dtype=np.float64)) @ V_B.T
    return A_prime, B_prime


def reconstruct_delta_w(U_A, V_A, U_B, V_B, sA, sB) -> np.ndarray:
    """Dense update of one candidate, as Algorithm 1 line 7 writes it: DeltaW = B' A' (m x n)."""
    A_prime, B_prime = reconstruct_factors(U_A, V_A, U_B, V_B, sA, sB)
    return B_prime @ A_prime


def apply_projection(W0, U_A, V_A, U_B, V_B, x, offsets, sigma, sA_col: int, sB_col: int, rank: int,
                     candidates: Optional[Iterable[int]] = None) -> np.ndarray:
    """y[T, m] (fp64): token t of candidate k gets y_t = (W0 + DeltaW_k) x_t.

    sigma is the population table [P, >= max(sA_col, sB_col) + rank]; candidate k reads
    sA = sigma[k, sA_col : sA_col + rank], sB likewise.  With `candidates`, only those
    candidates' rows are computed and all other rows are NaN.
    """
    W0 = np.asarray(W0, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    sigma = np.asarray(sigma, dtype=np.float64)
    offsets = np.asarray(offsets, dtype=np.int64)
    T, m = x.shape[0], W0.shape[0]
    y = np.full((T, m), np.nan, dtype=np.float64)
    ks = range(offsets.shape[0] - 1) if candidates is None else candidates
    for k in ks:
        a, b = int(offsets[k]), int(offsets[k + 1])
        if b <= a:
            continue
        dW = reconstruct_delta_w(U_A, V_A, U_B, V_B, sigma[k, sA_col:sA_col + rank], sigma[k, sB_col:sB_col + rank])
        W_prime = W0 + dW
        y[a:b] = x[a:b] @ W_prime.T
    return y


def relative_error(got, want) -> float:
    """max_i |g_i - o_i| / max(|o_i|, rms(o)) -- the projection parity metric (rows with NaN in `want` ignored)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    mask = ~np.isnan(want)
    if not mask.any():
        return 0.0
    w = want[mask]
    g = got[mask]
    rms = np.sqrt(np.mean(w * w))
    denom = np.maximum(np.abs(w), rms if rms > 0 else 1.0)
    return float(np.max(np.abs(g - w) / denom))
