"""Pins for the CPU oracle: every check here compares the oracle against something other than
itself -- published vectors, closed forms, invariants, library routines, or scalar brute force."""
import math

import numpy as np
import pytest
import scipy.stats

from oracle import essa_oracle as orc


# ------------------------------------------------------------------ Philox / uniforms / normals
def test_philox_known_answers(philox_kat):
    assert len(philox_kat) >= 3
    for ctr, key, want in philox_kat:
        got = orc.philox4x32_10(np.array(ctr, dtype=np.uint32), np.array(key, dtype=np.uint32))
        assert [int(v) for v in got] == want


def test_philox_batched_equals_single(philox_kat):
    ctr = np.array([c for c, _, _ in philox_kat], dtype=np.uint32)
    key = np.array([k for _, k, _ in philox_kat], dtype=np.uint32)
    want = np.array([w for _, _, w in philox_kat], dtype=np.uint32)
    assert np.array_equal(orc.philox4x32_10(ctr, key), want)


def test_philox_is_a_bijection_on_a_counter_range():
    # A block cipher in counter mode never repeats an output block for distinct counters.
    ctr = np.zeros((4096, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(4096)
    out = orc.philox4x32_10(ctr, np.broadcast_to(np.array([7, 9], dtype=np.uint32), (4096, 2)))
    assert len({tuple(r) for r in out.tolist()}) == 4096


def test_uniform_closed_form_values():
    u = orc.uniform_open01(np.array([0, 0xFFFFFFFF, 0x80000000, 0x1FF, 0x200], dtype=np.uint32))
    assert u[0] == 2.0 ** -24
    assert u[1] == 1.0 - 2.0 ** -24
    assert u[2] == 0.5 + 2.0 ** -24
    assert u[3] == 2.0 ** -24  # low 9 bits are dropped
    assert u[4] == 3.0 * 2.0 ** -24
    assert np.all(u.astype(np.float32).astype(np.float64) == u)  # representable in fp32


def test_box_muller_radius_identity_and_bound():
    rng = np.random.default_rng(5)
    w0 = rng.integers(0, 2 ** 32, size=10000, dtype=np.uint64).astype(np.uint32)
    w1 = rng.integers(0, 2 ** 32, size=10000, dtype=np.uint64).astype(np.uint32)
    z0, z1 = orc.box_muller(w0, w1)
    u0 = (2 * (w0.astype(np.int64) >> 9) + 1) / 2.0 ** 24
    np.testing.assert_allclose(z0 ** 2 + z1 ** 2, -2.0 * np.log(u0), rtol=1e-12)
    # angle comes from the second word: atan2 recovers it
    u1 = (2 * (w1.astype(np.int64) >> 9) + 1) / 2.0 ** 24
    ang = np.mod(np.arctan2(z1, z0), 2 * np.pi)
    np.testing.assert_allclose(ang, 2 * np.pi * u1, atol=1e-9)
    assert np.max(np.abs(np.concatenate([z0, z1]))) <= math.sqrt(-2.0 * math.log(2.0 ** -24)) + 1e-12


def test_extreme_words_give_extreme_radius():
    z0, z1 = orc.box_muller(np.array([0], dtype=np.uint32), np.array([0], dtype=np.uint32))
    rho = math.sqrt(-2 * math.log(2.0 ** -24))
    phi = 2 * math.pi * 2.0 ** -24
    assert abs(z0[0] - rho * math.cos(phi)) < 1e-12 and abs(z1[0] - rho * math.sin(phi)) < 1e-12


def test_normals_moments_and_ks():
    z = orc.standard_normals(seed=12345, k=np.arange(2048), d=512).reshape(-1)  # ~1e6 draws
    n = z.size
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 5 * math.sqrt(2.0 / n)
    assert abs(scipy.stats.kurtosis(z, fisher=False) - 3.0) < 0.02
    assert abs(scipy.stats.skew(z)) < 0.01
    ks = scipy.stats.kstest(z[:200000], "norm")
    assert ks.pvalue > 1e-3
    # the four lanes of a block and neighbouring candidates are uncorrelated
    zz = orc.standard_normals(seed=12345, k=np.arange(4096), d=8)
    c = np.corrcoef(zz.T)
    assert np.max(np.abs(c - np.eye(8))) < 0.08


def test_stream_layout_regenerable_from_seed_and_index():
    # Any member can be regenerated alone, in any order, from <seed, k>.
    full = orc.sample_population(np.zeros(13), 1.0, None, None, seed=99, P=17)
    for k in (16, 0, 5):
        one = orc.sample_population(np.zeros(13), 1.0, None, None, seed=99, P=1, k_begin=k)
        assert np.array_equal(one[0], full[k])
    # different seeds and different members differ; the high seed word matters
    a = orc.standard_normals(1, np.arange(2), 8)
    assert not np.array_equal(a[0], a[1])
    assert not np.array_equal(a, orc.standard_normals(2, np.arange(2), 8))
    assert not np.array_equal(a, orc.standard_normals(1 + (1 << 32), np.arange(2), 8))
    # d not a multiple of 4: prefix property (tail of the last block is discarded)
    assert np.array_equal(orc.standard_normals(1, np.arange(2), 7), orc.standard_normals(1, np.arange(2), 8)[:, :7])


def test_stream_counter_convention():
    w = orc.candidate_stream_words(seed=(0x299F31D0 << 32) | 0xA4093822, k=np.array([0x85A308D3]), n_blocks=3)
    # block j of candidate k is Philox(ctr=(j,k,0,0), key=(seed_lo, seed_hi))
    for j in range(3):
        ref = orc.philox4x32_10(np.array([j, 0x85A308D3, 0, 0], dtype=np.uint32),
                                np.array([0xA4093822, 0x299F31D0], dtype=np.uint32))
        assert np.array_equal(w[0, j], ref)


# ------------------------------------------------------------------ shaping to N(m, step^2 C)
def test_identity_covariance_reduces_to_mean_plus_step_z():
    mean = np.linspace(-1, 1, 16)
    z = orc.standard_normals(0, np.arange(4), 16)
    got = orc.sample_population(mean, 0.1, None, None, 0, 4)
    np.testing.assert_allclose(got, mean[None] + 0.1 * z, rtol=0, atol=1e-15)
    got_I = orc.sample_population(mean, 0.1, np.eye(16), np.ones(16), 0, 4)
    np.testing.assert_allclose(got_I, got, rtol=0, atol=1e-15)


def test_zero_step_returns_mean():
    mean = np.arange(8.0)
    assert np.array_equal(orc.sample_population(mean, 0.0, None, None, 3, 5), np.tile(mean, (5, 1)))


def test_orthogonal_factor_preserves_norm_and_matches_matvec():
    rng = np.random.default_rng(0)
    d = 24
    Q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    D = rng.uniform(0.5, 1.5, d)
    z = orc.standard_normals(7, np.arange(6), d)
    s = orc.sample_population(np.zeros(d), 1.0, Q, D, 7, 6)
    np.testing.assert_allclose(np.linalg.norm(s, axis=1), np.linalg.norm(z * D, axis=1), rtol=1e-12)
    for k in range(6):  # explicit scalar matvec, row-major B[i][j]
        want = [sum(Q[i, j] * D[j] * z[k, j] for j in range(d)) for i in range(d)]
        np.testing.assert_allclose(s[k], want, rtol=1e-12, atol=1e-14)


def test_non_symmetric_factor_orientation():
    # B[i][j] multiplies coordinate j of D*z and lands in coordinate i (not the transpose).
    d = 4
    Bf = np.zeros((d, d))
    Bf[2, 0] = 1.0
    z = orc.standard_normals(1, np.arange(1), d)
    s = orc.sample_population(np.zeros(d), 2.0, Bf, np.array([3.0, 1, 1, 1]), 1, 1)
    np.testing.assert_allclose(s[0], [0, 0, 2.0 * 3.0 * z[0, 0], 0], rtol=1e-14)


def test_empirical_covariance_matches_step2_BD2Bt():
    rng = np.random.default_rng(1)
    d, P = 6, 200000
    Bf = rng.standard_normal((d, d))
    D = rng.uniform(0.5, 1.5, d)
    mean = rng.standard_normal(d)
    s = orc.sample_population(mean, 0.3, Bf, D, 2024, P)
    C = 0.09 * Bf @ np.diag(D ** 2) @ Bf.T
    emp = np.cov(s.T)
    assert np.max(np.abs(emp - C)) < 6 * np.max(np.abs(C)) / math.sqrt(P) * 2
    assert np.max(np.abs(s.mean(axis=0) - mean)) < 6 * math.sqrt(np.max(np.diag(C)) / P)


# ------------------------------------------------------------------ reconstruction / projection
def _random_problem(rng, m, n, r, P, lens=None):
    W0 = rng.standard_normal((m, n)) / math.sqrt(n)
    U_A, _ = np.linalg.qr(rng.standard_normal((r, r)))
    V_A, _ = np.linalg.qr(rng.standard_normal((n, r)))
    U_B, _ = np.linalg.qr(rng.standard_normal((m, r)))
    V_B, _ = np.linalg.qr(rng.standard_normal((r, r)))
    lens = rng.integers(0, 5, size=P) if lens is None else np.asarray(lens)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    x = rng.standard_normal((int(off[-1]), n))
    sigma = rng.standard_normal((P, 2 * r + 3))
    return W0, U_A, V_A, U_B, V_B, x, off, sigma


def test_svd_round_trip_reproduces_lora_product():
    # With sigma equal to the singular values of the LoRA factors, B'A' = BA (Section 3).
    rng = np.random.default_rng(2)
    m, n, r = 40, 56, 8
    A = rng.standard_normal((r, n))
    B = rng.standard_normal((m, r))
    U_A, sA, V_At = np.linalg.svd(A, full_matrices=False)
    U_B, sB, V_Bt = np.linalg.svd(B, full_matrices=False)
    dW = orc.reconstruct_delta_w(U_A, V_At.T, U_B, V_Bt.T, sA, sB)
    np.testing.assert_allclose(dW, B @ A, rtol=0, atol=1e-12)
    # and through the full projection: y = (W0 + BA) x
    W0 = rng.standard_normal((m, n))
    x = rng.standard_normal((5, n))
    sigma = np.concatenate([sA, sB])[None, :]
    y = orc.apply_projection(W0, U_A, V_At.T, U_B, V_Bt.T, x, [0, 5], sigma, 0, r, r)
    np.testing.assert_allclose(y, x @ (W0 + B @ A).T, rtol=0, atol=1e-11)


def test_core_identity_special_case_has_known_singular_values():
    # U_A = V_B makes V_B^T U_A = I, so DeltaW = U_B diag(sB*sA) V_A^T with orthonormal U_B, V_A:
    # its singular values are |sA*sB| -- checked with a library SVD.
    rng = np.random.default_rng(3)
    m, n, r = 30, 44, 6
    _, U_A, V_A, U_B, _, _, _, _ = _random_problem(rng, m, n, r, 1)
    sA = rng.standard_normal(r)
    sB = rng.standard_normal(r)
    dW = orc.reconstruct_delta_w(U_A, V_A, U_B, U_A, sA, sB)
    sv = np.linalg.svd(dW, compute_uv=False)
    np.testing.assert_allclose(sv[:r], np.sort(np.abs(sA * sB))[::-1], rtol=1e-10, atol=1e-12)
    assert np.all(sv[r:] < 1e-12)
    np.testing.assert_allclose(dW, U_B @ np.diag(sA * sB) @ V_A.T, atol=1e-13)


def test_delta_w_has_rank_at_most_r_and_lives_in_frozen_subspaces():
    rng = np.random.default_rng(4)
    W0, U_A, V_A, U_B, V_B, _, _, sigma = _random_problem(rng, 20, 28, 4, 1)
    dW = orc.reconstruct_delta_w(U_A, V_A, U_B, V_B, sigma[0, :4], sigma[0, 4:8])
    assert np.linalg.matrix_rank(dW, tol=1e-10) <= 4
    # column space inside span(U_B), row space inside span(V_A)
    np.testing.assert_allclose(U_B @ (U_B.T @ dW), dW, atol=1e-12)
    np.testing.assert_allclose((dW @ V_A) @ V_A.T, dW, atol=1e-12)


def test_zero_sigma_reproduces_base_output_exactly():
    rng = np.random.default_rng(5)
    W0, U_A, V_A, U_B, V_B, x, off, sigma = _random_problem(rng, 24, 32, 4, 3, lens=[2, 3, 1])
    base = x @ W0.T
    sA0 = sigma.copy(); sA0[:, 0:4] = 0.0
    sB0 = sigma.copy(); sB0[:, 4:8] = 0.0
    # the reconstructed update is exactly the zero matrix, so W' is W0 bit for bit ...
    assert not np.any(orc.reconstruct_delta_w(U_A, V_A, U_B, V_B, sA0[0, 0:4], sA0[0, 4:8]))
    assert not np.any(orc.reconstruct_delta_w(U_A, V_A, U_B, V_B, sB0[0, 0:4], sB0[0, 4:8]))
    # ... and the output is the base output (segment-wise products: same summation order)
    seg = np.concatenate([x[off[k]:off[k + 1]] @ W0.T for k in range(3)])
    assert np.array_equal(orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, sA0, 0, 4, 4), seg)
    assert np.array_equal(orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, sB0, 0, 4, 4), seg)
    np.testing.assert_allclose(seg, base, rtol=0, atol=1e-13)


def test_bilinear_in_singular_values():
    rng = np.random.default_rng(6)
    W0, U_A, V_A, U_B, V_B, x, off, sigma = _random_problem(rng, 24, 32, 4, 2, lens=[3, 2])
    r = 4
    f = lambda s: orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, s, 0, r, r) - x @ W0.T
    s1 = sigma.copy()
    s2 = sigma.copy(); s2[:, 0:r] = rng.standard_normal((2, r))
    s12 = sigma.copy(); s12[:, 0:r] = s1[:, 0:r] + s2[:, 0:r]
    np.testing.assert_allclose(f(s12), f(s1) + f(s2), atol=1e-12)  # additive in sA
    sc = sigma.copy(); sc[:, r:2 * r] *= -2.5
    np.testing.assert_allclose(f(sc), -2.5 * f(sigma), atol=1e-12)  # homogeneous in sB
    e = np.zeros_like(sigma); e[:, 1] = 1.0; e[:, r + 2] = 1.0  # single (i,j) pair: rank-one response
    M = V_B.T @ U_A
    want = np.outer(x @ V_A[:, 1], U_B[:, 2]) * M[2, 1]
    np.testing.assert_allclose(f(e), want, atol=1e-12)


def test_brute_force_factored_formula_scalar_loops():
    # y = W0 x + U_B (sB * (M (sA * (V_A^T x)))), M = V_B^T U_A, in pure-Python scalar loops.
    rng = np.random.default_rng(7)
    m, n, r, P = 7, 9, 3, 3
    W0, U_A, V_A, U_B, V_B, x, off, sigma = _random_problem(rng, m, n, r, P, lens=[2, 0, 3])
    sA_col, sB_col = 1, 5
    sigma = rng.standard_normal((P, 9))
    got = orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, sigma, sA_col, sB_col, r)
    M = [[sum(V_B[l][j] * U_A[l][i] for l in range(r)) for i in range(r)] for j in range(r)]
    for k in range(P):
        for t in range(off[k], off[k + 1]):
            p = [sum(V_A[i][a] * x[t][i] for i in range(n)) for a in range(r)]
            q = [sigma[k][sA_col + a] * p[a] for a in range(r)]
            v = [sum(M[j][a] * q[a] for a in range(r)) for j in range(r)]
            u = [sigma[k][sB_col + j] * v[j] for j in range(r)]
            for o in range(m):
                want = sum(W0[o][i] * x[t][i] for i in range(n)) + sum(U_B[o][j] * u[j] for j in range(r))
                assert abs(got[t][o] - want) < 1e-12


def test_each_candidate_uses_its_own_sigma_and_tokens():
    rng = np.random.default_rng(8)
    W0, U_A, V_A, U_B, V_B, x, off, sigma = _random_problem(rng, 10, 12, 2, 4, lens=[1, 4, 0, 2])
    full = orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, sigma, 0, 2, 2)
    for k in range(4):
        a, b = off[k], off[k + 1]
        alone = orc.apply_projection(W0, U_A, V_A, U_B, V_B, x[a:b], [0, b - a], sigma[k:k + 1], 0, 2, 2)
        assert np.array_equal(alone, full[a:b])
    sub = orc.apply_projection(W0, U_A, V_A, U_B, V_B, x, off, sigma, 0, 2, 2, candidates=[1])
    assert np.array_equal(sub[off[1]:off[2]], full[off[1]:off[2]]) and np.isnan(sub[0]).all()


def test_segment_map_vs_library_search():
    rng = np.random.default_rng(9)
    for _ in range(50):
        lens = rng.integers(0, 4, size=rng.integers(1, 12))
        off = np.concatenate([[0], np.cumsum(lens)])
        T = int(off[-1])
        cand = orc.candidate_of_token(off, T)
        want = np.searchsorted(off, np.arange(T), side="right") - 1
        assert np.array_equal(cand, want)
        assert np.all(np.diff(cand) >= 0)
        assert np.array_equal(np.bincount(cand, minlength=len(lens)) if T else np.zeros(len(lens), int), lens)


def test_int8_dequant_identity_and_agreement_with_plain_weights():
    rng = np.random.default_rng(10)
    q = rng.integers(-127, 128, size=(6, 8)).astype(np.int8)
    scale = rng.uniform(0.001, 0.01, 6).astype(np.float16)
    W = orc.dequantize_int8(q, scale)
    for o in range(6):
        for i in range(8):
            assert W[o, i] == float(q[o, i]) * float(scale[o])  # exact in fp64
    assert np.array_equal(orc.dequantize_int8(q, np.ones(6, np.float16)), q.astype(np.float64))


def test_dimension_bookkeeping():
    # d = layers * 4 matrices * 2 factors * r  (Appendix "Countdown": 28 * 4 * 2r ~ 1.8K for r = 8)
    assert 28 * 4 * 2 * 8 == 1792
    from paper_2507_04453_b200 import workloads as wl
    assert wl.CONFIGS["2"].d == 128 and wl.CONFIGS["4"].d == 256 and wl.CONFIGS["5a"].d == 512
    assert wl.CONFIGS["1"].d == 16
    assert wl.CONFIGS["2"].sigma_cols(3) == (96, 112)


def test_relative_error_metric():
    want = np.array([[1.0, -2.0], [0.0, 4.0]])
    got = want + np.array([[0.1, 0.0], [0.0, 0.0]])
    rms = math.sqrt(21 / 4)
    assert abs(orc.relative_error(got, want) - 0.1 / rms) < 1e-15


# ------------------------------------------------------------------ top-alpha selection (Section 3; sensitivity-figure caption)
def test_top_alpha_rounds_down_as_the_paper_states():
    # the paper's own example: rank 8 with alpha = 0.1 leaves zero trainable singular values
    assert orc.top_alpha_index(8, 8, 0.1).size == 0
    # decimal fractions are taken exactly: 0.29 * 100 is 29, not floor(28.999999999999996)
    assert orc.top_alpha_index(1, 100, 0.29).size == 29
    # alpha = 1: every coordinate, in order; alpha = 0.5 of rank 4 on three factors: the two leading ones of each slice
    assert np.array_equal(orc.top_alpha_index(3, 4, 1.0), np.arange(12))
    assert np.array_equal(orc.top_alpha_index(3, 4, 0.5), np.array([0, 1, 4, 5, 8, 9]))
    assert np.array_equal(orc.top_alpha_index(2, 16, 0.3), np.array([0, 1, 2, 3, 16, 17, 18, 19]))  # floor(4.8) = 4


def test_masked_population_special_cases():
    rng = np.random.default_rng(5)
    d, P, seed = 24, 7, (3 << 32) + 11
    frozen = rng.standard_normal(d)
    # nothing optimised: every candidate is the frozen vector
    assert np.array_equal(orc.sample_population_masked(frozen, [], None, 0.3, None, None, seed, P), np.tile(frozen, (P, 1)))
    # everything optimised: the unmasked draw, whatever `frozen` holds
    mean = rng.standard_normal(d)
    Bf = rng.standard_normal((d, d)) / 5
    Dv = rng.uniform(0.5, 1.5, d)
    full = orc.sample_population(mean, 0.3, Bf, Dv, seed, P)
    assert np.array_equal(orc.sample_population_masked(frozen, np.arange(d), mean, 0.3, Bf, Dv, seed, P), full)
    # a proper subset: the optimised columns are the draw of the SMALL problem (its own stream numbering), scattered;
    # the others are untouched; a permuted index scatters the same draw to the permuted columns
    idx = orc.top_alpha_index(3, 8, 0.5)          # 12 of 24 columns
    dt = idx.size
    small = orc.sample_population(mean[:dt], 0.3, Bf[:dt, :dt], Dv[:dt], seed, P, k_begin=2)
    got = orc.sample_population_masked(frozen, idx, mean[:dt], 0.3, Bf[:dt, :dt], Dv[:dt], seed, P, k_begin=2)
    assert np.array_equal(got[:, idx], small)
    rest = np.setdiff1d(np.arange(d), idx)
    assert np.array_equal(got[:, rest], np.tile(frozen[rest], (P, 1)))
    perm = idx[::-1].copy()
    got_p = orc.sample_population_masked(frozen, perm, mean[:dt], 0.3, Bf[:dt, :dt], Dv[:dt], seed, P, k_begin=2)
    assert np.array_equal(got_p[:, perm], small)
    # moments of the optimised columns (diagonal case): mean m_i, standard deviation step * D_i
    many = orc.sample_population_masked(frozen, idx, mean[:dt], 0.5, None, Dv[:dt], 9, 20000)
    assert np.allclose(many[:, idx].mean(axis=0), mean[:dt], atol=0.03)
    assert np.allclose(many[:, idx].std(axis=0), 0.5 * Dv[:dt], rtol=0.03)


# ------------------------------------------------------------------ candidate reconstruction (Algorithm 1, line 7)
def test_reconstructed_factors_round_trip_the_svd():
    """With the singular values the thin SVD of a LoRA factor produced, the reconstruction is that factor again
    (library SVD as the independent routine); scaling one singular value scales exactly its rank-one term."""
    rng = np.random.default_rng(17)
    m, n, r = 24, 40, 6
    A = rng.standard_normal((r, n))
    Bm = rng.standard_normal((m, r))
    UA, SA, VAt = np.linalg.svd(A, full_matrices=False)    # A = UA diag(SA) VAt, UA r x r, VAt r x n
    UB, SB, VBt = np.linalg.svd(Bm, full_matrices=False)   # B = UB diag(SB) VBt, UB m x r, VBt r x r
    A2, B2 = orc.reconstruct_factors(UA, VAt.T, UB, VBt.T, SA, SB)
    assert np.allclose(A2, A, atol=1e-12) and np.allclose(B2, Bm, atol=1e-12)
    assert np.allclose(orc.reconstruct_delta_w(UA, VAt.T, UB, VBt.T, SA, SB), Bm @ A, atol=1e-11)
    s2 = SA.copy(); s2[2] *= 3.0
    A3, _ = orc.reconstruct_factors(UA, VAt.T, UB, VBt.T, s2, SB)
    assert np.allclose(A3 - A, 2.0 * SA[2] * np.outer(UA[:, 2], VAt[2, :]), atol=1e-12)
    # element by element, scalar loops
    A4 = np.zeros((r, n))
    for i in range(r):
        for c in range(n):
            A4[i, c] = sum(UA[i, j] * SA[j] * VAt[j, c] for j in range(r))
    assert np.allclose(A4, A2, atol=1e-12)


# ---------------------------------------------------------------------------------------------- INT4 storage
def test_int4_dequant_scalar_loops_and_nibble_table():
    rng = np.random.default_rng(41)
    m, n, group = 5, 256, 128
    packed = rng.integers(0, 256, size=(m, n // 2), dtype=np.uint8)
    scale = rng.uniform(0.01, 0.2, size=(m, n // group)).astype(np.float16)
    got = orc.dequantize_int4(packed, scale, group)
    table = [0, 1, 2, 3, 4, 5, 6, 7, -8, -7, -6, -5, -4, -3, -2, -1]  # 4-bit two's complement, written out
    for o in range(m):
        for i in range(n):
            byte = int(packed[o, i // 2])
            nib = (byte >> 4) if (i & 1) else (byte & 15)
            assert got[o, i] == table[nib] * float(scale[o, i // group])


def test_int4_agrees_with_int8_when_codes_fit_and_groups_share_a_scale():
    rng = np.random.default_rng(42)
    m, n = 6, 384
    q = rng.integers(-8, 8, size=(m, n)).astype(np.int8)
    row_scale = rng.uniform(0.01, 0.1, size=m).astype(np.float16)
    u = (q.astype(np.int16) & 15).astype(np.uint8)
    packed = (u[:, 0::2] | (u[:, 1::2] << 4)).astype(np.uint8)
    w4 = orc.dequantize_int4(packed, np.repeat(row_scale[:, None], n // 128, axis=1))
    w8 = orc.dequantize_int8(q, row_scale)
    assert np.array_equal(w4, w8)


def test_int4_workload_quantiser_round_trip_error_bound():
    """The generator's codes stay in [-7, 7] and the stored pair reproduces the weight to half a step per entry."""
    rng = np.random.default_rng(43)
    W = (rng.standard_normal((8, 512)) / np.sqrt(512)).astype(np.float32)
    from paper_2507_04453_b200 import workloads as wl
    packed, scale = wl.quantize_int4_groupwise(W)
    assert packed.shape == (8, 256) and scale.shape == (8, 4) and scale.dtype == np.float16
    deq = orc.dequantize_int4(packed, scale)
    step = np.repeat(scale.astype(np.float64), 128, axis=1)
    # half a step, plus the clip at +-7 when the fp16 rounding made the scale a little smaller than max / 7
    assert np.all(np.abs(deq - W) <= (0.5 + 7 * 2.0 ** -11) * step + 1e-12)
    assert np.max(np.abs(deq / step)) <= 7
