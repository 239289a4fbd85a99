"""Pins of the CMA-ES update oracle (oracle/cma_oracle.py) against what the mathematics fixes (CPU only).

The paper prints no formulas and no worked example for the update (Section 3, "Evolutionary optimization";
Algorithm 1, the CMA-ES update after the <seed, reward> exchange), so the oracle is pinned by closed forms,
special cases that reduce to a library routine, invariances that rank-based selection must have, the
stationarity of the evolution paths and of C under neutral selection, and convergence on the sphere function.
"""
import dataclasses
import math

import numpy as np
import pytest

from oracle import cma_oracle as cma


def random_spd(rng, n, cond=20.0):
    q, _ = np.linalg.qr(rng.standard_normal((n, n)))
    ev = np.exp(rng.uniform(0.0, math.log(cond), n))
    return (q * ev) @ q.T


def test_weights_closed_form():
    for lam in (2, 3, 4, 12, 48, 400):
        p = cma.default_params(7, lam)
        mu = lam // 2
        assert p.mu == mu and p.weights.shape == (mu,)
        assert abs(p.weights.sum() - 1.0) < 1e-14
        assert np.all(p.weights > 0) and np.all(np.diff(p.weights) < 0 if mu > 1 else True)
        # sum_{i<=mu} (ln((lam+1)/2) - ln i) = mu ln((lam+1)/2) - ln(mu!)
        total = mu * math.log((lam + 1) / 2.0) - math.lgamma(mu + 1)
        assert abs(p.weights[0] - math.log((lam + 1) / 2.0) / total) < 1e-13
        assert abs(p.mu_eff - 1.0 / sum(w * w for w in p.weights)) < 1e-12
        assert 1.0 <= p.mu_eff <= mu + 1e-12
    p4 = cma.default_params(5, 4)  # by hand: w' = (ln 2.5, ln 1.25)
    a, b = math.log(2.5), math.log(1.25)
    assert np.allclose(p4.weights, [a / (a + b), b / (a + b)], rtol=0, atol=1e-15)


def test_default_parameters_are_in_range():
    for n, lam in ((2, 6), (16, 4), (128, 256), (512, 128), (1792, 48)):
        p = cma.default_params(n, lam)
        assert 0 < p.c_sigma < 1 and 0 < p.c_c <= 1 and p.d_sigma >= 1
        assert 0 < p.c_1 < 1 and 0 <= p.c_mu <= 1 - p.c_1
        # E|N(0,I_n)| = sqrt(2) Gamma((n+1)/2) / Gamma(n/2); the tutorial's approximation is good to ~1e-3 relative
        exact = math.sqrt(2.0) * math.exp(math.lgamma((n + 1) / 2.0) - math.lgamma(n / 2.0))
        assert abs(p.chi_n - exact) / exact < 2e-3


def test_single_parent_moves_the_mean_onto_the_best_candidate():
    rng = np.random.default_rng(1)
    st = cma.init_state(rng.standard_normal(5), 0.3, lam=2)
    x = st.mean[None, :] + 0.3 * rng.standard_normal((2, 5))
    new = cma.tell(st, x, [0.1, 0.7])
    assert np.allclose(new.mean, x[1], atol=1e-15)
    new = cma.tell(st, x, [0.7, 0.1])
    assert np.allclose(new.mean, x[0], atol=1e-15)


def test_rewards_are_maximised_and_ties_keep_order():
    assert list(cma.rank_rewards([1.0, 3.0, 2.0])) == [1, 2, 0]
    assert list(cma.rank_rewards([2.0, 2.0, 5.0, 2.0])) == [2, 0, 1, 3]
    assert list(cma.rank_rewards([float("nan"), 1.0, -np.inf])) == [1, 0, 2] or list(cma.rank_rewards([float("nan"), 1.0, -np.inf]))[0] == 1


def test_update_depends_on_reward_ranks_only():
    rng = np.random.default_rng(2)
    n, lam = 6, 10
    st = cma.init_state(rng.standard_normal(n), 0.5, lam, C0=random_spd(rng, n))
    x = cma.ask_from_normals(st, rng.standard_normal((lam, n)))
    f = rng.standard_normal(lam)
    ref = cma.tell(st, x, f)
    for g in (np.exp(f), f ** 3, 5.0 * f - 2.0, np.arctan(f)):
        out = cma.tell(st, x, g)
        for name in ("mean", "C", "p_sigma", "p_c"):
            assert np.array_equal(getattr(out, name), getattr(ref, name))
        assert out.sigma == ref.sigma


def test_zero_learning_rates_leave_the_covariance_alone():
    rng = np.random.default_rng(3)
    n, lam = 5, 8
    p = dataclasses.replace(cma.default_params(n, lam), c_1=0.0, c_mu=0.0)
    C0 = random_spd(rng, n)
    st = cma.init_state(rng.standard_normal(n), 0.4, lam, C0=C0, params=p)
    x = cma.ask_from_normals(st, rng.standard_normal((lam, n)))
    new = cma.tell(st, x, rng.standard_normal(lam))
    assert np.array_equal(new.C, C0)
    p0 = dataclasses.replace(cma.default_params(n, lam), c_sigma=0.0)
    st0 = cma.init_state(rng.standard_normal(n), 0.4, lam, params=p0)
    new0 = cma.tell(st0, x, rng.standard_normal(lam))
    assert new0.sigma == 0.4 and np.array_equal(new0.p_sigma, np.zeros(n))


def test_rank_mu_update_with_equal_weights_is_a_sample_covariance():
    """weights 1/mu, c_1 = 0, c_mu = 1: C_new is the second moment of the selected steps about the old mean,
    i.e. numpy.cov (biased) plus the outer product of their average."""
    rng = np.random.default_rng(4)
    n, lam = 4, 12
    base = cma.default_params(n, lam)
    p = dataclasses.replace(base, weights=np.full(base.mu, 1.0 / base.mu), mu_eff=float(base.mu), c_1=0.0, c_mu=1.0)
    st = cma.init_state(np.zeros(n), 2.0, lam, params=p)
    x = rng.standard_normal((lam, n)) * 3.0
    f = rng.standard_normal(lam)
    new = cma.tell(st, x, f)
    sel = x[np.argsort(-f)[:base.mu]] / 2.0
    want = np.cov(sel.T, bias=True) + np.outer(sel.mean(axis=0), sel.mean(axis=0))
    assert np.allclose(new.C, want, atol=1e-13)
    assert np.allclose(new.mean, 2.0 * sel.mean(axis=0), atol=1e-14)


def test_conjugate_path_sees_the_whitened_step():
    """For x_k = m + sigma B (D .* z_k):  C^{-1/2} <y>_w = B sum_i w_i z_{i:lambda} (orientation of B, inverse of D)."""
    rng = np.random.default_rng(5)
    n, lam = 7, 9
    st = cma.init_state(rng.standard_normal(n), 0.8, lam, C0=random_spd(rng, n, cond=1e3))
    z = rng.standard_normal((lam, n))
    x = cma.ask_from_normals(st, z)
    # the population really has covariance sigma^2 C:  (x - m)/sigma = z D B^T
    assert np.allclose(((x - st.mean) / st.sigma) @ st.B / st.D, z, atol=1e-10)
    f = rng.standard_normal(lam)
    new = cma.tell(st, x, f)
    p = st.params
    order = np.argsort(-f)
    want = math.sqrt(p.c_sigma * (2 - p.c_sigma) * p.mu_eff) * st.B @ (p.weights @ z[order[:p.mu]])
    assert np.allclose(new.p_sigma, want, atol=1e-10)


def test_decomposition_is_valid_after_many_updates():
    rng = np.random.default_rng(6)
    n, lam = 10, 14
    st = cma.init_state(rng.standard_normal(n), 0.32, lam)
    for _ in range(60):
        x = cma.ask_from_normals(st, rng.standard_normal((lam, n)))
        st = cma.tell(st, x, rng.standard_normal(lam))
        assert np.array_equal(st.C, st.C.T)
    assert np.all(np.linalg.eigvalsh(st.C) > 0)
    assert np.allclose(st.B.T @ st.B, np.eye(n), atol=1e-12)
    assert np.allclose((st.B * st.D ** 2) @ st.B.T, st.C, atol=1e-12)
    assert np.all(np.diff(st.D) >= 0)
    assert st.generation == 60


def test_neutral_selection_keeps_paths_and_covariance_stationary():
    """With rewards independent of the candidates, p_sigma ~ N(0, I) and p_c ~ N(0, C) are stationary and the
    expected C does not move (the normalisation sqrt(c (2 - c) mu_eff) and the coefficients summing to one)."""
    rng = np.random.default_rng(7)
    n, lam, trials = 4, 8, 6000
    C0 = random_spd(rng, n, cond=5.0)
    base = cma.init_state(np.zeros(n), 1.0, lam, C0=C0)
    L = np.linalg.cholesky(C0)
    acc_ps, acc_pc, acc_C = 0.0, np.zeros((n, n)), np.zeros((n, n))
    for _ in range(trials):
        st = dataclasses.replace(base, p_sigma=rng.standard_normal(n), p_c=L @ rng.standard_normal(n), generation=10 ** 6)
        x = cma.ask_from_normals(st, rng.standard_normal((lam, n)))
        new = cma.tell(st, x, rng.standard_normal(lam))
        acc_ps += float(new.p_sigma @ new.p_sigma) / n
        acc_pc += np.outer(new.p_c, new.p_c)
        acc_C += new.C
    assert abs(acc_ps / trials - 1.0) < 0.05
    # h_sigma = 0 happens for a small fraction of the draws and only shrinks p_c, so allow a one-sided margin
    assert np.allclose(acc_pc / trials, C0, atol=0.12 * np.abs(C0).max())
    assert np.allclose(acc_C / trials, C0, atol=0.03 * np.abs(C0).max())


def test_stalled_path_update_when_the_step_is_too_long():
    rng = np.random.default_rng(8)
    n, lam = 5, 6
    st = cma.init_state(np.zeros(n), 1.0, lam)
    st = dataclasses.replace(st, p_c=rng.standard_normal(n))
    x = 50.0 * np.ones((lam, n)) + rng.standard_normal((lam, n))   # every candidate far along one direction
    new = cma.tell(st, x, rng.standard_normal(lam))
    p = st.params
    assert np.allclose(new.p_c, (1 - p.c_c) * st.p_c, atol=1e-15)   # h_sigma = 0: no new step enters p_c
    assert new.sigma > st.sigma                                     # and the step size grows


@pytest.mark.parametrize("n,lam", [(8, 12), (16, 16)])
def test_converges_on_the_sphere_function(n, lam):
    rng = np.random.default_rng(100 + n)
    st = cma.init_state(np.full(n, 3.0), 0.32, lam)
    best = np.inf
    for gen in range(700):
        x = cma.ask_from_normals(st, rng.standard_normal((lam, n)))
        f = np.sum(x * x, axis=1)
        best = min(best, float(f.min()))
        if best < 1e-10:
            break
        st = cma.tell(st, x, -f)
    assert best < 1e-10, (gen, best)
