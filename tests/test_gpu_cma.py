"""GPU parity of the device-resident CMA-ES update (essa_tell / essa_cma_*) against the fp64 CPU oracle.

Data flow is one-way: every population and every reward fed to both sides comes from the oracle side or from a
seeded generator; nothing the CUDA path produced is given to the oracle.  m, sigma, C and the two paths are unique
and compared element by element; the decomposition is not (eigenvector signs, order inside equal eigenvalues), so B
and D are checked for validity: B orthonormal, B diag(D^2) B^T = C, D ascending.
"""
import numpy as np
import pytest

from oracle import cma_oracle as cma
from oracle import essa_oracle as orc
from paper_2507_04453_b200 import binding

pytestmark = pytest.mark.gpu
REL = 1e-6


@pytest.fixture(scope="module")
def torch():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    return torch


@pytest.fixture(scope="module")
def ctx(torch):
    c = binding.Context(0)
    yield c
    assert c.get_status() == 0
    c.close()


def rel_err(got, want):
    want = np.asarray(want, dtype=np.float64)
    scale = max(float(np.max(np.abs(want))), 1e-300)
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - want))) / scale


def check_decomposition(st, tag):
    d = st["C"].shape[0]
    B, D, C = st["B"], st["D"], st["C"]
    assert np.array_equal(C, C.T), tag
    assert np.max(np.abs(B.T @ B - np.eye(d))) <= 1e-6, tag
    assert rel_err((B * D ** 2) @ B.T, C) <= 1e-6, tag
    assert np.all(np.diff(D) >= 0), tag


def reward_fn(x, target):
    """A seeded, smooth, non-separable reward (larger is better)."""
    z = x - target[None, :]
    return -(np.sum(z * z, axis=1) + 0.5 * np.sum(z[:, :-1] * z[:, 1:], axis=1))


def test_strategy_parameters_match_oracle(ctx):
    for d, lam in ((16, 4), (128, 32), (256, 64), (512, 128), (37, 9)):
        st = ctx.cma_state(d, lam, np.zeros(d, dtype=np.float32), 0.32)
        got, want = st.params(), cma.default_params(d, lam)
        for k in ("mu", "mu_eff", "c_sigma", "d_sigma", "c_c", "c_1", "c_mu", "c_m", "chi_n"):
            assert abs(got[k] - float(getattr(want, k))) <= 1e-13 * max(1.0, abs(float(getattr(want, k)))), (d, lam, k)
        st.close()


@pytest.mark.parametrize("d,lam,gens", [(16, 8, 20), (37, 9, 20), (128, 32, 20), (256, 64, 6)])
def test_tell_matches_oracle_over_generations(torch, ctx, d, lam, gens):
    rng = np.random.default_rng(1000 + d)
    mean0 = rng.standard_normal(d).astype(np.float32)
    target = rng.standard_normal(d)
    ost = cma.init_state(mean0.astype(np.float64), 0.32, lam)
    gst = ctx.cma_state(d, lam, mean0, 0.32)
    for g in range(gens):
        # the population both sides are told about: the ORACLE's draw from its own state, stored as fp32
        pop = orc.sample_population(ost.mean.astype(np.float32), np.float32(ost.sigma), ost.B.astype(np.float32),
                                    ost.D.astype(np.float32), seed=77 + g, P=lam).astype(np.float32)
        rew = reward_fn(pop.astype(np.float64), target).astype(np.float32)
        ost = cma.tell(ost, pop, rew)
        gst.tell(torch.from_numpy(pop).cuda(), torch.from_numpy(rew).cuda())
        st = gst.get()
        tag = (d, lam, g)
        assert st["generation"] == g + 1
        assert rel_err(st["mean"], ost.mean) <= REL, tag
        assert abs(st["step"] - ost.sigma) <= REL * ost.sigma, tag
        assert rel_err(st["C"], ost.C) <= REL, tag
        assert rel_err(st["p_sigma"], ost.p_sigma) <= REL, tag
        assert rel_err(st["p_c"], ost.p_c) <= REL, tag
        check_decomposition(st, tag)
        assert rel_err(np.sort(st["D"]), np.sort(ost.D)) <= 1e-6, tag  # the eigenvalues themselves are unique
        assert 1 <= st["sweeps"] <= 30
    gst.close()


def test_tell_ranks_ties_and_nan_like_the_oracle(torch, ctx):
    d, lam = 8, 10
    rng = np.random.default_rng(5)
    mean0 = rng.standard_normal(d).astype(np.float32)
    ost = cma.init_state(mean0.astype(np.float64), 0.5, lam)
    gst = ctx.cma_state(d, lam, mean0, 0.5)
    pop = (mean0[None, :] + 0.5 * rng.standard_normal((lam, d))).astype(np.float32)
    rew = np.array([1.0, 3.0, 3.0, np.nan, -np.inf, 2.0, 3.0, 0.0, np.nan, 2.0], dtype=np.float32)
    ost = cma.tell(ost, pop, rew)
    gst.tell(torch.from_numpy(pop).cuda(), torch.from_numpy(rew).cuda())
    st = gst.get()
    assert rel_err(st["mean"], ost.mean) <= REL and rel_err(st["C"], ost.C) <= REL
    gst.close()


def test_set_state_and_stalled_path(torch, ctx):
    """A given (C, p_sigma, p_c, generation) and a population far along one direction: h_sigma = 0 on both sides."""
    d, lam = 12, 8
    rng = np.random.default_rng(6)
    q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    C0 = (q * np.exp(rng.uniform(0, 3, d))) @ q.T
    C0 = (C0 + C0.T) / 2
    mean0 = rng.standard_normal(d)
    ost = cma.init_state(mean0, 0.7, lam, C0=C0)
    import dataclasses
    ost = dataclasses.replace(ost, p_sigma=rng.standard_normal(d), p_c=rng.standard_normal(d), generation=3)
    gst = ctx.cma_state(d, lam, mean0.astype(np.float32), 0.7)
    gst.set(mean=mean0, step=0.7, C_=C0, p_sigma=ost.p_sigma, p_c=ost.p_c, generation=3)
    st0 = gst.get()
    check_decomposition(st0, "after set")
    assert rel_err(np.sort(st0["D"]), np.sort(ost.D)) <= 1e-9
    pop = (mean0[None, :] + 40.0 + rng.standard_normal((lam, d))).astype(np.float32)
    rew = rng.standard_normal(lam).astype(np.float32)
    new = cma.tell(ost, pop, rew)
    assert np.allclose(new.p_c, (1 - ost.params.c_c) * ost.p_c)  # the oracle did stall the path
    gst.tell(torch.from_numpy(pop).cuda(), torch.from_numpy(rew).cuda())
    st = gst.get()
    for k, want in (("mean", new.mean), ("C", new.C), ("p_sigma", new.p_sigma), ("p_c", new.p_c)):
        assert rel_err(st[k], want) <= REL, k
    assert abs(st["step"] - new.sigma) <= REL * new.sigma
    check_decomposition(st, "after tell")
    gst.close()


def test_ask_draws_from_the_state(torch, ctx):
    """x_k = m + sigma B (D .* z_k) for SOME valid decomposition: |C^{-1/2} (x_k - m) / sigma| = |z_k| with the oracle's
    own normals and the oracle's own inverse square root of the same C; candidates regenerate from <seed, k>."""
    d, lam = 24, 16
    rng = np.random.default_rng(8)
    q, _ = np.linalg.qr(rng.standard_normal((d, d)))
    C0 = (q * np.exp(rng.uniform(0, 2, d))) @ q.T
    C0 = (C0 + C0.T) / 2
    mean0 = rng.standard_normal(d)
    gst = ctx.cma_state(d, lam, mean0.astype(np.float32), 0.4)
    gst.set(mean=mean0, step=0.4, C_=C0)
    x = gst.ask(seed=123).cpu().numpy().astype(np.float64)
    z = orc.standard_normals(123, np.arange(lam), d)
    lam_c, Bc = np.linalg.eigh(C0)
    inv_sqrt = (Bc / np.sqrt(lam_c)) @ Bc.T
    y = (x - mean0.astype(np.float32).astype(np.float64)[None, :]) / float(np.float32(0.4))
    got = np.linalg.norm(y @ inv_sqrt.T, axis=1)
    assert np.max(np.abs(got - np.linalg.norm(z, axis=1)) / np.linalg.norm(z, axis=1)) <= 1e-5
    part = gst.ask(seed=123, P=5, k_begin=7).cpu().numpy()
    assert np.array_equal(part, x[7:12].astype(np.float32))
    gst.close()


def test_ask_tell_loop_converges_on_device(torch, ctx):
    """ask -> rewards -> tell entirely on the device (the rewards are a torch expression: plumbing) on a shifted sphere."""
    d, lam = 32, 16
    rng = np.random.default_rng(9)
    target = torch.from_numpy(rng.standard_normal(d).astype(np.float32)).cuda()
    gst = ctx.cma_state(d, lam, np.zeros(d, dtype=np.float32), 0.32)
    best = np.inf
    for g in range(400):
        x = gst.ask(seed=g)
        f = ((x - target[None, :]) ** 2).sum(dim=1)
        gst.tell(x, -f)
        if g % 20 == 19:
            best = min(best, float(f.min().item()))
            if best < 1e-8:
                break
    assert best < 1e-8, best
    st = gst.get()
    check_decomposition(st, "after the loop")
    assert np.max(np.abs(st["mean"] - target.cpu().numpy())) < 1e-3
    gst.close()
