"""GPU tests of the library's behaviour around the numerics: a bounded device-side wait that runs out (no fault, no
trap: the kernel gives up, records the status and the context stays usable), calls on one context from two streams,
and the rank-term isolation check at full size."""
import numpy as np
import pytest

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import binding, workloads as wl
from tests.parity_utils import TOL_BF16, TOL_INT8, Case, oracle_weight, to_dev

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    return torch


def test_bounded_wait_runs_out_and_the_context_recovers(torch):
    """One-CTA cluster (d_in = 64: a single K block, no split): with ESSA_OPT_DEBUG_STALL_RANK_ROWS the up-projection
    waits for a row of u that nobody publishes; with a limit of a few million cycles the wait runs out, the kernel
    leaves through its give-up path (drains its copies, joins the cluster barriers, frees tensor memory), the status
    word says ESSA_ERR_DEVICE_TIMEOUT, and the next call on the same context is correct."""
    ctx = binding.Context(0)
    cfg = wl.scaled_config("1", d_model=64, d_kv=64, rank=4, P=3, seg_len=2)
    case = Case(torch, ctx, cfg)
    x = case.tokens(0)
    dx = to_dev(torch, x, torch.bfloat16)
    sA, sB = cfg.sigma_cols(0)
    plan = binding.plan_projection(64, 64, 4, binding.ESSA_W0_BF16, case.T)
    assert plan["decode"] == 1 and plan["splits"] == 1
    want = case.oracle_projection(0, x)
    ok0 = ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)
    torch.cuda.synchronize()
    assert orc.relative_error(ok0.float().cpu().numpy(), want) <= TOL_BF16 and ctx.get_status() == 0
    ctx.set_option(binding.ESSA_OPT_WAIT_LIMIT_MCYCLES, 5)
    ctx.set_option(binding.ESSA_OPT_DEBUG_STALL_RANK_ROWS, 1)
    ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)  # gives up after ~3 ms
    ctx.set_option(binding.ESSA_OPT_DEBUG_STALL_RANK_ROWS, 0)
    ctx.set_option(binding.ESSA_OPT_WAIT_LIMIT_MCYCLES, 3000)
    assert ctx.get_status() == binding.ESSA_ERR_DEVICE_TIMEOUT   # reads, clears and repairs
    assert ctx.get_status() == 0
    for _ in range(2):
        y = ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)
        torch.cuda.synchronize()
        assert orc.relative_error(y.float().cpu().numpy(), want) <= TOL_BF16
    assert ctx.get_status() == 0
    case.close()
    ctx.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("3", 1024, 192, 16, 128, 1),    # decode schedule (context-owned u, counters)
                                               ("2", 512, 128, 16, 6, 150)])   # prefill schedule (u buffer, split-K scratch)
def test_two_streams_on_one_context_are_ordered(torch, base, dm, dkv, r, P, L):
    """The calls of a context share its scratch; alternating two streams must still give every call its own correct
    result (the library orders a call behind the context's previous one with an event)."""
    ctx = binding.Context(0)
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    xs_h = [case.tokens(i) for i in range(2)]
    xs = [to_dev(torch, x, torch.bfloat16) for x in xs_h]
    wants = [case.oracle_projection(i, xs_h[i]) for i in range(2)]
    torch.cuda.synchronize()
    outs = []
    for rep in range(6):
        i = rep % 2
        sA, sB = cfg.sigma_cols(i)
        with torch.cuda.stream(streams[rep % 2]):
            outs.append((i, ctx.apply_projection(case.handles[i], xs[i], case.d_offsets, case.d_sigma, sA, sB, stream=streams[rep % 2])))
    torch.cuda.synchronize()
    for i, y in outs:
        assert orc.relative_error(y.float().cpu().numpy(), wants[i]) <= TOL_BF16
    assert ctx.get_status() == 0
    case.close()
    ctx.close()


@pytest.mark.parametrize("name,n_cands", [("5a", 12), ("5b", 3), ("6a", 12)])
def test_rank_term_alone_matches_oracle_at_full_size(torch, name, n_cands):
    """y(sigma) - y(sigma = 0) from the GPU against the oracle's DeltaW_k x, same metric on the DIFFERENCE: the base
    contraction cancels, so a wrong candidate's singular values (e.g. the neighbour's row) cannot hide behind it."""
    ctx = binding.Context(0)
    cfg = wl.CONFIGS[name]
    case = Case(torch, ctx, cfg, projections=[0, 1])
    cands = wl.stratified_candidates(cfg, case.offsets)[:n_cands]
    zero = torch.zeros_like(case.d_sigma)
    for i in (0, 1):
        ad = case.adapters[i]
        sA, sB = cfg.sigma_cols(i)
        x = case.tokens(i)
        dx = to_dev(torch, x, torch.bfloat16)
        y1 = ctx.apply_projection(case.handles[i], dx, case.d_offsets, case.d_sigma, sA, sB).float()
        y0 = ctx.apply_projection(case.handles[i], dx, case.d_offsets, zero, sA, sB).float()
        torch.cuda.synchronize()
        got = (y1 - y0).cpu().numpy().astype(np.float64)
        want = np.full(got.shape, np.nan)
        wrong = np.full(got.shape, np.nan)  # the same with every candidate reading its neighbour's row
        x64 = x.astype(np.float64)
        for k in cands:
            a, b = int(case.offsets[k]), int(case.offsets[k + 1])
            for tbl, dst in ((case.sigma32, want), (np.roll(case.sigma32, 1, axis=0), wrong)):
                dW = orc.reconstruct_delta_w(ad.U_A, ad.V_A, ad.U_B, ad.V_B, tbl[k, sA:sA + ad.rank], tbl[k, sB:sB + ad.rank])
                dst[a:b] = x64[a:b] @ dW.T
        # Both y's are rounded to bf16: 2^-9 of |y|, and |y| is some thirty times the rank term, so the difference
        # carries rounding noise of about 5 % of its own size on EVERY element; a max-type metric over a million
        # elements would measure that noise's tail, so the difference is compared in the Frobenius norm.  The
        # candidates' tables differ by the perturbation only (step 0.05 around a common mean), so the neighbour's
        # rows change the rank term by ~17 %: the GPU result must be within 12 % of the right one AND at least twice
        # as close to it as to the planted mistake.
        mask = ~np.isnan(want)
        dist = lambda a, b: float(np.sqrt(np.sum((a[mask] - b[mask]) ** 2) / np.sum(want[mask] ** 2)))
        err, err_vs_wrong, planted = dist(got, want), dist(got, wrong), dist(wrong, want)
        assert planted > 0.12, (name, i, planted)  # the planted mistake (in the oracle) is visible in this metric
        assert err <= 0.12 and err < 0.5 * err_vs_wrong, (name, i, err, err_vs_wrong, planted)
    case.close()
    ctx.close()
