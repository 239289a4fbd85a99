"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle cannot cover these sizes in full within seconds, so per projection it computes a fixed stratified
subset of candidates (first, last, shortest, longest, tile-straddling, a few seeded random ones) -- all their
tokens and all channels -- and the tensor-core path is compared with it element by element.  On top of that
the tensor-core output is compared on EVERY element with the CUDA-core cross-check path (itself checked
against the oracle on the same subset), which catches tile- or schedule-dependent faults anywhere in the output.
"""
import numpy as np
import pytest

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import workloads as wl
from tests.parity_utils import TOL_BF16, TOL_INT8, Case

pytestmark = pytest.mark.gpu

MAX_ORACLE_CANDIDATES = {"2": 6, "3": 24, "4": 6, "5a": 12, "5b": 5, "6a": 12, "6b": 4}


@pytest.fixture(scope="module")
def torch():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    return torch


@pytest.fixture(scope="module")
def ctx(torch):
    from paper_2507_04453_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.get_status() == 0, "a kernel recorded a device-side error"
    c.close()


@pytest.mark.parametrize("name", ["2", "3", "4", "5a", "5b", "6a", "6b"])
def test_full_size_config(torch, ctx, name):
    cfg = wl.CONFIGS[name]
    case = Case(torch, ctx, cfg)
    tol = TOL_BF16 if cfg.w0_dtype == "bf16" else TOL_INT8
    cands = wl.stratified_candidates(cfg, case.offsets)[:MAX_ORACLE_CANDIDATES[name]]
    assert case.T == int(case.offsets[-1]) and len(cands) >= 2
    for i in range(len(cfg.projections)):
        x = case.tokens(i)
        got_tc = case.gpu_projection(i, x, "tc")
        got_simt = case.gpu_projection(i, x, "simt")
        assert np.isfinite(got_tc).all()
        # every element: tensor-core path vs CUDA-core path (both round the result to bf16)
        assert orc.relative_error(got_tc, got_simt.astype(np.float64)) <= tol, (name, i, "tc vs simt")
        # sampled candidates: both against the oracle
        want = case.oracle_projection(i, x, cands)
        e_tc, e_simt = orc.relative_error(got_tc, want), orc.relative_error(got_simt, want)
        assert e_tc <= tol and e_simt <= tol, (name, cfg.projections[i], e_tc, e_simt)
        del x, got_tc, got_simt, want
    case.close()
