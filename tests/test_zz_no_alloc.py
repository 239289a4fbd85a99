"""essa_apply_projection_static: the allocation-free variant of the projection call.

Some users of the library cannot allocate device memory at call time (another allocator owns the GPU's memory,
or an implicit cudaMalloc synchronisation is not acceptable in their loop).  The variant keeps its scratch in a
fixed array inside the library; it must return what essa_apply_projection returns.  This file is collected last
so that a run stopping at the first failure has already run every other test; it also passes on its own in a
fresh process (the first call performs the one-time symbol look-up).
"""
import numpy as np
import pytest

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import workloads as wl
from tests.parity_utils import TOL_BF16, TOL_INT8, Case, to_dev

pytestmark = pytest.mark.gpu


def _rel_err(got, want):
    got, want = got.astype(np.float64), want.astype(np.float64)
    rms = np.sqrt(np.mean(want * want))
    return float(np.max(np.abs(got - want) / np.maximum(np.abs(want), rms)))


@pytest.mark.parametrize("base,dm,dkv,r,P,L,tol", [("2", 512, 128, 16, 8, 200, TOL_BF16),      # 1600 tokens, several tiles
                                                  ("3", 1024, 192, 16, 200, 1, TOL_BF16),     # decode-sized, ragged tile
                                                  ("5b", 512, 128, 64, 6, 70, TOL_INT8)])     # INT8 weights, rank 64
def test_static_variant_matches_regular_entry_point_twice(base, dm, dkv, r, P, L, tol):
    import torch
    from paper_2507_04453_b200 import binding
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    ctx = binding.Context(0)
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg, projections=[0, 1])
    if cfg.w0_dtype == "int8":
        ctx.reserve_dequant(dm, dm)  # set-up time: the allocation-free call will not size this scratch itself
    for i in (0, 1):
        x = to_dev(torch, case.tokens(i), torch.bfloat16)
        sA, sB = cfg.sigma_cols(i)
        want = ctx.apply_projection(case.handles[i], x, case.d_offsets, case.d_sigma, sA, sB).float().cpu().numpy()
        want_oracle = case.oracle_projection(i, case.tokens(i))  # ... and the CPU oracle, not only the sibling entry point
        out = torch.empty((case.T, case.handles[i].d_out), dtype=torch.bfloat16, device="cuda")
        free_before = None
        for call in range(2):  # two calls in a row share the fixed scratch: the second must not see stale data
            out.fill_(float("nan"))
            torch.cuda.synchronize()
            if call == 1:  # (the first call on a device may look up the array's address; after that nothing is allocated)
                free_before = torch.cuda.mem_get_info()[0]
            ctx.apply_projection_static(case.handles[i], x, case.d_offsets, case.d_sigma, sA, sB, out)
            torch.cuda.synchronize()
            if call == 1:
                assert torch.cuda.mem_get_info()[0] == free_before, "the allocation-free call changed the free device memory"
            got = out.float().cpu().numpy()
            assert np.isfinite(got).all(), (i, call)
            assert _rel_err(got, want) <= tol, (i, call)
            assert orc.relative_error(got, want_oracle) <= tol, (i, call)
    assert ctx.get_status() == 0
    case.close()
    ctx.close()


def test_static_variant_rejects_oversized_batches():
    import torch
    from paper_2507_04453_b200 import binding
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    ctx = binding.Context(0)
    cfg = wl.scaled_config("1", d_model=128, d_kv=128, rank=8, P=1, seg_len=4097)
    case = Case(torch, ctx, cfg)
    x = to_dev(torch, case.tokens(0), torch.bfloat16)
    out = torch.empty((case.T, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.EssaError) as e:
        ctx.apply_projection_static(case.handles[0], x, case.d_offsets, case.d_sigma, 0, 8, out)
    assert e.value.status == binding.ESSA_ERR_UNSUPPORTED_SHAPE and "ESSA_STATIC_MAX_TOKENS" in str(e.value)
    case.close()
    ctx.close()


def test_static_variant_at_its_token_limit_and_without_reserved_dequant_scratch():
    """T = ESSA_STATIC_MAX_TOKENS exactly is accepted and correct; an INT8-stored adapter without a sized
    dequantisation scratch is refused with ESSA_ERR_ALLOC (the entry point never allocates it itself)."""
    import torch
    from paper_2507_04453_b200 import binding
    if not torch.cuda.is_available():
        pytest.fail("CUDA device required for -m gpu tests")
    ctx = binding.Context(0)
    cfg = wl.scaled_config("1", d_model=128, d_kv=128, rank=8, P=2, seg_len=2048)  # 4096 tokens
    case = Case(torch, ctx, cfg)
    assert case.T == 4096
    x_h = case.tokens(0)
    out = torch.full((case.T, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    ctx.apply_projection_static(case.handles[0], to_dev(torch, x_h, torch.bfloat16), case.d_offsets, case.d_sigma, 0, 8, out)
    torch.cuda.synchronize()
    assert orc.relative_error(out.float().cpu().numpy(), case.oracle_projection(0, x_h)) <= TOL_BF16
    case.close()
    ctx.close()
    ctx = binding.Context(0)  # a fresh context: its dequantisation scratch is empty
    cfg8 = wl.scaled_config("5b", d_model=256, d_kv=128, rank=16, P=2, seg_len=300)
    case8 = Case(torch, ctx, cfg8, projections=[0])
    out8 = torch.empty((case8.T, 256), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.EssaError) as e:
        ctx.apply_projection_static(case8.handles[0], to_dev(torch, case8.tokens(0), torch.bfloat16), case8.d_offsets, case8.d_sigma,
                                    *cfg8.sigma_cols(0), out8)
    assert e.value.status == binding.ESSA_ERR_ALLOC
    case8.close()
    ctx.close()
