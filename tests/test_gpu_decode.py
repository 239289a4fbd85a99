"""GPU parity of the decode schedule (at most 256 tokens in the call: one launch, W0 rows on the MMA M side,
reduction over d_in split across a thread-block cluster) against the CPU oracle, element by element.

Sizes span one and several W0 row tiles, ragged channel counts, every padded rank, token counts around the
16-token MMA granularity and the 128-token half boundary, ragged and empty segments, both W0 storage types.
"""
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


@pytest.fixture(scope="module")
def ctx(torch):
    c = binding.Context(0)
    yield c
    assert c.get_status() == 0, "a kernel recorded a device-side error"
    c.close()


def _run(torch, ctx, case, i, offsets, T, tol):
    cfg = case.cfg
    ad, h = case.adapters[i], case.handles[i]
    sA, sB = cfg.sigma_cols(i)
    offsets = np.asarray(offsets, dtype=np.int32)
    dtype = {"bf16": binding.ESSA_W0_BF16, "int8": binding.ESSA_W0_INT8_PERCHANNEL, "int4": binding.ESSA_W0_INT4_GROUP128}[ad.w0_dtype]
    plan = binding.plan_projection(ad.d_in, ad.d_out, ad.rank, dtype, T)
    # INT4 storage has the tensor-memory decode mode only (at most 128 tokens); larger calls take the prefill kernels
    assert plan["decode"] == (0 if ad.w0_dtype == "int4" and T > 128 else 1)
    x = wl.make_tokens(cfg, i, T)
    want = orc.apply_projection(oracle_weight(ad), ad.U_A, ad.V_A, ad.U_B, ad.V_B, x, offsets, case.sigma32, sA, sB, ad.rank)
    y = ctx.apply_projection(h, to_dev(torch, x, torch.bfloat16), to_dev(torch, offsets), case.d_sigma, sA, sB)
    torch.cuda.synchronize()
    got = y.float().cpu().numpy()
    assert got.shape == want.shape and np.isfinite(got).all()
    err = orc.relative_error(got, want)
    assert err <= tol, (cfg.name, ad.d_in, ad.d_out, ad.rank, T, plan, err)
    return y, err


def _offsets(rng, P, T):
    """P segments (some empty) covering T tokens."""
    cuts = np.sort(rng.integers(0, T + 1, size=P - 1))
    return np.concatenate([[0], cuts, [T]]).astype(np.int32)


@pytest.mark.parametrize("T", [1, 5, 16, 17, 100, 128, 129, 200, 255, 256])
def test_token_counts(torch, ctx, T):
    cfg = wl.scaled_config("3", d_model=1024, d_kv=192, rank=16, P=9, seg_len=1)
    case = Case(torch, ctx, cfg)
    rng = np.random.default_rng(100 + T)
    for i in (0, 1):  # 1024 -> 1024 (8 row tiles) and 1024 -> 192 (1.5 row tiles)
        _run(torch, ctx, case, i, _offsets(rng, cfg.P, T), T, TOL_BF16)
    case.close()


@pytest.mark.parametrize("rank", [1, 3, 8, 17, 33, 48, 64])
@pytest.mark.parametrize("w0", ["bf16", "int8", "int4"])
def test_ranks_and_storage(torch, ctx, rank, w0):
    cfg = wl.scaled_config({"int8": "5a", "int4": "6a", "bf16": "3"}[w0], d_model=512, d_kv=200, rank=rank, P=7, seg_len=1)
    case = Case(torch, ctx, cfg)
    rng = np.random.default_rng(rank)
    tol = TOL_BF16 if w0 == "bf16" else TOL_INT8
    for i, T in ((0, 77), (1, 192)):
        _run(torch, ctx, case, i, _offsets(rng, cfg.P, T), T, tol)
    case.close()


def test_single_k_block_and_tiny_shapes(torch, ctx):
    cfg = wl.scaled_config("1", d_model=64, d_kv=64, rank=4, P=3, seg_len=2)  # d_in = 64: one K block, no split
    case = Case(torch, ctx, cfg)
    _run(torch, ctx, case, 0, [0, 2, 2, 6], 6, TOL_BF16)
    case.close()
    cfg = wl.scaled_config("1", d_model=128, d_kv=128, rank=8, P=1, seg_len=1)
    case = Case(torch, ctx, cfg)
    _run(torch, ctx, case, 0, [0, 1], 1, TOL_BF16)
    case.close()


def test_decode_is_deterministic_and_matches_cuda_core_path(torch, ctx):
    """The cluster reduction sums the partial tiles in fixed rank order: repeated calls are bit-identical."""
    cfg = wl.scaled_config("3", d_model=2048, d_kv=256, rank=16, P=256, seg_len=1)
    case = Case(torch, ctx, cfg, projections=[0])
    y0, _ = _run(torch, ctx, case, 0, case.offsets, case.T, TOL_BF16)
    y0 = y0.clone()
    dx = to_dev(torch, case.tokens(0), torch.bfloat16)
    sA, sB = cfg.sigma_cols(0)
    for _ in range(4):
        y = ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)
        assert torch.equal(y, y0)
    ys = ctx.apply_projection_simt(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)
    assert orc.relative_error(y0.float().cpu().numpy(), ys.float().cpu().numpy().astype(np.float64)) <= TOL_BF16
    case.close()


def test_zero_sigma_gives_base_projection(torch, ctx):
    cfg = wl.scaled_config("3", d_model=768, d_kv=128, rank=16, P=40, seg_len=1)
    case = Case(torch, ctx, cfg, projections=[0])
    x = case.tokens(0)
    sA, sB = cfg.sigma_cols(0)
    y = ctx.apply_projection(case.handles[0], to_dev(torch, x, torch.bfloat16), case.d_offsets,
                             torch.zeros_like(case.d_sigma), sA, sB).float().cpu().numpy()
    base = x.astype(np.float64) @ oracle_weight(case.adapters[0]).T
    assert orc.relative_error(y, base) <= 6e-3  # only the final bf16 rounding
    case.close()


@pytest.mark.parametrize("w0", ["int8", "int4"])
@pytest.mark.parametrize("T", [1, 16, 33, 100, 128])
def test_quantised_storage_token_counts_in_tensor_memory_mode(torch, ctx, w0, T):
    """At most 128 tokens: the codes are converted straight into tensor memory (INT8 and INT4 storage alike); several
    row tiles, a ragged last row tile (d_kv = 200), more K blocks than ring slots, ragged and empty segments."""
    cfg = wl.scaled_config("5a" if w0 == "int8" else "6a", d_model=1280, d_kv=200, rank=24, P=6, seg_len=1)
    case = Case(torch, ctx, cfg)
    rng = np.random.default_rng(7 * T)
    for i in (0, 1):
        y, _ = _run(torch, ctx, case, i, _offsets(rng, cfg.P, T), T, TOL_INT8)
    case.close()


@pytest.mark.parametrize("w0,T", [("bf16", 256), ("bf16", 96), ("int8", 128), ("int4", 64)])
def test_cta_pair_variant(torch, w0, T):
    """ESSA_OPT_DECODE_PAIRS: two W0 row tiles per MMA of 256 rows (cta_group::2), each CTA loading half of the token
    rows; an odd number of row tiles (d_kv = 200 -> 2 tiles, d_model 640 -> 5) pairs the last tile with an empty one."""
    c = binding.Context(0)
    c.set_option(binding.ESSA_OPT_DECODE_PAIRS, 1)
    cfg = wl.scaled_config({"int8": "5a", "int4": "6a", "bf16": "3"}[w0], d_model=640, d_kv=200, rank=24, P=5, seg_len=1)
    case = Case(torch, c, cfg)
    rng = np.random.default_rng(T)
    for i in (0, 1):
        _run(torch, c, case, i, _offsets(rng, cfg.P, T), T, TOL_BF16 if w0 == "bf16" else TOL_INT8)
    assert c.get_status() == 0
    case.close()
    c.close()


@pytest.mark.parametrize("w0,T,r", [("bf16", 256, 16), ("bf16", 77, 33), ("int8", 128, 64), ("int8", 200, 24), ("int4", 100, 16)])
def test_slices_on_the_row_tiles_when_no_down_projection_ctas(torch, w0, T, r):
    """ESSA_OPT_DECODE_DOWN_CTAS = 0: the down-projection rides as slices on the K loops of the first row tiles (the
    scheme a launch without spare thread blocks uses), same results."""
    c = binding.Context(0)
    c.set_option(binding.ESSA_OPT_DECODE_DOWN_CTAS, 0)
    cfg = wl.scaled_config({"int8": "5a", "int4": "6a", "bf16": "3"}[w0], d_model=1024, d_kv=200, rank=r, P=6, seg_len=1)
    case = Case(torch, c, cfg)
    rng = np.random.default_rng(T + r)
    for i in (0, 1):
        _run(torch, c, case, i, _offsets(rng, cfg.P, T), T, TOL_BF16 if w0 == "bf16" else TOL_INT8)
    assert c.get_status() == 0
    case.close()
    c.close()
