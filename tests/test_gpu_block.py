"""GPU parity of essa_apply_block (the q, k, v, o projections of a block in one call) against the CPU oracle.

At decode sizes the block runs as one launch of the decode kernel; at prefill sizes as the projections' rank-down
launches followed by one launch for the base + up step of all of them, where the shapes suit that, else as one call
per projection.  Either way every projection's output must match the oracle like a single call does.
"""
import numpy as np
import pytest

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import binding, workloads as wl
from tests.parity_utils import TOL_BF16, TOL_INT8, Case, to_dev

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


def _block(torch, ctx, case, candidates=None):
    cfg = case.cfg
    n = len(cfg.projections)
    xs_host = [case.tokens(i) for i in range(n)]
    xs = [to_dev(torch, x, torch.bfloat16) for x in xs_host]
    cols = [cfg.sigma_cols(i) for i in range(n)]
    launches0 = ctx.gpu_launches
    ys = ctx.apply_block([case.handles[i] for i in range(n)], xs, case.d_offsets, case.d_sigma, cols)
    torch.cuda.synchronize()
    launches = ctx.gpu_launches - launches0
    tol = TOL_BF16 if cfg.w0_dtype == "bf16" else TOL_INT8
    for i in range(n):
        got = ys[i].float().cpu().numpy()
        want = case.oracle_projection(i, xs_host[i], candidates)
        assert np.isfinite(got).all()
        err = orc.relative_error(got, want)
        assert err <= tol, (cfg.name, cfg.projections[i], err)
    return launches, xs, ys


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("3", 1024, 192, 16, 256, 1),      # decode block, bf16: one launch
                                               ("5a", 1024, 256, 64, 128, 1),     # decode block, INT8, rank 64
                                               ("6a", 1024, 256, 64, 128, 1),     # decode block, INT4 group-wise
                                               ("4", 512, 128, 32, 9, 20),        # ragged segments, T = sum L_k <= 180
                                               ("2", 256, 64, 16, 3, 100)])       # T = 300: prefill sizes, one call each
def test_block_matches_oracle(torch, ctx, base, dm, dkv, r, P, L):
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    launches, _, _ = _block(torch, ctx, case)
    if case.T <= 256:
        assert launches == 1, "a decode-sized block is one kernel launch"
    else:
        assert launches == 2 * len(cfg.projections)
    case.close()


def test_block_equals_single_calls_in_structure_and_is_deterministic(torch, ctx):
    """Same inputs, two block calls: bit-identical (the cluster reduction and the rank path sum in fixed order)."""
    cfg = wl.scaled_config("3", d_model=2048, d_kv=256, rank=16, P=200, seg_len=1)
    case = Case(torch, ctx, cfg)
    _, xs, ys = _block(torch, ctx, case)
    first = [y.clone() for y in ys]
    cols = [cfg.sigma_cols(i) for i in range(4)]
    for _ in range(3):
        again = ctx.apply_block([case.handles[i] for i in range(4)], xs, case.d_offsets, case.d_sigma, cols)
        for a, b in zip(first, again):
            assert torch.equal(a, b)
    # single calls take another split of the reduction, so they agree to rounding, not bit for bit
    for i in range(4):
        single = ctx.apply_projection(case.handles[i], xs[i], case.d_offsets, case.d_sigma, *cols[i])
        assert orc.relative_error(first[i].float().cpu().numpy(), single.float().cpu().numpy().astype(np.float64)) <= TOL_BF16
    case.close()


def test_prefill_block_with_odd_channel_counts(torch, ctx):
    """One base + up launch for projections of 1024 and 1000 channels (1000 = 3.9 channel tiles of 256, not a multiple of
    the 32-channel store boxes: the last box of a row is clipped) over 2400 tokens."""
    cfg = wl.scaled_config("2", d_model=1024, d_kv=1000, rank=16, P=6, seg_len=400)
    case = Case(torch, ctx, cfg)
    try:
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 2)
        launches, _, _ = _block(torch, ctx, case)
        assert launches == len(cfg.projections) + 1
    finally:
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 1)
    case.close()


def test_prefill_block_is_one_base_up_launch(torch, ctx):
    """A prefill-sized block whose projections all suit the wide pair tiles: four rank-down launches, then ONE launch for
    the base + up step of all four (ragged segments, T = 4348: the last 512-token tile holds 252 rows); with the wide
    tiles switched off the block degrades to one call (two launches) per projection.  Both match the oracle."""
    cfg = wl.scaled_config("4", d_model=1024, d_kv=1024, rank=32, P=12, seg_len=600)
    case = Case(torch, ctx, cfg)
    try:
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 2)
        launches, xs, ys = _block(torch, ctx, case)
        assert launches == len(cfg.projections) + 1  # (too few tokens for the CTA-pair rank-down kernel: one launch each)
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 0)
        launches0, _, ys0 = _block(torch, ctx, case)
        assert launches0 == 2 * len(cfg.projections)
        for a, b in zip(ys, ys0):  # same K order in fp32; u may differ in its last bit (split-K rank-down launches)
            assert orc.relative_error(a.float().cpu().numpy(), b.float().cpu().numpy().astype(np.float64)) <= 8e-3
    finally:
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 1)
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L,pairs", [("4", 512, 512, 32, 40, 1000, True),    # ragged, T = 21 394: 335 units of 64 rows per projection
                                                     ("2", 512, 512, 16, 30, 650, True),     # T = 19 500
                                                     ("2", 512, 512, 16, 16, 500, True),     # T = 8 000: fewer than twelve units per pair, 256-row tiles
                                                     ("5c", 512, 512, 17, 150, 256, True),   # INT8 storage (one call per projection), padded rank 32, mixed lengths
                                                     ("2", 512, 512, 33, 30, 650, False)])   # padded rank 48: stays on the single-CTA kernel
def test_rank_down_on_cta_pairs(torch, ctx, base, dm, dkv, r, P, L, pairs):
    """Prefill-sized block with enough tokens for the CTA-pair rank-down kernel (every pair of the grid gets at least four
    64-row units; the last tile of a pair's range is partial): bf16 blocks run ONE rank-down launch and ONE base + up
    launch.  The result matches the oracle and, to the last bit or so, the single-CTA rank-down launches
    (ESSA_OPT_DOWN_PAIRS = 0), which add the same K blocks in the same order; 256-row and 512-row tiles
    (ESSA_OPT_DOWN_TILE_UNITS) give the same bits."""
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    assert len(cfg.projections) * ((case.T + 63) // 64) >= 4 * 74
    cands = wl.stratified_candidates(cfg, case.offsets)[:10]
    n = len(cfg.projections)
    bf16 = cfg.w0_dtype == "bf16"
    try:
        launches, xs, ys = _block(torch, ctx, case, cands)
        # quantised storage: dequantisation pass, rank-down, base + up per projection
        assert launches == ((2 if pairs else n + 1) if bf16 else 3 * n)
        if pairs:
            for units in (3, 4, 8):
                ctx.set_option(binding.ESSA_OPT_DOWN_TILE_UNITS, units)
                _, _, ys_u = _block(torch, ctx, case, cands)
                for a, b in zip(ys, ys_u):
                    assert torch.equal(a, b), units
            ctx.set_option(binding.ESSA_OPT_DOWN_TILE_UNITS, 0)
        ctx.set_option(binding.ESSA_OPT_DOWN_PAIRS, 0)
        launches0, _, ys0 = _block(torch, ctx, case, cands)
        assert launches0 == (n + 1 if bf16 else 3 * n)
        for a, b in zip(ys, ys0):
            a, b = a.float().cpu().numpy(), b.float().cpu().numpy()
            assert np.mean(a != b) < 0.01 and orc.relative_error(a, b.astype(np.float64)) <= 8e-3
    finally:
        ctx.set_option(binding.ESSA_OPT_DOWN_PAIRS, 5)
        ctx.set_option(binding.ESSA_OPT_DOWN_TILE_UNITS, 0)
    case.close()


@pytest.mark.parametrize("name,max_cands,want_launches", [("3", 24, 1), ("5a", 12, 1), ("4", 4, 2)])
def test_block_full_size(torch, ctx, name, max_cands, want_launches):
    """The benchmark's configurations through the block call, in the launch configuration bench.py times."""
    cfg = wl.CONFIGS[name]
    case = Case(torch, ctx, cfg)
    cands = wl.stratified_candidates(cfg, case.offsets)[:max_cands]
    launches, xs, ys = _block(torch, ctx, case, cands)
    assert launches == want_launches
    tol = TOL_INT8 if cfg.w0_dtype == "int8" else TOL_BF16
    for i in range(4):  # every element against the CUDA-core path
        ref = ctx.apply_projection_simt(case.handles[i], xs[i], case.d_offsets, case.d_sigma, *cfg.sigma_cols(i))
        assert orc.relative_error(ys[i].float().cpu().numpy(), ref.float().cpu().numpy().astype(np.float64)) <= tol
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("3", 1024, 192, 16, 200, 1),     # decode sizes: one device call for the block
                                               ("5a", 1024, 256, 64, 96, 1),     # ... INT8 storage
                                               ("4", 512, 128, 32, 24, 300),     # ragged prefill: pipelined (projection, chunk) units
                                               ("5b", 512, 128, 64, 20, 256)])   # ... INT8 storage: every chunk dequantises W0 again
def test_block_host_entry_point(torch, ctx, base, dm, dkv, r, P, L):
    """essa_apply_block_host: host buffers in, host buffers out, against the oracle for every projection."""
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    n = len(cfg.projections)
    xs = [case.tokens(i) for i in range(n)]
    xh = [torch.from_numpy(x).to(torch.bfloat16).pin_memory() for x in xs]
    yh = [torch.zeros((case.T, case.adapters[i].d_out), dtype=torch.bfloat16).pin_memory() for i in range(n)]
    cols = [cfg.sigma_cols(i) for i in range(n)]
    hs = [case.handles[i] for i in range(n)]
    for _ in range(2):  # the second call re-uses the staging buffers
        ctx.apply_block_host(hs, xh, torch.from_numpy(case.offsets), torch.from_numpy(case.sigma32), cols, yh)
    tol = TOL_INT8 if cfg.w0_dtype == "int8" else TOL_BF16
    for i in range(n):
        got = yh[i].float().numpy()
        assert np.isfinite(got).all()
        assert orc.relative_error(got, case.oracle_projection(i, xs[i])) <= tol, (cfg.name, cfg.projections[i])
    assert ctx.get_status() == 0
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("3", 1024, 192, 16, 256, 1),    # decode, full covariance factor
                                               ("5a", 1024, 256, 64, 128, 1),   # decode, INT8 storage, diagonal draw
                                               ("2", 256, 64, 16, 3, 100)])     # prefill sizes: plain stream order
def test_fused_draw_and_block_equals_separate_calls_and_oracle(torch, ctx, base, dm, dkv, r, P, L):
    """essa_sample_apply_block: the table and every output equal the two separate calls bit for bit (the block
    kernel only starts earlier), and both match the oracle; repeated calls stay identical (the draw's completion
    count is monotonic across calls)."""
    from tests.parity_utils import TOL_SIGMA, sigma_error
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    n = len(cfg.projections)
    cma = case.cma
    xs_host = [case.tokens(i) for i in range(n)]
    xs = [to_dev(torch, x, torch.bfloat16) for x in xs_host]
    cols = [cfg.sigma_cols(i) for i in range(n)]
    hs = [case.handles[i] for i in range(n)]
    d_mean = to_dev(torch, cma.mean)
    d_B = None if cma.Bfactor is None else to_dev(torch, cma.Bfactor)
    d_D = None if cma.Dvec is None else to_dev(torch, cma.Dvec)
    sig_sep = ctx.sample_population(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P)
    ys_sep = ctx.apply_block(hs, xs, case.d_offsets, sig_sep, cols)
    torch.cuda.synchronize()
    for rep in range(3):
        sig_f, ys_f = ctx.sample_apply_block(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, hs, xs, case.d_offsets, cols)
        torch.cuda.synchronize()
        assert torch.equal(sig_f, sig_sep)
        for a, b in zip(ys_f, ys_sep):
            if case.T <= 256:
                assert torch.equal(a, b), (cfg.name, rep)
            else:  # prefill split-K adds partial tiles in arrival order: equal to rounding, not bit for bit
                assert orc.relative_error(a.float().cpu().numpy(), b.float().cpu().numpy()) <= 1e-2
    want_sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    assert sigma_error(sig_f.cpu().numpy(), want_sigma) <= TOL_SIGMA
    tol = TOL_INT8 if cfg.w0_dtype == "int8" else TOL_BF16
    sig32 = sig_f.cpu().numpy()
    for i in range(n):
        ad = case.adapters[i]
        from tests.parity_utils import oracle_weight
        want = orc.apply_projection(oracle_weight(ad), ad.U_A, ad.V_A, ad.U_B, ad.V_B, xs_host[i], case.offsets, sig32,
                                    *cols[i], ad.rank)
        assert orc.relative_error(ys_f[i].float().cpu().numpy(), want) <= tol
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L,n_layers", [("3", 768, 128, 16, 200, 1, 2),     # decode, bf16, two layers
                                                        ("3", 512, 192, 16, 64, 1, 8),      # eight layers (both scratch sets reused)
                                                        ("5a", 512, 128, 64, 100, 1, 3),    # INT8 storage, tensor-memory mode
                                                        ("2", 256, 64, 16, 3, 100, 2)])     # prefill sizes: issued block by block
def test_layers_call_matches_block_calls_and_oracle(torch, ctx, base, dm, dkv, r, P, L, n_layers):
    """essa_apply_layers over n_layers blocks (each layer its own adapters, activations and slice of the table):
    every output equals the per-block call bit for bit at decode sizes and matches the oracle; repeated calls agree."""
    import dataclasses
    from tests.parity_utils import oracle_weight
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    n = len(cfg.projections)
    offsets = wl.make_segments(cfg)
    T = int(offsets[-1])
    d_off = to_dev(torch, offsets)
    # one table for all layers: layer l owns columns [l * d, (l + 1) * d), drawn by the oracle
    rng = np.random.default_rng(77)
    sigma = rng.uniform(0.05, 1.0, size=(cfg.P, n_layers * cfg.d)).astype(np.float32)
    d_sigma = to_dev(torch, sigma)
    layers, host = [], []
    for l in range(n_layers):
        cfg_l = dataclasses.replace(cfg, cfg_id=cfg.cfg_id * 100 + l)  # another seed per layer: distinct weights and tokens
        ads = [wl.make_adapter(cfg_l, i) for i in range(n)]
        hs = [ctx.load_adapter(a) for a in ads]
        xs_h = [wl.make_tokens(cfg_l, i, T) for i in range(n)]
        xs = [to_dev(torch, x, torch.bfloat16) for x in xs_h]
        ys = [torch.empty((T, a.d_out), dtype=torch.bfloat16, device="cuda") for a in ads]
        cols = [(l * cfg.d + a, l * cfg.d + b) for a, b in (cfg.sigma_cols(i) for i in range(n))]
        layers.append([(hs[i], xs[i], cols[i], ys[i]) for i in range(n)])
        host.append((ads, xs_h, cols))
    launches0 = ctx.gpu_launches
    ctx.apply_layers(layers, d_off, d_sigma)
    torch.cuda.synchronize()
    if T <= 256:
        assert ctx.gpu_launches - launches0 == n_layers, "one launch per layer at decode sizes"
    first = [[y.clone() for (_, _, _, y) in layer] for layer in layers]
    tol = TOL_BF16 if cfg.w0_dtype == "bf16" else TOL_INT8
    for l, (ads, xs_h, cols) in enumerate(host):
        ys_blk = ctx.apply_block([it[0] for it in layers[l]], [it[1] for it in layers[l]], d_off, d_sigma, cols)
        torch.cuda.synchronize()
        for i in range(n):
            if T <= 256:
                assert torch.equal(first[l][i], ys_blk[i]), (l, i)
            want = orc.apply_projection(oracle_weight(ads[i]), ads[i].U_A, ads[i].V_A, ads[i].U_B, ads[i].V_B, xs_h[i], offsets,
                                        sigma, cols[i][0], cols[i][1], ads[i].rank)
            assert orc.relative_error(first[l][i].float().cpu().numpy(), want) <= tol, (l, i)
    for _ in range(3):  # the chained launches reuse the two scratch sets: results must not depend on timing
        ctx.apply_layers(layers, d_off, d_sigma)
    torch.cuda.synchronize()
    if T <= 256:
        for l in range(n_layers):
            for i in range(n):
                assert torch.equal(first[l][i], layers[l][i][3]), (l, i)
    for layer in layers:
        for it in layer:
            it[0].free()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("3", 512, 128, 16, 100, 1),     # decode sizes: one copy in, one block launch
                                               ("2", 512, 128, 16, 5, 1000)])  # 5000 tokens: the chunked three-stage pipeline
def test_host_block_call_with_shared_activations(torch, ctx, base, dm, dkv, r, P, L):
    """q, k and v reading ONE host activation buffer (as in an attention block): the host-buffer call stages it once;
    every output still matches the oracle."""
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    n = len(cfg.projections)
    x_qkv, x_o = case.tokens(0), case.tokens(3)
    xh_qkv = torch.from_numpy(x_qkv).to(torch.bfloat16).pin_memory()
    xh_o = torch.from_numpy(x_o).to(torch.bfloat16).pin_memory()
    xs_h = [xh_qkv, xh_qkv, xh_qkv, xh_o]
    ys_h = [torch.empty((case.T, case.adapters[i].d_out), dtype=torch.bfloat16).pin_memory() for i in range(n)]
    off_h = torch.from_numpy(case.offsets).pin_memory()
    sig_h = torch.from_numpy(case.sigma32).pin_memory()
    cols = [cfg.sigma_cols(i) for i in range(n)]
    ctx.apply_block_host([case.handles[i] for i in range(n)], xs_h, off_h, sig_h, cols, ys_h)
    for i in range(n):
        want = case.oracle_projection(i, x_o if i == 3 else x_qkv)
        assert orc.relative_error(ys_h[i].float().numpy(), want) <= TOL_BF16, i
    case.close()
