"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Integer work (Philox words, segment map) must match bit for bit; sampled singular values within 1e-6;
bf16 projection outputs within 2e-2 (4e-2 with INT8 weights) of max(|o|, rms(o)).
"""
import dataclasses

import numpy as np
import pytest

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import workloads as wl
from tests.parity_utils import TOL_BF16, TOL_INT8, TOL_SIGMA, Case, oracle_weight, sigma_error, to_dev

pytestmark = pytest.mark.gpu


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


# ------------------------------------------------------------------ integer stream, segment map
def test_device_philox_known_answers(ctx, philox_kat):
    for ctr, key, want in philox_kat:
        assert ctx.debug_philox(ctr, key) == want


def test_stream_words_bit_exact(ctx):
    for seed, k_begin, k_count, nb in [(0, 0, 4, 4), (3, 0, 256, 32), ((0xDEADBEEF << 32) | 0x1234567, 1000, 37, 129)]:
        got = ctx.debug_stream_words(seed, k_begin, k_count, nb).cpu().numpy().view(np.uint32)
        want = orc.candidate_stream_words(seed, np.arange(k_begin, k_begin + k_count), nb)
        assert np.array_equal(got, want)


def test_segment_map_bit_exact(torch, ctx):
    rng = np.random.default_rng(11)
    cases = [np.array([0, 16, 32, 48, 64]), np.arange(257), wl.make_segments(wl.CONFIGS["4"]),
             wl.make_segments(wl.CONFIGS["5c"])]
    for _ in range(5):
        lens = rng.integers(0, 7, size=rng.integers(1, 300))
        lens[rng.integers(0, len(lens))] += 1  # at least one token
        cases.append(np.concatenate([[0], np.cumsum(lens)]))
    for off in cases:
        off = off.astype(np.int32)
        T = int(off[-1])
        got = ctx.debug_segment_map(to_dev(torch, off), T).cpu().numpy()
        assert np.array_equal(got, orc.candidate_of_token(off, T))


# ------------------------------------------------------------------ sampling
@pytest.mark.parametrize("name", ["1", "2", "3", "4", "5a"])
def test_sampled_sigma_matches_oracle(torch, ctx, name):
    cfg = wl.CONFIGS[name]
    adapters = [wl.make_adapter(_tiny_like(cfg), i) for i in range(len(cfg.projections))]
    cma = wl.make_cma_state(_tiny_like(cfg), adapters)
    want = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    got = ctx.sample_population(to_dev(torch, cma.mean), cma.step,
                                None if cma.Bfactor is None else to_dev(torch, cma.Bfactor),
                                None if cma.Dvec is None else to_dev(torch, cma.Dvec), cma.seed, cfg.P)
    torch.cuda.synchronize()
    assert got.shape == (cfg.P, cfg.d)
    assert sigma_error(got.cpu().numpy(), want) <= TOL_SIGMA


def _tiny_like(cfg):
    """Same rank / P / CMA-ES structure, small matrices (the sampler does not depend on d_model)."""
    if len(cfg.projections) == 1:
        return cfg
    return dataclasses.replace(cfg, projections=wl._qkvo(128, 64))


def test_sampler_general_cases(torch, ctx):
    rng = np.random.default_rng(12)
    for d, P, full, step, seed in [(1, 1, False, 1.0, 1), (7, 5, True, 0.32, 2), (130, 33, True, 0.32, (9 << 32) + 5),
                                   (512, 128, True, 0.32, 77), (1792, 64, False, 0.32, 4), (1030, 9, True, 2.0, 8)]:
        mean = rng.standard_normal(d).astype(np.float32)
        Dv = rng.uniform(0.5, 1.5, d).astype(np.float32)
        Bf = (rng.standard_normal((d, d)) / np.sqrt(d)).astype(np.float32) if full else None
        want = orc.sample_population(mean, np.float32(step), Bf, Dv, seed, P)
        got = ctx.sample_population(to_dev(torch, mean), step, None if Bf is None else to_dev(torch, Bf),
                                    to_dev(torch, Dv), seed, P)
        assert sigma_error(got.cpu().numpy(), want) <= TOL_SIGMA, (d, P, full)
    # zero candidates is a no-op
    out = ctx.sample_population(to_dev(torch, np.zeros(4, np.float32)), 1.0, None, None, 0, 0)
    assert out.shape == (0, 4)


def test_masked_sampler_matches_oracle(torch, ctx):
    """Top-alpha selection: only some columns of the table are drawn, the rest keep their frozen values."""
    from paper_2507_04453_b200 import binding
    rng = np.random.default_rng(21)
    for n_f, r, alpha, P, full, k_begin in [(8, 16, 0.5, 64, True, 0), (8, 16, 0.25, 33, False, 5), (8, 8, 0.1, 4, True, 0),
                                            (2, 64, 1.0, 16, True, 0), (6, 33, "1/3", 9, True, 3)]:
        d = n_f * r
        idx = orc.top_alpha_index(n_f, r, alpha)
        assert binding.top_alpha_index(n_f, r, alpha) == [int(v) for v in idx]
        dt = idx.size
        frozen = rng.standard_normal(d).astype(np.float32)
        mean_t = rng.standard_normal(dt).astype(np.float32)
        Dv = rng.uniform(0.5, 1.5, dt).astype(np.float32)
        Bf = (rng.standard_normal((dt, dt)) / np.sqrt(max(dt, 1))).astype(np.float32) if full and dt else None
        seed = (7 << 32) + 13
        want = orc.sample_population_masked(frozen, idx, mean_t, np.float32(0.32), Bf, Dv, seed, P, k_begin)
        got = ctx.sample_population_masked(to_dev(torch, frozen), to_dev(torch, idx.astype(np.int32)) if dt else None,
                                           to_dev(torch, mean_t) if dt else None, 0.32,
                                           None if Bf is None else to_dev(torch, Bf), to_dev(torch, Dv) if dt else None,
                                           seed, P, k_begin=k_begin)
        torch.cuda.synchronize()
        got = got.cpu().numpy()
        assert got.shape == (P, d)
        assert sigma_error(got, want) <= TOL_SIGMA, (n_f, r, alpha)
        rest = np.setdiff1d(np.arange(d), idx)
        assert np.array_equal(got[:, rest], np.tile(frozen[rest], (P, 1)))  # frozen columns are bit-exact copies


def test_sampler_range_regenerates_any_member(torch, ctx):
    rng = np.random.default_rng(13)
    d, P = 128, 64
    mean = to_dev(torch, rng.standard_normal(d).astype(np.float32))
    Bf = to_dev(torch, np.linalg.qr(rng.standard_normal((d, d)))[0].astype(np.float32))
    full = ctx.sample_population(mean, 0.05, Bf, None, 5, P).cpu().numpy()
    part = ctx.sample_population(mean, 0.05, Bf, None, 5, 10, k_begin=37).cpu().numpy()
    assert np.array_equal(part, full[37:47])  # bit-identical: a member depends on <seed, k> only


# ------------------------------------------------------------------ adapter preparation
def test_core_matrix(torch, ctx):
    cfg = wl.CONFIGS["1"]
    ad = wl.make_adapter(cfg, 0)
    h = ctx.load_adapter(ad)
    M = ctx.debug_core_matrix(h)
    want = ad.V_B.astype(np.float64).T @ ad.U_A.astype(np.float64)
    np.testing.assert_allclose(M, want, rtol=0, atol=2e-6)
    h.free()


# ------------------------------------------------------------------ projection, full outputs vs oracle
def _check_projection(case, i, tol, paths=("tc", "simt"), candidates=None):
    x = case.tokens(i)
    want = case.oracle_projection(i, x, candidates)
    errs = {}
    for path in paths:
        got = case.gpu_projection(i, x, path)
        assert got.shape == want.shape
        assert np.isfinite(got).all()
        errs[path] = orc.relative_error(got, want)
        assert errs[path] <= tol, (case.cfg.name, case.cfg.projections[i], path, errs[path])
    return errs


def test_config1_full(torch, ctx):
    case = Case(torch, ctx, wl.CONFIGS["1"])
    errs = _check_projection(case, 0, TOL_BF16)
    assert errs["tc"] < 8e-3, errs  # expected ~4e-3: bf16 output rounding + bf16 rank-r intermediate
    case.close()


SCALED = {
    # name: (base, d_model, d_kv, rank, P, seg_len)
    "prefill-r16": ("2", 512, 128, 16, 8, 200),     # T = 1600: 12.5 token tiles, 2-4 channel tiles
    "decode-r16": ("3", 1024, 192, 16, 256, 1),      # T = 256, split-K path, d_kv not a tile multiple
    "ragged-r32": ("4", 640, 128, 32, 24, 300),      # ragged segments, d_out = 640 = 2.5 x 256
    "int8-decode-r64": ("5a", 1024, 256, 64, 128, 1),
    "int8-prefill-r64": ("5b", 768, 128, 64, 16, 100),
    "int8-mixed-r64": ("5c", 512, 128, 64, 32, 90),
    "int4-decode-r64": ("6a", 1024, 256, 64, 128, 1),     # INT4 group-wise storage, tensor-memory decode mode
    "int4-prefill-r64": ("6b", 768, 128, 64, 16, 100),    # ... dequantised per call for the prefill kernels
    "int4-decode-256": ("6a", 512, 128, 32, 200, 1),      # 200 tokens: above the decode mode's limit, prefill kernels
}


@pytest.mark.parametrize("name", list(SCALED))
def test_scaled_configs_full_outputs(torch, ctx, name):
    base, dm, dkv, r, P, L = SCALED[name]
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg)
    tol = TOL_BF16 if cfg.w0_dtype == "bf16" else TOL_INT8
    for i in range(len(cfg.projections)):
        _check_projection(case, i, tol)
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("2", 1024, 256, 16, 4, 700),    # T = 2800: the last 512-token tile holds 240 rows
                                               ("4", 768, 256, 32, 24, 300),    # ragged segments, three channel tiles
                                               ("2", 1024, 256, 33, 13, 197),   # T = 2561: one row in the last tile; padded rank 48
                                               ("5b", 2048, 512, 64, 16, 128),  # INT8 storage: two rank slabs, scale in the epilogue
                                               ("6b", 2048, 512, 64, 9, 130),   # INT4 group-wise storage
                                               ("4", 640, 640, 32, 24, 300)])   # 640 channels = 2.5 channel tiles: W0 rows beyond d_out read as zeros, stores clipped
def test_wide_pair_tiles(torch, ctx, base, dm, dkv, r, P, L):
    """Prefill base + up on 512-token x 256-channel pair tiles (ESSA_OPT_WIDE_TILES = 2) matches the oracle, and the
    256 x 256 pair tiles (ESSA_OPT_WIDE_TILES = 0) to the last bit or so: both add the K blocks in the same order in
    fp32; only u can differ in its last bit between two calls (the rank-down launch splits K at these token counts and
    adds its partial sums in arrival order)."""
    from paper_2507_04453_b200 import binding
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg, projections=[0])
    tol = TOL_BF16 if cfg.w0_dtype == "bf16" else TOL_INT8
    code = {"bf16": 0, "int8": 1, "int4": 2}[cfg.w0_dtype]
    plan = binding.plan_projection(dm, dm, r, code, case.T)
    assert plan["block_n"] == 256 and plan["splits"] == 1 and case.T >= 512  # the shape the pair tiles take
    x = case.tokens(0)
    want = case.oracle_projection(0, x)
    try:
        outs = {}
        for wide in (2, 0):
            ctx.set_option(binding.ESSA_OPT_WIDE_TILES, wide)
            outs[wide] = case.gpu_projection(0, x)
            assert np.isfinite(outs[wide]).all()
        assert orc.relative_error(outs[2], want) <= tol
        assert np.mean(outs[2] != outs[0]) < 0.02 and orc.relative_error(outs[2], outs[0].astype(np.float64)) <= 8e-3
    finally:
        ctx.set_option(binding.ESSA_OPT_WIDE_TILES, 1)
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P,L", [("2", 1024, 256, 16, 4, 700),    # T = 2800: 11 token tiles, ragged last tile
                                               ("2", 1024, 256, 33, 8, 300),    # padded rank 48
                                               ("5b", 2048, 512, 64, 16, 128)])  # INT8 storage, rank 64, five stages
def test_pair_tiles_with_fused_down_projection(torch, ctx, base, dm, dkv, r, P, L):
    """Prefill-sized call on 256-channel tiles: the pair-tile launch that also computes u (ESSA_OPT_FUSE_DOWN = 2) and the
    two-launch schedule (ESSA_OPT_FUSE_DOWN = 0) both match the oracle; the fused one is deterministic."""
    from paper_2507_04453_b200 import binding
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=L)
    case = Case(torch, ctx, cfg, projections=[0])
    tol = TOL_INT8 if cfg.w0_dtype == "int8" else TOL_BF16
    plan = binding.plan_projection(dm, dm, r, 1 if cfg.w0_dtype == "int8" else 0, case.T)
    assert plan["block_n"] == 256 and plan["splits"] == 1 and case.T >= 512  # the shape the pair tiles take
    x = case.tokens(0)
    want = case.oracle_projection(0, x)
    try:
        outs, counts = {}, {}
        for fuse in (2, 0):  # 2 = fused at any token count, 0 = the default two-launch schedule
            ctx.set_option(binding.ESSA_OPT_FUSE_DOWN, fuse)
            n0 = ctx.gpu_launches
            got = case.gpu_projection(0, x, "tc")
            counts[fuse] = ctx.gpu_launches - n0
            assert np.isfinite(got).all()
            assert orc.relative_error(got, want) <= tol, (cfg.name, fuse)
            outs[fuse] = got
        assert counts[0] - counts[2] == 1  # the rank-down launch is gone
        ctx.set_option(binding.ESSA_OPT_FUSE_DOWN, 2)
        again = case.gpu_projection(0, x, "tc")
        assert np.array_equal(again, outs[2])
    finally:
        ctx.set_option(binding.ESSA_OPT_FUSE_DOWN, 0)
    case.close()


@pytest.mark.parametrize("rank", [1, 3, 8, 17, 33, 48, 64])
def test_rank_padding(torch, ctx, rank):
    cfg = wl.scaled_config("1", d_model=256, d_kv=256, rank=rank, P=5, seg_len=37)
    case = Case(torch, ctx, cfg)
    _check_projection(case, 0, TOL_BF16)
    case.close()


def test_edge_cases(torch, ctx):
    cfg = wl.scaled_config("1", d_model=192, d_kv=192, rank=8, P=6, seg_len=1)
    case = Case(torch, ctx, cfg)
    ad, h = case.adapters[0], case.handles[0]
    sA, sB = cfg.sigma_cols(0)
    W = oracle_weight(ad)

    def run(offsets, T):
        x = wl.make_tokens(cfg, 0, T)
        d_off = to_dev(torch, np.asarray(offsets, dtype=np.int32))
        want = orc.apply_projection(W, ad.U_A, ad.V_A, ad.U_B, ad.V_B, x, offsets, case.sigma32, sA, sB, ad.rank)
        for fn in (ctx.apply_projection, ctx.apply_projection_simt):
            got = fn(h, to_dev(torch, x, torch.bfloat16) if T else torch.empty((0, 192), dtype=torch.bfloat16, device="cuda"),
                     d_off, case.d_sigma, sA, sB)
            torch.cuda.synchronize()
            assert got.shape == (T, 192)
            if T:
                assert orc.relative_error(got.float().cpu().numpy(), want) <= TOL_BF16

    run([0, 0, 0, 0, 0, 0, 0], 0)            # empty input: legal no-op
    run([0, 1, 1, 1, 1, 1, 1], 1)            # one token, trailing empty segments
    run([0, 0, 0, 0, 0, 0, 129], 129)        # leading empty segments, one token past a tile
    run([0, 127, 128, 129, 129, 300, 385], 385)  # boundaries around the 128-token tile edge, ragged tail
    case.close()


def test_zero_sigma_gives_base_projection_and_is_deterministic(torch, ctx):
    cfg = wl.scaled_config("2", d_model=512, d_kv=128, rank=16, P=4, seg_len=160)
    case = Case(torch, ctx, cfg)
    x = case.tokens(0)
    dx = to_dev(torch, x, torch.bfloat16)
    sA, sB = cfg.sigma_cols(0)
    zero = torch.zeros_like(case.d_sigma)
    y0 = ctx.apply_projection(case.handles[0], dx, case.d_offsets, zero, sA, sB).float().cpu().numpy()
    base = x.astype(np.float64) @ oracle_weight(case.adapters[0]).T
    assert orc.relative_error(y0, base) <= 6e-3  # only the final bf16 rounding
    case.close()


@pytest.mark.parametrize("P,split_k", [(64, False), (4, True)])
def test_repeated_calls_agree(torch, ctx, P, split_k):
    """No data race, no dependence on stale TMEM / shared memory / workspace contents between calls.
    Without split-K the result is bit-identical run to run; with split-K the fp32 partial sums meet in
    arrival order, so runs may differ by the last bf16 bit."""
    from paper_2507_04453_b200 import binding
    cfg = wl.scaled_config("2", d_model=512, d_kv=128, rank=16, P=P, seg_len=160)
    plan = binding.plan_projection(512, 512, 16, binding.ESSA_W0_BF16, P * 160, 148)
    assert (plan["splits"] > 1) == split_k
    case = Case(torch, ctx, cfg, projections=[0])
    dx = to_dev(torch, case.tokens(0), torch.bfloat16)
    sA, sB = cfg.sigma_cols(0)
    a = ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB).clone()
    for _ in range(4):
        b = ctx.apply_projection(case.handles[0], dx, case.d_offsets, case.d_sigma, sA, sB)
        if split_k:
            assert torch.allclose(a.float(), b.float(), rtol=2.0 ** -7, atol=1e-3)
        else:
            assert torch.equal(a, b)
    case.close()


def test_host_buffer_entry_point(torch, ctx):
    cfg = wl.scaled_config("4", d_model=256, d_kv=64, rank=32, P=7, seg_len=50)
    case = Case(torch, ctx, cfg)
    x = case.tokens(1)
    sA, sB = cfg.sigma_cols(1)
    xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    yh = torch.empty((case.T, 64), dtype=torch.bfloat16).pin_memory()
    ctx.apply_projection_host(case.handles[1], xh, torch.from_numpy(case.offsets), torch.from_numpy(case.sigma32),
                              sA, sB, yh)
    want = case.oracle_projection(1, x)
    assert orc.relative_error(yh.float().numpy(), want) <= TOL_BF16
    # offsets that do not end at T are rejected on the host
    from paper_2507_04453_b200.binding import EssaError
    bad = torch.from_numpy(case.offsets.copy())
    bad[-1] += 1
    with pytest.raises(EssaError):
        ctx.apply_projection_host(case.handles[1], xh, bad, torch.from_numpy(case.sigma32), sA, sB, yh)
    case.close()


def test_host_buffer_entry_point_pipelined_chunks(torch, ctx):
    """A call of several thousand tokens is cut into chunks of whole candidates that pipeline copies and compute:
    ragged segments (some empty), pinned and pageable host memory, all against the oracle and equal to each
    other up to the last bf16 bit; later calls re-use the staging buffers."""
    cfg = wl.scaled_config("4", d_model=512, d_kv=128, rank=32, P=40, seg_len=300)  # ragged lengths, T of several thousand
    case = Case(torch, ctx, cfg, projections=[0])
    off = case.offsets.copy()
    off[5] = off[4]            # an empty candidate inside a chunk
    off[21:23] = off[20]       # ... and two at what would be a chunk boundary
    assert case.T >= 3 * 2048 and np.all(np.diff(off) >= 0)
    x = case.tokens(0)
    sA, sB = cfg.sigma_cols(0)
    ad = case.adapters[0]
    want = orc.apply_projection(oracle_weight(ad), ad.U_A, ad.V_A, ad.U_B, ad.V_B, x, off, case.sigma32, sA, sB, ad.rank)
    xh = torch.from_numpy(x).to(torch.bfloat16)
    outs = []
    for pinned in (True, False, True):
        xin = xh.pin_memory() if pinned else xh.clone()
        yh = torch.zeros((case.T, ad.d_out), dtype=torch.bfloat16)
        yh = yh.pin_memory() if pinned else yh
        ctx.apply_projection_host(case.handles[0], xin, torch.from_numpy(off), torch.from_numpy(case.sigma32), sA, sB, yh)
        got = yh.float().numpy()
        assert np.isfinite(got).all()
        assert orc.relative_error(got, want) <= TOL_BF16
        outs.append(got)
    for other in outs[1:]:  # (chunks of this size take the split-K schedule, whose fp32 add order varies: last-bit differences)
        assert np.max(np.abs(outs[0] - other) / np.maximum(1.0, np.abs(outs[0]))) <= 2.0 ** -7
    assert ctx.get_status() == 0
    case.close()


@pytest.mark.parametrize("base,dm,dkv,r,P", [("2", 512, 128, 16, 9), ("4", 640, 128, 33, 5), ("5b", 512, 192, 64, 3)])
def test_exported_candidates_match_oracle(torch, ctx, base, dm, dkv, r, P):
    """essa_export_candidates: A'_k and B'_k of a range of candidates against the oracle's reconstruction, and the
    product B'_k A'_k x against the library's own projection of the same candidate (the two routes to W' x)."""
    cfg = wl.scaled_config(base, d_model=dm, d_kv=dkv, rank=r, P=P, seg_len=40)
    case = Case(torch, ctx, cfg, projections=[1])
    ad = case.adapters[1]
    sA, sB = cfg.sigma_cols(1)
    k0, kc = 1, P - 1
    A, B = ctx.export_candidates(case.handles[1], case.d_sigma, sA, sB, k0, kc)
    torch.cuda.synchronize()
    assert A.shape == (kc, ad.rank, ad.d_in) and B.shape == (kc, ad.d_out, ad.rank)
    A, B = A.float().cpu().numpy(), B.float().cpu().numpy()
    for kk in range(kc):
        srow = case.sigma32[k0 + kk].astype(np.float64)
        wa, wb = orc.reconstruct_factors(ad.U_A, ad.V_A, ad.U_B, ad.V_B, srow[sA:sA + ad.rank], srow[sB:sB + ad.rank])
        assert orc.relative_error(A[kk], wa) <= 2.0 ** -8, (cfg.name, kk)   # one bf16 rounding of an fp32 sum
        assert orc.relative_error(B[kk], wb) <= 2.0 ** -8, (cfg.name, kk)
    # only one of the two outputs
    A_only, none = ctx.export_candidates(case.handles[1], case.d_sigma, sA, sB, 0, 2, want_b=False)
    assert none is None and A_only.shape[0] == 2
    # the exported factors reproduce the library's projection of that candidate's tokens
    x = case.tokens(1)
    y = case.gpu_projection(1, x)
    lo, hi = int(case.offsets[k0]), int(case.offsets[k0 + 1])
    W0 = oracle_weight(ad)
    via_export = x[lo:hi].astype(np.float64) @ (W0 + B[0].astype(np.float64) @ A[0].astype(np.float64)).T
    tol = TOL_INT8 if cfg.w0_dtype == "int8" else TOL_BF16
    assert orc.relative_error(y[lo:hi], via_export) <= tol
    case.close()


def test_argument_validation(torch, ctx):
    from paper_2507_04453_b200.binding import EssaError
    cfg = wl.scaled_config("1", d_model=128, d_kv=128, rank=8, P=2, seg_len=4)
    case = Case(torch, ctx, cfg)
    x = to_dev(torch, case.tokens(0), torch.bfloat16)
    with pytest.raises(EssaError):  # sigma columns outside the row
        ctx.apply_projection(case.handles[0], x, case.d_offsets, case.d_sigma, 12, 8)
    bad = dataclasses.replace(case.adapters[0], d_in=100)
    with pytest.raises(EssaError):  # d_in not a multiple of 64
        ctx.load_adapter(bad)
    case.close()


def test_sampler_to_projection_end_to_end(torch, ctx):
    """Both chains run on their own: GPU sampler -> GPU projection vs oracle sampler -> oracle projection."""
    cfg = wl.scaled_config("3", d_model=512, d_kv=128, rank=16, P=64, seg_len=1)
    case = Case(torch, ctx, cfg)
    cma = case.cma
    d_sig = ctx.sample_population(to_dev(torch, cma.mean), cma.step, to_dev(torch, cma.Bfactor), to_dev(torch, cma.Dvec),
                                  cma.seed, cfg.P)
    want_sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    for i in range(4):
        x = case.tokens(i)
        ad = case.adapters[i]
        sA, sB = cfg.sigma_cols(i)
        y = ctx.apply_projection(case.handles[i], to_dev(torch, x, torch.bfloat16), case.d_offsets, d_sig, sA, sB)
        want = orc.apply_projection(oracle_weight(ad), ad.U_A, ad.V_A, ad.U_B, ad.V_B, x, case.offsets, want_sigma,
                                    sA, sB, ad.rank)
        assert orc.relative_error(y.float().cpu().numpy(), want) <= TOL_BF16
    case.close()
