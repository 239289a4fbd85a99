"""CPU-side checks of the C-ABI library: it loads, exports what include/essa.h declares, and its host-only
entry points (planner, segment validation, status strings) behave.  No kernel runs here."""
import os
import re

import numpy as np
import pytest

from paper_2507_04453_b200 import binding, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2507_04453_b200 import build
    build.build()
    return binding.load_library()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "essa.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(essa_[a-z0-9_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTED_SYMBOLS)
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.essa_version() >= 100


def test_status_strings(lib):
    seen = set()
    for code in range(0, -7, -1):
        s = lib.essa_status_string(code).decode()
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 7
    assert lib.essa_status_string(-99).decode() == "unknown status"


def test_create_without_device_fails_loudly(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.EssaError) as e:
        binding.Context(0)
    assert e.value.status == binding.ESSA_ERR_NO_DEVICE


def test_validate_segments(lib):
    ok = binding.ESSA_OK
    assert binding.validate_segments([0, 3, 3, 7], 7) == ok
    assert binding.validate_segments([0], 0) == ok
    assert binding.validate_segments([0, 0, 0], 0) == ok
    assert binding.validate_segments([1, 3, 7], 7) != ok     # does not start at 0
    assert binding.validate_segments([0, 5, 4, 7], 7) != ok  # decreasing
    assert binding.validate_segments([0, 3, 6], 7) != ok     # does not end at T
    for name in ("1", "2", "3", "4", "5a", "5b", "5c"):
        off = wl.make_segments(wl.CONFIGS[name])
        assert binding.validate_segments(off, int(off[-1])) == ok


@pytest.mark.parametrize("name", ["1", "2", "3", "4", "5a", "5b", "5c", "6a", "6b"])
def test_plan_is_consistent(lib, name):
    cfg = wl.CONFIGS[name]
    T = int(wl.make_segments(cfg)[-1])
    dtype = {"bf16": binding.ESSA_W0_BF16, "int8": binding.ESSA_W0_INT8_PERCHANNEL, "int4": binding.ESSA_W0_INT4_GROUP128}[cfg.w0_dtype]
    for _, n, m in cfg.projections:
        p = binding.plan_projection(n, m, cfg.rank, dtype, T, 148)
        ext = 2 if dtype == binding.ESSA_W0_INT8_PERCHANNEL else 1
        assert p["k_blocks"] == n // 64 + ext
        if T <= 256:
            # decode schedule: 128 W0 rows per CTA, all tokens in one tile, reduction split over a cluster
            assert p["decode"] == 1 and p["block_m"] == 128 and p["block_k"] == 64
            assert p["block_n"] == -(-T // 16) * 16 and p["tiles"] == -(-m // 128)
            assert p["splits"] in (1, 2, 4, 8) and p["splits"] <= n // 64 and p["grid"] <= {1: 148, 2: 148, 4: 132, 8: 120}[p["splits"]]
            assert p["grid"] == p["tiles"] * p["splits"] and p["scratch_bytes"] == 0
            # bf16 storage: 16 KB W0 tiles.  Quantised storage: 8 KB (INT8) or 4 KB (INT4) tiles of codes; at most 128
            # tokens the converted tiles live in tensor memory and two 16 KB slots hold the U_B slabs, above that
            # (INT8 only) four converted tiles sit in shared memory.  Two 8 KB tiles of V_A^T in every mode.
            w_slot = {binding.ESSA_W0_BF16: 128 * 128, binding.ESSA_W0_INT8_PERCHANNEL: 64 * 128, binding.ESSA_W0_INT4_GROUP128: 32 * 128}[dtype]
            slots16k = 0 if dtype == binding.ESSA_W0_BF16 else 2 if p["block_n"] <= 128 else 4
            rings = 2 * 64 * 128 + p["stages"] * w_slot + slots16k * 128 * 128 + p["x_stages"] * p["block_n"] * 128
            assert 1 <= p["stages"] <= 16 and 1 <= p["x_stages"] <= 6
            assert 1024 + rings + 8192 <= 227 * 1024
            per = -(-(-(-p["block_n"] // p["splits"])) // 16) * 16
            assert rings >= p["splits"] * per * 128 * 4  # the receive buffer overlays the rings
            continue
        assert p["decode"] == 0
        assert p["block_m"] == 128 and p["block_k"] == 64 and p["block_n"] in (64, 128, 256)
        m_tiles = -(-T // 128)
        assert p["tiles"] == m_tiles * -(-m // p["block_n"])
        assert 1 <= p["splits"] <= p["k_blocks"]
        assert 1 <= p["grid"] <= 148 and p["grid"] <= p["tiles"] * p["splits"]
        assert 1 <= p["down_splits"] <= n // 64 and 1 <= p["down_grid"] <= 148
        assert p["stages"] >= 3
        if p["tiles"] >= 148:
            assert p["splits"] == 1  # enough tiles: no split-K
        else:
            assert p["tiles"] * p["splits"] <= 148 + p["tiles"]  # one wave
        assert p["scratch_bytes"] >= T * 128


def test_plan_rejects_bad_shapes(lib):
    with pytest.raises(binding.EssaError):
        binding.plan_projection(100, 128, 8, 0, 16)      # d_in not a multiple of 64
    with pytest.raises(binding.EssaError):
        binding.plan_projection(128, 130, 8, 0, 16)      # d_out not a multiple of 8
    with pytest.raises(binding.EssaError):
        binding.plan_projection(128, 128, 65, 0, 16)     # rank too large
    with pytest.raises(binding.EssaError):
        binding.plan_projection(128, 128, 8, 7, 16)      # unknown dtype
    assert binding.plan_projection(128, 128, 8, 0, 0)["tiles"] == 0


def test_workload_generator_is_deterministic_and_exact():
    cfg = wl.scaled_config("5c", d_model=128, d_kv=64, rank=8, P=6, seg_len=5)
    a, b = wl.make_adapter(cfg, 1), wl.make_adapter(cfg, 1)
    assert np.array_equal(a.W0_q, b.W0_q) and np.array_equal(a.V_A, b.V_A)
    assert a.W0_q.dtype == np.int8 and np.abs(a.W0_q.astype(int)).max() <= 127 and a.W0_scale.dtype == np.float16
    wl.bf16_bits(a.U_B)  # raises if not bf16-representable
    x = wl.make_tokens(cfg, 0, 11)
    assert np.array_equal(wl.bf16_bits_to_f32(wl.bf16_bits(x)), x)
    off = wl.make_segments(cfg)
    assert list(np.diff(off)) == [1, 5, 1, 5, 1, 5]
    # bf16 rounding is round-to-nearest-even
    v = np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -9], dtype=np.float32)
    assert list(wl.round_to_bf16(v)) == [1.0, 1.0 + 2.0 ** -6, 1.0]
    assert abs(np.linalg.norm(a.V_A.astype(np.float64).T @ a.V_A.astype(np.float64) - np.eye(8))) < 0.05


def test_top_alpha_index_host(lib):
    """essa_top_alpha_index against the paper's stated rounding and the oracle's own count."""
    from oracle import essa_oracle as orc
    assert binding.top_alpha_index(8, 8, 0.1) == []                      # rank 8, alpha 0.1: zero trainable values
    assert binding.top_alpha_index(1, 100, 0.29) == list(range(29))      # exact decimal arithmetic
    for n_f, r, alpha in [(3, 4, 0.5), (2, 16, 0.3), (8, 16, 1.0), (4, 64, 0.75), (2, 7, "1/3")]:
        want = orc.top_alpha_index(n_f, r, alpha if alpha != "1/3" else "1/3")
        assert binding.top_alpha_index(n_f, r, alpha) == [int(v) for v in want]
    with pytest.raises(binding.EssaError):
        binding.top_alpha_index(2, 8, 1.5)
