"""Helpers shared by the GPU parity tests: run one workload through the C-ABI library and the CPU oracle.

Data flow is one-way: seeded generator -> {oracle, CUDA}.  Nothing the CUDA path produced is ever fed to the
oracle; the sigma table used for projection parity is the ORACLE's sample rounded to fp32 (both sides then
consume identical fp32 values).
"""
from __future__ import annotations

import numpy as np

from oracle import essa_oracle as orc
from paper_2507_04453_b200 import workloads as wl

TOL_BF16 = 2e-2   # max |g-o| / max(|o|, rms(o)) for bf16 outputs
TOL_INT8 = 4e-2   # same, INT8-weight variant
TOL_SIGMA = 1e-6  # max |g-o| / max(1, |o|) for fp32 sampled singular values


def sigma_error(got: np.ndarray, want: np.ndarray) -> float:
    want = np.asarray(want, dtype=np.float64)
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - want) / np.maximum(1.0, np.abs(want)))) if want.size else 0.0


def oracle_weight(ad: wl.Adapter) -> np.ndarray:
    if ad.w0_dtype == "bf16":
        return ad.W0.astype(np.float64)
    if ad.w0_dtype == "int4":
        return orc.dequantize_int4(ad.W0_q, ad.W0_scale)
    return orc.dequantize_int8(ad.W0_q, ad.W0_scale)


def oracle_sigma_fp32(cma: wl.CmaState, P: int) -> np.ndarray:
    """The oracle's population, rounded once to fp32 (the storage type of the sigma table)."""
    s = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, P)
    return s.astype(np.float32)


def to_dev(torch, a, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(a))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


class Case:
    """All inputs of one configuration, on host (numpy) and device (torch)."""

    def __init__(self, torch, ctx, cfg: wl.WorkloadConfig, projections=None):
        self.torch, self.ctx, self.cfg = torch, ctx, cfg
        self.proj_ids = list(range(len(cfg.projections))) if projections is None else list(projections)
        self.adapters = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
        self.cma = wl.make_cma_state(cfg, self.adapters)
        self.offsets = wl.make_segments(cfg)
        self.T = int(self.offsets[-1])
        self.sigma32 = oracle_sigma_fp32(self.cma, cfg.P)
        self.d_offsets = to_dev(torch, self.offsets)
        self.d_sigma = to_dev(torch, self.sigma32)
        self.handles = {i: ctx.load_adapter(self.adapters[i]) for i in self.proj_ids}

    def tokens(self, i):
        return wl.make_tokens(self.cfg, i, self.T)

    def gpu_projection(self, i, x_host, path="tc"):
        torch = self.torch
        x = to_dev(torch, x_host, torch.bfloat16)
        sA, sB = self.cfg.sigma_cols(i)
        fn = self.ctx.apply_projection if path == "tc" else self.ctx.apply_projection_simt
        y = fn(self.handles[i], x, self.d_offsets, self.d_sigma, sA, sB)
        torch.cuda.synchronize()
        return y.float().cpu().numpy()

    def oracle_projection(self, i, x_host, candidates=None):
        ad = self.adapters[i]
        sA, sB = self.cfg.sigma_cols(i)
        return orc.apply_projection(oracle_weight(ad), ad.U_A, ad.V_A, ad.U_B, ad.V_B, x_host, self.offsets,
                                    self.sigma32, sA, sB, ad.rank, candidates=candidates)

    def close(self):
        for h in self.handles.values():
            h.free()
