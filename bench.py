#!/usr/bin/env python
"""Benchmark of the ESSA population-projection hot path on B200.

One step = one pass of the whole hot path over one synthetic batch: draw the population's singular values
(essa_sample_population) and run the q, k, v, o adapted projections for every candidate's tokens
(essa_apply_block at decode sizes, 4 x essa_apply_projection otherwise).  Metric: candidate-tokens/s (a
candidate-token = one token of one candidate through all projections of the block).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

Without --config the run times the five benchmark workloads (2, 3, 4, 5a, 5b) one after the other in one
process and prints ONE JSON line: its top-level fields describe the largest single-GPU bf16 workload (config 4)
and config.per_config holds the same measurements for each of the five.  With --config C only that workload runs.

N > 1: one rank per GPU (the launcher's RANK / LOCAL_RANK / WORLD_SIZE are used when present; otherwise this
script re-executes itself under torch.distributed.run with N local ranks).  Candidates are independent, so ranks
take disjoint candidate ranges of an N-times larger population with no data-path collective (weak scaling).
Rank 0 prints the line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_2507_04453_b200 import workloads as wl

METRIC = "candidate-tokens/sec through q/k/v/o SVD-LoRA projections"
UNIT = "candidate-tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_PEAKS = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}  # chip figures, printed beside the measured ones
ALL_CONFIGS = ("2", "3", "4", "5a", "5b", "6a", "6b")  # 6a / 6b: the 72B-shaped block with INT4 group-wise weights
HEADLINE = "4"
L2_BYTES = 126e6
CSRC = os.path.join(ROOT, "paper_2507_04453_b200", "csrc")
# DRAM bytes (read + write) per launch of the dominant kernel from the ncu captures summarised under profiles/,
# with the SHA-256 (first 16 hex digits) of the kernel's source file at capture time: a kernel that has changed
# since reports "traffic": null until it is captured again.
NCU_TRAFFIC = {
    "2": {"bytes": 792e6, "source": "proj_tc3.cu", "sha16": "13fd60855285679d", "profile": "profiles/essa_tcw_kernel_cfg2_cfg4_prefill.md",
          "note": "captured at half the population (425.2 MB) and scaled: W0 traffic fixed, x and y traffic doubled"},
    "4": {"bytes": 4787e6, "source": "proj_tc3.cu", "sha16": "13fd60855285679d", "profile": "profiles/essa_tcw_kernel_cfg2_cfg4_prefill.md",
          "note": "full size; captures of the same kernel range from 3.4 to 5.4 GB (how well the CTA pairs stay in step)"},
    "3": {"bytes": 67.9e6, "source": "proj_decode.cu", "sha16": "853fbc3271e38da6", "profile": "profiles/essa_decode_kernel_cfg3_cfg5a.md"},
    "5a": {"bytes": 170.7e6, "source": "proj_decode.cu", "sha16": "853fbc3271e38da6", "profile": "profiles/essa_decode_kernel_cfg3_cfg5a.md"},
}


def source_sha16(name):
    try:
        with open(os.path.join(CSRC, name), "rb") as f:
            return hashlib.sha256(f.read()).hexdigest()[:16]
    except OSError:
        return None


def ncu_traffic(config_key):
    rec = NCU_TRAFFIC.get(config_key)
    if rec is None or not rec["sha16"] or source_sha16(rec["source"]) != rec["sha16"]:
        return None
    return rec["bytes"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ---------------------------------------------------------------------------------------------- work model
def projection_work(n, m, r, T, P, w_bytes):
    """Algorithmic FLOPs and bytes of one projection call and of its dominant (base + up) kernel."""
    flops_call = 2.0 * T * m * n + 2.0 * T * r * (n + m + r) + 3.0 * T * r
    bytes_call = m * n * w_bytes + (2 * m if w_bytes == 1 else 2 * m * n / 128 if w_bytes == 0.5 else 0) + 2.0 * T * n + 2.0 * T * m + 2.0 * n * r + 2.0 * m * r \
        + 4.0 * r * r + 8.0 * P * r + 4.0 * (P + 1)
    flops_main = 2.0 * T * m * (n + r)                       # base contraction + up-projection
    bytes_main = m * n * w_bytes + 2.0 * T * n + 2.0 * T * m + 2.0 * m * r + 2.0 * T * r  # W0, x, y, U_B, u
    return flops_call, bytes_call, flops_main, bytes_main


def block_model(cfg, T):
    """Algorithmic work of the block's projection calls, each bounded by whichever of its FLOPs and bytes is slower
    at NOMINAL peak ratios (the bound does not depend on which measured peak is used: the configurations are far
    from the ridge except 3 and 5a, which are HBM-bound by bytes / copy bandwidth vs FLOPs / burst peak)."""
    w = {"int8": 1, "int4": 0.5}.get(cfg.w0_dtype, 2)  # bytes per weight as stored
    rows = []
    for _, n, m in cfg.projections:
        rows.append(projection_work(n, m, cfg.rank, T, cfg.P, w))
    return rows


def block_roofline(cfg, T, tflops, gbs):
    tf, bw = tflops * 1e12, gbs * 1e9
    t_total, fl, by, fl_main, by_main = 0.0, 0.0, 0.0, 0.0, 0.0
    votes = {"tensor": 0.0, "hbm": 0.0}
    for f, b, fm, bm in block_model(cfg, T):
        t = max(f / tf, b / bw)
        votes["tensor" if f / tf >= b / bw else "hbm"] += t
        t_total += t
        fl += f; by += b; fl_main += fm; by_main += bm
    return {"time_s": t_total, "flops": fl, "bytes": by, "flops_main": fl_main, "bytes_main": by_main,
            "bound": max(votes, key=votes.get)}


# ---------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch, device_index):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            props = torch.cuda.get_device_properties(device_index)
            try:
                bus = "%08x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
                self.h = pynvml.nvmlDeviceGetHandleByPciBusId(bus.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.nv = pynvml
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # no NVML: report that clocks could not be read
            self.nv = None
            self.err = repr(e)

    def _sample(self):
        nv = self.nv
        try:
            self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
            self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._sample()
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join()
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "power_w_max": max(self.power) if self.power else None}


# ---------------------------------------------------------------------------------------------- CPU oracle timing
def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, cands):
    """The oracle, as it stands, on the given candidates (all their tokens, all channels, all projections)."""
    from oracle import essa_oracle as orc
    for i, ad in enumerate(adapters):
        sA, sB = cfg.sigma_cols(i)
        orc.apply_projection(weights[i], ad.U_A, ad.V_A, ad.U_B, ad.V_B, xs[i], offsets, sigma, sA, sB, ad.rank,
                             candidates=cands)


def oracle_setup(cfg, max_candidates=None):
    """Oracle inputs.  Only the tokens of the first max_candidates candidates are generated as fp64 (the timed sample
    never touches the others, and the full fp64 activations of the largest workloads would not fit host memory)."""
    from oracle import essa_oracle as orc
    adapters = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
    offsets = wl.make_segments(cfg)
    T = int(offsets[-1])
    cma = wl.make_cma_state(cfg, adapters)
    weights = [a.W0.astype(np.float64) if a.w0_dtype == "bf16" else orc.dequantize_int4(a.W0_q, a.W0_scale) if a.w0_dtype == "int4"
               else orc.dequantize_int8(a.W0_q, a.W0_scale) for a in adapters]
    kmax = cfg.P if max_candidates is None else min(cfg.P, max_candidates)
    t_need = int(offsets[kmax])
    xs = []
    for i in range(len(adapters)):
        x = wl.make_tokens(cfg, i, T)
        xs.append(np.ascontiguousarray(x[:t_need]).astype(np.float64))
        del x
    return adapters, weights, offsets, T, cma, xs, kmax


def warm_blas():
    """A few fp64 products before timing: the first BLAS calls of a process pay for thread start-up."""
    a = np.ones((512, 512))
    for _ in range(3):
        a = (a @ a) * 1e-3


def time_oracle_sample(cfg, budget_s=15.0, max_candidates=32):
    """cpu_baseline: the oracle timed on a bounded sample (whole candidates, in order) of the workload."""
    from oracle import essa_oracle as orc
    adapters, weights, offsets, T, cma, xs, kmax = oracle_setup(cfg, max_candidates)
    warm_blas()
    oracle_candidates_pass(cfg, adapters, weights, offsets, orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, 1),
                           xs, [0])  # untimed warm-up pass on one candidate
    t0 = time.perf_counter()
    sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    t_sample = time.perf_counter() - t0
    done_tokens, done_c, elapsed = 0, 0, t_sample
    for k in range(kmax):
        t0 = time.perf_counter()
        oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, [k])
        elapsed += time.perf_counter() - t0
        done_tokens += int(offsets[k + 1] - offsets[k])
        done_c += 1
        if elapsed >= budget_s:
            break
    return {"value": done_tokens / elapsed, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"first {done_c} of {cfg.P} candidates ({done_tokens} of {T} tokens), all {len(adapters)} projections, "
                      f"all channels, plus the full population draw; {elapsed:.1f} s after one untimed warm-up candidate; "
                      "numpy fp64 with BLAS matrix products"}


def run_reference(args, cfg):
    """--impl reference: the fp64 CPU oracle on the host cores; each step is a bounded sample of the workload."""
    from oracle import essa_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    adapters, weights, offsets, T, cma, xs, kmax = oracle_setup(cfg, 32)
    warm_blas()
    sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, [0])
    t0 = time.perf_counter()
    oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, [0])
    t1 = max(time.perf_counter() - t0, 1e-4)
    total_steps = args.steps + args.warmup
    c = int(max(1, min(kmax, 100.0 / (total_steps * t1))))  # whole run within a couple of minutes
    cands = list(range(c))
    tokens = int(offsets[c] - offsets[0])
    for _ in range(args.warmup):
        oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, cands)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
        oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, cands)
    dt = time.perf_counter() - t0
    value = tokens * args.steps / dt
    sample = (f"each step: full population draw + first {c} of {cfg.P} candidates ({tokens} of {T} tokens), all projections, "
              "all channels; numpy fp64 with BLAS matrix products")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "tokens_per_step": tokens, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- GPU arm
def measure_config(key, cfg, args, env):
    """All measurements of one workload on this rank's GPU; returns the per-config record (max over ranks applied)."""
    torch, binding, dist = env["torch"], env["binding"], env["dist"]
    world, rank, local_rank = env["world"], env["rank"], env["local_rank"]
    peaks, peak_src = env["peaks"], env["peak_src"]

    ctx = binding.Context(local_rank)
    if args.pair_tiles >= 0:
        ctx.set_option(binding.ESSA_OPT_PAIR_TILES, args.pair_tiles)
    if args.fuse_down >= 0:
        ctx.set_option(binding.ESSA_OPT_FUSE_DOWN, args.fuse_down)
    for item in args.set_option:
        opt, val = item.split("=")
        ctx.set_option(int(opt), int(val))
    adapters = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
    offsets = wl.make_segments(cfg)
    T = int(offsets[-1])
    cma = wl.make_cma_state(cfg, adapters)
    # Weights that fit L2 (decode configurations) would be served from it on every step: rotate through enough
    # device copies of the block's adapters that each step streams its W0 from HBM, as a forward pass over many
    # layers does.
    w_bytes = int(sum(a.d_in * a.d_out * {"int8": 1, "int4": 0.5}.get(cfg.w0_dtype, 2) for a in adapters))  # as stored
    copies = 1 if w_bytes > 2 * L2_BYTES else int(np.ceil(2 * L2_BYTES / w_bytes)) + 1
    handle_sets = [[ctx.load_adapter(a) for a in adapters] for _ in range(copies)]
    handles = handle_sets[0]
    del adapters[:]  # the host copies of the weights are not needed any more
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).cuda()
    xs_host = []
    for i in range(len(handles)):
        xs_host.append(torch.from_numpy(wl.make_tokens(cfg, i, T)).to(torch.bfloat16))
    xs = [x.cuda() for x in xs_host]
    ys = [torch.empty((T, h.d_out), dtype=torch.bfloat16, device="cuda") for h in handles]
    d_off = dev(offsets)
    d_mean = dev(cma.mean)
    d_B = None if cma.Bfactor is None else dev(cma.Bfactor)
    d_D = None if cma.Dvec is None else dev(cma.Dvec)
    sigma = torch.empty((cfg.P, cfg.d), dtype=torch.float32, device="cuda")
    k_begin = rank * cfg.P  # weak scaling: rank g evaluates candidates [g*P, (g+1)*P) of an N*P population
    ctx.reserve(T, max(h.d_in for h in handles), max(h.d_out for h in handles))
    if cfg.w0_dtype != "bf16":
        ctx.reserve_dequant(max(h.d_in for h in handles), max(h.d_out for h in handles))
    stream = torch.cuda.current_stream()

    step_no = [0]
    cols = [cfg.sigma_cols(i) for i in range(len(handles))]
    decode = T <= 256  # one-launch decode schedule (essa_plan.decode)
    # the block's projections share tokens, segments and the table -> one essa_apply_block call (decode sizes: one launch;
    # prefill sizes: the rank-down launches, then one launch for the base + up step of all projections)
    block_call = len(handles) > 1 and not args.single_calls

    # Decode steps are tens of microseconds: their two calls are marshalled once (binding.PreparedSample /
    # PreparedBlock: the same C entry points, argument tuples built ahead of time) so that the host keeps ahead.
    stream_handle = stream.cuda_stream
    prep_sample = ctx.prepare_sample(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, sigma, k_begin)
    prep_blocks = [ctx.prepare_block(hs, xs, d_off, sigma, cols, ys) for hs in handle_sets] if block_call else None
    fused_call = block_call and decode and not args.separate_calls  # (at prefill sizes the draw is a separate call)
    prep_fused = [ctx.prepare_sample_block(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, sigma, hs, xs, d_off, cols, ys, k_begin)
                  for hs in handle_sets] if fused_call else None

    def step():
        c = step_no[0] % copies
        step_no[0] += 1
        if fused_call:  # draw + block in one call: the block kernel streams W0 while the draw runs
            prep_fused[c].run(stream_handle)
            return
        prep_sample.run(stream_handle)
        if block_call:  # decode sizes: the block's projections share tokens, segments and the table -> one call
            prep_blocks[c].run(stream_handle)
        else:
            for i, h in enumerate(handle_sets[c]):
                ctx.apply_projection(h, xs[i], d_off, sigma, cols[i][0], cols[i][1], out=ys[i])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        if dist is None:
            return v
        t = torch.tensor([v], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    steps = args.steps
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    barrier()
    sampler = ClockSampler(torch, local_rank)
    launches0 = ctx.gpu_launches
    # Per-launch durations for the roofline come from CUDA events that the library records around every launch.
    # At prefill sizes they are recorded inside the timed steps (three event records per call are ~1 % of a step).
    # At decode sizes they would be a fifth of a step, and an event between two kernels also defeats the dependent
    # launch that lets the decode kernel's set-up overlap the population draw, so there the timed steps run without
    # them and the same K steps run once more, right after, with them.
    events_inside = not decode
    if events_inside:
        ctx.profile_begin(steps * len(handles))
    # The K timed steps are bracketed by one pair of events (the mean); events between groups of steps (every step
    # at prefill sizes, every `group` steps at decode sizes, where a step is tens of microseconds) give the spread.
    group = 1 if not decode else max(1, min(10, steps // 5))
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(steps // group + 2)]
    sampler.start()
    t_host0 = time.perf_counter()
    marks[0].record(stream)
    n_marks = 1
    for s in range(steps):
        step()
        if (s + 1) % group == 0 or s + 1 == steps:
            marks[n_marks].record(stream)
            n_marks += 1
    host_issue_ms = (time.perf_counter() - t_host0) * 1e3  # wall clock of issuing the K steps without synchronising
    barrier()
    launches = ctx.gpu_launches - launches0
    clocks = sampler.stop()
    if not events_inside:
        ctx.profile_begin(steps * len(handles))
        for _ in range(steps):
            step()
        barrier()
    prof = ctx.profile_end()
    ms = max_over_ranks(marks[0].elapsed_time(marks[n_marks - 1]))
    per_group = []
    for g in range(1, n_marks):
        n_in = group if g * group <= steps else steps - (g - 1) * group
        per_group.append(marks[g - 1].elapsed_time(marks[g]) / max(n_in, 1))
    status = ctx.get_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region of config {key}")
    ms_per_step = ms / steps
    value = world * T * steps / (ms * 1e-3)

    # ---- L2-warm regime (decode configurations): the same steps on ONE copy of the weights, which then stay in L2
    warm_ms = None
    if copies > 1:
        hs0 = handle_sets[0]

        def step_warm():
            ctx.sample_population(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, out=sigma, k_begin=k_begin)
            if block_call:
                ctx.apply_block(hs0, xs, d_off, sigma, cols, outs=ys)
            else:
                for i, h in enumerate(hs0):
                    ctx.apply_projection(h, xs[i], d_off, sigma, cols[i][0], cols[i][1], out=ys[i])
        for _ in range(3):
            step_warm()
        barrier()
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        w0.record(stream)
        for _ in range(steps):
            step_warm()
        w1.record(stream)
        barrier()
        warm_ms = max_over_ranks(w0.elapsed_time(w1)) / steps

    # ---- multi-layer call (decode configurations): L layers' blocks in ONE essa_apply_layers call, each layer with its
    # own device copy of the adapters (so every layer streams its W0 from HBM); per-layer time beside the single block's
    layers_rec = None
    if block_call and decode and world == 1 and not args.no_layers:
        L = {"3": 28, "5a": 80, "6a": 80}.get(key, 8)  # decoder layers of the backbone the shapes come from
        adapters_again = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
        while len(handle_sets) < L:
            handle_sets.append([ctx.load_adapter(a) for a in adapters_again])
        del adapters_again
        ys_alt = [torch.empty_like(y) for y in ys]
        layers = [[(handle_sets[l][i], xs[i], cols[i], (ys if l % 2 == 0 else ys_alt)[i]) for i in range(len(handles))]
                  for l in range(L)]
        prep_layers = ctx.prepare_layers(layers, d_off, sigma)
        reps = 5
        for _ in range(2):
            prep_layers.run(stream_handle)
        barrier()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0.record(stream)
        for _ in range(reps):
            prep_layers.run(stream_handle)
        l1.record(stream)
        barrier()
        ms_layers = l0.elapsed_time(l1) / reps
        layers_rec = {"n_layers": L, "ms_per_call": ms_layers, "ms_per_layer": ms_layers / L,
                      "block_frac_per_layer": None, "note": "one essa_apply_layers call; the population draw is not part of it"}

    # ---- end to end through the host-buffer entry points (H2D of x/offsets/sigma and D2H of y inside the call)
    xh = [x.pin_memory() for x in xs_host]
    del xs_host
    yh = [torch.empty((T, h.d_out), dtype=torch.bfloat16).pin_memory() for h in handles]
    off_h = torch.from_numpy(offsets).pin_memory()
    sig_h = torch.empty((cfg.P, cfg.d), dtype=torch.float32).pin_memory()

    def step_e2e():
        ctx.sample_population(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, out=sigma, k_begin=k_begin)
        sig_h.copy_(sigma, non_blocking=True)
        stream.synchronize()
        if args.single_calls:
            for i, h in enumerate(handles):
                sA, sB = cfg.sigma_cols(i)
                ctx.apply_projection_host(h, xh[i], off_h, sig_h, sA, sB, yh[i])
        else:  # the block's projections in one host call: offsets and the table travel once
            ctx.apply_block_host(handles, xh, off_h, sig_h, cols, yh)

    e2e_steps = max(1, min(steps, args.e2e_steps))
    for _ in range(2):
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_e2e()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks((time.perf_counter() - t0) * 1e3)
    # the same with q, k and v reading ONE activation buffer (as in an attention block): it is copied in once
    e2e_shared = None
    if len(handles) == 4 and not args.single_calls and handles[0].d_in == handles[1].d_in == handles[2].d_in:
        xh_shared = [xh[0], xh[0], xh[0], xh[3]]

        def step_e2e_shared():
            ctx.sample_population(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, out=sigma, k_begin=k_begin)
            sig_h.copy_(sigma, non_blocking=True)
            stream.synchronize()
            ctx.apply_block_host(handles, xh_shared, off_h, sig_h, cols, yh)
        for _ in range(2):
            step_e2e_shared()
        barrier()
        t0 = time.perf_counter()
        for _ in range(e2e_steps):
            step_e2e_shared()
        torch.cuda.synchronize()
        es_ms = max_over_ranks((time.perf_counter() - t0) * 1e3)
        e2e_shared = {"value": world * T * e2e_steps / (es_ms * 1e-3), "unit": UNIT, "ms_per_step": es_ms / e2e_steps,
                      "h2d_bytes_per_step": int(xh[0].numel() * 2 + xh[3].numel() * 2 + off_h.numel() * 4 + sig_h.numel() * 4)}
    h2d = sum(x.numel() * 2 for x in xh) + (len(handles) if args.single_calls else 1) * (off_h.numel() * 4 + sig_h.numel() * 4)
    d2h = sum(y.numel() * 2 for y in yh) + sig_h.numel() * 4
    e2e = {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}

    # ---- roofline of the dominant kernel (base contraction + up-projection), timed live by the library's events.
    # Tensor peak: the sustained figure only if this workload's own clock samples show the power cap, else burst.
    capped = "sw_power_cap" in clocks.get("reasons", [])
    tf_key = "bf16_tflops_sustained" if capped else "bf16_tflops"
    model = block_roofline(cfg, T, peaks[tf_key], peaks["hbm_gbs"])
    nominal = block_roofline(cfg, T, NOMINAL_PEAKS["bf16_tflops"], NOMINAL_PEAKS["hbm_gbs"])
    calls = max(prof["calls"], 1)
    main_s = prof["base_up_ms"] * 1e-3 / calls  # average launch duration
    # timed launches of the dominant kernel per step: 1 when a block call covers all projections with one launch
    per_call = max(1, round(prof["calls"] / steps))
    if model["bound"] == "tensor":
        per_launch = model["flops_main"] / per_call
        achieved, peak, peak_nom, unit = per_launch / main_s / 1e12, peaks[tf_key], NOMINAL_PEAKS["bf16_tflops"], "TFLOP/s"
        peak_kind = "sustained bf16 (sw_power_cap sampled during the timed steps)" if capped else "burst bf16 (no power cap sampled)"
    else:
        per_launch = model["bytes_main"] / per_call
        achieved, peak, peak_nom, unit = per_launch / main_s / 1e9, peaks["hbm_gbs"], NOMINAL_PEAKS["hbm_gbs"], "GB/s"
        peak_kind = "copy bandwidth"
    traffic = None
    if not ((decode and not block_call) or args.candidates > 0 or args.pair_tiles == 0 or args.fuse_down > 0):
        traffic = ncu_traffic(key)
    if decode:
        kernel = "essa_decode_kernel (one launch for the block's projections)" if block_call else "essa_decode_kernel (whole call)"
    else:
        kernel = ("essa_tcw_kernel (base contraction + up-projection of the block's projections in one launch)" if per_call == 1 and block_call
                  else "essa_tcw_kernel / essa_tc2_kernel / essa_tc_kernel (base contraction + up-projection)")
    roofline = {"bound": model["bound"], "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
                "traffic": traffic, "kernel": kernel, "peak_kind": peak_kind, "peak_source": f"{peak_src} ({peak_kind})",
                "peak_nominal": peak_nom, "frac_of_nominal": achieved / peak_nom,
                "algorithmic_per_launch": per_launch, "avg_launch_us": main_s * 1e6, "launches_timed": prof["calls"],
                "rank_down_avg_us": prof["rank_down_ms"] * 1e3 / calls,
                "block_roofline_us": model["time_s"] * 1e6, "block_frac": model["time_s"] * 1e3 / ms_per_step,
                "block_roofline_us_nominal": nominal["time_s"] * 1e6,
                "block_frac_of_nominal": nominal["time_s"] * 1e3 / ms_per_step}

    rec = {"workload": cfg.name, "tokens_per_gpu_step": T, "candidates_per_gpu": cfg.P, "rank": cfg.rank,
           "dtype": "bf16" if cfg.w0_dtype == "bf16" else f"bf16 ({cfg.w0_dtype} weights)",
           "projections": [f"{nm}:{n}->{m}" for nm, n, m in cfg.projections],
           "value": value, "steps": steps, "warmup": warmup,
           "ms_per_step": ms_per_step, "ms_per_step_median": float(np.median(per_group)), "ms_per_step_min": float(np.min(per_group)),
           "timing_group": group, "ms_per_step_l2_warm": warm_ms, "host_issue_ms_per_step": host_issue_ms / steps,
           "l2": "inputs larger than L2 (x, W0 and y of the projections exceed 126 MB per step)"
                 if copies == 1 else f"weights rotate through {copies} device copies ({copies * w_bytes / 1e6:.0f} MB > 2 x L2): "
                                     "every step streams W0 from HBM (ms_per_step_l2_warm: one copy, W0 served from L2)",
           "calls_per_step": "1 x essa_sample_apply_block (population draw + the block's projections)" if fused_call
                             else "essa_sample_population + 1 x essa_apply_block" if block_call
                             else f"essa_sample_population + {len(handles)} x essa_apply_projection",
           "kernel_timing": "CUDA events around every launch, inside the timed steps" if events_inside
                            else "CUDA events around every launch in a second pass of the same steps (not inside the timed steps)",
           "roofline": roofline, "e2e": e2e, "gpu_launches": launches, "clocks": clocks}
    if layers_rec is not None:
        layers_rec["block_frac_per_layer"] = model["time_s"] * 1e3 / layers_rec["ms_per_layer"]
        rec["layers"] = layers_rec
    if e2e_shared is not None:
        rec["e2e_shared_x"] = e2e_shared
    for hs in handle_sets:
        for h in hs:
            h.free()
    ctx.close()
    del xs, ys, xh, yh
    torch.cuda.empty_cache()
    return rec


def run_ours(args):
    import torch
    from paper_2507_04453_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    if not torch.cuda.is_available():
        raise SystemExit(f"bench.py: rank {rank} has no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_src = load_peaks()
    env = {"torch": torch, "binding": binding, "dist": dist, "world": world, "rank": rank, "local_rank": local_rank,
           "peaks": peaks, "peak_src": peak_src}

    keys = [args.config] if args.config else list(ALL_CONFIGS)
    head_key = args.config if args.config else HEADLINE
    per_config = {}
    for key in keys:
        cfg = wl.CONFIGS[key]
        if args.candidates > 0:
            import dataclasses
            cfg = dataclasses.replace(cfg, P=args.candidates, name=f"{cfg.name}-P{args.candidates}")
        per_config[key] = measure_config(key, cfg, args, env)
    head = per_config[head_key]

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            cpu = time_oracle_sample(wl.CONFIGS[head_key], budget_s=args.cpu_budget)
        config = {k: head[k] for k in ("workload", "tokens_per_gpu_step", "candidates_per_gpu", "rank", "projections", "l2",
                                       "calls_per_step", "kernel_timing")}
        config["parallelism"] = f"dp{world} (candidate-sharded, no data-path collective)"
        config["headline"] = ("largest single-GPU bf16 workload of the five" if not args.config else "--config given")
        config["peaks"] = {"source": peak_src, "bf16_tflops_burst": peaks["bf16_tflops"],
                           "bf16_tflops_sustained": peaks["bf16_tflops_sustained"], "hbm_gbs": peaks["hbm_gbs"],
                           "nominal_bf16_tflops": NOMINAL_PEAKS["bf16_tflops"], "nominal_hbm_gbs": NOMINAL_PEAKS["hbm_gbs"]}
        config["per_config"] = per_config
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
                "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "ms_per_step_median": head["ms_per_step_median"],
                "ms_per_step_min": head["ms_per_step_min"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": head["dtype"], "data": "synthetic", "config": config, "roofline": head["roofline"],
                "cpu_baseline": cpu, "e2e": head["e2e"], "gpu_launches": head["gpu_launches"], "clocks": head["clocks"]}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def spawn_ranks(args):
    """--gpus N without a launcher: re-execute this script under torch.distributed.run with N local ranks."""
    port = 29500 + (os.getpid() % 2000)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    raise SystemExit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=None, choices=list(wl.CONFIGS),
                    help="one workload only (default: 2, 3, 4, 5a, 5b in turn, config 4 as the headline)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--pair-tiles", type=int, default=-1, help="override ESSA_OPT_PAIR_TILES (0 / 1)")
    ap.add_argument("--fuse-down", type=int, default=-1, help="override ESSA_OPT_FUSE_DOWN (0 / 1)")
    ap.add_argument("--single-calls", action="store_true",
                    help="decode configurations: one essa_apply_projection per projection instead of one essa_apply_block")
    ap.add_argument("--set-option", action="append", default=[], metavar="ID=VALUE",
                    help="essa_set_option(ID, VALUE) on every context (scheduling experiments), e.g. 6=0")
    ap.add_argument("--no-layers", action="store_true", help="skip the multi-layer (essa_apply_layers) measurement of decode configurations")
    ap.add_argument("--separate-calls", action="store_true",
                    help="decode configurations: essa_sample_population then essa_apply_block instead of the fused call")
    ap.add_argument("--candidates", type=int, default=0, help="override the population size (smaller case for profiler captures)")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("bench.py: --gpus must be at least 1")
    if args.impl == "reference":
        run_reference(args, wl.CONFIGS[args.config or HEADLINE])
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args)
    run_ours(args)


if __name__ == "__main__":
    main()
