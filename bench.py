#!/usr/bin/env python
"""Benchmark of the ESSA population-projection hot path on B200.

One step = one pass of the whole hot path over one synthetic batch: draw the population's singular values
(essa_sample_population) and run the q, k, v, o adapted projections for every candidate's tokens
(4 x essa_apply_projection).  Metric: candidate-tokens/s (a candidate-token = one token of one candidate
through all projections of the block).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2] [--impl ours|reference]

N > 1 is launched with torch.distributed.run (one rank per GPU).  Candidates are independent, so ranks take
disjoint candidate ranges of an N-times larger population with no data-path collective (weak scaling).
Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
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
# DRAM bytes per launch of the dominant kernel from an ncu capture (profiles/), keyed by config; None = not captured.
NCU_TRAFFIC_BYTES = {"2": 184.4e6, "3": 67.9e6, "5a": 171.4e6}  # configs 3, 5a: the block launch


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
    bytes_call = m * n * w_bytes + (2 * m if w_bytes == 1 else 0) + 2.0 * T * n + 2.0 * T * m + 2.0 * n * r + 2.0 * m * r \
        + 4.0 * r * r + 8.0 * P * r + 4.0 * (P + 1)
    flops_main = 2.0 * T * m * (n + r)                       # base contraction + up-projection
    bytes_main = m * n * w_bytes + 2.0 * T * n + 2.0 * T * m + 2.0 * m * r + 2.0 * T * r  # W0, x, y, U_B, u
    return flops_call, bytes_call, flops_main, bytes_main


def block_roofline(cfg, T, peaks, sustained=True):
    tf = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"] * 1e12
    bw = peaks["hbm_gbs"] * 1e9
    w = 1 if cfg.w0_dtype == "int8" else 2
    t_total, fl, by, fl_main, by_main = 0.0, 0.0, 0.0, 0.0, 0.0
    bound_votes = {"tensor": 0.0, "hbm": 0.0}
    for _, n, m in cfg.projections:
        f, b, fm, bm = projection_work(n, m, cfg.rank, T, cfg.P, w)
        t = max(f / tf, b / bw)
        bound_votes["tensor" if f / tf >= b / bw else "hbm"] += t
        t_total += t
        fl += f; by += b; fl_main += fm; by_main += bm
    bound = max(bound_votes, key=bound_votes.get)
    return {"time_s": t_total, "flops": fl, "bytes": by, "flops_main": fl_main, "bytes_main": by_main, "bound": bound}


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

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
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
            time.sleep(0.004)

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


def oracle_setup(cfg):
    from oracle import essa_oracle as orc
    adapters = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
    offsets = wl.make_segments(cfg)
    T = int(offsets[-1])
    cma = wl.make_cma_state(cfg, adapters)
    weights = [a.W0.astype(np.float64) if a.w0_dtype == "bf16" else orc.dequantize_int8(a.W0_q, a.W0_scale) for a in adapters]
    xs = [wl.make_tokens(cfg, i, T).astype(np.float64) for i in range(len(adapters))]
    return adapters, weights, offsets, T, cma, xs


def time_oracle_sample(cfg, budget_s=15.0, prepared=None):
    """cpu_baseline: the oracle timed on a bounded sample (whole candidates, in order) of the workload."""
    from oracle import essa_oracle as orc
    adapters, weights, offsets, T, cma, xs = prepared or oracle_setup(cfg)
    t0 = time.perf_counter()
    sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    t_sample = time.perf_counter() - t0
    done_tokens, done_c, elapsed = 0, 0, t_sample
    for k in range(cfg.P):
        t0 = time.perf_counter()
        oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, [k])
        elapsed += time.perf_counter() - t0
        done_tokens += int(offsets[k + 1] - offsets[k])
        done_c += 1
        if elapsed >= budget_s:
            break
    return {"value": done_tokens / elapsed, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"first {done_c} of {cfg.P} candidates ({done_tokens} of {T} tokens), all {len(adapters)} projections, "
                      f"all channels, plus the full population draw; {elapsed:.1f} s"}


def run_reference(args, cfg):
    """--impl reference: the fp64 CPU oracle on the host cores; each step is a bounded sample of the workload."""
    from oracle import essa_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    prepared = oracle_setup(cfg)
    adapters, weights, offsets, T, cma, xs = prepared
    sigma = orc.sample_population(cma.mean, cma.step, cma.Bfactor, cma.Dvec, cma.seed, cfg.P)
    t0 = time.perf_counter()
    oracle_candidates_pass(cfg, adapters, weights, offsets, sigma, xs, [0])
    t1 = max(time.perf_counter() - t0, 1e-4)
    total_steps = args.steps + args.warmup
    c = int(max(1, min(cfg.P, 100.0 / (total_steps * t1))))  # whole run within a couple of minutes
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
    sample = f"each step: full population draw + first {c} of {cfg.P} candidates ({tokens} of {T} tokens), all projections, all channels"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "tokens_per_step": tokens, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg):
    import torch
    from paper_2507_04453_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_src = load_peaks()

    ctx = binding.Context(local_rank)
    if args.pair_tiles >= 0:
        ctx.set_option(binding.ESSA_OPT_PAIR_TILES, args.pair_tiles)
    if args.fuse_down >= 0:
        ctx.set_option(binding.ESSA_OPT_FUSE_DOWN, args.fuse_down)
    adapters = [wl.make_adapter(cfg, i) for i in range(len(cfg.projections))]
    offsets = wl.make_segments(cfg)
    T = int(offsets[-1])
    cma = wl.make_cma_state(cfg, adapters)
    # Weights that fit L2 (decode configurations) would be served from it on every step: rotate through enough
    # device copies of the block's adapters that each step streams its W0 from HBM, as a forward pass over many
    # layers does.
    w_bytes = sum(a.d_in * a.d_out * (1 if cfg.w0_dtype == 'int8' else 2) for a in adapters)  # as stored
    L2_BYTES = 126e6
    copies = 1 if w_bytes > 2 * L2_BYTES else int(np.ceil(2 * L2_BYTES / w_bytes)) + 1
    handle_sets = [[ctx.load_adapter(a) for a in adapters] for _ in range(copies)]
    handles = handle_sets[0]
    dev = lambda a, dt=None: (torch.from_numpy(np.ascontiguousarray(a)).to(dt) if dt else torch.from_numpy(np.ascontiguousarray(a))).cuda()
    xs_host = [torch.from_numpy(wl.make_tokens(cfg, i, T)).to(torch.bfloat16) for i in range(len(adapters))]
    xs = [x.cuda() for x in xs_host]
    ys = [torch.empty((T, a.d_out), dtype=torch.bfloat16, device="cuda") for a in adapters]
    d_off = dev(offsets)
    d_mean = dev(cma.mean)
    d_B = None if cma.Bfactor is None else dev(cma.Bfactor)
    d_D = None if cma.Dvec is None else dev(cma.Dvec)
    sigma = torch.empty((cfg.P, cfg.d), dtype=torch.float32, device="cuda")
    k_begin = rank * cfg.P  # weak scaling: rank g evaluates candidates [g*P, (g+1)*P) of an N*P population
    ctx.reserve(T, max(a.d_in for a in adapters), max(a.d_out for a in adapters))
    if cfg.w0_dtype == "int8":
        ctx.reserve_dequant(max(a.d_in for a in adapters), max(a.d_out for a in adapters))
    stream = torch.cuda.current_stream()

    step_no = [0]
    cols = [cfg.sigma_cols(i) for i in range(len(adapters))]
    block_call = T <= 256 and len(adapters) > 1 and not args.single_calls

    def step():
        hs = handle_sets[step_no[0] % copies]
        step_no[0] += 1
        ctx.sample_population(d_mean, cma.step, d_B, d_D, cma.seed, cfg.P, out=sigma, k_begin=k_begin)
        if block_call:  # decode sizes: the block's projections share tokens, segments and the table -> one call
            ctx.apply_block(hs, xs, d_off, sigma, cols, outs=ys)
        else:
            for i, h in enumerate(hs):
                ctx.apply_projection(h, xs[i], d_off, sigma, cols[i][0], cols[i][1], out=ys[i])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    sampler = ClockSampler(torch, local_rank)
    launches0 = ctx.gpu_launches
    # Per-launch durations for the roofline come from CUDA events that the library records around every launch.
    # At prefill sizes they are recorded inside the timed steps (three event records per call are ~1 % of a step).
    # At decode sizes they would be a fifth of a step, and an event between two kernels also defeats the dependent
    # launch that lets the decode kernel's set-up overlap the population draw, so there the timed steps run without
    # them and the same K steps run once more, right after, with them.
    events_inside = T > 256
    if events_inside:
        ctx.profile_begin(args.steps * len(handles))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    launches = ctx.gpu_launches - launches0
    if not events_inside:
        ctx.profile_begin(args.steps * len(handles))
        for _ in range(args.steps):
            step()
        barrier()
    clocks = sampler.stop()
    prof = ctx.profile_end()
    ms = e0.elapsed_time(e1)
    if dist is not None:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    status = ctx.get_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the timed region")
    ms_per_step = ms / args.steps
    value = world * T * args.steps / (ms * 1e-3)

    # ---- end to end through the host-buffer entry points (H2D of x/offsets/sigma and D2H of y inside the call)
    xh = [x.pin_memory() for x in xs_host]
    yh = [torch.empty((T, a.d_out), dtype=torch.bfloat16).pin_memory() for a in adapters]
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
            ctx.apply_block_host(handles, xh, off_h, sig_h, [cfg.sigma_cols(i) for i in range(len(handles))], yh)

    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    for _ in range(2):
        step_e2e()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        step_e2e()
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t0) * 1e3
    if dist is not None:
        t = torch.tensor([e2e_ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    h2d = sum(x.numel() * 2 for x in xh) + (len(handles) if args.single_calls else 1) * (off_h.numel() * 4 + sig_h.numel() * 4)
    d2h = sum(y.numel() * 2 for y in yh) + sig_h.numel() * 4
    e2e = {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps}

    # ---- roofline of the dominant kernel (base contraction + up-projection), timed live by the library's events
    decode = T <= 256  # one-launch decode schedule (essa_plan.decode)
    # a kernel inside a long, power-capped step is held against the sustained tensor peak, a short one against the burst peak
    model = block_roofline(cfg, T, peaks, sustained=not decode)
    calls = max(prof["calls"], 1)
    main_s = prof["base_up_ms"] * 1e-3 / calls  # average launch duration
    per_call = 1 if block_call else len(handles)  # a block call is one launch for all projections
    if model["bound"] == "tensor":
        per_launch = model["flops_main"] / per_call
        achieved, peak, unit = per_launch / main_s / 1e12, peaks["bf16_tflops" if decode else "bf16_tflops_sustained"], "TFLOP/s"
    else:
        per_launch = model["bytes_main"] / per_call
        achieved, peak, unit = per_launch / main_s / 1e9, peaks["hbm_gbs"], "GB/s"
    roofline = {"bound": model["bound"], "achieved": achieved, "peak": peak, "unit": unit, "frac": achieved / peak,
                "traffic": None if (decode and not block_call) or args.candidates > 0 or args.pair_tiles == 0 or args.fuse_down > 0
                           else NCU_TRAFFIC_BYTES.get(args.config), "kernel": ("essa_decode_kernel (one launch for the block's projections)" if block_call else "essa_decode_kernel (whole call)") if decode else "essa_tc2_kernel / essa_tc_kernel (base + up; --fuse-down 1|2 puts the down-projection inside the pair-tile launch)",
                "peak_source": f"{peak_src} ({('burst bf16' if decode else 'sustained bf16') if unit == 'TFLOP/s' else 'copy'})",
                "avg_launch_us": main_s * 1e6, "launches_timed": prof["calls"],
                "rank_down_avg_us": prof["rank_down_ms"] * 1e3 / calls,
                "block_roofline_us": model["time_s"] * 1e6, "block_frac": model["time_s"] * 1e3 / ms_per_step}

    if rank == 0:
        cpu = time_oracle_sample(cfg, budget_s=args.cpu_budget) if world == 1 and not args.no_cpu_baseline else None
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16" if cfg.w0_dtype == "bf16" else "bf16 (int8 weights)", "data": "synthetic",
                "config": {"workload": cfg.name, "tokens_per_gpu_step": T, "candidates_per_gpu": cfg.P, "rank": cfg.rank,
                           "projections": [f"{nm}:{n}->{m}" for nm, n, m in cfg.projections],
                           "l2": "inputs larger than L2 (x, W0 and y of the projections exceed 126 MB per step)"
                                 if copies == 1 else f"weights rotate through {copies} device copies ({copies * w_bytes / 1e6:.0f} MB > 2 x L2): "
                                                     "every step streams W0 from HBM",
                           "calls_per_step": "essa_sample_population + 1 x essa_apply_block" if block_call
                                             else f"essa_sample_population + {len(handles)} x essa_apply_projection",
                           "kernel_timing": "CUDA events around every launch, inside the timed steps" if events_inside
                                            else "CUDA events around every launch in a second pass of the same steps (not inside the timed steps)",
                           "parallelism": f"dp{world} (candidate-sharded, no data-path collective)"},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks}
        print(json.dumps(line), flush=True)
    for hs in handle_sets:
        for h in hs:
            h.free()
    ctx.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="2", choices=list(wl.CONFIGS))
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--pair-tiles", type=int, default=-1, help="override ESSA_OPT_PAIR_TILES (0 / 1)")
    ap.add_argument("--fuse-down", type=int, default=-1, help="override ESSA_OPT_FUSE_DOWN (0 / 1)")
    ap.add_argument("--single-calls", action="store_true",
                    help="decode configurations: one essa_apply_projection per projection instead of one essa_apply_block")
    ap.add_argument("--candidates", type=int, default=0, help="override the population size (smaller case for profiler captures)")
    args = ap.parse_args()
    cfg = wl.CONFIGS[args.config]
    if args.candidates > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, P=args.candidates, name=f"{cfg.name}-P{args.candidates}")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
