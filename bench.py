#!/usr/bin/env python
"""Benchmark of the Thanos per-layer hot path on B200.

A "step" is one pass of the whole hot path over one transformer block's layer set: for every
distinct layer input the calibration Hessian (thanos_hessian_accumulate over all tokens) and
its factorisation (thanos_prepare_inverse), then thanos_prune_layer for every layer.

Prints ONE JSON line (rank 0).  `--impl reference` times the float64 CPU oracle on a bounded
sample of the same workload instead.
"""

from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import workloads as WL

METRIC = "pruned_weights_per_sec"
UNIT = "weights/s"
TOKEN_CHUNK = 262144  # tokens per thanos_hessian_accumulate call (the activations are resident)


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of ONE launch of the Hessian kernel,
# taken once with ncu on launches short enough to capture: width b -> (bytes, tokens of the captured
# launch).  A launch streams X once per wave of tile pairs, so its traffic grows in proportion to
# its tokens; the figure reported with the bench line is scaled that way.  Set an entry to None
# when the kernel has changed since its counters were taken (the line then reports null).
HESSIAN_DRAM_CAPTURE = {4096: (2.016e9, 65536), 11008: (3.819e9, 16384)}


def hessian_traffic_per_launch(launch_shapes):
    """Average scaled DRAM bytes per launch over (b, tokens) launches; None if a width was never
    captured."""
    tot = 0.0
    for b, tok in launch_shapes:
        if HESSIAN_DRAM_CAPTURE.get(b) is None:
            return None
        byt, cap_tok = HESSIAN_DRAM_CAPTURE[b]
        tot += byt * tok / cap_tok
    return tot / max(1, len(launch_shapes))


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None

    def _nvml_loop(self):
        import pynvml as N
        names = [("hw_slowdown", "nvmlClocksThrottleReasonHwSlowdown"),
                 ("hw_thermal_slowdown", "nvmlClocksThrottleReasonHwThermalSlowdown"),
                 ("sw_thermal_slowdown", "nvmlClocksThrottleReasonSwThermalSlowdown"),
                 ("sw_power_cap", "nvmlClocksThrottleReasonSwPowerCap")]
        bits = [(nm, getattr(N, const)) for nm, const in names if hasattr(N, const)]
        while not self._stop.is_set():
            try:
                self._sm.append(float(N.nvmlDeviceGetClockInfo(self._h, N.NVML_CLOCK_SM)))
                r = int(N.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for nm, bit in bits:
                    if r & bit:
                        self._reasons.add(nm)
            except Exception:
                pass
            self._stop.wait(0.02)

    def start(self):
        """Read-only NVML queries every 20 ms from a thread; nvidia-smi (200 ms) if NVML is not
        importable."""
        import threading
        self._sm, self._reasons, self._thread = [], set(), None
        try:
            import pynvml as N
            N.nvmlInit()
            self._h = N.nvmlDeviceGetHandleByIndex(self.gpu)
            self._smax = float(N.nvmlDeviceGetMaxClockInfo(self._h, N.NVML_CLOCK_SM))
            self._stop = threading.Event()
            self._thread = threading.Thread(target=self._nvml_loop, daemon=True)
            self._thread.start()
            return
        except Exception:
            self._thread = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "200"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if getattr(self, "_thread", None) is not None:
            self._stop.set()
            self._thread.join(timeout=2)
            sm = self._sm
            return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": self._smax,
                    "samples": len(sm), "reasons": sorted(self._reasons)}
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [t.strip() for t in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(smax)) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time: one all_reduce(MAX) over the default process group (any backend);
    the value itself when no group is up.  Replicas exchange nothing else."""
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(weights_per_replica: int, steps: int, world: int, ms_total: float) -> float:
    """Weights swept per second by all replicas together, given the slowest rank's time."""
    return world * weights_per_replica * steps / (ms_total * 1e-3)


def layer_set_weights(cfg):
    return sum(L.c * L.b for L in cfg.layers)


def mode_args(cfg, T):
    if cfg.mode == "unstructured":
        return dict(mode=T.UNSTRUCTURED, p=cfg.p)
    return dict(mode=T.NM, n=cfg.n, m=cfg.m)


def select_mode(cfg, index: int):
    """index 0: the configuration's own sparsity mode; k > 0: its k-th additional mode (the
    LLaMA-2-70B-shaped set is also pruned to 60 % unstructured)."""
    if index == 0:
        return cfg
    kind, val = cfg.extra_modes[index - 1]
    if kind == "unstructured":
        return dataclasses.replace(cfg, mode="unstructured", p=float(val))
    n, m = val
    return dataclasses.replace(cfg, mode="nm", n=int(n), m=int(m))


def kernel_trace(fn):
    """Runs fn() under a CUPTI activity trace (torch.profiler, device activities only) and returns
    {kernel name: [launches, device ms]} plus the copies / memsets; None when no trace can be had.
    Used for ONE extra, untimed step whose calls are issued on a single stream, so that the step's
    time can be split by kernel; nothing measured under the trace is reported as a bench value."""
    try:
        from torch.profiler import ProfilerActivity, profile
        with profile(activities=[ProfilerActivity.CUDA]) as prof:
            fn()
            torch.cuda.synchronize()
        agg = {}
        for e in prof.events():
            if e.device_type == torch.autograd.DeviceType.CUDA:
                d = agg.setdefault(e.name, [0, 0.0])
                d[0] += 1
                d[1] += e.device_time * 1e-3
        return agg or None
    except Exception:
        return None


def short_kernel_name(name: str) -> str:
    n = name.replace("thanos::(anonymous namespace)::", "").replace("void ", "")
    return n.split("(")[0]


def measure_fp32_peak(T, dev):
    """Plain fp32 FMA throughput of this device from the library's FMA-chain kernel (best of 5
    launches of about a millisecond, CUDA events): the roofline of the per-row solves."""
    ctas = 148 * 8
    out = torch.empty(ctas * 256, dtype=torch.float32, device=dev)
    T.fp32_fma_probe(out, ctas, 64)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        flop = T.fp32_fma_probe(out, ctas, 16384)
        e1.record()
        torch.cuda.synchronize()
        best = max(best, flop / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    return best


def solve_flop(masks, cfg):
    """Arithmetic of the per-row systems of one step from the masks it produced: per row and
    block, with s removed of B and n = min(s, B - s) unknowns (direct or complement form),
    n^3 / 3 + 2 n^2 + 2 s (B - s) floating-point operations (factorisation, two triangular
    solves, the product that spreads the solution over the block)."""
    tot = 0.0
    B = cfg.B
    for M in masks:
        c, b = M.shape
        nb = b // B
        if nb == 0:
            continue
        s_ = M[:, : nb * B].reshape(c, nb, B).sum(dim=2, dtype=torch.int32).double()
        n_ = torch.minimum(s_, B - s_)
        tot += float((n_ ** 3 / 3.0 + 2.0 * n_ ** 2 + 2.0 * s_ * (B - s_)).sum())
    return tot


def roofline_by_kernel(trace_factor, trace_sweep, cfg, peaks, fp32_peak, masks, n_inputs_by_b):
    """Fractions of the governing roofline for the kernels next to the Hessian, from the per-kernel
    device times of one serialised step (trace_factor: Hessians + factorisations, trace_sweep: the
    sweeps) and the algorithmic work of that step."""
    def t_of(trace, key):
        if not trace:
            return None, 0
        ms = sum(v[1] for k, v in trace.items() if key in k)
        n = sum(v[0] for k, v in trace.items() if key in k)
        return (ms if n else None), n

    out = {}
    unstructured = cfg.mode == "unstructured"
    B = cfg.B
    resid_elems = 0.0   # sum over layers and blocks of c (b - j1): one look at the residual per block
    upd_elems = 0.0     # sum over layers and blocks of c (b - j2): what a block's update changes
    grouped_layers = 0
    for L in cfg.layers:
        # n:m sweeps of wide layers update in groups of 512 columns: a block's update reaches the
        # rest of its group at once, the columns to the right of the group once per group
        group = 1
        if not unstructured and L.b >= 2048 and B < 512:
            group = max(1, min(8, 512 // B))
            grouped_layers += 1
        for j1 in range(0, L.b, B):
            j2 = min(L.b, j1 + B)
            resid_elems += float(L.c) * (L.b - j1)
            ge = min(L.b, (j1 // (group * B) + 1) * group * B)   # end of the block's group
            upd_elems += float(L.c) * (ge - j2)
            if j2 == ge:
                upd_elems += float(L.c) * (L.b - ge)
    hbm = peaks["hbm_gbs"]
    if unstructured:
        ms, n = t_of(trace_sweep, "::select_")   # select_pass_kernel and select_rest_kernel
        if ms:
            ach = 4.0 * resid_elems / (ms * 1e-3) / 1e9
            out["select_pass_kernel"] = {
                "bound": "hbm", "achieved": round(ach, 1), "peak": hbm, "unit": "GB/s",
                "frac": round(ach / hbm, 4), "ms_per_step": round(ms, 3), "launches": n,
                "work": "4 c (b - j1) bytes per block: one read of the residual"}
    ms, n = t_of(trace_sweep, "tc_gemm_")   # tc_gemm_kernel and tc_gemm_pair_kernel
    if ms:
        ach = 8.0 * upd_elems / (ms * 1e-3) / 1e9
        out["tc_gemm_kernel (sweep update)"] = {
            "bound": "hbm", "achieved": round(ach, 1), "peak": hbm, "unit": "GB/s",
            "frac": round(ach / hbm, 4), "ms_per_step": round(ms, 3), "launches": n,
            "work": "8 bytes per weight an update changes: c (b - j2) per block; in n:m sweeps of "
                    "wide layers c (group end - j2) per block and c (b - group end) per group "
                    "of 512 columns"}
        if grouped_layers:
            # with K = 512 per group the update is a tensor-bound product: also against that bound
            flop = sum(float(L.c) * float(L.b) * float(L.b) for L in cfg.layers)   # 2 c B (b - j2) / block
            tf = flop / (ms * 1e-3) / 1e12
            pk = peaks["bf16_tflops_sustained"]
            out["tc_gemm_kernel (sweep update)"].update({
                "tensor_useful_tflops": round(tf, 1), "tensor_frac_useful": round(tf / pk, 4),
                "tensor_frac_executed": round(6.0 * tf / pk, 4),
                "tensor_note": "c b^2 useful FLOP per layer; the kernel executes six bf16-plane "
                               "products per fp32 product"})
    ms, n = t_of(trace_factor, "tc_gemm_")
    if ms:
        flop = sum(k * (2.0 / 3.0) * float(b) ** 3 for b, k in n_inputs_by_b.items())
        ach = flop / (ms * 1e-3) / 1e12
        pk = peaks["bf16_tflops_sustained"]
        out["tc_gemm_kernel (factorisation)"] = {
            "bound": "tensor", "achieved": round(ach, 2), "peak": pk, "unit": "TFLOP/s",
            "frac": round(ach / pk, 4), "ms_per_step": round(ms, 3), "launches": n,
            "work": "2/3 b^3 useful FLOP per factorisation (Cholesky + triangular inverse); the "
                    "kernel executes six bf16-plane products per fp32 product"}
    ms, n = t_of(trace_sweep, "solve_rows")
    if ms and fp32_peak:
        ach = solve_flop(masks, cfg) / (ms * 1e-3) / 1e12
        out["solve_rows kernels"] = {
            "bound": "alu", "achieved": round(ach, 2), "peak": round(fp32_peak, 2),
            "unit": "TFLOP/s", "frac": round(ach / fp32_peak, 4), "ms_per_step": round(ms, 3),
            "launches": n, "peak_source": "measured: FMA-chain kernel of this library, this run",
            "work": "n^3/3 + 2 n^2 + 2 s (B - s) FLOP per row and block, n = min(s, B - s), "
                    "counted from the step's masks"}
    return out


# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch.distributed as dist

    import paper_2504_05346_b200 as T
    from paper_2504_05346_b200 import build as B_

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        B_.build()
    if world > 1:
        dist.barrier()
    T.load_library()

    cfg = select_mode(WL.CONFIGS[args.workload], args.mode_index)
    a = args.tokens or cfg.a
    dt = T.BF16 if cfg.dtype == "bf16" else T.F32
    margs = mode_args(cfg, T)

    # ---- resident inputs: one activation matrix per distinct layer input, all weights
    inputs = {}
    for L in cfg.layers:
        if L.input_id not in inputs:
            inputs[L.input_id] = WL.config_activations(cfg, L.input_id, L.b, device=dev, a=a)
    weights = [WL.config_weight(cfg, i, device=dev) for i in range(len(cfg.layers))]
    outs = [torch.empty_like(w) for w in weights]
    masks = [torch.empty(w.shape, dtype=torch.uint8, device=dev) for w in weights]
    # Layers of a block are pruned independently of each other, so every distinct input gets a
    # stream (Hessian + factorisation) and every layer a stream (sweep) with buffers of their own:
    # the serial chains of small kernels of one call then fill the gaps of the others.
    overlap = not args.no_overlap
    main = torch.cuda.current_stream()
    in_ids = list(inputs.keys())
    s_in = {iid: (torch.cuda.Stream() if overlap else main) for iid in in_ids}
    s_layer = [torch.cuda.Stream() if overlap else main for _ in cfg.layers]
    Hbuf, Ubuf, xnbuf, ws_in = {}, {}, {}, {}
    for iid in in_ids:
        b = inputs[iid].shape[1]
        Hbuf[iid] = torch.empty((b, b), dtype=torch.float32, device=dev)
        Ubuf[iid] = torch.empty((b, b), dtype=torch.float32, device=dev)
        xnbuf[iid] = torch.empty((b,), dtype=torch.float32, device=dev)
        nb = max(T.workspace_bytes(0, 0, b, 0, dt), T.workspace_bytes(1, 0, b, 0, T.F32))
        ws_in[iid] = torch.empty(nb, dtype=torch.uint8, device=dev)
    ws_layer = [torch.empty(T.workspace_bytes(2, L.c, L.b, cfg.B, dt), dtype=torch.uint8, device=dev)
                for L in cfg.layers]
    torch.cuda.synchronize()

    hess_events = []  # (start, end, flops, (b, tokens)) per thanos_hessian_accumulate call
    hess_status = {iid: torch.zeros(1, dtype=torch.int32, device=dev) for iid in in_ids}

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def one_step(record, serial=False, do_factor=True, do_sweep=True):
        """One pass over the layer set.  `serial` issues every call on the main stream (used by
        the untimed per-kernel trace); `do_factor` / `do_sweep` select the two halves of the step
        (Hessians + factorisations, sweeps) for that trace."""
        stats_all = [None] * len(cfg.layers)
        ready = {}
        if do_factor:
            # the Hessians fill the whole GPU by themselves: one after the other on the main stream
            for iid in in_ids:
                X = inputs[iid]
                b = X.shape[1]
                H = Hbuf[iid]
                H.zero_()
                for t0 in range(0, a, TOKEN_CHUNK):
                    xc = X[t0:t0 + TOKEN_CHUNK]
                    if record:
                        hs, he = ev(), ev()
                        hs.record(main)
                    T.hessian_accumulate(H, xc, workspace=ws_in[iid])
                    if record:
                        he.record(main)
                        hess_events.append((hs, he, float(xc.shape[0]) * b * (b + 1),
                                            (b, int(xc.shape[0]))))
                    # the call's status word sits in the workspace the factorisation reuses
                    torch.maximum(hess_status[iid], ws_in[iid][:4].view(torch.int32),
                                  out=hess_status[iid])
            e_h = ev()
            e_h.record(main)
            # factorisations: one stream per input
            for iid in in_ids:
                s = main if serial else s_in[iid]
                s.wait_event(e_h)
                with torch.cuda.stream(s):
                    T.prepare_inverse(Hbuf[iid], cfg.damp_rel, workspace=ws_in[iid], check=False,
                                      factor=Ubuf[iid], xnorm=xnbuf[iid])
                    e2 = ev()
                    e2.record(s)
                    ready[iid] = e2
        if not do_sweep:
            for e in ready.values():
                main.wait_event(e)
            return stats_all
        done = []
        for i, L in enumerate(cfg.layers):
            s = main if serial else s_layer[i]
            if L.input_id in ready:
                s.wait_event(ready[L.input_id])
            with torch.cuda.stream(s):
                _, _, st = T.prune_layer(weights[i], Ubuf[L.input_id], xnbuf[L.input_id], B=cfg.B,
                                         workspace=ws_layer[i], out=outs[i], mask=masks[i],
                                         read_stats=False, **margs)
                p1 = ev()
                p1.record(s)
            stats_all[i] = st
            done.append(p1)
        for e in done:
            main.wait_event(e)
        return stats_all

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        one_step(False)
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = T.launch_count()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_start.record()
    stats_last = None
    for _ in range(args.steps):
        stats_last = one_step(True)
    t_end.record()
    barrier()
    launches = T.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    ms_total = t_start.elapsed_time(t_end)
    ms_total = max_over_ranks(ms_total, dev)
    # device status of the last step
    select_misses = 0
    for st in stats_last:
        ps = T.PruneStats.from_bytes(bytes(st.cpu().numpy().tobytes()))
        if ps.status != 0:
            raise RuntimeError("device status %d in prune_layer" % ps.status)
        select_misses += ps.select_misses
    for iid, hs in hess_status.items():
        if int(hs.item()) != 0:
            raise RuntimeError("device status %d in hessian_accumulate" % int(hs.item()))

    nweights = layer_set_weights(cfg)
    ms_per_step = ms_total / args.steps
    value = whole_job_rate(nweights, args.steps, world, ms_total)

    # ---- roofline of the dominant kernel: the Hessian contraction
    peaks = _peaks()
    h_ms = sum(ev[0].elapsed_time(ev[1]) for ev in hess_events)
    h_flops = sum(ev[2] for ev in hess_events)
    traffic = hessian_traffic_per_launch([ev[3] for ev in hess_events])
    achieved = h_flops / (h_ms * 1e-3) / 1e12 if h_ms > 0 else 0.0
    peak = peaks["bf16_tflops_sustained"]
    roofline = {"kernel": "hessian_tc2_kernel (thanos_hessian_accumulate)", "bound": "tensor", "achieved": round(achieved, 2),
                "peak": peak, "unit": "TFLOP/s", "frac": round(achieved / peak, 4),
                "peak_source": peaks["source"] + " (sustained bf16)",
                "traffic": None if traffic is None else round(traffic),
                "traffic_unit": "DRAM bytes per launch, ncu capture of a shorter launch scaled by tokens",
                "launches": len(hess_events), "avg_launch_ms": round(h_ms / max(1, len(hess_events)), 4)}

    # ---- the rest of the step by kernel: ONE extra untimed step, every call on one stream, under
    #      a device-activity trace, in two halves so that the tensor-core products of the
    #      factorisations and of the sweeps are told apart
    by_kernel, kernel_ms, fp32_peak = None, None, None
    if rank == 0 and not args.no_kernel_split:
        fp32_peak = measure_fp32_peak(T, dev)
        tr_f = kernel_trace(lambda: one_step(False, serial=True, do_sweep=False))
        tr_s = kernel_trace(lambda: one_step(False, serial=True, do_factor=False))
        if tr_f and tr_s:
            n_by_b = {}
            for iid in in_ids:
                n_by_b[inputs[iid].shape[1]] = n_by_b.get(inputs[iid].shape[1], 0) + 1
            by_kernel = roofline_by_kernel(tr_f, tr_s, cfg, peaks, fp32_peak, masks, n_by_b)
            kernel_ms = {}
            for half, tr in (("hessians+factorisations", tr_f), ("sweeps", tr_s)):
                kernel_ms[half] = {short_kernel_name(k): [v[0], round(v[1], 3)]
                                   for k, v in sorted(tr.items(), key=lambda kv: -kv[1][1])
                                   if v[1] >= 0.05}
                kernel_ms[half]["total_ms"] = round(sum(v[1] for v in tr.values()), 3)

    # ---- end to end through the host-buffer entry point
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(T, cfg, a, dev, dt, margs, world, args)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample(cfg, args.cpu_budget_s)

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype if cfg.dtype != "f32" else "f32",
            "data": "synthetic",
            "config": {"workload": "%s layer set: %s; %d calibration tokens; %s; B=%d; damp %.2g"
                                   % (cfg.name, ", ".join("%dx%d" % (L.c, L.b) for L in cfg.layers),
                                      a, ("%d%% unstructured" % round(100 * cfg.p))
                                      if cfg.mode == "unstructured" else "%d:%d" % (cfg.n, cfg.m),
                                      cfg.B, cfg.damp_rel),
                       "weights_per_step": nweights, "l2": "inputs larger than L2",
                       "parallelism": "replicas only" if world > 1 else "single GPU",
                       "streams": "one per layer input and one per layer (calls overlap)"
                       if overlap else "one",
                       "token_chunk": TOKEN_CHUNK},
            "ms_per_layer": ms_per_step / len(cfg.layers),
            "select_misses_last_step": int(select_misses),
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "roofline": roofline, "roofline_by_kernel": by_kernel,
            "fp32_fma_peak_tflops_measured": None if fp32_peak is None else round(fp32_peak, 2),
            "kernel_ms_serialised_step": kernel_ms,
            "kernel_ms_note": "device time per kernel [launches, ms] of one extra untimed step "
                              "issued on a single stream, from a device-activity trace; the timed "
                              "steps overlap these calls on several streams",
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_e2e(T, cfg, a, dev, dt, margs, world, args):
    """Same metric through thanos_prune_layer_host: pinned host inputs, copies timed."""
    import torch.distributed as dist

    steps = max(1, min(args.steps, args.e2e_steps))
    host_in = {}
    for L in cfg.layers:
        if L.input_id not in host_in:
            x = WL.config_activations(cfg, L.input_id, L.b, device=dev, a=a)
            host_in[L.input_id] = x.cpu().pin_memory()
            del x
    host_w = [WL.config_weight(cfg, i, device=dev).cpu().pin_memory() for i in range(len(cfg.layers))]
    host_o = [torch.empty_like(w).pin_memory() for w in host_w]
    host_m = [torch.empty(w.shape, dtype=torch.uint8).pin_memory() for w in host_w]
    torch.cuda.empty_cache()
    arena_bytes = max(T.workspace_bytes(3, L.c, L.b, cfg.B, dt) for L in cfg.layers)
    h2d = sum(x.numel() * x.element_size() for x in host_in.values()) + \
        sum(w.numel() * w.element_size() for w in host_w)
    d2h = sum(w.numel() * w.element_size() + w.numel() + 64 for w in host_w)

    # Layers that share an input share its factor, so they stay together and in order; the
    # groups are dealt to host threads (largest first, to the lighter thread), each with its own
    # stream and arena, so that one group's copies overlap another group's kernels.
    groups = {}
    for i, L in enumerate(cfg.layers):
        groups.setdefault(L.input_id, []).append(i)
    n_workers = max(1, min(args.e2e_workers, len(groups)))
    load = [0] * n_workers
    plan = [[] for _ in range(n_workers)]
    for gid in sorted(groups, key=lambda g: -host_in[g].numel()):
        k = load.index(min(load))
        plan[k].append(gid)
        load[k] += host_in[gid].numel() + sum(host_w[i].numel() for i in groups[gid])
    arenas = [torch.empty(arena_bytes, dtype=torch.uint8, device=dev) for _ in range(n_workers)]
    streams = [torch.cuda.Stream(device=dev) for _ in range(n_workers)]
    errors = []

    def work(k):
        try:
            torch.cuda.set_device(dev)
            for gid in plan[k]:
                for pos, i in enumerate(groups[gid]):
                    reuse = pos > 0
                    T.prune_layer_host(host_w[i], None if reuse else host_in[gid], cfg.damp_rel,
                                       B=cfg.B, arena=arenas[k], reuse_factor=reuse,
                                       out=host_o[i], mask=host_m[i], stream=streams[k], **margs)
        except Exception as e:  # reported by the caller's thread
            errors.append(e)

    def step():
        import threading
        if n_workers == 1:
            work(0)
        else:
            ts = [threading.Thread(target=work, args=(k,)) for k in range(n_workers)]
            for t in ts:
                t.start()
            for t in ts:
                t.join()
        if errors:
            raise errors[0]

    step()  # warm-up
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    torch.cuda.synchronize()
    dt_s = time.perf_counter() - t0
    dt_s = max_over_ranks(dt_s, dev)
    return {"value": world * layer_set_weights(cfg) * steps / dt_s, "unit": UNIT,
            "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": steps,
            "ms_per_step": dt_s * 1e3 / steps, "host_threads": n_workers}


# ------------------------------------------------------------------------------------------
def oracle_sample(cfg, budget_s=20.0):
    """Times the float64 oracle, as it stands, on a bounded sample of the workload: the first
    layer of the set with a reduced token count and only the first column blocks of the sweep;
    the per-weight rate is extrapolated to the full layer (stated in `sample`)."""
    from oracle import thanos_oracle as O

    try:
        import threadpoolctl
        info = threadpoolctl.threadpool_info()
        cores = max([i.get("num_threads", 1) for i in info] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    L = cfg.layers[0]
    c, b, B = L.c, L.b, cfg.B
    a_s = min(cfg.a, 4096)
    W = WL.config_weight(cfg, 0).double().numpy()
    Xt = WL.config_activations(cfg, L.input_id, b, a=a_s).double().numpy()
    t0 = time.perf_counter()
    H = O.hessian(Xt.T)
    t_h = time.perf_counter() - t0
    t0 = time.perf_counter()
    Hd = O.damped(H, cfg.damp_rel)
    U = O.inverse_factor(Hd)
    xn = O.feature_norms(H)
    t_f = time.perf_counter() - t0
    # sweep: as many leading blocks as fit the budget (at least one)
    Wc = W.copy()
    r = int(np.floor(cfg.p * c * b)) if cfg.mode == "unstructured" else 0
    nblk_total = -(-b // B)
    t_sweep, nblk = 0.0, 0
    for j1 in range(0, b, B):
        t0 = time.perf_counter()
        j2 = min(b, j1 + B)
        if cfg.mode == "unstructured":
            Mb = O.psi(Wc[:, j1:], xn[j1:], r)[:, : j2 - j1]
            r -= int(Mb.sum())
        else:
            Mb = O.nm_block_mask(Wc[:, j1:j2], xn[j1:j2], cfg.n, cfg.m)
        O.block_update_from_factor(Wc, Mb, U, j1, j2)
        t_sweep += time.perf_counter() - t0
        nblk += 1
        if t_h + t_f + t_sweep > budget_s:
            break
    t_full = t_h * (cfg.a / a_s) + t_f + t_sweep * (nblk_total / nblk)
    return {"value": c * b / t_full, "unit": UNIT, "cores": int(cores), "kind": "oracle",
            "sample": "layer %dx%d: Hessian on %d of %d tokens (%.1fs, scaled by token count), "
                      "factor (%.1fs), first %d of %d column blocks of the sweep (%.1fs, scaled by "
                      "block count)" % (c, b, a_s, cfg.a, t_h, t_f, nblk, nblk_total, t_sweep),
            "seconds_measured": round(t_h + t_f + t_sweep, 2),
            "seconds_extrapolated_layer": round(t_full, 1)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = select_mode(WL.CONFIGS[args.workload], args.mode_index)
    vals, last = [], None
    t0 = time.perf_counter()
    for i in range(args.warmup + args.steps):
        last = oracle_sample(cfg, budget_s=min(args.cpu_budget_s, 12.0))
        if i >= args.warmup:
            vals.append(last["value"])
        if time.perf_counter() - t0 > 240 and vals:
            break
    value = float(np.mean(vals))
    nweights = cfg.layers[0].c * cfg.layers[0].b
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
            "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": len(vals),
            "warmup": args.warmup, "ms_per_step": 1e3 * nweights / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": "%s (float64 CPU oracle on a bounded sample, extrapolated)"
                                   % cfg.name},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"],
                             "kind": "oracle", "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def run_single_layer(args):
    """One layer (c, b) with `a` calibration tokens through the three calls, `--reps` times: a
    small, fixed workload for profiler captures of single kernels."""
    import paper_2504_05346_b200 as T
    from paper_2504_05346_b200 import build as B_

    B_.build()
    T.load_library()
    c, b, a = [int(v) for v in args.single_layer.split(",")]
    cfg = select_mode(WL.CONFIGS[args.workload], args.mode_index)
    if args.block > 0:
        cfg = dataclasses.replace(cfg, B=args.block)
    dev = torch.device("cuda", 0)
    margs = mode_args(cfg, T)
    W = WL.make_weight(c, b, cfg.dtype, seed=cfg.seed, layer_index=0, device=dev)
    X = WL.make_activations(a, b, cfg.dtype, cfg.x_dist, cfg.outlier_frac, cfg.outlier_count,
                            cfg.outlier_scale, cfg.seed, 0, device=dev)
    H = torch.zeros((b, b), dtype=torch.float32, device=dev)
    out = []
    for _ in range(args.reps):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        H.zero_()
        ev[0].record()
        T.hessian_accumulate(H, X)
        ev[1].record()
        if args.hessian_only:
            torch.cuda.synchronize()
            ms = ev[0].elapsed_time(ev[1])
            out.append({"hessian_ms": round(ms, 4),
                        "hessian_tflops": round(a * b * (b + 1.0) / ms / 1e9, 1)})
            continue
        U, xn = T.prepare_inverse(H, cfg.damp_rel)
        ev[2].record()
        if args.structured > 0.0:   # Algorithm 2: whole columns, with --alpha outlier rows
            al = max(args.alpha, 0.0)
            _, _, _, st = T.prune_layer_structured(W, U, xn, args.structured, al,
                                                   H=H if al > 0 else None)
        elif args.alpha >= 0.0:   # n:m with outlier rows (2:4 unless the workload names an n:m)
            n_, m_ = (cfg.n, cfg.m) if cfg.mode == "nm" else (2, 4)
            _, _, _, st = T.prune_layer_outliers(W, U, xn, H, n_, m_, args.alpha, B=cfg.B)
        else:
            _, _, st = T.prune_layer(W, U, xn, B=cfg.B, **margs)
        ev[3].record()
        torch.cuda.synchronize()
        out.append({"hessian_ms": round(ev[0].elapsed_time(ev[1]), 4),
                    "prepare_ms": round(ev[1].elapsed_time(ev[2]), 4),
                    "prune_ms": round(ev[2].elapsed_time(ev[3]), 4), "n_pruned": st.n_pruned,
                    "select_misses": st.select_misses})
    print(json.dumps({"single_layer": [c, b, a], "workload": cfg.name, "runs": out}))


def replica_launch_command(n_gpus: int, argv, port: int):
    """Command that starts `n_gpus` replicas of this script, one process per GPU, on this node."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
            "--nproc-per-node", str(n_gpus), "--master-addr", "127.0.0.1",
            "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def _free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return int(sk.getsockname()[1])


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama2_7b", choices=sorted(WL.CONFIGS))
    ap.add_argument("--tokens", type=int, default=0, help="override the calibration token count")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-overlap", action="store_true",
                    help="issue every call on one stream instead of one stream per input / layer")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-workers", type=int, default=3,
                    help="host threads (each with a stream and an arena) of the end-to-end leg")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-split", action="store_true",
                    help="skip the extra untimed step that splits the step's time by kernel")
    ap.add_argument("--mode-index", type=int, default=0,
                    help="0: the workload's own sparsity mode; k: its k-th additional mode "
                         "(llama2_70b: 1 = 60 %% unstructured)")
    ap.add_argument("--cpu-budget-s", type=float, default=20.0)
    ap.add_argument("--single-layer", default="", metavar="C,B,A",
                    help="profile driver: one c x b layer with a tokens instead of the layer set")
    ap.add_argument("--hessian-only", action="store_true", help="with --single-layer: stop after H")
    ap.add_argument("--reps", type=int, default=1)
    ap.add_argument("--alpha", type=float, default=-1.0,
                    help="with --single-layer: n:m sweep with this fraction of outlier rows")
    ap.add_argument("--block", type=int, default=0,
                    help="with --single-layer: block width B instead of the workload's")
    ap.add_argument("--structured", type=float, default=0.0, metavar="P",
                    help="with --single-layer: structured pruning of this fraction of the columns")
    args = ap.parse_args()
    if args.single_layer:
        run_single_layer(args)
        return
    world_env = os.environ.get("WORLD_SIZE")
    if world_env is None and args.gpus > 1:
        # not under a launcher: start one replica per GPU and hand over
        cmd = replica_launch_command(args.gpus, sys.argv[1:], _free_port())
        sys.exit(subprocess.call(cmd))
    if world_env is not None and int(world_env) != args.gpus:
        sys.exit("bench.py: --gpus %d but the launcher started %s ranks" % (args.gpus, world_env))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
