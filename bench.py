#!/usr/bin/env python
"""Benchmark of the folded quantized linear layer on B200.

Default workload (``backbone_layer``): one pi0.5-like language-backbone layer at M = 816
tokens -- four activation sites, seven projections (q/k/v fused, o, gate/up fused, down),
o_proj/down_proj at W8A8 and the rest W4A4.  A step is one pass of the whole hot path over
one batch: per site the prologue kernel (scale + FWHT + per-token quantization) and the
tcgen05 integer GEMM with its dequant/bias epilogue.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-large-m] [--no-cpu-baseline]
                    [--workload backbone_layer|backbone_layer_w4|backbone_forward|backbone_forward_w4|expert_layer|expert_loop|sweep:M,K,N,block,bits[,after|composite]|w4a16:M,K,N|gptq:N,K,Mc,block]

Prints ONE JSON line (rank 0).  ``--impl reference`` times the CPU oracle on host cores.
``--gpus N`` without a torchrun environment starts the N ranks itself (one process per GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2609_24433_b200 import replicas, synth  # noqa: E402

METRIC = "fused FWHT+quant+W4A4/W8A8 GEMM throughput (whole layer)"
UNIT = "TOPS"
ROTATE = 4            # distinct weight/activation sets cycled so that no step finds its operands in L2
CPU_SAMPLE_ROWS = 512  # token rows the oracle arm processes per step (about 10 s on 8 cores)
INT8_DATASHEET_TOPS = 4500.0   # dense INT8 tensor rate of the B200 data sheet
LARGE_M_POINT = (16384, 8192, 8192, 128, 4)   # M, K, N, block, bits of the long-batch record in the default line


def layer_ops(sites) -> float:
    return float(sum(2 * s.M * s.K * s.N_total for s in sites))


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_burst=p["bf16_tflops"], bf16_sustained=p["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------ clock sampling ----
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while a region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        while not self._stop.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                mask = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self, note: str = ""):
        d = {"sm_mhz": (int(statistics.median(self.samples)) if self.samples else None),
             "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if note:
            d["note"] = note
        return d


# ------------------------------------------------------------------------ our arm ----
class LayerOnDevice:
    """Folded weights, inputs, outputs and workspace of ROTATE copies of one layer."""

    def __init__(self, sites, seed: int, device, rotate: int = 0):
        import torch
        from paper_2609_24433_b200 import fq
        self.sites, self.fq, self.torch = sites, fq, torch
        self.rotate = rotate if rotate > 0 else ROTATE
        self.sets = []
        for r in range(self.rotate):
            entry = []
            shared = {}          # expert loop: the 18 layers' handles serve all 10 denoising steps
            for i, site in enumerate(sites):
                wkey = site.name.split(".", 1)[1] if site.name.startswith("S") and "." in site.name else None
                if wkey is not None and wkey in shared:
                    # same weights as step 0 of this layer; only the activations (their scale drifts) are new
                    h0, y0, ws0 = shared[wkey]
                    data = synth.make_site(site, seed + 1000 * r + i, with_weights=False)
                    x = self._dev(data.x, site.x_dtype, device)
                    entry.append(dict(x=x, h=h0, y=y0, ws=ws0, host_x=data.x, site=site, rot=None))
                    continue
                data = synth.make_site(site, seed + 1000 * r + i)
                x = self._dev(data.x, site.x_dtype, device)
                W = torch.from_numpy(np.concatenate([data.W[n] for n, _ in site.consumers], 0)).to(device)
                b = torch.from_numpy(np.concatenate([data.bias[n] for n, _ in site.consumers], 0)).to(device)
                smooth = None
                if site.alpha is not None:      # SmoothQuant scale from the calibration batch, on the device
                    a = fq.col_absmax(torch.from_numpy(data.calib).to(device))
                    smooth = fq.smooth_scale(a, fq.col_absmax(W), site.alpha)
                rot = None
                if site.composite:      # stored rotation: permutation + per-block matrices (synthetic stand-ins)
                    perm, blocks = synth.composite_rotation(site.K, site.beta, seed + 1000 * r + i)
                    rot = (torch.from_numpy(perm).to(device), torch.from_numpy(blocks).to(device),
                           torch.empty(4 * site.M * site.K, dtype=torch.uint8, device=device),
                           torch.empty((site.M, site.K * site.bits // 8), dtype=torch.uint8, device=device),
                           torch.empty(site.M, dtype=torch.float32, device=device))
                    h = fq.fold_weights_composite(W, smooth, b, rot[0], rot[1], site.bits)
                elif site.fold_after:
                    pscale = torch.from_numpy(synth.post_scale(site, seed + 1000 * r + i)).to(device)
                    h = fq.fold_weights_after(W, pscale, b, site.beta, site.bits)
                else:
                    h = fq.fold_weights(W, smooth, b, site.beta, site.bits)
                ydt = torch.float32 if site.y_dtype == "f32" else torch.bfloat16
                y = torch.empty((site.M, site.N_total), dtype=ydt, device=device)
                ws = torch.empty(fq.workspace_bytes(site.M, site.K, site.N_total, site.bits), dtype=torch.uint8,
                                 device=device)
                entry.append(dict(x=x, h=h, y=y, ws=ws, host_x=data.x, site=site, rot=rot))
                if wkey is not None:
                    shared[wkey] = (h, y, ws)
                del W, data
            self.sets.append(entry)
        torch.cuda.synchronize()

    @staticmethod
    def _dev(a, dtype, device):
        import torch
        if dtype == "bf16":
            return torch.from_numpy(a.view(np.int16)).to(device).view(torch.bfloat16)
        return torch.from_numpy(a).to(device)

    def step(self, k: int, events=None):
        """One pass of the layer. ``events``: optional list of (e0, mark, e1) per site."""
        fq = self.fq
        for i, e in enumerate(self.sets[k % self.rotate]):
            if events is not None:
                e0, mark, e1 = events[i]
                e0.record()
                fq.profile_mark(mark)
            self.run_site(e, None if events is None else events[i][1])
            if events is not None:
                fq.profile_mark(None)
                e1.record()

    def run_site(self, e, mark=None):
        """Prologue + GEMM of one site: one call, or two for a stored composite rotation."""
        fq = self.fq
        if e["rot"] is None:
            fq.linear(e["x"], e["h"], 1.0, y=e["y"], workspace=e["ws"])
            return
        perm, blocks, scratch, codes, delta = e["rot"]
        fq.quantize_act_composite(e["x"], e["h"], perm, blocks, e["site"].bits, 1.0, codes=codes, delta=delta,
                                  workspace=scratch)
        if mark is not None:
            mark.record()
        (fq.gemm_w4a4 if e["site"].bits == 4 else fq.gemm_w8a8)(codes, delta, e["h"], y=e["y"], workspace=e["ws"])

    def capture(self):
        """One CUDA graph per rotating set (the step's kernels back to back, no host launch gaps),
        and a second graph per set that also carries external event-record nodes around and
        inside every site so that single-kernel durations can be read after a replay."""
        torch = self.torch
        self.graphs, self.ev_graphs, self.ev, self.ev_empty = [], [], [], []
        for r in range(self.rotate):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self.step(r)
            self.graphs.append(g)
            evs = [tuple(torch.cuda.Event(enable_timing=True, external=True) for _ in range(3)) for _ in self.sites]
            for trio in evs:
                for e in trio:
                    e.record()          # creates the underlying event before the capture
            torch.cuda.synchronize()
            pair = tuple(torch.cuda.Event(enable_timing=True, external=True) for _ in range(2))
            for e in pair:
                e.record()
            torch.cuda.synchronize()
            g2 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g2):
                self.step(r, evs)
                pair[0].record()        # two event nodes with nothing between: the cost of a record node
                pair[1].record()
            self.ev_graphs.append(g2)
            self.ev.append(evs)
            self.ev_empty.append(pair)
        torch.cuda.synchronize()

    def kernel_durations(self, replays: int):
        """Mean (prologue_ms, gemm_ms) per site over ``replays`` replays of the evented graphs, and
        the mean interval between two adjacent event-record nodes (what a record node itself costs:
        every interval between events contains one, so it is subtracted from the kernel figures)."""
        torch = self.torch
        act = [[] for _ in self.sites]
        gemm = [[] for _ in self.sites]
        empty = []
        for k in range(replays):
            self.ev_graphs[k % self.rotate].replay()
            torch.cuda.synchronize()
            for i, (e0, mark, e1) in enumerate(self.ev[k % self.rotate]):
                act[i].append(e0.elapsed_time(mark))
                gemm[i].append(mark.elapsed_time(e1))
            p0, p1 = self.ev_empty[k % self.rotate]
            empty.append(p0.elapsed_time(p1))
        ov = statistics.mean(empty)
        return ([max(statistics.mean(a) - ov, 1e-6) for a in act], [max(statistics.mean(g) - ov, 1e-6) for g in gemm], ov)

    def site_pair_us(self, i: int, calls: int = 8, replays: int = 5) -> float:
        """Microseconds per call of site i alone: ``calls`` back-to-back calls (rotating sets) captured as one
        graph with nothing between the prologue and the GEMM, so the two kernels overlap as they do in a step."""
        torch = self.torch
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for c in range(calls):
                self.run_site(self.sets[c % self.rotate][i])
        g.replay()
        torch.cuda.synchronize()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for _ in range(replays):
            g.replay()
        end.record()
        torch.cuda.synchronize()
        return start.elapsed_time(end) * 1e3 / (calls * replays)

    @property
    def launches_per_step(self) -> int:
        return 2 * len(self.sites)


def measure_int8_library_rate(device, local_rank: int) -> dict:
    """A yardstick, not part of the path: the INT8 rate a vendor-library GEMM (torch._int_mm, 8192^3) reaches on this
    very GPU, as a burst (best of 10) and sustained for two seconds under the power cap, with the clocks seen."""
    import torch
    n = 8192
    a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device)
    b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device=device).t()      # column-major second operand
    try:
        for _ in range(3):
            torch._int_mm(a, b)
    except Exception as exc:                                                         # not available in this build
        return {"unavailable": str(exc)[:120]}
    torch.cuda.synchronize()
    ops = 2.0 * n ** 3
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    best = float("inf")
    for _ in range(10):
        start.record()
        torch._int_mm(a, b)
        end.record()
        torch.cuda.synchronize()
        best = min(best, start.elapsed_time(end))
    sampler = ClockSampler(local_rank)
    with sampler:
        reps, t_end = 0, time.time() + 2.0
        start.record()
        while time.time() < t_end:
            for _ in range(20):
                torch._int_mm(a, b)
            reps += 20
            torch.cuda.synchronize()
        end.record()
        torch.cuda.synchronize()
    sustained_ms = start.elapsed_time(end) / reps
    return {"kernel": "torch._int_mm 8192^3 (vendor library; yardstick only)", "burst_tops": round(ops / (best * 1e-3) / 1e12, 1),
            "sustained_tops": round(ops / (sustained_ms * 1e-3) / 1e12, 1), "clocks_sustained": sampler.summary()}


def tensor_fractions(tops: float, peaks) -> dict:
    """One achieved INT8 rate against the three denominators in use: twice the measured bf16 cuBLAS rate, as a
    burst (a kernel timed alone or in a short region) and sustained (seconds under the power cap) -- dense int8 is
    nominally 2 x bf16 -- and the data-sheet dense INT8 figure."""
    return {"frac_burst": round(tops / (2.0 * peaks["bf16_burst"]), 4),
            "frac_sustained": round(tops / (2.0 * peaks["bf16_sustained"]), 4),
            "frac_datasheet_4500": round(tops / INT8_DATASHEET_TOPS, 4)}


def large_m_record(device, local_rank: int, peaks, seed: int):
    """The long-batch point of the throughput sweep, measured in the same process as the default step: the
    integer GEMM against the tensor peak and the prologue against the copy rate, with the clocks seen meanwhile."""
    import torch
    M, K, N, beta, bits = LARGE_M_POINT
    site = synth.sweep_site(M, K, N, beta, bits)
    layer = LayerOnDevice([site], seed=seed, device=device, rotate=1)     # 268 MB of activations per step: beyond L2
    for k in range(3):
        layer.step(k)
    torch.cuda.synchronize()
    layer.capture()
    for _ in range(3):
        layer.graphs[0].replay()
    steps = 12
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    torch.cuda.synchronize()
    with sampler:
        start.record()
        for _ in range(steps):
            layer.graphs[0].replay()
        end.record()
        torch.cuda.synchronize()
        t_end = time.time() + 0.4          # keep the same load up long enough for NVML to see it
        while time.time() < t_end:
            layer.graphs[0].replay()
            torch.cuda.synchronize()
    ms_step = start.elapsed_time(end) / steps
    act_ms, gemm_ms, ov = layer.kernel_durations(8)
    ops = 2.0 * M * K * N
    gemm_tops = ops / (gemm_ms[0] * 1e-3) / 1e12
    act_bytes = M * K * 2 + M * K + 4 * M
    act_gbs = act_bytes / (act_ms[0] * 1e-3) / 1e9
    rec = {"workload": workload_name(f"sweep:{M},{K},{N},{beta},{bits}"), "steps": steps,
           "us_per_step": round(ms_step * 1e3, 1), "tops_per_step": round(ops / (ms_step * 1e-3) / 1e12, 1),
           "l2": "268 MB of activations and 268 MB of outputs per step (beyond the 126 MB L2); 32 MB of weights stay resident",
           "gemm": dict({"us": round(gemm_ms[0] * 1e3, 1), "achieved_tops": round(gemm_tops, 1)}, **tensor_fractions(gemm_tops, peaks)),
           "prologue": {"us": round(act_ms[0] * 1e3, 1), "bytes": act_bytes, "achieved_gbs": round(act_gbs, 1),
                        "peak_gbs": peaks["hbm_gbs"], "frac": round(act_gbs / peaks["hbm_gbs"], 4)},
           "timing": "kernel figures from event-record nodes inside the step graph (they serialise the two kernels)",
           "clocks": sampler.summary()}
    del layer
    torch.cuda.empty_cache()
    return rec


def run_ours(args, rank: int, world: int, local_rank: int):
    import torch
    from paper_2609_24433_b200 import fq
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)

    global ROTATE, CPU_SAMPLE_ROWS
    if args.workload in ("backbone_forward", "backbone_forward_w4", "expert_loop"):
        ROTATE = 1              # a step already walks far more weight bytes than L2 holds
        CPU_SAMPLE_ROWS = 32    # keeps the oracle arm's sample to tens of seconds
    sites = workload_sites(args.workload)
    if args.workload.startswith("sweep:") and sites[0].M * sites[0].K >= (1 << 26):
        ROTATE = 1              # one step's activations and outputs alone are several times L2
    layer = LayerOnDevice(sites, seed=replicas.replica_seed(2, rank), device=device)
    ops = layer_ops(sites)
    K, Wm = args.steps, max(args.warmup, 3)

    for k in range(Wm):
        layer.step(k)
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: exactly K steps, each one replay of a captured step graph ----
    layer.capture()
    for k in range(Wm):
        layer.graphs[k % ROTATE].replay()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    barrier()
    with sampler:
        start.record()
        for k in range(K):
            layer.graphs[(Wm + k) % ROTATE].replay()
        end.record()
        torch.cuda.synchronize()
    barrier()
    ms_total = start.elapsed_time(end)
    note = ""
    if len(sampler.samples) < 5:
        # The timed region is shorter than NVML's refresh period: replay the same loop untimed for
        # about half a second and sample the clocks under that identical load.
        sampler = ClockSampler(local_rank)
        t_end = time.time() + 0.5
        with sampler:
            k = 0
            while time.time() < t_end:
                layer.graphs[k % ROTATE].replay()
                k += 1
                if k % 64 == 0:
                    torch.cuda.synchronize()
            torch.cuda.synchronize()
        note = "sampled during an immediate untimed replay of the timed loop (timed region < NVML period)"
    ms_per_step = replicas.max_over_ranks(ms_total, dist, device) / K
    value = replicas.job_throughput(ops * K, ms_total * 1e-3, dist, device) / 1e12

    st, word = fq.device_status()
    if st != fq.OK:
        raise RuntimeError(f"device watchdog fired during the benchmark: {word:#x}")

    # per-kernel durations: the same step graphs with event-record nodes between the kernels
    act_ms, gemm_ms, ev_overhead_ms = layer.kernel_durations(max(8, min(K, 40)))
    peaks = read_peaks()
    dom = max(range(len(sites)), key=lambda i: gemm_ms[i])
    s = sites[dom]
    gemm_ops = 2.0 * s.M * s.K * s.N_total
    achieved = gemm_ops / (gemm_ms[dom] * 1e-3) / 1e12
    # dense int8 : bf16 = 2 : 1 (4.5 vs 2.25 PFLOP/s nominal).  A timed region of well under a second runs at boost
    # clocks: the burst figure is its denominator; a region of seconds under the power cap takes the sustained one.
    short_region = ms_total < 1000.0
    which = "bf16_burst" if short_region else "bf16_sustained"
    int8_peak = 2.0 * peaks[which]
    roofline = {"bound": "tensor", "kernel": f"gemm_tcgen05_kernel<{s.bits},1> ({s.name}: M={s.M} K={s.K} N={s.N_total})",
                "achieved": round(achieved, 1), "peak": round(int8_peak, 1), "unit": "TOP/s",
                "frac": round(achieved / int8_peak, 4),
                "peak_source": f"{peaks['source']}: {'burst' if short_region else 'sustained'} bf16 cuBLAS {peaks[which]} TFLOP/s x 2 "
                               f"(int8:bf16), chosen because the timed region lasted {ms_total:.1f} ms",
                "traffic": TRAFFIC_BYTES.get((args.workload, s.name)),
                "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one launch in an ncu capture of this workload, "
                                  "taken separately (not re-measured by this run)" if (args.workload, s.name) in TRAFFIC_BYTES else None,
                "event_node_overhead_us": round(ev_overhead_ms * 1e3, 2),
                "per_site_us": {sites[i].name: {"prologue": round(act_ms[i] * 1e3, 2), "gemm": round(gemm_ms[i] * 1e3, 2)}
                                for i in range(min(len(sites), 8))},
                "per_site_us_note": "from event-record nodes between the kernels of the step graph: the nodes serialise kernels "
                                    "that otherwise overlap (programmatic dependent launch), so these durations are upper bounds, "
                                    "`achieved` is a lower bound, and their sum exceeds the step"}
    roofline.update(tensor_fractions(achieved, peaks))
    if len(sites) <= 8:
        roofline["site_us_alone"] = {sites[i].name: round(layer.site_pair_us(i), 2) for i in range(len(sites))}
        roofline["site_us_alone_note"] = "each site's two kernels replayed back to back on rotating sets, no event nodes"
    act_i = max(range(len(sites)), key=lambda i: act_ms[i])
    sa = sites[act_i]
    act_bytes = sa.M * sa.K * (2 if sa.x_dtype == "bf16" else 4) + sa.M * sa.K + 4 * sa.M
    roofline["prologue"] = {"site": sa.name, "bytes": act_bytes,
                            "achieved_gbs": round(act_bytes / (act_ms[act_i] * 1e-3) / 1e9, 1),
                            "peak_gbs": peaks["hbm_gbs"],
                            "frac": round(act_bytes / (act_ms[act_i] * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}

    # ---- end to end: host buffers, copies inside the timed region ----
    e2e = run_e2e(layer, sites, ops, world, K, Wm, dist, device)

    out = {
        "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": round(ms_per_step, 5), "us_per_layer": round(ms_per_step * 1e3, 2),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8/int4 codes, int32 accumulate, f32 transform",
        "data": "synthetic", "impl": "ours",
        "config": bench_config(args.workload, sites),
        "clocks": sampler.summary(note), "e2e": e2e, "gpu_launches": layer.launches_per_step * K,
        "roofline": roofline,
    }
    if world == 1 and args.workload == "backbone_layer" and not args.no_large_m:
        del layer
        torch.cuda.empty_cache()
        out["large_m"] = large_m_record(device, local_rank, peaks, seed=5)
        # last, so that its two seconds of full load do not heat the measurements above
        lib = measure_int8_library_rate(device, local_rank)
        out["int8_library_rate"] = lib
        if "burst_tops" in lib:
            out["roofline"]["frac_int8_library_burst"] = round(achieved / lib["burst_tops"], 4)
            out["large_m"]["gemm"]["frac_int8_library_sustained"] = round(out["large_m"]["gemm"]["achieved_tops"] / lib["sustained_tops"], 4)
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline(args.workload, steps=1)
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(layer, sites, ops, world, K, Wm, dist, device):
    """Same step through the public API with HOST buffers: pinned host -> device copies of the
    step's inputs, the kernels, and the device -> pinned host copy of every output, each step."""
    import torch
    entry = layer.sets[0]
    host_x = []
    for e in entry:
        site = e["site"]
        t = torch.from_numpy(e["host_x"].view(np.int16) if site.x_dtype == "bf16" else e["host_x"]).pin_memory()
        host_x.append(t)
    host_y = [torch.empty(e["y"].shape, dtype=e["y"].dtype).pin_memory() for e in entry]
    h2d = sum(t.numel() * t.element_size() for t in host_x)
    d2h = sum(t.numel() * t.element_size() for t in host_y)

    # Copies in, kernels and copies out run on three streams chained by events, so that a site's
    # result travels to the host while the next site's input travels to the device (PCIe is full
    # duplex) and its kernels run; every step still moves all inputs and all outputs.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    s_run = torch.cuda.current_stream()
    ev_in = [torch.cuda.Event() for _ in entry]
    ev_done = [torch.cuda.Event() for _ in entry]

    def step():
        for i, (e, hx, hy) in enumerate(zip(entry, host_x, host_y)):
            dst = e["x"].view(torch.int16) if e["x"].dtype == torch.bfloat16 else e["x"]
            with torch.cuda.stream(s_in):
                dst.copy_(hx, non_blocking=True)
                ev_in[i].record(s_in)
            s_run.wait_event(ev_in[i])
            layer.run_site(e)
            ev_done[i].record(s_run)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                hy.copy_(e["y"], non_blocking=True)
        torch.cuda.synchronize()

    n = max(3, min(K, 20))
    for _ in range(3):
        step()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(n):
        step()                      # ends with a synchronize: host time between steps is inside the interval
    end.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    seconds = start.elapsed_time(end) * 1e-3
    dt = replicas.max_over_ranks(seconds, dist, device) / n
    return {"value": round(replicas.job_throughput(ops * n, seconds, dist, device) / 1e12, 3), "unit": UNIT,
            "ms_per_step": round(dt * 1e3, 4),
            "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": n}


# --------------------------------------- weight-only W4A16 projection (its own workload) ----
def w4a16_shape(name: str):
    M, K, N = (int(v) for v in name[len("w4a16:"):].split(","))
    return M, K, N


def w4a16_inputs(M: int, K: int, N: int, seed: int):
    rng = np.random.default_rng(seed)
    W = synth.draw_weights(rng, N, K)
    b = rng.standard_normal(N).astype(np.float32)
    x = synth.as_dtype(rng.standard_normal((M, K)).astype(np.float32), "bf16")
    return W, b, x


def w4a16_cpu_baseline(M: int, K: int, N: int, steps: int):
    import oracle
    W, b, x = w4a16_inputs(M, K, N, 2)
    rows = min(N, max(8, (1 << 28) // max(1, M * K) // 8 * 8))     # bound the sample to ~2.7e8 multiply-adds
    wc, ws, _ = oracle.fold_weights(W[:rows], "f32", None, 1, 4)     # offline, untimed
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        oracle.linear_wonly(x, "bf16", wc, ws, b[:rows], 4, "bf16")
        times.append(time.perf_counter() - t0)
    dt = statistics.mean(times)
    return {"value": round(2.0 * M * K * rows / dt / 1e12, 6), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{rows} of {N} output channels, all {M} tokens (binary64 products and sums), {dt:.2f} s per step",
            "seconds_per_step": round(dt, 3)}


def run_w4a16(args, rank: int, world: int, local_rank: int):
    """fq_linear_w4a16 alone: y = s^W (qW x) + b on bf16 activations, weights rotating through enough
    handles that every call streams its 4-bit codes from HBM.  The bound is HBM (weight bytes)."""
    import torch
    from paper_2609_24433_b200 import fq
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=device)
    M, K, N = w4a16_shape(args.workload)
    sets = max(ROTATE, min(64, -(-300_000_000 // (N * K // 2))))      # > 2 x L2 of packed weights in rotation
    hs, xs = [], []
    for r in range(sets):
        W, b, x = w4a16_inputs(M, K, N, replicas.replica_seed(2, rank) + r)
        hs.append(fq.fold_weights(torch.from_numpy(W).to(device), None, torch.from_numpy(b).to(device), 1, 4))
        xs.append(torch.from_numpy(x.view(np.int16)).to(device).view(torch.bfloat16))
    y = torch.empty((M, N), dtype=torch.bfloat16, device=device)
    steps, Wm = args.steps, max(args.warmup, 3)
    for k in range(Wm):
        fq.linear_w4a16(xs[k % sets], hs[k % sets], y=y)
    torch.cuda.synchronize()
    # the K timed steps are ONE captured graph (K kernel nodes, handles rotating): a replay per step would
    # time the graph launch (4-5 us) rather than this microsecond-scale kernel
    timed = torch.cuda.CUDAGraph()
    with torch.cuda.graph(timed):
        for k in range(steps):
            fq.linear_w4a16(xs[(Wm + k) % sets], hs[(Wm + k) % sets], y=y)
    timed.replay()                      # untimed: every handle touched once more before the timed replay
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    with sampler:
        start.record()
        timed.replay()
        end.record()
        torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    ms_total = start.elapsed_time(end)
    note = ""
    if len(sampler.samples) < 5:
        sampler = ClockSampler(local_rank)
        t_end = time.time() + 0.5
        with sampler:
            while time.time() < t_end:
                timed.replay()
                torch.cuda.synchronize()
        note = "sampled during an immediate untimed replay of the timed loop (timed region < NVML period)"
    st, word = fq.device_status()
    if st != fq.OK:
        raise RuntimeError(f"device watchdog fired during the benchmark: {word:#x}")
    ops = 2.0 * M * K * N
    ms_per_step = replicas.max_over_ranks(ms_total, dist, device) / steps
    value = replicas.job_throughput(ops * steps, ms_total * 1e-3, dist, device) / 1e12
    peaks = read_peaks()
    alg_bytes = N * K // 2 + 8 * N + 2 * M * K + 2 * M * N          # codes + scale/bias + x + y
    gbs = alg_bytes / (ms_total / steps * 1e-3) / 1e9
    # end to end: x from pinned host memory, y back to pinned host memory, every step
    hx = torch.from_numpy(w4a16_inputs(M, K, N, 2)[2].view(np.int16)).pin_memory()
    hy = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
    n = max(3, min(steps, 50))

    def e2e_step(k):
        xs[k % sets].view(torch.int16).copy_(hx, non_blocking=True)
        fq.linear_w4a16(xs[k % sets], hs[k % sets], y=y)
        hy.copy_(y, non_blocking=True)
        torch.cuda.synchronize()
    for k in range(3):
        e2e_step(k)
    start.record()
    for k in range(n):
        e2e_step(k)
    end.record()
    torch.cuda.synchronize()
    sec = start.elapsed_time(end) * 1e-3
    e2e = {"value": round(replicas.job_throughput(ops * n, sec, dist, device) / 1e12, 4), "unit": UNIT,
           "ms_per_step": round(replicas.max_over_ranks(sec, dist, device) / n * 1e3, 4),
           "h2d_bytes_per_step": 2 * M * K, "d2h_bytes_per_step": 2 * M * N, "steps": n}
    out = {"metric": "weight-only W4A16 projection (fq_linear_w4a16)", "value": round(value, 3), "unit": UNIT,
           "n_gpus": world, "steps": steps, "warmup": Wm, "ms_per_step": round(ms_per_step, 5),
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
           "dtype": "int4 codes expanded to bf16 (exact), bf16 activations, f32 accumulate", "data": "synthetic", "impl": "ours",
           "config": {"workload": f"weight-only INT4 projection, M={M} tokens, K={K}, N={N}, bf16 in/out",
                      "l2": f"{sets} rotating weight handles ({sets * N * K // 2 >> 20} MiB of codes), no flush kernel",
                      "launch": "the K steps are one CUDA graph of K kernel nodes", "parallelism": "replicas only"},
           "clocks": sampler.summary(note), "e2e": e2e, "gpu_launches": steps,
           "roofline": {"bound": "hbm", "kernel": "weight_stream_kernel<bf16>", "achieved": round(gbs, 1),
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": round(gbs / peaks["hbm_gbs"], 4),
                        "bytes": alg_bytes, "traffic": None, "peak_source": f"{peaks['source']}: copy rate"}}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = w4a16_cpu_baseline(M, K, N, steps=1)
        print(json.dumps(out), flush=True)
    if dist is not None:
        dist.destroy_process_group()


# ------------------------------------------------ GPTQ fold (offline step, its own workload) ----
def gptq_shape(name: str):
    N, K, Mc, block = (int(v) for v in name[len("gptq:"):].split(","))
    return N, K, Mc, block


def gptq_inputs(N: int, K: int, Mc: int, seed: int):
    """Weights and calibration tokens with cross-channel correlation (a rank-32 mixture plus noise): the
    structure that gives error compensation something to do."""
    rng = np.random.default_rng(seed)
    W = synth.draw_weights(rng, N, K)
    mix = rng.standard_normal((32, K)).astype(np.float32)
    calib = (0.85 * rng.standard_normal((Mc, 32)).astype(np.float32) @ mix
             + 0.15 * rng.standard_normal((Mc, K)).astype(np.float32)).astype(np.float32)
    return W, calib


def gptq_flops(N: int, K: int, Mc: int) -> float:
    # fused multiply-adds x 2: second moment K^2 Mc, factorisation K^3/3, triangular inverse K^3/6, sweep N K^2/2
    return 2.0 * (K * K * Mc + K ** 3 / 3.0 + K ** 3 / 6.0 + N * K * K / 2.0)


def gptq_cpu_baseline(N: int, K: int, Mc: int, block: int, steps: int):
    import oracle
    Ks = min(K, 512)                                  # the oracle's factorisation is cubic: a narrower site
    Ns = min(N, 256)
    W, calib = gptq_inputs(Ns, Ks, min(Mc, 1024), 2)
    times = []
    for _ in range(steps):
        t0 = time.perf_counter()
        oracle.fold_weights_gptq(W, "f32", None, min(block, Ks), calib, "f32", 0.01, 4)
        times.append(time.perf_counter() - t0)
    dt = statistics.mean(times)
    return {"value": round(gptq_flops(Ns, Ks, min(Mc, 1024)) / dt / 1e12, 6), "unit": "TFLOP/s", "cores": oracle.num_threads(),
            "kind": "oracle", "sample": f"a narrower site of the same kind: N={Ns}, K={Ks}, {min(Mc, 1024)} tokens, {dt:.2f} s per fold",
            "seconds_per_step": round(dt, 3)}


def run_gptq(args, rank: int, world: int, local_rank: int):
    """fq_fold_weights_gptq alone (offline): one fold per step, timed with CUDA events around the call."""
    import torch
    from paper_2609_24433_b200 import fq
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    N, K, Mc, block = gptq_shape(args.workload)
    W, calib = gptq_inputs(N, K, Mc, replicas.replica_seed(2, rank))
    Wd, cd = torch.from_numpy(W).to(device), torch.from_numpy(calib).to(device)
    steps, Wm = max(1, min(args.steps, 10)), 3
    for _ in range(Wm):
        fq.fold_weights_gptq(Wd, None, None, cd, block, 4, 0.01)
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local_rank)
    torch.cuda.synchronize()
    each = []
    with sampler:
        for _ in range(steps):
            start.record()
            fq.fold_weights_gptq(Wd, None, None, cd, block, 4, 0.01)      # synchronises its stream (offline call)
            end.record()
            torch.cuda.synchronize()
            each.append(start.elapsed_time(end))
    # the call allocates, frees and issues ~K launches from the host: the median keeps a busy host out of the figure
    ms = statistics.median(each)
    flops = gptq_flops(N, K, Mc)
    peak = 148 * 128 * 2 * 1.965e9 / 1e12            # binary32 fma lanes x 2 flops x boost clock, TFLOP/s
    ach = flops / (ms * 1e-3) / 1e12
    out = {"metric": "GPTQ fold in transformed coordinates (fq_fold_weights_gptq, offline): arithmetic rate", "value": round(ach, 4),
           "unit": "TFLOP/s", "n_gpus": world, "steps": steps, "warmup": Wm, "ms_per_step": round(ms, 3), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f32 (fixed-order fma chains), int4 codes", "data": "synthetic",
           "impl": "ours", "config": {"workload": f"GPTQ fold N={N} K={K}, {Mc} calibration tokens, block {block}, W4",
                                      "timing": f"median of {steps} folds; min {min(each):.1f} ms, max {max(each):.1f} ms",
                                      "parallelism": "replicas only"},
           "clocks": sampler.summary(""), "gpu_launches": steps * (K + 8),
           "e2e": {"value": round(ach, 4), "unit": "TFLOP/s", "ms_per_step": round(ms, 3), "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 4,
                   "note": "the call itself is the user-facing API and ends with a host synchronisation; inputs are device tensors"},
           "roofline": {"bound": "alu", "kernel": "rev_chol_col_kernel x K (column-sequential)", "achieved": round(ach, 4),
                        "peak": round(peak, 1), "unit": "TFLOP/s", "frac": round(ach / peak, 5), "traffic": None,
                        "peak_source": "derived: 148 SMs x 128 binary32 lanes x 2 flops x 1.965 GHz"}}
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = gptq_cpu_baseline(N, K, Mc, block, steps=1)
        print(json.dumps(out), flush=True)


# ------------------------------------------------------------------- oracle arm ----
def cpu_baseline(workload: str, steps: int, warmup: int = 0):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    sites = workload_sites(workload)
    rows = CPU_SAMPLE_ROWS
    prepared = []
    for i, site in enumerate(sites):
        data = synth.make_site(site, 2 + i)
        W = np.concatenate([data.W[n] for n, _ in site.consumers], 0)
        b = np.concatenate([data.bias[n] for n, _ in site.consumers], 0)
        smooth = None
        if site.alpha is not None:
            smooth = oracle.smooth_scale(oracle.col_absmax(data.calib), oracle.col_absmax(W), site.alpha)
        rot = None
        if site.composite:
            rot = synth.composite_rotation(site.K, site.beta, 2 + i)
            wc, ws, g = oracle.fold_weights_composite(W, "f32", smooth, rot[0], rot[1], site.bits)
        elif site.fold_after:
            wc, ws, g = oracle.fold_weights_after(W, "f32", synth.post_scale(site, 2 + i), site.beta, site.bits)
        else:
            wc, ws, g = oracle.fold_weights(W, "f32", smooth, site.beta, site.bits)      # offline, untimed
        prepared.append((site, np.ascontiguousarray(data.x[:rows]), g, wc, ws, b, rot))
    times = []
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        for site, x, g, wc, ws, b, rot in prepared:
            if site.composite:
                ac, ad = oracle.composite_quantize(x, site.x_dtype, g, rot[0], rot[1], site.bits)
                oracle.epilogue(oracle.gemm_i32(ac, wc, site.K, site.bits), ad, ws, b, site.y_dtype)
            elif site.fold_after:
                ac, ad = oracle.quantize_act_after(x, site.x_dtype, g, site.beta, site.bits)
                oracle.epilogue(oracle.gemm_i32(ac, wc, site.K, site.bits), ad, ws, b, site.y_dtype)
            else:
                oracle.linear(x, site.x_dtype, g, site.beta, site.bits, 1.0, wc, ws, b, site.y_dtype)
        if it >= warmup:
            times.append(time.perf_counter() - t0)
    ops = sum(2.0 * rows * s.K * s.N_total for s in sites)
    dt = statistics.mean(times)
    return {"value": round(ops / dt / 1e12, 6), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{rows} of {sites[0].M} token rows through all {len(sites)} sites "
                      f"(prologue + integer GEMM + epilogue, all N), {dt:.2f} s per step",
            "seconds_per_step": round(dt, 3)}


def bench_config(workload: str, sites) -> dict:
    """The `config` object of the JSON line: the workload and how the GPU arm stages and launches it.  Both arms
    print the same object (the oracle arm runs a bounded sample of this workload; its `cpu_baseline.sample` says
    which)."""
    rotate = 1 if workload in ("backbone_forward", "backbone_forward_w4", "expert_loop") or \
        (workload.startswith("sweep:") and sites[0].M * sites[0].K >= (1 << 26)) else ROTATE
    return {"workload": workload_name(workload), "M": sites[0].M,
            "sites": {s.name: {"K": s.K, "N": s.N_total, "bits": s.bits, "block": s.beta} for s in sites[:8]},
            "n_sites": len(sites), "ops_per_step": layer_ops(sites),
            "parallelism": "replicas only (one batch per GPU, no collective)",
            "l2": f"{rotate} rotating weight+activation sets (> 126 MB L2 in total), no flush kernel",
            "launch": "one CUDA-graph replay per step"}


def run_reference(args):
    global CPU_SAMPLE_ROWS
    if args.workload in ("backbone_forward", "backbone_forward_w4", "expert_loop"):
        CPU_SAMPLE_ROWS = 32
    if args.workload.startswith("gptq:"):
        N, K, Mc, block = gptq_shape(args.workload)
        base = gptq_cpu_baseline(N, K, Mc, block, steps=max(1, min(args.steps, 3)))
        print(json.dumps({"metric": "GPTQ fold in transformed coordinates (fq_fold_weights_gptq, offline): arithmetic rate",
                          "value": base["value"], "unit": "TFLOP/s", "n_gpus": args.gpus,
                          "steps": max(1, min(args.steps, 3)), "warmup": 0, "ms_per_step": round(base["seconds_per_step"] * 1e3, 3),
                          "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                          "impl": "reference", "config": {"workload": "GPTQ fold, " + base["sample"]}, "cpu_baseline": base,
                          "e2e": {"value": base["value"], "unit": "TFLOP/s",
                                  "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}), flush=True)
        return
    if args.workload.startswith("w4a16:"):
        M, K, N = w4a16_shape(args.workload)
        steps = max(1, min(args.steps, 5))
        base = w4a16_cpu_baseline(M, K, N, steps)
        print(json.dumps({"metric": "weight-only W4A16 projection (fq_linear_w4a16)", "value": base["value"], "unit": UNIT,
                          "n_gpus": args.gpus, "steps": steps, "warmup": 0,
                          "ms_per_step": round(base["seconds_per_step"] * 1e3, 2), "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "binary64 products and sums", "data": "synthetic",
                          "impl": "reference", "config": {"workload": f"weight-only INT4 projection, M={M}, K={K}, N={N}"},
                          "cpu_baseline": base,
                          "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}),
              flush=True)
        return
    sites = workload_sites(args.workload)
    # Exactly --steps timed steps after --warmup untimed ones, like the GPU arm; the per-step sample of token rows
    # shrinks with the number of steps so that the whole run stays within about two minutes of host time.
    steps, warm = max(1, args.steps), max(0, args.warmup)
    CPU_SAMPLE_ROWS = max(16, min(CPU_SAMPLE_ROWS, sites[0].M, CPU_SAMPLE_ROWS * 12 // (steps + warm) // 16 * 16))
    base = cpu_baseline(args.workload, steps=steps, warmup=warm)
    out = {"metric": METRIC, "value": base["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
           "warmup": warm, "ms_per_step": round(base["seconds_per_step"] * 1e3, 2), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "int8/int4 codes, int32 accumulate, f32 transform",
           "data": "synthetic", "impl": "reference",
           "config": bench_config(args.workload, sites),
           "cpu_baseline": base,
           "e2e": {"value": base["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out), flush=True)


# -------------------------------------------------------------------- workloads ----
# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture).
TRAFFIC_BYTES = {("backbone_layer", "gate_up"): 41771776}


def workload_sites(name: str):
    if name == "backbone_layer":
        return synth.backbone_layer_sites(selective_int8=True)
    if name == "backbone_layer_w4":
        return synth.backbone_layer_sites(selective_int8=False)
    if name == "expert_layer":
        return synth.expert_layer_sites()
    if name in ("backbone_forward", "backbone_forward_w4"):   # 18 layers with distinct weights: one forward per step
        import dataclasses
        return [dataclasses.replace(s, name=f"L{layer:02d}.{s.name}")
                for layer in range(18) for s in synth.backbone_layer_sites(selective_int8=name == "backbone_forward")]
    if name == "expert_loop":                                  # 18 layers x 10 denoising steps, activation scale drifting
        import dataclasses
        return [dataclasses.replace(s, name=f"S{step}.L{layer:02d}.{s.name}")
                for step in range(10) for layer in range(18)
                for s in synth.expert_layer_sites(sigma=synth.expert_step_sigma(step))]
    if name.startswith("sweep:"):        # one site of the throughput sweep: sweep:M,K,N,block,bits[,after]
        f = name[6:].split(",")
        M, K, N, beta, bits = (int(v) for v in f[:5])
        return [synth.sweep_site(M, K, N, beta, bits, fold_after=len(f) > 5 and f[5] == "after",
                                 composite=len(f) > 5 and f[5] == "composite")]
    raise ValueError(name)


def workload_name(name: str) -> str:
    if name.startswith("sweep:"):
        f = name[6:].split(",")
        M, K, N, beta, bits = (int(v) for v in f[:5])
        return f"throughput sweep point M={M} K={K} N={N}, block {beta}, W{bits}A{bits}" + \
               (", fold-after" if len(f) > 5 and f[5] == "after" else "") + \
               (", stored composite rotation" if len(f) > 5 and f[5] == "composite" else "")
    return {"backbone_forward": "18-layer pi0.5-like backbone forward (distinct weights per layer), M=816, o/down W8A8, rest W4A4",
            "backbone_forward_w4": "18-layer pi0.5-like backbone forward (distinct weights per layer), M=816, uniform W4A4",
            "expert_loop": "action-expert denoising loop: 10 steps x 18 layers (one set of layer weights serves all steps), M=50, "
                           "width 1024, MLP 4096, W4A4, block 64, activation scale drifting 1.0 -> 0.1",
            "backbone_layer": "pi0.5-like backbone layer, M=816, hidden 2048, MLP 16384, o/down W8A8, rest W4A4",
            "backbone_layer_w4": "pi0.5-like backbone layer, M=816, uniform W4A4",
            "expert_layer": "action-expert layer, M=50, width 1024, MLP 4096, W4A4, block 64"}[name]


def spawn_ranks(args) -> int:
    """`--gpus N` outside a torchrun environment: start the N ranks here, one process per GPU, the way a launcher
    would (rendezvous on 127.0.0.1).  Refuses loudly when the machine does not have N GPUs."""
    if not args.dry_run and args.impl == "ours":
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            print(f"bench.py: --gpus {args.gpus} needs {args.gpus} CUDA devices, this machine shows {have}", file=sys.stderr)
            return 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ)
    env.setdefault("NCCL_DEBUG", "INFO")            # the communicator's own log (one line per rank) stays on
    env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def run_dry(args, rank: int, world: int):
    """The multi-rank bookkeeping of the benchmark without any GPU: every rank reports a made-up duration of
    (rank + 1) ms for 10 units of work, and rank 0 prints the line that MAX-over-ranks timing gives."""
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("gloo")
    ms = float(rank + 1)
    slowest = replicas.max_over_ranks(ms, dist)
    rate = replicas.job_throughput(10.0, ms * 1e-3, dist)
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ms_per_step": slowest, "value": rate,
                          "seed_of_last_rank": replicas.replica_seed(2, world - 1)}), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="backbone_layer")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-large-m", action="store_true", help="skip the long-batch record of the default workload")
    ap.add_argument("--dry-run", action="store_true",
                    help="rank plumbing only: CPU ranks (gloo) exchange a per-rank duration; used by the CPU tests")
    args = ap.parse_args()
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(spawn_ranks(args))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s): start one rank per GPU")
    if args.dry_run:
        run_dry(args, rank, world)
        return
    if args.impl == "reference":
        if rank == 0:
            run_reference(args)
        return
    if args.workload.startswith("w4a16:"):
        run_w4a16(args, rank, world, local_rank)
        return
    if args.workload.startswith("gptq:"):
        run_gptq(args, rank, world, local_rank)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
