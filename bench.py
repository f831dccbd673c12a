#!/usr/bin/env python
"""Benchmark of the SpeCa feature-cache hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic input: a reference-step
cache update of every entry (Eq. 3), a forecast of every entry (Eq. 2) -- the verification entry's
forecast comes out of the verification launch -- the fused forecast + verification of the
verification entry (Eq. 4 and the accept rule) and the per-sample selection. ``value`` is the
algorithmic bytes of a step divided by its device time (GB/s), with the inputs already resident in
HBM; ``e2e`` repeats the measurement with the step's inputs in pinned host memory and its outputs
copied back.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config flux] [--impl reference]
                    [--detail PATH] [--full]

The LAST line printed (rank 0) is one compact JSON object (under 2 KB) with the headline numbers.
Everything else -- per-kernel tables, the other configurations, the optional sweeps of ``--full`` --
goes to the JSON file named by ``--detail``. With ``--gpus N`` and no process group in the
environment the script starts its own N ranks (one per GPU).
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2509_11628_b200 import dist as D  # noqa: E402
from paper_2509_11628_b200 import workloads as W  # noqa: E402

METRIC = "forecast+verify GB/s"
VALUE_COVERS = "update+forecast+verify+select (whole step)"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
MAX_LINE_BYTES = 2000

# DRAM bytes per cached element per launch: (dram__bytes_read.sum + dram__bytes_write.sum) / elements
# from the ncu capture of the DiT-XL/2-shaped case (1.6 GB cache; see the file named in TRAFFIC_SOURCE).
# The kernels are reuse-free streams, so traffic grows in proportion to the elements a launch covers;
# other workloads scale by that (the verify figure is from profiles/verify_kernel_dit_xl2.md and counts
# reads only: the forecast it stores is still dirty in L2 when the kernel ends). An entry is None while
# its kernel has changed since the counters were taken.
NCU_DRAM_BYTES_PER_ELEM = {"update": 11.80, "forecast": 7.93, "verify": 8.01}
TRAFFIC_SOURCE = "ncu dram bytes/elem on the DiT-shaped capture (profiles/stream_kernels_dit_xl2.md) x elems"


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def make_workload(name: str) -> W.Workload:
    if name == "flux_b8":
        return W.flux_adaptive(max_order=2, batch=8)
    return W.BY_NAME[name]()


def algorithmic_bytes(w: W.Workload, order: int, layout: int = 0, pred_from_verify: bool = True):
    """Bytes a step must move per kernel, from the per-element figures: update reads the feature
    and `order` old planes and writes order+1 planes (a cache that keeps raw features, layout 1, reads
    the feature and writes one plane); forecast reads order+1 planes and writes one; verify reads
    order+1 planes and the fresh feature. With `pred_from_verify` the verification entry's forecast
    is written by the verify launch (one more word per element there) and left out of the forecast
    launch."""
    eb = w.elem_bytes
    n_all = w.elems_per_order
    n_ver = w.batch * w.entry_elems(w.vidx)
    return {
        "update": (2 if layout == 1 else 2 * order + 2) * eb * n_all,
        "forecast": (order + 2) * eb * (n_all - n_ver if pred_from_verify else n_all),
        "verify": (order + (3 if pred_from_verify else 2)) * eb * n_ver,
        "select": 0,
    }


class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.stop_flag = [], set(), False
        self.max_mhz, self.ok = None, False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def summary(self):
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"], "samples": 0}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


class Harness:
    """Device-resident state for one workload: cache, two alternating feature sets, outputs."""

    def __init__(self, w: W.Workload, device: str, seed_offset: int = 0, path: int = 0, fused_select: bool = True,
                 layout: int = 0):
        from paper_2509_11628_b200 import binding as S
        self.S, self.w, self.device = S, w, torch.device(device)
        self.fused_select, self.layout = fused_select, layout
        self.B, self.m = w.batch, w.max_order
        self.cache = S.SpecaCache(w.entries, w.batch, w.max_order, w.dtype, device, path=path, layout=layout)
        self.src = W.FeatureSource(w, device, seed_offset)
        ne = len(w.entries)
        # warm the tables with max_order + 1 fully computed steps of the generator
        for step in range(self.m + 1):
            t = [w.times[step]] * self.B
            for e in range(ne):
                f = self.src.feature(e, step, t)
                one = [None] * ne
                one[e] = f
                self.cache.update(one, t)
                del f
            self.cache.commit_step()
        torch.cuda.synchronize(self.device)
        self.step0 = self.m + 1
        # inputs of the timed steps: two feature sets used alternately, outputs, verification feature
        self.feats = [[self.src.feature(e, self.step0 + k, [w.times[self.step0 + k]] * self.B) for e in range(ne)]
                      for k in range(2)]
        self.fresh = [self.src.feature(w.vidx, self.step0 + 2 + k, [w.times[self.step0 + 2 + k]] * self.B)
                      for k in range(2)]
        self.outs = [torch.empty(self.B, n, d, dtype=w.torch_dtype, device=self.device) for n, d in w.entries]
        self.err = torch.zeros(self.B, dtype=torch.float32, device=self.device)
        self.accept = torch.zeros(self.B, dtype=torch.uint8, device=self.device)
        self.active = torch.ones(self.B, dtype=torch.uint8, device=self.device)
        self.active_next = torch.ones(self.B, dtype=torch.uint8, device=self.device)
        self.spec = torch.zeros(self.B, dtype=torch.int32, device=self.device)
        self.idx = torch.zeros(self.B, dtype=torch.int32, device=self.device)
        self.n_active = torch.zeros(1, dtype=torch.int32, device=self.device)
        self.j = 0
        self.t_base = w.times[self.m]
        torch.cuda.synchronize(self.device)

    def times_for(self, j):
        gap = 0.02
        t_ref = self.t_base - gap * (j + 1)
        return [t_ref] * self.B, [t_ref - 0.5 * gap] * self.B

    def step(self, events=None, feats=None, fresh=None, outs=None):
        """update -> commit -> forecast -> verify -> select on the current stream: three launches
        (speca_cache_update_activate, speca_forecast, speca_verify_select), or five with
        fused_select=False (update, activate, forecast, verify, select). The verification entry is
        forecast once: by the verification launch, which writes it to that entry's output."""
        S, c, w = self.S, self.cache, self.w
        j = self.j
        self.j += 1
        t_ref, t_tgt = self.times_for(j)
        feats = feats if feats is not None else self.feats[j & 1]
        fresh = fresh if fresh is not None else self.fresh[j & 1]
        outs = outs if outs is not None else self.outs
        others = list(outs)
        others[w.vidx] = None
        tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - (j % w.total_steps), w.total_steps)] * self.B
        if events is not None:
            events[0].record()
        if self.fused_select:
            c.update_activate(feats, t_ref, None, self.spec, self.active)   # the re-arming rides in the update launch
            c.commit_step()
            if events is not None:
                events[1].record()
        else:
            c.update(feats, t_ref)
            c.commit_step()
            if events is not None:
                events[1].record()
            c.activate(None, self.spec, self.active)
        if events is not None:
            events[2].record()
        c.forecast(t_tgt, others, self.active)
        if events is not None:
            events[3].record()
        if self.fused_select:
            c.verify_select(fresh, t_tgt, tau, self.err, self.accept, self.active, self.active_next, 1 << 30, 1, self.spec,
                            self.idx, self.n_active, out_pred=outs[w.vidx])
            self.active, self.active_next = self.active_next, self.active
            if events is not None:
                events[4].record()
        else:
            c.verify(fresh, t_tgt, tau, self.err, self.accept, self.active, out_pred=outs[w.vidx])
            if events is not None:
                events[4].record()
            c.select_adaptive(self.accept, 1 << 30, 1, self.spec, self.active, self.idx, self.n_active)
        if events is not None:
            events[5].record()

    def close(self):
        self.cache.close()


def time_device_resident(h: Harness, steps: int, warmup: int, info: D.RankInfo, sample_clocks: bool):
    """The timed region: exactly `steps` steps between two events on the launching stream, nothing else
    in the stream (no per-kernel event records), barrier + synchronize on both sides, clocks sampled
    meanwhile. A second, untimed pass of at most 20 steps records events around each launch for the
    per-kernel breakdown; in the three-launch step nothing runs between the update and the forecast or
    after the verification, so no gap is timed there."""
    dev = h.device
    for _ in range(warmup):
        h.step()
    torch.cuda.synchronize(dev)
    launches0 = h.cache.launches
    sampler = ClockSampler(physical_gpu_index(dev.index or 0)) if sample_clocks else None
    D.barrier()
    torch.cuda.synchronize(dev)
    if sampler:
        sampler.start()
    t_start = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_start.record()
    for k in range(steps):
        h.step()
    t_end.record()
    torch.cuda.synchronize(dev)
    D.barrier()
    if sampler:
        sampler.stop_flag = True
        sampler.join(timeout=2.0)
    total_ms = t_start.elapsed_time(t_end)
    launches = h.cache.launches - launches0
    n = max(1, min(steps, 20))
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(n)]
    for k in range(n):
        h.step(ev[k])
    torch.cuda.synchronize(dev)
    per = {"update": 0.0, "forecast": 0.0, "verify": 0.0, "select": 0.0}
    for k in range(n):
        per["update"] += ev[k][0].elapsed_time(ev[k][1])
        per["forecast"] += ev[k][2].elapsed_time(ev[k][3])
        per["verify"] += ev[k][3].elapsed_time(ev[k][4])
        if not h.fused_select:   # activate + select launches of the five-launch step
            per["select"] += ev[k][1].elapsed_time(ev[k][2]) + ev[k][4].elapsed_time(ev[k][5])
    per = {k: v / n for k, v in per.items()}
    return total_ms, per, launches, (sampler.summary() if sampler else None)


def time_multi_horizon(h: Harness, peak: float, forecast_ms: float, K: int = 4, reps: int = 20):
    """K speculative steps forecast from one read of the tables (speca_forecast_multi) against K
    single-target launches: device time, algorithmic GB/s over (order + 1 + K) words per element."""
    w, dev = h.w, h.device
    outs = [torch.empty(K, h.B, n, d, dtype=w.torch_dtype, device=dev) for n, d in w.entries]
    t0 = h.t_base - 0.02 * (h.j + 1)
    targets = [[t0 - 0.01 * (k + 1)] * h.B for k in range(K)]
    for _ in range(3):
        h.cache.forecast_multi(targets, outs, h.active)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        h.cache.forecast_multi(targets, outs, h.active)
    e1.record()
    torch.cuda.synchronize(dev)
    ms = e0.elapsed_time(e1) / reps
    nbytes = (w.max_order + 1 + K) * w.elem_bytes * w.elems_per_order
    gbs = nbytes / (ms * 1e-3) / 1e9
    del outs
    torch.cuda.empty_cache()
    return {"targets": K, "ms": ms, "algorithmic_bytes": nbytes, "gbs": gbs, "frac_of_measured_peak": gbs / peak,
            "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS, "ms_of_k_single_forecasts": K * forecast_ms,
            "speedup_vs_single_forecasts": K * forecast_ms / ms}


def time_graph_replay(h: Harness, K: int = 4, reps: int = 20):
    """K consecutive speculative steps (forecast of every other entry + verification / continuation) issued
    call by call, against the same K steps captured once into a CUDA graph and replayed: the calls neither
    allocate nor synchronise, and the masks chain on the device, so a whole speculative run needs no host
    round trip. The threshold is set so that every sample stays active (constant work per step)."""
    w, dev = h.w, h.device
    others = list(h.outs)
    others[w.vidx] = None
    tau = [1e30] * h.B
    masks = [torch.ones(h.B, dtype=torch.uint8, device=dev) for _ in range(2)]
    t0 = h.t_base - 0.02 * (h.j + 1)
    targets = [[t0 - 0.004 * (k + 1)] * h.B for k in range(K)]

    def run():
        for k in range(K):
            h.cache.forecast(targets[k], others, masks[k & 1])
            h.cache.verify_select(h.fresh[k & 1], targets[k], tau, h.err, h.accept, masks[k & 1], masks[(k + 1) & 1], 1 << 30, 1,
                                  h.spec, h.idx, h.n_active, out_pred=h.outs[w.vidx])

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize(dev)
        return e0.elapsed_time(e1) / reps / K

    eager_ms = timed(run)
    side = torch.cuda.Stream(dev)
    side.wait_stream(torch.cuda.current_stream(dev))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run()                                   # the capture must not be the first use of anything
        torch.cuda.synchronize(dev)
        with torch.cuda.graph(graph, stream=side):
            run()
    torch.cuda.current_stream(dev).wait_stream(side)
    graph_ms = timed(graph.replay)
    return {"steps_per_graph": K, "eager_ms_per_step": eager_ms, "graph_ms_per_step": graph_ms,
            "eager_steps_per_s": 1e3 / eager_ms, "graph_steps_per_s": 1e3 / graph_ms}


def time_fused_reference_step(h: Harness, peak: float, reps: int = 20):
    """A reference step and the first forecast after it as ONE launch (speca_cache_update_forecast): the
    forecast is evaluated from the planes the update has just formed, so the tables are not read again --
    2 * order + 3 words per element (order + 2 of them writes) instead of (2 * order + 2) + (order + 2).
    A cache that keeps raw features copies the feature into its ring plane and sums the planes with the
    feature still in registers: order + 3 words instead of 2 + (order + 2).
    The verification entry is only updated (its forecast comes out of the verification launch)."""
    w, dev = h.w, h.device
    others = list(h.outs)
    others[w.vidx] = None
    m, eb = w.max_order, w.elem_bytes
    n_ver = w.batch * w.entry_elems(w.vidx)
    ab = algorithmic_bytes(w, m, layout=h.layout)
    # the update's traffic, one more store where a forecast is written and, for raw features, the other planes' reads
    nbytes = ab["update"] + (1 + (m if h.layout == 1 else 0)) * eb * (w.elems_per_order - n_ver)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0.0
    for r in range(reps + 3):
        j = h.j
        h.j += 1
        t_ref, t_tgt = h.times_for(j)
        e0.record()
        h.cache.update_forecast(h.feats[j & 1], t_ref, t_tgt, others, spec_count=h.spec, rearm=h.active)
        e1.record()
        torch.cuda.synchronize(dev)
        if r >= 3:
            total += e0.elapsed_time(e1)
    ms = total / reps
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"ms": ms, "algorithmic_bytes": nbytes, "gbs": gbs, "frac_of_measured_peak": gbs / peak,
            "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS,
            "bytes_of_the_two_launches": ab["update"] + ab["forecast"],
            "traffic_saved_vs_two_launches": 1.0 - nbytes / float(ab["update"] + ab["forecast"])}


def time_fused_reference_step_multi(h: Harness, peak: float, K: int = 4, reps: int = 10):
    """The same with K speculative times forecast in the reference step's pass (speca_cache_update_forecast_multi):
    2 * order + 2 + K words per element against (2 * order + 2) + (order + 1 + K) for update + speca_forecast_multi."""
    w, dev = h.w, h.device
    m, eb = w.max_order, w.elem_bytes
    outs = [torch.empty(K, h.B, n, d, dtype=w.torch_dtype, device=dev) for n, d in w.entries]
    nbytes = (2 * m + 2 + K) * eb * w.elems_per_order
    two_bytes = ((2 * m + 2) + (m + 1 + K)) * eb * w.elems_per_order
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    res = {}
    for name in ("fused", "two_launches"):
        total = 0.0
        for r in range(reps + 3):
            j = h.j
            h.j += 1
            t_ref, _ = h.times_for(j)
            targets = [[t_ref[0] - 0.003 * (k + 1)] * h.B for k in range(K)]
            e0.record()
            if name == "fused":
                h.cache.update_forecast_multi(h.feats[j & 1], t_ref, targets, outs)
            else:
                h.cache.update(h.feats[j & 1], t_ref)
                h.cache.commit_step()
                h.cache.forecast_multi(targets, outs)
            e1.record()
            torch.cuda.synchronize(dev)
            if r >= 3:
                total += e0.elapsed_time(e1)
        res[name + "_ms"] = total / reps
    del outs
    torch.cuda.empty_cache()
    gbs = nbytes / (res["fused_ms"] * 1e-3) / 1e9
    return dict(res, targets=K, algorithmic_bytes=nbytes, gbs=gbs, frac_of_measured_peak=gbs / peak,
                bytes_of_the_two_launches=two_bytes, speedup_vs_two_launches=res["two_launches_ms"] / res["fused_ms"])


def time_update_per_entry(h: Harness, reps: int = 5):
    """A model hands over one block output at a time: the same reference step as one launch per entry."""
    w, dev = h.w, h.device
    ne = len(w.entries)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    total = 0.0
    for r in range(reps + 1):
        j = h.j
        h.j += 1
        t_ref, _ = h.times_for(j)
        e0.record()
        for e in range(ne):
            one = [None] * ne
            one[e] = h.feats[j & 1][e]
            h.cache.update(one, t_ref)
        h.cache.commit_step()
        e1.record()
        torch.cuda.synchronize(dev)
        if r > 0:
            total += e0.elapsed_time(e1)
    ms = total / reps
    nbytes = algorithmic_bytes(w, w.max_order)["update"]
    return {"launches": ne, "ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9}


def time_forecast_sum(h: Harness, peak: float, reps: int = 20):
    """base + sum of the forecasts of the largest group of equally shaped entries (all 56 block outputs
    of the DiT shape, the 38 single blocks of the FLUX shape, ...) in one pass, in place on a residual
    buffer: E (order + 1) + 2 words per element."""
    w, dev = h.w, h.device
    groups = {}
    for e, shape in enumerate(w.entries):
        groups.setdefault(shape, []).append(e)
    shape, ids = max(groups.items(), key=lambda kv: len(kv[1]) * kv[0][0] * kv[0][1])
    resid = torch.zeros(h.B, shape[0], shape[1], dtype=w.torch_dtype, device=dev)
    t = [h.t_base - 0.02 * (h.j + 1) - 0.01] * h.B
    for _ in range(3):
        h.cache.forecast_sum(ids, t, resid, resid, h.active)
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        resid.zero_()
        h.cache.forecast_sum(ids, t, resid, resid, h.active)
    e1.record()
    torch.cuda.synchronize(dev)
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for _ in range(reps):
        resid.zero_()
    e3.record()
    torch.cuda.synchronize(dev)
    ms = (e0.elapsed_time(e1) - e2.elapsed_time(e3)) / reps
    n = h.B * shape[0] * shape[1]
    nbytes = (len(ids) * (w.max_order + 1) + 2) * w.elem_bytes * n
    separate = len(ids) * (w.max_order + 2) * w.elem_bytes * n
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"entries": len(ids), "shape": list(shape), "ms": ms, "algorithmic_bytes": nbytes, "gbs": gbs,
            "frac_of_measured_peak": gbs / peak, "bytes_of_separate_forecasts": separate,
            "traffic_saved_vs_separate": 1.0 - nbytes / separate}


def time_draft_models(w: W.Workload, device: str, path: int, reps: int = 10):
    """The other draft models of the ablation on the same tables (Newton-form divided differences, the
    Adams-Bashforth predictor): they differ from Eq. 2-3 in host-computed scalars only, so the kernels and
    their times must be the same. Device time of a reference step and of a forecast per basis."""
    from paper_2509_11628_b200 import binding as S
    dev = torch.device(device)
    ne = len(w.entries)
    src = W.FeatureSource(w, device)
    feats = [[src.feature(e, k, [w.times[k]] * w.batch) for e in range(ne)] for k in range(2)]
    outs = [torch.empty(w.batch, n, d, dtype=w.torch_dtype, device=dev) for n, d in w.entries]
    ab = algorithmic_bytes(w, w.max_order, pred_from_verify=False)
    res = {}
    for basis, name in ((S.SPECA_BASIS_TAYLOR, "taylor_eq2_3"), (S.SPECA_BASIS_NEWTON, "newton"),
                        (S.SPECA_BASIS_ADAMS_BASHFORTH, "adams_bashforth")):
        cache = S.SpecaCache(w.entries, w.batch, w.max_order, w.dtype, device, basis=basis, path=path)
        t = 1.0
        for k in range(w.max_order + 2):
            t -= 0.02
            cache.update(feats[k & 1], [t] * w.batch)
            cache.commit_step()
        torch.cuda.synchronize(dev)
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        upd = fc = 0.0
        for r in range(reps):
            t -= 0.02
            e0.record()
            cache.update(feats[r & 1], [t] * w.batch)
            cache.commit_step()
            e1.record()
            cache.forecast([t - 0.01] * w.batch, outs)
            e2.record()
            torch.cuda.synchronize(dev)
            upd += e0.elapsed_time(e1)
            fc += e1.elapsed_time(e2)
        res[name] = {"update_ms": upd / reps, "update_gbs": ab["update"] / (upd / reps * 1e-3) / 1e9,
                     "forecast_ms": fc / reps, "forecast_gbs": ab["forecast"] / (fc / reps * 1e-3) / 1e9}
        cache.close()
        del cache
        torch.cuda.empty_cache()
    return res


def time_metrics(h: Harness, reps: int = 20):
    """Device time of the fused verification with each error metric (same traffic: order + 2 words per
    element of the verification entry)."""
    w, dev = h.w, h.device
    names = {0: "l2", 1: "l1", 2: "linf", 3: "cosine"}
    t = [h.t_base - 0.02 * (h.j + 1) - 0.01] * h.B
    tau = [0.1] * h.B
    nbytes = (w.max_order + 2) * w.elem_bytes * w.batch * w.entry_elems(w.vidx)
    out = {}
    for metric, name in names.items():
        for _ in range(3):
            h.cache.verify(h.fresh[0], t, tau, h.err, h.accept, h.active, metric=metric)
        torch.cuda.synchronize(dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            h.cache.verify(h.fresh[0], t, tau, h.err, h.accept, h.active, metric=metric)
        e1.record()
        torch.cuda.synchronize(dev)
        ms = e0.elapsed_time(e1) / reps
        out[name] = {"ms": ms, "gbs": nbytes / (ms * 1e-3) / 1e9, "err": [round(float(x), 6) for x in h.err.cpu().tolist()]}
    return out


def _slab_layout(sizes, align=256):
    """Offsets of consecutive byte ranges, each starting on an `align`-byte boundary; (offsets, total)."""
    offs, off = [], 0
    for s in sizes:
        offs.append(off)
        off = (off + s + align - 1) // align * align
    return offs, off


def time_end_to_end(h: Harness, steps: int, warmup: int):
    """Same step, but every step's inputs start in pinned host memory and its results end there.
    A step's inputs (every entry's feature and the verification feature) sit in ONE pinned slab and
    its results (every forecast, err, accept, next mask) in another, so each direction is a single
    large copy per step. The three legs of a step -- host-to-device copy, the library calls,
    device-to-host copy -- run on three streams with two sets of device buffers, so the copy-in of
    step k+1 and the copy-out of step k-1 overlap step k (PCIe is full duplex). Time is the host's
    wall clock from the first enqueue to the moment every result is in host memory."""
    w, dev = h.w, h.device
    eb = w.elem_bytes
    ne = len(w.entries)
    in_sizes = [h.B * n * d * eb for n, d in w.entries] + [h.B * w.entry_elems(w.vidx) * eb]
    in_offs, in_total = _slab_layout(in_sizes)
    out_sizes = [h.B * n * d * eb for n, d in w.entries] + [h.B * 4, h.B, h.B]
    out_offs, out_total = _slab_layout(out_sizes)

    def views(slab, offs, sizes, shapes):
        return [slab[o: o + s].view(w.torch_dtype).view(shape) for o, s, shape in zip(offs, sizes, shapes)]

    shapes_in = [(h.B, n, d) for n, d in w.entries] + [(h.B,) + tuple(w.entries[w.vidx])]
    shapes_out = [(h.B, n, d) for n, d in w.entries]
    host_in = [torch.empty(in_total, dtype=torch.uint8).pin_memory() for _ in range(2)]
    for p in range(2):
        for v, src in zip(views(host_in[p], in_offs, in_sizes, shapes_in), h.feats[p] + [h.fresh[p]]):
            v.copy_(src)
    host_out = [torch.empty(out_total, dtype=torch.uint8).pin_memory() for _ in range(2)]
    dev_in = [torch.empty(in_total, dtype=torch.uint8, device=dev) for _ in range(2)]
    dev_out = [torch.empty(out_total, dtype=torch.uint8, device=dev) for _ in range(2)]
    dev_in_views = [views(s, in_offs, in_sizes, shapes_in) for s in dev_in]
    dev_out_views = [views(s, out_offs[:ne], out_sizes[:ne], shapes_out) for s in dev_out]
    h2d = sum(in_sizes)
    d2h = sum(out_sizes)
    main = torch.cuda.current_stream(dev)
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in, ev_done, ev_out = {}, {}, {}

    def one(k):
        p = k & 1
        with torch.cuda.stream(s_in):
            if k - 2 in ev_done:
                s_in.wait_event(ev_done[k - 2])      # the step that last read this buffer set has run
            dev_in[p].copy_(host_in[p], non_blocking=True)          # one copy: the step's whole input
            ev_in[k] = torch.cuda.Event()
            ev_in[k].record(s_in)
        main.wait_event(ev_in[k])
        if k - 2 in ev_out:
            main.wait_event(ev_out[k - 2])           # the previous results in this output set are on the host
        h.step(feats=dev_in_views[p][:ne], fresh=dev_in_views[p][ne], outs=dev_out_views[p])
        tail = dev_out[p]
        tail[out_offs[ne]: out_offs[ne] + 4 * h.B].copy_(h.err.view(torch.uint8))
        tail[out_offs[ne + 1]: out_offs[ne + 1] + h.B].copy_(h.accept)
        tail[out_offs[ne + 2]: out_offs[ne + 2] + h.B].copy_(h.active)
        ev_done[k] = torch.cuda.Event()
        ev_done[k].record(main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[k])
            host_out[p].copy_(dev_out[p], non_blocking=True)        # one copy: the step's whole result
            ev_out[k] = torch.cuda.Event()
            ev_out[k].record(s_out)
        for old in (k - 3,):
            ev_in.pop(old, None), ev_done.pop(old, None), ev_out.pop(old, None)

    for k in range(warmup):
        one(k)
    torch.cuda.synchronize(dev)
    ev_in.clear(), ev_done.clear(), ev_out.clear()
    D.barrier()
    wall0 = time.perf_counter()
    for k in range(steps):
        one(k)
    torch.cuda.synchronize(dev)
    wall = (time.perf_counter() - wall0) * 1e3
    D.barrier()
    # one direction alone, for the PCIe rate each copy reaches when the link is not shared
    e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
    e0.record()
    dev_in[0].copy_(host_in[0], non_blocking=True)
    e1.record()
    host_out[0].copy_(dev_out[0], non_blocking=True)
    e2.record()
    torch.cuda.synchronize(dev)
    alone = {"h2d_gbs_alone": h2d / (e0.elapsed_time(e1) * 1e-3) / 1e9, "d2h_gbs_alone": d2h / (e1.elapsed_time(e2) * 1e-3) / 1e9}
    del host_in, host_out, dev_in, dev_out
    torch.cuda.empty_cache()
    return wall / steps, h2d, d2h, alone


def adaptive_sweep(device: str, peak: float, path: int, orders=(1, 2, 3), horizon: int = 6):
    """FLUX-shaped batch of 8 samples with different noise levels: after max_order + 1 reference
    steps, k = 1..horizon speculative steps run from the same table; samples whose verification
    fails drop out of later forecasts (sequential validation). Per (order, k): samples forecast,
    their accept flags, device times and GB/s over the bytes of the samples still active."""
    from paper_2509_11628_b200 import binding as S
    out = {}
    dev = torch.device(device)
    for m in orders:
        w = W.flux_adaptive(max_order=m, batch=8)
        B, ne = w.batch, len(w.entries)
        src = W.FeatureSource(w, device)
        cache = S.SpecaCache(w.entries, B, m, w.dtype, device, path=path)
        for step in range(m + 1):
            t = [w.times[step]] * B
            for e in range(ne):
                one = [None] * ne
                one[e] = src.feature(e, step, t)
                cache.update(one, t)
            cache.commit_step()
        outs = [torch.empty(B, n, d, dtype=w.torch_dtype, device=dev) for n, d in w.entries]
        err = torch.zeros(B, dtype=torch.float32, device=dev)
        acc = torch.zeros(B, dtype=torch.uint8, device=dev)
        active = torch.ones(B, dtype=torch.uint8, device=dev)
        spec = torch.zeros(B, dtype=torch.int32, device=dev)
        rows = []
        for k in range(1, horizon + 1):
            step = m + k
            t = [w.times[step]] * B
            tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
            fresh = src.feature(w.vidx, step, t)
            act_in = active.cpu().tolist()
            n_act = sum(act_in)
            if n_act == 0:
                rows.append({"k": k, "active": 0})
                continue

            def timed(fn, reps=5):
                ts = []
                for _ in range(reps):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    fn()
                    e1.record()
                    torch.cuda.synchronize(dev)
                    ts.append(e0.elapsed_time(e1))
                return sorted(ts)[len(ts) // 2]

            f_ms = timed(lambda: cache.forecast(t, outs, active))
            v_ms = timed(lambda: cache.verify(fresh, t, tau, err, acc, active))
            cache.select_adaptive(acc, horizon, 1, spec, active)
            torch.cuda.synchronize(dev)
            per_sample = sum(n * d for n, d in w.entries)
            f_bytes = (m + 2) * w.elem_bytes * per_sample * n_act
            v_bytes = (m + 2) * w.elem_bytes * w.entry_elems(w.vidx) * n_act
            gbs = (f_bytes + v_bytes) / ((f_ms + v_ms) * 1e-3) / 1e9
            rows.append({"k": k, "active": n_act, "active_mask": act_in,
                         "accept": [int(a) if act_in[i] else None for i, a in enumerate(acc.cpu().tolist())],
                         "err": [round(float(x), 5) if act_in[i] else None for i, x in enumerate(err.cpu().tolist())],
                         "tau": round(tau[0], 5), "forecast_ms": f_ms, "verify_ms": v_ms,
                         "forecast_verify_gbs": gbs, "frac_of_measured_peak": gbs / peak,
                         "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS})
            del fresh
        out["order_%d" % m] = {"sigma": w.sigma, "cache_bytes": w.elems_per_order * (m + 1) * w.elem_bytes,
                               "steps": rows}
        cache.close()
        del cache, outs, src
        torch.cuda.empty_cache()
    return out


def sampler_run(device: str, path: int, name: str, layout: int = 0, horizon: int = 1):
    """The whole forecast-then-verify loop (50 sampler steps) over the library with the seeded feature
    generator standing in for the transformer: which steps each sample took in full, acceptance rate,
    speed-up by the paper's cost model next to Eq. 8, and the device time the cache path itself took.
    With `horizon` > 1 a reference step of the whole batch forecasts that many coming steps in its pass."""
    from paper_2509_11628_b200 import binding as S
    from paper_2509_11628_b200 import scheduler as SCH
    w = W.flux_adaptive(max_order=2, batch=8) if name == "flux_adaptive" else W.BY_NAME[name]()
    gamma = 1.0 / {"dit_xl2": 28, "flux": 57, "flux_adaptive": 57, "hunyuan_video": 60}[name]
    cache = S.SpecaCache(w.entries, w.batch, w.max_order, w.dtype, device, path=path, layout=layout)
    src = W.FeatureSource(w, device)

    class Model:
        def full(self, step, times, mask):
            return [src.feature(e, step, times) for e in range(len(w.entries))]

        def verify_feature(self, step, times):
            return src.feature(w.vidx, step, times)

    class Timed(SCH.SpecaCacheBackend):
        def __init__(self, cache):
            super().__init__(cache, horizon=horizon)
            self.spans = {"forecast": [], "verify+select": [], "update": []}

        def _timed(self, key, fn):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            out = fn()
            e1.record()
            self.spans[key].append((e0, e1))
            return out

        def forecast(self, t, t_later=()):
            return self._timed("forecast", lambda: SCH.SpecaCacheBackend.forecast(self, t, t_later))

        def verify_and_select(self, fresh, t, tau, period):
            return self._timed("verify+select", lambda: SCH.SpecaCacheBackend.verify_and_select(self, fresh, t, tau, period))

        def reference_step(self, feats, t, mask, t_next=None, t_later=()):
            return self._timed("update", lambda: SCH.SpecaCacheBackend.reference_step(self, feats, t, mask, t_next, t_later))

    be = Timed(cache)
    wall0 = time.perf_counter()
    tr = SCH.run_sampler(be, Model(), w.times, w.tau0, w.beta, w.period, w.warm_refs, gamma, total_steps=w.total_steps)
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    ms = {k: [a.elapsed_time(b_) for a, b_ in v] for k, v in be.spans.items()}
    lib_ms = sum(sum(v) for v in ms.values())
    res = {
        "workload": w.name, "horizon": horizon, "sampler_steps": len(w.times), "period": w.period, "warm_refs": w.warm_refs, "gamma": gamma,
        "sigma": w.sigma, "acceptance_rate": tr.acceptance_rate(), "speedup_cost_model": tr.speedup(),
        "speedup_eq8": tr.predicted_speedup(), "full_steps_histogram": tr.full_steps_histogram(),
        "per_sample": ["".join(row[b] for row in tr.steps) for b in range(w.batch)],
        "library_ms_total": lib_ms, "calls": {k: len(v) for k, v in ms.items()},
        "ms_mean": {k: (sum(v) / len(v) if v else None) for k, v in ms.items()},
        "sampler_steps_per_s_library_only": len(w.times) / (lib_ms * 1e-3) if lib_ms > 0 else None,
        "wall_s_with_standin_model": wall,
    }
    cache.close()
    del be, cache
    torch.cuda.empty_cache()
    return res


# ------------------------------------------------------------------------------------------------
# the CPU oracle timed on the same configuration (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def _host_array(x: torch.Tensor, B: int):
    import numpy as np
    x = x.detach().contiguous().cpu()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16).reshape(B, -1).copy()
    return x.numpy().reshape(B, -1).copy()


def oracle_entry_steps(w: W.Workload, src: W.FeatureSource, e: int, n_steps: int, t_base: float):
    """The CPU oracle, as it stands, on ONE entry of the workload with the workload's own seeded
    features: max_order + 1 warming reference steps (untimed), then `n_steps` whole steps -- update,
    commit, forecast, and for the verification entry Eq. 4, the accept rule and the selection -- at
    the reference / target times the GPU harness uses. Returns the seconds each step took."""
    from oracle import speca_oracle as O
    B, m = w.batch, w.max_order
    is_v = e == w.vidx
    cache = O.OracleCache([w.entry_elems(e)], B, m, w.dtype)
    for step in range(m + 1):
        t = [w.times[step]] * B
        cache.update([_host_array(src.feature(e, step, t), B)], t)
        cache.commit_step()
    step0 = m + 1
    feats = [_host_array(src.feature(e, step0 + k, [w.times[step0 + k]] * B), B) for k in range(2)]
    fresh = [_host_array(src.feature(e, step0 + 2 + k, [w.times[step0 + 2 + k]] * B), B) for k in range(2)] if is_v else None
    out = None
    secs = []
    for j in range(n_steps):
        t_ref = [t_base - 0.02 * (j + 1)] * B
        t_tgt = [t_ref[0] - 0.01] * B
        tau = [O.tau_schedule(w.tau0, w.beta, w.total_steps - (j % w.total_steps), w.total_steps)] * B
        t0 = time.perf_counter()
        cache.update([feats[j & 1]], t_ref)
        cache.commit_step()
        if is_v:
            _, acc, _ = cache.verify(fresh[j & 1], t_tgt, tau)      # the entry's forecast is part of this
            O.select_adaptive([max(int(a), 0) for a in acc], 1 << 30, 1, [0] * B, [1] * B)
        else:
            out = cache.forecast_entry(0, t_tgt, out=out)
        secs.append(time.perf_counter() - t0)
    return secs


def oracle_config_run(w: W.Workload, n_steps: int, budget_s: float, gen_device: str):
    """Times the oracle over the whole configuration, entry by entry (the entries are independent, so a
    step's time is the sum of its entries' times; only one entry's tables are in host memory at a
    time). If the whole configuration would not fit `budget_s` seconds of oracle work, every k-th entry
    (always with the verification entry) is the step's sample instead, and the result says so.
    Returns a dict with the per-step seconds, the algorithmic bytes those steps covered, the threads
    the oracle used and a description of the sample."""
    from oracle import speca_oracle as O
    src = W.FeatureSource(w, gen_device)
    ne = len(w.entries)
    t_base = w.times[w.max_order]
    per_elem = lambda e: ((2 * w.max_order + 2) + (w.max_order + (3 if e == w.vidx else 2))) * w.elem_bytes  # noqa: E731
    # calibrate on the smallest entry: seconds per element of one step
    e_small = min(range(ne), key=lambda e: w.entry_elems(e))
    cal = oracle_entry_steps(w, src, e_small, 2, t_base)
    rate = min(cal) / (w.batch * w.entry_elems(e_small))
    est = rate * w.elems_per_order * n_steps
    stride = 1 if est <= budget_s else int(-(-est // budget_s))
    chosen = sorted(set(list(range(0, ne, stride)) + [w.vidx]))
    secs = [0.0] * n_steps
    nbytes = 0
    for e in chosen:
        for j, s in enumerate(oracle_entry_steps(w, src, e, n_steps, t_base)):
            secs[j] += s
        nbytes += per_elem(e) * w.batch * w.entry_elems(e)
    if len(chosen) == ne:
        sample = "all %d entries of %s, every step: update+forecast+verify+select on the workload's seeded features" % (ne, w.name)
    else:
        sample = "%d of %d entries of %s (every %d-th and the verification entry), every step: update+forecast+verify+select" % (
            len(chosen), ne, w.name, stride)
    return {"secs": secs, "bytes_per_step": nbytes, "threads": O.threads(), "sample": sample, "entries": len(chosen)}


def oracle_one_thread_gbs(w: W.Workload, gen_device: str):
    """One step of the verification entry alone with the oracle held to one thread: GB/s."""
    from oracle import speca_oracle as O
    n = O.threads()
    O.set_threads(1)
    try:
        src = W.FeatureSource(w, gen_device)
        secs = oracle_entry_steps(w, src, w.vidx, 1, w.times[w.max_order])
    finally:
        O.set_threads(n)
    nbytes = ((2 * w.max_order + 2) + (w.max_order + 3)) * w.elem_bytes * w.batch * w.entry_elems(w.vidx)
    return nbytes / secs[0] / 1e9


def parity_on_verify_entry(w: W.Workload, device: str, path: int):
    """The same seeded features through the library and through the oracle, on the workload's
    verification entry alone (full size): norm-wise forecast difference, verification errors,
    decisions. Part of the CPU-baseline leg: the one place the benchmark runs the oracle."""
    import numpy as np
    from oracle import speca_oracle as O
    from paper_2509_11628_b200 import binding as S
    B, m = w.batch, w.max_order
    n_tok, dim = w.entries[w.vidx]
    one = W.Workload(name=w.name + "_verify_entry", index=w.index, entries=[(n_tok, dim)], batch=B, max_order=m,
                     dtype=w.dtype, times=w.times, poly_degree=w.poly_degree, sigma=w.sigma, outlier_frac=w.outlier_frac,
                     frame_tokens=w.frame_tokens, n_frames=w.n_frames, video_tokens=min(w.video_tokens, n_tok))
    src = W.FeatureSource(one, device)
    gpu = S.SpecaCache(one.entries, B, m, w.dtype, device, path=path)
    cpu = O.OracleCache([n_tok * dim], B, m, w.dtype)

    def f64(a):
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64) if a.dtype == np.uint16 else a.astype(np.float64)

    for step in range(m + 1):
        t = [w.times[step]] * B
        f = src.feature(0, step, t)
        gpu.update([f], t)
        gpu.commit_step()
        cpu.update([_host_array(f, B)], t)
        cpu.commit_step()
    step = m + 1
    t = [w.times[step]] * B
    tau = [0.1] * B
    fresh = src.feature(0, step, t)
    pred = torch.empty_like(fresh)
    err = torch.zeros(B, dtype=torch.float32, device=device)
    acc = torch.zeros(B, dtype=torch.uint8, device=device)
    gpu.verify(fresh, t, tau, err, acc, out_pred=pred)
    torch.cuda.synchronize()
    e_want, a_want, p_want = cpu.verify(_host_array(fresh, B), t, tau)
    g, o = f64(_host_array(pred, B)), f64(p_want)
    rel = [float(np.linalg.norm(g[b] - o[b]) / max(np.linalg.norm(o[b]), 1e-30)) for b in range(B)]
    e_got = [float(x) for x in err.cpu().tolist()]
    out = {"entry_elems": n_tok * dim, "samples": B,
           "forecast_norm_rel_diff_max": max(rel), "forecast_tolerance": 2e-3,
           "err_library": e_got, "err_oracle": [float(x) for x in e_want],
           "err_abs_diff_max": max(abs(a - b_) for a, b_ in zip(e_got, e_want)), "err_tolerance": 1e-4,
           "decisions_equal": [int(x) for x in acc.cpu().tolist()] == [int(x) for x in a_want]}
    gpu.close()
    return out


def generation_device() -> str:
    """Where the seeded features are drawn: the GPU when there is one (the same bits the library's
    arm sees), else the host."""
    return "cuda:0" if torch.cuda.is_available() else "cpu"


def run_reference(args, info: D.RankInfo):
    """--impl reference: the oracle timed on the host cores for the same metric, configuration and
    step (rank 0 alone; the other ranks leave at once)."""
    if not info.is_main:
        return
    w = make_workload(args.config)
    steps, warm = max(1, args.steps), max(0, args.warmup)
    res = oracle_config_run(w, steps + warm, args.oracle_budget_s, generation_device())
    timed = res["secs"][warm:]
    dt = sum(timed) / len(timed)
    gbs = res["bytes_per_step"] / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": _r(gbs, 4), "unit": "GB/s", "n_gpus": args.gpus,
        "steps": steps, "warmup": warm, "ms_per_step": _r(dt * 1e3, 3), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "value_covers": VALUE_COVERS, "config": workload_config(w),
        "cpu_baseline": {"value": _r(gbs, 4), "unit": "GB/s", "cores": res["threads"], "kind": "oracle",
                         "sample": res["sample"]},
        "e2e": {"value": _r(gbs, 4), "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line, separators=(",", ":")), flush=True)


def workload_config(w: W.Workload, layout: str = "tables"):
    return {
        "workload": "%s (config %d)" % (w.name, w.index),
        "entries": len(w.entries), "batch": w.batch, "order": w.max_order,
        "storage": "bf16" if w.dtype == W.BF16 else "f32", "layout": layout,
        "elems_per_order": w.elems_per_order,
        "l2": ("no flush: working set >> 126 MB L2" if w.elems_per_order * w.elem_bytes * (w.max_order + 1) > (1 << 30)
               else "no flush: small case, fits L2 (parity configuration, not an HBM figure)"),
        "parallelism": "one cache per GPU, no collective",
    }


def summarize(w, per_ms, total_ms, steps, n_gpus, peak, layout=0):
    ab = algorithmic_bytes(w, w.max_order, layout)
    step_bytes = ab["update"] + ab["forecast"] + ab["verify"]
    ms_step = total_ms / steps
    kernels = {}
    for k in ("update", "forecast", "verify", "select"):
        gbs = ab[k] / (per_ms[k] * 1e-3) / 1e9 if per_ms[k] > 0 else 0.0
        kernels[k] = {"ms": per_ms[k], "algorithmic_bytes": ab[k], "gbs": gbs, "frac_of_measured_peak": gbs / peak,
                      "frac_of_nominal_8TBs": gbs / NOMINAL_HBM_GBS}
    value = n_gpus * step_bytes / (ms_step * 1e-3) / 1e9
    spec_ms = per_ms["forecast"] + per_ms["verify"] + per_ms["select"]
    fv_gbs = (ab["forecast"] + ab["verify"]) / (spec_ms * 1e-3) / 1e9
    return value, ms_step, kernels, {"speculative_steps_per_s": 1e3 / spec_ms, "forecast_verify_gbs": fv_gbs,
                                     "forecast_verify_frac_of_nominal_8TBs": fv_gbs / NOMINAL_HBM_GBS,
                                     "forecast_verify_frac_of_measured_peak": fv_gbs / peak}


def time_history_layout(w, device, path, steps, info, peak, tables_ms_step, tables_kernels):
    """The same step on a cache that keeps the raw features of the last references instead of the
    difference tables (SPECA_LAYOUT_HISTORY): the reference step becomes one copy."""
    h = Harness(w, device, path=path, layout=1)
    total_ms, per_ms, _, _ = time_device_resident(h, steps, 3, info, False)
    value, ms_step, kernels, extra = summarize(w, per_ms, total_ms, steps, 1, peak, layout=1)
    h.close()
    del h
    torch.cuda.empty_cache()
    return {"ms_per_step": ms_step, "value": value, "unit": "GB/s", "kernels": kernels,
            "speculative_steps_per_s": extra["speculative_steps_per_s"],
            "update_ms_tables_layout": tables_kernels["update"]["ms"],
            "update_speedup_vs_tables_layout": tables_kernels["update"]["ms"] / kernels["update"]["ms"],
            "step_speedup_vs_tables_layout": tables_ms_step / ms_step,
            "note": "update moves 2 words per element instead of 2 * order + 2; forecast and verify move the same bytes"}


# ------------------------------------------------------------------------------------------------
# the one line
# ------------------------------------------------------------------------------------------------

def _r(x, digits=5):
    """A float to `digits` significant digits (keeps the line short); other values unchanged."""
    if isinstance(x, float):
        if x != x or x in (float("inf"), float("-inf")):
            return None
        return float("%.*g" % (digits, x))
    return x


def build_line(*, value, ms_per_step, n_gpus, steps, warmup, config, roofline, cpu_baseline, e2e, gpu_launches, clocks,
               kernels, forecast_verify_gbs, speculative_steps_per_s, also=None, detail_path=None, scaling="weak", fused=None):
    """The compact JSON object of the benchmark's last line, kept under MAX_LINE_BYTES: whatever does
    not fit belongs in the detail file. Raises only if the contract keys alone are too long."""
    line = {
        "metric": METRIC, "value": _r(value), "unit": "GB/s", "n_gpus": n_gpus, "steps": steps, "warmup": warmup,
        "ms_per_step": _r(ms_per_step), "higher_is_better": True, "scaling": scaling, "vs_baseline": None,
        "dtype": "f32",  # the arithmetic type: every kernel computes in fp32 registers, whatever config.storage is
        "data": "synthetic", "value_covers": VALUE_COVERS, "config": config,
        "roofline": {k: _r(v) for k, v in roofline.items()} if roofline else None,
        "cpu_baseline": {k: _r(v, 4) for k, v in cpu_baseline.items()} if cpu_baseline else None,
        "e2e": {k: _r(v, 4) for k, v in e2e.items()} if e2e else None,
        "gpu_launches": gpu_launches, "clocks": clocks,
        "forecast_verify_gbs": _r(forecast_verify_gbs), "speculative_steps_per_s": _r(speculative_steps_per_s),
        "kernels_ms_gbs": {k: [_r(v["ms"], 4), _r(v["gbs"], 4)] for k, v in kernels.items() if k != "select"},
    }
    if fused:   # update + first forecast as one launch: [ms, GB/s over its own 2*order+3 words, ms of the two launches]
        line["fused_update_forecast_ms_gbs_vs_ms"] = [_r(fused["ms"], 4), _r(fused["gbs"], 4), _r(fused["ms_of_the_two_launches"], 4)]
    if also:
        line["also_value_fv_gbs_steps_per_s"] = {k: [_r(x, 4) for x in v] for k, v in also.items()}
    if detail_path:
        line["detail"] = detail_path
    # the contract keys always go out; the extras are dropped, last first, if the line would grow too long
    for extra in (None, "also_value_fv_gbs_steps_per_s", "fused_update_forecast_ms_gbs_vs_ms", "kernels_ms_gbs", "detail",
                  "value_covers"):
        if extra is not None:
            line.pop(extra, None)
        text = json.dumps(line, separators=(",", ":"))
        if len(text) < MAX_LINE_BYTES:
            return text
    raise ValueError("benchmark line is %d bytes; the limit is %d" % (len(text), MAX_LINE_BYTES))


def write_detail(path, detail):
    """Best effort: the detail file is a by-product, the line is the result."""
    if not path:
        return None
    try:
        d = os.path.dirname(os.path.abspath(path))
        os.makedirs(d, exist_ok=True)
        with open(path, "w") as f:
            json.dump(detail, f, indent=1)
        return path
    except Exception:
        return None


# ------------------------------------------------------------------------------------------------
# one process per GPU
# ------------------------------------------------------------------------------------------------

def free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(n: int, argv, extra_env=None, timeout_s: float = 3600.0) -> int:
    """Starts `n` copies of `argv` (a full command line), one per rank, with the process-group
    environment torchrun would give them (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR, MASTER_PORT),
    and waits for all of them. Rank 0 inherits stdout, so its one line is the job's line; the other
    ranks' stdout is dropped. If a rank fails the others are stopped (by their own PIDs). Returns
    the largest exit status."""
    port = free_port()
    procs = []
    for r in range(n):
        env = dict(os.environ)
        env.update(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        env.update(extra_env or {})
        procs.append(subprocess.Popen(list(argv), env=env, stdout=None if r == 0 else subprocess.DEVNULL))
    deadline = time.time() + timeout_s
    rc = 0
    live = list(procs)
    while live:
        for p in list(live):
            code = p.poll()
            if code is None:
                continue
            live.remove(p)
            if code != 0:
                rc = max(rc, abs(code) or 1)
        if (rc != 0 or time.time() > deadline) and live:
            for p in live:
                p.terminate()
            for p in live:
                try:
                    p.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    p.kill()
            rc = rc or 124
            break
        time.sleep(0.05)
    return rc


def job_value(step_bytes_per_rank: float, world: int, slowest_ms_per_step: float) -> float:
    """Whole-job GB/s: every rank moves its own step's bytes; the job is as fast as its slowest rank."""
    return world * step_bytes_per_rank / (slowest_ms_per_step * 1e-3) / 1e9


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="flux", choices=["tiny", "dit_xl2", "flux", "hunyuan_video", "flux_b8"])
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--also", default="dit_xl2,hunyuan_video",
                    help="comma list of further configs measured device-resident (three numbers each in the line)")
    ap.add_argument("--path", default="auto", choices=["auto", "direct", "bulk", "wide"],
                    help="kernel variant (speca_path_t); results are identical, only speed differs")
    ap.add_argument("--layout", default="tables", choices=["tables", "history"],
                    help="what the cache keeps: the paper's difference tables (default) or the raw features of "
                         "the last references (speca_layout_t)")
    ap.add_argument("--separate-select", action="store_true",
                    help="five launches per step (update, activate, forecast, verify, select) instead of the three fused ones")
    ap.add_argument("--detail", default="bench_detail.json",
                    help="JSON file for everything that does not belong in the last line ('' = none)")
    ap.add_argument("--full", action="store_true",
                    help="also run the sweeps reported only in the detail file: multi-horizon and summed forecasts, "
                         "other metrics and draft models, the raw-feature layout, the B=8 adaptive sweep, the sampler loop")
    ap.add_argument("--oracle-budget-s", type=float, default=150.0,
                    help="--impl reference: seconds of oracle work the run may take; above it a step samples every k-th entry")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-adaptive", action="store_true", help="accepted for older command lines; the sweep needs --full")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args(argv)
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup

    if args.impl == "reference":
        run_reference(args, D.rank_info_from_env())
        return 0

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher gave us a process group: start one rank per GPU ourselves
        if not torch.cuda.is_available() or torch.cuda.device_count() < args.gpus:
            raise SystemExit("bench.py --gpus %d: only %d CUDA devices visible" % (
                args.gpus, torch.cuda.device_count() if torch.cuda.is_available() else 0))
        return spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + list(sys.argv[1:] if argv is None else argv))

    info = D.rank_info_from_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    from paper_2509_11628_b200 import build as _b
    if info.local_rank == 0:
        _b.build()
    torch.cuda.set_device(info.local_rank)
    device = "cuda:%d" % info.local_rank
    info = D.init("nccl")
    D.barrier()
    peak, peak_src = measured_peak()
    solo = info.world == 1

    w = make_workload(args.config)
    path = {"auto": 0, "direct": 1, "bulk": 2, "wide": 3}[args.path]
    layout = 1 if args.layout == "history" else 0
    h = Harness(w, device, seed_offset=17 * info.rank, path=path, fused_select=not args.separate_select, layout=layout)
    total_ms, per_ms, launches, clocks = time_device_resident(h, args.steps, args.warmup, info, True)
    total_ms = D.max_over_ranks(total_ms, device)
    value, ms_step, kernels, extra = summarize(w, per_ms, total_ms, args.steps, info.world, peak, layout=layout)
    detail = {"config": workload_config(w, args.layout), "kernels": kernels, **extra,
              "frac_of_measured_peak": value / info.world / peak, "frac_of_nominal_8TBs": value / info.world / NOMINAL_HBM_GBS,
              "select": "its own launches (speca_select_adaptive, speca_activate)" if args.separate_select else
                        "inside the verify launch (speca_verify_select); re-arming inside the update launch",
              "paper_context": {"end_to_end_speedups": {"flux_h800": 6.34, "dit_xl2_a800": 7.3, "hunyuan_video_h800": 6.1},
                                "verification_overhead": "1.67%-3.5% of a full forward pass",
                                "note": "other hardware, whole-model numbers; context only"}}

    tables = solo and layout == 0      # these calls exist for the table layout only
    fused = None
    if path in (0, 3):
        fused = time_fused_reference_step(h, peak)
        fused["ms_of_the_two_launches"] = per_ms["update"] + per_ms["forecast"]
        fused["speedup_vs_two_launches"] = fused["ms_of_the_two_launches"] / fused["ms"]
        detail["fused_reference_step"] = fused
    if args.full and solo:
        detail["verify_metrics"] = time_metrics(h)
    if args.full and tables:
        detail["multi_horizon"] = time_multi_horizon(h, peak, per_ms["forecast"])
        if path in (0, 3):
            detail["fused_reference_step_4_targets"] = time_fused_reference_step_multi(h, peak)
        try:
            detail["speculative_run_as_cuda_graph"] = time_graph_replay(h)
        except Exception as exc:  # report, do not hide
            detail["speculative_run_as_cuda_graph"] = {"error": repr(exc)}
        detail["update_one_launch_per_entry"] = time_update_per_entry(h)
        detail["forecast_sum"] = time_forecast_sum(h, peak)

    e2e = None
    if not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 24))
        e2e_ms, h2d, d2h, alone = time_end_to_end(h, e2e_steps, 3)
        e2e_ms = D.max_over_ranks(e2e_ms, device)
        ab = algorithmic_bytes(w, w.max_order, layout)
        e2e = {"value": job_value(ab["update"] + ab["forecast"] + ab["verify"], info.world, e2e_ms),
               "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
               "h2d_gbs": h2d / (e2e_ms * 1e-3) / 1e9, "d2h_gbs": d2h / (e2e_ms * 1e-3) / 1e9,
               "pcie_gbs_one_direction_alone": [_r(alone["h2d_gbs_alone"], 3), _r(alone["d2h_gbs_alone"], 3)]}
        detail["e2e"] = dict(e2e, steps=e2e_steps, **alone,
                             note="one pinned slab per direction per step (features + verification feature in, forecasts + "
                                  "decisions out), one copy each; copy-in, library calls and copy-out pipelined on three "
                                  "streams; host wall clock; *_gbs = bytes / step time with both directions busy")
    h.close()
    del h
    torch.cuda.empty_cache()

    if args.full and tables:
        try:
            detail["draft_models"] = time_draft_models(w, device, path)
        except Exception as exc:  # report, do not hide
            detail["draft_models"] = {"error": repr(exc)}
        if path in (0, 3):
            try:
                detail["history_layout"] = time_history_layout(w, device, path, min(args.steps, 100), info, peak, ms_step, kernels)
            except Exception as exc:  # report, do not hide
                detail["history_layout"] = {"error": repr(exc)}

    also, per_config = {}, {}
    if tables:
        for name in [n for n in args.also.split(",") if n and n != args.config]:
            try:
                w2 = make_workload(name)
                h2 = Harness(w2, device, path=path, fused_select=not args.separate_select)
                k2 = max(5, min(args.steps, 2000 // max(1, len(w2.entries)) * 4))
                t2, p2, _, _ = time_device_resident(h2, k2, 3, info, False)
                v2, ms2, kern2, ex2 = summarize(w2, p2, t2, k2, 1, peak)
                per_config[name] = {"value": v2, "unit": "GB/s", "ms_per_step": ms2, "steps": k2,
                                    "config": workload_config(w2), "kernels": kern2, **ex2}
                if path in (0, 3):
                    per_config[name]["fused_reference_step"] = time_fused_reference_step(h2, peak)
                    per_config[name]["fused_reference_step"]["ms_of_the_two_launches"] = p2["update"] + p2["forecast"]
                also[name] = [v2, ex2["forecast_verify_gbs"], ex2["speculative_steps_per_s"]]
                if args.full:
                    try:
                        per_config[name]["speculative_run_as_cuda_graph"] = time_graph_replay(h2)
                    except Exception as exc:  # report, do not hide
                        per_config[name]["speculative_run_as_cuda_graph"] = {"error": repr(exc)}
                    per_config[name].update(multi_horizon=time_multi_horizon(h2, peak, p2["forecast"]),
                                            update_one_launch_per_entry=time_update_per_entry(h2),
                                            forecast_sum=time_forecast_sum(h2, peak))
                h2.close()
                del h2
                torch.cuda.empty_cache()
                if args.full and path in (0, 3):
                    per_config[name]["history_layout"] = time_history_layout(w2, device, path, k2, info, peak, ms2, kern2)
            except Exception as exc:  # report, do not hide
                per_config[name] = {"error": repr(exc)}
    detail["per_config"] = per_config

    if args.full and solo and not args.no_adaptive:
        try:
            detail["adaptive"] = adaptive_sweep(device, peak, path)
        except Exception as exc:  # report, do not hide
            detail["adaptive"] = {"error": repr(exc)}
        detail["sampler"] = {}
        for name in ("dit_xl2", "flux", "flux_adaptive"):
            try:
                detail["sampler"][name] = sampler_run(device, path, name)
                if path in (0, 3) and name != "flux_adaptive":
                    # batches whose samples stay in step: a reference step hands over the whole run that follows
                    far = sampler_run(device, path, name, horizon=W.BY_NAME[name]().period)
                    assert far["per_sample"] == detail["sampler"][name]["per_sample"]     # same decisions
                    detail["sampler"][name]["with_horizon"] = {k: far[k] for k in (
                        "horizon", "library_ms_total", "calls", "ms_mean", "sampler_steps_per_s_library_only")}
                if path in (0, 3):   # the same run on a cache that keeps raw features: cache-path time only
                    hist = sampler_run(device, path, name, layout=1)
                    detail["sampler"][name]["history_layout"] = {k: hist[k] for k in (
                        "acceptance_rate", "library_ms_total", "ms_mean", "sampler_steps_per_s_library_only")}
            except Exception as exc:  # report, do not hide
                detail["sampler"][name] = {"error": repr(exc)}

    if not info.is_main:
        D.shutdown()
        return 0

    dominant = max(("update", "forecast", "verify"), key=lambda k: per_ms[k])
    dom = kernels[dominant]
    per_elem = None if (layout == 1 and dominant == "update") else NCU_DRAM_BYTES_PER_ELEM.get(dominant)
    n_dom = w.batch * w.entry_elems(w.vidx) if dominant == "verify" else w.elems_per_order
    if dominant == "forecast":
        n_dom -= w.batch * w.entry_elems(w.vidx)
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": dom["gbs"], "peak": peak, "unit": "GB/s",
                "frac": dom["gbs"] / peak, "peak_source": peak_src,
                "traffic": (per_elem * n_dom) if per_elem is not None else None,
                "traffic_source": TRAFFIC_SOURCE if per_elem is not None else "none: kernel changed since the last capture",
                "algorithmic_bytes_per_launch": dom["algorithmic_bytes"],
                "frac_of_nominal_8TBs": dom["gbs"] / NOMINAL_HBM_GBS}

    cpu_baseline = None
    if not args.no_cpu_baseline and solo:      # timed on rank 0 of a one-GPU run only
        res = oracle_config_run(w, 1, 60.0, device)
        dt = res["secs"][0]
        cpu_baseline = {"value": res["bytes_per_step"] / dt / 1e9, "unit": "GB/s", "cores": res["threads"], "kind": "oracle",
                        "sample": "1 step, " + res["sample"].replace(", every step", ""), "s_per_step": dt,
                        "value_1_thread_verify_entry_only": oracle_one_thread_gbs(w, device)}
        try:
            detail["parity_on_verify_entry"] = parity_on_verify_entry(w, device, path)
        except Exception as exc:  # report, do not hide
            detail["parity_on_verify_entry"] = {"error": repr(exc)}
        detail["cpu_baseline"] = cpu_baseline

    detail_path = write_detail(args.detail, dict(detail, roofline=roofline, clocks=clocks, value=value, ms_per_step=ms_step,
                                                 gpu_launches=launches, n_gpus=info.world, steps=args.steps, warmup=args.warmup))
    clocks_line = {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")} if clocks else None
    print(build_line(value=value, ms_per_step=ms_step, n_gpus=info.world, steps=args.steps, warmup=args.warmup,
                     config=workload_config(w, args.layout), roofline=roofline, cpu_baseline=cpu_baseline, e2e=e2e,
                     gpu_launches=launches, clocks=clocks_line, kernels=kernels,
                     forecast_verify_gbs=extra["forecast_verify_gbs"],
                     speculative_steps_per_s=extra["speculative_steps_per_s"], also=also, detail_path=detail_path,
                     fused=fused), flush=True)
    D.shutdown()
    return 0


if __name__ == "__main__":
    sys.exit(main())
