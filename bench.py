#!/usr/bin/env python
"""Benchmark of the SpeCa feature-cache hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic input: a reference-step
cache update of every entry (Eq. 3), a forecast of every entry (Eq. 2), the fused
forecast+verification of the verification entry (Eq. 4 and the accept rule) and the per-sample
selection. The headline value is the algorithmic bytes of a step divided by its device time
(GB/s), with the inputs already resident in HBM; ``e2e`` repeats the measurement with the step's
inputs in pinned host memory and its outputs copied back.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config flux] [--impl reference]

Prints exactly one JSON line (rank 0).
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

import torch  # noqa: E402

from paper_2509_11628_b200 import dist as D  # noqa: E402
from paper_2509_11628_b200 import workloads as W  # noqa: E402

METRIC = "forecast+verify GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM bytes per cached element per launch: (dram__bytes_read.sum + dram__bytes_write.sum) / elements,
# from the one-pass ncu capture of this benchmark's default workload at full size (FLUX-shaped cache,
# order 2, bf16; profiles/dram_traffic_flux_full_size.md). Other workloads scale by the elements a
# launch covers. Set an entry to None when its kernel changes until the counters have been taken again.
NCU_DRAM_BYTES_PER_ELEM_HISTORY_UPDATE = 3.956   # profiles/history_layout_flux_full_size.md
NCU_DRAM_BYTES_PER_ELEM = {"update": 12.000, "forecast": 8.052, "verify": 8.147}


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def make_workload(name: str) -> W.Workload:
    if name == "flux_b8":
        return W.flux_adaptive(max_order=2, batch=8)
    return W.BY_NAME[name]()


def algorithmic_bytes(w: W.Workload, order: int, layout: int = 0):
    """Bytes a step must move per kernel, from the per-element figures: update reads the feature
    and `order` old planes and writes order+1 planes (a cache that keeps raw features, layout 1, reads
    the feature and writes one plane); forecast reads order+1 planes and writes one; verify reads
    order+1 planes and the fresh feature."""
    eb = w.elem_bytes
    n_all = w.elems_per_order
    n_ver = w.batch * w.entry_elems(w.vidx)
    return {
        "update": (2 if layout == 1 else 2 * order + 2) * eb * n_all,
        "forecast": (order + 2) * eb * n_all,
        "verify": (order + 2) * eb * n_ver,
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
        self.fused_select = fused_select
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
        self.ones = [1] * self.B
        self.j = 0
        self.t_base = w.times[self.m]
        torch.cuda.synchronize(self.device)

    def times_for(self, j):
        gap = 0.02
        t_ref = self.t_base - gap * (j + 1)
        return [t_ref] * self.B, [t_ref - 0.5 * gap] * self.B

    def step(self, events=None, feats=None, fresh=None):
        """update -> commit -> forecast -> verify -> select on the current stream: three launches
        (speca_cache_update_activate, speca_forecast, speca_verify_select), or five with
        fused_select=False (update, activate, forecast, verify, select)."""
        S, c, w = self.S, self.cache, self.w
        j = self.j
        self.j += 1
        t_ref, t_tgt = self.times_for(j)
        feats = feats if feats is not None else self.feats[j & 1]
        fresh = fresh if fresh is not None else self.fresh[j & 1]
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
        c.forecast(t_tgt, self.outs, self.active)
        if events is not None:
            events[3].record()
        if self.fused_select:
            c.verify_select(fresh, t_tgt, tau, self.err, self.accept, self.active, self.active_next, 1 << 30, 1, self.spec,
                            self.idx, self.n_active)
            self.active, self.active_next = self.active_next, self.active
            if events is not None:
                events[4].record()
        else:
            c.verify(fresh, t_tgt, tau, self.err, self.accept, self.active)
            if events is not None:
                events[4].record()
            c.select_adaptive(self.accept, 1 << 30, 1, self.spec, self.active, self.idx, self.n_active)
        if events is not None:
            events[5].record()

    def close(self):
        self.cache.close()


def time_device_resident(h: Harness, steps: int, warmup: int, info: D.RankInfo, sample_clocks: bool):
    dev = h.device
    for _ in range(warmup):
        h.step()
    torch.cuda.synchronize(dev)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(6)] for _ in range(steps)]
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
        h.step(ev[k])
    t_end.record()
    torch.cuda.synchronize(dev)
    D.barrier()
    if sampler:
        sampler.stop_flag = True
        sampler.join(timeout=2.0)
    total_ms = t_start.elapsed_time(t_end)
    per = {"update": 0.0, "forecast": 0.0, "verify": 0.0, "select": 0.0}
    for k in range(steps):
        per["update"] += ev[k][0].elapsed_time(ev[k][1])
        per["forecast"] += ev[k][2].elapsed_time(ev[k][3])
        per["verify"] += ev[k][3].elapsed_time(ev[k][4])
        per["select"] += ev[k][1].elapsed_time(ev[k][2]) + ev[k][4].elapsed_time(ev[k][5])  # activate + select
    per = {k: v / steps for k, v in per.items()}
    return total_ms, per, h.cache.launches - launches0, (sampler.summary() if sampler else None)


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
    ab = algorithmic_bytes(w, w.max_order)
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


def time_end_to_end(h: Harness, steps: int, warmup: int):
    """Same step, but every step's inputs start in pinned host memory and its results end there.
    The three legs of a step -- host-to-device copy of the features, the library calls, device-to-host
    copy of forecasts and decisions -- run on three streams with two sets of device buffers, so the
    copy-in of step k+1 and the copy-out of step k-1 overlap step k (PCIe is full duplex). Time is the
    host's wall clock from the first enqueue to the moment every result is in host memory."""
    w, dev = h.w, h.device
    host_feats = [[f.cpu().pin_memory() for f in fs] for fs in h.feats]
    host_fresh = [f.cpu().pin_memory() for f in h.fresh]
    host_outs = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in h.outs]
    host_small = [torch.empty(h.B * 6, dtype=torch.uint8).pin_memory() for _ in range(2)]
    dev_feats = [[torch.empty_like(f) for f in h.feats[0]] for _ in range(2)]
    dev_fresh = [torch.empty_like(h.fresh[0]) for _ in range(2)]
    dev_outs = [h.outs, [torch.empty_like(o) for o in h.outs]]
    dev_small = [torch.empty(h.B * 6, dtype=torch.uint8, device=dev) for _ in range(2)]
    h2d = sum(f.numel() * f.element_size() for f in host_feats[0]) + host_fresh[0].numel() * host_fresh[0].element_size()
    d2h = sum(o.numel() * o.element_size() for o in host_outs) + h.B * (4 + 1 + 1)
    main = torch.cuda.current_stream(dev)
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in, ev_done, ev_out = {}, {}, {}

    def one(k):
        p = k & 1
        with torch.cuda.stream(s_in):
            if k - 2 in ev_done:
                s_in.wait_event(ev_done[k - 2])      # the step that last read this buffer set has run
            for dst, src in zip(dev_feats[p], host_feats[p]):
                dst.copy_(src, non_blocking=True)
            dev_fresh[p].copy_(host_fresh[p], non_blocking=True)
            ev_in[k] = torch.cuda.Event()
            ev_in[k].record(s_in)
        main.wait_event(ev_in[k])
        if k - 2 in ev_out:
            main.wait_event(ev_out[k - 2])           # the previous results in this output set are on the host
        saved, h.outs = h.outs, dev_outs[p]
        h.step(feats=dev_feats[p], fresh=dev_fresh[p])
        h.outs = saved
        dev_small[p][: 4 * h.B].copy_(h.err.view(torch.uint8))
        dev_small[p][4 * h.B: 5 * h.B].copy_(h.accept)
        dev_small[p][5 * h.B:].copy_(h.active)
        ev_done[k] = torch.cuda.Event()
        ev_done[k].record(main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[k])
            for dst, src in zip(host_outs, dev_outs[p]):
                dst.copy_(src, non_blocking=True)
            host_small[p].copy_(dev_small[p], non_blocking=True)
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
    return wall / steps, h2d, d2h


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


def sampler_run(device: str, path: int, name: str, layout: int = 0):
    """The whole forecast-then-verify loop (50 sampler steps) over the library with the seeded feature
    generator standing in for the transformer: which steps each sample took in full, acceptance rate,
    speed-up by the paper's cost model next to Eq. 8, and the device time the cache path itself took."""
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
            super().__init__(cache)
            self.spans = {"forecast": [], "verify+select": [], "update": []}

        def _timed(self, key, fn):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            out = fn()
            e1.record()
            self.spans[key].append((e0, e1))
            return out

        def forecast(self, t):
            return self._timed("forecast", lambda: SCH.SpecaCacheBackend.forecast(self, t))

        def verify_and_select(self, fresh, t, tau, period):
            return self._timed("verify+select", lambda: SCH.SpecaCacheBackend.verify_and_select(self, fresh, t, tau, period))

        def reference_step(self, feats, t, mask):
            return self._timed("update", lambda: SCH.SpecaCacheBackend.reference_step(self, feats, t, mask))

    be = Timed(cache)
    wall0 = time.perf_counter()
    tr = SCH.run_sampler(be, Model(), w.times, w.tau0, w.beta, w.period, w.warm_refs, gamma, total_steps=w.total_steps)
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    ms = {k: [a.elapsed_time(b_) for a, b_ in v] for k, v in be.spans.items()}
    lib_ms = sum(sum(v) for v in ms.values())
    res = {
        "workload": w.name, "sampler_steps": len(w.times), "period": w.period, "warm_refs": w.warm_refs, "gamma": gamma,
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


def oracle_sample_run(w: W.Workload, sample_elems: int, repeats: int, seed: int = 0):
    """The CPU oracle, as it stands, on a bounded sample of the workload: `sample_elems` elements
    per sample of the verification entry go through one full step (update at order m, forecast,
    Eq. 4, accept, select). Returns (seconds per step, algorithmic bytes per step, threads)."""
    import numpy as np
    from oracle import speca_oracle as O
    B, m = w.batch, w.max_order
    n = min(sample_elems, w.entry_elems(w.vidx))
    g = torch.Generator().manual_seed(W.SEED_BASE + seed)

    def feat():
        x = torch.randn(B, n, generator=g)
        if w.dtype == W.BF16:
            return x.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16).copy()
        return x.numpy().copy()

    cache = O.OracleCache([n], B, m, w.dtype)
    for k in range(m + 1):
        cache.update([feat()], [1.0 - 0.02 * k] * B)
        cache.commit_step()
    fa, fb = feat(), feat()
    eb = w.elem_bytes
    bytes_step = ((2 * m + 2) + (m + 2) + (m + 2)) * eb * n * B
    t0 = time.perf_counter()
    for r in range(repeats):
        t_ref = 1.0 - 0.02 * (m + 1 + r)
        cache.update([fa if r & 1 else fb], [t_ref] * B)
        cache.commit_step()
        cache.forecast_entry(0, [t_ref - 0.01] * B)
        err, acc, _ = cache.verify(fb if r & 1 else fa, [t_ref - 0.01] * B, [0.1] * B)
        O.select_adaptive([max(int(a), 0) for a in acc], 1 << 30, 1, [0] * B, [1] * B)
    dt = (time.perf_counter() - t0) / repeats
    return dt, bytes_step, O.threads(), n


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

    def host(x):
        x = x.detach().contiguous().cpu()
        if x.dtype == torch.bfloat16:
            return x.view(torch.int16).numpy().view(np.uint16).reshape(B, -1).copy()
        return x.numpy().reshape(B, -1).copy()

    def f64(a):
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64) if a.dtype == np.uint16 else a.astype(np.float64)

    for step in range(m + 1):
        t = [w.times[step]] * B
        f = src.feature(0, step, t)
        gpu.update([f], t)
        gpu.commit_step()
        cpu.update([host(f)], t)
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
    e_want, a_want, p_want = cpu.verify(host(fresh), t, tau)
    g, o = f64(host(pred)), f64(p_want)
    rel = [float(np.linalg.norm(g[b] - o[b]) / max(np.linalg.norm(o[b]), 1e-30)) for b in range(B)]
    e_got = [float(x) for x in err.cpu().tolist()]
    out = {"entry_elems": n_tok * dim, "samples": B,
           "forecast_norm_rel_diff_max": max(rel), "forecast_tolerance": 2e-3,
           "err_library": e_got, "err_oracle": [float(x) for x in e_want],
           "err_abs_diff_max": max(abs(a - b_) for a, b_ in zip(e_got, e_want)), "err_tolerance": 1e-4,
           "decisions_equal": [int(x) for x in acc.cpu().tolist()] == [int(x) for x in a_want]}
    gpu.close()
    return out


def run_reference(args, info: D.RankInfo):
    """The oracle timed on the host cores for the same metric (bounded sample per step)."""
    if not info.is_main:
        return
    w = make_workload(args.config)
    sample = 1 << 20
    for _ in range(max(0, args.warmup)):
        oracle_sample_run(w, sample, 1)
    dt, bytes_step, threads, n = oracle_sample_run(w, sample, max(1, args.steps))
    gbs = bytes_step / dt / 1e9
    sample_desc = "update+forecast+verify+select over %d elements x %d samples of the verification entry per step" % (
        n, w.batch)
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample_desc},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(w: W.Workload):
    return {
        "workload": "%s (benchmark config %d)" % (w.name, w.index),
        "entries": len(w.entries), "batch": w.batch, "taylor_order": w.max_order,
        "storage": "bf16" if w.dtype == W.BF16 else "f32",
        "elems_per_order": w.elems_per_order,
        "cache_bytes": w.elems_per_order * (w.max_order + 1) * w.elem_bytes,
        "l2": "no flush: every step streams a working set far larger than the 126 MB L2",
        "step": "update(all entries) + forecast(all entries) + verify(last entry) + select",
        "parallelism": "one independent cache per GPU (sample-sharded, no collective on the data path)",
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="flux", choices=["tiny", "dit_xl2", "flux", "hunyuan_video", "flux_b8"])
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--also", default="dit_xl2,hunyuan_video",
                    help="comma list of further configs measured device-resident and reported under per_config")
    ap.add_argument("--path", default="auto", choices=["auto", "direct", "bulk", "wide"],
                    help="kernel variant (speca_path_t); results are identical, only speed differs")
    ap.add_argument("--layout", default="tables", choices=["tables", "history"],
                    help="what the cache keeps: the paper's difference tables (default) or the raw features of "
                         "the last references (speca_layout_t)")
    ap.add_argument("--separate-select", action="store_true",
                    help="five launches per step (update, activate, forecast, verify, select) instead of the three fused ones")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-adaptive", action="store_true",
                    help="skip the B=8 sample-adaptive sweep (orders 1-3, horizon 1-6) reported under 'adaptive'")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup

    info = D.rank_info_from_env()
    if args.impl == "reference":
        run_reference(args, info)
        return

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

    w = make_workload(args.config)
    path = {"auto": 0, "direct": 1, "bulk": 2, "wide": 3}[args.path]
    layout = 1 if args.layout == "history" else 0
    h = Harness(w, device, seed_offset=17 * info.rank, path=path, fused_select=not args.separate_select, layout=layout)
    total_ms, per_ms, launches, clocks = time_device_resident(h, args.steps, args.warmup, info, True)
    total_ms = D.max_over_ranks(total_ms, device)
    value, ms_step, kernels, extra = summarize(w, per_ms, total_ms, args.steps, info.world, peak, layout=layout)

    tables = info.world == 1 and layout == 0      # these calls exist for the table layout only
    multi = time_multi_horizon(h, peak, per_ms["forecast"]) if tables else None
    metrics = time_metrics(h) if info.world == 1 else None
    per_entry = time_update_per_entry(h) if tables else None
    fsum = time_forecast_sum(h, peak) if tables else None

    e2e = None
    if not args.no_e2e:
        e2e_steps = max(3, min(args.steps, 24))
        e2e_ms, h2d, d2h = time_end_to_end(h, e2e_steps, 3)
        e2e_ms = D.max_over_ranks(e2e_ms, device)
        ab = algorithmic_bytes(w, w.max_order, layout)
        e2e = {"value": info.world * (ab["update"] + ab["forecast"] + ab["verify"]) / (e2e_ms * 1e-3) / 1e9,
               "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms,
               "steps": e2e_steps,
               "note": "features and verification feature copied from pinned host memory, forecasts and decisions copied back, "
                       "every step; copy-in, library calls and copy-out pipelined on three streams; host wall clock"}
    h.close()
    del h
    torch.cuda.empty_cache()

    drafts = None
    if info.world == 1 and layout == 0:
        try:
            drafts = time_draft_models(w, device, path)
        except Exception as exc:  # report, do not hide
            drafts = {"error": repr(exc)}

    history = None
    if info.world == 1 and path in (0, 3) and layout == 0:
        try:
            history = time_history_layout(w, device, path, min(args.steps, 100), info, peak, ms_step, kernels)
        except Exception as exc:  # report, do not hide
            history = {"error": repr(exc)}

    per_config = {}
    if info.world == 1 and layout == 0:
        for name in [n for n in args.also.split(",") if n and n != args.config]:
            try:
                w2 = make_workload(name)
                h2 = Harness(w2, device, path=path, fused_select=not args.separate_select)
                k2 = max(5, min(args.steps, 2000 // max(1, len(w2.entries)) * 4))
                t2, p2, _, _ = time_device_resident(h2, k2, 3, info, False)
                v2, ms2, kern2, ex2 = summarize(w2, p2, t2, k2, 1, peak)
                per_config[name] = {"value": v2, "unit": "GB/s", "ms_per_step": ms2, "steps": k2,
                                    "config": workload_config(w2), "kernels": kern2, **ex2,
                                    "multi_horizon": time_multi_horizon(h2, peak, p2["forecast"]),
                                    "update_one_launch_per_entry": time_update_per_entry(h2),
                                    "forecast_sum": time_forecast_sum(h2, peak)}
                h2.close()
                del h2
                torch.cuda.empty_cache()
                if path in (0, 3):
                    per_config[name]["history_layout"] = time_history_layout(w2, device, path, k2, info, peak, ms2, kern2)
            except Exception as exc:  # report, do not hide
                per_config[name] = {"error": repr(exc)}

    adaptive = None
    if info.world == 1 and not args.no_adaptive:
        try:
            adaptive = adaptive_sweep(device, peak, path)
        except Exception as exc:  # report, do not hide
            adaptive = {"error": repr(exc)}

    sampler = None
    if info.world == 1 and not args.no_adaptive:
        sampler = {}
        for name in ("dit_xl2", "flux_adaptive"):
            try:
                sampler[name] = sampler_run(device, path, name)
                if path in (0, 3):   # the same run on a cache that keeps raw features: cache-path time only
                    hist = sampler_run(device, path, name, layout=1)
                    sampler[name]["history_layout"] = {k: hist[k] for k in (
                        "acceptance_rate", "library_ms_total", "ms_mean", "sampler_steps_per_s_library_only")}
            except Exception as exc:  # report, do not hide
                sampler[name] = {"error": repr(exc)}

    if not info.is_main:
        D.shutdown()
        return

    dominant = max(("update", "forecast", "verify"), key=lambda k: per_ms[k])
    dom = kernels[dominant]
    per_elem = NCU_DRAM_BYTES_PER_ELEM.get(dominant)
    if layout == 1 and dominant == "update":
        per_elem = NCU_DRAM_BYTES_PER_ELEM_HISTORY_UPDATE
    n_dom = w.batch * w.entry_elems(w.vidx) if dominant == "verify" else w.elems_per_order
    roofline = {"bound": "hbm", "kernel": dominant, "achieved": dom["gbs"], "peak": peak, "unit": "GB/s",
                "frac": dom["gbs"] / peak, "peak_source": peak_src,
                "traffic": (per_elem * n_dom) if per_elem is not None else None,
                "algorithmic_bytes_per_launch": dom["algorithmic_bytes"],
                "frac_of_nominal_8TBs": dom["gbs"] / NOMINAL_HBM_GBS}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        n_s = w.entry_elems(w.vidx)
        dt1, _, _, _ = oracle_sample_run(w, n_s, 1)          # size the run: about 10 s of oracle work
        reps = max(1, min(50, int(10.0 / max(dt1, 1e-3))))
        dt, bytes_step, threads, n = oracle_sample_run(w, n_s, reps)
        cpu_baseline = {"value": bytes_step / dt / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
                        "sample": "%d steps of update+forecast+verify+select over the verification entry only "
                                  "(%d elements x %d samples), not all %d entries" % (reps, n, w.batch, len(w.entries)),
                        "s_per_step": dt}
        from oracle import speca_oracle as _O
        n_threads = _O.threads()
        _O.set_threads(1)
        dt_one, _, _, _ = oracle_sample_run(w, n_s, 1)
        _O.set_threads(n_threads)
        cpu_baseline["value_1_thread"] = bytes_step / dt_one / 1e9
        try:
            cpu_baseline["parity"] = parity_on_verify_entry(w, device, path)
        except Exception as exc:  # report, do not hide
            cpu_baseline["parity"] = {"error": repr(exc)}

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": info.world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": dict(workload_config(w), layout=args.layout, select="its own launch (speca_select_adaptive); re-arming its own launch (speca_activate)"
                       if args.separate_select else
                       "inside the verify launch (speca_verify_select); re-arming inside the update launch "
                       "(speca_cache_update_activate)"),
        "metric_note": "value = algorithmic bytes of the whole step (update + forecast + verify/select) / step time; "
                       "forecast + verify alone (one speculative step) is forecast_verify_gbs, the update alone kernels.update.gbs",
        "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": launches,
        "clocks": clocks, "kernels": kernels, **extra,
        "frac_of_measured_peak": value / info.world / peak, "frac_of_nominal_8TBs": value / info.world / NOMINAL_HBM_GBS,
        "multi_horizon": multi, "verify_metrics": metrics, "update_one_launch_per_entry": per_entry, "forecast_sum": fsum, "draft_models": drafts, "history_layout": history, "per_config": per_config, "adaptive": adaptive, "sampler": sampler,
        "paper_context": {"end_to_end_speedups": {"flux_h800": 6.34, "dit_xl2_a800": 7.3, "hunyuan_video_h800": 6.1},
                          "verification_overhead": "1.67%-3.5% of a full forward pass",
                          "note": "other hardware, whole-model numbers; context only"},
    }
    print(json.dumps(line))
    D.shutdown()


if __name__ == "__main__":
    main()
