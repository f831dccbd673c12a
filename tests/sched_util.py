"""Scheduler backends for tests: the CPU oracle behind the same methods the CUDA backend offers, a
scripted backend whose decisions are written down in advance, and a stand-in model that serves
features from the seeded generator."""
from __future__ import annotations

import numpy as np

from oracle import speca_oracle as O
from paper_2509_11628_b200 import workloads as W


class OracleBackend:
    def __init__(self, w: W.Workload, metric: int = O.METRIC_L2, layout: int = O.LAYOUT_TABLES):
        self.w, self.batch, self.metric = w, w.batch, metric
        self.cache = O.OracleCache([n * d for n, d in w.entries], w.batch, w.max_order, w.dtype, layout=layout)
        self.reset_run()

    def reset_run(self):
        self.cache.reset()
        self.active = [0] * self.batch
        self.spec = [0] * self.batch

    def tau(self, tau0, beta, t, T):
        return O.tau_schedule(tau0, beta, t, T)

    def forecast(self, t_target):
        pass  # the stand-in model does not consume forecasts; verify recomputes the one it needs

    def verify_and_select(self, fresh, t_target, tau, period):
        err, acc, _ = self.cache.verify(fresh, t_target, tau, self.active, metric=self.metric)
        acc = [1 if a == 1 else 0 for a in acc]
        self.active, self.spec, _ = O.select_adaptive(acc, period, 1, self.spec, self.active)
        return [float(e) for e in err], acc

    def active_mask(self):
        return list(self.active)

    def reference_step(self, feats, t_ref, mask, t_next=None):
        self.cache.update(feats, t_ref, mask)
        self.cache.commit_step()
        for b in range(self.batch):
            if mask[b]:
                self.active[b], self.spec[b] = 1, 0


class ScriptedBackend:
    """Accept flags come from a script {(step, sample): 0/1} (default accept); no arithmetic at all."""

    def __init__(self, batch, script):
        self.batch, self.script, self.step = batch, script, -1
        self.reset_run()

    def reset_run(self):
        self.active, self.spec, self.calls = [0] * self.batch, [0] * self.batch, []

    def tau(self, tau0, beta, t, T):
        self.step += 1
        return tau0

    def forecast(self, t_target):
        self.calls.append(("forecast", self.step, tuple(self.active)))

    def verify_and_select(self, fresh, t_target, tau, period):
        acc = [self.script.get((self.step, b), 1) if self.active[b] else 0 for b in range(self.batch)]
        self.calls.append(("verify", self.step, tuple(self.active)))
        self.active, self.spec, _ = O.select_adaptive(acc, period, 1, self.spec, self.active)
        return [0.0] * self.batch, acc

    def active_mask(self):
        return list(self.active)

    def reference_step(self, feats, t_ref, mask, t_next=None):
        self.calls.append(("update", self.step, tuple(mask)))
        for b in range(self.batch):
            if mask[b]:
                self.active[b], self.spec[b] = 1, 0


class NullModel:
    def full(self, step, times, mask):
        return None

    def verify_feature(self, step, times):
        return None


class GeneratorModel:
    """Stand-in for the diffusion transformer: block outputs come from the seeded feature generator.
    `to_backend` converts a device tensor to what the backend expects (identity for the CUDA one)."""

    def __init__(self, w: W.Workload, device="cpu", to_backend=None):
        self.w, self.src = w, W.FeatureSource(w, device)
        self.conv = to_backend or (lambda x: x)

    def full(self, step, times, mask):
        return [self.conv(self.src.feature(e, step, times)) for e in range(len(self.w.entries))]

    def verify_feature(self, step, times):
        return self.conv(self.src.feature(self.w.vidx, step, times))


def to_oracle_array(x):
    import torch
    x = x.detach().contiguous().cpu()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16).reshape(x.shape[0], -1).copy()
    return x.numpy().reshape(x.shape[0], -1).copy()
