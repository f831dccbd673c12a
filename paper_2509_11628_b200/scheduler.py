"""Forecast-then-verify control flow over the cache library (Section 3.2 workflow, Section 3.4.2
sequential validation, the forced activation period of the appendix's hyper-parameters).

This module holds control flow and bookkeeping only: every number it branches on (accept flags,
active masks, thresholds) comes from the backend it drives -- the CUDA library through
``SpecaCacheBackend`` below, or any object with the same methods. The model is a stand-in supplied by
the caller: ``full(step, times, mask)`` returns the block outputs of a complete forward pass,
``verify_feature(step, times)`` the freshly computed verification-layer feature of a speculative step.

Per sampler step, per sample:
  * a sample that is *active* attempts the step speculatively: its block outputs are forecast
    (Eq. 2), the verification layer is computed for real, Eq. 4 is compared with tau_t;
  * accepted (e <= tau_t): the step costs gamma (verification only) and the sample stays active
    until it has taken ``period`` speculative steps in a row;
  * rejected: the step is recomputed in full (Eq. 6 puts the rejected step in the rejection set), the
    tables are updated from it, and the sample becomes active again;
  * a sample that is not active takes a full step, updates its tables and becomes active.
Samples of one batch therefore drift apart: each gets as many full steps as its own errors demand
(sample-adaptive computation allocation).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence

FULL, ACCEPTED, REJECTED = "F", "A", "R"


@dataclass
class Trace:
    """What happened: ``steps[i][b]`` is FULL, ACCEPTED or REJECTED (rejected = verified, failed,
    then recomputed in full). ``err[i][b]`` is the verification error where one was computed."""
    batch: int
    gamma: float
    steps: List[List[str]] = field(default_factory=list)
    err: List[List[float]] = field(default_factory=list)
    tau: List[float] = field(default_factory=list)

    def counts(self, b: int):
        col = [row[b] for row in self.steps]
        return col.count(FULL), col.count(ACCEPTED), col.count(REJECTED)

    def acceptance_rate(self, b: int = None) -> float:
        """alpha = speculative steps that were accepted / all steps (Section 3.5)."""
        cols = range(self.batch) if b is None else [b]
        acc = sum(self.counts(c)[1] for c in cols)
        return acc / float(len(self.steps) * len(list(cols)))

    def cost(self, b: int) -> float:
        """In units of one full forward pass: full = 1, accepted = gamma, rejected = gamma + 1."""
        f, a, r = self.counts(b)
        return f + a * self.gamma + r * (1.0 + self.gamma)

    def speedup(self, b: int = None) -> float:
        cols = list(range(self.batch)) if b is None else [b]
        return len(self.steps) * len(cols) / sum(self.cost(c) for c in cols)

    def predicted_speedup(self, b: int = None) -> float:
        """Eq. 8 with the measured acceptance rate: S = 1 / (1 - alpha + alpha * gamma)."""
        a = self.acceptance_rate(b)
        return 1.0 / (1.0 - a + a * self.gamma)

    def full_steps_histogram(self):
        """{number of full forward passes: how many samples needed that many}."""
        hist = {}
        for b in range(self.batch):
            f, _, r = self.counts(b)
            hist[f + r] = hist.get(f + r, 0) + 1
        return dict(sorted(hist.items()))


def run_sampler(backend, model, times: Sequence[float], tau0: float, beta: float, period: int, warm_refs: int,
                gamma: float, total_steps: int = None) -> Trace:
    """Drive ``backend`` through the whole timeline. ``times[i]`` is the sampler time of step i;
    the first ``warm_refs`` steps are always full. ``period`` is the largest number of consecutive
    speculative steps a sample may take."""
    B = backend.batch
    T = total_steps if total_steps is not None else len(times)
    trace = Trace(batch=B, gamma=gamma)
    active = [0] * B                      # host mirror of the device mask, refreshed once per step
    backend.reset_run()
    for i, t in enumerate(times):
        tt = [t] * B
        row = [FULL] * B
        errs = [float("nan")] * B
        tau_i = backend.tau(tau0, beta, T - i, T)
        trace.tau.append(tau_i)
        attempted = [b for b in range(B) if active[b]] if i >= warm_refs else []
        horizon = getattr(backend, "horizon", 1)
        if attempted:
            if horizon > 1:                                        # this step's forecasts, and the following steps' with them
                backend.forecast(tt, [[x] * B for x in times[i + 1:i + horizon]])
            else:
                backend.forecast(tt)                               # forecasts for the active samples
            fresh = model.verify_feature(i, tt)                    # the model computes the verify layer
            e, acc = backend.verify_and_select(fresh, tt, [tau_i] * B, period)
            for b in attempted:
                errs[b] = e[b]
                row[b] = ACCEPTED if acc[b] else REJECTED
            active = backend.active_mask()
        # everyone who did not get through speculatively takes the step in full and refreshes the tables
        need_full = [0 if row[b] == ACCEPTED else 1 for b in range(B)]
        if any(need_full):
            feats = model.full(i, tt, need_full)
            # the next step is speculative for everyone who is active after this one: a backend that can
            # may hand over that step's forecasts from the same pass over the tables
            t_next = [times[i + 1]] * B if i + 1 < len(times) and i + 1 >= warm_refs else None
            if horizon > 1 and t_next is not None:
                # up to `period` speculative steps follow a reference step: a backend with a horizon forecasts
                # them all from the one pass (Fig. 1: the draft predicts the next steps from one reference)
                later = [[x] * B for x in times[i + 2:i + 1 + min(horizon, period)]]
                backend.reference_step(feats, tt, need_full, t_next, later)
            else:
                backend.reference_step(feats, tt, need_full, t_next)
            active = backend.active_mask()
        trace.steps.append(row)
        trace.err.append(errs)
    return trace


class SpecaCacheBackend:
    """The CUDA library as a scheduler backend. Device buffers are allocated once; one small
    device-to-host copy of the decisions per speculative step is the only synchronisation."""

    def __init__(self, cache, metric=None, use_fused=True, horizon=1):
        """``horizon`` K > 1: a reference step that the whole batch takes forecasts the next K steps in its
        own pass over the tables (2v + 2 + K words per element for all K, where K single forecasts would read
        the tables K times), and the speculative steps that follow launch only their verification. Costs K
        output buffers per entry. A handed-over step costs one word per element if the run ends before it and
        saves v + 1 if it is reached, so the number handed over follows the runs seen: one more than the
        speculative run that has just ended (the first time: K). While the samples of a batch are out of step
        with one another (reference steps that only some samples take come every step or two) only the next
        step is handed over."""
        import torch
        from . import binding as S
        self.S, self.torch, self.cache = S, torch, cache
        self.use_fused = use_fused      # reference steps also hand over the next step's forecasts (one launch)
        self.horizon = max(1, min(int(horizon), S.SPECA_MAX_HORIZON)) if use_fused else 1
        self.handed = {}                # time of a coming step (per sample, as a tuple) -> row of `multi` that holds its forecasts
        self.in_step = False            # the last reference step was taken by the whole batch
        self.run = None                 # speculative steps the whole batch has passed since then (None: no run seen yet)
        self.batch = cache.batch
        dev = cache.device
        self.metric = metric
        tdt = torch.bfloat16 if cache.dtype == S.SPECA_BF16 else torch.float32
        # [K, B, N_e, D] per entry; `outs` are the rows the current step's forecasts are in
        self.multi = [torch.empty(self.horizon, cache.batch, n, d, dtype=tdt, device=dev) for n, d in cache.entries]
        self.outs = [m[0] for m in self.multi]
        # What the host reads back every step sits in ONE device buffer with ONE pinned mirror, so that a step
        # costs one small copy and one stream synchronisation: errors | accept flags | the two mask buffers
        # that the fused verification alternates between (the next mask goes to the buffer that is not read).
        B = self.batch
        self.pack = torch.zeros(7 * B, dtype=torch.uint8, device=dev)
        self.h_pack = torch.zeros(7 * B, dtype=torch.uint8).pin_memory()
        self.err = self.pack[:4 * B].view(torch.float32)
        self.accept = self.pack[4 * B:5 * B]
        self.masks = [self.pack[5 * B:6 * B], self.pack[6 * B:7 * B]]
        self.cur = 0                    # which of the two masks is the current one
        self.spec = torch.zeros(B, dtype=torch.int32, device=dev)
        self.idx = torch.zeros(B, dtype=torch.int32, device=dev)
        self.n_active = torch.zeros(1, dtype=torch.int32, device=dev)
        self.h_err = self.h_pack[:4 * B].view(torch.float32)
        self.h_accept = self.h_pack[4 * B:5 * B]

    @property
    def active(self):
        """The device mask of the samples that are speculating (the current one of the two buffers)."""
        return self.masks[self.cur]

    @property
    def active_next(self):
        return self.masks[1 - self.cur]

    @property
    def h_active(self):
        B = self.batch
        return self.h_pack[(5 + self.cur) * B:(6 + self.cur) * B]

    def reset_run(self):
        self.cache.reset()
        self.handed, self.in_step, self.run = {}, False, None
        self.pack.zero_()
        self.spec.zero_()
        self.h_pack.zero_()

    def _fetch(self, with_decisions):
        self.h_pack.copy_(self.pack, non_blocking=True)
        self.torch.cuda.current_stream(self.cache.device).synchronize()

    def tau(self, tau0, beta, t, T):
        return self.S.speca_tau(tau0, beta, t, T)

    def forecast(self, t_target, t_later=()):
        row = self.handed.get(tuple(t_target))
        if row is not None:               # an earlier call already wrote these forecasts
            self.outs = [m[row] for m in self.multi]
            return
        targets = [list(t_target)]
        if self.in_step:                  # a run longer than expected: its next stretch in one read of the tables
            targets += [list(t) for t in t_later][:self._expected_run() - 1]
        self.handed = {tuple(t): k for k, t in enumerate(targets)}
        self.outs = [m[0] for m in self.multi]
        if len(targets) == 1:
            self.cache.forecast(t_target, self.outs, self.active)
        else:                             # the following steps' forecasts from the same read of the tables
            self.cache.forecast_multi(targets, [m[:len(targets)] for m in self.multi], self.active)

    def verify_and_select(self, fresh, t_target, tau, period):
        # Eq. 4 and the continuation rule in one launch; the next mask arrives in the other buffer
        self.cache.verify_select(fresh, t_target, tau, self.err, self.accept, self.active, self.active_next, period, 1,
                                 self.spec, self.idx, self.n_active, metric=self.metric or 0)
        attempted = self.h_active.tolist()
        self.cur = 1 - self.cur
        self._fetch(with_decisions=True)
        # the launch writes the flags of the samples it verified; the others' are stale and read as "no"
        accepted = [int(a) if on else 0 for a, on in zip(self.h_accept.tolist(), attempted)]
        if self.run is not None and all(a for a, on in zip(accepted, attempted) if on):
            self.run += 1
        return self.h_err.tolist(), accepted

    def _expected_run(self):
        """How many coming steps to forecast at once: one more than the run that is ending (or under way)."""
        return self.horizon if self.run is None else max(1, min(self.horizon, self.run + 1))

    def active_mask(self):
        return self.h_active.tolist()

    def reference_step(self, feats, t_ref, mask, t_next=None, t_later=()):
        S = self.S
        fused = self.use_fused and t_next is not None and self.cache.path in (S.SPECA_PATH_AUTO, S.SPECA_PATH_WIDE)
        self.handed = {}                  # the tables change: forecasts handed over earlier are void for the updated samples
        self.in_step = all(mask)
        if fused:
            # Eq. 3, the re-arming and Eq. 2 at the coming steps' times in one launch: samples that took this
            # step are forecast from the planes just written, the ones still speculating from theirs
            targets = [list(t_next)]
            if self.in_step:              # the speculative run that follows, as long as the last one was (and one more)
                targets += [list(t) for t in t_later][:self._expected_run() - 1]
            self.cache.update_forecast_multi(feats, t_ref, targets, [m[:len(targets)] for m in self.multi], mask=mask,
                                             active=self.active, spec_count=self.spec, rearm=self.active)
            self.handed = {tuple(t): k for k, t in enumerate(targets)}
        else:
            self.cache.update_activate(feats, t_ref, mask, self.spec, self.active)   # Eq. 3 and the re-arming, one launch
            self.cache.commit_step()
        if fused:
            self.run = 0                  # a new run starts (warm-up references, which forecast nothing, do not count)
        self._fetch(with_decisions=False)
