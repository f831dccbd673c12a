"""Seeded synthetic workloads shaped like the paper's three models.

This module only *describes* and *generates inputs*: entry lists (which block outputs are cached
and how big they are), the sampler's time grid, threshold-schedule parameters, and a seeded
feature generator. It holds none of the method's arithmetic (no differences, no extrapolation,
no error norm, no threshold formula), so the CPU oracle's tests and the CUDA path's tests and
benchmarks can both draw inputs from it.

The activations of DiT-XL/2, FLUX.1-dev and HunyuanVideo (Section 4.1 of the paper; 28 blocks,
19 dual + 38 single blocks, 20 dual + 40 single blocks -- the block counts agree with the
verification-cost ratios 1/28, 1/57, 1/60 quoted in the appendix) are replaced by features with
the same shapes and a similar value structure: a smooth polynomial in the sampler time per
element, plus fresh Gaussian noise per step, plus a few outlier channels scaled x50. They stand
in for the ImageNet / DrawBench / VBench runs of the paper, whose weights and data are not needed
to exercise an element-wise cache.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import torch

F32, BF16 = 0, 1
_TORCH_DTYPE = {F32: torch.float32, BF16: torch.bfloat16}
SEED_BASE = 20250911


@dataclass
class Workload:
    name: str
    index: int                          # position in the benchmark's config list (1-based)
    entries: List[Tuple[int, int]]      # (tokens N_e, dim D) per cached tensor
    batch: int
    max_order: int
    dtype: int
    times: List[float]                  # sampler time of step i, i = 0 .. n_steps-1 (decreasing)
    poly_degree: int                    # degree of the smooth part of the features in t
    sigma: List[float]                  # per-sample noise scale
    outlier_frac: float = 0.0           # fraction of channels scaled x50 (at least one if > 0)
    tau0: float = 0.1
    beta: float = 0.5
    total_steps: int = 50               # T of the threshold schedule (step-index coordinate)
    warm_refs: int = 3                  # fully computed steps before the first speculative one
    period: int = 5                     # forced activation period: a reference every `period` steps
    frame_tokens: int = 0               # > 0: per-frame drift over the first video_tokens tokens
    n_frames: int = 0
    video_tokens: int = 0
    verify_entry: int = -1
    notes: str = ""
    labels: List[str] = field(default_factory=list)

    @property
    def torch_dtype(self):
        return _TORCH_DTYPE[self.dtype]

    @property
    def elem_bytes(self) -> int:
        return 2 if self.dtype == BF16 else 4

    def entry_elems(self, e: int) -> int:
        n, d = self.entries[e]
        return n * d

    @property
    def elems_per_order(self) -> int:
        return self.batch * sum(n * d for n, d in self.entries)

    @property
    def vidx(self) -> int:
        return self.verify_entry if self.verify_entry >= 0 else len(self.entries) - 1


def _uniform_times(n: int) -> List[float]:
    return [1.0 - i / n for i in range(n)]


def _shifted_sigmoid_times(n: int, mu: float) -> List[float]:
    """Flow-matching time grid with an exponential shift: s_i = 1 - i/n,
    t_i = e^mu / (e^mu + 1/s_i - 1). Gaps are uneven."""
    out = []
    for i in range(n):
        s = 1.0 - i / n
        out.append(math.exp(mu) / (math.exp(mu) + 1.0 / s - 1.0))
    return out


def _linear_shift_times(n: int, shift: float) -> List[float]:
    """Flow time grid with a rational shift: t_i = shift*s_i / (1 + (shift-1)*s_i)."""
    out = []
    for i in range(n):
        s = 1.0 - i / n
        out.append(shift * s / (1.0 + (shift - 1.0) * s))
    return out


def tiny() -> Workload:
    return Workload(
        name="tiny_dit_s", index=1, entries=[(64, 384)] * 8, batch=2, max_order=2, dtype=F32,
        times=[1.0, 0.9, 0.8, 0.775, 0.75, 0.725, 0.7], poly_degree=2, sigma=[0.01, 0.01],
        tau0=0.05, beta=1.0, total_steps=7, warm_refs=3, period=5,
        notes="4 layers x (attn, mlp); refs at t=1.0,0.9,0.8 then 4 forecasts 0.025 apart",
        labels=["L%d.%s" % (l, br) for l in range(4) for br in ("attn", "mlp")])


def dit_xl2() -> Workload:
    return Workload(
        name="dit_xl2_256", index=2, entries=[(256, 1152)] * 56, batch=16, max_order=2, dtype=BF16,
        times=_uniform_times(50), poly_degree=2, sigma=[0.02] * 16, outlier_frac=0.001,
        tau0=0.3, beta=0.5, notes="28 blocks x (attn, mlp), 8 images x CFG pair, 50-step DDIM grid",
        labels=["B%d.%s" % (l, br) for l in range(28) for br in ("attn", "mlp")])


def _dual_single(n_dual, n_single, n_main, n_txt, dim):
    entries, labels = [], []
    for l in range(n_dual):
        entries += [(n_main, dim), (n_txt, dim)]
        labels += ["D%d.main" % l, "D%d.txt" % l]
    for l in range(n_single):
        entries.append((n_main + n_txt, dim))
        labels.append("S%d" % l)
    return entries, labels


def flux(batch: int = 1, max_order: int = 2, sigma: Optional[Sequence[float]] = None) -> Workload:
    entries, labels = _dual_single(19, 38, 4096, 512, 3072)
    return Workload(
        name="flux_dev_1024" if batch == 1 else "flux_dev_1024_b%d" % batch, index=3 if batch == 1 else 5,
        entries=entries, batch=batch, max_order=max_order, dtype=BF16,
        times=_shifted_sigmoid_times(50, 1.15), poly_degree=3,
        sigma=list(sigma) if sigma is not None else [0.02] * batch, outlier_frac=0.001,
        tau0=0.1, beta=0.2, notes="19 dual (img 4096 + txt 512) + 38 single (4608) blocks, D=3072",
        labels=labels)


def hunyuan_video() -> Workload:
    entries, labels = _dual_single(20, 40, 20670, 256, 3072)
    return Workload(
        name="hunyuan_video_480p_2s", index=4, entries=entries, batch=1, max_order=2, dtype=BF16,
        times=_linear_shift_times(50, 7.0), poly_degree=3, sigma=[0.02], outlier_frac=0.001,
        tau0=0.1, beta=0.2, frame_tokens=30 * 53, n_frames=13, video_tokens=20670,
        notes="20 dual (video 13x30x53 + txt 256) + 40 single blocks, D=3072", labels=labels)


def flux_adaptive(max_order: int = 2, batch: int = 8) -> Workload:
    """FLUX-shaped batch whose samples carry different noise scales (seeded draw from three
    levels), so that they accept and reject differently."""
    g = torch.Generator().manual_seed(SEED_BASE + 5)
    levels = [0.005, 0.02, 0.08]
    pick = torch.randint(0, 3, (batch,), generator=g).tolist()
    w = flux(batch=batch, max_order=max_order, sigma=[levels[i] for i in pick])
    w.name = "flux_adaptive_b%d_m%d" % (batch, max_order)
    w.warm_refs = max_order + 1
    return w


def scaled(w: Workload, max_entries: int = 0, max_tokens: int = 0) -> Workload:
    """A cut-down copy (fewer entries and/or fewer tokens per entry) for tests: same dim, dtype,
    time grid and value structure. The verification entry stays the last one."""
    import copy
    c = copy.deepcopy(w)
    if max_entries and len(c.entries) > max_entries:
        keep = list(range(max_entries - 1)) + [len(c.entries) - 1]
        c.entries = [c.entries[i] for i in keep]
        c.labels = [c.labels[i] for i in keep] if c.labels else []
    if max_tokens:
        c.entries = [(min(n, max_tokens), d) for n, d in c.entries]
        c.video_tokens = min(c.video_tokens, max_tokens)
    c.verify_entry = -1
    c.name = w.name + "_cut"
    return c


BY_NAME = {
    "tiny": tiny, "dit_xl2": dit_xl2, "flux": flux, "hunyuan_video": hunyuan_video,
    "flux_adaptive": flux_adaptive,
}


class FeatureSource:
    """f_e(b, n, c; t) = s_c * poly_{e,n,c}(t) + s_c * sigma_b * xi, rounded to the storage dtype.

    The polynomial coefficients are N(0,1) per element, fixed for the run and re-drawn from the
    entry's seed on every call (so nothing the size of the cache is kept); xi is N(0,1), fresh
    per (entry, step). s_c = 50 on a seeded choice of outlier channels, else 1. With frames
    configured, video tokens get a smooth per-frame drift of the constant and linear terms.
    """

    def __init__(self, w: Workload, device: str = "cpu", seed_offset: int = 0):
        self.w, self.device = w, torch.device(device)
        self.seed = SEED_BASE + 1000 * w.index + seed_offset

    def _gen(self, seed: int) -> torch.Generator:
        g = torch.Generator(device=self.device)
        g.manual_seed(seed)
        return g

    def coefficients(self, e: int) -> torch.Tensor:
        """[degree+1, N_e, D] fp32 coefficients of entry e (shared by the samples of a batch; the
        samples differ through a per-sample factor applied in `feature`)."""
        n, d = self.w.entries[e]
        g = self._gen(self.seed + e)
        a = torch.randn(self.w.poly_degree + 1, n, d, generator=g, device=self.device, dtype=torch.float32)
        if self.w.frame_tokens > 0:
            nv = min(n, self.w.video_tokens)
            frame = torch.arange(nv, device=self.device) // self.w.frame_tokens
            phase = frame.to(torch.float32) / float(self.w.n_frames)
            a[1, :nv] *= (1.0 + 0.25 * torch.sin(2.0 * math.pi * phase))[:, None]
            a[0, :nv] += (0.1 * phase)[:, None]
        return a

    def channel_scale(self, e: int) -> torch.Tensor:
        n, d = self.w.entries[e]
        s = torch.ones(d, device=self.device, dtype=torch.float32)
        if self.w.outlier_frac > 0:
            k = max(1, round(self.w.outlier_frac * d))
            g = torch.Generator().manual_seed(self.seed + 7919 * (e + 1))
            idx = torch.randperm(d, generator=g)[:k].to(self.device)
            s[idx] = 50.0
        return s

    def feature(self, e: int, step: int, t: Sequence[float], noise: bool = True) -> torch.Tensor:
        """[B, N_e, D] in the storage dtype: entry e at sampler step `step`, sample b at time t[b]."""
        w = self.w
        n, d = w.entries[e]
        a = self.coefficients(e)
        tt = torch.tensor(list(t), device=self.device, dtype=torch.float32).view(w.batch, 1, 1)
        # per-sample variation of the smooth part: sample b scales coefficient i by (1 + 0.1*b/(B))^i
        sample_gain = 1.0 + 0.1 * torch.arange(w.batch, device=self.device, dtype=torch.float32) / max(1, w.batch)
        f = torch.zeros(w.batch, n, d, device=self.device, dtype=torch.float32)
        for i in range(w.poly_degree, -1, -1):
            f = f * (tt * sample_gain.view(-1, 1, 1)) + a[i]
        if noise:
            g = self._gen(self.seed + 104729 * (step + 1) + e)
            xi = torch.randn(w.batch, n, d, generator=g, device=self.device, dtype=torch.float32)
            sig = torch.tensor(w.sigma, device=self.device, dtype=torch.float32).view(w.batch, 1, 1)
            f = f + sig * xi
        f = f * self.channel_scale(e).view(1, 1, d)
        return f.to(w.torch_dtype).contiguous()


def reference_pattern(w: Workload) -> List[bool]:
    """is_reference[i] for each step of the grid: the first `warm_refs` steps are fully computed,
    after that one step in every `period`."""
    out = []
    for i in range(len(w.times)):
        out.append(i < w.warm_refs or (i - (w.warm_refs - 1)) % w.period == 0)
    return out
