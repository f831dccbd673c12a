"""Helpers shared by the GPU parity tests: tensor <-> oracle array conversion, tolerances, and a
driver that feeds identical seeded inputs to the CUDA library and to the CPU oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import speca_oracle as O
from paper_2509_11628_b200 import binding as S

BF16_ULP_REL = 2.0 ** -7   # one bfloat16 ulp is at most 2^-7 of the value
FORECAST_NORM_TOL = 2e-3   # ||gpu - oracle|| / ||oracle|| per (entry, sample)
ERR_TOL = 1e-4             # |e_gpu - e_oracle| <= ERR_TOL * max(1, e_oracle)


def to_oracle(x: torch.Tensor) -> np.ndarray:
    """Storage bits of a tensor as the oracle's array type (float32, or uint16 bf16 patterns)."""
    x = x.detach().contiguous().cpu()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16).copy()
    assert x.dtype == torch.float32
    return x.numpy().copy()


def as_f64(a: np.ndarray) -> np.ndarray:
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def storage_ulp(ref: np.ndarray, dtype: int) -> np.ndarray:
    """Size of one unit in the last place of the storage type at |ref|."""
    mant = 7 if dtype == O.BF16 else 23
    a = np.maximum(np.abs(ref), 2.0 ** -126)
    return 2.0 ** (np.floor(np.log2(a)) - mant)


def assert_close_storage(got: np.ndarray, want: np.ndarray, dtype: int, scale: np.ndarray | float, what: str):
    """got/want: storage arrays. Element-wise: within one storage ulp of the oracle's value plus the
    fp32-vs-fp64 evaluation error of a sum whose terms have magnitude `scale`. Norm-wise: 2e-3."""
    g, w = as_f64(got), as_f64(want)
    both_nan = np.isnan(g) & np.isnan(w)
    g, w = np.where(both_nan, 0.0, g), np.where(both_nan, 0.0, w)
    tol = storage_ulp(w, dtype) + 1e-6 * np.asarray(scale, dtype=np.float64) + 1e-30
    bad = np.abs(g - w) > tol
    assert not bad.any(), "%s: %d elements off by more than one ulp; worst %g vs %g" % (
        what, int(bad.sum()), float(g[bad][0]), float(w[bad][0]))
    den = float(np.linalg.norm(w))
    if den > 0 and w.size >= 1024:  # a single one-ulp flip dominates the norm of a tiny segment
        rel = float(np.linalg.norm(g - w)) / den
        assert rel <= FORECAST_NORM_TOL, "%s: norm-wise error %g" % (what, rel)


def assert_equal_or_tie(got: np.ndarray, want: np.ndarray, unrounded: np.ndarray, dtype: int, scale, what: str) -> float:
    """Where a result is a rounding of a value that sits (within the fp32 evaluation error of its terms,
    4e-6 of their magnitude `scale`) on the midpoint of two neighbouring storage values, both neighbours
    are correct roundings. `got` must equal the oracle's `want` bit for bit everywhere else; where it
    differs it must be the neighbour on the other side of such a midpoint (`unrounded` is the oracle's
    float64 value before rounding), or -- where the terms cancel to something smaller than their own
    evaluation error -- lie within that error of the oracle's value. Returns the share of elements that
    differ at all."""
    g, w = as_f64(got), as_f64(want)
    diff = (got != want) & ~(np.isnan(g) & np.isnan(w))
    if not diff.any():
        return 0.0
    mid = 0.5 * (g[diff] + w[diff])
    ulp = storage_ulp(w[diff], dtype)
    sc = np.broadcast_to(np.asarray(scale, dtype=np.float64), g.shape)[diff]
    adjacent = np.abs(g[diff] - w[diff]) <= 1.0001 * np.maximum(ulp, storage_ulp(g[diff], dtype))
    near_tie = np.abs(unrounded[diff] - mid) <= 4e-6 * sc + 1e-30
    cancelled = np.abs(g[diff] - w[diff]) <= 4e-6 * sc
    bad = ~((adjacent & near_tie) | cancelled)
    assert not bad.any(), "%s: %d elements differ from the oracle away from a rounding tie; first: got %g want %g unrounded %.17g" % (
        what, int(bad.sum()), float(g[diff][bad][0]), float(w[diff][bad][0]), float(unrounded[diff][bad][0]))
    return float(diff.sum()) / got.size


def term_scale(planes: np.ndarray, weights) -> np.ndarray:
    """Sum of |plane_i * w_i| per element: magnitude of the terms the forecast adds up."""
    p = as_f64(planes)
    return sum(np.abs(p[i]) * abs(w) for i, w in enumerate(weights))


class Pair:
    """A CUDA cache and an oracle cache driven with identical inputs."""

    def __init__(self, entries, batch, max_order, dtype, basis=S.SPECA_BASIS_TAYLOR, verify_entry=-1,
                 device="cuda:0", path=S.SPECA_PATH_AUTO, layout=S.SPECA_LAYOUT_TABLES):
        self.entries = list(entries)
        self.B, self.m, self.dtype, self.basis = batch, max_order, dtype, basis
        self.device = torch.device(device)
        self.tdt = torch.bfloat16 if dtype == S.SPECA_BF16 else torch.float32
        self.layout = layout
        self.gpu = S.SpecaCache(entries, batch, max_order, dtype, device, basis, verify_entry, path=path, layout=layout)
        self.cpu = O.OracleCache([n * d for n, d in entries], batch, max_order, dtype, basis, verify_entry, layout=layout)
        self.vidx = self.gpu.verify_entry

    def close(self):
        self.gpu.close()

    def update(self, feats, t_ref, mask=None, per_entry_calls=False):
        """feats: list of device tensors [B, N, D] (None = skip)."""
        if per_entry_calls:
            for e, f in enumerate(feats):
                if f is None:
                    continue
                one = [None] * len(feats)
                one[e] = f
                self.gpu.update(one, t_ref, mask)
        else:
            self.gpu.update(feats, t_ref, mask)
        self.cpu.update([None if f is None else to_oracle(f).reshape(self.B, -1) for f in feats], t_ref, mask)

    def commit(self):
        self.gpu.commit_step()
        self.cpu.commit_step()

    def check_tables(self, what="tables"):
        torch.cuda.synchronize()
        if self.layout == S.SPECA_LAYOUT_HISTORY:
            # the planes hold copies of the last features: age j sits in plane (references - 1 - j) mod (m + 1)
            for e in range(len(self.entries)):
                for b in range(self.B):
                    got = to_oracle(self.gpu.plane_tensor(e, b))
                    for j, want in enumerate(self.cpu.hist[e][b][: min(self.cpu.n_refs[b], self.m + 1)]):
                        phys = (self.cpu.n_refs[b] - 1 - j) % (self.m + 1)
                        assert np.array_equal(got[phys], want), "%s entry %d sample %d age %d" % (what, e, b, j)
            return
        for e in range(len(self.entries)):
            for b in range(self.B):
                v = min(self.m, self.cpu.n_refs[b] - 1)
                if v < 0:
                    continue
                got = to_oracle(self.gpu.plane_tensor(e, b))
                want = self.cpu.planes[e][b]
                R = self._max_recip(b)
                for i in range(v + 1):
                    # the fp32 chain c_{j+1} = (c_j - D_j) / gap carries the rounding error of every
                    # earlier link, amplified by 1/gap per step: sum_j |plane_j| * R^(i-j)
                    scale = sum(np.abs(as_f64(want[j])) * R ** (i - j) for j in range(i + 1))
                    assert_close_storage(got[i], want[i], self.dtype, scale * 0.5,
                                         "%s entry %d sample %d plane %d" % (what, e, b, i))

    def sync_tables(self):
        """Overwrite the GPU tables with the oracle's bits so that both sides continue from the same
        state (a one-ulp rounding flip in a stored plane would otherwise be amplified by 1/gap at
        the next reference step and hide real errors behind a loose tolerance)."""
        if self.layout == S.SPECA_LAYOUT_HISTORY:
            return  # the planes are bit-exact copies of the features: nothing can drift
        for e in range(len(self.entries)):
            for b in range(self.B):
                src = torch.from_numpy(self.cpu.planes[e][b].view(np.int16) if self.dtype == O.BF16
                                       else self.cpu.planes[e][b])
                if self.dtype == O.BF16:
                    src = src.view(torch.bfloat16)
                self.gpu.plane_tensor(e, b).copy_(src.to(self.device))
        torch.cuda.synchronize()

    def _max_recip(self, b):
        h = self.cpu.t_hist[b]
        if len(h) < 2:
            return 0.0
        gaps = [abs(h[0] - h[j]) for j in range(1, len(h))]
        return 1.0 / min(gaps)

    def history_scale(self, e, b, t):
        """sum_j |a_j * F_j| per element for the raw-feature cache: the weight a_j of the feature of age j
        is read off by forecasting one-hot features."""
        k = min(self.cpu.n_refs[b], self.m + 1)
        unit = [np.eye(k, dtype=np.float32)[j].copy() for j in range(k)]
        a = np.zeros(k, dtype=np.float32)
        O.forecast_history_segment(O.F32, self.m, self.basis, self.cpu.t_hist[b], t, unit, a)
        return sum(np.abs(as_f64(self.cpu.hist[e][b][j])) * abs(float(a[j])) for j in range(k))

    def forecast_weights(self, b, t):
        h = self.cpu.t_hist[b]
        v = min(self.m, self.cpu.n_refs[b] - 1)
        w = [1.0]
        if self.basis == S.SPECA_BASIS_ADAMS_BASHFORTH:
            x, hh = t - h[0], (h[0] - h[1]) if len(h) > 1 else 0.0
            return w + [x * c * hh ** i for i, c in enumerate([1.0, 1 / 2, 5 / 12, 3 / 8][:v])]
        for i in range(1, v + 1):
            if self.basis == S.SPECA_BASIS_NEWTON:
                w.append(w[-1] * (t - h[i - 1]))
            else:
                w.append(w[-1] * (t - h[0]) / i)
        return w

    def check_forecast(self, t_target, active=None, sentinel=None, what="forecast"):
        """Runs forecast on both sides for all entries and compares. Returns the GPU outputs."""
        outs = []
        for (n, d) in self.entries:
            o = torch.empty(self.B, n, d, dtype=self.tdt, device=self.device)
            o.fill_(sentinel if sentinel is not None else 0.0)
            outs.append(o)
        mask_dev = None
        if active is not None:
            mask_dev = torch.tensor(active, dtype=torch.uint8, device=self.device)
        self.gpu.forecast(t_target, outs, mask_dev)
        torch.cuda.synchronize()
        for e in range(len(self.entries)):
            got = to_oracle(outs[e]).reshape(self.B, -1)
            init = got.copy()
            init[...] = to_oracle(torch.full((1,), sentinel if sentinel is not None else 0.0, dtype=self.tdt))[0]
            want = self.cpu.forecast_entry(e, t_target, active, out=init)
            for b in range(self.B):
                if (active is not None and not active[b]) or self.cpu.n_refs[b] < 1:
                    assert np.array_equal(got[b], want[b]), "%s: inactive sample %d of entry %d was written" % (what, b, e)
                    continue
                if self.layout == S.SPECA_LAYOUT_HISTORY:
                    scale = self.history_scale(e, b, t_target[b])
                else:
                    scale = term_scale(self.cpu.planes[e][b], self.forecast_weights(b, t_target[b]))
                assert_close_storage(got[b], want[b], self.dtype, scale, "%s entry %d sample %d" % (what, e, b))
        return outs

    def check_verify(self, fresh: torch.Tensor, t_target, tau, active=None, with_pred=True, what="verify", metric=None, ulp_slack=False):
        """ulp_slack: also allow the error to move by one storage ulp of the largest forecast value over
        the largest feature value. The l-infinity metric is decided by a single element, so a forecast
        that rounds the other way by one ulp (allowed: fp32 against fp64 evaluation) moves it by that much."""
        n, d = self.entries[self.vidx]
        err = torch.full((self.B,), -7.0, dtype=torch.float32, device=self.device)
        acc = torch.full((self.B,), 9, dtype=torch.uint8, device=self.device)
        pred = torch.zeros(self.B, n, d, dtype=self.tdt, device=self.device) if with_pred else None
        mask_dev = torch.tensor(active, dtype=torch.uint8, device=self.device) if active is not None else None
        self.gpu.verify(fresh, t_target, tau, err, acc, mask_dev, pred, metric=metric)
        torch.cuda.synchronize()
        e_want, a_want, p_want = self.cpu.verify(to_oracle(fresh).reshape(self.B, -1), t_target, tau, active,
                                                 metric=metric or 0)
        e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
        for b in range(self.B):
            if a_want[b] < 0:
                assert e_got[b] == -7.0 and a_got[b] == 9, "%s: skipped sample %d was written" % (what, b)
                continue
            if np.isnan(e_want[b]):
                assert np.isnan(e_got[b]) and a_got[b] == 0
                continue
            slack = 0.0
            if ulp_slack:
                pw, fw = as_f64(p_want[b]), as_f64(to_oracle(fresh[b]).reshape(-1))
                slack = float(storage_ulp(np.array([np.abs(pw).max()]), self.dtype)[0]) / (float(np.abs(fw).max()) + 1e-8)
            assert abs(e_got[b] - e_want[b]) <= ERR_TOL * max(1.0, e_want[b]) + slack, \
                "%s sample %d: err %g vs oracle %g" % (what, b, e_got[b], e_want[b])
            if abs(e_want[b] - float(np.float32(tau[b]))) >= ERR_TOL + slack:
                assert int(a_got[b]) == int(a_want[b]), "%s sample %d: decision differs (e=%g tau=%g)" % (
                    what, b, e_want[b], tau[b])
            else:
                assert int(a_got[b]) in (0, 1)
            if with_pred:
                if self.layout == S.SPECA_LAYOUT_HISTORY:
                    scale = self.history_scale(self.vidx, b, t_target[b])
                else:
                    scale = term_scale(self.cpu.planes[self.vidx][b], self.forecast_weights(b, t_target[b]))
                assert_close_storage(to_oracle(pred[b]).reshape(-1), p_want[b], self.dtype, scale,
                                     "%s pred sample %d" % (what, b))
        return e_got, a_got, e_want, a_want
