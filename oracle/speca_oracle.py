"""CPU oracle of the SpeCa feature-cache hot path (arXiv 2509.11628). TEST INFRASTRUCTURE ONLY.

Thin state keeping around ``speca_oracle.c`` (double arithmetic, one loop per equation). The class
mirrors the sequence of calls a sampler makes -- reference step (Eq. 3), speculative step (Eq. 2),
verification (Eq. 4 and the accept rule of Section 3.4.2), per-sample continuation -- so tests can
drive it and the CUDA library with the same inputs. It shares nothing with the CUDA path and must
never be imported by the product package.

Arrays are numpy: ``float32`` for fp32 storage, ``uint16`` holding bfloat16 bit patterns for bf16
storage. A tensor of entry ``e`` is ``[B, n_e]`` with ``n_e = tokens * dim`` (row-major flattening
of ``[B, N_e, D]``).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "speca_oracle.c")
_LIB = os.path.join(_HERE, "libspeca_oracle.so")

F32, BF16 = 0, 1
TAYLOR, NEWTON, ADAMS_BASHFORTH = 0, 1, 2
METRIC_L2, METRIC_L1, METRIC_LINF, METRIC_COSINE = 0, 1, 2, 3
LAYOUT_TABLES, LAYOUT_HISTORY = 0, 1   # what the cache keeps: difference quotients, or the raw features
EPS_PAPER = 1e-8  # Eq. 4


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP over elements) if it is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-shared", "-fPIC",
             "-std=c99", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        # SPECA_ORACLE_LIB: a library built elsewhere from (a variant of) speca_oracle.c; the mutation
        # tests use it to check that the pins notice mistakes planted in the C source
        L = ctypes.CDLL(os.environ.get("SPECA_ORACLE_LIB") or build())
        i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        dp = ctypes.POINTER(ctypes.c_double)
        L.oracle_update_segment.argtypes = [i32, i64, i32, i32, i32, dp, dbl, vp, vp, i64]
        L.oracle_update_segment.restype = i32
        L.oracle_forecast_segment.argtypes = [i32, i64, i32, i32, i32, dp, dbl, vp, i64, vp]
        L.oracle_forecast_segment.restype = i32
        L.oracle_forecast_history_segment.argtypes = [i32, i64, i32, i32, i32, dp, dbl, ctypes.POINTER(vp), vp]
        L.oracle_forecast_history_segment.restype = i32
        L.oracle_forecast_history_accumulate_segment.argtypes = [i32, i64, i32, i32, i32, dp, dbl, ctypes.POINTER(vp), vp]
        L.oracle_forecast_history_accumulate_segment.restype = i32
        L.oracle_forecast_accumulate_segment.argtypes = [i32, i64, i32, i32, i32, dp, dbl, vp, i64, vp]
        L.oracle_forecast_accumulate_segment.restype = i32
        L.oracle_accumulate_elems.argtypes = [i32, i64, vp, vp]
        L.oracle_accumulate_elems.restype = None
        L.oracle_round_store.argtypes = [i32, i64, vp, vp]
        L.oracle_round_store.restype = None
        L.oracle_rel_l2.argtypes = [i32, i64, vp, vp, dbl]
        L.oracle_rel_l2.restype = dbl
        for fn in (L.oracle_rel_l1, L.oracle_rel_linf, L.oracle_cos_dist):
            fn.argtypes = [i32, i64, vp, vp, dbl]
            fn.restype = dbl
        L.oracle_metric_sums.argtypes = [i32, i32, i64, vp, vp, dp]
        L.oracle_metric_sums.restype = None
        L.oracle_metric_from_sums.argtypes = [i32, dp, dbl]
        L.oracle_metric_from_sums.restype = dbl
        L.oracle_accept.argtypes = [dbl, dbl]
        L.oracle_accept.restype = i32
        L.oracle_tau.argtypes = [dbl, dbl, dbl, dbl]
        L.oracle_tau.restype = dbl
        L.oracle_speedup.argtypes = [dbl, dbl]
        L.oracle_speedup.restype = dbl
        L.oracle_double_to_bf16_bits.argtypes = [dbl]
        L.oracle_double_to_bf16_bits.restype = ctypes.c_uint16
        L.oracle_threads.restype = i32
        L.oracle_set_threads.argtypes = [i32]
        _lib = L
    return _lib


def np_dtype(dtype: int):
    return np.float32 if dtype == F32 else np.uint16


def _ptr(a: np.ndarray) -> ctypes.c_void_p:
    return ctypes.c_void_p(a.ctypes.data)


def _hist(t_hist: Sequence[float], m: int):
    buf = (ctypes.c_double * (m + 1))()
    for i, t in enumerate(list(t_hist)[: m + 1]):
        buf[i] = t
    return buf


# ---- stateless, one (entry, sample) segment ------------------------------------------------------

def update_segment(dtype, m, basis, n_refs, t_hist, t_new, feat: np.ndarray, planes: np.ndarray) -> None:
    """Eq. 3. ``planes`` is ``[m+1, n]`` (C-contiguous rows), rewritten in place."""
    assert planes.ndim == 2 and planes.shape[0] == m + 1 and planes.flags.c_contiguous
    assert feat.flags.c_contiguous and feat.dtype == planes.dtype == np_dtype(dtype)
    n = feat.size
    assert planes.shape[1] == n
    rc = lib().oracle_update_segment(dtype, n, m, basis, n_refs, _hist(t_hist, m), float(t_new),
                                     _ptr(feat), _ptr(planes), planes.strides[0] // planes.itemsize)
    if rc != 0:
        raise ZeroDivisionError("reference time repeats: zero gap")


def forecast_segment(dtype, m, basis, n_refs, t_hist, t_target, planes: np.ndarray, out: np.ndarray) -> None:
    """Eq. 2. Writes the forecast of one segment into ``out`` (``[n]``)."""
    assert planes.ndim == 2 and planes.shape[0] == m + 1 and planes.flags.c_contiguous
    assert out.flags.c_contiguous and out.dtype == planes.dtype == np_dtype(dtype)
    rc = lib().oracle_forecast_segment(dtype, out.size, m, basis, n_refs, _hist(t_hist, m), float(t_target),
                                       _ptr(planes), planes.strides[0] // planes.itemsize, _ptr(out))
    if rc != 0:
        raise RuntimeError("forecast from an empty table")


def forecast_history_segment(dtype, m, basis, t_hist, t_target, hist: Sequence[np.ndarray], out: np.ndarray) -> None:
    """Eq. 2-3 from the raw features of the last references: ``hist[0]`` at ``t_hist[0]`` (the latest),
    ``hist[1]`` the one before, ...; at most ``m + 1`` of them."""
    k = len(hist)
    assert 1 <= k <= m + 1 and len(t_hist) >= k
    assert all(h.flags.c_contiguous and h.dtype == np_dtype(dtype) and h.size == out.size for h in hist)
    assert out.flags.c_contiguous and out.dtype == np_dtype(dtype)
    ptrs = (ctypes.c_void_p * k)(*[h.ctypes.data for h in hist])
    rc = lib().oracle_forecast_history_segment(dtype, out.size, m, basis, k, _hist(t_hist, m), float(t_target), ptrs, _ptr(out))
    if rc != 0:
        raise RuntimeError("forecast from an empty history, or a repeated reference time")


def forecast_history_unrounded(dtype, m, basis, t_hist, t_target, hist: Sequence[np.ndarray]) -> np.ndarray:
    """The same forecast before it is rounded to the storage type, as float64 (tests use it to tell which
    elements sit so close to a rounding tie of the storage type that either neighbour is a correct result)."""
    k = len(hist)
    assert 1 <= k <= m + 1 and len(t_hist) >= k
    n = hist[0].size
    assert all(h.flags.c_contiguous and h.dtype == np_dtype(dtype) and h.size == n for h in hist)
    acc = np.zeros(n, dtype=np.float64)
    ptrs = (ctypes.c_void_p * k)(*[h.ctypes.data for h in hist])
    rc = lib().oracle_forecast_history_accumulate_segment(dtype, n, m, basis, k, _hist(t_hist, m), float(t_target), ptrs, _ptr(acc))
    if rc != 0:
        raise RuntimeError("forecast from an empty history, or a repeated reference time")
    return acc


def rel_l2(dtype, pred: np.ndarray, fresh: np.ndarray, eps: float = EPS_PAPER) -> float:
    """Eq. 4 over one sample."""
    assert pred.flags.c_contiguous and fresh.flags.c_contiguous and pred.size == fresh.size
    assert pred.dtype == fresh.dtype == np_dtype(dtype)
    return float(lib().oracle_rel_l2(dtype, pred.size, _ptr(pred), _ptr(fresh), float(eps)))


def rel_err(metric: int, dtype, pred: np.ndarray, fresh: np.ndarray, eps: float = EPS_PAPER) -> float:
    """Eq. 4 (metric 0) or one of the appendix's other metrics over one sample."""
    assert pred.flags.c_contiguous and fresh.flags.c_contiguous and pred.size == fresh.size
    assert pred.dtype == fresh.dtype == np_dtype(dtype)
    fn = {METRIC_L2: lib().oracle_rel_l2, METRIC_L1: lib().oracle_rel_l1, METRIC_LINF: lib().oracle_rel_linf,
          METRIC_COSINE: lib().oracle_cos_dist}[metric]
    return float(fn(dtype, pred.size, _ptr(pred), _ptr(fresh), float(eps)))


def metric_sums(metric: int, dtype, pred: np.ndarray, fresh: np.ndarray):
    """Running values of one part of a sample (sums; maxima for l-infinity): [a0, a1, a2]."""
    assert pred.flags.c_contiguous and fresh.flags.c_contiguous and pred.size == fresh.size
    out = (ctypes.c_double * 3)()
    lib().oracle_metric_sums(metric, dtype, pred.size, _ptr(pred), _ptr(fresh), out)
    return [out[0], out[1], out[2]]


def metric_from_sums(metric: int, sums: Sequence[float], eps: float = EPS_PAPER) -> float:
    buf = (ctypes.c_double * 3)(*[float(x) for x in sums])
    return float(lib().oracle_metric_from_sums(metric, buf, float(eps)))


def accept(err: float, tau: float) -> bool:
    return bool(lib().oracle_accept(float(err), float(tau)))


def tau_schedule(tau0: float, beta: float, t: float, T: float) -> float:
    return float(lib().oracle_tau(tau0, beta, t, T))


def speedup(alpha: float, gamma: float) -> float:
    return float(lib().oracle_speedup(alpha, gamma))


def to_bf16_bits(x: float) -> int:
    return int(lib().oracle_double_to_bf16_bits(float(x)))


def threads() -> int:
    return int(lib().oracle_threads())


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def select_adaptive(accept_flags, k_max: int, group: int, spec_count, active):
    """Sequential validation + forced activation period + group fate sharing (Section 3.4.2,
    Appendix A). Pure integer logic; returns (active', spec_count', idx list)."""
    B = len(active)
    assert B % group == 0 and k_max >= 1
    count = [int(c) for c in spec_count]
    keep = [0] * B
    for b in range(B):
        if active[b]:
            if accept_flags[b]:
                count[b] += 1
            keep[b] = 1 if (accept_flags[b] and count[b] < k_max) else 0
    new_active = [0] * B
    for g in range(0, B, group):
        ok = all(keep[g + i] for i in range(group))
        for i in range(group):
            new_active[g + i] = 1 if ok else 0
    idx = [b for b in range(B) if new_active[b]]
    return new_active, count, idx


# ---- stateful mirror of the library's call sequence ----------------------------------------------

class OracleCache:
    """Derivative tables for a list of entries, with per-sample reference history."""

    def __init__(self, entry_elems: Sequence[int], batch: int, max_order: int, dtype: int,
                 basis: int = TAYLOR, verify_entry: int = -1, eps: float = EPS_PAPER, layout: int = LAYOUT_TABLES):
        self.entry_elems = [int(n) for n in entry_elems]
        self.B, self.m, self.dtype, self.basis = batch, max_order, dtype, basis
        self.layout = layout
        # LAYOUT_HISTORY: hist[e][b] = stored features of the last <= m + 1 references, latest first
        self.hist: List[List[List[np.ndarray]]] = [[[] for _ in range(batch)] for _ in self.entry_elems]
        self.verify_entry = verify_entry if verify_entry >= 0 else len(self.entry_elems) - 1
        self.eps = eps
        self.planes: List[np.ndarray] = [np.zeros((batch, max_order + 1, n), dtype=np_dtype(dtype))
                                         for n in self.entry_elems]
        self.n_refs = [0] * batch
        self.t_hist: List[List[float]] = [[] for _ in range(batch)]
        self._pending = None  # (t_ref, mask)

    def update(self, feats: Sequence[Optional[np.ndarray]], t_ref: Sequence[float],
               mask: Optional[Sequence[int]] = None) -> None:
        mask = [1] * self.B if mask is None else [int(bool(x)) for x in mask]
        self._pending = (list(t_ref), mask)
        for e, f in enumerate(feats):
            if f is None:
                continue
            f = np.ascontiguousarray(f).reshape(self.B, self.entry_elems[e])
            for b in range(self.B):
                if mask[b] and self.layout == LAYOUT_HISTORY:
                    if self.n_refs[b] >= 1 and float(t_ref[b]) == self.t_hist[b][0]:
                        raise ZeroDivisionError("reference time repeats: zero gap")
                    kept = self.hist[e][b] if self.n_refs[b] >= 1 else []   # a reset sample starts over
                    self.hist[e][b] = ([f[b].copy()] + kept)[: self.m + 1]
                elif mask[b]:
                    update_segment(self.dtype, self.m, self.basis, self.n_refs[b], self.t_hist[b], t_ref[b],
                                   f[b], self.planes[e][b])

    def commit_step(self) -> None:
        t_ref, mask = self._pending
        for b in range(self.B):
            if mask[b]:
                self.t_hist[b] = ([float(t_ref[b])] + self.t_hist[b])[: self.m + 1]
                self.n_refs[b] += 1
        self._pending = None

    def reset(self, mask: Optional[Sequence[int]] = None) -> None:
        for b in range(self.B):
            if mask is None or mask[b]:
                self.n_refs[b] = 0
                self.t_hist[b] = []

    def forecast_entry(self, e: int, t_target: Sequence[float], active: Optional[Sequence[int]] = None,
                       out: Optional[np.ndarray] = None) -> np.ndarray:
        if out is None:
            out = np.zeros((self.B, self.entry_elems[e]), dtype=np_dtype(self.dtype))
        for b in range(self.B):
            if (active is None or active[b]) and self.n_refs[b] >= 1:
                if self.layout == LAYOUT_HISTORY:
                    forecast_history_segment(self.dtype, self.m, self.basis, self.t_hist[b], t_target[b],
                                             self.hist[e][b][: min(self.n_refs[b], self.m + 1)], out[b])
                else:
                    forecast_segment(self.dtype, self.m, self.basis, self.n_refs[b], self.t_hist[b], t_target[b],
                                     self.planes[e][b], out[b])
        return out

    def forecast_multi(self, e: int, t_targets: Sequence[Sequence[float]], active: Optional[Sequence[int]] = None,
                       out: Optional[np.ndarray] = None) -> np.ndarray:
        """Eq. 2 for K speculative steps from the same table (Fig. 1: the draft predicts the next
        steps t-1 .. t-K): simply K forecasts. Returns [K, B, n_e]."""
        K = len(t_targets)
        if out is None:
            out = np.zeros((K, self.B, self.entry_elems[e]), dtype=np_dtype(self.dtype))
        for k in range(K):
            self.forecast_entry(e, t_targets[k], active, out=out[k])
        return out

    def forecast_sum(self, entry_ids: Sequence[int], t_target: Sequence[float], base: Optional[np.ndarray] = None,
                     active: Optional[Sequence[int]] = None, out: Optional[np.ndarray] = None) -> np.ndarray:
        """out[b] = round(base[b] + sum over the listed entries of their unrounded forecasts), the form
        in which a residual stream consumes the forecasts of equally shaped blocks. Inactive samples
        keep what `out` held."""
        n = self.entry_elems[entry_ids[0]]
        assert all(self.entry_elems[e] == n for e in entry_ids)
        if out is None:
            out = np.zeros((self.B, n), dtype=np_dtype(self.dtype))
        for b in range(self.B):
            if (active is not None and not active[b]) or self.n_refs[b] < 1:
                continue
            acc = np.zeros(n, dtype=np.float64)
            if base is not None:
                lib().oracle_accumulate_elems(self.dtype, n, _ptr(np.ascontiguousarray(base[b])), _ptr(acc))
            for e in entry_ids:
                if self.layout == LAYOUT_HISTORY:
                    hist = self.hist[e][b][: min(self.n_refs[b], self.m + 1)]
                    ptrs = (ctypes.c_void_p * len(hist))(*[h.ctypes.data for h in hist])
                    rc = lib().oracle_forecast_history_accumulate_segment(self.dtype, n, self.m, self.basis, len(hist),
                                                                          _hist(self.t_hist[b], self.m), float(t_target[b]),
                                                                          ptrs, _ptr(acc))
                    assert rc == 0
                    continue
                p = self.planes[e][b]
                rc = lib().oracle_forecast_accumulate_segment(self.dtype, n, self.m, self.basis, self.n_refs[b],
                                                              _hist(self.t_hist[b], self.m), float(t_target[b]),
                                                              _ptr(p), p.strides[0] // p.itemsize, _ptr(acc))
                assert rc == 0
            lib().oracle_round_store(self.dtype, n, _ptr(acc), _ptr(out[b]))
        return out

    def verify(self, fresh: np.ndarray, t_target: Sequence[float], tau: Sequence[float],
               active: Optional[Sequence[int]] = None, metric: int = METRIC_L2):
        """Returns (err[B] float64 with NaN for skipped samples, accept[B] int with -1 for skipped,
        pred [B, n_v])."""
        e = self.verify_entry
        fresh = np.ascontiguousarray(fresh).reshape(self.B, self.entry_elems[e])
        pred = self.forecast_entry(e, t_target, active)
        err = np.full(self.B, np.nan)
        acc = np.full(self.B, -1, dtype=np.int64)
        for b in range(self.B):
            if (active is None or active[b]) and self.n_refs[b] >= 1:
                err[b] = rel_err(metric, self.dtype, pred[b], fresh[b], self.eps)
                acc[b] = 1 if accept(err[b], float(np.float32(tau[b]))) else 0
        return err, acc, pred
