"""ctypes binding of ``libspeca.so``: the same entry points as ``include/speca.h``.

Argument marshalling only -- every arithmetic step runs in the CUDA kernels behind the C ABI.
Device buffers are torch tensors (or raw integer addresses); host arrays are Python sequences.
There is no fallback: if the library is missing or cannot be loaded, importing the entry points
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libspeca.so")

SPECA_OK = 0
SPECA_ERR_INVALID_ARG, SPECA_ERR_SHAPE, SPECA_ERR_ALIGNMENT, SPECA_ERR_STATE = 1, 2, 3, 4
SPECA_ERR_ZERO_GAP, SPECA_ERR_NOMEM, SPECA_ERR_CUDA, SPECA_ERR_UNSUPPORTED = 5, 6, 7, 8
SPECA_F32, SPECA_BF16 = 0, 1
SPECA_BASIS_TAYLOR, SPECA_BASIS_NEWTON, SPECA_BASIS_ADAMS_BASHFORTH = 0, 1, 2
SPECA_METRIC_L2, SPECA_METRIC_L1, SPECA_METRIC_LINF, SPECA_METRIC_COSINE = 0, 1, 2, 3
SPECA_PATH_AUTO, SPECA_PATH_DIRECT, SPECA_PATH_BULK, SPECA_PATH_WIDE = 0, 1, 2, 3
SPECA_LAYOUT_TABLES, SPECA_LAYOUT_HISTORY = 0, 1
SPECA_FEATURE_IN_PLACE = 1   # as feats[entry]: the features already sit in the planes speca_cache_next_slot names
SPECA_MAX_ORDER, SPECA_MAX_BATCH, SPECA_MAX_ENTRIES, SPECA_MAX_HORIZON = 4, 64, 512, 8

EXPORTS = [
    "speca_cache_arena_bytes", "speca_cache_create", "speca_cache_destroy", "speca_cache_reset",
    "speca_cache_update", "speca_cache_update_activate", "speca_cache_update_forecast", "speca_cache_update_forecast_multi", "speca_cache_commit_step", "speca_forecast", "speca_verify",
    "speca_select_adaptive", "speca_activate", "speca_tau", "speca_cache_state", "speca_cache_plane",
    "speca_cache_launch_count", "speca_cache_stats", "speca_cache_check", "speca_cache_next_slot", "speca_forecast_weights", "speca_status_string", "speca_last_error", "speca_version",
    "speca_verify_pred_static", "speca_forecast_multi", "speca_verify_metric",
    "speca_verify_partial", "speca_verify_decide", "speca_cache_get_history", "speca_cache_set_history",
    "speca_forecast_sum", "speca_verify_select",
]


class SpecaError(RuntimeError):
    def __init__(self, status: int, detail: str = ""):
        self.status = status
        name = _lib().speca_status_string(status).decode()
        super().__init__("speca status %d (%s)%s" % (status, name, (": " + detail) if detail else ""))


class EntryDesc(ctypes.Structure):
    _fields_ = [("tokens", ctypes.c_int64), ("dim", ctypes.c_int32)]


class CacheStats(ctypes.Structure):
    _fields_ = [(name, ctypes.c_uint64) for name in (
        "update_launches", "forecast_launches", "forecast_multi_launches", "forecast_sum_launches",
        "verify_launches", "select_launches", "activate_launches", "update_forecast_launches")] + [
        ("reference_steps", ctypes.c_uint64 * 64), ("resets", ctypes.c_uint64 * 64)]


class CacheConfig(ctypes.Structure):
    _fields_ = [
        ("n_entries", ctypes.c_int32), ("entries", ctypes.POINTER(EntryDesc)), ("batch", ctypes.c_int32),
        ("max_order", ctypes.c_int32), ("dtype", ctypes.c_int32), ("basis", ctypes.c_int32),
        ("verify_entry", ctypes.c_int32), ("eps", ctypes.c_float), ("arena", ctypes.c_void_p),
        ("arena_bytes", ctypes.c_size_t), ("device", ctypes.c_int32), ("path", ctypes.c_int32),
        ("layout", ctypes.c_int32),
    ]


_LIB = None


def _lib() -> ctypes.CDLL:
    global _LIB
    if _LIB is not None:
        return _LIB
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libspeca.so is not built (%s). Run `python -m paper_2509_11628_b200.build`; "
            "there is no CPU fallback." % LIB_PATH)
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_double
    cfgp = ctypes.POINTER(CacheConfig)
    L.speca_cache_arena_bytes.argtypes = [cfgp, ctypes.POINTER(ctypes.c_size_t)]
    L.speca_cache_create.argtypes = [cfgp, ctypes.POINTER(vp)]
    L.speca_cache_destroy.argtypes = [vp]
    L.speca_cache_reset.argtypes = [vp, vp]
    L.speca_cache_update.argtypes = [vp, vp, vp, vp, vp]
    L.speca_cache_update_activate.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.speca_cache_update_forecast.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.speca_cache_update_forecast_multi.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, vp, vp, vp]
    L.speca_cache_commit_step.argtypes = [vp]
    L.speca_forecast.argtypes = [vp, vp, vp, vp, vp]
    L.speca_forecast_sum.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    L.speca_forecast_multi.argtypes = [vp, i32, vp, vp, vp, vp]
    L.speca_verify.argtypes = [vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.speca_verify_metric.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
    L.speca_verify_select.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    L.speca_verify_partial.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp]
    L.speca_verify_decide.argtypes = [i32, vp, i32, vp, ctypes.c_float, vp, vp, vp, vp]
    L.speca_select_adaptive.argtypes = [vp, vp, i32, i32, vp, vp, vp, vp, vp]
    L.speca_activate.argtypes = [vp, vp, vp, vp, vp]
    L.speca_verify_pred_static.argtypes = [vp, vp, ctypes.c_int64, i32, i32, vp, ctypes.c_float, vp, vp, vp, i32, vp]
    L.speca_tau.argtypes = [dbl, dbl, dbl, dbl]
    L.speca_tau.restype = dbl
    L.speca_cache_state.argtypes = [vp, vp, vp]
    L.speca_cache_get_history.argtypes = [vp, vp, vp]
    L.speca_cache_set_history.argtypes = [vp, vp, vp]
    L.speca_cache_plane.argtypes = [vp, i32, i32, ctypes.POINTER(vp), ctypes.POINTER(ctypes.c_size_t)]
    L.speca_cache_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_uint64)]
    L.speca_cache_stats.argtypes = [vp, ctypes.POINTER(CacheStats)]
    L.speca_cache_check.argtypes = [vp, vp]
    L.speca_cache_next_slot.argtypes = [vp, i32, i32, ctypes.POINTER(vp)]
    L.speca_forecast_weights.argtypes = [i32, i32, i32, i32, vp, dbl, ctypes.POINTER(i32), vp]
    L.speca_status_string.argtypes = [i32]
    L.speca_status_string.restype = ctypes.c_char_p
    L.speca_last_error.argtypes = [vp]
    L.speca_last_error.restype = ctypes.c_char_p
    L.speca_version.restype = ctypes.c_char_p
    for name in EXPORTS:
        if getattr(L, name).restype is ctypes.c_int:  # default restype: status codes
            getattr(L, name).restype = i32
    _LIB = L
    return L


# ---- marshalling helpers -------------------------------------------------------------------------

def _dev_ptr(x) -> Optional[int]:
    """torch CUDA tensor / int address / None -> integer address or None."""
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        if not x.is_cuda:
            raise TypeError("device buffer expected, got a CPU tensor")
        if not x.is_contiguous():
            raise TypeError("device buffers must be contiguous")
        return x.data_ptr()
    return int(x)


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream or None
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream or None
    return int(stream) or None


def _doubles(xs: Sequence[float]):
    return (ctypes.c_double * len(xs))(*[float(x) for x in xs])


def _floats(xs: Sequence[float]):
    return (ctypes.c_float * len(xs))(*[float(x) for x in xs])


def _bytes(xs: Optional[Sequence[int]]):
    if xs is None:
        return None
    return (ctypes.c_uint8 * len(xs))(*[1 if x else 0 for x in xs])


def _ptr_array(xs: Sequence):
    return (ctypes.c_void_p * len(xs))(*[_dev_ptr(x) for x in xs])


def _check(status: int, handle=None):
    if status != SPECA_OK:
        detail = _lib().speca_last_error(handle).decode() if handle else ""
        raise SpecaError(status, detail)


def _config(entries, batch, max_order, dtype, basis, verify_entry, eps, arena, arena_bytes, device, path,
            layout=SPECA_LAYOUT_TABLES):
    arr = (EntryDesc * len(entries))(*[EntryDesc(int(n), int(d)) for n, d in entries])
    cfg = CacheConfig(len(entries), arr, batch, max_order, dtype, basis, verify_entry, eps,
                      _dev_ptr(arena), arena_bytes, device, path, layout)
    cfg._keep = arr
    return cfg


# ---- the entry points, same names as the header ----------------------------------------------------

def speca_cache_arena_bytes(entries, batch, max_order, dtype, basis=SPECA_BASIS_TAYLOR, verify_entry=-1,
                            path=SPECA_PATH_AUTO, layout=SPECA_LAYOUT_TABLES) -> int:
    cfg = _config(entries, batch, max_order, dtype, basis, verify_entry, 0.0, None, 0, 0, path, layout)
    out = ctypes.c_size_t(0)
    _check(_lib().speca_cache_arena_bytes(ctypes.byref(cfg), ctypes.byref(out)))
    return out.value


def speca_cache_create(entries, batch, max_order, dtype, arena, basis=SPECA_BASIS_TAYLOR, verify_entry=-1,
                       eps=0.0, device=None, path=SPECA_PATH_AUTO, arena_bytes=None, layout=SPECA_LAYOUT_TABLES) -> int:
    """Returns the opaque handle (an integer address). ``arena`` is a CUDA uint8 tensor the caller
    keeps alive, or a raw device address together with ``arena_bytes``."""
    if isinstance(arena, torch.Tensor):
        if device is None:
            device = arena.device.index
        if arena_bytes is None:
            arena_bytes = arena.numel() * arena.element_size()
    cfg = _config(entries, batch, max_order, dtype, basis, verify_entry, eps, arena, arena_bytes or 0,
                  device or 0, path, layout)
    out = ctypes.c_void_p(None)
    _check(_lib().speca_cache_create(ctypes.byref(cfg), ctypes.byref(out)))
    return out.value


def speca_cache_destroy(cache) -> None:
    _check(_lib().speca_cache_destroy(cache))


def speca_cache_reset(cache, host_sample_mask=None) -> None:
    _check(_lib().speca_cache_reset(cache, _bytes(host_sample_mask)), cache)


def speca_cache_update(cache, feats, t_ref, host_sample_mask=None, stream=None) -> None:
    _check(_lib().speca_cache_update(cache, _ptr_array(feats), _doubles(t_ref), _bytes(host_sample_mask),
                                     _stream_ptr(stream)), cache)


def speca_cache_update_activate(cache, feats, t_ref, host_sample_mask, dev_spec_count, dev_active_mask, stream=None) -> None:
    """speca_cache_update + speca_activate for the masked samples in one launch."""
    _check(_lib().speca_cache_update_activate(cache, _ptr_array(feats), _doubles(t_ref), _bytes(host_sample_mask),
                                              _dev_ptr(dev_spec_count), _dev_ptr(dev_active_mask), _stream_ptr(stream)), cache)


def speca_cache_update_forecast(cache, feats, t_ref, host_sample_mask, t_target, dev_active_mask, outs, dev_spec_count=None,
                                dev_rearm_mask=None, stream=None) -> None:
    """A whole reference step (update + commit) and the forecast at t_target in one launch."""
    _check(_lib().speca_cache_update_forecast(cache, _ptr_array(feats), _doubles(t_ref), _bytes(host_sample_mask),
                                              _doubles(t_target), _dev_ptr(dev_active_mask), _ptr_array(outs),
                                              _dev_ptr(dev_spec_count), _dev_ptr(dev_rearm_mask), _stream_ptr(stream)), cache)


def speca_cache_update_forecast_multi(cache, feats, t_ref, host_sample_mask, t_targets, dev_active_mask, outs,
                                      dev_spec_count=None, dev_rearm_mask=None, stream=None) -> None:
    """The same with K speculative times: t_targets is K lists of B times, outs[e] a [K, B, N_e, D] tensor."""
    flat = [t for row in t_targets for t in row]
    _check(_lib().speca_cache_update_forecast_multi(cache, _ptr_array(feats), _doubles(t_ref), _bytes(host_sample_mask),
                                                    len(t_targets), _doubles(flat), _dev_ptr(dev_active_mask), _ptr_array(outs),
                                                    _dev_ptr(dev_spec_count), _dev_ptr(dev_rearm_mask), _stream_ptr(stream)), cache)


def speca_cache_commit_step(cache) -> None:
    _check(_lib().speca_cache_commit_step(cache), cache)


def speca_forecast(cache, t_target, dev_active_mask, outs, stream=None) -> None:
    _check(_lib().speca_forecast(cache, _doubles(t_target), _dev_ptr(dev_active_mask), _ptr_array(outs),
                                 _stream_ptr(stream)), cache)


def speca_forecast_sum(cache, entry_ids, t_target, dev_active_mask, base, out, stream=None) -> None:
    """out = base + sum of the forecasts of the listed (equally shaped) entries; base may be None."""
    ids = (ctypes.c_int32 * len(entry_ids))(*[int(e) for e in entry_ids])
    _check(_lib().speca_forecast_sum(cache, ids, len(entry_ids), _doubles(t_target), _dev_ptr(dev_active_mask),
                                     _dev_ptr(base), _dev_ptr(out), _stream_ptr(stream)), cache)


def speca_forecast_multi(cache, t_targets, dev_active_mask, outs, stream=None) -> None:
    """``t_targets``: K lists of B times; ``outs[e]``: device tensor [K, B, N_e, D] (None = skip)."""
    flat = [float(t) for row in t_targets for t in row]
    _check(_lib().speca_forecast_multi(cache, len(t_targets), _doubles(flat), _dev_ptr(dev_active_mask),
                                       _ptr_array(outs), _stream_ptr(stream)), cache)


def speca_verify(cache, fresh, t_target, tau, dev_active_mask, out_pred, dev_err, dev_accept, stream=None) -> None:
    _check(_lib().speca_verify(cache, _dev_ptr(fresh), _doubles(t_target), _floats(tau), _dev_ptr(dev_active_mask),
                               _dev_ptr(out_pred), _dev_ptr(dev_err), _dev_ptr(dev_accept), _stream_ptr(stream)),
           cache)


def speca_verify_metric(cache, metric, fresh, t_target, tau, dev_active_mask, out_pred, dev_err, dev_accept,
                        stream=None) -> None:
    _check(_lib().speca_verify_metric(cache, int(metric), _dev_ptr(fresh), _doubles(t_target), _floats(tau),
                                      _dev_ptr(dev_active_mask), _dev_ptr(out_pred), _dev_ptr(dev_err),
                                      _dev_ptr(dev_accept), _stream_ptr(stream)), cache)


def speca_verify_select(cache, metric, fresh, t_target, tau, dev_active_mask, dev_next_active_mask, out_pred, dev_err,
                        dev_accept, k_max, group, dev_spec_count, dev_active_idx=None, dev_n_active=None, stream=None) -> None:
    """speca_verify_metric + speca_select_adaptive in one launch; the next mask goes to its own buffer."""
    _check(_lib().speca_verify_select(cache, int(metric), _dev_ptr(fresh), _doubles(t_target), _floats(tau),
                                      _dev_ptr(dev_active_mask), _dev_ptr(dev_next_active_mask), _dev_ptr(out_pred),
                                      _dev_ptr(dev_err), _dev_ptr(dev_accept), int(k_max), int(group),
                                      _dev_ptr(dev_spec_count), _dev_ptr(dev_active_idx), _dev_ptr(dev_n_active),
                                      _stream_ptr(stream)), cache)


def speca_verify_partial(cache, metric, fresh, t_target, dev_active_mask, out_pred, dev_sums, stream=None) -> None:
    """``dev_sums``: CUDA float64 tensor [B, 4] that receives the metric's running values of this shard."""
    _check(_lib().speca_verify_partial(cache, int(metric), _dev_ptr(fresh), _doubles(t_target), _dev_ptr(dev_active_mask),
                                       _dev_ptr(out_pred), _dev_ptr(dev_sums), _stream_ptr(stream)), cache)


def speca_verify_decide(metric, dev_sums, batch, tau, eps, dev_active_mask, dev_err, dev_accept, stream=None) -> None:
    _check(_lib().speca_verify_decide(int(metric), _dev_ptr(dev_sums), int(batch), _floats(tau), float(eps),
                                      _dev_ptr(dev_active_mask), _dev_ptr(dev_err), _dev_ptr(dev_accept),
                                      _stream_ptr(stream)))


def speca_select_adaptive(cache, dev_accept, k_max, group, dev_spec_count, dev_active_mask, dev_active_idx=None,
                          dev_n_active=None, stream=None) -> None:
    _check(_lib().speca_select_adaptive(cache, _dev_ptr(dev_accept), int(k_max), int(group), _dev_ptr(dev_spec_count),
                                        _dev_ptr(dev_active_mask), _dev_ptr(dev_active_idx), _dev_ptr(dev_n_active),
                                        _stream_ptr(stream)), cache)


def speca_activate(cache, host_sample_mask, dev_spec_count, dev_active_mask, stream=None) -> None:
    _check(_lib().speca_activate(cache, _bytes(host_sample_mask), _dev_ptr(dev_spec_count), _dev_ptr(dev_active_mask),
                                 _stream_ptr(stream)), cache)


def speca_verify_pred_static(pred, fresh, n_elems, batch, dtype, tau, eps, dev_active_mask, dev_err, dev_accept,
                             device=0, stream=None) -> None:
    """Eq. 4 + accept rule on a forecast the caller holds, with the reduction scratch inside the
    library image: for callers that cannot allocate device memory or hand over an arena. Calls
    whose kernels overlap on the GPU race on that shared scratch; keep them in stream order."""
    _check(_lib().speca_verify_pred_static(_dev_ptr(pred), _dev_ptr(fresh), int(n_elems), int(batch), int(dtype),
                                           _floats(tau), float(eps), _dev_ptr(dev_active_mask), _dev_ptr(dev_err),
                                           _dev_ptr(dev_accept), int(device), _stream_ptr(stream)))


def speca_tau(tau0: float, beta: float, t: float, T: float) -> float:
    return float(_lib().speca_tau(tau0, beta, t, T))


def speca_cache_state(cache, batch: int):
    n = (ctypes.c_int32 * batch)()
    t = (ctypes.c_double * batch)()
    _check(_lib().speca_cache_state(cache, n, t), cache)
    return list(n), list(t)


def speca_cache_get_history(cache, batch: int):
    """(n_refs[B], t_hist[B][SPECA_MAX_ORDER + 1]) -- with the arena bytes, everything a checkpoint needs."""
    n = (ctypes.c_int32 * batch)()
    t = (ctypes.c_double * (batch * (SPECA_MAX_ORDER + 1)))()
    _check(_lib().speca_cache_get_history(cache, n, t), cache)
    w = SPECA_MAX_ORDER + 1
    return list(n), [list(t[b * w:(b + 1) * w]) for b in range(batch)]


def speca_cache_set_history(cache, n_refs, t_hist) -> None:
    n = (ctypes.c_int32 * len(n_refs))(*[int(x) for x in n_refs])
    flat = [float(x) for row in t_hist for x in row]
    t = (ctypes.c_double * len(flat))(*flat)
    _check(_lib().speca_cache_set_history(cache, n, t), cache)


def speca_cache_plane(cache, entry: int, sample: int):
    p = ctypes.c_void_p(None)
    s = ctypes.c_size_t(0)
    _check(_lib().speca_cache_plane(cache, entry, sample, ctypes.byref(p), ctypes.byref(s)), cache)
    return p.value, s.value


def speca_forecast_weights(layout: int, basis: int, max_order: int, n_refs: int, t_hist: Sequence[float], t_target: float):
    """(order, coefficients) a forecast at ``t_target`` hands to the kernels; host only, no GPU needed."""
    order = ctypes.c_int32(0)
    coef = (ctypes.c_float * (SPECA_MAX_ORDER + 1))()
    _check(_lib().speca_forecast_weights(layout, basis, max_order, n_refs, _doubles(t_hist), float(t_target),
                                         ctypes.byref(order), coef))
    return order.value, [float(x) for x in coef]


def speca_cache_next_slot(cache, entry: int, sample: int) -> int:
    """Device address of the plane the next reference step of ``sample`` fills for ``entry`` (raw-feature cache)."""
    out = ctypes.c_void_p(None)
    _check(_lib().speca_cache_next_slot(cache, int(entry), int(sample), ctypes.byref(out)), cache)
    return out.value


def speca_cache_stats(cache, batch: int) -> dict:
    """Host-side counters of the handle: launches per kernel kind, reference steps and resets per sample."""
    st = CacheStats()
    _check(_lib().speca_cache_stats(cache, ctypes.byref(st)), cache)
    out = {name: int(getattr(st, name)) for name, _ in CacheStats._fields_[:8]}
    out["reference_steps"] = [int(x) for x in st.reference_steps[:batch]]
    out["resets"] = [int(x) for x in st.resets[:batch]]
    return out


def speca_cache_check(cache, stream=None) -> None:
    _check(_lib().speca_cache_check(cache, _stream_ptr(stream)), cache)


def speca_cache_launch_count(cache) -> int:
    n = ctypes.c_uint64(0)
    _check(_lib().speca_cache_launch_count(cache, ctypes.byref(n)), cache)
    return n.value


def speca_status_string(status: int) -> str:
    return _lib().speca_status_string(status).decode()


def speca_last_error(cache) -> str:
    return _lib().speca_last_error(cache).decode()


def speca_version() -> str:
    return _lib().speca_version().decode()


class SpecaCache:
    """Owns an arena tensor and a handle; forwards to the entry points above."""

    def __init__(self, entries, batch, max_order, dtype, device="cuda:0", basis=SPECA_BASIS_TAYLOR,
                 verify_entry=-1, eps=0.0, path=SPECA_PATH_AUTO, layout=SPECA_LAYOUT_TABLES):
        self.entries = [(int(n), int(d)) for n, d in entries]
        self.batch, self.max_order, self.dtype, self.basis = batch, max_order, dtype, basis
        self.layout, self.path = layout, path
        self.device = torch.device(device)
        self.verify_entry = verify_entry if verify_entry >= 0 else len(self.entries) - 1
        nbytes = speca_cache_arena_bytes(self.entries, batch, max_order, dtype, basis, verify_entry, path, layout)
        self.arena = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        assert self.arena.data_ptr() % 256 == 0
        self.handle = speca_cache_create(self.entries, batch, max_order, dtype, self.arena, basis, verify_entry,
                                         eps, self.device.index or 0, path, layout=layout)

    def close(self):
        if self.handle:
            speca_cache_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def update(self, feats, t_ref, mask=None, stream=None):
        speca_cache_update(self.handle, feats, t_ref, mask, stream)

    def update_activate(self, feats, t_ref, mask, spec_count, active, stream=None):
        speca_cache_update_activate(self.handle, feats, t_ref, mask, spec_count, active, stream)

    def update_forecast(self, feats, t_ref, t_target, outs, mask=None, active=None, spec_count=None, rearm=None, stream=None):
        """A whole reference step and the first forecast after it in one launch (commits the step)."""
        speca_cache_update_forecast(self.handle, feats, t_ref, mask, t_target, active, outs, spec_count, rearm, stream)

    def update_forecast_multi(self, feats, t_ref, t_targets, outs, mask=None, active=None, spec_count=None, rearm=None, stream=None):
        """The same for K speculative times: outs[e] is [K, B, N_e, D]."""
        speca_cache_update_forecast_multi(self.handle, feats, t_ref, mask, t_targets, active, outs, spec_count, rearm, stream)

    def commit_step(self):
        speca_cache_commit_step(self.handle)

    def forecast(self, t_target, outs, active=None, stream=None):
        speca_forecast(self.handle, t_target, active, outs, stream)

    def forecast_sum(self, entry_ids, t_target, out, base=None, active=None, stream=None):
        speca_forecast_sum(self.handle, entry_ids, t_target, active, base, out, stream)

    def forecast_multi(self, t_targets, outs, active=None, stream=None):
        speca_forecast_multi(self.handle, t_targets, active, outs, stream)

    def verify(self, fresh, t_target, tau, err, accept, active=None, out_pred=None, stream=None, metric=None):
        if metric is None:
            speca_verify(self.handle, fresh, t_target, tau, active, out_pred, err, accept, stream)
        else:
            speca_verify_metric(self.handle, metric, fresh, t_target, tau, active, out_pred, err, accept, stream)

    def verify_select(self, fresh, t_target, tau, err, accept, active, next_active, k_max, group, spec_count, idx=None,
                      n_active=None, out_pred=None, stream=None, metric=0):
        speca_verify_select(self.handle, metric, fresh, t_target, tau, active, next_active, out_pred, err, accept, k_max,
                            group, spec_count, idx, n_active, stream)

    def select_adaptive(self, accept, k_max, group, spec_count, active, idx=None, n_active=None, stream=None):
        speca_select_adaptive(self.handle, accept, k_max, group, spec_count, active, idx, n_active, stream)

    def activate(self, mask, spec_count, active, stream=None):
        speca_activate(self.handle, mask, spec_count, active, stream)

    def reset(self, mask=None):
        speca_cache_reset(self.handle, mask)

    def state(self):
        return speca_cache_state(self.handle, self.batch)

    def plane_tensor(self, entry: int, sample: int) -> torch.Tensor:
        """View of the (entry, sample) table as ``[m+1, n_elems]`` in the storage dtype."""
        ptr, stride = speca_cache_plane(self.handle, entry, sample)
        esz = 2 if self.dtype == SPECA_BF16 else 4
        tdt = torch.bfloat16 if self.dtype == SPECA_BF16 else torch.float32
        n = self.entries[entry][0] * self.entries[entry][1]
        off = ptr - self.arena.data_ptr()
        raw = self.arena[off: off + stride * (self.max_order + 1)].view(tdt).view(self.max_order + 1, stride // esz)
        return raw[:, :n]

    @property
    def launches(self) -> int:
        return speca_cache_launch_count(self.handle)

    def stats(self):
        return speca_cache_stats(self.handle, self.batch)

    def check(self, stream=None):
        """Waits for `stream` and raises if a staged copy of the bulk path gave up."""
        speca_cache_check(self.handle, stream)

    def next_slot_batch(self, entry: int) -> torch.Tensor:
        """All samples' next planes of ``entry`` as one strided ``[B, N_e, D]`` view of the arena (raw-feature
        cache whose samples are at the same ring position): write the block output here and pass
        ``SPECA_FEATURE_IN_PLACE`` for the entry to ``update``."""
        ptrs = [speca_cache_next_slot(self.handle, entry, b) for b in range(self.batch)]
        n, d = self.entries[entry]
        esz = 2 if self.dtype == SPECA_BF16 else 4
        tdt = torch.bfloat16 if self.dtype == SPECA_BF16 else torch.float32
        step = (ptrs[1] - ptrs[0]) if self.batch > 1 else n * d * esz
        if any(ptrs[b] - ptrs[0] != b * step for b in range(self.batch)):
            raise ValueError("the samples are at different ring positions: use next_slot_tensor per sample")
        off = ptrs[0] - self.arena.data_ptr()
        flat = self.arena[off:].view(tdt)
        return torch.as_strided(flat, (self.batch, n, d), (step // esz, d, 1))

    def next_slot_tensor(self, entry: int, sample: int = 0) -> torch.Tensor:
        """The plane that the next reference step of ``sample`` fills, as an ``[N_e, D]`` view of the arena
        (raw-feature cache): write the block output here and pass it to ``update`` to skip the copy."""
        ptr = speca_cache_next_slot(self.handle, entry, sample)
        n, d = self.entries[entry]
        tdt = torch.bfloat16 if self.dtype == SPECA_BF16 else torch.float32
        off = ptr - self.arena.data_ptr()
        return self.arena[off: off + n * d * (2 if self.dtype == SPECA_BF16 else 4)].view(tdt).view(n, d)
