"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (every entry of a
step in one call, library-default kernel path).

The oracle cannot walk a 23 GB cache, so it is run on sampled blocks -- first and last elements of
rows, blocks straddling tile boundaries, unaligned random blocks -- plus the whole verification
entry (which Eq. 4 needs in full). Two properties that hold at any size cover every element without
the oracle: after an update plane 0 is the feature bit for bit, and a forecast to the latest
reference time returns plane 0 bit for bit (Eq. 2 with k = 0).

As in the small-shape tests, after each reference step the compared blocks of the GPU tables are
overwritten with the oracle's bits, so that a one-ulp rounding flip is not amplified by 1/gap at
the next step and real errors cannot hide behind a loose tolerance.
"""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O
from paper_2509_11628_b200 import workloads as W

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


@pytest.fixture(scope="module")
def U():
    from tests import gpu_util
    return gpu_util


def choose_blocks(w, rng):
    """{entry: [(sample, start, length), ...]}; the verification entry gets whole rows."""
    ne = len(w.entries)
    picked = sorted(set([0, 1, ne // 2, ne - 2]) - {w.vidx})
    blocks = {}
    for e in picked:
        n = w.entry_elems(e)
        lst = []
        for b in sorted(set([0, w.batch - 1, int(rng.integers(0, w.batch))])):
            lst.append((b, 0, min(n, 4096)))                                  # head of the row
            lst.append((b, max(0, n - 3001), min(n, 3001)))                   # ragged tail
            for tile_elems in (16384, 8192):                                  # 32 KB / 16 KB tile edges (bf16)
                k = int(rng.integers(1, max(2, n // tile_elems)))
                s = max(0, min(n - 2048, k * tile_elems - 1000))
                lst.append((b, s, min(2048, n - s)))
            s = int(rng.integers(0, max(1, n - 5000))) | 1                    # odd start: no vector alignment
            lst.append((b, s, min(4999, n - s)))
        blocks[e] = lst
    blocks[w.vidx] = [(b, 0, w.entry_elems(w.vidx)) for b in range(w.batch)]
    return blocks


def plane_slice(cache, e, b, start, length):
    return cache.plane_tensor(e, b)[:, start:start + length]


def bits_to_tensor(a, tdt):
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    return torch.from_numpy(a)


def reference_steps(U, w, cache, src, blocks, name):
    """max_order + 1 reference steps, every entry in one launch as the benchmark does. After each, on
    every element: plane 0 is the feature bit for bit; on the sampled blocks: the tables against the
    oracle's, then overwritten with the oracle's bits. Returns the oracle's tables per block and the
    reference times (latest first)."""
    B, m, ne = w.batch, w.max_order, len(w.entries)
    tdt = w.torch_dtype
    it = torch.int16 if w.dtype == W.BF16 else torch.int32
    orc = {(e, blk): np.zeros((m + 1, blk[2]), dtype=O.np_dtype(w.dtype)) for e, lst in blocks.items() for blk in lst}
    hist = []
    for step in range(m + 1):
        t = [w.times[step]] * B
        feats = [src.feature(e, step, t) for e in range(ne)]
        cache.update(feats, t)           # all entries, one launch: the benchmark's configuration
        cache.commit_step()
        torch.cuda.synchronize()
        for e in range(ne):
            for b in range(B):
                assert torch.equal(cache.plane_tensor(e, b)[0].view(it), feats[e][b].reshape(-1).view(it)), \
                    "%s step %d entry %d sample %d: plane 0 differs from the feature" % (name, step, e, b)
        R = 0.0 if not hist else 1.0 / min(abs(t[0] - h) for h in hist)
        for e, lst in blocks.items():
            for blk in lst:
                b, s, ln = blk
                fb = U.to_oracle(feats[e][b].reshape(-1)[s:s + ln])
                want = orc[(e, blk)]
                O.update_segment(w.dtype, m, O.TAYLOR, step, hist, t[b], fb, want)
                got = U.to_oracle(plane_slice(cache, e, b, s, ln))
                for i in range(min(m, step) + 1):
                    scale = sum(np.abs(U.as_f64(want[j])) * R ** (i - j) for j in range(i + 1))
                    U.assert_close_storage(got[i], want[i], w.dtype, scale * 0.5,
                                           "%s step %d entry %d block %r plane %d" % (name, step, e, blk, i))
                plane_slice(cache, e, b, s, ln).copy_(bits_to_tensor(want, tdt).to(DEV))
        hist = [t[0]] + hist
        del feats
    torch.cuda.synchronize()
    return orc, hist


def taylor_weights(m, x):
    ws = [1.0]
    for i in range(1, m + 1):
        ws.append(ws[-1] * x / i)
    return ws


FULL = [
    ("dit_xl2", {}, 0),
    ("flux", {}, 0),
    ("hunyuan_video", {}, 0),
    ("flux_adaptive", {"max_order": 3}, 0),
    ("flux_adaptive", {"max_order": 2}, 0),
    ("flux_adaptive", {"max_order": 1}, 0),
    ("flux", {}, 2),          # the TMA-staged kernels at full size
    ("dit_xl2", {}, 1),       # the 16-byte register path at full size
]


@pytest.mark.parametrize("name,kw,path", FULL)
def test_full_size_config_on_sampled_blocks(S, U, name, kw, path):
    w = W.BY_NAME[name](**kw)
    B, m, ne = w.batch, w.max_order, len(w.entries)
    rng = np.random.default_rng(1234 + w.index)
    blocks = choose_blocks(w, rng)
    src = W.FeatureSource(w, DEV)
    cache = S.SpecaCache(w.entries, B, m, w.dtype, DEV, path=path)
    tdt = w.torch_dtype
    orc, hist = reference_steps(U, w, cache, src, blocks, name)

    def weights(x):
        return taylor_weights(m, x)

    # forecast of every entry in one launch, compared on the blocks
    step = m + 1
    t_tgt = [w.times[step]] * B
    outs = [torch.full((B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in w.entries]
    cache.forecast(t_tgt, outs)
    torch.cuda.synchronize()
    for e, lst in blocks.items():
        if e == w.vidx:
            continue
        for blk in lst:
            b, s, ln = blk
            want = np.zeros(ln, dtype=O.np_dtype(w.dtype))
            O.forecast_segment(w.dtype, m, O.TAYLOR, m + 1, hist, t_tgt[b], orc[(e, blk)], want)
            got = U.to_oracle(outs[e][b].reshape(-1)[s:s + ln])
            scale = U.term_scale(orc[(e, blk)], weights(t_tgt[b] - hist[0]))
            U.assert_close_storage(got, want, w.dtype, scale, "%s forecast entry %d block %r" % (name, e, blk))

    # verification on the whole verify entry
    fresh = src.feature(w.vidx, step, t_tgt)
    tau = [0.12 if name == "flux_adaptive" else S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
    err = torch.full((B,), -7.0, dtype=torch.float32, device=DEV)
    acc = torch.full((B,), 9, dtype=torch.uint8, device=DEV)
    cache.verify(fresh, t_tgt, tau, err, acc)
    torch.cuda.synchronize()
    e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
    fresh_np = U.to_oracle(fresh).reshape(B, -1)
    a_want = []
    for b in range(B):
        blk = (b, 0, w.entry_elems(w.vidx))
        pred = np.zeros(blk[2], dtype=O.np_dtype(w.dtype))
        O.forecast_segment(w.dtype, m, O.TAYLOR, m + 1, hist, t_tgt[b], orc[(w.vidx, blk)], pred)
        e_want = O.rel_l2(w.dtype, pred, fresh_np[b])
        assert abs(e_got[b] - e_want) <= U.ERR_TOL * max(1.0, e_want), (name, b, e_got[b], e_want)
        ok = O.accept(e_want, float(np.float32(tau[b])))
        a_want.append(1 if ok else 0)
        if abs(e_want - float(np.float32(tau[b]))) >= U.ERR_TOL:
            assert int(a_got[b]) == a_want[-1], (name, b, e_want, tau[b])
        # the forecast launch wrote the same prediction for this entry
        got = U.to_oracle(outs[w.vidx][b].reshape(-1))
        scale = U.term_scale(orc[(w.vidx, blk)], weights(t_tgt[b] - hist[0]))
        U.assert_close_storage(got, pred, w.dtype, scale, "%s forecast of the verify entry sample %d" % (name, b))
    del fresh

    # rejected samples drop out: their rows of every output stay untouched, accepted rows are rewritten
    spec = torch.zeros(B, dtype=torch.int32, device=DEV)
    active = torch.ones(B, dtype=torch.uint8, device=DEV)
    flags = list(a_want)
    if B == 1:
        flags = [1]                      # keep the only sample active so that the k = 0 property is exercised
    elif len(set(flags)) == 1:
        flags[-1] = 1 - flags[-1]        # make sure both an active and an inactive row are exercised
    d_acc = torch.tensor(flags, dtype=torch.uint8, device=DEV)
    cache.select_adaptive(d_acc, 6, 1, spec, active)
    act_want, _, _ = O.select_adaptive(flags, 6, 1, [0] * B, [1] * B)
    torch.cuda.synchronize()
    assert active.cpu().tolist() == act_want
    for o in outs:
        o.fill_(5.0)
    # forecast to the latest reference time: Eq. 2 with k = 0 returns the cached feature itself
    cache.forecast([hist[0]] * B, outs, active)
    torch.cuda.synchronize()
    it = torch.int16 if w.dtype == W.BF16 else torch.int32
    five = torch.full((1,), 5.0, dtype=tdt, device=DEV).view(it)
    for e in range(ne):
        for b in range(B):
            row = outs[e][b].reshape(-1).view(it)
            if act_want[b]:
                assert torch.equal(row, cache.plane_tensor(e, b)[0].view(it)), (name, e, b)
            else:
                assert bool((row == five).all()), "%s: inactive sample %d of entry %d was written" % (name, b, e)
    cache.close()


def test_full_size_adaptive_batch_over_a_speculative_run(S, U):
    """The sample-adaptive configuration (FLUX shape, 8 samples with three noise levels, order 2) at full
    size over a run of speculative steps k = 1, 2, 3 from the same tables. At every k the oracle's own
    accept flags decide who stays active: the forecast launch is checked on the sampled blocks (active
    samples against the oracle, inactive rows untouched), the fused verification on the whole
    verification entry per active sample, and the continuation rule against the oracle's."""
    name = "flux_adaptive_m2"
    w = W.flux_adaptive(max_order=2, batch=8)
    B, m, ne = w.batch, w.max_order, len(w.entries)
    rng = np.random.default_rng(977)
    blocks = choose_blocks(w, rng)
    src = W.FeatureSource(w, DEV)
    cache = S.SpecaCache(w.entries, B, m, w.dtype, DEV)
    tdt = w.torch_dtype
    it = torch.int16 if w.dtype == W.BF16 else torch.int32
    orc, hist = reference_steps(U, w, cache, src, blocks, name)
    outs = [torch.empty(B, n, d, dtype=tdt, device=DEV) for n, d in w.entries]
    err = torch.zeros(B, dtype=torch.float32, device=DEV)
    acc = torch.zeros(B, dtype=torch.uint8, device=DEV)
    active = torch.ones(B, dtype=torch.uint8, device=DEV)
    nxt = torch.ones(B, dtype=torch.uint8, device=DEV)
    spec = torch.zeros(B, dtype=torch.int32, device=DEV)
    act, cnt = [1] * B, [0] * B
    seven = torch.full((1,), 7.0, dtype=tdt, device=DEV).view(it)
    seen_inactive = False
    for k in range(1, 4):
        step = m + k
        t_tgt = [w.times[step]] * B
        tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
        for o in outs:
            o.fill_(7.0)
        err.fill_(-7.0)
        acc.fill_(9)
        fresh = src.feature(w.vidx, step, t_tgt)
        others = list(outs)
        others[w.vidx] = None            # as the benchmark's step: the verification launch writes that entry's forecast
        cache.forecast(t_tgt, others, active)
        cache.verify_select(fresh, t_tgt, tau, err, acc, active, nxt, 6, 1, spec, out_pred=outs[w.vidx])
        torch.cuda.synchronize()
        fresh_np = U.to_oracle(fresh).reshape(B, -1)
        e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
        flags = [0] * B
        for e, lst in blocks.items():
            for blk in lst:
                b, s, ln = blk
                got_t = outs[e][b].reshape(-1)[s:s + ln]
                if not act[b]:
                    seen_inactive = True
                    assert bool((got_t.view(it) == seven).all()), "%s k=%d: inactive sample %d of entry %d was written" % (name, k, b, e)
                    continue
                want = np.zeros(ln, dtype=O.np_dtype(w.dtype))
                O.forecast_segment(w.dtype, m, O.TAYLOR, m + 1, hist, t_tgt[b], orc[(e, blk)], want)
                scale = U.term_scale(orc[(e, blk)], taylor_weights(m, t_tgt[b] - hist[0]))
                U.assert_close_storage(U.to_oracle(got_t), want, w.dtype, scale, "%s k=%d forecast entry %d block %r" % (name, k, e, blk))
                if e == w.vidx:
                    e_want = O.rel_l2(w.dtype, want, fresh_np[b])
                    assert abs(e_got[b] - e_want) <= U.ERR_TOL * max(1.0, e_want), (name, k, b, e_got[b], e_want)
                    flags[b] = 1 if O.accept(e_want, float(np.float32(tau[b]))) else 0
                    if abs(e_want - float(np.float32(tau[b]))) >= U.ERR_TOL:
                        assert int(a_got[b]) == flags[b], (name, k, b, e_want, tau[b])
                    else:
                        flags[b] = int(a_got[b])     # inside the tolerance band either decision is right: follow the library
        for b in range(B):
            if not act[b]:
                assert e_got[b] == -7.0 and a_got[b] == 9, (name, k, b)
        act, cnt, _ = O.select_adaptive(flags, 6, 1, cnt, act)
        assert nxt.cpu().tolist() == act and spec.cpu().tolist() == cnt, (name, k)
        active, nxt = nxt, active
        del fresh
    assert seen_inactive and any(act), "the noise levels were chosen so that some samples drop out and some stay: %r" % (act,)
    cache.close()


@pytest.mark.parametrize("name", ["dit_xl2", "flux", "hunyuan_video"])
def test_full_size_raw_feature_cache_on_sampled_blocks(S, U, name):
    """The same at full size for the cache that keeps raw features: reference steps past the point where
    the ring wraps (every element: the newest plane is the feature, bit for bit), forecast of every entry
    in one launch against the oracle on the sampled blocks, Eq. 4 on the whole verification entry, and
    the k = 0 property on every element."""
    w = W.BY_NAME[name]()
    B, m, ne = w.batch, w.max_order, len(w.entries)
    rng = np.random.default_rng(4321 + w.index)
    blocks = choose_blocks(w, rng)
    src = W.FeatureSource(w, DEV)
    cache = S.SpecaCache(w.entries, B, m, w.dtype, DEV, layout=S.SPECA_LAYOUT_HISTORY)
    tdt = w.torch_dtype
    it = torch.int16 if w.dtype == W.BF16 else torch.int32
    kept = {(e, blk): [] for e, lst in blocks.items() for blk in lst}      # raw feature blocks, latest first
    hist = []
    n_steps = m + 2
    for step in range(n_steps):
        t = [w.times[step]] * B
        feats = [src.feature(e, step, t) for e in range(ne)]
        cache.update(feats, t)
        cache.commit_step()
        torch.cuda.synchronize()
        slot = step % (m + 1)
        for e in range(ne):
            for b in range(B):
                assert torch.equal(cache.plane_tensor(e, b)[slot].view(it), feats[e][b].reshape(-1).view(it)), \
                    "%s step %d entry %d sample %d: the newest plane differs from the feature" % (name, step, e, b)
        for e, lst in blocks.items():
            for blk in lst:
                b, s, ln = blk
                kept[(e, blk)] = ([U.to_oracle(feats[e][b].reshape(-1)[s:s + ln])] + kept[(e, blk)])[: m + 1]
        hist = ([t[0]] + hist)[: m + 1]
        del feats
    step = n_steps
    t_tgt = [w.times[step]] * B
    outs = [torch.full((B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in w.entries]
    cache.forecast(t_tgt, outs)
    torch.cuda.synchronize()
    unit = [np.eye(m + 1, dtype=np.float32)[j].copy() for j in range(m + 1)]
    a = np.zeros(m + 1, dtype=np.float32)
    O.forecast_history_segment(O.F32, m, O.TAYLOR, hist, t_tgt[0], unit, a)            # weights, for the tolerance only

    def oracle_forecast(e, blk):
        want = np.zeros(blk[2], dtype=O.np_dtype(w.dtype))
        O.forecast_history_segment(w.dtype, m, O.TAYLOR, hist, t_tgt[blk[0]], kept[(e, blk)], want)
        scale = sum(np.abs(U.as_f64(f)) * abs(float(a[j])) for j, f in enumerate(kept[(e, blk)]))
        return want, scale

    for e, lst in blocks.items():
        for blk in lst:
            b, s, ln = blk
            want, scale = oracle_forecast(e, blk)
            got = U.to_oracle(outs[e][b].reshape(-1)[s:s + ln])
            U.assert_close_storage(got, want, w.dtype, scale, "%s forecast entry %d block %r" % (name, e, blk))
    fresh = src.feature(w.vidx, step, t_tgt)
    tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
    err = torch.full((B,), -7.0, dtype=torch.float32, device=DEV)
    acc = torch.full((B,), 9, dtype=torch.uint8, device=DEV)
    pred_gpu = torch.empty_like(fresh)
    cache.verify(fresh, t_tgt, tau, err, acc, out_pred=pred_gpu)
    torch.cuda.synchronize()
    fresh_np = U.to_oracle(fresh).reshape(B, -1)
    pred_np = U.to_oracle(pred_gpu).reshape(B, -1)
    for b in range(B):
        blk = (b, 0, w.entry_elems(w.vidx))
        pred, scale = oracle_forecast(w.vidx, blk)
        # The forecast of a raw-feature cache is rounded ONCE, from an exact combination of stored values.
        # On a uniform time grid the weights are ratios of small integers, so a few per cent of the
        # results sit exactly on a rounding tie of the storage type, where fp32 and fp64 evaluation may
        # pick different neighbours and both are correct roundings. So: (1) every element of the
        # library's forecast equals the oracle's, or is the other neighbour of such a tie; (2) Eq. 4 and
        # the accept rule, by the oracle, ON THAT FORECAST agree with the library's err / accept within
        # the usual bound -- no widened tolerance anywhere.
        raw = O.forecast_history_unrounded(w.dtype, m, O.TAYLOR, hist, t_tgt[b], kept[(w.vidx, blk)])
        share = U.assert_equal_or_tie(pred_np[b], pred, raw, w.dtype, scale, "%s forecast of the verify entry sample %d" % (name, b))
        assert share < 0.1, (name, b, share)
        e_on_it = O.rel_l2(w.dtype, np.ascontiguousarray(pred_np[b]), fresh_np[b])
        assert abs(float(err[b]) - e_on_it) <= U.ERR_TOL * max(1.0, e_on_it), (name, b, float(err[b]), e_on_it)
        if abs(e_on_it - float(np.float32(tau[b]))) >= U.ERR_TOL:
            assert int(acc[b]) == (1 if O.accept(e_on_it, float(np.float32(tau[b]))) else 0)
        # for the record: how far the ties move the error from the oracle's own end-to-end value
        e_want = O.rel_l2(w.dtype, pred, fresh_np[b])
        print("%s sample %d: %.3f %% of the forecast on the other side of a tie; err %.6f, oracle end to end %.6f (%.2e relative)" % (
            name, b, 100 * share, float(err[b]), e_want, abs(float(err[b]) - e_want) / max(e_want, 1e-30)))
        assert abs(float(err[b]) - e_want) <= 2e-2 * max(e_want, 1e-3)     # sanity only; the bound that binds is the one above
    for o in outs:
        o.fill_(5.0)
    cache.forecast([hist[0]] * B, outs)          # k = 0: the newest feature itself
    torch.cuda.synchronize()
    newest = (n_steps - 1) % (m + 1)
    for e in range(ne):
        for b in range(B):
            assert torch.equal(outs[e][b].reshape(-1).view(it), cache.plane_tensor(e, b)[newest].view(it)), (name, e, b)
    cache.close()
