"""The cache that keeps raw features (SPECA_LAYOUT_HISTORY): a reference step only copies the feature
into the next plane of a ring; Eq. 2-3 are evaluated from the stored features at forecast time. Parity
against the oracle's history layout (which folds the features in double, in the order Eq. 3 does)."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RAGGED = [(37, 129), (5, 3), (64, 384), (1, 8192 * 2 + 24), (3, 8192), (1, 1)]
HIST = 1


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


@pytest.fixture(scope="module")
def U():
    from tests import gpu_util
    return gpu_util


def rand_feats(entries, B, tdt, gen):
    return [torch.randn(B, n, d, generator=gen, device=DEV, dtype=torch.float32).to(tdt) for n, d in entries]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("basis", [0, 1, 2])
@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_ragged_shapes_all_orders(S, U, dtype, basis, m):
    B = 3
    gen = torch.Generator(device=DEV).manual_seed(7000 + 10 * m + basis)
    pair = U.Pair(RAGGED, B, m, dtype, basis, layout=HIST)
    times = [1.0, 0.93, 0.9, 0.81, 0.8, 0.74, 0.7, 0.66]
    for step in range(m + 4):                       # past the point where the ring wraps
        t = [times[step], times[step] - 0.003, times[step] + 0.001]
        pair.update(rand_feats(RAGGED, B, pair.tdt, gen), t, per_entry_calls=(step % 2 == 1))
        pair.commit()
        pair.check_tables("step %d" % step)
        tt = [times[step] - 0.02, times[step] - 0.035, times[step] - 0.011]
        pair.check_forecast(tt, what="m=%d basis=%d step %d" % (m, basis, step))
    outs = pair.check_forecast(tt)
    n, d = RAGGED[-1] if pair.vidx == len(RAGGED) - 1 else RAGGED[pair.vidx]
    fresh = (outs[pair.vidx].float() * 1.02).to(pair.tdt)
    pair.check_verify(fresh, tt, [0.5, 0.01, 0.03])
    pair.close()


@pytest.mark.parametrize("dtype", [0, 1])
def test_masks_resets_and_verification_on_many_tiles(S, U, dtype):
    entries = [(16, 520), (301, 1160)]
    B, m = 5, 2
    gen = torch.Generator(device=DEV).manual_seed(11)
    pair = U.Pair(entries, B, m, dtype, layout=HIST)
    clock = 1.0
    masks = [None, None, [1, 0, 1, 1, 0], None, [0, 1, 1, 0, 1], [1, 1, 0, 0, 0]]
    for step, mask in enumerate(masks):
        clock -= 0.04
        pair.update(rand_feats(entries, B, pair.tdt, gen), [clock - 0.001 * b for b in range(B)], mask)
        pair.commit()
        pair.check_tables("masked step %d" % step)
        if step == 3:
            pair.gpu.reset([0, 0, 0, 1, 0])
            pair.cpu.reset([0, 0, 0, 1, 0])
    n_refs, _ = pair.gpu.state()
    assert n_refs == pair.cpu.n_refs == [5, 5, 5, 0, 4]
    act = [1, 1, 1, 0, 1]
    tt = [clock - 0.03] * B
    outs = pair.check_forecast(tt, active=act, sentinel=2.5)
    noise = torch.randn(B, 301, 1160, generator=gen, device=DEV) * torch.tensor([0.0, 0.01, 0.05, 0.2, 1.0], device=DEV).view(B, 1, 1)
    fresh = (outs[1].float() + noise).to(pair.tdt)
    for metric in (None, O.METRIC_L1, O.METRIC_LINF, O.METRIC_COSINE):
        tau = [1e-3] * B if metric == O.METRIC_COSINE else [0.03] * B
        e, a, _, _ = pair.check_verify(fresh, tt, tau, active=act, metric=metric, ulp_slack=(metric == O.METRIC_LINF))
    # the fused continuation works on this layout too
    err = torch.zeros(B, device=DEV); acc = torch.zeros(B, dtype=torch.uint8, device=DEV)
    cur = torch.tensor(act, dtype=torch.uint8, device=DEV); nxt = torch.zeros(B, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(B, dtype=torch.int32, device=DEV)
    pair.gpu.verify_select(fresh, tt, [0.03] * B, err, acc, cur, nxt, 3, 1, cnt)
    torch.cuda.synchronize()
    _, a_want, _ = pair.cpu.verify(U.to_oracle(fresh).reshape(B, -1), tt, [0.03] * B, act)
    want_act, want_cnt, _ = O.select_adaptive([max(int(a), 0) for a in a_want], 3, 1, [0] * B, act)
    assert nxt.cpu().tolist() == want_act and cnt.cpu().tolist() == want_cnt
    assert want_act[0] == 1 and want_act[3] == 0 and want_act[4] == 0     # exact match kept; inactive and noisy dropped
    pair.close()


def test_the_ring_wraps_and_other_kernel_paths_are_refused(S):
    entries = [(8, 64), (4, 32)]
    B = 2
    c = S.SpecaCache(entries, B, 2, 1, DEV, layout=HIST)
    f = [torch.ones(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    for t in (1.0, 0.9, 0.8, 0.7):
        c.update([x * t for x in f], [t] * B)
        c.commit_step()
    torch.cuda.synchronize()
    # four references in a ring of three planes: 0.7 overwrote 1.0 in plane 0
    planes = c.plane_tensor(0, 1).float().cpu()
    assert torch.allclose(planes[:, 0], torch.tensor([0.7, 0.9, 0.8]), atol=4e-3)
    outs = [torch.zeros_like(x) for x in f]
    c.forecast([0.6] * B, outs)
    torch.cuda.synchronize()
    assert torch.allclose(outs[0].float().cpu(), torch.full((B, 8, 64), 0.6), atol=8e-3)   # linear in t: exact

    def status_of(fn):
        with pytest.raises(S.SpecaError) as ei:
            fn()
        return ei.value.status

    assert status_of(lambda: c.update(f, [0.7] * B)) == S.SPECA_ERR_ZERO_GAP
    assert status_of(lambda: S.SpecaCache(entries, B, 2, 1, DEV, path=S.SPECA_PATH_BULK, layout=HIST)) == S.SPECA_ERR_UNSUPPORTED
    c.close()


def test_history_and_tables_agree_on_exactly_representable_inputs(S):
    # integer features, power-of-two gaps, fp32, order 2 (x^2 / 2 is dyadic; order 3 would bring in thirds):
    # both layouts compute the same numbers without any rounding, so they must agree bit for bit
    entries = [(33, 130)]
    B, m = 2, 2
    gen = torch.Generator(device=DEV).manual_seed(3)
    a = S.SpecaCache(entries, B, m, 0, DEV)
    b = S.SpecaCache(entries, B, m, 0, DEV, layout=HIST)
    t = 64.0
    for k in range(7):
        f = [(torch.randint(-8, 8, (B, 33, 130), generator=gen, device=DEV) * 64).float()]
        t -= [1.0, 2.0, 4.0][k % 3]
        for c in (a, b):
            c.update(f, [t, t - 0.5])
            c.commit_step()
        oa, ob = [torch.zeros_like(f[0])], [torch.zeros_like(f[0])]
        a.forecast([t - 2.0, t - 1.0], oa)
        b.forecast([t - 2.0, t - 1.0], ob)
        torch.cuda.synchronize()
        assert torch.equal(oa[0], ob[0]), k
    a.close(); b.close()


def test_features_written_in_place_cost_no_launch(S, U):
    """B = 1: the model writes each block output straight into the plane that is next in the ring and
    hands that address to update: nothing is copied, the reference step launches nothing."""
    entries = [(37, 129), (64, 384), (3, 8192)]
    m = 2
    gen = torch.Generator(device=DEV).manual_seed(23)
    pair = U.Pair(entries, 1, m, 1, layout=HIST)
    clock = 1.0
    for step in range(6):
        clock -= 0.03 + 0.01 * (step % 2)
        slots = [pair.gpu.next_slot_tensor(e, 0) for e in range(len(entries))]
        for s, f in zip(slots, rand_feats(entries, 1, pair.tdt, gen)):
            s.copy_(f[0])
        launches = pair.gpu.launches
        if step == 3:   # one entry handed over from elsewhere: only that one is copied
            other = slots[1].clone().view(1, *entries[1])
            pair.update([slots[0].view(1, *entries[0]), other, slots[2].view(1, *entries[2])], [clock])
            assert pair.gpu.launches == launches + 1
        else:
            pair.update([s.view(1, n, d) for s, (n, d) in zip(slots, entries)], [clock])
            assert pair.gpu.launches == launches
        pair.commit()
        pair.check_tables("in place, step %d" % step)
        pair.check_forecast([clock - 0.02], what="in place, step %d" % step)
    assert pair.gpu.stats()["update_launches"] == 1 and pair.gpu.stats()["reference_steps"] == [6]
    # a cache that keeps tables has no such slot
    c = S.SpecaCache(entries, 1, m, 1, DEV)
    with pytest.raises(S.SpecaError) as ei:
        S.speca_cache_next_slot(c.handle, 0, 0)
    assert ei.value.status == S.SPECA_ERR_UNSUPPORTED
    c.close()
    pair.close()


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("basis", [0, 1, 2])
@pytest.mark.parametrize("m", [0, 1, 2, 4])
def test_multi_horizon_and_summed_forecasts(S, U, dtype, basis, m):
    """speca_forecast_multi and speca_forecast_sum on the raw-feature cache: K targets bit-identical to K
    single forecasts and equal to the oracle; the sum of several entries equal to the oracle's sum."""
    shape = (37, 129)
    E, B, K = 7, 3, 3
    entries = [shape] * E + [(3, 8192 + 8)]
    gen = torch.Generator(device=DEV).manual_seed(9100 + 10 * m + basis)
    pair = U.Pair(entries, B, m, dtype, basis, layout=HIST)
    times = [1.0, 0.93, 0.9, 0.84, 0.8, 0.77, 0.71]
    for step in range(m + 3):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [times[step], times[step] - 0.003, times[step] + 0.001])
        pair.commit()
    t_last = times[m + 2]
    targets = [[t_last - 0.011 * (k + 1) - 0.001 * b for b in range(B)] for k in range(K)]
    active = [1, 0, 1]
    mask = torch.tensor(active, dtype=torch.uint8, device=DEV)
    outs = [torch.full((K, B, n, d), 3.0, dtype=pair.tdt, device=DEV) for n, d in entries]
    pair.gpu.forecast_multi(targets, outs, mask)
    it = torch.int16 if dtype == 1 else torch.int32
    three = U.to_oracle(torch.full((1,), 3.0, dtype=pair.tdt))[0]
    for k in range(K):
        single = [torch.full((B, n, d), 3.0, dtype=pair.tdt, device=DEV) for n, d in entries]
        pair.gpu.forecast(targets[k], single, mask)
        torch.cuda.synchronize()
        for e, (n, d) in enumerate(entries):
            assert torch.equal(outs[e][k].view(it), single[e].view(it)), (k, e)
            init = np.full((B, n * d), three, dtype=O.np_dtype(dtype))
            want = pair.cpu.forecast_entry(e, targets[k], active, out=init)
            got = U.to_oracle(outs[e][k]).reshape(B, -1)
            for b in range(B):
                if not active[b]:
                    assert np.array_equal(got[b], want[b])
                else:
                    U.assert_close_storage(got[b], want[b], dtype, pair.history_scale(e, b, targets[k][b]), "multi %d %d %d" % (k, e, b))
    tt = targets[0]
    base = torch.randn(B, *shape, generator=gen, device=DEV).to(pair.tdt)
    for ids, use_base in [(list(range(E)), True), ([3], False), ([4, 0, 4, 6, 5, 1], True)]:
        out = torch.full((B, *shape), 3.0, dtype=pair.tdt, device=DEV)
        pair.gpu.forecast_sum(ids, tt, out, base if use_base else None)
        torch.cuda.synchronize()
        want = pair.cpu.forecast_sum(ids, tt, U.to_oracle(base).reshape(B, -1) if use_base else None)
        got = U.to_oracle(out).reshape(B, -1)
        for b in range(B):
            scale = sum(pair.history_scale(e, b, tt[b]) for e in ids)
            if use_base:
                scale = scale + np.abs(U.as_f64(U.to_oracle(base).reshape(B, -1)[b]))
            U.assert_close_storage(got[b], want[b], dtype, scale, "sum %r sample %d" % (ids, b))
    pair.close()


def test_checkpoint_and_resume_continue_bit_for_bit(S):
    """Arena bytes + reference history are the whole state of a raw-feature cache too: the ring position
    follows from the number of references, so a restored cache continues exactly where the saved one was."""
    entries = [(16, 520), (33, 1031)]
    B, m = 3, 2
    gen = torch.Generator(device=DEV).manual_seed(13)
    a = S.SpecaCache(entries, B, m, 1, DEV, layout=HIST)
    steps = [([1.0, 1.0, 1.0], None), ([0.95, 0.96, 0.95], [1, 1, 0]), ([0.9, 0.91, 0.9], None), ([0.85, 0.85, 0.85], [1, 0, 1]),
             ([0.8, 0.8, 0.8], None)]
    for t, mask in steps:
        a.update(rand_feats(entries, B, torch.bfloat16, gen), t, mask)
        a.commit_step()
    torch.cuda.synchronize()
    saved = a.arena.clone()
    n_refs, t_hist = S.speca_cache_get_history(a.handle, B)
    assert n_refs == [5, 4, 4]                     # past the wrap of the three-plane ring, at different positions
    b = S.SpecaCache(entries, B, m, 1, DEV, layout=HIST)
    b.arena.copy_(saved)
    S.speca_cache_set_history(b.handle, n_refs, t_hist)
    nxt = rand_feats(entries, B, torch.bfloat16, gen)
    for c in (a, b):
        c.update(nxt, [0.75, 0.74, 0.76], [0, 1, 1])
        c.commit_step()
    oa = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    ob = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    a.forecast([0.7] * B, oa)
    b.forecast([0.7] * B, ob)
    torch.cuda.synchronize()
    for x, y in zip(oa, ob):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    assert torch.equal(a.arena, b.arena)
    a.close(); b.close()


def test_a_batch_written_in_place_through_a_strided_view(S, U):
    """B = 3 in lockstep: the next planes of all samples form one strided [B, N, D] tensor; the model
    writes there and the reference step copies nothing. When a masked step has moved the samples to
    different ring positions the per-sample views still work."""
    entries = [(37, 129), (64, 384)]
    B, m = 3, 2
    gen = torch.Generator(device=DEV).manual_seed(29)
    pair = U.Pair(entries, B, m, 1, layout=HIST)
    clock = 1.0
    for step in range(5):
        clock -= 0.03
        feats = rand_feats(entries, B, pair.tdt, gen)
        for e in range(len(entries)):
            pair.gpu.next_slot_batch(e).copy_(feats[e])
        launches = pair.gpu.launches
        pair.gpu.update([S.SPECA_FEATURE_IN_PLACE] * len(entries), [clock] * B)
        pair.cpu.update([U.to_oracle(f).reshape(B, -1) for f in feats], [clock] * B)
        assert pair.gpu.launches == launches
        pair.commit()
        pair.check_tables("strided in place, step %d" % step)
        pair.check_forecast([clock - 0.02] * B)
    # a masked step: samples 0 and 2 advance, sample 1 stays; per-sample planes from now on
    for step in range(3):
        clock -= 0.03
        mask = [1, 0, 1] if step == 0 else None
        feats = rand_feats(entries, B, pair.tdt, gen)
        for e in range(len(entries)):
            for b in range(B):
                if mask is None or mask[b]:
                    pair.gpu.next_slot_tensor(e, b).copy_(feats[e][b])
        if step == 1:
            with pytest.raises(ValueError):
                pair.gpu.next_slot_batch(0)
        pair.gpu.update([S.SPECA_FEATURE_IN_PLACE] * len(entries), [clock] * B, mask)
        pair.cpu.update([U.to_oracle(f).reshape(B, -1) for f in feats], [clock] * B, mask)
        pair.commit()
        pair.check_tables("per-sample in place, step %d" % step)
        pair.check_forecast([clock - 0.02] * B)
    assert pair.gpu.stats()["update_launches"] == 0
    # the marker means nothing to a cache that keeps tables
    c = S.SpecaCache(entries, B, m, 1, DEV)
    with pytest.raises(S.SpecaError) as ei:
        c.update([S.SPECA_FEATURE_IN_PLACE, None], [1.0] * B)
    assert ei.value.status == S.SPECA_ERR_INVALID_ARG
    c.close()
    pair.close()
