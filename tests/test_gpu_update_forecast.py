"""speca_cache_update_forecast: a whole reference step and the first speculative step after it in one
pass over the tables. It must be, bit for bit, speca_cache_update_activate + speca_cache_commit_step +
speca_forecast -- which the other tests hold against the oracle -- and it is held against the oracle
here as well (tables after every step, forecasts of every step), over ragged shapes, orders 0-4, the
three draft models, both storage types, warm-up orders, samples that skip a reference step and keep
speculating, samples that have dropped out, and entries that are only updated."""
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


def bits(x):
    return x.contiguous().view(torch.uint8)


ENTRIES = [(3, 520), (9, 1031), (65, 1024), (40, 1030)]   # rows that are and are not 32-byte aligned, several tiles


@pytest.mark.parametrize("dtype", [1, 0])
@pytest.mark.parametrize("basis", [0, 1, 2])
@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_fused_reference_step_equals_the_three_calls_and_the_oracle(S, U, dtype, basis, m):
    B = 4
    pair = U.Pair(ENTRIES, B, m, dtype, basis=basis)          # the three calls + the oracle
    fused = S.SpecaCache(ENTRIES, B, m, dtype, DEV, basis=basis)
    gen = torch.Generator(device=DEV).manual_seed(100 * dtype + 10 * basis + m)
    ne = len(ENTRIES)
    st = {k: torch.zeros(B, dtype=torch.int32, device=DEV) for k in ("spec_a", "spec_b")}
    act_a = torch.ones(B, dtype=torch.uint8, device=DEV)
    act_b = torch.ones(B, dtype=torch.uint8, device=DEV)
    t = 1.0
    # who takes which reference step: everybody warms up, then sample 1 skips one (and keeps speculating),
    # sample 2 skips one after having dropped out (inactive: not forecast), sample 3 always takes part
    plan = [([1, 1, 1, 1], None)] * (m + 1) + [([1, 0, 1, 1], None), ([1, 1, 0, 1], 2), ([1, 1, 1, 1], None)]
    for k, (mask, drop) in enumerate(plan):
        t -= 0.03 + 0.004 * (k % 3)                          # uneven gaps
        t_ref = [t - 0.001 * b for b in range(B)]            # every sample on its own clock
        t_tgt = [x - 0.011 for x in t_ref]
        if drop is not None:                                 # a sample the verification rejected earlier
            act_a[drop] = 0
            act_b[drop] = 0
            st["spec_a"][drop] = 3
            st["spec_b"][drop] = 3
        feats = [torch.randn(B, n, d, generator=gen, device=DEV).to(pair.tdt) for n, d in ENTRIES]
        outs_a = [torch.full((B, n, d), 7.0, dtype=pair.tdt, device=DEV) for n, d in ENTRIES]
        only_update = ne - 1 if k % 2 == 1 else None        # every other step one entry gets no forecast
        give = list(outs_a)
        if only_update is not None:
            give[only_update] = None
        launches = fused.launches
        fused.update_forecast(feats, t_ref, t_tgt, give, mask=mask, active=act_a, spec_count=st["spec_a"], rearm=act_a)
        assert fused.launches == launches + 1
        # the same through the three calls (update with the re-arming, commit, forecast) and the oracle
        pair.gpu.update_activate(feats, t_ref, mask, st["spec_b"], act_b)
        pair.cpu.update([U.to_oracle(f).reshape(B, -1) for f in feats], t_ref, mask)
        pair.commit()
        pair.check_tables("step %d" % k)
        active_host = [int(x) for x in act_b.cpu().tolist()]
        outs_b = [torch.full((B, n, d), 7.0, dtype=pair.tdt, device=DEV) for n, d in ENTRIES]
        pair.gpu.forecast(t_tgt, outs_b, act_b)
        torch.cuda.synchronize()
        # Eq. 2 by the oracle on the very planes the library holds (its tables were checked against the
        # oracle's just above; they are re-synchronised only after the step, as the fused call forecasts
        # from what it has just written)
        for e in range(ne):
            for b in range(B):
                row = U.to_oracle(outs_b[e][b].reshape(-1))
                if not active_host[b]:
                    assert bool((outs_b[e][b].float() == 7.0).all()), ("an inactive sample was forecast", k, e, b)
                    continue
                planes = U.to_oracle(pair.gpu.plane_tensor(e, b))
                planes[min(m, pair.cpu.n_refs[b] - 1) + 1:] = 0      # planes above the sample's order hold nothing yet
                want = np.zeros(row.size, dtype=O.np_dtype(dtype))
                O.forecast_segment(dtype, m, basis, pair.cpu.n_refs[b], pair.cpu.t_hist[b], t_tgt[b], planes, want)
                scale = U.term_scale(planes, pair.forecast_weights(b, t_tgt[b]))
                U.assert_close_storage(row, want, dtype, scale, "step %d forecast entry %d sample %d" % (k, e, b))
        refs = fused.state()[0]
        for e in range(ne):
            for b in range(B):
                live = min(m, refs[b] - 1) + 1               # planes above the sample's order are not defined yet
                assert torch.equal(bits(fused.plane_tensor(e, b)[:live]), bits(pair.gpu.plane_tensor(e, b)[:live])), ("planes", k, e, b)
            if e == only_update:
                assert bool((outs_a[e].float() == 7.0).all()), ("an entry without an output was written", k, e)
            else:
                assert torch.equal(bits(outs_a[e]), bits(outs_b[e])), ("forecast", k, e)
        assert torch.equal(act_a, act_b) and torch.equal(st["spec_a"], st["spec_b"])
        assert fused.state() == pair.gpu.state()
        # both sides continue from the oracle's bits (see gpu_util.Pair.sync_tables)
        pair.sync_tables()
        for e in range(ne):
            for b in range(B):
                fused.plane_tensor(e, b).copy_(pair.gpu.plane_tensor(e, b))
    assert fused.stats()["update_forecast_launches"] == len(plan) and fused.stats()["update_launches"] == 0
    assert fused.stats()["reference_steps"] == pair.gpu.stats()["reference_steps"]
    fused.close()
    pair.close()


def test_fused_reference_step_refuses_what_it_cannot_do_and_leaves_the_history_alone(S):
    entries = [(8, 512), (5, 520)]
    B = 2
    feats = [torch.randn(B, n, d, device=DEV).bfloat16() for n, d in entries]
    outs = [torch.empty_like(f) for f in feats]

    def status(fn):
        with pytest.raises(S.SpecaError) as ei:
            fn()
        return ei.value.status

    bulk = S.SpecaCache(entries, B, 2, 1, DEV, path=S.SPECA_PATH_BULK)
    assert status(lambda: bulk.update_forecast(feats, [1.0] * B, [0.9] * B, outs)) == S.SPECA_ERR_UNSUPPORTED
    bulk.close()
    c = S.SpecaCache(entries, B, 2, 1, DEV)
    assert status(lambda: c.update_forecast([feats[0], None], [1.0] * B, [0.9] * B, outs)) == S.SPECA_ERR_INVALID_ARG
    assert status(lambda: c.update_forecast(feats, [float("nan")] * B, [0.9] * B, outs)) == S.SPECA_ERR_INVALID_ARG
    assert status(lambda: c.update_forecast(feats, [1.0] * B, [float("inf")] * B, outs)) == S.SPECA_ERR_INVALID_ARG
    # a sample that is not part of the step and has never had a reference, with no device mask to excuse it
    assert status(lambda: c.update_forecast(feats, [1.0] * B, [0.9] * B, outs, mask=[1, 0])) == S.SPECA_ERR_STATE
    assert c.state()[0] == [0, 0] and c.launches == 0
    c.update_forecast(feats, [1.0] * B, [0.9] * B, outs)
    before = c.state()
    assert before[0] == [1, 1]
    assert status(lambda: c.update_forecast(feats, [1.0, 0.95], [0.9] * B, outs)) == S.SPECA_ERR_ZERO_GAP   # sample 0 repeats t = 1.0
    assert c.state() == before
    c.update([feats[0], None], [0.9] * B)                                 # an open reference step
    assert status(lambda: c.update_forecast(feats, [0.9] * B, [0.8] * B, outs)) == S.SPECA_ERR_STATE
    torch.cuda.synchronize()
    c.close()


@pytest.mark.parametrize("layout", [0, 1])
def test_fused_reference_step_at_full_size(S, layout):
    """FLUX-shaped cache at full size, every entry in the one launch, the verification entry updated only:
    every plane and every forecast bit for bit equal to the three calls, for difference tables and for a
    cache that keeps raw features (there one step further, past the ring's wrap)."""
    w = W.flux()
    B, m, ne = w.batch, w.max_order, len(w.entries)
    src = W.FeatureSource(w, DEV)
    a = S.SpecaCache(w.entries, B, m, w.dtype, DEV, layout=layout)
    b = S.SpecaCache(w.entries, B, m, w.dtype, DEV, layout=layout)
    outs_a = [torch.empty(B, n, d, dtype=w.torch_dtype, device=DEV) for n, d in w.entries]
    outs_b = [torch.empty(B, n, d, dtype=w.torch_dtype, device=DEV) for n, d in w.entries]
    give_a, give_b = list(outs_a), list(outs_b)
    give_a[w.vidx] = None
    give_b[w.vidx] = None
    for step in range(m + 2 + layout):                       # orders 0, 1, 2 warming up, then steady state
        t = [w.times[step]] * B
        t_tgt = [w.times[step + 1]] * B
        feats = [src.feature(e, step, t) for e in range(ne)]
        a.update_forecast(feats, t, t_tgt, give_a)
        b.update(feats, t)
        b.commit_step()
        b.forecast(t_tgt, give_b)
        torch.cuda.synchronize()
        for e in range(ne):
            live = min(m, step) + 1
            assert torch.equal(bits(a.plane_tensor(e, 0)[:live]), bits(b.plane_tensor(e, 0)[:live])), (step, e)
            if e != w.vidx:
                assert torch.equal(bits(outs_a[e]), bits(outs_b[e])), (step, e)
        del feats
    a.close()
    b.close()


@pytest.mark.parametrize("dtype,tdt", [(1, torch.bfloat16), (0, torch.float32)])
@pytest.mark.parametrize("m,K", [(0, 2), (1, 8), (2, 3), (2, 8), (3, 2), (4, 5)])
def test_fused_reference_step_with_several_targets_equals_update_commit_forecast_multi(S, dtype, tdt, m, K):
    """K speculative times forecast in the reference step's own pass: tables and all K forecasts bit for bit
    those of update + commit + speca_forecast_multi (which the multi-horizon tests hold against the oracle),
    with warm-up orders, a sample that skips a step and keeps speculating, one that has dropped out, and an
    entry that is only updated."""
    B, ne = 3, len(ENTRIES)
    a = S.SpecaCache(ENTRIES, B, m, dtype, DEV)
    b = S.SpecaCache(ENTRIES, B, m, dtype, DEV)
    gen = torch.Generator(device=DEV).manual_seed(7 * m + K)
    active = torch.tensor([1, 1, 1], dtype=torch.uint8, device=DEV)
    active_b = active.clone()
    spec_a, spec_b = torch.zeros(B, dtype=torch.int32, device=DEV), torch.zeros(B, dtype=torch.int32, device=DEV)
    t = 1.0
    for k, mask in enumerate([[1, 1, 1]] * (m + 1) + [[1, 0, 1], [0, 1, 1], [1, 1, 1]]):
        t -= 0.04
        t_ref = [t - 0.002 * s for s in range(B)]
        targets = [[x - 0.006 * (j + 1) for x in t_ref] for j in range(K)]
        if k == m + 2:
            active[0] = 0                                    # sample 0 skips this step AND has dropped out: no forecast
            active_b[0] = 0                                  # (the next step, which it takes, re-arms it)
        feats = [torch.randn(B, n, d, generator=gen, device=DEV).to(tdt) for n, d in ENTRIES]
        outs_a = [torch.full((K, B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in ENTRIES]
        outs_b = [torch.full((K, B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in ENTRIES]
        skip = k % ne
        give_a = [None if e == skip else o for e, o in enumerate(outs_a)]
        give_b = [None if e == skip else o for e, o in enumerate(outs_b)]
        a.update_forecast_multi(feats, t_ref, targets, give_a, mask=mask, active=active, spec_count=spec_a, rearm=active)
        b.update_activate(feats, t_ref, mask, spec_b, active_b)
        b.commit_step()
        b.forecast_multi(targets, give_b, active_b)
        torch.cuda.synchronize()
        assert torch.equal(active, active_b) and torch.equal(spec_a, spec_b)
        refs = a.state()[0]
        assert refs == b.state()[0]
        for e in range(ne):
            for s in range(B):
                live = min(m, refs[s] - 1) + 1
                assert torch.equal(bits(a.plane_tensor(e, s)[:live]), bits(b.plane_tensor(e, s)[:live])), ("planes", k, e, s)
            assert torch.equal(bits(outs_a[e]), bits(outs_b[e])), ("forecasts", k, e)
            if e == skip:
                assert bool((outs_a[e].float() == 7.0).all())
        if k == m + 2:
            assert bool((outs_a[(skip + 1) % ne][:, 0].float() == 7.0).all())     # the dropped-out sample's rows are untouched
    assert a.stats()["update_forecast_launches"] == m + 4
    with pytest.raises(S.SpecaError):
        a.update_forecast_multi(feats, [t - 1.0] * B, [[0.0] * B] * 9, give_a)   # more targets than SPECA_MAX_HORIZON
    a.close()
    b.close()


def test_fused_reference_step_can_be_captured_into_a_cuda_graph(S):
    """The call neither allocates nor synchronises: captured once into a CUDA graph (nothing runs during the
    capture; the host-side history advances then) and replayed, it leaves the same tables and forecasts
    as the eager call on a twin cache."""
    entries = [(40, 1030), (301, 1152)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(91)
    a = S.SpecaCache(entries, B, m, 1, DEV)
    b = S.SpecaCache(entries, B, m, 1, DEV)
    feats = [torch.randn(B, n, d, generator=gen, device=DEV).bfloat16() for n, d in entries]
    for k, t in enumerate((1.0, 0.93)):                      # two ordinary reference steps on both
        f0 = [torch.randn(B, n, d, generator=gen, device=DEV).bfloat16() for n, d in entries]
        for c in (a, b):
            c.update(f0, [t] * B)
            c.commit_step()
    outs_a = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    outs_b = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    act = torch.ones(B, dtype=torch.uint8, device=DEV)
    a.update_forecast(feats, [0.9] * B, [0.87] * B, outs_a, mask=[1, 1, 0, 1], active=act)
    torch.cuda.synchronize()
    side = torch.cuda.Stream(DEV)
    side.wait_stream(torch.cuda.current_stream(DEV))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            b.update_forecast(feats, [0.9] * B, [0.87] * B, outs_b, mask=[1, 1, 0, 1], active=act)
    torch.cuda.current_stream(DEV).wait_stream(side)
    torch.cuda.synchronize()
    assert all(bool((o == 0).all()) for o in outs_b)          # captured, not run
    assert a.state()[0] == b.state()[0] == [3, 3, 2, 3]       # the history advanced at capture time
    graph.replay()
    torch.cuda.synchronize()
    for e in range(len(entries)):
        assert torch.equal(bits(outs_a[e]), bits(outs_b[e]))
        for s, refs in enumerate(a.state()[0]):               # the planes that hold a difference (the rest is unwritten memory)
            assert torch.equal(bits(a.plane_tensor(e, s)[:refs]), bits(b.plane_tensor(e, s)[:refs]))
    a.close()
    b.close()


@pytest.mark.parametrize("dtype,tdt", [(1, torch.bfloat16), (0, torch.float32)])
@pytest.mark.parametrize("basis", [0, 1, 2])
@pytest.mark.parametrize("m,K", [(0, 1), (1, 2), (2, 1), (2, 3), (3, 1), (4, 2)])
def test_fused_reference_step_on_a_raw_feature_cache(S, dtype, tdt, basis, m, K):
    """SPECA_LAYOUT_HISTORY: the step copies the feature into its ring plane and forms the weighted sum with
    the feature still in registers. Ring planes and forecasts bit for bit those of update + commit +
    speca_forecast_multi on a twin cache (which the raw-feature tests hold against the oracle), through
    the warm-up, past the ring's wrap, with a sample that skips a step and one that has dropped out."""
    B, ne = 3, len(ENTRIES)
    a = S.SpecaCache(ENTRIES, B, m, dtype, DEV, basis=basis, layout=S.SPECA_LAYOUT_HISTORY)
    b = S.SpecaCache(ENTRIES, B, m, dtype, DEV, basis=basis, layout=S.SPECA_LAYOUT_HISTORY)
    gen = torch.Generator(device=DEV).manual_seed(1000 + 10 * m + K)
    act_a = torch.ones(B, dtype=torch.uint8, device=DEV)
    act_b = torch.ones(B, dtype=torch.uint8, device=DEV)
    spec_a, spec_b = torch.zeros(B, dtype=torch.int32, device=DEV), torch.zeros(B, dtype=torch.int32, device=DEV)
    t = 1.0
    plan = [[1, 1, 1]] * (m + 1) + [[1, 0, 1], [0, 1, 1], [1, 1, 1], [1, 1, 1]]
    for k, mask in enumerate(plan):
        t -= 0.04 + 0.003 * (k % 2)
        t_ref = [t - 0.002 * s for s in range(B)]
        targets = [[x - 0.007 * (j + 1) for x in t_ref] for j in range(K)]
        if k == m + 2:
            act_a[0] = 0
            act_b[0] = 0
        feats = [torch.randn(B, n, d, generator=gen, device=DEV).to(tdt) for n, d in ENTRIES]
        outs_a = [torch.full((K, B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in ENTRIES]
        outs_b = [torch.full((K, B, n, d), 7.0, dtype=tdt, device=DEV) for n, d in ENTRIES]
        skip = k % ne
        give_a = [None if e == skip else o for e, o in enumerate(outs_a)]
        give_b = [None if e == skip else o for e, o in enumerate(outs_b)]
        a.update_forecast_multi(feats, t_ref, targets, give_a, mask=mask, active=act_a, spec_count=spec_a, rearm=act_a)
        b.update_activate(feats, t_ref, mask, spec_b, act_b)
        b.commit_step()
        b.forecast_multi(targets, give_b, act_b)
        torch.cuda.synchronize()
        refs = a.state()[0]
        assert refs == b.state()[0]
        for e in range(ne):
            for s in range(B):
                live = min(m + 1, refs[s])                   # ring planes that hold a feature
                assert torch.equal(bits(a.plane_tensor(e, s)[:live]), bits(b.plane_tensor(e, s)[:live])), ("ring", k, e, s)
            assert torch.equal(bits(outs_a[e]), bits(outs_b[e])), ("forecasts", k, e)
        assert torch.equal(act_a, act_b) and torch.equal(spec_a, spec_b)
    a.close()
    b.close()


def test_fused_reference_step_with_features_already_in_their_ring_planes(S):
    """A model that writes its block output straight into the next ring plane (speca_cache_next_slot) passes
    that pointer, or SPECA_FEATURE_IN_PLACE: nothing is copied and the forecast reads the feature where it is."""
    entries = [(64, 1024), (9, 1031)]
    m = 2
    a = S.SpecaCache(entries, 1, m, 1, DEV, layout=S.SPECA_LAYOUT_HISTORY)
    b = S.SpecaCache(entries, 1, m, 1, DEV, layout=S.SPECA_LAYOUT_HISTORY)
    gen = torch.Generator(device=DEV).manual_seed(5)
    t = 1.0
    for k in range(m + 3):
        t -= 0.05
        feats = [torch.randn(1, n, d, generator=gen, device=DEV).bfloat16() for n, d in entries]
        slots = [a.next_slot_tensor(e) for e in range(len(entries))]
        for sl, f in zip(slots, feats):
            sl.copy_(f[0])
        outs_a = [torch.full((1, n, d), 7.0, dtype=torch.bfloat16, device=DEV) for n, d in entries]
        outs_b = [torch.full((1, n, d), 7.0, dtype=torch.bfloat16, device=DEV) for n, d in entries]
        launches = a.launches
        how = [slots[0], S.SPECA_FEATURE_IN_PLACE] if k % 2 else [S.SPECA_FEATURE_IN_PLACE, slots[1]]
        a.update_forecast(how, [t], [t - 0.02], outs_a)
        b.update(feats, [t])
        b.commit_step()
        b.forecast([t - 0.02], outs_b)
        torch.cuda.synchronize()
        assert a.launches == launches + 1
        for e in range(len(entries)):
            live = min(m + 1, k + 1)
            assert torch.equal(bits(a.plane_tensor(e, 0)[:live]), bits(b.plane_tensor(e, 0)[:live])), (k, e)
            assert torch.equal(bits(outs_a[e]), bits(outs_b[e])), (k, e)
    a.close()
    b.close()
