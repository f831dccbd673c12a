"""speca_verify_select (verification and the per-sample continuation rule in one launch) against the
two separate calls on the same inputs -- bit for bit -- and against the oracle's decisions."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

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


def rand_feats(entries, B, tdt, gen):
    return [torch.randn(B, n, d, generator=gen, device=DEV, dtype=torch.float32).to(tdt) for n, d in entries]


def both_ways(pair, fresh, t, tau, act, cnt, k_max, group, metric=0):
    """Runs verify + select, then the fused call, from the same state. Returns both result sets."""
    B = pair.B
    n, d = pair.entries[pair.vidx]
    dev = lambda x, dt: torch.tensor(x, dtype=dt, device=DEV)
    # two calls
    err_a = torch.full((B,), -7.0, device=DEV)
    acc_a = torch.zeros(B, dtype=torch.uint8, device=DEV)
    act_a, cnt_a = dev(act, torch.uint8), dev(cnt, torch.int32)
    idx_a, n_a = torch.full((B,), -1, dtype=torch.int32, device=DEV), torch.full((1,), -1, dtype=torch.int32, device=DEV)
    pred_a = torch.zeros(B, n, d, dtype=pair.tdt, device=DEV)
    pair.gpu.verify(fresh, t, tau, err_a, acc_a, act_a, pred_a, metric=metric)
    pair.gpu.select_adaptive(acc_a, k_max, group, cnt_a, act_a, idx_a, n_a)
    # one call
    err_b = torch.full((B,), -7.0, device=DEV)
    acc_b = torch.zeros(B, dtype=torch.uint8, device=DEV)
    act_b, cnt_b = dev(act, torch.uint8), dev(cnt, torch.int32)
    nxt_b = torch.full((B,), 5, dtype=torch.uint8, device=DEV)
    idx_b, n_b = torch.full((B,), -1, dtype=torch.int32, device=DEV), torch.full((1,), -1, dtype=torch.int32, device=DEV)
    pred_b = torch.zeros(B, n, d, dtype=pair.tdt, device=DEV)
    launches = pair.gpu.launches
    pair.gpu.verify_select(fresh, t, tau, err_b, acc_b, act_b, nxt_b, k_max, group, cnt_b, idx_b, n_b, pred_b, metric=metric)
    assert pair.gpu.launches == launches + 1
    torch.cuda.synchronize()
    assert act_b.cpu().tolist() == act, "the step's own mask must stay as it was"
    two = dict(err=err_a.cpu().numpy(), acc=acc_a.cpu().tolist(), act=act_a.cpu().tolist(), cnt=cnt_a.cpu().tolist(),
               n=n_a.item(), idx=idx_a.cpu().tolist(), pred=pred_a)
    one = dict(err=err_b.cpu().numpy(), acc=acc_b.cpu().tolist(), act=nxt_b.cpu().tolist(), cnt=cnt_b.cpu().tolist(),
               n=n_b.item(), idx=idx_b.cpu().tolist(), pred=pred_b)
    return two, one


def assert_same(two, one):
    assert np.array_equal(two["err"].view(np.uint32), one["err"].view(np.uint32))
    assert two["acc"] == one["acc"] and two["act"] == one["act"] and two["cnt"] == one["cnt"]
    assert two["n"] == one["n"] and two["idx"][: two["n"]] == one["idx"][: one["n"]]
    assert torch.equal(two["pred"].view(torch.uint8), one["pred"].view(torch.uint8))


@pytest.mark.parametrize("metric", [O.METRIC_L2, O.METRIC_LINF])
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("B,group,entry", [(8, 1, (301, 1160)), (8, 2, (301, 1160)), (6, 3, (5, 24)), (64, 8, (17, 130)),
                                           (1, 1, (2050, 1152))])
def test_fused_call_equals_the_two_calls_and_the_oracle(S, U, metric, dtype, B, group, entry):
    entries = [(3, 16), entry]
    m = 2
    gen = torch.Generator(device=DEV).manual_seed(4100 + B + group + metric)
    rng = np.random.default_rng(B * 7 + group)
    pair = U.Pair(entries, B, m, dtype)
    for t in (1.0, 0.93, 0.9):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t] * B)
        pair.commit()
        pair.sync_tables()
    t = [0.86] * B
    outs = pair.check_forecast(t)
    level = torch.tensor(rng.choice([0.0, 0.01, 0.05, 0.3], B), device=DEV, dtype=torch.float32).view(B, 1, 1)
    fresh = (outs[1].float() + level * torch.randn(B, *entry, generator=gen, device=DEV)).to(pair.tdt)
    tau = [0.03] * B
    for trial in range(3):
        act = rng.integers(0, 2, B).tolist() if trial else [1] * B
        cnt = rng.integers(0, 4, B).tolist()
        k_max = int(rng.integers(1, 6))
        two, one = both_ways(pair, fresh, t, tau, act, cnt, k_max, group, metric)
        assert_same(two, one)
        # and the decisions the oracle takes (skipping samples within tolerance of the threshold)
        e_want, a_want, _ = pair.cpu.verify(U.to_oracle(fresh).reshape(B, -1), t, tau, act, metric=metric)
        near = [a_want[b] >= 0 and abs(e_want[b] - float(np.float32(tau[b]))) < 1e-3 for b in range(B)]
        if not any(near):
            want_act, want_cnt, want_idx = O.select_adaptive([max(int(a), 0) for a in a_want], k_max, group, cnt, act)
            assert one["act"] == want_act and one["cnt"] == want_cnt
            assert one["n"] == len(want_idx) and one["idx"][: one["n"]] == want_idx
    pair.close()


def test_nobody_active_and_nobody_with_a_table(S, U):
    entries = [(4, 32), (40, 256)]
    B = 4
    gen = torch.Generator(device=DEV).manual_seed(5)
    pair = U.Pair(entries, B, 1, 1)
    fresh = rand_feats(entries, B, pair.tdt, gen)[1]
    # no reference step yet: nothing is verified, the continuation rule still runs on what it is given
    two, one = both_ways(pair, fresh, [0.9] * B, [0.5] * B, [1, 0, 1, 0], [0, 1, 2, 3], 4, 1)
    assert_same(two, one)
    assert one["act"] == [0, 0, 0, 0] and one["n"] == 0 and (one["err"] == -7.0).all()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [1.0] * B)
    pair.commit()
    # tables exist, nobody active
    two, one = both_ways(pair, fresh, [0.9] * B, [0.5] * B, [0] * B, [1] * B, 4, 2)
    assert_same(two, one)
    assert one["act"] == [0] * B and one["n"] == 0 and one["cnt"] == [1] * B and (one["err"] == -7.0).all()
    pair.close()


def test_argument_errors(S):
    B = 4
    c = S.SpecaCache([(8, 64)], B, 1, 1, DEV)
    f = torch.zeros(B, 8, 64, dtype=torch.bfloat16, device=DEV)
    c.update([f], [1.0] * B)
    c.commit_step()
    err, acc = torch.zeros(B, device=DEV), torch.zeros(B, dtype=torch.uint8, device=DEV)
    masks = torch.ones(2 * B, dtype=torch.uint8, device=DEV)
    cnt = torch.zeros(B, dtype=torch.int32, device=DEV)
    launches = c.launches

    def status_of(fn):
        with pytest.raises(S.SpecaError) as ei:
            fn()
        return ei.value.status

    t, tau = [0.9] * B, [0.1] * B
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, masks[:B], masks[:B], 2, 1, cnt)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, masks[:B], masks[2:2 + B], 2, 1, cnt)) == S.SPECA_ERR_INVALID_ARG
    assert "overlap" in S.speca_last_error(c.handle)
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, None, masks[B:], 2, 1, cnt)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, masks[:B], masks[B:], 0, 1, cnt)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, masks[:B], masks[B:], 2, 3, cnt)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.verify_select(f, t, tau, err, acc, masks[:B], masks[B:], 2, 1, None)) == S.SPECA_ERR_INVALID_ARG
    assert c.launches == launches
    c.verify_select(f, t, tau, err, acc, masks[:B], masks[B:], 2, 1, cnt)   # adjacent buffers are fine
    torch.cuda.synchronize()
    assert acc.cpu().tolist() == [1] * B and masks[B:].cpu().tolist() == [1] * B and cnt.cpu().tolist() == [1] * B
    c.close()


def test_speculative_steps_replay_from_a_cuda_graph(S, U):
    """The calls neither synchronise nor allocate, so a run of speculative steps (forecast, then
    verification + continuation, at two successive times) can be captured once into a CUDA graph and
    replayed on new verification features: same bits as the eager calls."""
    entries = [(40, 1030), (301, 1160)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(31)
    pair = U.Pair(entries, B, m, 1)
    for t in (1.0, 0.93, 0.9):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t] * B)
        pair.commit()
    t1, t2, tau = [0.87] * B, [0.84] * B, [0.05] * B
    c = pair.gpu

    def buffers():
        return dict(outs=[[torch.zeros(B, n, d, dtype=pair.tdt, device=DEV) for n, d in entries] for _ in range(2)],
                    err=torch.zeros(2, B, device=DEV), acc=torch.zeros(2, B, dtype=torch.uint8, device=DEV),
                    masks=torch.ones(3, B, dtype=torch.uint8, device=DEV), cnt=torch.zeros(B, dtype=torch.int32, device=DEV))

    fresh = [torch.zeros(B, *entries[1], dtype=pair.tdt, device=DEV) for _ in range(2)]

    def steps(x):
        c.forecast(t1, x["outs"][0], x["masks"][0])
        c.verify_select(fresh[0], t1, tau, x["err"][0], x["acc"][0], x["masks"][0], x["masks"][1], 4, 1, x["cnt"])
        c.forecast(t2, x["outs"][1], x["masks"][1])
        c.verify_select(fresh[1], t2, tau, x["err"][1], x["acc"][1], x["masks"][1], x["masks"][2], 4, 1, x["cnt"])

    def new_fresh(seed):
        g = torch.Generator(device=DEV).manual_seed(seed)
        ref = buffers()
        c.forecast(t1, ref["outs"][0]); c.forecast(t2, ref["outs"][1])
        level = torch.tensor([0.0, 0.01, 0.4, 0.02], device=DEV).view(B, 1, 1).roll(seed, 0)
        for k in range(2):
            fresh[k].copy_((ref["outs"][k][1].float() + level * torch.randn(B, *entries[1], generator=g, device=DEV)).to(pair.tdt))

    graphed = buffers()
    new_fresh(1)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    launches = c.launches
    with torch.cuda.graph(graph):
        steps(graphed)
    assert c.launches == launches + 4
    for seed in (1, 2, 3):
        new_fresh(seed)
        eager = buffers()
        steps(eager)
        graphed["masks"].fill_(1); graphed["cnt"].zero_(); graphed["acc"].zero_(); graphed["err"].zero_()
        for o in graphed["outs"][0] + graphed["outs"][1]:
            o.zero_()          # rows of samples that this replay leaves out must compare equal to the eager zeros
        graph.replay()
        torch.cuda.synchronize()
        for k in ("err", "acc", "masks", "cnt"):
            assert torch.equal(eager[k].view(torch.uint8), graphed[k].view(torch.uint8)), (seed, k)
        for a, b_ in zip(eager["outs"], graphed["outs"]):
            for x, y in zip(a, b_):
                assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))
        want = [0 if lv == 0.4 else 1 for lv in np.roll([0.0, 0.01, 0.4, 0.02], seed)]
        assert eager["acc"][0].cpu().tolist() == want and eager["masks"][1].cpu().tolist() == want
        assert eager["outs"][1][1][want.index(0)].abs().sum().item() == 0     # dropped after step 1: not forecast at step 2
    pair.close()


def test_two_handles_on_two_streams_do_not_disturb_each_other(S, U):
    """Each handle carries its own reduction scratch and ticket, so two caches can work on two streams at
    once: results equal those of running them one after the other."""
    entries = [(40, 1030), (301, 1160)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(57)
    caches = [S.SpecaCache(entries, B, m, 1, DEV) for _ in range(2)]
    feats = [[rand_feats(entries, B, torch.bfloat16, gen) for _ in range(3)] for _ in range(2)]
    fresh = [rand_feats(entries, B, torch.bfloat16, gen)[1] for _ in range(2)]

    def run(streams, rounds=6):
        res = []
        for c in caches:
            c.reset()
        bufs = [dict(outs=[torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries],
                     err=torch.zeros(rounds, B, device=DEV), acc=torch.zeros(rounds, B, dtype=torch.uint8, device=DEV),
                     cur=torch.ones(B, dtype=torch.uint8, device=DEV), nxt=torch.zeros(rounds, B, dtype=torch.uint8, device=DEV),
                     cnt=torch.zeros(B, dtype=torch.int32, device=DEV)) for _ in caches]
        torch.cuda.synchronize()
        for k, t in enumerate((1.0, 0.93, 0.9)):
            for i, c in enumerate(caches):
                c.update(feats[i][k], [t] * B, stream=streams[i])
                c.commit_step()
        for r in range(rounds):
            tt = [0.88 - 0.01 * r] * B
            for i, c in enumerate(caches):      # interleaved enqueue: the two streams overlap on the device
                c.forecast(tt, bufs[i]["outs"], stream=streams[i])
                c.verify_select(fresh[i], tt, [1e30] * B, bufs[i]["err"][r], bufs[i]["acc"][r], bufs[i]["cur"],
                                bufs[i]["nxt"][r], 1 << 20, 1, bufs[i]["cnt"], stream=streams[i])
        torch.cuda.synchronize()
        return [(b["err"].clone(), b["acc"].clone(), b["nxt"].clone(), b["cnt"].clone(), [o.clone() for o in b["outs"]]) for b in bufs]

    main = torch.cuda.current_stream()
    serial = run([main, main])
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    overlapped = run([s1, s2])
    for a, b_ in zip(serial, overlapped):
        for x, y in zip(a[:4], b_[:4]):
            assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))
        for x, y in zip(a[4], b_[4]):
            assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))
    assert bool((serial[0][1] == 1).all()) and serial[0][3].tolist() == [6] * B
    for c in caches:
        c.close()


@pytest.mark.parametrize("path,layout", [(0, 0), (1, 0), (2, 0), (0, 1)])
def test_update_that_also_rearms_the_samples(S, U, path, layout):
    """speca_cache_update_activate = speca_cache_update + speca_activate for the masked samples: same
    tables, same mask and counters, one launch fewer (the staged kernels keep a launch of their own)."""
    entries = [(37, 129), (64, 384)]
    B, m = 5, 2
    gen = torch.Generator(device=DEV).manual_seed(61)
    a = S.SpecaCache(entries, B, m, 1, DEV, path=path, layout=layout)
    b = S.SpecaCache(entries, B, m, 1, DEV, path=path, layout=layout)
    act = [torch.tensor([0, 1, 0, 1, 0], dtype=torch.uint8, device=DEV) for _ in range(2)]
    cnt = [torch.tensor([3, 1, 4, 1, 5], dtype=torch.int32, device=DEV) for _ in range(2)]
    clock = 1.0
    for step, mask in enumerate([None, [1, 0, 1, 0, 0], [0, 0, 0, 0, 1], None]):
        clock -= 0.04
        feats = rand_feats(entries, B, torch.bfloat16, gen)
        la, lb = a.launches, b.launches
        a.update(feats, [clock] * B, mask)
        a.commit_step()
        a.activate(mask, cnt[0], act[0])
        b.update_activate(feats, [clock] * B, mask, cnt[1], act[1])
        b.commit_step()
        torch.cuda.synchronize()
        assert a.launches - la == 2 and b.launches - lb == (2 if path == 2 else 1)
        la, lb = a.launches, b.launches
        assert torch.equal(act[0], act[1]) and torch.equal(cnt[0], cnt[1])
        if step >= 1:     # every sample has a reference by now: the two caches must forecast the same bits
            oa = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
            ob = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
            a.forecast([clock - 0.02] * B, oa)
            b.forecast([clock - 0.02] * B, ob)
            torch.cuda.synchronize()
            assert all(torch.equal(x.view(torch.int16), y.view(torch.int16)) for x, y in zip(oa, ob))
        act[0][2] = act[1][2] = 0                      # something for the next step to re-arm
        cnt[0][2] = cnt[1][2] = 7
    if layout == 1:   # features already in place: nothing is copied, the re-arming runs on its own
        nxt = rand_feats(entries, B, torch.bfloat16, gen)
        for e in range(len(entries)):
            for smp in range(B):      # the masked steps above left the samples at different ring positions
                b.next_slot_tensor(e, smp).copy_(nxt[e][smp])
        lb = b.launches
        b.update_activate([S.SPECA_FEATURE_IN_PLACE] * len(entries), [clock - 0.04] * B, None, cnt[1], act[1])
        b.commit_step()
        torch.cuda.synchronize()
        st = b.stats()
        assert b.launches - lb == 1 and st["activate_launches"] == 1 and act[1].tolist() == [1] * B and cnt[1].tolist() == [0] * B
    err = S.SpecaError
    with pytest.raises(err) as ei:
        b.update_activate(rand_feats(entries, B, torch.bfloat16, gen), [0.1] * B, None, None, act[1])
    assert ei.value.status == S.SPECA_ERR_INVALID_ARG
    a.close(); b.close()
