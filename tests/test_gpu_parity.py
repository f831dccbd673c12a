"""CUDA path vs CPU oracle, element by element, on identical seeded inputs (through the C ABI)."""
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
    binding._lib()  # fail loudly if the CUDA library is missing
    return binding


@pytest.fixture(scope="module")
def U():
    from tests import gpu_util
    return gpu_util


def rand_feats(entries, B, tdt, gen, scale=1.0):
    return [(torch.randn(B, n, d, generator=gen, device=DEV, dtype=torch.float32) * scale).to(tdt) for n, d in entries]


# ---------------------------------------------------------------------------------------------
# config 1: the tiny fp32 cache, whole sequence
# ---------------------------------------------------------------------------------------------

def test_tiny_config_full_sequence(S, U):
    w = W.tiny()
    src = W.FeatureSource(w, DEV)
    pair = U.Pair(w.entries, w.batch, w.max_order, w.dtype)
    B = w.batch
    for step in range(3):
        t = [w.times[step]] * B
        feats = [src.feature(e, step, t) for e in range(len(w.entries))]
        pair.update(feats, t)
        pair.commit()
        pair.check_tables("tiny ref %d" % step)
        pair.sync_tables()
    spec = torch.zeros(B, dtype=torch.int32, device=DEV)
    active = torch.ones(B, dtype=torch.uint8, device=DEV)
    act_cpu, cnt_cpu = [1] * B, [0] * B
    for k in range(1, 5):
        step = 2 + k
        t = [w.times[step]] * B
        pair.check_forecast(t, active=act_cpu, what="tiny forecast k=%d" % k)
        fresh = src.feature(pair.vidx, step, t)
        tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
        assert tau[0] == pytest.approx(O.tau_schedule(w.tau0, w.beta, w.total_steps - step, w.total_steps), rel=1e-15)
        e_got, a_got, e_want, a_want = pair.check_verify(fresh, t, tau, active=act_cpu, what="tiny verify k=%d" % k)
        acc_dev = torch.tensor([int(a) if a >= 0 else 0 for a in a_want], dtype=torch.uint8, device=DEV)
        idx = torch.full((B,), -1, dtype=torch.int32, device=DEV)
        n_act = torch.zeros(1, dtype=torch.int32, device=DEV)
        pair.gpu.select_adaptive(acc_dev, 3, 1, spec, active, idx, n_act)
        act_cpu, cnt_cpu, idx_cpu = O.select_adaptive([max(int(a), 0) for a in a_want], 3, 1, cnt_cpu, act_cpu)
        torch.cuda.synchronize()
        assert active.cpu().tolist() == act_cpu and spec.cpu().tolist() == cnt_cpu
        assert n_act.item() == len(idx_cpu) and idx.cpu().tolist()[: len(idx_cpu)] == idx_cpu
    assert pair.gpu.launches > 0
    pair.close()


# ---------------------------------------------------------------------------------------------
# ragged shapes, all orders, both bases, both dtypes
# ---------------------------------------------------------------------------------------------

RAGGED = [(37, 129), (5, 3), (64, 384), (1, 8192 * 2 + 24), (3, 8192), (1, 1)]


@pytest.mark.parametrize("path", [1, 2, 3])  # SPECA_PATH_DIRECT, SPECA_PATH_BULK, SPECA_PATH_WIDE
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("basis", [0, 1, 2])  # Taylor (Eq. 2-3), Newton, Adams-Bashforth
@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_ragged_shapes_all_orders(S, U, dtype, basis, m, path):
    B = 3
    gen = torch.Generator(device=DEV).manual_seed(1000 + 10 * m + basis)
    pair = U.Pair(RAGGED, B, m, dtype, basis, path=path)
    times = [1.0, 0.93, 0.9, 0.81, 0.8, 0.74]
    for step in range(m + 2):
        t = [times[step], times[step] - 0.003, times[step] + 0.001]  # per-sample times
        feats = rand_feats(RAGGED, B, pair.tdt, gen)
        pair.update(feats, t, per_entry_calls=(step % 2 == 1))
        pair.commit()
        pair.check_tables("ragged ref %d" % step)
        pair.sync_tables()
        tt = [x - 0.02 for x in t]
        pair.check_forecast(tt, what="ragged forecast after ref %d" % step)
    fresh = rand_feats([RAGGED[pair.vidx]], B, pair.tdt, gen)[0]
    pair.check_verify(fresh, [0.7] * B, [0.5, 1.5, 2.5])
    pair.close()


def test_verify_entry_spanning_many_tiles_and_clusters(S, U):
    """A verification entry large enough that every cluster gets several units and samples change
    inside a cluster's walk; also a non-default verify entry."""
    entries = [(300, 1152), (8, 64)]
    B, m = 5, 2
    gen = torch.Generator(device=DEV).manual_seed(77)
    pair = U.Pair(entries, B, m, 1, verify_entry=0)
    for step, t in enumerate([1.0, 0.9, 0.85]):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t] * B)
        pair.commit()
        pair.sync_tables()
    # fresh = forecast + small perturbation so that errors are spread around tau
    t = [0.8] * B
    outs = pair.check_forecast(t)
    noise = torch.randn(B, 300, 1152, generator=gen, device=DEV) * torch.tensor(
        [0.0, 0.01, 0.05, 0.2, 1.0], device=DEV).view(B, 1, 1)
    fresh = (outs[0].float() + noise).to(pair.tdt)
    e1, a1, _, _ = pair.check_verify(fresh, t, [0.03] * B)
    assert a1[0] == 1 and a1[-1] == 0
    # run to run identical (fixed reduction order)
    e2, a2, _, _ = pair.check_verify(fresh, t, [0.03] * B)
    assert np.array_equal(e1, e2) and np.array_equal(a1, a2)
    # exact match -> zero error, accepted even at tau = 0
    e3, a3, _, _ = pair.check_verify(outs[0], t, [0.0] * B)
    assert np.all(e3 == 0.0) and np.all(a3 == 1)
    pair.close()


# ---------------------------------------------------------------------------------------------
# masks: untouched means bit-for-bit untouched
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", [0, 1])
def test_masks_leave_other_samples_untouched(S, U, dtype):
    entries = [(16, 520), (33, 1031)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(5)
    pair = U.Pair(entries, B, m, dtype)
    pair.update(rand_feats(entries, B, pair.tdt, gen), [1.0] * B)
    pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.9] * B)
    pair.commit()
    pair.sync_tables()
    before = [[U.to_oracle(pair.gpu.plane_tensor(e, b)) for b in range(B)] for e in range(len(entries))]
    mask = [1, 0, 0, 1]
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.8, 0.8, 0.8, 0.75], mask)
    pair.commit()
    pair.check_tables("masked update")
    torch.cuda.synchronize()
    for e in range(len(entries)):
        for b in (1, 2):
            assert np.array_equal(U.to_oracle(pair.gpu.plane_tensor(e, b)), before[e][b])
    n_refs, t_last = pair.gpu.state()
    assert n_refs == [3, 2, 2, 3] and t_last == [0.8, 0.9, 0.9, 0.75]
    pair.sync_tables()
    # mixed orders (2,1,1,2) in one launch, device mask, sentinel in skipped rows
    pair.check_forecast([0.7] * B, active=[1, 1, 0, 1], sentinel=3.0, what="masked forecast")
    fresh = rand_feats([entries[1]], B, pair.tdt, gen)[0]
    pair.check_verify(fresh, [0.7] * B, [1.0] * B, active=[0, 1, 1, 0])
    # reset one sample: it is skipped under a device mask and refused without one
    pair.gpu.reset([0, 0, 1, 0])
    pair.cpu.reset([0, 0, 1, 0])
    pair.check_forecast([0.7] * B, active=[1, 1, 1, 1], sentinel=-2.0, what="forecast after reset")
    with pytest.raises(S.SpecaError) as ei:
        pair.gpu.forecast([0.7] * B, [torch.empty(B, n, d, dtype=pair.tdt, device=DEV) for n, d in entries])
    assert ei.value.status == S.SPECA_ERR_STATE
    pair.close()


@pytest.mark.parametrize("entry", [(17, 130), (40, 1030), (301, 1160)])   # 1, 3 and 22 tiles per sample
def test_verify_with_any_number_of_active_samples(S, U, entry):
    """The grid is sized for the whole batch, so with few active samples there are more clusters than
    tiles and some clusters own nothing; every ratio of clusters to tiles must find its partials."""
    entries = [(2, 8), entry]
    B, m = 64, 1
    gen = torch.Generator(device=DEV).manual_seed(911)
    rng = np.random.default_rng(12)
    pair = U.Pair(entries, B, m, 1)
    for t in (1.0, 0.9):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t] * B)
        pair.commit()
    pair.sync_tables()
    fresh = rand_feats([entry], B, pair.tdt, gen)[0]
    for n_on in (1, 2, 3, 5, 7, 11, 15, 23, 30, 31, 33, 47, 63, 64):
        act = [0] * B
        for b in rng.choice(B, n_on, replace=False):
            act[int(b)] = 1
        e, a, ew, aw = pair.check_verify(fresh, [0.85] * B, [1.0] * B, active=act, with_pred=(n_on % 2 == 0),
                                         what="%d of %d active" % (n_on, B))
        assert all(e[b] > 0.1 for b in range(B) if act[b])
    pair.close()


# ---------------------------------------------------------------------------------------------
# degenerate inputs
# ---------------------------------------------------------------------------------------------

def test_nan_inf_and_zero_features(S, U):
    entries = [(4, 2056)]
    B, m = 4, 1
    gen = torch.Generator(device=DEV).manual_seed(9)
    pair = U.Pair(entries, B, m, 1)
    f0 = rand_feats(entries, B, pair.tdt, gen)
    f1 = rand_feats(entries, B, pair.tdt, gen)
    pair.update(f0, [1.0] * B); pair.commit()
    pair.update(f1, [0.9] * B); pair.commit()
    pair.sync_tables()
    fresh = rand_feats(entries, B, pair.tdt, gen)[0]
    fresh[0, 1, 7] = float("nan")        # NaN anywhere rejects
    fresh[1] = 0                          # zero feature: only epsilon in the denominator
    fresh[2, 0, 0] = float("inf")         # inf/inf -> NaN -> reject
    e, a, ew, aw = pair.check_verify(fresh, [0.85] * B, [1e30] * B)
    assert a.tolist() == [0, 0, 0, 1] or a.tolist() == [0, 1, 0, 1]
    assert np.isnan(e[0]) and np.isnan(e[2]) and e[1] > 1e6
    pair.close()


def test_select_adaptive_random_against_oracle(S, U):
    rng = np.random.default_rng(3)
    for B, group in [(1, 1), (8, 1), (8, 2), (16, 2), (12, 4), (64, 1), (64, 8)]:
        cache = S.SpecaCache([(1, 8)], B, 0, 0, DEV)
        for trial in range(6):
            acc = rng.integers(0, 2, B).tolist()
            act = rng.integers(0, 2, B).tolist()
            cnt = rng.integers(0, 5, B).tolist()
            k_max = int(rng.integers(1, 6))
            d_acc = torch.tensor(acc, dtype=torch.uint8, device=DEV)
            d_act = torch.tensor(act, dtype=torch.uint8, device=DEV)
            d_cnt = torch.tensor(cnt, dtype=torch.int32, device=DEV)
            d_idx = torch.full((B,), -1, dtype=torch.int32, device=DEV)
            d_n = torch.full((1,), -1, dtype=torch.int32, device=DEV)
            cache.select_adaptive(d_acc, k_max, group, d_cnt, d_act, d_idx, d_n)
            want_act, want_cnt, want_idx = O.select_adaptive(acc, k_max, group, cnt, act)
            torch.cuda.synchronize()
            assert d_act.cpu().tolist() == want_act
            assert d_cnt.cpu().tolist() == want_cnt
            assert d_n.item() == len(want_idx)
            assert d_idx.cpu().tolist()[: len(want_idx)] == want_idx
        # re-activation after a reference step
        d_act = torch.zeros(B, dtype=torch.uint8, device=DEV)
        d_cnt = torch.full((B,), 3, dtype=torch.int32, device=DEV)
        mask = [b % 2 for b in range(B)]
        cache.activate(mask, d_cnt, d_act)
        torch.cuda.synchronize()
        assert d_act.cpu().tolist() == mask and d_cnt.cpu().tolist() == [0 if x else 3 for x in mask]
        cache.close()


# ---------------------------------------------------------------------------------------------
# argument errors: a status, never a launch
# ---------------------------------------------------------------------------------------------

def test_argument_errors_return_status(S):
    entries = [(8, 64), (4, 32)]
    B = 2
    c = S.SpecaCache(entries, B, 2, 1, DEV)
    f = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    launches0 = c.launches

    def status_of(fn):
        with pytest.raises(S.SpecaError) as ei:
            fn()
        return ei.value.status

    assert status_of(lambda: c.forecast([0.5] * B, f)) == S.SPECA_ERR_STATE          # nothing cached yet
    assert status_of(lambda: c.commit_step()) == S.SPECA_ERR_STATE                     # no step open
    assert status_of(lambda: c.update(f, [float("nan")] * B)) == S.SPECA_ERR_INVALID_ARG
    c.update([f[0], None], [1.0] * B)
    assert status_of(lambda: c.commit_step()) == S.SPECA_ERR_STATE                     # entry 1 missing
    assert status_of(lambda: c.update([f[0], None], [1.0] * B)) == S.SPECA_ERR_STATE   # entry 0 twice
    assert status_of(lambda: c.update([None, f[1]], [0.9] * B)) == S.SPECA_ERR_STATE   # other time, same step
    assert status_of(lambda: c.forecast([0.5] * B, f)) == S.SPECA_ERR_STATE            # step still open
    c.update([None, f[1]], [1.0] * B)
    c.commit_step()
    assert status_of(lambda: c.update(f, [1.0] * B)) == S.SPECA_ERR_ZERO_GAP
    odd = torch.zeros(B * 8 * 64 + 1, dtype=torch.bfloat16, device=DEV)
    assert status_of(lambda: S.speca_forecast(c.handle, [0.5] * B, None, [odd.data_ptr() + 1, None])) == S.SPECA_ERR_ALIGNMENT
    err = torch.zeros(B, device=DEV)
    acc = torch.zeros(B, dtype=torch.uint8, device=DEV)
    assert status_of(lambda: c.verify(f[1], [0.5] * B, [float("nan")] * B, err, acc)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.select_adaptive(acc, 0, 1, torch.zeros(B, dtype=torch.int32, device=DEV), acc)) == S.SPECA_ERR_INVALID_ARG
    assert status_of(lambda: c.select_adaptive(acc, 2, 3, torch.zeros(B, dtype=torch.int32, device=DEV), acc)) == S.SPECA_ERR_INVALID_ARG
    assert "select" in S.speca_last_error(c.handle)
    assert c.launches == launches0 + 2  # only the two valid updates launched
    # creation errors
    assert status_of(lambda: S.speca_cache_arena_bytes([(0, 4)], 1, 1, 1)) == S.SPECA_ERR_SHAPE
    assert status_of(lambda: S.speca_cache_arena_bytes([(4, 4)], 65, 1, 1)) == S.SPECA_ERR_SHAPE
    assert status_of(lambda: S.speca_cache_arena_bytes([(4, 4)], 1, 5, 1)) == S.SPECA_ERR_SHAPE
    small = torch.empty(1024, dtype=torch.uint8, device=DEV)
    assert status_of(lambda: S.speca_cache_create(entries, B, 2, 1, small)) == S.SPECA_ERR_NOMEM
    big = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
    assert status_of(lambda: S.speca_cache_create(entries, B, 2, 1, big.data_ptr() + 16, arena_bytes=(1 << 20) - 16,
                                                  device=0)) == S.SPECA_ERR_ALIGNMENT
    c.close()


# ---------------------------------------------------------------------------------------------
# cut-down copies of the model-shaped configs (same dim, dtype, time grid, value structure)
# ---------------------------------------------------------------------------------------------

@pytest.mark.parametrize("path", [0, 2])  # library default, and the TMA-staged variant
@pytest.mark.parametrize("name,kw", [
    ("dit_xl2", dict(max_entries=6, max_tokens=0)),
    ("flux", dict(max_entries=5, max_tokens=300)),
    ("hunyuan_video", dict(max_entries=4, max_tokens=1700)),
])
def test_model_shaped_configs_cut_down(S, U, name, kw, path):
    w = W.scaled(W.BY_NAME[name](), **kw)
    src = W.FeatureSource(w, DEV)
    B = w.batch
    pair = U.Pair(w.entries, B, w.max_order, w.dtype, path=path)
    pattern = W.reference_pattern(w)
    spec = torch.zeros(B, dtype=torch.int32, device=DEV)
    active = torch.ones(B, dtype=torch.uint8, device=DEV)
    n_spec = 0
    for step in range(9):
        t = [w.times[step]] * B
        if pattern[step]:
            feats = [src.feature(e, step, t) for e in range(len(w.entries))]
            pair.update(feats, t)
            pair.commit()
            pair.check_tables("%s ref step %d" % (name, step))
            pair.sync_tables()
        else:
            pair.check_forecast(t, what="%s forecast step %d" % (name, step))
            fresh = src.feature(pair.vidx, step, t)
            tau = [S.speca_tau(w.tau0, w.beta, w.total_steps - step, w.total_steps)] * B
            pair.check_verify(fresh, t, tau, what="%s verify step %d" % (name, step))
            n_spec += 1
    assert n_spec >= 4
    pair.close()


def test_adaptive_batch_rejected_samples_stop_forecasting(S, U):
    """FLUX-shaped, cut down: samples with different noise levels accept or reject differently;
    a rejected sample drops out of later forecasts (its output rows stay untouched)."""
    for m in (1, 2, 3):
        w = W.scaled(W.flux_adaptive(max_order=m, batch=8), max_entries=3, max_tokens=200)
        src = W.FeatureSource(w, DEV)
        B = w.batch
        pair = U.Pair(w.entries, B, m, w.dtype)
        for step in range(m + 1):
            t = [w.times[step]] * B
            pair.update([src.feature(e, step, t) for e in range(len(w.entries))], t)
            pair.commit()
            pair.sync_tables()
        spec = torch.zeros(B, dtype=torch.int32, device=DEV)
        active = torch.ones(B, dtype=torch.uint8, device=DEV)
        act_cpu, cnt_cpu = [1] * B, [0] * B
        seen_reject = False
        for k in range(1, 7):
            step = m + k
            t = [w.times[step]] * B
            pair.check_forecast(t, active=act_cpu, sentinel=5.0, what="adaptive m=%d k=%d" % (m, k))
            fresh = src.feature(pair.vidx, step, t)
            tau = [0.12] * B
            _, a_got, e_want, a_want = pair.check_verify(fresh, t, tau, active=act_cpu)
            acc = [1 if a == 1 else 0 for a in a_want]
            d_acc = torch.tensor(acc, dtype=torch.uint8, device=DEV)
            pair.gpu.select_adaptive(d_acc, 6, 1, spec, active)
            act_cpu, cnt_cpu, _ = O.select_adaptive(acc, 6, 1, cnt_cpu, act_cpu)
            torch.cuda.synchronize()
            assert active.cpu().tolist() == act_cpu
            seen_reject |= (0 in act_cpu)
            if not any(act_cpu):
                break
        assert seen_reject
        pair.close()


# ---------------------------------------------------------------------------------------------
# checkpoint / resume: arena bytes + reference history are the whole state
# ---------------------------------------------------------------------------------------------

def test_checkpoint_and_resume_continue_bit_for_bit(S, U):
    entries = [(16, 520), (33, 1031)]
    B, m = 3, 2
    gen = torch.Generator(device=DEV).manual_seed(12)
    a = S.SpecaCache(entries, B, m, 1, DEV)
    feats = [rand_feats(entries, B, torch.bfloat16, gen) for _ in range(4)]
    a.update(feats[0], [1.0, 1.0, 1.0]); a.commit_step()
    a.update(feats[1], [0.9, 0.91, 0.9], [1, 1, 0]); a.commit_step()
    torch.cuda.synchronize()
    saved_arena = a.arena.clone()
    n_refs, t_hist = S.speca_cache_get_history(a.handle, B)
    assert n_refs == [2, 2, 1] and t_hist[1][:2] == [0.91, 1.0] and np.isnan(t_hist[2][1])
    # a second cache over a copy of the bytes, history installed
    b = S.SpecaCache(entries, B, m, 1, DEV)
    b.arena.copy_(saved_arena)
    S.speca_cache_set_history(b.handle, n_refs, t_hist)
    assert b.state() == a.state()
    for c in (a, b):
        c.update(feats[2], [0.8, 0.8, 0.8]); c.commit_step()
    outs_a = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    outs_b = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    a.forecast([0.77] * B, outs_a)
    b.forecast([0.77] * B, outs_b)
    torch.cuda.synchronize()
    for x, y in zip(outs_a, outs_b):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    with pytest.raises(S.SpecaError) as ei:
        S.speca_cache_set_history(b.handle, [1, -1, 0], t_hist)
    assert ei.value.status == S.SPECA_ERR_INVALID_ARG
    b.update(feats[3], [0.7] * B)
    with pytest.raises(S.SpecaError) as ei:
        S.speca_cache_set_history(b.handle, n_refs, t_hist)
    assert ei.value.status == S.SPECA_ERR_STATE
    a.close(); b.close()


def test_arena_that_is_only_256_byte_aligned(S, U):
    """4 KB alignment of the arena is a speed matter only: at base + 256 the planes start 256 bytes
    off their 4 KB boundaries and every result must be the same."""
    entries = [(37, 129), (64, 384), (3, 8192)]
    B, m = 2, 2
    gen = torch.Generator(device=DEV).manual_seed(31)
    nbytes = S.speca_cache_arena_bytes(entries, B, m, 1)
    raw = torch.empty(nbytes + 4096, dtype=torch.uint8, device=DEV)
    aligned = S.SpecaCache(entries, B, m, 1, DEV)
    handle = S.speca_cache_create(entries, B, m, 1, raw.data_ptr() + 256, arena_bytes=nbytes, device=0)
    feats = [rand_feats(entries, B, torch.bfloat16, gen) for _ in range(3)]
    for k, f in enumerate(feats):
        t = [1.0 - 0.1 * k] * B
        aligned.update(f, t); aligned.commit_step()
        S.speca_cache_update(handle, f, t); S.speca_cache_commit_step(handle)
    oa = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    ob = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
    aligned.forecast([0.72] * B, oa)
    S.speca_forecast(handle, [0.72] * B, None, ob)
    ea, eb = torch.zeros(B, device=DEV), torch.zeros(B, device=DEV)
    aa, ab = torch.zeros(B, dtype=torch.uint8, device=DEV), torch.zeros(B, dtype=torch.uint8, device=DEV)
    fresh = rand_feats([entries[-1]], B, torch.bfloat16, gen)[0]
    aligned.verify(fresh, [0.72] * B, [1.5] * B, ea, aa)
    S.speca_verify(handle, fresh, [0.72] * B, [1.5] * B, None, None, eb, ab)
    torch.cuda.synchronize()
    for x, y in zip(oa, ob):
        assert torch.equal(x.view(torch.int16), y.view(torch.int16))
    assert torch.equal(ea, eb) and torch.equal(aa, ab)
    S.speca_cache_destroy(handle)
    aligned.close()
