"""Seeded random scenarios: random shapes, batch sizes, orders, bases, storage types and kernel paths,
and a random sequence of masked reference steps, speculative steps (forecast, multi-horizon and summed
forecasts, verify under a random metric, the fused verify + continuation call) and resets -- every result
compared with the oracle. The hand-written cases elsewhere pick the shapes someone thought of; this file picks the others."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
MAX_ELEMS = 3_000_000   # per scenario, over all entries and samples: keeps the oracle in the seconds


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


@pytest.fixture(scope="module")
def U():
    from tests import gpu_util
    return gpu_util


def draw_shape(rng):
    B = int(rng.choice([1, 2, 3, 5, 8, 16, 33, 64]))
    n_entries = int(rng.integers(1, 6))
    budget = MAX_ELEMS // B
    entries = []
    for _ in range(n_entries):
        kind = rng.integers(0, 4)
        if kind == 0:      # a handful of elements
            n, d = int(rng.integers(1, 6)), int(rng.integers(1, 40))
        elif kind == 1:    # odd row length, around one tile
            n, d = int(rng.integers(1, 40)), int(rng.integers(100, 1400))
        elif kind == 2:    # model-like width, several tiles
            n, d = int(rng.integers(20, 400)), int(rng.choice([1152, 3072, 768]))
        else:              # one long row
            n, d = 1, int(rng.integers(8000, 70000))
        while n * d > budget // n_entries and n > 1:
            n = max(1, n // 2)
        if n * d > budget // n_entries:
            d = max(1, budget // n_entries)
        entries.append((n, d))
    return B, entries


@pytest.mark.parametrize("seed", list(range(64)))
def test_random_scenario(S, U, seed):
    rng = np.random.default_rng(90_000 + seed)
    gen = torch.Generator(device=DEV).manual_seed(90_000 + seed)
    B, entries = draw_shape(rng)
    m = int(rng.integers(0, 5))
    dtype = int(rng.integers(0, 2))
    basis = int(rng.integers(0, 3))
    path = int(rng.integers(0, 4))
    vidx = int(rng.integers(-1, len(entries)))
    layout = int(seed % 3 == 2)               # every third scenario runs on the raw-feature cache
    if layout == 1:
        path = int(rng.choice([0, 3]))        # which only the default kernels serve
    pair = U.Pair(entries, B, m, dtype, basis, verify_entry=vidx, path=path, layout=layout)
    nv, dv = entries[pair.vidx]
    # a second cache takes every reference step through the fused call (where that call exists): its planes
    # and its forecast must be, bit for bit, those of update + commit + forecast on the first one
    shadow = S.SpecaCache(entries, B, m, dtype, DEV, basis, vidx, path=path, layout=layout) if path in (0, 3) else None
    ones = torch.ones(B, dtype=torch.uint8, device=DEV)
    what = "seed %d (B=%d m=%d dtype=%d basis=%d path=%d layout=%d entries=%s)" % (seed, B, m, dtype, basis, path, layout, entries)

    def feats():
        return [torch.randn(B, n, d, generator=gen, device=DEV, dtype=torch.float32).to(pair.tdt) for n, d in entries]

    clock = 1.0
    cnt = [0] * B
    for step in range(int(rng.integers(m + 2, m + 7))):
        have = [int(r >= 1) for r in pair.cpu.n_refs]
        kind = "ref" if step == 0 or not any(have) else rng.choice(["ref", "spec", "spec", "reset"], p=[0.4, 0.3, 0.2, 0.1])
        clock -= float(rng.uniform(0.012, 0.06))
        jitter = rng.uniform(-0.004, 0.004, B)
        t = [clock + float(j) for j in jitter]
        if kind == "ref":
            mask = None if rng.random() < 0.4 else rng.integers(0, 2, B).tolist()
            if mask is not None and not any(mask):
                mask[int(rng.integers(0, B))] = 1
            fs = feats()
            pair.update(fs, t, mask, per_entry_calls=bool(rng.integers(0, 2)))
            pair.commit()
            pair.check_tables(what + " step %d tables" % step)
            if shadow is not None:
                t_next = [x - 0.009 for x in t]
                give = [torch.full((B, n, d), 2.5, dtype=pair.tdt, device=DEV) for n, d in entries]
                plain = [torch.full((B, n, d), 2.5, dtype=pair.tdt, device=DEV) for n, d in entries]
                skip = int(rng.integers(-1, len(entries)))          # one entry may be updated only
                if skip >= 0:
                    give[skip] = None
                shadow.update_forecast(fs, t, t_next, give, mask=mask, active=ones)
                pair.gpu.forecast(t_next, [None if e == skip else o for e, o in enumerate(plain)], ones)
                torch.cuda.synchronize()
                assert shadow.state()[0] == pair.gpu.state()[0], what
                for e in range(len(entries)):
                    for b in range(B):
                        live = min(m, pair.cpu.n_refs[b] - 1) + 1
                        if live > 0:
                            assert torch.equal(shadow.plane_tensor(e, b)[:live].contiguous().view(torch.uint8),
                                               pair.gpu.plane_tensor(e, b)[:live].contiguous().view(torch.uint8)), \
                                what + " step %d fused tables entry %d sample %d" % (step, e, b)
                    if e != skip:
                        assert torch.equal(give[e].view(torch.uint8), plain[e].view(torch.uint8)), what + " step %d fused forecast entry %d" % (step, e)
            pair.sync_tables()
            if shadow is not None:
                for e in range(len(entries)):
                    for b in range(B):
                        shadow.plane_tensor(e, b).copy_(pair.gpu.plane_tensor(e, b))
        elif kind == "reset":
            mask = rng.integers(0, 2, B).tolist()
            pair.gpu.reset(mask)
            pair.cpu.reset(mask)
            if shadow is not None:
                shadow.reset(mask)
        else:
            act = [h & int(a) for h, a in zip(have, rng.integers(0, 2, B).tolist())]
            if rng.random() < 0.3:
                act = list(have)
            outs = pair.check_forecast(t, active=act, sentinel=2.5, what=what + " step %d forecast" % step)
            # several targets at once: row 0 is this very forecast, bit for bit
            t2 = [x - 0.007 for x in t]
            mask_dev = torch.tensor(act, dtype=torch.uint8, device=DEV)
            multi = [torch.full((2, B, n, d), 2.5, dtype=pair.tdt, device=DEV) for n, d in entries]
            pair.gpu.forecast_multi([t, t2], multi, mask_dev)
            # and an entry consumed twice as a sum, against the oracle's sum
            e0 = int(rng.integers(0, len(entries)))
            total = torch.full((B, *entries[e0]), 2.5, dtype=pair.tdt, device=DEV)
            pair.gpu.forecast_sum([e0, e0], t, total, None, mask_dev)
            torch.cuda.synchronize()
            for e in range(len(entries)):
                assert torch.equal(multi[e][0].view(torch.uint8), outs[e].view(torch.uint8)), what + " multi row 0 entry %d" % e
            init = U.to_oracle(torch.full((B, entries[e0][0] * entries[e0][1]), 2.5, dtype=pair.tdt))
            want_sum = pair.cpu.forecast_sum([e0, e0], t, None, act, out=init)
            got_sum = U.to_oracle(total).reshape(B, -1)
            for b in range(B):
                if not act[b]:
                    assert np.array_equal(got_sum[b], want_sum[b]), what
                    continue
                scale = 2 * (pair.history_scale(e0, b, t[b]) if layout == 1 else
                             U.term_scale(pair.cpu.planes[e0][b], pair.forecast_weights(b, t[b])))
                U.assert_close_storage(got_sum[b], want_sum[b], dtype, scale, what + " sum of entry %d twice, sample %d" % (e0, b))
            level = torch.tensor(rng.choice([0.0, 0.02, 0.3], B), device=DEV, dtype=torch.float32).view(B, 1, 1)
            fresh = (outs[pair.vidx].float() + level * torch.randn(B, nv, dv, generator=gen, device=DEV)).to(pair.tdt)
            metric = int(rng.integers(0, 4))
            tau = [1e-3 if metric == O.METRIC_COSINE else 0.05] * B
            pair.check_verify(fresh, t, tau, active=act, with_pred=bool(rng.integers(0, 2)), metric=metric,
                              ulp_slack=(metric == O.METRIC_LINF), what=what + " step %d verify metric %d" % (step, metric))
            # the fused call against the two calls, from the same state
            k_max, group = int(rng.integers(1, 5)), int(rng.choice([g for g in (1, 2, 4) if B % g == 0]))
            err2, acc2 = torch.zeros(B, device=DEV), torch.zeros(B, dtype=torch.uint8, device=DEV)
            err1, acc1 = torch.zeros(B, device=DEV), torch.zeros(B, dtype=torch.uint8, device=DEV)
            m2, m1 = torch.tensor(act, dtype=torch.uint8, device=DEV), torch.tensor(act, dtype=torch.uint8, device=DEV)
            c2, c1 = torch.tensor(cnt, dtype=torch.int32, device=DEV), torch.tensor(cnt, dtype=torch.int32, device=DEV)
            nxt = torch.zeros(B, dtype=torch.uint8, device=DEV)
            pair.gpu.verify(fresh, t, tau, err2, acc2, m2, metric=metric)
            pair.gpu.select_adaptive(acc2, k_max, group, c2, m2)
            pair.gpu.verify_select(fresh, t, tau, err1, acc1, m1, nxt, k_max, group, c1, metric=metric)
            torch.cuda.synchronize()
            assert torch.equal(err1.view(torch.int32), err2.view(torch.int32)) and torch.equal(acc1, acc2), what
            assert torch.equal(nxt, m2) and torch.equal(c1, c2), what
            want_act, want_cnt, _ = O.select_adaptive(acc2.cpu().tolist(), k_max, group, cnt, act)
            assert nxt.cpu().tolist() == want_act and c1.cpu().tolist() == want_cnt, what
            cnt = want_cnt
    if shadow is not None:
        shadow.close()
    pair.close()
