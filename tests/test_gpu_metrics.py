"""The other verification metrics (l1, l-infinity, cosine distance) through speca_verify_metric,
against the oracle's plain loops, on ragged shapes, with masks and degenerate inputs."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
METRICS = [O.METRIC_L2, O.METRIC_L1, O.METRIC_LINF, O.METRIC_COSINE]


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


@pytest.mark.parametrize("metric", METRICS)
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("m", [0, 2, 3])
def test_metrics_on_an_entry_spanning_many_tiles(S, U, metric, dtype, m):
    entries = [(8, 64), (301, 1152 + 8)]       # verify entry: ragged, ~21 tiles of 16 KB per sample
    B = 5
    gen = torch.Generator(device=DEV).manual_seed(700 + 10 * m + metric)
    pair = U.Pair(entries, B, m, dtype)
    for step, t in enumerate([1.0, 0.9, 0.85, 0.78][: m + 1]):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t] * B)
        pair.commit()
        pair.sync_tables()
    t = [0.75] * B
    outs = pair.check_forecast(t)
    noise = torch.randn(B, 301, 1160, generator=gen, device=DEV) * torch.tensor(
        [0.0, 0.01, 0.05, 0.2, 1.0], device=DEV).view(B, 1, 1)
    fresh = (outs[1].float() + noise).to(pair.tdt)
    tau = {O.METRIC_COSINE: [1e-3] * B}.get(metric, [0.03] * B)
    e1, a1, e_want, a_want = pair.check_verify(fresh, t, tau, metric=metric, ulp_slack=(metric == O.METRIC_LINF))
    assert a1[0] == 1 and a1[-1] == 0
    assert e1[0] == pytest.approx(0.0, abs=1e-6)      # fresh[0] is the library's own forecast
    # same inputs, same bits (fixed reduction order)
    e1b, a1b, _, _ = pair.check_verify(fresh, t, tau, metric=metric, ulp_slack=(metric == O.METRIC_LINF))
    assert np.array_equal(e1b, e1) and np.array_equal(a1b, a1)
    # masked samples are left alone (checked inside); the others only see another split of the tiles
    e2, a2, _, _ = pair.check_verify(fresh, t, tau, active=[1, 0, 1, 1, 0], metric=metric, ulp_slack=(metric == O.METRIC_LINF))
    assert np.allclose(e2[[0, 2, 3]], e1[[0, 2, 3]], rtol=1e-4, atol=1e-7) and np.array_equal(a2[[0, 2, 3]], a1[[0, 2, 3]])
    pair.close()


@pytest.mark.parametrize("metric", METRICS)
def test_metrics_nan_and_zero_features(S, U, metric):
    entries = [(4, 2056)]
    B, m = 4, 1
    gen = torch.Generator(device=DEV).manual_seed(9)
    pair = U.Pair(entries, B, m, 1)
    pair.update(rand_feats(entries, B, pair.tdt, gen), [1.0] * B); pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.9] * B); pair.commit()
    pair.sync_tables()
    fresh = rand_feats(entries, B, pair.tdt, gen)[0]
    fresh[0, 1, 7] = float("nan")        # NaN anywhere rejects, whatever the metric
    fresh[1] = 0                          # zero feature: only epsilon in the denominator
    fresh[2, 3, 2055] = float("nan")      # in the last, ragged vector of the row
    e, a, ew, aw = pair.check_verify(fresh, [0.85] * B, [1e30] * B, metric=metric)
    assert np.isnan(e[0]) and np.isnan(e[2]) and a[0] == 0 and a[2] == 0 and a[3] == 1
    pair.close()


def test_unknown_metric_is_refused(S):
    c = S.SpecaCache([(4, 32)], 1, 0, 1, DEV)
    f = torch.zeros(1, 4, 32, dtype=torch.bfloat16, device=DEV)
    c.update([f], [1.0]); c.commit_step()
    err = torch.zeros(1, device=DEV)
    acc = torch.zeros(1, dtype=torch.uint8, device=DEV)
    n = c.launches
    for bad in (-1, 4):
        with pytest.raises(S.SpecaError) as ei:
            c.verify(f, [0.9], [0.1], err, acc, metric=bad)
        assert ei.value.status == S.SPECA_ERR_INVALID_ARG
    assert c.launches == n
    c.close()
