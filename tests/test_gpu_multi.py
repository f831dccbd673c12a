"""Multi-horizon forecast (speca_forecast_multi): K speculative steps from one read of the tables.
Checked against the oracle (K plain forecasts) and, bit for bit, against K calls of speca_forecast."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
RAGGED = [(37, 129), (5, 3), (64, 384), (1, 8192 * 2 + 24), (3, 8192), (1, 1)]


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


def bits(x):
    return x.view(torch.int16 if x.dtype == torch.bfloat16 else torch.int32)


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("m", [0, 1, 2, 4])
@pytest.mark.parametrize("K", [1, 3, 8])
def test_multi_horizon_matches_oracle_and_single_forecasts(S, U, dtype, m, K):
    B = 3
    gen = torch.Generator(device=DEV).manual_seed(4000 + 10 * m + K)
    pair = U.Pair(RAGGED, B, m, dtype)
    times = [1.0, 0.93, 0.9, 0.81, 0.8]
    for step in range(m + 1):
        t = [times[step], times[step] - 0.003, times[step] + 0.001]
        pair.update(rand_feats(RAGGED, B, pair.tdt, gen), t)
        pair.commit()
        pair.sync_tables()
    t_last = pair.cpu.t_hist
    targets = [[t_last[b][0] - 0.011 * (k + 1) - 0.001 * b for b in range(B)] for k in range(K)]
    active = [1, 0, 1] if K == 3 else None
    mask = torch.tensor(active, dtype=torch.uint8, device=DEV) if active else None
    outs = [torch.full((K, B, n, d), 3.0, dtype=pair.tdt, device=DEV) for n, d in RAGGED]
    pair.gpu.forecast_multi(targets, outs, mask)
    singles = []
    for k in range(K):
        o = [torch.full((B, n, d), 3.0, dtype=pair.tdt, device=DEV) for n, d in RAGGED]
        pair.gpu.forecast(targets[k], o, mask)
        singles.append(o)
    torch.cuda.synchronize()
    three = U.to_oracle(torch.full((1,), 3.0, dtype=pair.tdt))[0]
    for e, (n, d) in enumerate(RAGGED):
        init = np.full((K, B, n * d), three, dtype=O.np_dtype(dtype))
        want = pair.cpu.forecast_multi(e, targets, active, out=init)
        got = U.to_oracle(outs[e]).reshape(K, B, -1)
        for k in range(K):
            assert torch.equal(bits(outs[e][k]), bits(singles[k][e])), "target %d of entry %d differs from speca_forecast" % (k, e)
            for b in range(B):
                if active is not None and not active[b]:
                    assert np.array_equal(got[k, b], want[k, b]), "inactive sample was written"
                    continue
                scale = U.term_scale(pair.cpu.planes[e][b], pair.forecast_weights(b, targets[k][b]))
                U.assert_close_storage(got[k, b], want[k, b], dtype, scale, "multi entry %d target %d sample %d" % (e, k, b))
    pair.close()


def test_multi_horizon_mixed_orders_and_errors(S, U):
    entries = [(16, 520), (33, 1031)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(6)
    pair = U.Pair(entries, B, m, 1)
    pair.update(rand_feats(entries, B, pair.tdt, gen), [1.0] * B)
    pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.9] * B)
    pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.8, 0.8, 0.8, 0.75], [1, 0, 0, 1])
    pair.commit()
    pair.sync_tables()            # orders are now (2, 1, 1, 2): one launch, two code paths
    K = 4
    targets = [[0.7 - 0.02 * k] * B for k in range(K)]
    outs = [torch.zeros(K, B, n, d, dtype=pair.tdt, device=DEV) for n, d in entries]
    pair.gpu.forecast_multi(targets, outs)
    torch.cuda.synchronize()
    for e, (n, d) in enumerate(entries):
        want = pair.cpu.forecast_multi(e, targets)
        got = U.to_oracle(outs[e]).reshape(K, B, -1)
        for k in range(K):
            for b in range(B):
                scale = U.term_scale(pair.cpu.planes[e][b], pair.forecast_weights(b, targets[k][b]))
                U.assert_close_storage(got[k, b], want[k, b], 1, scale, "mixed entry %d target %d sample %d" % (e, k, b))
    # only one entry requested; the other output stays untouched
    outs2 = [None, torch.full((K, B, 33, 1031), 2.0, dtype=pair.tdt, device=DEV)]
    pair.gpu.forecast_multi(targets, outs2)
    torch.cuda.synchronize()
    assert torch.equal(bits(outs2[1]), bits(outs[1]))
    launches = pair.gpu.launches
    for bad in ([], [[0.5] * B] * 9, [[float("inf")] * B]):
        with pytest.raises(S.SpecaError) as ei:
            pair.gpu.forecast_multi(bad, outs)
        assert ei.value.status == S.SPECA_ERR_INVALID_ARG
    assert pair.gpu.launches == launches
    pair.close()
