"""speca_forecast_sum: base + sum of the forecasts of equally shaped entries, against the oracle's
unrounded double accumulation."""
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


def sum_scale(pair, ids, b, t, base_row):
    s = 0.0 if base_row is None else np.abs(U_as64(base_row))
    for e in ids:
        w = pair.forecast_weights(b, t)
        p = U_as64(pair.cpu.planes[e][b])
        s = s + sum(np.abs(p[i]) * abs(wi) for i, wi in enumerate(w))
    return s


def U_as64(a):
    from tests import gpu_util
    return gpu_util.as_f64(a)


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("basis", [0, 1, 2])
@pytest.mark.parametrize("shape", [(37, 129), (3, 8192 + 8), (1, 5)])
@pytest.mark.parametrize("m", [0, 1, 2, 4])   # orders 0 and 1 take the entries in groups of 4 and 2
def test_summed_forecast_matches_oracle(S, U, dtype, basis, shape, m):
    E, B = 7, 3
    entries = [shape] * E + [(2, 7)]                      # a differently shaped entry that is never listed
    gen = torch.Generator(device=DEV).manual_seed(300 + 10 * basis + dtype)
    pair = U.Pair(entries, B, m, dtype, basis)
    for k, t in enumerate([1.0, 0.93, 0.9, 0.84, 0.8][: m + 1]):
        pair.update(rand_feats(entries, B, pair.tdt, gen), [t, t - 0.003, t + 0.001])
        pair.commit()
        pair.sync_tables()
    t_last = [1.0, 0.93, 0.9, 0.84, 0.8][m]
    tt = [t_last - 0.04, t_last - 0.05, t_last - 0.03]
    n = shape[0] * shape[1]
    base = torch.randn(B, shape[0], shape[1], generator=gen, device=DEV).to(pair.tdt)
    for ids, use_base, active in [([0, 1, 2, 3, 4, 5, 6], True, None), ([3], False, None), ([4, 0, 4], True, [1, 0, 1]),
                                  ([6, 5, 4, 3, 2, 1], False, [0, 1, 1])]:
        out = torch.full((B, shape[0], shape[1]), 3.0, dtype=pair.tdt, device=DEV)
        mask = torch.tensor(active, dtype=torch.uint8, device=DEV) if active else None
        pair.gpu.forecast_sum(ids, tt, out, base if use_base else None, mask)
        torch.cuda.synchronize()
        init = U.to_oracle(torch.full((B, n), 3.0, dtype=pair.tdt))
        want = pair.cpu.forecast_sum(ids, tt, U.to_oracle(base).reshape(B, -1) if use_base else None, active, out=init)
        got = U.to_oracle(out).reshape(B, -1)
        for b in range(B):
            if active is not None and not active[b]:
                assert np.array_equal(got[b], want[b])
                continue
            scale = sum_scale(pair, ids, b, tt[b], U.to_oracle(base).reshape(B, -1)[b] if use_base else None)
            U.assert_close_storage(got[b], want[b], dtype, scale, "sum ids %r sample %d" % (ids, b))
    # one entry, no base: exactly speca_forecast
    single = [torch.zeros(B, n_, d_, dtype=pair.tdt, device=DEV) for n_, d_ in entries]
    pair.gpu.forecast(tt, single)
    out = torch.zeros(B, shape[0], shape[1], dtype=pair.tdt, device=DEV)
    pair.gpu.forecast_sum([2], tt, out)
    torch.cuda.synchronize()
    it = torch.int16 if dtype == 1 else torch.int32
    assert torch.equal(out.view(it), single[2].view(it))
    # in place on the residual buffer
    resid = base.clone()
    pair.gpu.forecast_sum([0, 1], tt, resid, resid)
    out2 = torch.zeros_like(base)
    pair.gpu.forecast_sum([0, 1], tt, out2, base)
    torch.cuda.synchronize()
    assert torch.equal(resid.view(it), out2.view(it))
    pair.close()


def test_summed_forecast_mixed_orders_and_errors(S, U):
    entries = [(16, 520)] * 3 + [(4, 4)]
    B, m = 4, 2
    gen = torch.Generator(device=DEV).manual_seed(8)
    pair = U.Pair(entries, B, m, 1)
    pair.update(rand_feats(entries, B, pair.tdt, gen), [1.0] * B); pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.9] * B); pair.commit()
    pair.update(rand_feats(entries, B, pair.tdt, gen), [0.8, 0.8, 0.8, 0.75], [1, 0, 0, 1]); pair.commit()
    pair.sync_tables()                                    # orders (2, 1, 1, 2)
    tt = [0.7] * B
    out = torch.zeros(B, 16, 520, dtype=pair.tdt, device=DEV)
    pair.gpu.forecast_sum([0, 1, 2], tt, out)
    torch.cuda.synchronize()
    want = pair.cpu.forecast_sum([0, 1, 2], tt)
    got = U.to_oracle(out).reshape(B, -1)
    for b in range(B):
        U.assert_close_storage(got[b], want[b], 1, sum_scale(pair, [0, 1, 2], b, tt[b], None), "mixed sample %d" % b)
    n0 = pair.gpu.launches
    for ids, status in [([0, 3], S.SPECA_ERR_SHAPE), ([], S.SPECA_ERR_INVALID_ARG), ([7], S.SPECA_ERR_INVALID_ARG)]:
        with pytest.raises(S.SpecaError) as ei:
            pair.gpu.forecast_sum(ids, tt, out)
        assert ei.value.status == status
    assert pair.gpu.launches == n0
    pair.close()
