"""Token-sharded verification on one device: the verification entry's tokens are split over two
caches (as two GPUs of a sequence-parallel run would hold them), each reduces its shard with
speca_verify_partial, the running values are combined the way the all-reduce would, and
speca_verify_decide takes the decision. Compared with the unsharded speca_verify_metric and with the
oracle. The shards run one after the other: nothing here waits on another kernel."""
import numpy as np
import pytest
import torch

from oracle import speca_oracle as O

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ERR_TOL = 1e-4


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


@pytest.fixture(scope="module")
def U():
    from tests import gpu_util
    return gpu_util


@pytest.mark.parametrize("metric", [0, 1, 2, 3])
@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("layout", [0, 1])    # difference tables, raw features
def test_two_token_shards_match_unsharded_and_oracle(S, U, metric, dtype, layout):
    from paper_2509_11628_b200 import dist as D
    B, tokens, dim, m = 4, 301, 1160, 2
    tdt = torch.bfloat16 if dtype == 1 else torch.float32
    gen = torch.Generator(device=DEV).manual_seed(900 + metric)
    ranges = [D.shard_tokens(tokens, 2, r) for r in range(2)]
    whole = U.Pair([(tokens, dim)], B, m, dtype, layout=layout)
    shards = [S.SpecaCache([(n, dim)], B, m, dtype, DEV, layout=layout) for _, n in ranges]
    for t in (1.0, 0.9, 0.85):
        f = torch.randn(B, tokens, dim, generator=gen, device=DEV).to(tdt)
        whole.update([f], [t] * B)
        whole.commit()
        for (t0, n), c in zip(ranges, shards):
            c.update([f[:, t0:t0 + n].contiguous()], [t] * B)
            c.commit_step()
    tt = [0.8] * B
    outs = whole.check_forecast(tt)
    noise = torch.randn(B, tokens, dim, generator=gen, device=DEV) * torch.tensor([0.0, 0.01, 0.05, 1.0], device=DEV).view(B, 1, 1)
    fresh = (outs[0].float() + noise).to(tdt)
    tau = [1e-3] * B if metric == 3 else [0.03] * B
    active = [1, 1, 0, 1]
    mask = torch.tensor(active, dtype=torch.uint8, device=DEV)
    # unsharded reference through the library and the oracle
    e_ref, a_ref, e_orc, a_orc = whole.check_verify(fresh, tt, tau, active=active, with_pred=False, metric=metric,
                                                    ulp_slack=(metric == 2))
    # shards
    total = None
    for (t0, n), c in zip(ranges, shards):
        sums = torch.full((B, 4), -5.0, dtype=torch.float64, device=DEV)
        S.speca_verify_partial(c.handle, metric, fresh[:, t0:t0 + n].contiguous(), tt, mask, None, sums)
        torch.cuda.synchronize()
        assert torch.all(sums[2] == -5.0)                      # inactive sample untouched
        total = sums if total is None else (torch.maximum(total, sums) if metric == 2 else total + sums)
    err = torch.full((B,), -7.0, dtype=torch.float32, device=DEV)
    acc = torch.full((B,), 9, dtype=torch.uint8, device=DEV)
    S.speca_verify_decide(metric, total, B, tau, 0.0, mask, err, acc)
    torch.cuda.synchronize()
    e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
    assert e_got[2] == -7.0 and a_got[2] == 9
    for b in (0, 1, 3):
        assert abs(e_got[b] - e_ref[b]) <= 1e-5 * max(1.0, e_ref[b]) + 1e-7   # same values, other summation split
        assert abs(e_got[b] - e_orc[b]) <= ERR_TOL * max(1.0, e_orc[b]) + (4e-3 if metric == 2 and dtype == 1 else 0.0)
        if abs(e_orc[b] - tau[b]) >= ERR_TOL + (4e-3 if metric == 2 and dtype == 1 else 0.0):
            assert a_got[b] == a_orc[b]
    # one shard holding everything: partial + decide is exactly speca_verify_metric
    sums = torch.zeros(B, 4, dtype=torch.float64, device=DEV)
    S.speca_verify_partial(whole.gpu.handle, metric, fresh, tt, mask, None, sums)
    S.speca_verify_decide(metric, sums, B, tau, 0.0, mask, err, acc)
    torch.cuda.synchronize()
    assert np.array_equal(err.cpu().numpy().astype(np.float64)[[0, 1, 3]], e_ref[[0, 1, 3]])
    assert np.array_equal(acc.cpu().numpy()[[0, 1, 3]], a_ref[[0, 1, 3]])
    for c in shards:
        c.close()
    whole.close()


def test_decide_argument_errors(S):
    sums = torch.zeros(2, 4, dtype=torch.float64, device=DEV)
    err = torch.zeros(2, device=DEV)
    acc = torch.zeros(2, dtype=torch.uint8, device=DEV)
    for args, status in [((7, sums, 2, [0.1, 0.1]), S.SPECA_ERR_INVALID_ARG), ((0, sums, 65, [0.1] * 65), S.SPECA_ERR_SHAPE),
                         ((0, None, 2, [0.1, 0.1]), S.SPECA_ERR_INVALID_ARG), ((0, sums, 2, [float("nan"), 0.1]), S.SPECA_ERR_INVALID_ARG)]:
        with pytest.raises(S.SpecaError) as ei:
            S.speca_verify_decide(args[0], args[1], args[2], args[3], 0.0, None, err, acc)
        assert ei.value.status == status
