"""speca_verify_pred_static: the verification entry point for callers that cannot allocate device
memory (a process whose memory pool already owns all of HBM, a plug-in that only receives input and
output tensors). Its reduction scratch is a fixed array inside the library image, shared by every
call, so the checks here are: same answer as the handle-based speca_verify on the same data, and
still the same answer on a second call that finds the first call's leftovers in the scratch.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
ERR_TOL = 1e-4  # same bound as the other verification parity tests: |e - e_ref| <= 1e-4 * max(1, e_ref)


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()  # no fallback: fail here if the CUDA library is missing
    return binding


def reference_through_a_handle(S, pred, fresh, tau, active, dtype):
    """The existing path: an order-0 cache whose only plane is `pred` (order 0 = plain reuse, so its
    forecast is `pred` itself), verified against `fresh` with speca_verify."""
    B, n = pred.shape
    cache = S.SpecaCache([(1, n)], B, 0, dtype, DEV)
    cache.update([pred], [1.0] * B)
    cache.commit_step()
    err = torch.full((B,), -3.0, dtype=torch.float32, device=DEV)
    acc = torch.full((B,), 7, dtype=torch.uint8, device=DEV)
    cache.verify(fresh, [0.9] * B, tau, err, acc, active)
    torch.cuda.synchronize()
    cache.close()
    return err.cpu().numpy().astype(np.float64), acc.cpu().numpy()


def make_case(B, n, tdt, seed, noise):
    g = torch.Generator(device=DEV).manual_seed(seed)
    fresh = torch.randn(B, n, generator=g, device=DEV).to(tdt)
    scale = torch.tensor(noise, device=DEV).view(B, 1)
    pred = (fresh.float() + scale * torch.randn(B, n, generator=g, device=DEV)).to(tdt)
    return pred.contiguous(), fresh.contiguous()


@pytest.mark.parametrize("dtype,tdt", [(1, torch.bfloat16), (0, torch.float32)])
def test_static_scratch_variant_matches_handle_variant_twice_in_a_row(S, dtype, tdt):
    # first call: several samples, rows spanning many tiles with a ragged tail, one sample inactive
    B1, n1 = 5, 3 * 8192 * 7 + 8 * 13
    noise1 = [0.0, 0.01, 0.05, 0.3, 1.0]
    tau1 = [0.04] * B1
    pred1, fresh1 = make_case(B1, n1, tdt, 101, noise1)
    active1 = torch.tensor([1, 1, 1, 0, 1], dtype=torch.uint8, device=DEV)
    # second call, straight after: other batch, other length, other data -- it meets the partial
    # sums, row descriptors and counter the first call left behind
    B2, n2 = 3, 8192 * 2 + 24
    noise2 = [0.2, 0.0, 0.02]
    tau2 = [0.1, 0.0, 0.001]
    pred2, fresh2 = make_case(B2, n2, tdt, 202, noise2)

    got = []
    for pred, fresh, tau, active, B, n in [(pred1, fresh1, tau1, active1, B1, n1), (pred2, fresh2, tau2, None, B2, n2)]:
        err = torch.full((B,), -3.0, dtype=torch.float32, device=DEV)
        acc = torch.full((B,), 7, dtype=torch.uint8, device=DEV)
        S.speca_verify_pred_static(pred, fresh, n, B, dtype, tau, 0.0, active, err, acc, device=0)
        got.append((err, acc))
    torch.cuda.synchronize()

    for (err, acc), (pred, fresh, tau, active) in zip(got, [(pred1, fresh1, tau1, active1), (pred2, fresh2, tau2, None)]):
        e_ref, a_ref = reference_through_a_handle(S, pred, fresh, tau, active, dtype)
        e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
        for b in range(len(e_ref)):
            if a_ref[b] == 7:  # inactive sample: both variants leave the outputs alone
                assert e_got[b] == -3.0 and a_got[b] == 7
                continue
            assert abs(e_got[b] - e_ref[b]) <= ERR_TOL * max(1.0, e_ref[b]), (b, e_got[b], e_ref[b])
            if abs(e_ref[b] - tau[b]) >= ERR_TOL:
                assert a_got[b] == a_ref[b], (b, e_ref[b], tau[b])
    # the cases were built to contain both outcomes
    assert got[0][1].cpu().tolist()[0] == 1 and got[0][1].cpu().tolist()[4] == 0
    assert got[1][1].cpu().tolist() == [0, 1, 0]


def test_static_scratch_variant_rejects_what_it_cannot_hold(S):
    x = torch.zeros(2, 64, dtype=torch.bfloat16, device=DEV)
    err = torch.zeros(65, dtype=torch.float32, device=DEV)
    acc = torch.zeros(65, dtype=torch.uint8, device=DEV)

    def status(fn):
        with pytest.raises(S.SpecaError) as ei:
            fn()
        return ei.value.status

    assert status(lambda: S.speca_verify_pred_static(x, x, 2, 65, 1, [0.1] * 65, 0.0, None, err, acc)) == S.SPECA_ERR_SHAPE
    assert status(lambda: S.speca_verify_pred_static(x, x, 1 << 31, 1, 1, [0.1], 0.0, None, err, acc)) == S.SPECA_ERR_SHAPE
    assert status(lambda: S.speca_verify_pred_static(x, x, 0, 1, 1, [0.1], 0.0, None, err, acc)) == S.SPECA_ERR_SHAPE
    # rows that would not start on a 16-byte boundary
    assert status(lambda: S.speca_verify_pred_static(x, x, 63, 2, 1, [0.1] * 2, 0.0, None, err, acc)) == S.SPECA_ERR_ALIGNMENT
    assert status(lambda: S.speca_verify_pred_static(x.data_ptr() + 2, x, 8, 1, 1, [0.1], 0.0, None, err, acc)) == S.SPECA_ERR_ALIGNMENT
    assert status(lambda: S.speca_verify_pred_static(None, x, 8, 1, 1, [0.1], 0.0, None, err, acc)) == S.SPECA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert err.abs().sum().item() == 0  # nothing was enqueued
