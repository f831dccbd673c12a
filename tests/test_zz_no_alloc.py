"""speca_verify_pred_static: the verification entry point for callers that cannot allocate device
memory (a process whose memory pool already owns all of HBM, a plug-in that only receives input and
output tensors). Its reduction scratch is a fixed array inside the library image, shared by every
call, so the checks here are: same answer as the handle-based speca_verify on the same data and as
the CPU oracle's Eq. 4 and accept rule on the host copies of the same tensors, and still the same
answer on a second call that finds the first call's leftovers in the scratch.

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


def oracle_of_eq4(pred, fresh, tau, active, dtype):
    """Eq. 4 and the accept rule by the CPU oracle, per active sample, on the host copies of the tensors."""
    from oracle import speca_oracle as O
    from tests import gpu_util as U
    p, f = U.to_oracle(pred), U.to_oracle(fresh)
    on = [1] * pred.shape[0] if active is None else [int(x) for x in active.cpu().tolist()]
    out = []
    for b in range(pred.shape[0]):
        if not on[b]:
            out.append(None)
            continue
        e = O.rel_l2(dtype, np.ascontiguousarray(p[b]), np.ascontiguousarray(f[b]))
        out.append((e, O.accept(e, float(np.float32(tau[b])))))
    return out


def check_against_oracle(err, acc, pred, fresh, tau, active, dtype):
    e_got, a_got = err.cpu().numpy().astype(np.float64), acc.cpu().numpy()
    for b, want in enumerate(oracle_of_eq4(pred, fresh, tau, active, dtype)):
        if want is None:  # inactive: outputs untouched
            assert e_got[b] == -3.0 and a_got[b] == 7
            continue
        e, a = want
        assert abs(e_got[b] - e) <= ERR_TOL * max(1.0, e), (b, e_got[b], e)
        if abs(e - tau[b]) >= ERR_TOL:
            assert int(a_got[b]) == int(a), (b, e, tau[b])


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
        check_against_oracle(err, acc, pred, fresh, tau, active, dtype)
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


@pytest.mark.parametrize("dtype,tdt", [(1, torch.bfloat16), (0, torch.float32)])
def test_static_scratch_variant_on_awkward_shapes_against_the_oracle(S, dtype, tdt):
    """The entry point's own pieces, each against the oracle's Eq. 4: one sample whose length is not a
    multiple of the vector width (rows then need no 16-byte pitch); tensors that start 16 bytes into
    an allocation (aligned to 16 but not to 32 bytes); and a batch with more tiles than the grid has
    CTAs, twice in a row, so that every cluster walks several tiles of several samples and the second
    call meets a scratch full of the first call's partial sums."""
    esz = 2 if dtype == 1 else 4
    cases = []
    # one ragged sample
    n = 8192 * 3 + 5
    pred, fresh = make_case(1, n, tdt, 303, [0.05])
    cases.append((pred, fresh, n, 1, [0.04], None))
    # 16 bytes into the allocation
    n = 8192 * 2 + 16
    big_p, big_f = make_case(1, 2 * n + 64, tdt, 404, [0.02])
    off = 16 // esz
    pred = big_p.view(-1)[off: off + 2 * n].view(2, n)
    fresh = big_f.view(-1)[off: off + 2 * n].view(2, n)
    assert pred.data_ptr() % 32 == 16 and fresh.data_ptr() % 32 == 16
    cases.append((pred, fresh, n, 2, [0.5, 0.001], None))
    # many tiles per cluster: 8 samples x 71 tiles (one tile is 8 KB of a sample's row), about twice the resident CTAs
    n = (8192 // esz) * 70 + 40
    pred, fresh = make_case(8, n, tdt, 505, [0.0, 0.01, 0.02, 0.05, 0.1, 0.2, 0.5, 1.0])
    act = torch.tensor([1, 1, 0, 1, 1, 1, 1, 1], dtype=torch.uint8, device=DEV)
    cases.append((pred, fresh, n, 8, [0.03] * 8, act))
    cases.append((pred, fresh, n, 8, [0.3] * 8, None))
    outs = []
    for pred, fresh, n, B, tau, act in cases:      # all enqueued back to back on one stream
        err = torch.full((B,), -3.0, dtype=torch.float32, device=DEV)
        acc = torch.full((B,), 7, dtype=torch.uint8, device=DEV)
        S.speca_verify_pred_static(pred, fresh, n, B, dtype, tau, 0.0, act, err, acc, device=0)
        outs.append((err, acc))
    torch.cuda.synchronize()
    for (err, acc), (pred, fresh, n, B, tau, act) in zip(outs, cases):
        check_against_oracle(err, acc, pred.contiguous(), fresh.contiguous(), tau, act, dtype)


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
