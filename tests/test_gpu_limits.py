"""The library at its stated limits: 64 samples, 512 entries, one row of almost 2^31 elements."""
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


def test_batch_of_64_samples(S, U):
    entries = [(3, 520), (9, 1031)]
    B, m = S.SPECA_MAX_BATCH, 2
    gen = torch.Generator(device=DEV).manual_seed(64)
    pair = U.Pair(entries, B, m, 1)
    for k in range(3):
        t = [1.0 - 0.1 * k - 0.001 * b for b in range(B)]            # every sample on its own clock
        pair.update([torch.randn(B, n, d, generator=gen, device=DEV).to(pair.tdt) for n, d in entries], t)
        pair.commit()
        pair.check_tables("B=64 ref %d" % k)
        pair.sync_tables()
    tt = [0.75 - 0.001 * b for b in range(B)]
    active = [(b * 7) % 3 != 0 for b in range(B)]
    pair.check_forecast(tt, active=[int(a) for a in active], sentinel=4.0)
    fresh = torch.randn(B, 9, 1031, generator=gen, device=DEV).to(pair.tdt)
    pair.check_verify(fresh, tt, [1.4] * B, active=[int(a) for a in active])
    K = 3
    outs = [torch.zeros(K, B, n, d, dtype=pair.tdt, device=DEV) for n, d in entries]
    targets = [[t - 0.01 * k for t in tt] for k in range(K)]
    pair.gpu.forecast_multi(targets, outs)
    torch.cuda.synchronize()
    for e in range(len(entries)):
        want = pair.cpu.forecast_multi(e, targets)
        got = U.to_oracle(outs[e]).reshape(K, B, -1)
        for k in range(K):
            for b in (0, 31, 32, 63):
                scale = U.term_scale(pair.cpu.planes[e][b], pair.forecast_weights(b, targets[k][b]))
                U.assert_close_storage(got[k, b], want[k, b], 1, scale, "B=64 multi %d %d %d" % (e, k, b))
    pair.close()


def test_512_entries_in_one_launch(S, U):
    rng = np.random.default_rng(512)
    entries = [(int(rng.integers(1, 9)), int(rng.integers(1, 300))) for _ in range(S.SPECA_MAX_ENTRIES)]
    B, m = 2, 1
    gen = torch.Generator(device=DEV).manual_seed(5)
    pair = U.Pair(entries, B, m, 0)
    for k in range(2):
        pair.update([torch.randn(B, n, d, generator=gen, device=DEV) for n, d in entries], [1.0 - 0.1 * k] * B)
        pair.commit()
        pair.check_tables("512 entries ref %d" % k)
        pair.sync_tables()
    pair.check_forecast([0.85] * B)
    assert pair.gpu.launches == 3            # two updates and one forecast: one launch each
    with pytest.raises(S.SpecaError) as ei:
        S.speca_cache_arena_bytes(entries + [(1, 1)], B, m, 0)
    assert ei.value.status == S.SPECA_ERR_SHAPE
    pair.close()


def test_row_of_almost_2_to_31_elements(S, U):
    """One (entry, sample) row of 2^31 - 3 elements (the limit is n < 2^31): 32-bit element and tile
    arithmetic at its edge, an odd length (scalar tail), checked on blocks at the start, around the
    middle tile boundaries and at the very end, plus the all-element plane-0 identity."""
    n = (1 << 31) - 3
    entries = [(1, n)]
    B, m = 1, 1
    with pytest.raises(S.SpecaError) as ei:
        S.speca_cache_arena_bytes([(1, 1 << 31)], B, m, 1)
    assert ei.value.status == S.SPECA_ERR_SHAPE
    cache = S.SpecaCache(entries, B, m, 1, DEV)
    blocks = [(0, 5000), ((1 << 30) - 3000, 6001), (n - 70001, 70001), (16384 * 60000 - 100, 300)]
    orc = {blk: np.zeros((m + 1, blk[1]), dtype=np.uint16) for blk in blocks}
    hist = []
    g = torch.Generator(device=DEV).manual_seed(2031)
    f = None
    for k, t in enumerate([1.0, 0.9]):
        del f
        f = torch.empty(1, 1, n, dtype=torch.bfloat16, device=DEV)
        for s in range(0, n, 1 << 28):                                # fill in pieces: bounded temporaries
            e = min(n, s + (1 << 28))
            f[0, 0, s:e] = torch.randn(e - s, generator=g, device=DEV).to(torch.bfloat16)
        cache.update([f], [t])
        cache.commit_step()
        torch.cuda.synchronize()
        assert torch.equal(cache.plane_tensor(0, 0)[0].view(torch.int16), f.view(-1).view(torch.int16))
        for blk in blocks:
            s, ln = blk
            O.update_segment(O.BF16, m, O.TAYLOR, k, hist, t, U.to_oracle(f.view(-1)[s:s + ln]), orc[blk])
            got = U.to_oracle(cache.plane_tensor(0, 0)[:, s:s + ln])
            for i in range(min(m, k) + 1):
                scale = sum(np.abs(U.as_f64(orc[blk][j])) * 10.0 ** (i - j) for j in range(i + 1))
                U.assert_close_storage(got[i], orc[blk][i], 1, scale * 0.5, "2^31 row block %r plane %d" % (blk, i))
        hist = [t] + hist
    out = torch.full((1, 1, n), 3.0, dtype=torch.bfloat16, device=DEV)
    cache.forecast([0.85], [out])
    err = torch.zeros(1, device=DEV)
    acc = torch.zeros(1, dtype=torch.uint8, device=DEV)
    cache.verify(out, [0.85], [0.0], err, acc)                        # forecast against itself: e = 0, accepted at tau = 0
    torch.cuda.synchronize()
    assert err.item() == 0.0 and acc.item() == 1
    for blk in blocks:
        s, ln = blk
        want = np.zeros(ln, dtype=np.uint16)
        O.forecast_segment(O.BF16, m, O.TAYLOR, 2, hist, 0.85, orc[blk], want)
        got = U.to_oracle(out.view(-1)[s:s + ln])
        scale = U.term_scale(orc[blk], [1.0, 0.85 - hist[0]])
        # tables were not re-synchronised here, so plane 1 may differ by an ulp: compare against the GPU's own planes too
        planes_gpu = U.to_oracle(cache.plane_tensor(0, 0)[:, s:s + ln])
        want_gpu = np.zeros(ln, dtype=np.uint16)
        O.forecast_segment(O.BF16, m, O.TAYLOR, 2, hist, 0.85, np.ascontiguousarray(planes_gpu), want_gpu)
        U.assert_close_storage(got, want_gpu, 1, scale, "2^31 row forecast block %r" % (blk,))
    assert out.view(-1)[-1].item() != 3.0 and out.view(-1)[0].item() != 3.0
    cache.close()


@pytest.mark.parametrize("path", [0, 2])
def test_health_check_after_a_step(S, path):
    """speca_cache_check waits for the stream and reports whether a staged copy of the bulk path ever gave
    up; after an ordinary step on either path it says OK, and it can be asked repeatedly."""
    entries = [(64, 1024), (33, 520)]
    B, m = 3, 2
    cache = S.SpecaCache(entries, B, m, 1, DEV, path=path)
    gen = torch.Generator(device=DEV).manual_seed(7)
    side = torch.cuda.Stream(DEV)
    with torch.cuda.stream(side):
        for k in range(3):
            cache.update([torch.randn(B, n, d, generator=gen, device=DEV).bfloat16() for n, d in entries], [1.0 - 0.1 * k] * B,
                         stream=side)
            cache.commit_step()
        outs = [torch.empty(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
        cache.forecast([0.75] * B, outs, stream=side)
    cache.check(side)
    cache.check(side)
    assert all(bool(torch.isfinite(o.float()).all()) for o in outs)   # the check has waited for the forecast
    cache.close()
