"""Out-of-bounds writes would land in guard zones: every buffer the library writes (arena, forecast
outputs, multi-horizon and summed outputs, prediction, decisions) is carved out of a larger allocation
whose borders are filled with a pattern and checked afterwards. Ragged shapes, every kernel path."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 1 << 16
PATTERN = 0xA5


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


class Guarded:
    """A tensor of `shape` in the middle of a byte buffer with GUARD bytes of pattern on both sides.
    `offset` shifts the tensor inside the buffer (to test rows that are not 32-byte aligned)."""

    def __init__(self, shape, dtype, offset=0, fill=None):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((GUARD + offset + n + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.lo, self.hi = GUARD + offset, GUARD + offset + n
        self.t = self.raw[self.lo:self.hi].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def intact(self):
        return bool((self.raw[:self.lo] == PATTERN).all()) and bool((self.raw[self.hi:] == PATTERN).all())


RAGGED = [(37, 129), (5, 3), (1, 8192 * 2 + 24), (3, 8192), (1, 1)]


@pytest.mark.parametrize("path", [1, 2, 3])
@pytest.mark.parametrize("dtype,tdt", [(0, torch.float32), (1, torch.bfloat16)])
@pytest.mark.parametrize("m", [0, 2, 4])
def test_nothing_is_written_outside_the_buffers(S, path, dtype, tdt, m):
    B = 3
    gen = torch.Generator(device=DEV).manual_seed(77)
    nbytes = S.speca_cache_arena_bytes(RAGGED, B, m, dtype, path=path)
    arena = Guarded((nbytes,), torch.uint8, offset=(256 - GUARD % 256) % 256)
    assert arena.t.data_ptr() % 256 == 0
    handle = S.speca_cache_create(RAGGED, B, m, dtype, arena.t, path=path, device=0)
    esz = 4 if dtype == 0 else 2
    for k in range(m + 1):
        feats = [torch.randn(B, n, d, generator=gen, device=DEV).to(tdt) for n, d in RAGGED]
        S.speca_cache_update(handle, feats, [1.0 - 0.1 * k] * B)
        S.speca_cache_commit_step(handle)
    for shift in (0, esz):                      # aligned rows, then rows one element off
        outs = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
        S.speca_forecast(handle, [0.45] * B, None, [o.t for o in outs])
        K = 3
        mouts = [Guarded((K, B, n, d), tdt, offset=shift) for n, d in RAGGED]
        S.speca_forecast_multi(handle, [[0.45 - 0.01 * k] * B for k in range(K)], None, [o.t for o in mouts])
        n_v, d_v = RAGGED[-1]
        pred = Guarded((B, n_v, d_v), tdt, offset=shift)
        err, acc = Guarded((B,), torch.float32), Guarded((B,), torch.uint8)
        fresh = torch.randn(B, n_v, d_v, generator=gen, device=DEV).to(tdt)
        S.speca_verify(handle, fresh, [0.45] * B, [0.1] * B, None, pred.t, err.t, acc.t)
        sums = Guarded((B, 4), torch.float64)
        S.speca_verify_partial(handle, 0, fresh, [0.45] * B, None, None, sums.t)
        total = Guarded((B, 3, 8192), tdt, offset=shift)
        S.speca_forecast_sum(handle, [3, 3], [0.45] * B, None, None, total.t)
        spec, active = Guarded((B,), torch.int32, fill=0), Guarded((B,), torch.uint8, fill=1)
        idx, n_act = Guarded((B,), torch.int32), Guarded((1,), torch.int32)
        S.speca_select_adaptive(handle, acc.t, 3, 1, spec.t, active.t, idx.t, n_act.t)
        S.speca_activate(handle, None, spec.t, active.t)
        fouts = []
        if path == 3:                           # the fused reference step exists on the default path only
            fouts = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
            ffeats = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
            for f in ffeats:
                f.t.copy_(torch.randn(f.t.shape, generator=gen, device=DEV).to(tdt))
            t_new = 0.4 - 0.05 * (1 if shift else 0)
            S.speca_cache_update_forecast(handle, [f.t for f in ffeats], [t_new] * B, [1, 0, 1], [t_new - 0.02] * B, active.t,
                                          [o.t for o in fouts], spec.t, active.t)
            fouts += ffeats
            # and with two speculative times in the same pass
            mf = [Guarded((2, B, n, d), tdt, offset=shift) for n, d in RAGGED]
            for f in ffeats:
                f.t.copy_(torch.randn(f.t.shape, generator=gen, device=DEV).to(tdt))
            S.speca_cache_update_forecast_multi(handle, [f.t for f in ffeats], [t_new - 0.03] * B, [0, 1, 1],
                                                [[t_new - 0.04] * B, [t_new - 0.05] * B], active.t, [o.t for o in mf],
                                                spec.t, active.t)
            fouts += mf
        torch.cuda.synchronize()
        for g in outs + mouts + fouts + [pred, err, acc, sums, total, spec, active, idx, n_act, arena]:
            assert g.intact(), "a guard zone was overwritten (path %d, dtype %d, order %d, shift %d)" % (path, dtype, m, shift)
        assert not bool((outs[2].t.view(torch.uint8) == PATTERN).all())       # and the outputs were written
    S.speca_cache_destroy(handle)
    assert arena.intact()


@pytest.mark.parametrize("dtype,tdt", [(0, torch.float32), (1, torch.bfloat16)])
@pytest.mark.parametrize("m", [0, 2, 4])
def test_nothing_is_written_outside_the_buffers_raw_feature_cache(S, dtype, tdt, m):
    """The same for a cache that keeps raw features: copies into the ring (past the wrap), weighted
    forecasts, verification with the continuation rule inside."""
    B = 3
    gen = torch.Generator(device=DEV).manual_seed(78)
    nbytes = S.speca_cache_arena_bytes(RAGGED, B, m, dtype, layout=S.SPECA_LAYOUT_HISTORY)
    arena = Guarded((nbytes,), torch.uint8, offset=(256 - GUARD % 256) % 256)
    handle = S.speca_cache_create(RAGGED, B, m, dtype, arena.t, device=0, layout=S.SPECA_LAYOUT_HISTORY)
    esz = 4 if dtype == 0 else 2
    for shift in (0, esz):
        for k in range(m + 3):
            feats = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
            for f in feats:
                f.t.copy_(torch.randn(f.t.shape, generator=gen, device=DEV).to(tdt))
            S.speca_cache_update(handle, [f.t for f in feats], [1.0 - 0.1 * k - shift] * B, [1, k % 2, 1])
            S.speca_cache_commit_step(handle)
        outs = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
        t = [0.1 - shift] * B
        S.speca_forecast(handle, t, None, [o.t for o in outs])
        n_v, d_v = RAGGED[-1]
        pred = Guarded((B, n_v, d_v), tdt, offset=shift)
        err, acc = Guarded((B,), torch.float32), Guarded((B,), torch.uint8)
        fresh = torch.randn(B, n_v, d_v, generator=gen, device=DEV).to(tdt)
        cur, nxt = Guarded((B,), torch.uint8, fill=1), Guarded((B,), torch.uint8)
        spec, idx, n_act = Guarded((B,), torch.int32, fill=0), Guarded((B,), torch.int32), Guarded((1,), torch.int32)
        S.speca_verify_select(handle, 0, fresh, t, [0.1] * B, cur.t, nxt.t, pred.t, err.t, acc.t, 3, 1, spec.t, idx.t, n_act.t)
        # the fused reference step: copy into the ring and two forecasts per entry in one launch
        ffeats = [Guarded((B, n, d), tdt, offset=shift) for n, d in RAGGED]
        for f in ffeats:
            f.t.copy_(torch.randn(f.t.shape, generator=gen, device=DEV).to(tdt))
        fouts = [Guarded((2, B, n, d), tdt, offset=shift) for n, d in RAGGED]
        t_new = 0.05 - shift
        S.speca_cache_update_forecast_multi(handle, [f.t for f in ffeats], [t_new] * B, [1, 1, 0],
                                            [[t_new - 0.02] * B, [t_new - 0.04] * B], None, [o.t for o in fouts], None, None)
        torch.cuda.synchronize()
        for g in outs + fouts + ffeats + [pred, err, acc, cur, nxt, spec, idx, n_act, arena]:
            assert g.intact(), "a guard zone was overwritten (dtype %d, order %d, shift %d)" % (dtype, m, shift)
        assert not bool((outs[2].t.view(torch.uint8) == PATTERN).all())
        assert not bool((fouts[1].t.view(torch.uint8) == PATTERN).all())
    S.speca_cache_destroy(handle)
    assert arena.intact()
