"""The host half of a forecast -- the per-sample scalars the kernels receive -- checked on the CPU
against the oracle: one-hot planes (difference tables) or one-hot features (raw-feature cache) pushed
through the oracle's forecast read off the weight of every plane, which must equal what
speca_forecast_weights computes. No GPU involved; the CUDA library is only loaded."""
import numpy as np
import pytest

from oracle import speca_oracle as O
from paper_2509_11628_b200 import binding as S


def random_history(rng, n):
    """n strictly decreasing reference times, latest first, uneven gaps."""
    t, out = 1.0, []
    for _ in range(n):
        out.append(t)
        t += float(rng.choice([0.02, 0.03, 0.05, 0.08])) * float(rng.uniform(0.7, 1.3))
    return out            # out[0] is the latest (smallest) time: time runs downwards


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON, O.ADAMS_BASHFORTH])
@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_table_layout_multipliers_give_the_oracles_plane_weights(basis, m):
    rng = np.random.default_rng(10 * m + basis)
    for n_refs in range(1, m + 4):
        hist = random_history(rng, min(n_refs, m + 1))
        for target in (hist[0] - 0.013, hist[0] - 0.07, hist[0] + 0.004):
            order, c = S.speca_forecast_weights(S.SPECA_LAYOUT_TABLES, basis, m, n_refs, hist, target)
            v = min(m, n_refs - 1)
            assert order == v
            got = [1.0]
            for i in range(v):
                got.append(got[-1] * c[i])                      # Horner: plane_0 + c_0 (plane_1 + c_1 (...))
            planes = np.eye(m + 1, dtype=np.float32)            # element i of plane i is one
            want = np.zeros(m + 1, dtype=np.float32)
            O.forecast_segment(O.F32, m, basis, n_refs, hist, target, planes, want)
            assert got == pytest.approx(want[: v + 1].tolist(), rel=2e-6, abs=1e-9)
            assert not want[v + 1:].any() and not any(c[v:])


@pytest.mark.parametrize("basis", [O.TAYLOR, O.NEWTON, O.ADAMS_BASHFORTH])
@pytest.mark.parametrize("m", [0, 1, 2, 3, 4])
def test_raw_feature_layout_weights_match_the_oracle_and_sit_in_ring_order(basis, m):
    rng = np.random.default_rng(100 + 10 * m + basis)
    for n_refs in range(1, 2 * m + 4):
        k = min(n_refs, m + 1)
        hist = random_history(rng, k)
        for target in (hist[0] - 0.013, hist[0] - 0.07, hist[0]):
            order, w = S.speca_forecast_weights(S.SPECA_LAYOUT_HISTORY, basis, m, n_refs, hist, target)
            assert order == k - 1
            unit = [np.eye(k, dtype=np.float32)[j].copy() for j in range(k)]       # feature of age j is e_j
            by_age = np.zeros(k, dtype=np.float32)
            O.forecast_history_segment(O.F32, m, basis, hist, target, unit, by_age)
            scale = float(np.abs(by_age).max())
            for j in range(k):
                phys = (n_refs - 1 - j) % (m + 1)               # where the ring keeps the feature of age j
                assert w[phys] == pytest.approx(float(by_age[j]), rel=2e-6, abs=2e-6 * scale), (n_refs, j)
            assert sum(w[:k]) == pytest.approx(1.0, abs=1e-5 * max(1.0, scale))    # constants are reproduced
            if target == hist[0]:
                latest = (n_refs - 1) % (m + 1)
                assert w[latest] == 1.0 and sum(abs(x) for x in w) == 1.0          # k = 0: the latest feature itself


def test_no_references_and_argument_errors():
    order, w = S.speca_forecast_weights(S.SPECA_LAYOUT_HISTORY, O.TAYLOR, 2, 0, [], 0.5)
    assert order == -1 and not any(w)
    for bad in (lambda: S.speca_forecast_weights(2, 0, 2, 1, [1.0], 0.5),
                lambda: S.speca_forecast_weights(0, 3, 2, 1, [1.0], 0.5),
                lambda: S.speca_forecast_weights(0, 0, 5, 1, [1.0], 0.5),
                lambda: S.speca_forecast_weights(0, 0, 2, 1, [float("nan")], 0.5),
                lambda: S.speca_forecast_weights(0, 0, 2, 1, [1.0], float("inf"))):
        with pytest.raises(S.SpecaError) as ei:
            bad()
        assert ei.value.status == S.SPECA_ERR_INVALID_ARG
