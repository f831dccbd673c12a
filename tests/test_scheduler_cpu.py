"""The forecast-then-verify control flow: scripted decisions against hand-derived traces (sequential
validation, Eq. 5-6; forced activation period), cost accounting against Eq. 8's worked number, and a
whole run on the CPU oracle with samples of different difficulty."""
import pytest

from oracle import speca_oracle as O
from paper_2509_11628_b200 import scheduler as SCH
from paper_2509_11628_b200 import workloads as W
from tests import sched_util as SU


def run_scripted(script, B=1, steps=12, period=3, warm=2, gamma=0.05):
    be = SU.ScriptedBackend(B, script)
    tr = SCH.run_sampler(be, SU.NullModel(), [1.0 - 0.05 * i for i in range(steps)], 0.1, 0.5, period, warm, gamma)
    return tr, be


def col(tr, b=0):
    return "".join(row[b] for row in tr.steps)


def test_all_accepted_runs_in_periods():
    tr, be = run_scripted({}, period=3, warm=2, steps=12)
    # two warm-up references, then 3 speculative steps, a forced full step, 3 speculative steps, ...
    assert col(tr) == "FF" + "AAAF" * 2 + "AA"
    assert tr.counts(0) == (4, 8, 0)
    assert tr.acceptance_rate() == pytest.approx(8 / 12)
    assert tr.cost(0) == pytest.approx(4 + 8 * 0.05)
    assert tr.speedup() == pytest.approx(12 / 4.4)
    assert tr.predicted_speedup() == pytest.approx(1 / (1 - 8 / 12 + 8 / 12 * 0.05))
    assert tr.speedup() == pytest.approx(tr.predicted_speedup())      # no rejection: Eq. 8 is exact


def test_first_reject_ends_the_speculative_run_and_recomputes_that_step():
    # step 3 (the second speculative step after the warm-up) fails: it is recomputed in full, the
    # table is refreshed from it, and speculation resumes from there (Eq. 5-6)
    tr, be = run_scripted({(3, 0): 0}, period=4, warm=2, steps=10)
    assert col(tr) == "FFARAAAAFA"
    f, a, r = tr.counts(0)
    assert (f, a, r) == (3, 6, 1)
    assert tr.cost(0) == pytest.approx(3 + 6 * 0.05 + 1.05)
    assert tr.speedup() < tr.predicted_speedup()                        # a rejected step costs gamma extra
    kinds = [(c[0], c[1]) for c in be.calls]
    assert ("verify", 3) in kinds and ("update", 3) in kinds           # verified, then recomputed
    assert ("update", 2) not in kinds and ("update", 4) not in kinds


def test_samples_of_a_batch_drift_apart():
    script = {(2, 1): 0, (3, 1): 0, (4, 1): 0, (6, 2): 0}
    tr, be = run_scripted(script, B=3, period=3, warm=2, steps=9)
    assert col(tr, 0) == "FFAAAFAAA"
    assert col(tr, 1) == "FFRRRAAAF"
    assert col(tr, 2) == "FFAAAFRAA"
    # the update at step 3 covers only sample 1; sample 1 is not forecast at step 3 ... it is: it was
    # re-armed by its full step at 2; check the masks the backend saw
    upd = {c[1]: c[2] for c in be.calls if c[0] == "update"}
    assert upd[3] == (0, 1, 0) and upd[5] == (1, 0, 1) and upd[6] == (0, 0, 1)
    assert tr.full_steps_histogram() == {3: 1, 4: 1, 6: 1}


def test_worked_speedup_number_from_the_appendix():
    # alpha = 0.85, gamma = 0.05 -> about 5.2x (golden file): a trace with exactly that acceptance rate
    tr = SCH.Trace(batch=1, gamma=0.05, steps=[["A"]] * 85 + [["F"]] * 15)
    assert tr.acceptance_rate() == pytest.approx(0.85)
    assert tr.predicted_speedup() == pytest.approx(O.speedup(0.85, 0.05), rel=1e-12)
    assert round(tr.predicted_speedup(), 1) == 5.2


def test_whole_run_on_the_oracle_adapts_to_sample_difficulty():
    w = W.scaled(W.dit_xl2(), max_entries=2, max_tokens=16)
    w.batch = 4
    w.sigma = [0.002, 0.002, 0.3, 0.3]                                  # two easy samples, two noisy ones
    w.times = w.times[:24]
    be = SU.OracleBackend(w)
    model = SU.GeneratorModel(w, "cpu", SU.to_oracle_array)
    tr = SCH.run_sampler(be, model, w.times, 0.3, 0.5, 4, 3, 1 / 28, total_steps=50)
    easy = [tr.counts(b) for b in (0, 1)]
    hard = [tr.counts(b) for b in (2, 3)]
    assert all(a > 10 for _, a, _ in easy)                              # easy samples mostly speculate
    assert all(r + f > 15 for f, _, r in hard)                          # noisy ones keep being recomputed
    assert tr.speedup(0) > 2.0 > tr.speedup(2)
    for i, row in enumerate(tr.steps):                                  # thresholds and decisions are consistent
        for b, kind in enumerate(row):
            if kind == SCH.ACCEPTED:
                assert tr.err[i][b] <= tr.tau[i]
            elif kind == SCH.REJECTED:
                assert not tr.err[i][b] <= tr.tau[i]
    assert tr.tau[0] == pytest.approx(0.3) and tr.tau[-1] < tr.tau[0]


class HorizonScripted(SU.ScriptedBackend):
    """A scripted backend that announces a horizon: records which future times the sampler offers it."""

    def __init__(self, batch, script, horizon):
        super().__init__(batch, script)
        self.horizon = horizon

    def forecast(self, t_target, t_later=()):
        self.calls.append(("forecast", self.step, tuple(t_target), tuple(tuple(t) for t in t_later)))

    def reference_step(self, feats, t_ref, mask, t_next=None, t_later=()):
        self.calls.append(("offer", self.step, None if t_next is None else tuple(t_next), tuple(tuple(t) for t in t_later)))
        super().reference_step(feats, t_ref, mask, t_next)


def test_a_backend_with_a_horizon_is_offered_the_times_of_the_whole_speculative_run():
    times = [1.0 - 0.05 * i for i in range(12)]
    B, period, warm = 2, 3, 2
    for horizon in (2, 3, 5):
        be = HorizonScripted(B, {(4, 1): 0}, horizon)
        tr = SCH.run_sampler(be, SU.NullModel(), times, 0.1, 0.5, period, warm, 0.05)
        plain = SU.ScriptedBackend(B, {(4, 1): 0})
        assert tr.steps == SCH.run_sampler(plain, SU.NullModel(), times, 0.1, 0.5, period, warm, 0.05).steps   # same control flow
        k = min(horizon, period)
        for c in be.calls:
            if c[0] == "offer":
                i = c[1]
                if i + 1 < warm:
                    assert c[2] is None and c[3] == ()             # the next step is a warm-up reference: nothing to forecast
                    continue
                assert c[2] == (times[i + 1],) * B if i + 1 < len(times) else c[2] is None
                want = times[i + 2:i + 1 + k]                      # never more than a run can hold, never past the end
                assert c[3] == tuple((x,) * B for x in want), (horizon, i)
            elif c[0] == "forecast":
                i = c[1]
                assert c[2] == (times[i],) * B
                assert c[3] == tuple((x,) * B for x in times[i + 1:i + horizon])
