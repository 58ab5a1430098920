"""Host-side retrieval schedule (Algorithm 1's doRetrieval; Section 3.2.1 last paragraph, Appendix D)."""
import pytest

from paper_2505_20776_b200.policy import RetrievalSchedule


def run(schedule, accepted):
    out = []
    for i, a in enumerate(accepted):
        out.append(schedule.do_retrieval())
        schedule.observe(a)
    return out


@pytest.mark.parametrize("period", [1, 2, 4, 8, 128])
def test_fixed_period_updates_on_step_zero_and_every_period_after(period):
    s = RetrievalSchedule(period=period)
    got = run(s, [3] * 300)
    assert got == [i % period == 0 for i in range(300)]
    assert s.updates == sum(got) == -(-300 // period) and s.steps == 300


def test_adaptive_updates_early_when_acceptance_drops_and_restarts_the_period():
    s = RetrievalSchedule(period=8, adaptive=True, drop=0.5, min_history=2)
    #            step: 0  1  2  3  4  5  6  7  8  9 10 11 12
    accepted = [4, 4, 4, 1, 4, 4, 4, 4, 4, 4, 4, 4, 4]
    got = run(s, accepted)
    # step 0 always; the drop to 1 (< 0.5 * mean 4) is seen before step 4; the period then counts from 4
    assert [i for i, g in enumerate(got) if g] == [0, 4, 12]


def test_adaptive_needs_history_and_never_delays_the_periodic_update():
    s = RetrievalSchedule(period=4, adaptive=True, drop=0.9, min_history=3)
    got = run(s, [5, 1, 5, 5, 5, 5, 5, 5])
    assert got[:4] == [True, False, False, False]      # the early drop is ignored: not enough history yet
    assert got[4] is True
    periodic = run(RetrievalSchedule(period=4), [0] * 40)
    adaptive = run(RetrievalSchedule(period=4, adaptive=True), [0] * 40)
    assert all(a or not p for a, p in zip(adaptive, periodic))


def test_bad_parameters():
    for kw in (dict(period=0), dict(drop=0.0), dict(drop=1.5), dict(min_history=0)):
        with pytest.raises(ValueError):
            RetrievalSchedule(**kw)
    with pytest.raises(ValueError):
        RetrievalSchedule().observe(-1)
