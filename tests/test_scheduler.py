"""The batch planner for unsynchronised arrivals (host logic; paper Section IV-A admission control
re-read for one shared launch sequence).  No GPU needed."""
import pytest

from paper_2402_04466_b200.binding import Scheduler, TTError

MS = 1_000_000
PERIOD = 16_666_667


def test_idle_release_coalescing_window_and_all_present_release():
    s = Scheduler(max_streams=4, window_ns=1 * MS, deadline_ns=PERIOD)
    ids = [s.admit() for _ in range(4)]
    assert ids == [0, 1, 2, 3]
    assert s.next(0) == ([], Scheduler.NEVER)                     # nothing waiting
    assert s.arrive(3, 7, 9 * MS)
    assert s.next(9 * MS)[0] == [(3, 7, 9 * MS)]                  # idle GPU: a lone frame launches at once
    # that batch is still in flight: later frames are held so they can coalesce
    assert s.arrive(0, 7, 10 * MS)
    batch, wake = s.next(10 * MS)
    assert batch == [] and wake == 11 * MS                        # hold for the window
    assert s.arrive(2, 7, 10 * MS + 400_000)
    batch, wake = s.next(10 * MS + 500_000)
    assert batch == [] and wake == 11 * MS
    batch, wake = s.next(11 * MS)                                 # window of the oldest frame is over
    assert batch == [(0, 7, 10 * MS), (2, 7, 10 * MS + 400_000)]
    s.complete(0.2, 11 * MS + 100_000)
    # every admitted stream present: released at once even with a batch in flight
    for i in ids:
        assert s.arrive(i, 8, 27 * MS)
    batch, _ = s.next(27 * MS)
    assert [b[0] for b in batch] == ids
    assert s.stats() == {"batches": 3, "frames": 7, "dropped": 0, "deadline_misses": 0}


def test_in_flight_cap_and_overrun_drop():
    s = Scheduler(max_streams=2, window_ns=0, max_in_flight=1)
    a, b = s.admit(), s.admit()
    assert s.arrive(a, 0, 0)
    assert len(s.next(0)[0]) == 1                                 # window 0: launch immediately
    assert s.arrive(b, 0, 100)
    batch, wake = s.next(200)
    assert batch == [] and wake == Scheduler.NEVER                # one batch in flight is the cap: wait for completion
    assert s.arrive(a, 1, 300)
    assert not s.arrive(a, 2, 400)                                # stream a still has frame 1 waiting: frame 2 dropped
    s.complete(0.1, 500)
    batch, _ = s.next(500)
    assert batch == [(a, 1, 300), (b, 0, 100)]
    assert s.stats()["dropped"] == 1
    with pytest.raises(TTError):
        s.complete(0.1, 600) or s.complete(0.1, 700)              # second completion has nothing in flight


def test_deadline_aware_release_and_miss_counting():
    # predicted tick 4 ms, budget 0.5 * 10 ms = 5 ms: a lone frame may wait at most 1 ms even with a long window
    s = Scheduler(max_streams=2, window_ns=8 * MS, deadline_ns=10 * MS, budget_fraction=0.5, tick_ms_base=4.0, tick_ms_per_stream=0.0)
    x, y = s.admit(), s.admit()
    assert s.arrive(y, 0, 0)
    assert s.next(0)[0] == [(y, 0, 0)]                            # idle: launches at once and stays in flight
    assert s.arrive(x, 0, 100)
    batch, wake = s.next(100)
    assert batch == [] and wake == 100 + 1 * MS                   # busy: hold, but only until the budget allows
    batch, _ = s.next(100 + 1 * MS)
    assert batch == [(x, 0, 100)]
    s.complete(4.0, 4 * MS)
    s.complete(4.0, 11 * MS)                                      # finished after arrival + deadline: a miss
    assert s.stats()["deadline_misses"] == 1


def test_admission_by_capacity_and_by_predicted_tick_time():
    s = Scheduler(max_streams=2, window_ns=0)
    s.admit(), s.admit()
    with pytest.raises(TTError) as e:
        s.admit()
    assert e.value.status == 5                                    # no slot left
    s.release(0)
    assert s.admit() == 0
    # budget 0.5 * 16.67 ms = 8.33 ms; prior 1 ms + 2 ms per stream: 3 streams (7 ms) fit, the 4th (9 ms) is refused
    s = Scheduler(max_streams=8, window_ns=0, tick_ms_base=1.0, tick_ms_per_stream=2.0)
    for _ in range(3):
        s.admit()
    with pytest.raises(TTError) as e:
        s.admit()
    assert e.value.status == 5
    # observed tick times replace the prior: ticks of 3 streams take 1 ms, so a 4th (1 + 2 = 3 ms predicted) is admitted
    for i in range(3):
        s.arrive(i, 0, 0)
    assert len(s.next(0)[0]) == 3
    s.complete(1.0, 1 * MS)
    assert s.predict_ms(3) == pytest.approx(1.0) and s.predict_ms(4) == pytest.approx(3.0)
    assert s.admit() == 3
    # exponential average of repeated observations
    for k in range(20):
        for i in range(4):
            s.arrive(i, k + 1, (k + 1) * PERIOD)
        assert len(s.next((k + 1) * PERIOD)[0]) == 4
        s.complete(2.0, (k + 1) * PERIOD + 2 * MS)
    assert s.predict_ms(4) == pytest.approx(2.0, abs=1e-3)


def test_prediction_below_the_only_observed_batch_size_stays_positive():
    """Only ticks of 8 streams have been seen (0.4 ms); the prior's slope (0.1 ms per stream) would put a
    one-stream tick at -0.3 ms.  The prediction is floored by the 1/8 share of the observed tick, and the
    planner keeps coalescing instead of treating every frame as deadline-critical."""
    s = Scheduler(max_streams=8, window_ns=1 * MS, deadline_ns=PERIOD, tick_ms_base=0.1, tick_ms_per_stream=0.1)
    ids = [s.admit() for _ in range(8)]
    for i in ids:
        s.arrive(i, 0, 0)
    assert len(s.next(0)[0]) == 8
    s.complete(0.4, 400_000)
    assert s.predict_ms(8) == pytest.approx(0.4)
    assert s.predict_ms(1) == pytest.approx(0.05)                 # 0.4 * 1/8, not 0.4 - 0.7
    assert all(s.predict_ms(k) > 0 for k in range(1, 9))
    assert s.predict_ms(7) == pytest.approx(0.35)                 # max(0.4 - 0.1, 0.4 * 7/8)
    # a batch in flight, one frame waiting: it is held for the window, not released as "deadline near"
    for i in ids:
        s.arrive(i, 1, PERIOD)
    assert len(s.next(PERIOD)[0]) == 8
    assert s.arrive(ids[0], 2, 2 * PERIOD)
    batch, wake = s.next(2 * PERIOD)
    assert batch == [] and wake == 2 * PERIOD + 1 * MS
