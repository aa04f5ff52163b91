"""The knob search's guards (paper Section 5, "Self-improving autoresearch"), exercised with fake effects on the
CPU: no latency without a correctness PASS, keep / revert decided by interleaved A/B rounds (a candidate that
only met a cooler clock is reverted), nothing below the physical floor is believed, infeasible points are
skipped."""
import pytest

from paper_2606_09682_b200.autotune import Knobs, tune


class FakeGpu:
    """True latencies per knob set; `drift` multiplies the FIRST measurement of chosen candidates (a lucky clock)."""

    def __init__(self, true_us, lucky=(), wrong=(), infeasible=()):
        self.true_us, self.lucky, self.wrong, self.infeasible = true_us, set(lucky), set(wrong), set(infeasible)
        self.measured = {}
        self.released = []
        self.live = 0

    def build(self, k):
        if k in self.infeasible:
            raise RuntimeError("ring does not fit")
        self.live += 1
        return k

    def correct(self, k):
        return k not in self.wrong

    def measure(self, k, steps):
        n = self.measured.get(k, 0)
        self.measured[k] = n + 1
        us = self.true_us.get(k, 1000.0)
        return us * (0.85 if (k in self.lucky and n == 0) else 1.0)

    def release(self, k):
        self.live -= 1
        self.released.append(k)


A, B, C, D, E = Knobs(16384, 2, 2), Knobs(24576, 3, 2), Knobs(32768, 4, 6), Knobs(49152, 2, 6), Knobs(49152, 4, 2)


def _run(gpu, grid, floor=500.0):
    return tune(gpu.build, gpu.correct, gpu.measure, gpu.release, floor, grid=grid, steps=5, ab_rounds=3)


def test_a_really_faster_candidate_is_kept_and_becomes_the_incumbent():
    gpu = FakeGpu({Knobs(): 1000.0, A: 900.0, B: 950.0})
    res = _run(gpu, [A, B])
    verdicts = {t.knobs: t.verdict for t in res["trials"]}
    assert res["best"] == A and res["best_us"] == pytest.approx(900.0)
    assert verdicts[A] == "kept" and verdicts[B] == "reverted"        # B is slower than the new incumbent A
    assert gpu.live == 0                                               # every handle released


def test_a_candidate_that_only_met_a_cooler_clock_is_reverted_by_the_interleaved_rounds():
    gpu = FakeGpu({Knobs(): 1000.0, C: 1000.0}, lucky=[C])
    res = _run(gpu, [C])
    t = [t for t in res["trials"] if t.knobs == C][0]
    assert t.verdict == "reverted" and t.ab_us is not None and t.ab_us[0] == pytest.approx(t.ab_us[1])
    assert res["best"] == Knobs()


def test_no_latency_is_recorded_without_a_correctness_pass():
    gpu = FakeGpu({Knobs(): 1000.0, D: 100.0}, wrong=[D])
    res = _run(gpu, [D])
    t = [t for t in res["trials"] if t.knobs == D][0]
    assert t.verdict == "rejected: correctness" and t.latency_us is None
    assert D not in gpu.measured                                       # it was never even timed
    assert res["best"] == Knobs()


def test_a_latency_below_the_physical_floor_is_withheld():
    gpu = FakeGpu({Knobs(): 1000.0, E: 87.6})                          # "faster than the weights can be read"
    res = _run(gpu, [E], floor=695.0)
    t = [t for t in res["trials"] if t.knobs == E][0]
    assert t.verdict.startswith("rejected") and "floor" in t.verdict and t.latency_us is None
    assert res["best"] == Knobs()


def test_infeasible_points_are_skipped_and_a_broken_default_stops_the_search():
    gpu = FakeGpu({Knobs(): 1000.0, A: 900.0}, infeasible=[B])
    res = _run(gpu, [B, A])
    assert [t.verdict.split(" (")[0] for t in res["trials"]] == ["kept", "rejected: build", "kept"]
    with pytest.raises(RuntimeError):
        _run(FakeGpu({Knobs(): 1000.0}, wrong=[Knobs()]), [A])
    with pytest.raises(RuntimeError):
        _run(FakeGpu({Knobs(): 100.0}), [A], floor=500.0)
