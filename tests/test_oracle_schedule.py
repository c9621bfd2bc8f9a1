"""Pins of the schedule oracle: the paper's worked example, closed-form special cases, and a
brute-force count of step kinds."""
import os

import pytest

from oracle import schedule as S

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "schedule_speedup.txt")


def test_worked_example_of_the_result_overview():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert rows
    for sparse, total, s, printed, tol in rows:
        got = S.schedule_speedup(int(sparse), int(total), float(s))
        assert abs(got - float(printed)) <= float(tol)


def test_schedule_speedup_special_cases():
    assert S.schedule_speedup(0, 1000, 2.2) == 1.0                 # no sparse step: nothing gained
    assert S.schedule_speedup(1000, 1000, 2.2) == pytest.approx(2.2)   # all sparse: the per-step figure
    assert S.schedule_speedup(500, 1000, 1.0) == 1.0               # a sparse step that is no faster
    # time view: 10 sparse steps of 1/2 unit + 30 dense steps of 1 unit = 35 units instead of 40
    assert S.schedule_speedup(10, 40, 2.0) == pytest.approx(40 / 35)
    # more sparse steps never hurt while a sparse step is faster
    v = [S.schedule_speedup(k, 100, 1.4) for k in range(101)]
    assert all(b > a for a, b in zip(v, v[1:]))


def test_step_kinds_by_counting():
    warm, sparse, total = 7, 12, 40
    kinds = [S.step_kind(i, warm, sparse, total) for i in range(total)]
    assert kinds.count(S.SPARSE) == sparse
    assert all(k == S.DENSE for k in kinds[:warm])                 # V:N:M starts after the warm-up
    assert all(k == S.SPARSE for k in kinds[warm:warm + sparse])   # sparse first ...
    assert all(k == S.DENSE for k in kinds[warm + sparse:])        # ... dense steps recover accuracy
    for bad in (-1, total):
        with pytest.raises(ValueError):
            S.step_kind(bad, warm, sparse, total)
    with pytest.raises(ValueError):
        S.step_kind(0, 30, 12, 40)                                 # phases longer than the run


def test_ffn_fraction_and_amdahl():
    # with no attention parameters the FFN is everything; with equal parameter counts it is half
    assert S.ffn_flop_fraction(64, 256, 0, 0, 16) == 1.0
    D, F, H = 128, 512, 32
    heads = 3 * F // (2 * H)                     # 2 D heads H == 3 D F
    assert S.ffn_flop_fraction(D, F, heads // 2, heads - heads // 2, H) == pytest.approx(0.5)
    # Section 3.1: "up to 80 %" of the FLOPs for large models -- a 405B-class shape with grouped
    # queries (D 16384, F 53248, 128 query and 8 key/value heads of 128) gives 0.82
    f = S.ffn_flop_fraction(16384, 53248, 128, 8, 128)
    assert 0.78 < f < 0.83
    assert S.end_to_end_speedup(0.0, 7.0) == 1.0
    assert S.end_to_end_speedup(1.0, 7.0) == pytest.approx(7.0)
    assert S.end_to_end_speedup(0.5, 2.0) == pytest.approx(1 / 0.75)
    assert S.end_to_end_speedup(0.8, 1e12) == pytest.approx(5.0)   # the unaccelerated share bounds it
