"""Host logic of the whole-tensor oracle checker used by the full-size GPU tests: every piece is visited
while the budget lasts, a cut is reported and never silent, the ragged end is always checked, and a
mismatch fails."""
import warnings

import pytest

import gpu_util as gu


def test_every_piece_is_visited_within_budget():
    chk = gu.WholeTensorChecker(budget_s=1e9, piece=10, threads=4)
    seen = []
    for call in range(3):
        chk.run(95, lambda a, b: seen.append((a, b)), remaining_calls=3 - call)
    assert sorted(set(seen)) == [(a, min(a + 10, 95)) for a in range(0, 100, 10)]
    assert len(seen) == 30 and chk.fraction == 1.0
    with warnings.catch_warnings():
        warnings.simplefilter("error")
        assert "100.0 %" in chk.report("all")


def test_a_cut_is_reported_and_keeps_the_ragged_end():
    import time
    chk = gu.WholeTensorChecker(budget_s=0.05, piece=10, threads=1)
    chk.run(100, lambda a, b: time.sleep(0.02))           # 0.2 s: the budget is gone after this call
    seen = []
    chk.run(1005, lambda a, b: seen.append((a, b)), remaining_calls=1)
    assert 0 < len(seen) < 101 and (1000, 1005) in seen
    assert chk.fraction < 1.0
    with pytest.warns(UserWarning, match="time budget"):
        chk.report("cut")


def test_a_mismatch_fails():
    chk = gu.WholeTensorChecker(budget_s=10, piece=10, threads=2)
    with pytest.raises(AssertionError, match="piece 30"):
        chk.run(100, lambda a, b: "piece %d" % a if a == 30 else None)
