"""The schedule replay used by the GPU tests, checked on made-up timelines (no GPU needed)."""
import numpy as np
import pytest

from tests.test_gpu_schedule import check_schedule


def test_the_checker_rejects_a_broken_schedule():
    """The replay itself: a timeline in which a gather overlaps the attention that still reads its slot, or ends
    after the attention that needs it, fails the corresponding rule."""
    ahead, n = 2, 8
    tr = np.zeros((n, 8))
    for i in range(n):
        t0 = 100.0 * i
        tr[i] = [t0, t0 + 60, t0 + 70, t0 + 80, t0 + 71, t0 + 71 + 100, -1, -1]
    assert check_schedule(tr, ahead, False) == 2 * n - ahead
    bad = tr.copy()
    bad[3, 4] = bad[3, 2] - 5.0                     # write-after-read broken
    with pytest.raises(AssertionError, match="released the slot"):
        check_schedule(bad, ahead, False)
    bad = tr.copy()
    bad[3, 5] = bad[5, 1] + 1.0                     # read-after-write broken
    with pytest.raises(AssertionError, match="before its gather was complete"):
        check_schedule(bad, ahead, False)
    ok = tr.copy()
    ok[:, 6] = ok[:, 1] - 20.0
    ok[:, 7] = ok[:, 1] - 5.0
    ok[:, 5] = ok[:, 4] + 60.0
    check_schedule(ok, ahead, True)
    bad = ok.copy()
    bad[4, 7] = bad[4, 1] + 3.0                     # attention before the missing pages arrived
    with pytest.raises(AssertionError, match="missing pages"):
        check_schedule(bad, ahead, True)
