"""hilberta_check_work_list: the host-side check that stands between the planner and the kernels.

The attention kernels read the query rows and key ranges of their work items without bounds checks,
so hilberta_plan_bind validates every list it builds.  Here the validator itself is tested, without a
GPU, on hand-written lists: a correct one, and one mistake at a time."""
import numpy as np
import pytest

from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200 import build

OK, BAD = hb.OK, hb.ERR_INVALID


@pytest.fixture(scope="module", autouse=True)
def _lib():
    build.build_library()


def item(q_start, q_rows, segs, block=128):
    """One record: q_start, q_rows, n_seg, seg_start[3], seg_len[3], kv_blocks."""
    st = [s for s, _ in segs] + [0] * (3 - len(segs))
    ln = [n for _, n in segs] + [0] * (3 - len(segs))
    return [q_start, q_rows, len(segs)] + st + ln + [sum(-(-n // block) for _, n in segs)]


def good_list():
    # S = 1000: 100 prefix rows that see everything; two tiles of 450 rows that see the prefix and
    # themselves, the second one through a wrapped pair of ranges
    return [item(0, 100, [(0, 1000)]),
            item(100, 256, [(0, 100), (100, 450)]), item(356, 194, [(0, 100), (100, 450)]),
            item(550, 256, [(0, 100), (700, 300), (550, 150)]), item(806, 194, [(0, 100), (700, 300), (550, 150)])]


def test_a_correct_list_passes():
    assert hb.check_work_list(good_list(), 1000, 256, 128) == OK
    # order of the items does not matter (the schedule sorts them by cost)
    assert hb.check_work_list(good_list()[::-1], 1000, 256, 128) == OK
    assert hb.check_work_list(np.zeros((0, 10), np.int32), 0, 256, 128) == OK


@pytest.mark.parametrize("what", ["rows_past_end", "gap", "overlap", "missing_tail", "too_many_rows", "zero_rows",
                                  "range_past_end", "negative_start", "empty_range", "ranges_overlap",
                                  "wrong_block_count", "no_ranges", "four_ranges"])
def test_one_mistake_at_a_time_is_caught(what):
    L = good_list()
    if what == "rows_past_end":
        L[4][1] = 195
    elif what == "gap":
        L[1][0], L[1][1] = 101, 255
    elif what == "overlap":
        L[2][0], L[2][1] = 355, 195
    elif what == "missing_tail":
        L = L[:4]
    elif what == "too_many_rows":
        L[0][1] = 100
        L = [item(0, 356, [(0, 1000)])] + L[2:]
    elif what == "zero_rows":
        L.append(item(1000, 0, [(0, 100)]))
    elif what == "range_past_end":
        L[3] = item(550, 256, [(0, 100), (700, 301), (550, 150)])
    elif what == "negative_start":
        L[1] = item(100, 256, [(-1, 100), (100, 450)])
    elif what == "empty_range":
        L[1][7] = 0          # seg_len[1] = 0 with n_seg = 2
        L[1][9] = 1
    elif what == "ranges_overlap":
        L[3] = item(550, 256, [(0, 100), (700, 300), (550, 151)])
    elif what == "wrong_block_count":
        L[0][9] += 1
    elif what == "no_ranges":
        L[0][2] = 0
    elif what == "four_ranges":
        L[0][2] = 4
    assert hb.check_work_list(L, 1000, 256, 128) == BAD


def test_argument_checks():
    assert hb.check_work_list(good_list(), 1000, 0, 128) == BAD
    assert hb.check_work_list(good_list(), 1000, 256, 0) == BAD
    assert hb.check_work_list(good_list(), 999, 256, 128) == BAD
    assert hb.check_work_list(good_list(), 1000, 128, 128) == BAD     # items of 256 rows against a 128-row kernel
