"""hilberta_schedule_units: the host-side assignment of (work item, batch * head) units to CTAs.

What any correct schedule must satisfy, and what longest-first list scheduling guarantees."""
import numpy as np
import pytest

from paper_2509_26538_b200 import binding as hb


def _loads(units, begin, cost, two):
    loads = []
    for c in range(len(begin) - 1):
        tot = 0
        for item, a, b in units[begin[c]:begin[c + 1]]:
            tot += two[item] if b >= 0 else cost[item]
        loads.append(tot)
    return np.array(loads)


@pytest.mark.parametrize("seed", range(30))
def test_every_unit_exactly_once_and_balanced(seed):
    rng = np.random.default_rng(seed)
    n_items, bh, n_cta = int(rng.integers(1, 40)), int(rng.integers(1, 30)), int(rng.integers(1, 160))
    cost = np.sort(rng.integers(20, 3000, n_items))[::-1].astype(np.int64)
    pairable = rng.random(n_items) < 0.4
    two = np.where(pairable, cost + rng.integers(1, 60, n_items), 0).astype(np.int64)
    units, begin, largest = hb.schedule_units(cost, two, bh, n_cta)
    # every (item, index) exactly once; paired units only for items with a two-head cost, on consecutive indices
    seen = set()
    for item, a, b in units:
        assert 0 <= item < n_items and 0 <= a < bh
        assert (int(item), int(a)) not in seen
        seen.add((int(item), int(a)))
        if b >= 0:
            assert two[item] > 0 and b == a + 1 and a % 2 == 0 and b < bh
            assert (int(item), int(b)) not in seen
            seen.add((int(item), int(b)))
    assert len(seen) == n_items * bh
    for i in range(n_items):
        singles = [a for item, a, b in units if item == i and b < 0]
        if two[i] > 0:
            assert singles == ([bh - 1] if bh % 2 else [])   # only an odd index is left single
    assert begin[0] == 0 and begin[-1] == len(units) and (np.diff(begin) >= 0).all()
    loads = _loads(units, begin, cost, two)
    assert loads.max() == largest
    # list scheduling: no CTA exceeds the least loaded one by more than one unit
    used = loads[: min(n_cta, len(units))]
    biggest = max(int(cost.max()), int(two.max()))
    assert used.max() - used.min() <= biggest
    # and the classical bound: largest load <= average + largest unit
    assert largest <= loads.sum() / min(n_cta, max(len(units), 1)) + biggest


def test_flux_like_schedule_pairs_the_one_tile_items():
    """Three prefix items per head at 1024^2 (two of two tiles, one of one tile: 576 = 4.5 tiles) and 16
    window items: the one-tile item is run for pairs of heads, everything else head by head."""
    cost = np.array([36 * 20 + 40] * 2 + [36 * 19 + 20] + [7 * 20 + 40] * 16, dtype=np.int64)
    two = np.array([0, 0, 36 * 21 + 40] + [0] * 16, dtype=np.int64)
    units, begin, largest = hb.schedule_units(cost, two, 24, 148)
    paired = [(i, a, b) for i, a, b in units if b >= 0]
    assert len(paired) == 12 and all(i == 2 for i, _, _ in paired)
    assert len(units) == 18 * 24 + 12
    assert largest <= 5 * 180   # five window units, or a prefix unit and a window unit
    # without pairing the one-tile item costs 24 long single units instead of 12
    units1, _, _ = hb.schedule_units(cost, None, 24, 148)
    assert len(units1) == 19 * 24 and all(b < 0 for _, _, b in units1)


def test_argument_errors():
    L = hb.lib()
    buf = np.zeros(8, dtype=np.int32)
    c = np.ones(1, dtype=np.int64)
    assert L.hilberta_schedule_units(1, c.ctypes.data, None, 0, 4, buf.ctypes.data, buf.ctypes.data, None) == hb.ERR_INVALID
    assert L.hilberta_schedule_units(1, c.ctypes.data, None, 1, 0, buf.ctypes.data, buf.ctypes.data, None) == hb.ERR_INVALID
    assert L.hilberta_schedule_units(1, None, None, 1, 4, buf.ctypes.data, buf.ctypes.data, None) == hb.ERR_INVALID
    assert L.hilberta_schedule_units(1, c.ctypes.data, None, 1, 4, None, buf.ctypes.data, None) == hb.ERR_INVALID
