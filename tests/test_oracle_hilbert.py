"""Pins for the oracle's Hilbert bijection (Sec. 3.1) -- CPU only."""
import os

import numpy as np
import pytest

from oracle import hilberta_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hilbert_tables.txt")


def _bitpair_d2xy(k, d):
    """Independent construction: consume d two bits at a time from the least
    significant pair, rotating/reflecting the partial coordinate (the classic
    iterative index-to-point conversion)."""
    x = y = 0
    t = d
    s = 1
    while s < (1 << k):
        rx = 1 & (t >> 1)
        ry = 1 & (t ^ rx)
        if ry == 0:
            if rx == 1:
                x = s - 1 - x
                y = s - 1 - y
            x, y = y, x
        x += s * rx
        y += s * ry
        t >>= 2
        s <<= 1
    return x, y


def _read_golden():
    tables = {}
    cur = None
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("grid"):
                cur = int(line.split()[1])
                tables[cur] = []
            else:
                tables[cur].append([int(t) for t in line.split()])
    return {n: np.array(t) for n, t in tables.items()}


@pytest.mark.parametrize("k", range(0, 9))
def test_bijection_and_neighbours(k):
    n = 1 << k
    d2t = orc.hilbert_d2t(n, n)
    assert sorted(d2t.tolist()) == list(range(n * n))
    r, c = np.divmod(d2t.astype(np.int64), n)
    step = np.abs(np.diff(r)) + np.abs(np.diff(c))
    assert np.all(step == 1)
    t2d = orc.hilbert_t2d(n, n)
    assert np.array_equal(d2t[t2d], np.arange(n * n))
    assert np.array_equal(t2d[d2t], np.arange(n * n))


@pytest.mark.parametrize("k", range(1, 9))
def test_endpoints_mirror_first_step(k):
    n = 1 << k
    d2t = orc.hilbert_d2t(n, n).astype(np.int64)
    r, c = np.divmod(d2t, n)
    assert (r[0], c[0]) == (0, 0)
    assert (r[-1], c[-1]) == (0, n - 1)
    # mirror law: the curve read backwards is its left-right reflection
    assert np.array_equal(r[::-1], r)
    assert np.array_equal(c[::-1], n - 1 - c)
    # first step goes down a row for odd order, along a column for even order
    if k % 2:
        assert (r[1], c[1]) == (1, 0)
    else:
        assert (r[1], c[1]) == (0, 1)


@pytest.mark.parametrize("k", range(1, 8))
def test_aligned_blocks_fill_aligned_squares(k):
    """Tiles of 4^j consecutive indices are 2^j x 2^j squares (Sec. 3.2:
    tiles of any size stay spatially coherent)."""
    n = 1 << k
    d2t = orc.hilbert_d2t(n, n).astype(np.int64)
    r, c = np.divmod(d2t, n)
    for j in range(1, k + 1):
        side = 1 << j
        blk = side * side
        for b in range(0, n * n, blk):
            rr, cc = r[b:b + blk], c[b:b + blk]
            assert rr.max() - rr.min() == side - 1 and cc.max() - cc.min() == side - 1
            assert rr.min() % side == 0 and cc.min() % side == 0


@pytest.mark.parametrize("k", range(1, 9))
def test_against_bitpair_construction(k):
    n = 1 << k
    d2t = orc.hilbert_d2t(n, n)
    ref = np.array([(lambda xy: xy[1] * n + xy[0])(_bitpair_d2xy(k, d)) for d in range(n * n)])
    assert np.array_equal(d2t, ref)


def test_golden_tables():
    for n, table in _read_golden().items():
        assert np.array_equal(orc.hilbert_t2d(n, n).reshape(n, n), table)


def test_worked_points_16():
    d2t = orc.hilbert_d2t(16, 16)
    got = {d: divmod(int(d2t[d]), 16) for d in (64, 128, 192, 255)}
    # quadrant entry points follow from the aligned-square property + mirror law
    assert got == {64: (8, 0), 128: (8, 8), 192: (7, 15), 255: (0, 15)}


@pytest.mark.parametrize("H,W", [(6, 6), (8, 16), (3, 5), (7, 2), (1, 9), (12, 20), (5, 5)])
def test_general_shapes_are_the_padded_curve_restricted(H, W):
    """Appendix (general shape): the curve of the enclosing power-of-two square,
    with the cells outside the H x W region dropped and the order kept."""
    n = orc.padded_side(H, W)
    assert n >= max(H, W) and n // 2 < max(H, W) and n & (n - 1) == 0
    k = n.bit_length() - 1
    pidx = orc.hilbert_cell_index(H, W)
    # independent construction of the padded index of every real cell
    where = {}
    for d in range(n * n):
        x, y = _bitpair_d2xy(k, d)
        where[(y, x)] = d
    ref = np.array([where[(r, c)] for r in range(H) for c in range(W)])
    assert np.array_equal(pidx, ref)
    d2t, t2d = orc.hilbert_d2t(H, W), orc.hilbert_t2d(H, W)
    assert sorted(d2t.tolist()) == list(range(H * W))
    assert np.array_equal(t2d[d2t], np.arange(H * W))
    # rank order = padded-curve order
    assert np.all(np.diff(pidx[d2t]) > 0)
    # the padded curve visits real cells in runs: consecutive ranks whose padded
    # indices are consecutive are grid neighbours
    r, c = np.divmod(d2t.astype(np.int64), W)
    consecutive = np.diff(pidx[d2t]) == 1
    step = np.abs(np.diff(r)) + np.abs(np.diff(c))
    assert np.all(step[consecutive] == 1)


def test_power_of_two_square_needs_no_padding():
    for n in (1, 2, 8, 32):
        assert orc.padded_side(n, n) == n
        assert np.array_equal(orc.hilbert_cell_index(n, n), orc.hilbert_t2d(n, n))
    with pytest.raises(ValueError):
        orc.padded_side(0, 4)
