"""Pins for the oracle's video (3-D) geometry: Sec. 5, "Extension to Video Diffusion".

The paper names a three-dimensional Hilbert curve over the spatio-temporal volume, tiles as
contiguous stretches of it, the same slide, and a central shared region that also extends
along time; it fixes neither the curve nor the box.  What is pinned here is what any such
construction must satisfy (bijection, unit steps, aligned index blocks fill aligned cubes), a
hand-derived table for the 2 x 2 x 2 cube, a brute-force mask written a second way, and the
ERF law of Sec. 3.2, which only depends on the one-dimensional tile arithmetic.
"""
import os

import numpy as np
import pytest

from oracle import hilberta_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hilbert3d_order1.txt")


@pytest.mark.parametrize("k", [1, 2, 3, 4])
def test_curve_is_a_hilbert_curve(k):
    n = 1 << k
    pts = np.array([orc.hilbert3d_point(d, k) for d in range(n ** 3)])
    assert len({tuple(p) for p in pts.tolist()}) == n ** 3                  # bijection
    assert np.all(np.abs(np.diff(pts, axis=0)).sum(axis=1) == 1)            # unit steps
    assert tuple(pts[0]) == (0, 0, 0) and tuple(pts[-1]) == (n - 1, 0, 0)   # adjacent corners
    for j in range(1, k + 1):                                               # aligned blocks are cubes
        blocks = pts.reshape(-1, 8 ** j, 3)
        lo, hi = blocks.min(axis=1), blocks.max(axis=1)
        assert np.all(hi - lo == (1 << j) - 1) and np.all(lo % (1 << j) == 0)


def test_order_one_table():
    rows = [tuple(int(x) for x in line.split()) for line in open(GOLDEN) if line[0] not in "#\n"]
    assert len(rows) == 8
    for d, f, r, c in rows:
        assert orc.hilbert3d_point(d, 1) == (f, r, c)


def _bitpair_d2xy(k, d):
    """The 2-D curve by the classic iterative index-to-point conversion (not the oracle's recursion)."""
    x = y = 0
    t, s = d, 1
    while s < (1 << k):
        rx = 1 & (t >> 1)
        ry = 1 & (t ^ rx)
        if ry == 0:
            if rx == 1:
                x, y = s - 1 - x, s - 1 - y
            x, y = y, x
        x += s * rx
        y += s * ry
        t >>= 2
        s <<= 1
    return x, y


def _naive_mask(F, H, W, tile, o, hs, fs, n_text):
    """The three clauses of the mask tested on grid coordinates, token by token; the curve index
    of a cell is looked up in tables built here: the 3-D curve inside a block of 2^a frames by
    2^a x 2^a pixels, and (for clips shorter than the image is wide) the 2-D order of the blocks."""
    a = 1
    while (1 << a) < F:
        a += 1
    b = 0
    while (1 << b) < max(H, W):
        b += 1
    if a >= b:
        NP = 1 << (3 * a)
        index_of = {orc.hilbert3d_point(d, a): d for d in range(NP)}
    else:
        NP = 1 << (2 * b + a)
        inner = {orc.hilbert3d_point(d, a): d for d in range(1 << (3 * a))}
        macro = {}
        for m in range(1 << (2 * (b - a))):
            x, y = _bitpair_d2xy(b - a, m)
            macro[(y, x)] = m
        index_of = {}
        for f in range(F):
            for r in range(H):
                for c in range(W):
                    index_of[(f, r, c)] = (macro[(r >> a, c >> a)] << (3 * a)) + inner[(f, r & ((1 << a) - 1), c & ((1 << a) - 1))]
    S = n_text + F * H * W
    f0, r0, c0 = F // 2 - fs // 2, H // 2 - hs // 2, W // 2 - hs // 2

    def describe(i):
        if i < n_text:
            return True, None
        cell = i - n_text
        f, r, c = cell // (H * W), (cell // W) % H, cell % W
        shared = hs > 0 and f0 <= f < f0 + fs and r0 <= r < r0 + hs and c0 <= c < c0 + hs
        return shared, ((index_of[(f, r, c)] + o) % NP) // tile

    info = [describe(i) for i in range(S)]
    M = np.zeros((S, S), dtype=bool)
    for i in range(S):
        for j in range(S):
            gi, ti = info[i]
            gj, tj = info[j]
            M[i, j] = gi or gj or (ti is not None and ti == tj)
    return M


@pytest.mark.parametrize("F,H,W,tile,o,hs,fs,n_text", [
    (4, 4, 4, 16, 5, 2, 2, 3),      # a cube, shared 2 x 2 x 2 box, text
    (2, 4, 4, 8, 3, 2, 2, 0),       # fewer frames than rows: padded to a 4-cube
    (3, 4, 2, 16, 0, 0, 0, 2),      # odd frame count, no shared box
])
def test_mask_bruteforce(F, H, W, tile, o, hs, fs, n_text):
    M = orc.mask(H, W, tile, o, hs, n_text, frames=F, shared_frames=fs)
    assert np.array_equal(M, _naive_mask(F, H, W, tile, o, hs, fs, n_text))
    assert np.array_equal(M, M.T) and M.diagonal().all()
    assert orc.nnz(H, W, tile, o, hs, n_text, frames=F, shared_frames=fs) == int(M.sum())


@pytest.mark.parametrize("tile,L", [(8, 4), (16, 2)])
def test_erf_law_on_a_volume(tile, L):
    """|ERF_i(t)| = N_T * min(T, t) on a 4 x 4 x 4 volume: the law of Sec. 3.2 carries over."""
    F = H = W = 4
    N = F * H * W
    T = N // tile
    d2t = orc.hilbert_d2t(H, W, F)
    reach = np.eye(N, dtype=np.int64)
    for t in range(1, T + 2):
        Ml = orc.mask(H, W, tile, (t - 1) * (tile // L), 0, 0, frames=F)[np.ix_(d2t, d2t)]
        reach = ((Ml.astype(np.int64) @ reach) > 0).astype(np.int64)
        assert np.all(reach.sum(axis=1) == tile * min(T, t))
    assert reach.all()


@pytest.mark.parametrize("F,H,W,tile,o,hs,fs,n_text", [
    (4, 4, 4, 16, 5, 2, 2, 3), (2, 4, 4, 8, 3, 2, 2, 0), (3, 4, 2, 16, 7, 0, 0, 2), (4, 8, 8, 64, 40, 4, 2, 5),
])
def test_plan_arrays_against_mask(F, H, W, tile, o, hs, fs, n_text):
    """Layout and key ranges reproduce the mask exactly when expanded."""
    p = orc.plan_arrays(H, W, tile, o, hs, n_text, frames=F, shared_frames=fs)
    M = orc.mask(H, W, tile, o, hs, n_text, frames=F, shared_frames=fs)
    S, P = M.shape[0], p["prefix"]
    p2o = p["phys2orig"]
    assert sorted(p2o.tolist()) == list(range(S))
    assert P == n_text + hs * hs * fs
    Mp = np.zeros((S, S), dtype=bool)
    Mp[:P, :] = True
    Mp[:, :P] = True
    covered = np.zeros(S, dtype=int)
    for (lo, s0, n0, s1, n1) in p["windows"].tolist():
        idx = list(range(s0, s0 + n0)) + list(range(s1, s1 + n1))
        covered[idx] += 1
        Mp[np.ix_(idx, idx)] = True
    assert np.all(covered[P:] == 1) and np.all(covered[:P] == 0)
    assert np.array_equal(Mp, M[np.ix_(p2o, p2o)])
    assert p["nnz"] == int(M.sum())


def test_single_frame_arguments_change_nothing():
    a = orc.plan_arrays(8, 8, 16, 4, 2, 5)
    b = orc.plan_arrays(8, 8, 16, 4, 2, 5, frames=1, shared_frames=0)
    for key in ("phys2orig", "windows", "hil_d2t"):
        assert np.array_equal(a[key], b[key])
