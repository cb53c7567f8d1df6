"""Pins for the oracle's mask, layout and counts (Sec. 3.2, 3.3, App. A) -- CPU only."""
import os

import numpy as np
import pytest

from oracle import hilberta_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table1_gflops.txt")


def _naive_mask(H, W, tile, o, hs, n_text):  # H x W need not be square or a power of two
    """Second, independent enumeration: loop over all pairs and test the three
    clauses on grid coordinates, finding the Hilbert index by searching the
    curve's point list."""
    n = 1
    while n < max(H, W):
        n *= 2
    pts = orc.hilbert_points(int(np.log2(n)))
    index_of = {(y, x): d for d, (x, y) in enumerate(pts)}   # index on the padded curve
    HW = H * W
    T = (n * n) // tile
    S = n_text + HW
    r0, c0 = H // 2 - hs // 2, W // 2 - hs // 2

    def is_global(i):
        if i < n_text:
            return True
        r, c = divmod(i - n_text, W)
        return r0 <= r < r0 + hs and c0 <= c < c0 + hs

    def tile_id(i):
        r, c = divmod(i - n_text, W)
        return ((index_of[(r, c)] + o) // tile) % T

    M = np.zeros((S, S), dtype=bool)
    for i in range(S):
        for j in range(S):
            if is_global(i) or is_global(j):
                M[i, j] = True
            elif tile_id(i) == tile_id(j):
                M[i, j] = True
    return M


@pytest.mark.parametrize("H,tile,o,hs,n_text", [
    (4, 4, 0, 0, 0), (4, 4, 1, 2, 0), (4, 8, 3, 2, 3), (8, 16, 4, 2, 5),
    (8, 8, 6, 4, 0), (8, 32, 17, 0, 2), (8, 64, 9, 0, 0), (8, 16, 70, 8, 1),
])
def test_mask_bruteforce_tiny(H, tile, o, hs, n_text):
    M = orc.mask(H, H, tile, o, hs, n_text)
    assert np.array_equal(M, _naive_mask(H, H, tile, o, hs, n_text))
    assert orc.nnz(H, H, tile, o, hs, n_text) == int(M.sum())
    # row-by-row form agrees
    ig, grp = orc.token_classes(H, H, tile, o, hs, n_text)
    for i in range(M.shape[0]):
        assert np.array_equal(orc.mask_row(i, ig, grp), M[i])


@pytest.mark.parametrize("H,tile,o,hs,n_text", [(16, 64, 16, 2, 0), (16, 32, 8, 4, 7), (8, 16, 0, 0, 0)])
def test_mask_structure(H, tile, o, hs, n_text):
    M = orc.mask(H, H, tile, o, hs, n_text)
    S = M.shape[0]
    assert np.array_equal(M, M.T)
    assert M.diagonal().all()
    ig, _ = orc.token_classes(H, H, tile, o, hs, n_text)
    g = ig.astype(bool)
    assert int(g.sum()) == n_text + hs * hs
    assert M[g].all() and M[:, g].all()
    if hs == 0 and n_text == 0:
        assert np.all(M.sum(axis=1) == tile)
        classes = {tuple(np.nonzero(row)[0]) for row in M}
        assert len(classes) == (H * H) // tile


@pytest.mark.parametrize("H,W,tile,o,hs,n_text", [
    (3, 5, 16, 0, 0, 0), (3, 5, 8, 3, 2, 2), (6, 4, 16, 5, 2, 1), (7, 2, 4, 1, 0, 3), (5, 5, 64, 9, 4, 0),
    (6, 6, 8, 60, 2, 2), (1, 9, 32, 7, 0, 1),
])
def test_mask_bruteforce_general_shapes(H, W, tile, o, hs, n_text):
    """Appendix (general shape): tiles are cut on the padded curve, padding is masked."""
    M = orc.mask(H, W, tile, o, hs, n_text)
    assert np.array_equal(M, _naive_mask(H, W, tile, o, hs, n_text))
    assert np.array_equal(M, M.T) and M.diagonal().all()
    assert orc.nnz(H, W, tile, o, hs, n_text) == int(M.sum())
    # layout and key ranges expand to the same mask
    p = orc.plan_arrays(H, W, tile, o, hs, n_text)
    S, P = M.shape[0], p["prefix"]
    p2o = p["phys2orig"]
    assert sorted(p2o.tolist()) == list(range(S))
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
    assert len(p["windows"]) == orc.padded_side(H, W) ** 2 // tile


def test_offset_zero_is_block_diagonal_in_hilbert_order():
    H, tile = 8, 16
    M = orc.mask(H, H, tile, 0, 0, 0)
    d2t = orc.hilbert_d2t(H, H)
    Mh = M[np.ix_(d2t, d2t)]
    ref = np.kron(np.eye((H * H) // tile, dtype=bool), np.ones((tile, tile), dtype=bool))
    assert np.array_equal(Mh, ref)


def test_offset_periodicity():
    H, tile, hs, nt = 8, 16, 2, 3
    HW = H * H
    base = orc.mask(H, H, tile, 5, hs, nt)
    assert np.array_equal(base, orc.mask(H, H, tile, 5 + tile, hs, nt))
    assert np.array_equal(base, orc.mask(H, H, tile, 5 + HW, hs, nt))
    assert np.array_equal(base, orc.mask(H, H, tile, 5 - tile, hs, nt))
    assert not np.array_equal(base, orc.mask(H, H, tile, 6, hs, nt))


@pytest.mark.parametrize("N_side,tile,L", [(8, 4, 4), (8, 8, 4), (8, 4, 2), (16, 16, 2), (8, 16, 4)])
def test_erf_law(N_side, tile, L):
    """|ERF_i(t)| = N_T * min(T, t) for every token, full coverage after T
    layers (Sec. 3.2).  (8, 4, 4) is the worked example L = 4, N_T = 4, Delta = 1."""
    HW = N_side * N_side
    T = HW // tile
    delta = tile // L
    d2t = orc.hilbert_d2t(N_side, N_side)
    # reach[i, j] = input token j of layer 0 influences token i after t layers
    reach = np.eye(HW, dtype=np.int64)
    for t in range(1, T + 3):
        Ml = orc.mask(N_side, N_side, tile, (t - 1) * delta, 0, 0)[np.ix_(d2t, d2t)]
        reach = ((Ml.astype(np.int64) @ reach) > 0).astype(np.int64)
        assert np.all(reach.sum(axis=1) == tile * min(T, t))
    assert reach.all()


def test_erf_law_rejects_literal_window_reading():
    """Reading the window formula literally (query i attends to the UNSHIFTED
    interval tile[q_i(l)]) breaks the ERF law, so the oracle's reading -- tokens
    see each other iff their q_i(l) agree -- is the one the section fixes."""
    N, tile, L = 64, 4, 4
    T = N // tile
    reach = np.eye(N, dtype=np.int64)
    sizes = []
    for t in range(1, 6):
        o = (t - 1) * (tile // L)
        q = ((np.arange(N) + o) // tile) % T
        Ml = (q[:, None] == (np.arange(N)[None, :] // tile)).astype(np.int64)
        reach = ((Ml @ reach) > 0).astype(np.int64)
        sizes.append(int(reach.sum(axis=1).max()))
    assert sizes != [tile * min(T, t) for t in range(1, 6)]


def test_shared_runs_three_symmetric():
    for (n, hs) in [(16, 2), (64, 8), (64, 16), (128, 16), (128, 32), (256, 32)]:
        sh = orc.shared_hilbert_indices(n, n, hs)
        HW = n * n
        m = hs * hs // 4
        runs = orc.plan_arrays(n, n, HW, 0, hs, 0)["shared_runs"]
        assert runs.shape == (3, 2)
        a = int(runs[0, 0])
        assert runs.tolist() == [[a, m], [HW // 2 - m, 2 * m], [HW - a - m, m]]
        assert sh.size == hs * hs
        # the cells really are the centred square
        d2t = orc.hilbert_d2t(n, n)
        r, c = np.divmod(d2t[sh].astype(np.int64), n)
        assert r.min() == n // 2 - hs // 2 and r.max() == n // 2 + hs // 2 - 1
        assert c.min() == n // 2 - hs // 2 and c.max() == n // 2 + hs // 2 - 1


@pytest.mark.parametrize("H,tile,o,hs,n_text", [
    (8, 16, 4, 2, 5), (8, 16, 0, 2, 0), (16, 64, 16, 2, 0), (16, 64, 48, 4, 3), (8, 64, 9, 0, 0),
    (16, 16, 250, 2, 1),
])
def test_plan_arrays_against_mask(H, tile, o, hs, n_text):
    """Layout and key ranges reproduce the mask exactly when expanded."""
    p = orc.plan_arrays(H, H, tile, o, hs, n_text)
    M = orc.mask(H, H, tile, o, hs, n_text)
    S = M.shape[0]
    P = p["prefix"]
    p2o, o2p = p["phys2orig"], p["orig2phys"]
    assert sorted(p2o.tolist()) == list(range(S))
    assert np.array_equal(p2o[o2p], np.arange(S))
    assert np.array_equal(p2o[:n_text], np.arange(n_text))
    # prefix = text then shared cells; tail sorted by Hilbert index
    t2d = p["hil_t2d"]
    assert np.all(np.diff(t2d[p2o[n_text:P] - n_text]) > 0)
    assert np.all(np.diff(t2d[p2o[P:] - n_text]) > 0)
    ig, _ = orc.token_classes(H, H, tile, o, hs, n_text)
    assert ig[p2o[:P]].all() and not ig[p2o[P:]].any()
    # expand the windows into a physical-order mask
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


def test_worked_window_tables():
    p = orc.plan_arrays(16, 16, 64, 16, 2, 0)
    assert p["windows"][:, 1:].tolist() == [[240, 16, 4, 47], [51, 64, 0, 0], [115, 62, 0, 0], [177, 63, 0, 0]]
    assert p["nnz"] == 17910
    assert orc.nnz(16, 16, 64, 0, 2, 0) == 17908


def test_nnz_closed_form_full_sizes():
    for (n, tile, o, hs, nt) in [(64, 256, 128, 8, 512), (64, 1024, 512, 8, 512), (128, 1024, 512, 16, 512),
                                  (256, 2048, 1024, 32, 512)]:
        p = orc.plan_arrays(n, n, tile, o, hs, nt)
        S = nt + n * n
        P = p["prefix"]
        R = S - P
        rw = p["windows"][:, 2].astype(np.int64) + p["windows"][:, 4]
        assert rw.sum() == R
        assert p["nnz"] == P * S + R * P + int((rw * rw).sum())


def test_table1_gflops_column():
    """The paper counts, per Table 1: non-shared image queries x prefix keys, plus
    the nominal tile term HW^2/T; dense rows count S^2."""
    with open(GOLDEN) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    for label, H, W, nt, hs, tiles, printed in rows:
        H, W, nt, hs, tiles, printed = map(int, (H, W, nt, hs, tiles, printed))
        HW = H * W
        tile = HW // tiles
        if tiles == 1:
            pairs = orc.nnz(H, W, HW, 0, 0, nt)
        else:
            ig, grp = orc.token_classes(H, W, tile, 0, hs, nt)
            n_global = int(ig.sum())
            n_local = int((ig == 0).sum())
            pairs = n_local * n_global + orc.nnz(H, W, tile, 0, 0, 0)
        gflops = 4 * 3072 * pairs / 1e9
        assert abs(gflops - printed) <= 0.51, (label, gflops, printed)
    # nominal sparsity 1 - 1/T printed as 75% and 94%
    assert 1 - orc.nnz(64, 64, 1024, 0, 0, 0) / 4096 ** 2 == 0.75
    assert round(100 * (1 - orc.nnz(64, 64, 256, 0, 0, 0) / 4096 ** 2)) == 94


def test_permute_roundtrip():
    p = orc.plan_arrays(8, 8, 16, 4, 2, 5)
    x = np.arange(2 * 69 * 3).reshape(2, 69, 3)
    y = orc.permute_rows(x, p["phys2orig"])
    assert np.array_equal(y[:, 7], x[:, p["phys2orig"][7]])
    assert np.array_equal(orc.unpermute_rows(y, p["phys2orig"]), x)


# ---- Appendix A group arithmetic (equal groups over the non-shared tokens) ----

def _naive_mask_compact(H, W, groups, o, hs, n_text):
    n = 1
    while n < max(H, W):
        n *= 2
    pts = orc.hilbert_points(int(np.log2(n)))
    r0, c0 = H // 2 - hs // 2, W // 2 - hs // 2
    shared = lambda r, c: r0 <= r < r0 + hs and c0 <= c < c0 + hs
    seq = [(y, x) for (x, y) in pts if y < H and x < W and not shared(y, x)]   # non-shared cells in curve order
    R = len(seq)
    size = R // groups
    gid = {cell: ((pos + o) % R) // size for pos, cell in enumerate(seq)}
    S = n_text + H * W
    M = np.zeros((S, S), dtype=bool)
    for i in range(S):
        for j in range(S):
            gi = i < n_text or (divmod(i - n_text, W) not in gid)
            gj = j < n_text or (divmod(j - n_text, W) not in gid)
            M[i, j] = gi or gj or gid[divmod(i - n_text, W)] == gid[divmod(j - n_text, W)]
    return M


@pytest.mark.parametrize("H,W,groups,o,hs,n_text", [
    (8, 8, 4, 0, 2, 3), (8, 8, 5, 7, 2, 0), (8, 8, 12, 100, 2, 1), (4, 4, 3, 2, 2, 2), (6, 4, 4, 3, 2, 1),
    (8, 8, 4, 9, 0, 2),
])
def test_compact_tiling_bruteforce(H, W, groups, o, hs, n_text):
    M = orc.mask_compact(H, W, groups, o, hs, n_text)
    assert np.array_equal(M, _naive_mask_compact(H, W, groups, o, hs, n_text))
    assert np.array_equal(M, M.T) and M.diagonal().all()
    p = orc.plan_arrays_compact(H, W, groups, o, hs, n_text)
    assert p["nnz"] == int(M.sum())
    S, P, p2o = M.shape[0], p["prefix"], p["phys2orig"]
    Mp = np.zeros((S, S), dtype=bool)
    Mp[:P, :] = True
    Mp[:, :P] = True
    covered = np.zeros(S, dtype=int)
    for (lo, s0, n0, s1, n1) in p["windows"].tolist():
        idx = list(range(s0, s0 + n0)) + list(range(s1, s1 + n1))
        covered[idx] += 1
        Mp[np.ix_(idx, idx)] = True
    assert np.all(covered[P:] == 1)
    assert np.array_equal(Mp, M[np.ix_(p2o, p2o)])


def test_compact_equals_curve_tiling_without_shared_region():
    for (H, groups, o, nt) in [(8, 4, 5, 3), (16, 8, 40, 0)]:
        A = orc.mask(H, H, H * H // groups, o, 0, nt)
        B = orc.mask_compact(H, H, groups, o, 0, nt)
        assert np.array_equal(A, B)


def test_compact_matches_table1_group_sizes():
    """Table 1's settings: 16x16 shared at 1024^2 leaves 3840 tokens -> 960 / 240 per group."""
    p = orc.plan_arrays_compact(64, 64, 4, 0, 16, 512)
    assert p["windows"][:, 2].tolist() == [960] * 4 and p["prefix"] == 768
    p = orc.plan_arrays_compact(64, 64, 16, 60, 16, 512)
    assert (p["windows"][:, 2] + p["windows"][:, 4]).tolist() == [240] * 16
