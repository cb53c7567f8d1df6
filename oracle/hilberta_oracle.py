"""CPU fp64 oracle for HilbertA sparse attention.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain restatement of what the method computes, written
from the paper's definitions.  It shares no code with the CUDA library and is
never imported by it; only the tests, the smoke check and the benchmark's CPU
baseline call it.  Everything works on the ORIGINAL token order

    [ text tokens 0..n_text ) ++ [ image tokens, row-major: n_text + r*W + c ]

and in float64.

Where each piece comes from
---------------------------
* padded_side / hilbert_cell_index : general H x W grids (Appendix "Hilbert Curve
  for General Shape"): the curve of the smallest enclosing power-of-two square,
  restricted to the real cells; tiles are cut on the padded curve.
* hilbert_d2t / hilbert_t2d : the bijection pi and its inverse (Sec. 3.1, the
  graph model of the grid and "a bijection pi that visits each cell once").
  The paper names the Hilbert curve but fixes no orientation; the recursion
  below (start at row 0 / col 0, end at row 0 / col W-1) is this build's
  reading.  Parity between the eight orientations is unpinned by the paper.
* shared_cells : the fixed central region (Sec. 3.3).
* hilbert3d_point and the `frames` arguments : Sec. 5 ("Extension to Video
  Diffusion"): a 3-D Hilbert curve over (frame, row, col), tiles as contiguous
  stretches of it, the same slide, and a central shared BOX.  The paper leaves
  the curve and the box unspecified; both are this build's reading.
* group_of : tile id of a Hilbert index at a given slide (Sec. 3.2, the
  formula for q_i(l)), read as "two tokens see each other iff their q_i(l)
  agree" -- the only reading that reproduces the ERF law of the same section.
* mask : tiles + shared region + text rule (Sec. 3.2, Sec. 3.3, Appendix A:
  text tokens are treated exactly like the shared anchor region).
* attention : softmax(s * q k^T restricted to the mask) v, the quantity
  Algorithm 1's online softmax reaches up to rounding.
* attention_backward : the derivative of that quantity (the paper fine-tunes
  through its kernel, Sec. 4.1, without printing the backward pass).
* token_classes_compact / mask_compact / plan_arrays_compact : Appendix A read
  literally (Algorithm 1's S = N / G over the non-shared tokens).
* plan arrays : the memory layout of Appendix A (prefix of text + shared
  tokens, then the remaining image tokens in Hilbert order) and the contiguous
  key ranges of each slid tile ("pointer shift", modular indexing, Sec. 3.2/3.4).

Pins (tests/test_oracle_*.py): bijection, 4-neighbour steps, aligned-block
squares, mirror law, an independent bit-pair construction, hand-derived 4x4 and
8x8 tables, mask symmetry/diagonal/row counts, the ERF law, periodicity in the
offset, reduction to dense attention (checked against torch SDPA in fp64), the
block-diagonal case, brute-force masks on tiny grids, Table 1's GFLOPs column;
attention_backward: central finite differences of attention(), torch autograd in
fp64, and the identities sum_j dK_j = 0 and sum_j dV_j = sum_i dO_i.
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------
# Sec. 3.1 -- Hilbert bijection on a 2^k x 2^k grid
# --------------------------------------------------------------------------


def hilbert_points(k: int):
    """Curve of order k as a list of (x, y) = (col, row), by self-similarity.

    C_0 = [(0,0)].  With s = 2^(k-1), C_k is four copies of C_(k-1):
    transposed in the top-left quadrant, plain in the bottom-left, plain in
    the bottom-right, anti-transposed in the top-right.
    """
    pts = [(0, 0)]
    for level in range(1, k + 1):
        s = 1 << (level - 1)
        q0 = [(y, x) for (x, y) in pts]
        q1 = [(x, y + s) for (x, y) in pts]
        q2 = [(x + s, y + s) for (x, y) in pts]
        q3 = [(2 * s - 1 - y, s - 1 - x) for (x, y) in pts]
        pts = q0 + q1 + q2 + q3
    return pts


def _log2_exact(n: int) -> int:
    k = int(n).bit_length() - 1
    if n < 1 or (1 << k) != n:
        raise ValueError(f"{n} is not a power of two")
    return k


def hilbert3d_point(d: int, k: int):
    """Cell (frame, row, col) of index d on the 3-D Hilbert curve of a 2^k cube
    (Sec. 5, "Extension to Video Diffusion": a three-dimensional Hilbert curve over
    the spatio-temporal volume; the paper fixes no particular curve).

    The curve used is the one of Skilling's transpose construction ("Programming
    the Hilbert curve", 2004) with axes (frame, row, col): the 3k bits of d are
    dealt round-robin to three k-bit words (most significant bit to the frame
    word), the words are Gray-decoded, and the per-level exchanges / inversions
    are undone from the finest level up.  Starts at (0, 0, 0).
    """
    X = [0, 0, 0]
    for bit in range(3 * k):
        if (d >> (3 * k - 1 - bit)) & 1:
            X[bit % 3] |= 1 << (k - 1 - bit // 3)
    if k == 0:
        return (0, 0, 0)
    t = X[2] >> 1
    X[2] ^= X[1]
    X[1] ^= X[0]
    X[0] ^= t
    Q = 2
    while Q != (1 << k):
        Pm = Q - 1
        for i in (2, 1, 0):
            if X[i] & Q:
                X[0] ^= Pm
            else:
                t = (X[0] ^ X[i]) & Pm
                X[0] ^= t
                X[i] ^= t
        Q <<= 1
    return (X[0], X[1], X[2])


def padded_side(H: int, W: int, frames: int = 1) -> int:
    """Side n = 2^k of the smallest enclosing power-of-two square (Appendix "Hilbert
    Curve for General Shape": the curve is built on an enclosing regular grid and the
    H x W sub-region is extracted; cells outside it are padding).  For a video volume
    the frame axis is padded separately (video_orders)."""
    if H < 1 or W < 1 or frames < 1:
        raise ValueError("empty grid")
    n = 1
    while n < max(H, W):
        n *= 2
    if frames > 1:
        a, b = video_orders(H, W, frames)
        n = 1 << max(a, b)
    return n


def video_orders(H: int, W: int, frames: int):
    """(a, b): the frame axis is padded to 2^a >= frames, the two image axes to 2^b."""
    a = 1
    while (1 << a) < frames:
        a += 1
    b = 0
    while (1 << b) < max(H, W):
        b += 1
    return a, b


def padded_length(H: int, W: int, frames: int = 1) -> int:
    """Length of the padded curve: n^2 for an image; for a video volume 2^(2b + a) when the clip
    is shorter than the image is wide (a < b), else the cube (2^a)^3."""
    if frames == 1:
        n = padded_side(H, W)
        return n * n
    a, b = video_orders(H, W, frames)
    return 1 << (2 * b + a) if a < b else 1 << (3 * a)


def hilbert_cell_index(H: int, W: int, frames: int = 1) -> np.ndarray:
    """row-major cell id r*W + c -> Hilbert index of the cell on the padded n x n grid.
    int32[HW].  For a power-of-two square this is pi^-1 itself.

    With frames > 1: cell id (f*H + r)*W + c -> index on the spatio-temporal curve (Sec. 5).
    A clip is usually much shorter than a frame is wide, and one cube around everything would
    be mostly padding.  So, with the frame axis padded to 2^a and the image axes to 2^b, a < b:
    the image plane is cut into macro cells of 2^a x 2^a pixels, visited in the order of the 2-D
    curve of Sec. 3.1 (order b - a); the 2^a x 2^a x 2^a block of cells above a macro cell (all
    frames) is walked by the 3-D curve.  index = macro index * 8^a + index inside the block.
    Tiles of a multiple of 8^j positions are then unions of compact spatio-temporal blocks.
    If a >= b the whole volume sits in one cube of side 2^a walked by the 3-D curve."""
    if frames > 1:
        a, b = video_orders(H, W, frames)
        out = np.empty(frames * H * W, dtype=np.int32)
        if a >= b:
            for d in range(1 << (3 * a)):
                f, y, x = hilbert3d_point(d, a)
                if f < frames and y < H and x < W:
                    out[(f * H + y) * W + x] = d
            return out
        block = 1 << (3 * a)
        inner = [hilbert3d_point(d, a) for d in range(block)]
        for m, (mx, my) in enumerate(hilbert_points(b - a)):        # (x, y) = (col, row) of the macro cell
            for d, (f, y, x) in enumerate(inner):
                r, c = (my << a) + y, (mx << a) + x
                if f < frames and r < H and c < W:
                    out[(f * H + r) * W + c] = m * block + d
        return out
    n = padded_side(H, W)
    pts = hilbert_points(_log2_exact(n))
    out = np.empty(H * W, dtype=np.int32)
    for d, (x, y) in enumerate(pts):
        if y < H and x < W:
            out[y * W + x] = d
    return out


def hilbert_d2t(H: int, W: int, frames: int = 1) -> np.ndarray:
    """d -> row-major cell id r*W + c (pi of Sec. 3.1). int32[HW].  On a general
    shape d is the RANK of the cell among the real cells in padded-curve order."""
    return np.argsort(hilbert_cell_index(H, W, frames), kind="stable").astype(np.int32)


def hilbert_t2d(H: int, W: int, frames: int = 1) -> np.ndarray:
    """row-major cell id -> Hilbert index d (pi^-1; rank on a general shape). int32[HW]."""
    d2t = hilbert_d2t(H, W, frames)
    t2d = np.empty_like(d2t)
    t2d[d2t] = np.arange(d2t.size, dtype=np.int32)
    return t2d


# --------------------------------------------------------------------------
# Sec. 3.3 -- central shared region
# --------------------------------------------------------------------------


def shared_cells(H: int, W: int, shared_region: int, frames: int = 1, shared_frames: int = 0) -> np.ndarray:
    """Row-major ids of the centred shared_region x shared_region block.  For a video
    volume (frames > 1) the region is the centred box of shared_frames frames by
    shared_region x shared_region cells ("shared anchors ... also along the temporal
    dimension", Sec. 5)."""
    hs = int(shared_region)
    if frames > 1:
        fs = int(shared_frames)
        if hs == 0 or fs == 0:
            if hs or fs:
                raise ValueError("a shared box needs both extents")
            return np.zeros(0, dtype=np.int32)
        if hs < 0 or hs > H or hs > W or hs % 2 or fs < 0 or fs > frames or fs % 2:
            raise ValueError("shared box extents must be even and fit the volume")
        f0, r0, c0 = frames // 2 - fs // 2, H // 2 - hs // 2, W // 2 - hs // 2
        cells = [(f * H + r) * W + c for f in range(f0, f0 + fs) for r in range(r0, r0 + hs)
                 for c in range(c0, c0 + hs)]
        return np.array(cells, dtype=np.int32)
    if hs == 0:
        return np.zeros(0, dtype=np.int32)
    if hs < 0 or hs > H or hs > W or hs % 2:
        raise ValueError("shared_region must be even and fit the grid")
    r0 = H // 2 - hs // 2
    c0 = W // 2 - hs // 2
    cells = [r * W + c for r in range(r0, r0 + hs) for c in range(c0, c0 + hs)]
    return np.array(cells, dtype=np.int32)


def shared_hilbert_indices(H: int, W: int, shared_region: int, frames: int = 1, shared_frames: int = 0) -> np.ndarray:
    """Sorted (padded) Hilbert indices of the shared cells."""
    pidx = hilbert_cell_index(H, W, frames)
    return np.sort(pidx[shared_cells(H, W, shared_region, frames, shared_frames)]).astype(np.int32)


# --------------------------------------------------------------------------
# Sec. 3.2 -- tiles and the sliding schedule
# --------------------------------------------------------------------------


def group_of(d, layer_offset: int, HW: int, tile: int):
    """q_i(l) = floor((i + l*Delta) / N_T) mod T with l*Delta = layer_offset."""
    if tile < 1 or HW % tile:
        raise ValueError("tile must divide H*W")
    T = HW // tile
    d = np.asarray(d, dtype=np.int64)
    return ((d + int(layer_offset)) // tile) % T


def token_classes(H, W, tile, layer_offset, shared_region, n_text, frames=1, shared_frames=0):
    """Per original token: is_global (uint8[S]) and group (int32[S], -1 = text).

    Text tokens and shared-region tokens are global (Appendix A / Sec. 3.3);
    every image token, shared or not, has a tile id from its Hilbert index.
    On a general shape the tiles are cut on the padded curve (padding positions
    stay in the sequence and are masked out, as the appendix says), so `tile`
    must divide the padded length n*n.
    """
    HW = frames * H * W
    S = n_text + HW
    pidx = hilbert_cell_index(H, W, frames)
    is_global = np.zeros(S, dtype=np.uint8)
    is_global[:n_text] = 1
    is_global[n_text + shared_cells(H, W, shared_region, frames, shared_frames)] = 1
    group = np.full(S, -1, dtype=np.int32)
    group[n_text:] = group_of(pidx, layer_offset, padded_length(H, W, frames), tile).astype(np.int32)
    return is_global, group


def mask(H, W, tile, layer_offset, shared_region, n_text, frames=1, shared_frames=0) -> np.ndarray:
    """Boolean S x S mask over original token indices.

    M[i,j] = 1 iff i is global, or j is global, or i and j are image tokens
    of the same slid tile.
    """
    is_global, group = token_classes(H, W, tile, layer_offset, shared_region, n_text, frames, shared_frames)
    g = is_global.astype(bool)
    img = group >= 0
    same = (group[:, None] == group[None, :]) & img[:, None] & img[None, :]
    return g[:, None] | g[None, :] | same


def mask_row(i, is_global, group) -> np.ndarray:
    """Row i of the mask (bool[S]) from the per-token classes."""
    if is_global[i]:
        return np.ones(is_global.shape[0], dtype=bool)
    return is_global.astype(bool) | ((group == group[i]) & (group >= 0))


def nnz(H, W, tile, layer_offset, shared_region, n_text, frames=1, shared_frames=0) -> int:
    """Number of ones in the mask, as the sum of the row counts."""
    is_global, group = token_classes(H, W, tile, layer_offset, shared_region, n_text, frames, shared_frames)
    S = is_global.size
    n_global = int(is_global.sum())
    nonshared_img = (group >= 0) & (is_global == 0)
    T = padded_length(H, W, frames) // tile
    per_group = np.bincount(group[nonshared_img], minlength=T).astype(np.int64)
    total = n_global * S
    # a non-global row sees every global column plus the non-global members of its tile
    total += int((per_group * (n_global + per_group)).sum())
    return total


# --------------------------------------------------------------------------
# Algorithm 1's result -- masked softmax attention, fp64
# --------------------------------------------------------------------------


def attention(q, k, v, M, scale=None, return_lse=False):
    """O = softmax(scale * Q K^T + log M) V per (batch, head), in float64.

    q, k, v: [B, heads, S, D] in the original token order; M: bool [S, S].
    LSE_i = max + ln(sum exp) of the scaled, masked logits (natural log).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    B, Hh, S, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty_like(q)
    lse = np.empty((B, Hh, S), dtype=np.float64)
    for b in range(B):
        for h in range(Hh):
            logits = scale * (q[b, h] @ k[b, h].T)
            logits = np.where(M, logits, -np.inf)
            m = logits.max(axis=1, keepdims=True)
            p = np.exp(logits - m)
            l = p.sum(axis=1, keepdims=True)
            out[b, h] = (p @ v[b, h]) / l
            lse[b, h] = (m + np.log(l))[:, 0]
    return (out, lse) if return_lse else out


def attention_rows(q, k, v, is_global, group, rows, scale=None):
    """Output rows `rows` only: [B, heads, len(rows), D] fp64.

    Each row is computed from its own mask row, so this scales to the largest
    configurations when only sampled rows are wanted.
    """
    B, Hh, S, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    out = np.empty((B, Hh, len(rows), D), dtype=np.float64)
    for n, i in enumerate(rows):
        cols = np.nonzero(mask_row(int(i), is_global, group))[0]
        for b in range(B):
            for h in range(Hh):
                kk = np.asarray(k[b, h, cols], dtype=np.float64)
                vv = np.asarray(v[b, h, cols], dtype=np.float64)
                qq = np.asarray(q[b, h, int(i)], dtype=np.float64)
                logits = scale * (kk @ qq)
                p = np.exp(logits - logits.max())
                out[b, h, n] = (p @ vv) / p.sum()
    return out


def attention_backward(q, k, v, M, dout, scale=None):
    """Gradients of  L = sum(O * dout)  with  O = attention(q, k, v, M), in float64.

    The paper trains through its kernel (Sec. 4.1, LoRA fine-tuning) but prints
    no backward formulas, so this is the plain derivative of the definition
    above, written out per (batch, head) with dense S x S matrices:

        P   = softmax over the allowed keys of  scale * Q K^T
        dV  = P^T dO
        dP  = dO V^T
        dS  = P * (dP - rowsum(P * dP))          (zero where M is zero)
        dQ  = scale * dS K,      dK = scale * dS^T Q

    Returns (dq, dk, dv), each [B, heads, S, D].
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    B, Hh, S, D = q.shape
    if scale is None:
        scale = 1.0 / np.sqrt(D)
    dq, dk, dv = np.empty_like(q), np.empty_like(k), np.empty_like(v)
    for b in range(B):
        for h in range(Hh):
            logits = np.where(M, scale * (q[b, h] @ k[b, h].T), -np.inf)
            p = np.exp(logits - logits.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            dp = dout[b, h] @ v[b, h].T
            ds = p * (dp - (p * dp).sum(axis=1, keepdims=True))
            dv[b, h] = p.T @ dout[b, h]
            dq[b, h] = scale * (ds @ k[b, h])
            dk[b, h] = scale * (ds.T @ q[b, h])
    return dq, dk, dv


# --------------------------------------------------------------------------
# Appendix A layout and the per-tile key ranges (canonical plan arrays)
# --------------------------------------------------------------------------


def plan_arrays(H, W, tile, layer_offset, shared_region, n_text, frames=1, shared_frames=0) -> dict:
    """Canonical integer arrays a plan must reproduce bit for bit.

    physical order = [text | shared image tokens by ascending Hilbert index |
    non-shared image tokens by ascending Hilbert index].

    windows[w] = (lo, seg0_start, seg0_len, seg1_start, seg1_len): tile w of
    the slid partition covers (padded) Hilbert indices [lo, lo + tile) modulo
    n*n; its non-shared real members occupy one or (if it wraps) two contiguous
    physical ranges.  seg0 is the range that starts at lo.  Empty ranges are (0, 0).
    shared_runs are maximal runs of shared (padded) Hilbert indices.
    """
    HW = frames * H * W
    S = n_text + HW
    n = padded_side(H, W, frames)
    NP = padded_length(H, W, frames)
    if tile < 1 or NP % tile:
        raise ValueError("tile must divide the (padded) curve length")
    T = NP // tile
    d2t = hilbert_d2t(H, W, frames)
    t2d = hilbert_t2d(H, W, frames)
    pidx = hilbert_cell_index(H, W, frames)              # cell -> padded index
    sh_cells = shared_cells(H, W, shared_region, frames, shared_frames)
    sh = np.sort(pidx[sh_cells]).astype(np.int32)        # shared padded indices
    n_sh = sh.size
    P = n_text + n_sh
    cell_of = np.full(NP, -1, dtype=np.int64)            # padded index -> cell or -1 (padding)
    cell_of[pidx] = np.arange(HW)
    is_sh = np.zeros(NP, dtype=bool)
    is_sh[sh] = True
    real_ns = (cell_of >= 0) & ~is_sh                    # real, non-shared, by padded index

    phys2orig = np.empty(S, dtype=np.int32)
    phys2orig[:n_text] = np.arange(n_text)
    phys2orig[n_text:P] = n_text + cell_of[sh]
    phys2orig[P:] = n_text + cell_of[real_ns]
    orig2phys = np.empty(S, dtype=np.int32)
    orig2phys[phys2orig] = np.arange(S, dtype=np.int32)

    runs = []
    for d in sh.tolist():
        if runs and runs[-1][0] + runs[-1][1] == d:
            runs[-1][1] += 1
        else:
            runs.append([d, 1])
    shared_runs = np.array(runs, dtype=np.int32).reshape(-1, 2)

    # c[d] = number of real non-shared cells with padded index below d, d in [0, NP]
    c = np.concatenate([[0], np.cumsum(real_ns)]).astype(np.int64)
    o = int(layer_offset) % NP
    windows = np.zeros((T, 5), dtype=np.int32)
    for w in range(T):
        lo = (w * tile - o) % NP
        hi = lo + tile
        if hi <= NP:
            segs = [(lo, hi)]
        else:
            segs = [(lo, NP), (0, hi - NP)]
        row = [lo]
        for (a, b) in segs:
            cnt = int(c[b] - c[a])
            row += [int(P + c[a]), cnt] if cnt > 0 else [0, 0]
        row += [0, 0] * (2 - len(segs))
        windows[w] = row
    return {
        "hil_d2t": d2t,
        "hil_t2d": t2d,
        "phys2orig": phys2orig,
        "orig2phys": orig2phys,
        "shared_runs": shared_runs,
        "windows": windows,
        "nnz": nnz(H, W, tile, layer_offset, shared_region, n_text, frames, shared_frames),
        "n_shared": int(n_sh),
        "prefix": int(P),
        "padded_side": int(n),
    }


# --------------------------------------------------------------------------
# Appendix A read literally: G equal groups over the NON-SHARED tokens
# --------------------------------------------------------------------------


def token_classes_compact(H, W, groups, layer_offset, shared_region, n_text):
    """Per original token: is_global and group, for the group arithmetic of Algorithm 1.

    There the shared tokens are taken out first; the remaining R = HW - n_shared image
    tokens, in Hilbert order, form a sequence of their own that is cut into `groups`
    equal groups of R / groups tokens (S = N / G, start = group_id * S).  The slide of
    Sec. 3.2 is applied to positions in that sequence.  With no shared region this is
    the same mask as token_classes(tile = HW / groups)."""
    HW = H * W
    S = n_text + HW
    pidx = hilbert_cell_index(H, W)
    is_global = np.zeros(S, dtype=np.uint8)
    is_global[:n_text] = 1
    sh_cells = shared_cells(H, W, shared_region)
    is_global[n_text + sh_cells] = 1
    R = HW - sh_cells.size
    if groups < 1 or R % groups:
        raise ValueError("groups must divide the number of non-shared image tokens")
    size = R // groups if R else 1
    group = np.full(S, -1, dtype=np.int32)
    order = np.argsort(pidx, kind="stable")               # cells in curve order
    nonshared = [c for c in order.tolist() if not is_global[n_text + c]]
    for pos, c in enumerate(nonshared):
        group[n_text + c] = ((pos + int(layer_offset)) % R) // size
    # shared image tokens are global; give them a tile id that matches nobody else
    for c in sh_cells.tolist():
        group[n_text + c] = groups
    return is_global, group


def mask_compact(H, W, groups, layer_offset, shared_region, n_text) -> np.ndarray:
    is_global, group = token_classes_compact(H, W, groups, layer_offset, shared_region, n_text)
    g = is_global.astype(bool)
    img = (group >= 0) & ~g
    same = (group[:, None] == group[None, :]) & img[:, None] & img[None, :]
    return g[:, None] | g[None, :] | same


def plan_arrays_compact(H, W, groups, layer_offset, shared_region, n_text) -> dict:
    """Canonical arrays for the compact tiling: same physical order as plan_arrays;
    windows[w] = (lo, seg0_start, seg0_len, seg1_start, seg1_len) with lo the position in
    the non-shared sequence where group w starts."""
    base = plan_arrays(H, W, padded_side(H, W) ** 2, 0, shared_region, n_text)   # layout only
    HW = H * W
    S = n_text + HW
    P = base["prefix"]
    R = S - P
    if groups < 1 or R % groups:
        raise ValueError("groups must divide the number of non-shared image tokens")
    size = R // groups if R else 0
    o = int(layer_offset) % R if R else 0
    windows = np.zeros((groups, 5), dtype=np.int32)
    for w in range(groups):
        if size == 0:
            continue
        lo = (w * size - o) % R
        hi = lo + size
        if hi <= R:
            windows[w] = [lo, P + lo, size, 0, 0]
        else:
            windows[w] = [lo, P + lo, R - lo, P, hi - R]
    is_global, group = token_classes_compact(H, W, groups, layer_offset, shared_region, n_text)
    n_glob = int(is_global.sum())
    total = n_glob * S + groups * size * (n_glob + size)
    out = dict(base)
    out.update({"windows": windows, "nnz": int(total)})
    return out


def permute_rows(x, phys2orig):
    """dst[b, p, :] = src[b, phys2orig[p], :] (entry gather, Sec. 3.4)."""
    return np.ascontiguousarray(np.asarray(x)[:, phys2orig])


def unpermute_rows(x, phys2orig):
    """dst[b, phys2orig[p], :] = src[b, p, :] (exit gather, Sec. 3.4)."""
    x = np.asarray(x)
    out = np.empty_like(x)
    out[:, phys2orig] = x
    return out


# --------------------------------------------------------------------------
# error metrics used by the parity tests
# --------------------------------------------------------------------------


def max_abs_err(got, ref) -> float:
    return float(np.max(np.abs(np.asarray(got, dtype=np.float64) - np.asarray(ref, dtype=np.float64))))


def rel_l2_err(got, ref) -> float:
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm((got - ref).ravel()) / np.linalg.norm(ref.ravel()))
