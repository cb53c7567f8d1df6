"""hilberta_check_overlap: the exact aliasing test the attention calls run on their pointers (host only).

Checked against brute force: the byte sets of both tensors written out on small shapes."""
import itertools

import numpy as np
import pytest

from paper_2509_26538_b200 import binding as hb


def _bytes_of(base, batch, heads, S, sb, sh, ss, row):
    out = set()
    for x, y, z in itertools.product(range(batch), range(heads), range(S)):
        o = base + x * sb + y * sh + z * ss
        out.update(range(o, o + row))
    return out


@pytest.mark.parametrize("seed", range(40))
def test_against_brute_force(seed):
    rng = np.random.default_rng(seed)
    batch, heads, S = (int(rng.integers(1, 4)) for _ in range(3))
    row = int(rng.integers(1, 5)) * 2
    layout = int(rng.integers(0, 3))
    if layout == 0:      # dense [batch, heads, S, row]
        ss, sh = row, row * S
        sb = sh * heads
    elif layout == 1:    # token-major with heads interleaved: [batch, S, heads, row]
        sh, ss = row, row * heads
        sb = ss * S
    else:                # slices of a packed [batch, S, 4, heads, row] buffer
        sh, ss = row, 4 * heads * row
        sb = ss * S
    base = 1 << 20
    a = _bytes_of(base, batch, heads, S, sb, sh, ss, row)
    span = max(a) - base + 1
    for d in list(rng.integers(-span - 3, span + 4, size=60)) + [0, row, -row, heads * row, sh, ss, sb, span, -span]:
        b = _bytes_of(base + int(d), batch, heads, S, sb, sh, ss, row)
        want = bool(a & b)
        assert hb.check_overlap(base, base + int(d), batch, heads, S, sb, sh, ss, row) == want, (batch, heads, S, sb, sh, ss, row, d)


def test_packed_slices_are_accepted_and_shifted_copies_are_not():
    """q, k, v and out as the four slices of one [B, S, 4, H, D] bf16 buffer do not alias; an output placed
    one head into an input does."""
    B, S, H, D = 2, 33, 3, 128
    row = 2 * D
    sh, ss = row, 4 * H * row
    sb = ss * S
    base = 0x7f0000000000
    for i, j in itertools.combinations(range(4), 2):
        assert not hb.check_overlap(base + i * H * row, base + j * H * row, B, H, S, sb, sh, ss, row)
    assert hb.check_overlap(base, base + row, B, H, S, sb, sh, ss, row)            # one head further: head 1 of a = head 0 of b
    assert hb.check_overlap(base, base + 16, B, H, S, sb, sh, ss, row)             # inside a row
    assert hb.check_overlap(base, base, B, H, S, sb, sh, ss, row)
    # dense layout: the next tensor starts right after the first one's last byte
    sh2, ss2 = S * row, row
    sb2 = H * sh2
    assert not hb.check_overlap(base, base + B * sb2, B, H, S, sb2, sh2, ss2, row)
    assert hb.check_overlap(base, base + B * sb2 - 2, B, H, S, sb2, sh2, ss2, row)
