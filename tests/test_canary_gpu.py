"""Guard words around every output: the kernels write nothing outside the tensors they are given.

The tensor-core kernels work on 128-row tiles and drop the rows beyond a ragged item with predicated
stores; a wrong predicate would write into whatever follows the tensor.  Each output here sits in
the middle of a larger allocation that is filled with a bit pattern first; after the launch the words
before and after the tensor must still hold the pattern.  Shapes are chosen so that the last item of
every range is ragged.  Plain, fused-exit, fused-entry and strided launches, forward (with
log-sum-exp) and backward."""
import pytest
import torch

from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu

GUARD = 4096          # elements on either side (a multiple of 16 bytes for every element type)
PATTERN16 = 0x5A5A    # as int16 / bf16 bits
PATTERN32 = 0x5A5A5A5A


class Guarded:
    """A tensor of `shape` (optionally a permuted view) in the middle of a pattern-filled allocation."""

    def __init__(self, shape, dtype, permute=None):
        n = 1
        for s in shape:
            n *= s
        self.bits = torch.int16 if dtype == torch.bfloat16 else torch.int32
        self.pattern = PATTERN16 if dtype == torch.bfloat16 else PATTERN32
        self.raw = torch.full((GUARD + n + GUARD,), self.pattern, dtype=self.bits, device="cuda")
        body = self.raw[GUARD:GUARD + n].view(dtype).view(shape)
        self.t = body.permute(*permute) if permute else body
        self.n = n

    def guards_intact(self):
        return bool((self.raw[:GUARD] == self.pattern).all()) and bool((self.raw[GUARD + self.n:] == self.pattern).all())

    def body_written(self):
        """(Nearly) every word of the tensor was overwritten: unwritten words still show the pattern,
        and a computed value equals the pattern only by accident."""
        if self.n == 0:
            return True
        return float((self.raw[GUARD:GUARD + self.n] == self.pattern).float().mean()) < 1e-3


CASES = [
    # H, W, tile, offset, shared, n_text, batch, heads
    (20, 28, 64, 10, 2, 33, 1, 2),      # S = 593: ragged prefix (37 rows), ragged tiles, ragged last block
    (16, 16, 64, 16, 2, 0, 2, 1),       # 62 / 63 / 64-row tiles
    (5, 3, 16, 3, 2, 40, 1, 3),         # S = 55: everything smaller than one tile
    (32, 32, 256, 100, 4, 77, 1, 2),    # S = 1101: items of 256 rows with ragged tails
]


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("D", [128, 64])
def test_forward_outputs_stay_inside_their_tensors(case, D):
    H, W, tile, o, hs, nt, B, heads = case
    S = nt + H * W
    g = torch.Generator().manual_seed(5)
    q, k, v = (torch.randn((B, heads, S, D), generator=g).to(torch.bfloat16).cuda() for _ in range(3))
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        plan.bind_like(q)
        for mode in ("plain", "lse", "fused_exit", "fused_both"):
            out = Guarded((B, heads, S, D), torch.bfloat16)
            lse = Guarded((B, heads, S), torch.float32)
            if mode == "plain":
                plan.forward(q, k, v, out.t)
            elif mode == "lse":
                plan.forward_lse(q, k, v, out.t, lse.t)
            elif mode == "fused_exit":
                plan.forward_unpermute(q, k, v, out.t)
            else:
                plan.forward_fused(q, k, v, out.t, in_original=True, out_original=True)
            torch.cuda.synchronize()
            assert plan.status() == 0
            assert out.guards_intact(), (mode, "out")
            assert out.body_written(), (mode, "out")
            assert lse.guards_intact(), (mode, "lse")
            assert torch.isfinite(out.t.float()).all(), mode
            if mode == "lse":
                assert lse.body_written() and torch.isfinite(lse.t).all()
    finally:
        plan.destroy()


@pytest.mark.parametrize("case", CASES[:2] + CASES[3:])
def test_strided_outputs_stay_inside_their_tensors(case):
    """Heads interleaved per token ([B, S, heads, D] memory viewed as [B, heads, S, D])."""
    H, W, tile, o, hs, nt, B, heads = case
    S = nt + H * W
    g = torch.Generator().manual_seed(6)
    packs = [torch.randn((B, S, heads, 128), generator=g).to(torch.bfloat16).cuda() for _ in range(3)]
    q, k, v = (t.permute(0, 2, 1, 3) for t in packs)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        plan.bind_like(q)
        for fused in (False, True):
            out = Guarded((B, S, heads, 128), torch.bfloat16, permute=(0, 2, 1, 3))
            if fused:
                plan.forward_unpermute(q, k, v, out.t)
            else:
                plan.forward(q, k, v, out.t)
            torch.cuda.synchronize()
            assert plan.status() == 0
            assert out.guards_intact() and out.body_written(), fused
    finally:
        plan.destroy()


@pytest.mark.parametrize("case", CASES)
@pytest.mark.parametrize("dtype,D", [(torch.bfloat16, 128), (torch.bfloat16, 64), (torch.float32, 64)])
def test_backward_outputs_stay_inside_their_tensors(case, dtype, D):
    H, W, tile, o, hs, nt, B, heads = case
    S = nt + H * W
    g = torch.Generator().manual_seed(7)
    q, k, v, do = (torch.randn((B, heads, S, D), generator=g).to(dtype).cuda() for _ in range(4))
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        plan.bind_like(q)
        out = Guarded((B, heads, S, D), dtype)
        lse = Guarded((B, heads, S), torch.float32)
        plan.forward_lse(q, k, v, out.t, lse.t)
        grads = [Guarded((B, heads, S, D), dtype) for _ in range(3)]
        plan.backward(do, q, k, v, out.t, lse.t, *(gd.t for gd in grads))
        torch.cuda.synchronize()
        assert plan.status() == 0
        assert out.guards_intact() and lse.guards_intact()
        for name, gd in zip(("dq", "dk", "dv"), grads):
            assert gd.guards_intact(), name
            assert gd.body_written(), name
            assert torch.isfinite(gd.t.float()).all(), name
    finally:
        plan.destroy()
