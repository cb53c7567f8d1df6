"""bf16 tensor-core forward and backward with head dim 64 (one 64-column slab per tile) against the
oracle, including the fused entry / exit gathers and the host-buffer entry point."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,W,tile,o,hs,nt,B,heads", [
    (16, 16, 64, 16, 2, 0, 1, 2),
    (32, 32, 128, 100, 4, 77, 2, 3),
    (24, 40, 256, 100, 4, 33, 1, 2),
    (1, 1, 1, 0, 0, 0, 1, 1),
    (64, 64, 1024, 512, 8, 512, 1, 2),
])
def test_head_dim_64_forward_and_backward(H, W, tile, o, hs, nt, B, heads):
    S = nt + H * W
    g = torch.Generator().manual_seed(640 + H)
    q, k, v = (torch.randn((B, heads, S, 64), generator=g).bfloat16() for _ in range(3))
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    ref, ref_lse = attn_c.attention_rows(q.float().numpy(), k.float().numpy(), v.float().numpy(), ig, grp,
                                         return_lse=True)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        qp, kp, vp, op, od, of = (torch.empty_like(qd) for _ in range(6))
        for src, dst in ((qd, qp), (kd, kp), (vd, vp)):
            plan.permute(src, dst)
        plan.bind_like(qp)
        lse = torch.empty((B, heads, S), device="cuda", dtype=torch.float32)
        plan.forward_lse(qp, kp, vp, op, lse)
        plan.unpermute(op, od)
        plan.forward_fused(qd, kd, vd, of, in_original=True, out_original=True)
        assert plan.status() == 0
        assert torch.equal(of.view(torch.int16), od.view(torch.int16))
        got = od.cpu().double().numpy()
        assert np.isfinite(got).all()
        assert orc.max_abs_err(got, ref) <= 1e-2 and orc.rel_l2_err(got, ref) <= 5e-3
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        got_lse = torch.empty((B, heads, S), dtype=torch.float64)
        got_lse[:, :, p2o] = lse.cpu().double()
        assert np.max(np.abs(got_lse.numpy() - ref_lse)) <= 2e-3
        # host-buffer path
        qh, kh, vh = (t.pin_memory() for t in (q, k, v))
        oh = torch.empty_like(qh).pin_memory()
        plan.bind_like(qd)
        plan.forward_host(qh, kh, vh, oh)
        assert plan.status() == 0
        assert torch.equal(oh.view(torch.int16), od.cpu().view(torch.int16))
        # backward pass on the same plan
        g2 = torch.Generator().manual_seed(641)
        do = torch.randn((B, heads, S, 64), generator=g2).bfloat16()
        ref_g = attn_c.attention_backward(q.float().numpy(), k.float().numpy(), v.float().numpy(),
                                          do.float().numpy(), ig, grp)
        dop = do[:, :, p2o].contiguous().cuda()
        plan.bind_like(qp)
        grads = [torch.full_like(qp, float("nan")) for _ in range(3)]
        plan.backward(dop, qp, kp, vp, op, lse, *grads)
        assert plan.status() == 0
        for name, t, r in zip(("dq", "dk", "dv"), grads, ref_g):
            full = torch.empty((B, heads, S, 64), dtype=torch.float64)
            full[:, :, p2o] = t.cpu().double()
            assert np.isfinite(full.numpy()).all(), name
            if np.abs(r).max() > 0:
                assert orc.rel_l2_err(full.numpy(), r) <= 5e-3, (name, orc.rel_l2_err(full.numpy(), r))
            assert orc.max_abs_err(full.numpy(), r) <= 1e-2 * max(1.0, np.abs(r).max()), name
    finally:
        plan.destroy()
