"""Per-row log-sum-exp output (the buffer a backward pass needs) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,tile,o,hs,nt,B,heads,D,dtype,tol", [
    (32, 256, 128, 4, 77, 1, 2, 128, torch.bfloat16, 2e-3),
    (16, 64, 16, 2, 0, 2, 2, 128, torch.bfloat16, 2e-3),
    (16, 64, 48, 2, 5, 1, 2, 64, torch.float32, 1e-5),
])
def test_lse_matches_oracle(H, tile, o, hs, nt, B, heads, D, dtype, tol):
    S = nt + H * H
    g = torch.Generator().manual_seed(99)
    q, k, v = (torch.randn((B, heads, S, D), generator=g).to(dtype) for _ in range(3))
    ig, grp = orc.token_classes(H, H, tile, o, hs, nt)
    ref_out, ref_lse = attn_c.attention_rows(q.float().numpy(), k.float().numpy(), v.float().numpy(), ig, grp,
                                             return_lse=True)
    plan = hb.Plan(H, H, tile, o, hs, nt)
    try:
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        qp, kp, vp = (t[:, :, p2o].contiguous().cuda() for t in (q, k, v))
        out = torch.empty_like(qp)
        out_plain = torch.empty_like(qp)
        lse = torch.full((B, heads, S), float("nan"), device="cuda", dtype=torch.float32)
        plan.bind_like(qp)
        plan.forward_lse(qp, kp, vp, out, lse)
        plan.forward(qp, kp, vp, out_plain)
        assert plan.status() == 0
        view = torch.int16 if dtype == torch.bfloat16 else torch.int32
        assert torch.equal(out.view(view), out_plain.view(view))  # the extra output changes nothing else
        got = torch.empty((B, heads, S), dtype=torch.float64)
        got[:, :, p2o] = lse.cpu().double()
    finally:
        plan.destroy()
    assert np.isfinite(got.numpy()).all()
    assert np.max(np.abs(got.numpy() - ref_lse)) <= tol
    # L.hilberta_forward_lse rejects a null lse pointer
    plan = hb.Plan(H, H, tile, o, hs, nt)
    try:
        plan.bind_like(qp)
        assert hb.lib().hilberta_forward_lse(qp.data_ptr(), kp.data_ptr(), vp.data_ptr(), out.data_ptr(), None,
                                             plan._h, None) == hb.ERR_INVALID
    finally:
        plan.destroy()
