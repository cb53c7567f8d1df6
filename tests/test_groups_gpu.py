"""The Appendix-A tiling (equal groups over the non-shared tokens): plan bit-exact and
forward in tolerance, including the settings of the paper's Table 1."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200.inputs import WORKLOADS, make_qkv, sample_rows

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,W,groups,o,hs,nt", [
    (8, 8, 4, 0, 2, 3), (8, 8, 12, 100, 2, 1), (6, 4, 4, 3, 2, 1), (64, 64, 4, 0, 16, 512),
    (64, 64, 16, 60, 16, 512), (128, 128, 16, 240, 32, 512), (16, 16, 252, 5, 2, 0), (8, 8, 1, 9, 0, 2),
])
def test_plan_groups_bit_exact(H, W, groups, o, hs, nt):
    ref = orc.plan_arrays_compact(H, W, groups, o, hs, nt)
    plan = hb.Plan(H, W, 0, o, hs, nt, groups=groups)
    try:
        assert np.array_equal(plan.export(hb.EXPORT_PHYS2ORIG), ref["phys2orig"])
        assert np.array_equal(plan.export(hb.EXPORT_ORIG2PHYS), ref["orig2phys"])
        assert np.array_equal(plan.export(hb.EXPORT_WINDOWS), ref["windows"])
        assert int(plan.export(hb.EXPORT_NNZ)[0]) == ref["nnz"]
    finally:
        plan.destroy()


def test_plan_groups_errors():
    import ctypes
    h = ctypes.c_void_p()
    L = hb.lib()
    assert L.hilberta_plan_groups(8, 8, 7, 0, 2, 0, ctypes.byref(h)) == hb.ERR_INVALID   # 60 % 7 != 0
    assert L.hilberta_plan_groups(8, 8, 0, 0, 2, 0, ctypes.byref(h)) == hb.ERR_INVALID
    assert L.hilberta_plan_groups(2, 2, 1, 0, 2, 0, ctypes.byref(h)) == hb.ERR_INVALID   # no non-shared token left


@pytest.mark.parametrize("dtype,D,tol", [(torch.bfloat16, 128, (1e-2, 5e-3)), (torch.float32, 64, (1e-5, 1e-5))])
def test_forward_groups_small(dtype, D, tol):
    H, W, groups, o, hs, nt = 16, 16, 4, 21, 2, 9
    S = nt + H * W
    g = torch.Generator().manual_seed(606)
    q, k, v = (torch.randn((1, 2, S, D), generator=g).to(dtype) for _ in range(3))
    ig, grp = orc.token_classes_compact(H, W, groups, o, hs, nt)
    ref = attn_c.attention_rows(q.float().numpy(), k.float().numpy(), v.float().numpy(), ig, grp)
    plan = hb.Plan(H, W, 0, o, hs, nt, groups=groups)
    try:
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        qp, kp, vp, od = (torch.empty_like(qd) for _ in range(4))
        plan.permute(qd, qp)
        plan.permute(kd, kp)
        plan.permute(vd, vp)
        plan.bind_like(qp)
        plan.forward_unpermute(qp, kp, vp, od)
        assert plan.status() == 0
        got = od.cpu().double().numpy()
    finally:
        plan.destroy()
    assert orc.max_abs_err(got, ref) <= tol[0] and orc.rel_l2_err(got, ref) <= tol[1]


def test_forward_table1_setting_sampled_rows():
    """Table 1's 16-tile setting at 1024^2: 16x16 shared region, groups of 240 tokens, all 24 heads."""
    wl = WORKLOADS["flux1024"]
    groups, o, hs = 16, 60, 16
    q, k, v = make_qkv(wl)
    plan = hb.Plan(wl.H, wl.W, 0, o, hs, wl.n_text, groups=groups)
    try:
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        qp, kp, vp, od = (torch.empty_like(qd) for _ in range(4))
        plan.permute(qd, qp)
        plan.permute(kd, kp)
        plan.permute(vd, vp)
        plan.bind_like(qp)
        plan.forward_unpermute(qp, kp, vp, od)
        assert plan.status() == 0
        got = od.cpu()
    finally:
        plan.destroy()
    rows = sample_rows(wl, 96)
    ig, grp = orc.token_classes_compact(wl.H, wl.W, groups, o, hs, wl.n_text)
    ref = attn_c.attention_rows(q.float().numpy(), k.float().numpy(), v.float().numpy(), ig, grp, rows=rows)
    g = got[:, :, rows].double().numpy()
    assert orc.max_abs_err(g, ref) <= 1e-2 and orc.rel_l2_err(g, ref) <= 5e-3
