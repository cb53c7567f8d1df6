"""fp32 forward parity with the fp64 oracle: max-abs and relative L2 <= 1e-5."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200.inputs import TINY_LAYER_OFFSETS, WORKLOADS, make_qkv

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5  # both metrics, fp32 inputs


def run_gpu(plan, q, k, v, scale=0.0):
    """Original-order host tensors in, original-order host tensor out; every
    step (permute, forward, unpermute) through the C ABI."""
    qd, kd, vd = (t.cuda() for t in (q, k, v))
    qp, kp, vp, op, od = (torch.empty_like(qd) for _ in range(5))
    plan.permute(qd, qp)
    plan.permute(kd, kp)
    plan.permute(vd, vp)
    plan.bind_like(qp, scale)
    plan.forward(qp, kp, vp, op)
    plan.unpermute(op, od)
    torch.cuda.synchronize()
    return od.cpu()


def oracle(H, tile, o, hs, nt, q, k, v, scale=None):
    ig, grp = orc.token_classes(H, H, tile, o, hs, nt)
    return attn_c.attention_rows(q.float().numpy(), k.float().numpy(), v.float().numpy(), ig, grp, scale=scale)


def test_tiny_config_four_layers():
    wl = WORKLOADS["tiny16"]
    q, k, v = make_qkv(wl)
    for o in TINY_LAYER_OFFSETS:
        plan = hb.Plan(wl.H, wl.W, wl.tile, o, wl.shared_region, wl.n_text)
        try:
            got = run_gpu(plan, q, k, v).double().numpy()
        finally:
            plan.destroy()
        ref = oracle(wl.H, wl.tile, o, wl.shared_region, wl.n_text, q, k, v)
        assert orc.max_abs_err(got, ref) <= TOL_FP32
        assert orc.rel_l2_err(got, ref) <= TOL_FP32


@pytest.mark.parametrize("H,tile,o,hs,nt,B,heads,D", [
    (8, 16, 4, 2, 5, 2, 3, 32),
    (16, 64, 48, 4, 7, 1, 2, 128),
    (8, 64, 9, 0, 0, 1, 1, 64),      # one tile, no prefix: dense
    (8, 16, 0, 0, 0, 1, 2, 64),      # block diagonal
    (4, 4, 1, 4, 0, 1, 1, 32),       # every token shared: dense
    (1, 1, 0, 0, 0, 1, 1, 32),       # a single token
    (32, 128, 32, 8, 33, 1, 2, 64),
])
def test_shapes_and_degenerate_cases(H, tile, o, hs, nt, B, heads, D):
    S = nt + H * H
    g = torch.Generator().manual_seed(100 + H + D)
    q, k, v = (torch.randn((B, heads, S, D), generator=g) for _ in range(3))
    plan = hb.Plan(H, H, tile, o, hs, nt)
    try:
        got = run_gpu(plan, q, k, v).double().numpy()
    finally:
        plan.destroy()
    ref = oracle(H, tile, o, hs, nt, q, k, v)
    assert orc.max_abs_err(got, ref) <= TOL_FP32
    assert orc.rel_l2_err(got, ref) <= TOL_FP32


def test_dense_case_matches_sdpa_and_custom_scale():
    H, nt, D = 8, 3, 64
    S = nt + H * H
    g = torch.Generator().manual_seed(3)
    q, k, v = (torch.randn((1, 2, S, D), generator=g) for _ in range(3))
    plan = hb.Plan(H, H, H * H, 11, 0, nt)
    try:
        got = run_gpu(plan, q, k, v, scale=0.2)
    finally:
        plan.destroy()
    ref = torch.nn.functional.scaled_dot_product_attention(q.double(), k.double(), v.double(), scale=0.2)
    assert (got.double() - ref).abs().max().item() <= TOL_FP32


def test_peaky_rows_and_strided_layout():
    H, tile, o, hs, nt, D = 8, 16, 4, 2, 5, 64
    S = nt + H * H
    g = torch.Generator().manual_seed(11)
    q, k, v = (torch.randn((1, 2, S, D), generator=g) for _ in range(3))
    q = q * 8.0
    ref = oracle(H, tile, o, hs, nt, q, k, v)
    plan = hb.Plan(H, H, tile, o, hs, nt)
    try:
        # [B, S, heads, D] storage viewed as [B, heads, S, D]
        def strided(t):
            return t.permute(0, 2, 1, 3).contiguous().cuda().permute(0, 2, 1, 3)
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        qp, kp, vp = (strided(t[:, :, p2o]) for t in (q, k, v))
        out = torch.empty_like(qp)
        assert not qp.is_contiguous()
        plan.bind_like(qp)
        plan.forward(qp, kp, vp, out)
        torch.cuda.synchronize()
        got = torch.empty_like(q)
        got[:, :, p2o] = out.cpu()
    finally:
        plan.destroy()
    assert orc.max_abs_err(got.double().numpy(), ref) <= TOL_FP32
    assert orc.rel_l2_err(got.double().numpy(), ref) <= TOL_FP32


def test_forward_errors():
    plan = hb.Plan(8, 8, 16, 0, 0, 0)
    try:
        x = torch.zeros((1, 1, 64, 64), device="cuda")
        y = torch.zeros_like(x)
        L = hb.lib()
        assert L.hilberta_forward(x.data_ptr(), x.data_ptr(), x.data_ptr(), y.data_ptr(), plan._h, None) == hb.ERR_UNBOUND
        assert L.hilberta_plan_bind(plan._h, 1, 1, 48, hb.FP32, 0, 0, 0, 0.0) == hb.ERR_UNSUPPORTED
        assert L.hilberta_plan_bind(plan._h, 1, 1, 64, 5, 0, 0, 0, 0.0) == hb.ERR_INVALID
        assert L.hilberta_plan_bind(plan._h, 0, 1, 64, hb.FP32, 0, 0, 0, 0.0) == hb.ERR_INVALID
        plan.bind(1, 1, 64, hb.FP32)
        assert L.hilberta_forward(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), plan._h, None) == hb.ERR_INVALID
        assert L.hilberta_forward(x.data_ptr(), x.data_ptr(), x.data_ptr(), None, plan._h, None) == hb.ERR_INVALID
    finally:
        plan.destroy()


def test_general_shape_fp32():
    H, W, tile, o, hs, nt = 12, 20, 64, 19, 4, 7
    S = nt + H * W
    g = torch.Generator().manual_seed(8)
    q, k, v = (torch.randn((1, 2, S, 64), generator=g) for _ in range(3))
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        got = run_gpu(plan, q, k, v).double().numpy()
    finally:
        plan.destroy()
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    ref = attn_c.attention_rows(q.numpy(), k.numpy(), v.numpy(), ig, grp)
    assert orc.max_abs_err(got, ref) <= TOL_FP32 and orc.rel_l2_err(got, ref) <= TOL_FP32
