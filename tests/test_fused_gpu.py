"""hilberta_forward_fused: the entry gather (and the exit gather) fused into the attention launch
must give exactly what permute -> forward (-> unpermute) gives."""
import pytest
import torch

from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,W,tile,o,hs,nt,B,heads,D,dtype", [
    (32, 32, 256, 128, 4, 77, 2, 3, 128, torch.bfloat16),   # ragged tiles, text prefix, batch 2
    (16, 16, 64, 16, 2, 0, 1, 2, 128, torch.bfloat16),
    (24, 40, 256, 100, 4, 33, 1, 2, 128, torch.bfloat16),   # non-square grid on the padded curve
    (64, 64, 1024, 512, 8, 512, 1, 4, 128, torch.bfloat16),  # Flux 1024^2 shape, four heads
    (16, 16, 64, 48, 2, 5, 1, 2, 64, torch.float32),
])
def test_fused_entry_and_exit_match_separate_gathers(H, W, tile, o, hs, nt, B, heads, D, dtype):
    S = nt + H * W
    g = torch.Generator().manual_seed(77)
    q, k, v = (torch.randn((B, heads, S, D), generator=g).to(dtype).cuda() for _ in range(3))
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        qp, kp, vp, out_phys, out_orig = (torch.empty_like(q) for _ in range(5))
        for src, dst in ((q, qp), (k, kp), (v, vp)):
            plan.permute(src, dst)
        plan.bind_like(qp)
        plan.forward(qp, kp, vp, out_phys)
        plan.unpermute(out_phys, out_orig)
        view = torch.int16 if dtype == torch.bfloat16 else torch.int32
        for in_o, out_o, want in ((True, False, out_phys), (True, True, out_orig), (False, True, out_orig),
                                  (False, False, out_phys)):
            got = torch.full_like(q, float("nan"))
            a = (q, k, v) if in_o else (qp, kp, vp)
            plan.forward_fused(*a, got, in_original=in_o, out_original=out_o)
            assert plan.status() == 0
            assert torch.equal(got.view(view), want.view(view)), (in_o, out_o)
    finally:
        plan.destroy()


def test_fused_strided_inputs():
    """q, k, v as slices of one packed [B, S, 3, heads, D] projection output, original order."""
    H = W = 32
    nt, heads, D = 40, 2, 128
    S = nt + H * W
    g = torch.Generator().manual_seed(78)
    qkv = torch.randn((1, S, 3, heads, D), generator=g).to(torch.bfloat16).cuda()
    q, k, v = (qkv[:, :, i].permute(0, 2, 1, 3) for i in range(3))   # [B, heads, S, D] views
    plan = hb.Plan(H, W, 256, 64, 4, nt)
    try:
        plan.bind_like(q)
        qc, kc, vc = (t.contiguous() for t in (q, k, v))
        qp, kp, vp = (torch.empty_like(qc) for _ in range(3))
        for src, dst in ((qc, qp), (kc, kp), (vc, vp)):
            plan.permute(src, dst)
        got = torch.empty_like(qkv)[:, :, 0].permute(0, 2, 1, 3)      # same strides as q
        plan.forward_fused(q, k, v, got, in_original=True, out_original=False)
        want = torch.empty_like(qp)
        plan.bind_like(qp)
        plan.forward(qp, kp, vp, want)
        assert plan.status() == 0
        assert torch.equal(got.contiguous().view(torch.int16), want.view(torch.int16))
    finally:
        plan.destroy()


@pytest.mark.parametrize("D,dtype,B,heads", [(128, torch.bfloat16, 1, 2), (128, torch.bfloat16, 2, 6),
                                              (128, torch.bfloat16, 1, 1), (64, torch.float32, 2, 3)])
def test_forward_host_matches_device_path(D, dtype, B, heads):
    """Host-buffer entry point (copies and fused launches pipelined over slices of heads) against
    permute -> forward -> unpermute."""
    H = W = 32
    nt = 21
    S = nt + H * W
    g = torch.Generator().manual_seed(79)
    q, k, v = (torch.randn((B, heads, S, D), generator=g).to(dtype).pin_memory() for _ in range(3))
    out_h = torch.empty_like(q).pin_memory()
    plan = hb.Plan(H, W, 256, 192, 4, nt)
    try:
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        qp, kp, vp, op, od = (torch.empty_like(qd) for _ in range(5))
        plan.bind_like(qd)
        for src, dst in ((qd, qp), (kd, kp), (vd, vp)):
            plan.permute(src, dst)
        plan.forward(qp, kp, vp, op)
        plan.unpermute(op, od)
        for _ in range(2):   # the second call reuses the workspace
            out_h.fill_(float("nan"))
            plan.forward_host(q, k, v, out_h)
            assert plan.status() == 0
            view = torch.int16 if dtype == torch.bfloat16 else torch.int32
            assert torch.equal(out_h.view(view), od.cpu().view(view))
    finally:
        plan.destroy()
