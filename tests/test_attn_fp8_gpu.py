"""e4m3 operands (q, k, v as 8-bit floats, bf16 output) against the fp64 oracle run on the same
8-bit values.

Tolerance.  The inputs are exact in both paths; the kernel's only extra rounding is that of the
softmax weights to e4m3 before they multiply V: three mantissa bits, relative error at most 2^-4
and, for round-to-nearest, root-mean-square at most 2^-4 / sqrt(3) = 3.6e-2.  The errors of
different keys are independent and zero-mean, so for the output row sum_j p_j v_j / sum_j p_j the
relative L2 error is bounded by that rms figure (it is what random V attains; correlated V does
better): rel-L2 <= 4e-2.  A single output element errs by at most 2^-4 sum_j p_j |v_j| / sum_j p_j;
the tests bound it by 2^-4 times the largest |v|.  Rows whose weights are exactly representable
(one kept key; equal scores) must meet the bf16 tolerance."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200.inputs import WORKLOADS, make_qkv, sample_rows

pytestmark = pytest.mark.gpu

F8 = torch.float8_e4m3fn
TOL_REL_L2 = 4e-2
TOL_EXACT_MAX_ABS, TOL_EXACT_REL_L2 = 1e-2, 5e-3


def draw(shape, seed, gain=1.0):
    g = torch.Generator().manual_seed(seed)
    return tuple((torch.randn(shape, generator=g) * (gain if i == 0 else 1.0)).to(F8) for i in range(3))


def run_gpu(plan, q, k, v, scale=0.0, lse=False):
    """Original-order e4m3 host tensors in; original-order bf16 output (and lse) out."""
    B, heads, S, D = q.shape
    qd, kd, vd = (t.cuda() for t in (q, k, v))
    qp, kp, vp = (torch.empty_like(qd) for _ in range(3))
    for src, dst in ((qd, qp), (kd, kp), (vd, vp)):
        plan.permute(src, dst)
    plan.bind_like(qp, scale)
    op = torch.full((B, heads, S, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    od = torch.empty_like(op)
    l = torch.empty((B, heads, S), device="cuda", dtype=torch.float32) if lse else None
    if lse:
        plan.forward_lse(qp, kp, vp, op, l)
    else:
        plan.forward(qp, kp, vp, op)
    assert plan.status() == 0
    op2 = torch.full_like(op, float("nan"))
    plan.forward(qp, kp, vp, op2)
    assert torch.equal(op.view(torch.int16), op2.view(torch.int16))  # deterministic
    plan.unpermute(op, od)
    # entry and exit gathers fused into the launch: the same bytes
    of = torch.full_like(op, float("nan"))
    plan.forward_fused(qd, kd, vd, of, in_original=True, out_original=True)
    assert plan.status() == 0
    assert torch.equal(of.view(torch.int16), od.view(torch.int16))
    ou = torch.full_like(op, float("nan"))
    plan.forward_unpermute(qp, kp, vp, ou)
    assert torch.equal(ou.view(torch.int16), od.view(torch.int16))
    torch.cuda.synchronize()
    if lse:
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        full = torch.empty((B, heads, S), dtype=torch.float64)
        full[:, :, p2o] = l.cpu().double()
        return od.cpu(), full.numpy()
    return od.cpu()


def f64(t):
    return t.float().numpy()


@pytest.mark.parametrize("H,W,tile,o,hs,nt,B,heads", [
    (16, 16, 64, 16, 2, 0, 1, 2),      # ragged 62/63/64-key ranges, wrapped tile
    (16, 16, 64, 0, 2, 5, 2, 2),       # text tokens, batch 2
    (16, 16, 256, 3, 0, 0, 1, 1),      # one tile, no prefix: dense
    (8, 8, 16, 4, 8, 0, 1, 1),         # every token shared
    (32, 32, 128, 100, 4, 77, 1, 3),   # ragged prefix, several blocks per range
    (24, 40, 256, 100, 4, 33, 1, 2),   # non-square grid
    (1, 1, 1, 0, 0, 0, 1, 1),          # a single token
    (2, 2, 1, 0, 0, 300, 1, 2),        # almost only text
    (64, 64, 1024, 512, 8, 512, 1, 2), # Flux 1024^2 shape, two heads
])
def test_small_cases_elementwise(H, W, tile, o, hs, nt, B, heads):
    S = nt + H * W
    q, k, v = draw((B, heads, S, 128), 800 + H + nt)
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    ref, ref_lse = attn_c.attention_rows(f64(q), f64(k), f64(v), ig, grp, return_lse=True)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        got, got_lse = run_gpu(plan, q, k, v, lse=True)
    finally:
        plan.destroy()
    got = got.double().numpy()
    assert np.isfinite(got).all()
    if np.abs(ref).max() > 0:
        assert orc.rel_l2_err(got, ref) <= TOL_REL_L2, orc.rel_l2_err(got, ref)
    assert orc.max_abs_err(got, ref) <= 2.0 ** -4 * float(np.abs(f64(v)).max()) + 1e-2
    # the row sum is kept in fp32 from unrounded weights: lse is as tight as the bf16 kernel's
    assert np.max(np.abs(got_lse - ref_lse)) <= 2e-3


def test_exactly_representable_weights_meet_the_bf16_tolerance():
    """q = 0: every kept key has the same weight, a power of two in e4m3, so the only roundings
    left are the fp32 accumulation and the bf16 output: out = mean of the kept V rows.  A wrong
    key set, a misplaced V row or a wrong weight count shows at the tight tolerance."""
    H, W, tile, o, hs, nt, B, heads = 32, 32, 128, 100, 4, 77, 1, 2
    S = nt + H * W
    _, k, v = draw((B, heads, S, 128), 901)
    q = torch.zeros((B, heads, S, 128)).to(F8)
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    ref = attn_c.attention_rows(f64(q), f64(k), f64(v), ig, grp)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        got = run_gpu(plan, q, k, v).double().numpy()
    finally:
        plan.destroy()
    assert orc.max_abs_err(got, ref) <= TOL_EXACT_MAX_ABS and orc.rel_l2_err(got, ref) <= TOL_EXACT_REL_L2


def test_one_hot_rows_return_the_selected_value_row():
    """With q_i = 16 e_{7 i mod 128}, k_j = 16 e_{j mod 128} and scale 1, a row's kept keys whose
    index matches score 256 and all others 0: the winners outweigh the rest by e^256, the losers'
    weights underflow to zero in both paths, and the output is the mean of the winners' V rows
    (rows without a winner average all their keys).  All weights are powers of two."""
    H, W, tile, o, hs, nt, B, heads = 16, 16, 64, 16, 2, 3, 1, 1
    S = nt + H * W
    g = torch.Generator().manual_seed(77)
    v = torch.randn((B, heads, S, 128), generator=g).to(F8)
    k = torch.zeros((B, heads, S, 128))
    k[0, 0, torch.arange(S), torch.arange(S) % 128] = 16.0
    q = torch.zeros((B, heads, S, 128))
    q[0, 0, torch.arange(S), (torch.arange(S) * 7) % 128] = 16.0
    q, k = q.to(F8), k.to(F8)
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    ref = attn_c.attention_rows(f64(q), f64(k), f64(v), ig, grp, scale=1.0)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        got = run_gpu(plan, q, k, v, scale=1.0).double().numpy()
    finally:
        plan.destroy()
    assert orc.max_abs_err(got, ref) <= TOL_EXACT_MAX_ABS and orc.rel_l2_err(got, ref) <= TOL_EXACT_REL_L2


def test_peaky_rows_and_custom_scale():
    """Large logits: the lazily advanced maximum has to move (weights may not exceed e4m3's range)."""
    H, W, tile, o, hs, nt, B, heads = 32, 32, 256, 64, 4, 40, 1, 2
    S = nt + H * W
    q, k, v = draw((B, heads, S, 128), 903, gain=4.0)
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    for scale in (0.25, 0.02):
        ref = attn_c.attention_rows(f64(q), f64(k), f64(v), ig, grp, scale=scale)
        plan = hb.Plan(H, W, tile, o, hs, nt)
        try:
            got = run_gpu(plan, q, k, v, scale=scale).double().numpy()
        finally:
            plan.destroy()
        assert np.isfinite(got).all()
        assert orc.rel_l2_err(got, ref) <= TOL_REL_L2, (scale, orc.rel_l2_err(got, ref))


def test_strided_layout():
    """q, k, v as slices of one packed [B, S, 3, heads, D] buffer; out with the same element strides."""
    H, W, tile, o, hs, nt, B, heads = 16, 16, 64, 16, 2, 5, 2, 3
    S = nt + H * W
    g = torch.Generator().manual_seed(905)
    packed = torch.randn((B, S, 3, heads, 128), generator=g).to(F8)
    q, k, v = (packed[:, :, i].permute(0, 2, 1, 3) for i in range(3))   # [B, heads, S, D] views
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        pd = packed[:, p2o].contiguous().cuda()                        # physical order, packed
        qd, kd, vd = (pd[:, :, i].permute(0, 2, 1, 3) for i in range(3))
        out_buf = torch.full((B, S, 3, heads, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
        od = out_buf[:, :, 0].permute(0, 2, 1, 3)
        assert od.stride() == qd.stride()
        plan.bind_like(qd)
        plan.forward(qd, kd, vd, od)
        assert plan.status() == 0
        got = torch.empty((B, heads, S, 128), dtype=torch.float64)
        got[:, :, p2o] = od.cpu().double()
    finally:
        plan.destroy()
    ref = attn_c.attention_rows(f64(q.contiguous()), f64(k.contiguous()), f64(v.contiguous()), ig, grp)
    assert orc.rel_l2_err(got.numpy(), ref) <= TOL_REL_L2
    assert torch.isnan(out_buf[:, :, 1:].float()).all()   # nothing written outside `out`


def test_full_size_sampled_rows():
    """The bench's launch configuration at 2048^2 (24 heads, full sequence); sampled rows by the oracle."""
    wl = WORKLOADS["flux2048"].with_(dtype="fp8")
    q, k, v = make_qkv(wl)
    plan = hb.Plan(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)
    try:
        got = run_gpu(plan, q, k, v)
    finally:
        plan.destroy()
    rows = sample_rows(wl, 24)
    ig, grp = orc.token_classes(wl.H, wl.W, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)
    ref = attn_c.attention_rows(f64(q), f64(k), f64(v), ig, grp, rows=rows)
    g = got[:, :, rows].double().numpy()
    assert torch.isfinite(got.float()).all()
    assert orc.rel_l2_err(g, ref) <= TOL_REL_L2, orc.rel_l2_err(g, ref)


def test_host_buffer_path_equals_the_device_path():
    """hilberta_forward_host with 8-bit inputs and a bf16 output: pipelined over slices of heads, the
    same bytes as the fused device call."""
    H, W, tile, o, hs, nt, B, heads = 32, 32, 128, 100, 4, 77, 2, 8
    S = nt + H * W
    q, k, v = draw((B, heads, S, 128), 907)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        plan.bind_like(qd)
        of = torch.full((B, heads, S, 128), float("nan"), device="cuda", dtype=torch.bfloat16)
        plan.forward_fused(qd, kd, vd, of, in_original=True, out_original=True)
        qh, kh, vh = (t.pin_memory() for t in (q, k, v))
        oh = torch.full((B, heads, S, 128), float("nan"), dtype=torch.bfloat16).pin_memory()
        plan.forward_host(qh, kh, vh, oh)
        assert plan.status() == 0
        assert torch.equal(oh.view(torch.int16), of.cpu().view(torch.int16))
    finally:
        plan.destroy()


def test_unsupported_calls_are_refused():
    H, W, tile, o, hs, nt = 16, 16, 64, 0, 2, 0
    S = H * W
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        with pytest.raises(hb.HilbertaError) as e:
            plan.bind(1, 1, 64, hb.FP8_E4M3)
        assert e.value.status == hb.ERR_UNSUPPORTED
        with pytest.raises(hb.HilbertaError) as e:
            plan.bind(1, 1, 128, hb.FP8_E4M3, strides=(S * 136, S * 136, 136))  # 136 is not a multiple of 16
        assert e.value.status == hb.ERR_INVALID
        q, k, v = (t.cuda() for t in draw((1, 1, S, 128), 5))
        plan.bind_like(q)
        x = torch.zeros((1, 1, S, 128), device="cuda", dtype=torch.bfloat16)
        lse = torch.zeros((1, 1, S), device="cuda", dtype=torch.float32)
        with pytest.raises(hb.HilbertaError) as e:
            plan.backward(x, q, k, v, x.clone(), lse, x.clone(), x.clone(), x.clone())
        assert e.value.status == hb.ERR_UNSUPPORTED
    finally:
        plan.destroy()
