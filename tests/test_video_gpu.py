"""hilberta_plan_video: plan tables bit-exact against the oracle's 3-D geometry, and the
attention kernels (forward and backward) in tolerance on a video volume."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("F,H,W,tile,o,hs,fs,nt", [
    (4, 4, 4, 16, 5, 2, 2, 3),
    (2, 4, 4, 8, 3, 2, 2, 0),
    (3, 4, 2, 16, 7, 0, 0, 2),
    (8, 16, 16, 512, 200, 4, 2, 77),      # a clip shorter than the image is wide: 2 x 2 macro cells of 8-cubes
    (16, 16, 16, 256, 64, 8, 4, 0),       # a full cube
    (5, 12, 20, 1024, 999, 2, 2, 9),      # nothing is a power of two
    (8, 64, 64, 2048, 512, 8, 4, 100),    # a video-shaped volume without any padding
    (32, 8, 8, 4096, 77, 2, 2, 0),        # more frames than pixels per side: one 32-cube
])
def test_video_plan_bit_exact(F, H, W, tile, o, hs, fs, nt):
    ref = orc.plan_arrays(H, W, tile, o, hs, nt, frames=F, shared_frames=fs)
    plan = hb.Plan(H, W, tile, o, hs, nt, frames=F, shared_frames=fs)
    try:
        assert np.array_equal(plan.export(hb.EXPORT_HIL_D2T), ref["hil_d2t"])
        assert np.array_equal(plan.export(hb.EXPORT_HIL_T2D), ref["hil_t2d"])
        assert np.array_equal(plan.export(hb.EXPORT_PHYS2ORIG), ref["phys2orig"])
        assert np.array_equal(plan.export(hb.EXPORT_ORIG2PHYS), ref["orig2phys"])
        assert np.array_equal(plan.export(hb.EXPORT_SHARED_RUNS), ref["shared_runs"])
        assert np.array_equal(plan.export(hb.EXPORT_WINDOWS), ref["windows"])
        assert int(plan.export(hb.EXPORT_NNZ)[0]) == ref["nnz"]
        info = plan.export(hb.EXPORT_INFO).tolist()
        n, NP = orc.padded_side(H, W, F), orc.padded_length(H, W, F)
        assert info == [H, W, tile, o % NP, hs, nt, hs * hs * fs, NP // tile, n, F, fs]
    finally:
        plan.destroy()


def test_video_plan_argument_checks():
    L = hb.lib()
    import ctypes
    h = ctypes.c_void_p()
    for args in ((1, 4, 4, 16, 0, 0, 0, 0),        # one frame is an image: use hilberta_plan
                 (4, 4, 4, 24, 0, 0, 0, 0),        # tile does not divide 64
                 (2, 4, 4, 64, 0, 0, 0, 0),        # the padded curve of a 2 x 4 x 4 clip has 32 positions
                 (4, 4, 4, 16, 0, 2, 0, 0),        # shared square without temporal extent
                 (4, 4, 4, 16, 0, 2, 3, 0),        # odd temporal extent
                 (4, 4, 4, 16, 0, 2, 6, 0)):       # longer than the clip
        assert L.hilberta_plan_video(*args, ctypes.byref(h)) == hb.ERR_INVALID
    assert L.hilberta_plan_video(200, 4, 4, 16, 0, 0, 0, 0, ctypes.byref(h)) == hb.ERR_UNSUPPORTED


def test_video_forward_and_backward_match_oracle():
    F, H, W, tile, o, hs, fs, nt, heads = 8, 16, 16, 512, 200, 4, 2, 40, 2
    S = nt + F * H * W
    g = torch.Generator().manual_seed(8)
    q, k, v, do = (torch.randn((1, heads, S, 128), generator=g).to(torch.bfloat16) for _ in range(4))
    ig, grp = orc.token_classes(H, W, tile, o, hs, nt, frames=F, shared_frames=fs)
    f32 = lambda t: t.float().numpy()
    ref_out = attn_c.attention_rows(f32(q), f32(k), f32(v), ig, grp)
    ref_g = attn_c.attention_backward(f32(q), f32(k), f32(v), f32(do), ig, grp)
    plan = hb.Plan(H, W, tile, o, hs, nt, frames=F, shared_frames=fs)
    try:
        qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
        plan.bind_like(qd)
        out = torch.empty_like(qd)
        plan.forward_fused(qd, kd, vd, out, in_original=True, out_original=True)
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64))
        qp, kp, vp, dop = (t[:, :, p2o.cuda()].contiguous() for t in (qd, kd, vd, dod))
        outp = torch.empty_like(qp)
        lse = torch.empty((1, heads, S), device="cuda", dtype=torch.float32)
        plan.forward_lse(qp, kp, vp, outp, lse)
        grads = [torch.empty_like(qp) for _ in range(3)]
        plan.backward(dop, qp, kp, vp, outp, lse, *grads)
        assert plan.status() == 0
        got = out.cpu().double().numpy()
        assert orc.max_abs_err(got, ref_out) <= 1e-2 and orc.rel_l2_err(got, ref_out) <= 5e-3
        for t, r in zip(grads, ref_g):
            full = torch.empty((1, heads, S, 128), dtype=torch.float64)
            full[:, :, p2o] = t.cpu().double()
            assert orc.rel_l2_err(full.numpy(), r) <= 5e-3
    finally:
        plan.destroy()
