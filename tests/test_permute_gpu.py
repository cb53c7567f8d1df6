"""Permute / unpermute parity with the oracle's gathers (exact equality)."""
import numpy as np
import pytest
import torch

from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("H,tile,o,hs,nt,batch,row,dtype", [
    (16, 64, 16, 2, 0, 2, 64, torch.float32),
    (8, 16, 4, 2, 5, 3, 8, torch.bfloat16),
    (64, 1024, 512, 8, 512, 1, 3072, torch.bfloat16),
    (64, 256, 128, 8, 512, 24, 128, torch.bfloat16),
    (1, 1, 0, 0, 3, 1, 4, torch.float32),
    (32, 64, 7, 4, 1, 5, 40, torch.bfloat16),
])
def test_permute_unpermute(H, tile, o, hs, nt, batch, row, dtype):
    S = nt + H * H
    g = torch.Generator().manual_seed(5)
    x = torch.randn((batch, S, row), generator=g, dtype=torch.float32).to(dtype)
    ref_p2o = orc.plan_arrays(H, H, tile, o, hs, nt)["phys2orig"]
    xn = x.view(torch.int16).numpy() if dtype == torch.bfloat16 else x.numpy()
    plan = hb.Plan(H, H, tile, o, hs, nt)
    try:
        xd = x.cuda()
        yd = torch.empty_like(xd)
        canary = torch.full_like(xd, 7.0)
        plan.permute(xd, yd)
        y = yd.cpu()
        yn = y.view(torch.int16).numpy() if dtype == torch.bfloat16 else y.numpy()
        assert np.array_equal(yn, orc.permute_rows(xn, ref_p2o))
        plan.unpermute(yd, canary)
        torch.cuda.synchronize()
        assert torch.equal(canary.cpu(), x)
        # the exit gather alone equals the oracle's
        zd = torch.empty_like(xd)
        plan.unpermute(xd, zd)
        z = zd.cpu()
        zn = z.view(torch.int16).numpy() if dtype == torch.bfloat16 else z.numpy()
        assert np.array_equal(zn, orc.unpermute_rows(xn, ref_p2o))
    finally:
        plan.destroy()


def test_permute_4d_heads_layout_and_errors():
    plan = hb.Plan(8, 8, 16, 4, 2, 5)
    try:
        x = torch.randn((2, 3, 69, 64), device="cuda")
        y = torch.empty_like(x)
        plan.permute(x, y)
        p2o = torch.from_numpy(plan.export(hb.EXPORT_PHYS2ORIG).astype(np.int64)).cuda()
        assert torch.equal(y, x[:, :, p2o])
        L = hb.lib()
        # in-place, misaligned rows, bad dtype
        assert L.hilberta_permute(x.data_ptr(), x.data_ptr(), plan._h, 6, 64, hb.FP32, None) == hb.ERR_INVALID
        assert L.hilberta_permute(x.data_ptr(), y.data_ptr(), plan._h, 6, 3, hb.FP32, None) == hb.ERR_INVALID
        assert L.hilberta_permute(x.data_ptr(), y.data_ptr(), plan._h, 6, 64, 9, None) == hb.ERR_INVALID
        assert L.hilberta_permute(x.data_ptr(), y.data_ptr(), plan._h, 0, 64, hb.FP32, None) == hb.ERR_INVALID
    finally:
        plan.destroy()
