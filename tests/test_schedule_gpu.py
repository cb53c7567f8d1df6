"""Full per-step layer schedule at 1024^2 (57 layers, offsets (layer * tile / 4) mod HW),
with the entry and exit gathers: plans per distinct offset are bit-exact, and the
forward matches the oracle over the WHOLE output tensor (all 4608 tokens, all 24 heads) for a layer of
each of the four distinct masks, and on sampled rows for later layers, all run through the schedule's own loop."""
import numpy as np
import pytest
import torch

from oracle import attn_c
from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200.inputs import SCHEDULE_LAYERS, WORKLOADS, make_qkv, sample_rows, schedule_offset

pytestmark = pytest.mark.gpu


def test_schedule_57_layers():
    wl = WORKLOADS["flux1024"]
    tile = 1024
    offsets = [schedule_offset(layer, tile, wl.HW) for layer in range(SCHEDULE_LAYERS)]
    assert len(set(o % tile for o in offsets)) == 4  # only four distinct masks
    plans = {}
    try:
        for o in sorted(set(offsets)):
            plans[o] = hb.Plan(wl.H, wl.W, tile, o, wl.shared_region, wl.n_text)
            ref = orc.plan_arrays(wl.H, wl.W, tile, o, wl.shared_region, wl.n_text)
            assert np.array_equal(plans[o].export(hb.EXPORT_WINDOWS), ref["windows"])
            assert np.array_equal(plans[o].export(hb.EXPORT_PHYS2ORIG), ref["phys2orig"])
            assert int(plans[o].export(hb.EXPORT_NNZ)[0]) == ref["nnz"]
        # the physical layout does not depend on the offset: one permute serves all layers
        base = plans[offsets[0]].export(hb.EXPORT_PHYS2ORIG)
        for p in plans.values():
            assert np.array_equal(p.export(hb.EXPORT_PHYS2ORIG), base)

        q, k, v = make_qkv(wl)
        qd, kd, vd = (t.cuda() for t in (q, k, v))
        qp, kp, vp, op, od = (torch.empty_like(qd) for _ in range(5))
        first = plans[offsets[0]]
        first.permute(qd, qp)
        first.permute(kd, kp)
        first.permute(vd, vp)
        for p in plans.values():
            p.bind_like(qp)
        rows = sample_rows(wl, 48)
        whole_layers = {0, 1, 2, 3}          # offsets 0, 256, 512, 768: the four masks
        sampled_layers = {17, 38, 56}
        qf, kf, vf = (t.float().numpy() for t in (q, k, v))
        for layer, o in enumerate(offsets):
            plans[o].forward(qp, kp, vp, op)
            if layer in whole_layers or layer in sampled_layers:
                first.unpermute(op, od)
                torch.cuda.synchronize()
                ig, grp = orc.token_classes(wl.H, wl.W, tile, o, wl.shared_region, wl.n_text)
                if layer in whole_layers:
                    got = od.cpu().double().numpy()
                    ref = attn_c.attention_rows(qf, kf, vf, ig, grp)
                else:
                    got = od[:, :, rows].cpu().double().numpy()
                    ref = attn_c.attention_rows(qf, kf, vf, ig, grp, rows=rows)
                assert np.isfinite(got).all()
                assert orc.max_abs_err(got, ref) <= 1e-2 and orc.rel_l2_err(got, ref) <= 5e-3, (layer, o)
        assert len({offsets[l] % tile for l in whole_layers}) == 4
        for p in plans.values():
            assert p.status() == 0
    finally:
        for p in plans.values():
            p.destroy()
