"""Plan parity: every table the library exports equals the oracle's, bit for bit."""
import numpy as np
import pytest

from oracle import hilberta_oracle as orc
from paper_2509_26538_b200 import binding as hb
from paper_2509_26538_b200.inputs import TINY_LAYER_OFFSETS, WORKLOADS

pytestmark = pytest.mark.gpu


def _check(H, tile, o, hs, nt, W=None):
    W = H if W is None else W
    ref = orc.plan_arrays(H, W, tile, o, hs, nt)
    plan = hb.Plan(H, W, tile, o, hs, nt)
    try:
        assert np.array_equal(plan.export(hb.EXPORT_HIL_D2T), ref["hil_d2t"])
        assert np.array_equal(plan.export(hb.EXPORT_HIL_T2D), ref["hil_t2d"])
        assert np.array_equal(plan.export(hb.EXPORT_PHYS2ORIG), ref["phys2orig"])
        assert np.array_equal(plan.export(hb.EXPORT_ORIG2PHYS), ref["orig2phys"])
        assert np.array_equal(plan.export(hb.EXPORT_SHARED_RUNS), ref["shared_runs"])
        assert np.array_equal(plan.export(hb.EXPORT_WINDOWS), ref["windows"])
        assert int(plan.export(hb.EXPORT_NNZ)[0]) == ref["nnz"]
        info = plan.export(hb.EXPORT_INFO).tolist()
        NP = orc.padded_side(H, W) ** 2
        assert info == [H, W, tile, o % NP, hs, nt, hs * hs, NP // tile, orc.padded_side(H, W), 1, 0]
    finally:
        plan.destroy()


def test_tiny_config_all_layers():
    wl = WORKLOADS["tiny16"]
    for o in TINY_LAYER_OFFSETS:
        _check(wl.H, wl.tile, o, wl.shared_region, wl.n_text)


@pytest.mark.parametrize("tile", [256, 512, 1024])
def test_flux1024(tile):
    wl = WORKLOADS["flux1024"]
    _check(wl.H, tile, tile // 2, wl.shared_region, wl.n_text)


def test_flux1024_schedule_offsets():
    wl = WORKLOADS["flux1024"]
    for layer in (0, 1, 2, 3, 17, 56):
        _check(wl.H, 1024, (layer * 1024 // 4) % wl.HW, wl.shared_region, wl.n_text)


def test_flux2048_and_4096():
    for name in ("flux2048", "flux4096"):
        wl = WORKLOADS[name]
        _check(wl.H, wl.tile, wl.layer_offset, wl.shared_region, wl.n_text)


def test_paper_table_settings():
    _check(64, 256, 64, 16, 512)
    _check(128, 1024, 256, 32, 512)


def test_random_small_geometries():
    rng = np.random.default_rng(7)
    for _ in range(40):
        k = int(rng.integers(0, 6))
        H = 1 << k
        HW = H * H
        divs = [t for t in range(1, HW + 1) if HW % t == 0]
        tile = int(rng.choice(divs))
        o = int(rng.integers(-3 * HW, 3 * HW + 1))
        hs = int(rng.choice([s for s in range(0, H + 1, 2)]))
        nt = int(rng.choice([0, 1, 5, 77]))
        ref_o = o  # the oracle reduces the offset itself
        ref = orc.plan_arrays(H, H, tile, ref_o, hs, nt)
        plan = hb.Plan(H, H, tile, o, hs, nt)
        try:
            assert np.array_equal(plan.export(hb.EXPORT_PHYS2ORIG), ref["phys2orig"]), (H, tile, o, hs, nt)
            assert np.array_equal(plan.export(hb.EXPORT_WINDOWS), ref["windows"]), (H, tile, o, hs, nt)
            assert np.array_equal(plan.export(hb.EXPORT_SHARED_RUNS).reshape(-1, 2), ref["shared_runs"])
            assert int(plan.export(hb.EXPORT_NNZ)[0]) == ref["nnz"]
        finally:
            plan.destroy()


def test_general_shapes():
    """Non-square and non-power-of-two grids (appendix on general shapes)."""
    _check(24, 256, 100, 4, 77, W=40)      # padded to 64 x 64
    _check(3, 8, 3, 2, 2, W=5)
    _check(96, 1024, 512, 8, 512, W=128)   # a 3:4 latent grid
    _check(1, 16, 7, 0, 1, W=9)
    _check(100, 4096, 1024, 16, 0, W=100)
    rng = np.random.default_rng(11)
    for _ in range(25):
        H, W = int(rng.integers(1, 40)), int(rng.integers(1, 40))
        NP = orc.padded_side(H, W) ** 2
        tile = int(rng.choice([t for t in (1, 2, 4, 8, 16, 32, 64, 128, 256, 1024, 4096) if NP % t == 0]))
        hs = int(rng.choice([s for s in range(0, min(H, W) + 1, 2)]))
        _check(H, tile, int(rng.integers(-NP, 2 * NP)), hs, int(rng.choice([0, 3, 50])), W=W)


def test_degenerate_and_maximum():
    _check(1, 1, 0, 0, 0)          # single image token
    _check(1, 1, 0, 0, 3)
    _check(2, 4, 1, 2, 0)          # every image token shared
    _check(16, 256, 5, 16, 4)      # shared region = whole grid, one tile
    _check(512, 4096, 2048, 64, 512)  # 262144 image tokens
    _check(1024, 4096, 2048, 64, 512)  # the largest grid the library accepts: 1048576 image tokens
    _check(1000, 16384, 777, 10, 5, W=1024)  # the largest padded side with a ragged real grid


def test_export_buffer_protocol():
    import ctypes
    plan = hb.Plan(8, 8, 16, 4, 2, 5)
    try:
        need = ctypes.c_size_t()
        L = hb.lib()
        assert L.hilberta_plan_export(plan._h, hb.EXPORT_PHYS2ORIG, None, 0, ctypes.byref(need)) == 0
        assert need.value == 69 * 4
        buf = np.zeros(10, dtype=np.int32)
        assert L.hilberta_plan_export(plan._h, hb.EXPORT_PHYS2ORIG, buf.ctypes.data, buf.nbytes, None) == hb.ERR_BUFFER
        assert L.hilberta_plan_export(plan._h, 99, None, 0, None) == hb.ERR_INVALID
    finally:
        plan.destroy()
