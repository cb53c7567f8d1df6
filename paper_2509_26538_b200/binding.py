"""ctypes binding over libhilberta.so: same names as the C ABI, marshalling only.

Tensors are torch CUDA tensors used as plain device memory; every step of the
path runs inside the library's kernels.  If the shared library is missing or
fails to load, every call raises -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhilberta.so")

OK = 0
ERR_INVALID, ERR_UNSUPPORTED, ERR_ARCH, ERR_CUDA, ERR_NOMEM, ERR_BUFFER, ERR_UNBOUND, ERR_TIMEOUT = (
    -1, -2, -3, -4, -5, -6, -7, -8)
BF16, FP32, FP8_E4M3 = 0, 1, 2
(EXPORT_HIL_D2T, EXPORT_HIL_T2D, EXPORT_PHYS2ORIG, EXPORT_ORIG2PHYS, EXPORT_SHARED_RUNS, EXPORT_WINDOWS,
 EXPORT_NNZ, EXPORT_INFO, EXPORT_LAUNCH_CLOCK) = range(9)

# every symbol include/hilberta.h declares
SYMBOLS = (
    "hilberta_plan", "hilberta_plan_groups", "hilberta_plan_video", "hilberta_plan_destroy", "hilberta_plan_export",
    "hilberta_plan_bind",
    "hilberta_forward", "hilberta_forward_unpermute", "hilberta_forward_fused", "hilberta_forward_lse",
    "hilberta_backward",
    "hilberta_backward_static", "hilberta_permute",
    "hilberta_unpermute",
    "hilberta_forward_host",
    "hilberta_check_work_list", "hilberta_check_overlap", "hilberta_schedule_units",
    "hilberta_plan_status", "hilberta_selftest_timeout", "hilberta_launch_count", "hilberta_status_string", "hilberta_version",
    "hilberta_last_cuda_error",
)

_lib = None


class HilbertaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().hilberta_status_string(status).decode()
        if status == ERR_CUDA:
            msg += f" (cudaError {lib().hilberta_last_cuda_error()})"
        super().__init__(f"{where}: {msg} [{status}]")


def lib():
    """Load the C-ABI library (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2509_26538_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    L.hilberta_plan.argtypes = [i32] * 6 + [ctypes.POINTER(vp)]
    L.hilberta_plan.restype = i32
    L.hilberta_plan_groups.argtypes = [i32] * 6 + [ctypes.POINTER(vp)]
    L.hilberta_plan_groups.restype = i32
    L.hilberta_plan_video.argtypes = [i32] * 8 + [ctypes.POINTER(vp)]
    L.hilberta_plan_video.restype = i32
    L.hilberta_plan_destroy.argtypes = [vp]
    L.hilberta_plan_destroy.restype = i32
    L.hilberta_plan_export.argtypes = [vp, i32, vp, sz, ctypes.POINTER(sz)]
    L.hilberta_plan_export.restype = i32
    L.hilberta_plan_bind.argtypes = [vp, i32, i32, i32, i32, i64, i64, i64, f32]
    L.hilberta_plan_bind.restype = i32
    L.hilberta_forward.argtypes = [vp, vp, vp, vp, vp, vp]
    L.hilberta_forward.restype = i32
    L.hilberta_forward_unpermute.argtypes = [vp, vp, vp, vp, vp, vp]
    L.hilberta_forward_unpermute.restype = i32
    L.hilberta_forward_fused.argtypes = [vp, vp, vp, vp, vp, i32, i32, vp]
    L.hilberta_forward_fused.restype = i32
    L.hilberta_forward_lse.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    L.hilberta_forward_lse.restype = i32
    L.hilberta_backward.argtypes = [vp] * 11
    L.hilberta_backward.restype = i32
    L.hilberta_backward_static.argtypes = [vp] * 11
    L.hilberta_backward_static.restype = i32
    L.hilberta_forward_host.argtypes = [vp, vp, vp, vp, vp, vp]
    L.hilberta_forward_host.restype = i32
    for name in ("hilberta_permute", "hilberta_unpermute"):
        f = getattr(L, name)
        f.argtypes = [vp, vp, vp, i32, i32, i32, vp]
        f.restype = i32
    L.hilberta_check_work_list.argtypes = [vp, i32, i32, i32, i32]
    L.hilberta_check_work_list.restype = i32
    i64, u64 = ctypes.c_int64, ctypes.c_uint64
    L.hilberta_check_overlap.argtypes = [u64, u64, i32, i32, i32, i64, i64, i64, i64]
    L.hilberta_check_overlap.restype = i32
    L.hilberta_schedule_units.argtypes = [i32, vp, vp, i32, i32, vp, vp, vp]
    L.hilberta_schedule_units.restype = i32
    L.hilberta_selftest_timeout.argtypes = [vp, vp]
    L.hilberta_selftest_timeout.restype = i32
    L.hilberta_plan_status.argtypes = [vp]
    L.hilberta_plan_status.restype = i32
    L.hilberta_launch_count.argtypes = []
    L.hilberta_launch_count.restype = ctypes.c_uint64
    L.hilberta_status_string.argtypes = [i32]
    L.hilberta_status_string.restype = ctypes.c_char_p
    L.hilberta_version.argtypes = []
    L.hilberta_version.restype = i32
    L.hilberta_last_cuda_error.argtypes = []
    L.hilberta_last_cuda_error.restype = i32
    _lib = L
    return L


def check_work_list(items, S: int, item_rows: int, block: int) -> int:
    """Status of hilberta_check_work_list for an [n, 10] int32 array of work items (host only)."""
    a = np.ascontiguousarray(items, dtype=np.int32).reshape(-1, 10)
    return int(lib().hilberta_check_work_list(a.ctypes.data, a.shape[0], int(S), int(item_rows), int(block)))


def check_overlap(a: int, b: int, batch: int, heads: int, S: int, stride_b: int, stride_h: int, stride_s: int,
                  row_bytes: int) -> bool:
    """hilberta_check_overlap: do two [batch, heads, S, row] tensors with these byte strides share a byte? (host only)"""
    return bool(lib().hilberta_check_overlap(int(a), int(b), int(batch), int(heads), int(S), int(stride_b),
                                             int(stride_h), int(stride_s), int(row_bytes)))


def schedule_units(cost, cost_two_heads, bh: int, n_cta: int):
    """hilberta_schedule_units (host only): (units [n, 3] int32, cta_begin [n_cta + 1] int32, largest load)."""
    c1 = np.ascontiguousarray(cost, dtype=np.int64)
    c2 = None if cost_two_heads is None else np.ascontiguousarray(cost_two_heads, dtype=np.int64)
    units = np.full((max(len(c1) * int(bh), 1), 3), -7, dtype=np.int32)
    begin = np.zeros(int(n_cta) + 1, dtype=np.int32)
    load = ctypes.c_int64(0)
    _check(lib().hilberta_schedule_units(len(c1), c1.ctypes.data, None if c2 is None else c2.ctypes.data, int(bh), int(n_cta),
                                         units.ctypes.data, begin.ctypes.data, ctypes.addressof(load)), "hilberta_schedule_units")
    return units[:begin[-1]], begin, int(load.value)


def _check(status: int, where: str):
    if status != OK:
        raise HilbertaError(status, where)


def _dtype_code(t) -> int:
    import torch
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float32:
        return FP32
    if t.dtype == torch.float8_e4m3fn:
        return FP8_E4M3
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream_ptr(stream) -> int:
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


_EXPORT_NP = {
    EXPORT_HIL_D2T: (np.int32, None), EXPORT_HIL_T2D: (np.int32, None),
    EXPORT_PHYS2ORIG: (np.int32, None), EXPORT_ORIG2PHYS: (np.int32, None),
    EXPORT_SHARED_RUNS: (np.int32, 2), EXPORT_WINDOWS: (np.int32, 5),
    EXPORT_NNZ: (np.uint64, None), EXPORT_INFO: (np.int32, None), EXPORT_LAUNCH_CLOCK: (np.int32, None),
}


class Plan:
    """Owner of a hilberta_plan_t*.  Methods mirror the C entry points."""

    def __init__(self, H, W, tile, layer_offset, shared_region, n_text, groups=0, frames=1, shared_frames=0):
        """tile > 0: hilberta_plan; groups > 0 (tile ignored): hilberta_plan_groups;
        frames > 1: hilberta_plan_video (a frames x H x W volume)."""
        self._h = ctypes.c_void_p()
        if frames > 1:
            _check(lib().hilberta_plan_video(int(frames), int(H), int(W), int(tile), int(layer_offset),
                                             int(shared_region), int(shared_frames), int(n_text),
                                             ctypes.byref(self._h)), "hilberta_plan_video")
        elif groups:
            _check(lib().hilberta_plan_groups(int(H), int(W), int(groups), int(layer_offset), int(shared_region),
                                              int(n_text), ctypes.byref(self._h)), "hilberta_plan_groups")
        else:
            _check(lib().hilberta_plan(int(H), int(W), int(tile), int(layer_offset), int(shared_region),
                                       int(n_text), ctypes.byref(self._h)), "hilberta_plan")
        self.H, self.W, self.tile, self.n_text = int(H), int(W), int(tile), int(n_text)
        self.S = int(n_text) + int(frames) * int(H) * int(W)
        self._bound = None

    @property
    def handle(self) -> int:
        return self._h.value

    def destroy(self):
        if self._h is not None and self._h.value:
            lib().hilberta_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def export(self, what: int) -> np.ndarray:
        need = ctypes.c_size_t()
        _check(lib().hilberta_plan_export(self._h, what, None, 0, ctypes.byref(need)), "hilberta_plan_export")
        dt, cols = _EXPORT_NP[what]
        buf = np.empty(need.value // np.dtype(dt).itemsize, dtype=dt)
        _check(lib().hilberta_plan_export(self._h, what, buf.ctypes.data, buf.nbytes, None),
               "hilberta_plan_export")
        return buf.reshape(-1, cols) if cols else buf

    def bind(self, batch, heads, head_dim, dtype, strides=(0, 0, 0), scale=0.0):
        _check(lib().hilberta_plan_bind(self._h, int(batch), int(heads), int(head_dim), int(dtype),
                                        int(strides[0]), int(strides[1]), int(strides[2]), float(scale)),
               "hilberta_plan_bind")
        self._bound = (int(batch), int(heads), int(head_dim), int(dtype), tuple(int(s) for s in strides))

    def bind_like(self, t, scale=0.0):
        """Bind to the shape and strides of a [B, heads, S, D] tensor."""
        B, Hh, S, D = t.shape
        if S != self.S or t.stride(3) != 1:
            raise ValueError("tensor does not match the plan")
        strides = (t.stride(0), t.stride(1), t.stride(2))
        if t.is_contiguous():
            strides = (0, 0, 0)
        self.bind(B, Hh, D, _dtype_code(t), strides, scale)

    def forward(self, q, k, v, out, stream=None):
        _check(lib().hilberta_forward(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), self._h,
                                      _stream_ptr(stream)), "hilberta_forward")
        return out

    def forward_unpermute(self, q, k, v, out, stream=None):
        """Forward whose output lands in ORIGINAL token order (exit gather fused in)."""
        _check(lib().hilberta_forward_unpermute(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                                self._h, _stream_ptr(stream)), "hilberta_forward_unpermute")
        return out

    def forward_fused(self, q, k, v, out, in_original=True, out_original=True, stream=None):
        """Forward with the entry gather (q, k, v in ORIGINAL order) and / or the exit gather fused in."""
        _check(lib().hilberta_forward_fused(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), self._h,
                                            int(bool(in_original)), int(bool(out_original)), _stream_ptr(stream)),
               "hilberta_forward_fused")
        return out

    def forward_lse(self, q, k, v, out, lse, stream=None):
        """Forward that also writes the per-row log-sum-exp (fp32 [B, heads, S], physical order)."""
        _check(lib().hilberta_forward_lse(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                          lse.data_ptr(), self._h, _stream_ptr(stream)), "hilberta_forward_lse")
        return out, lse

    def backward(self, dout, q, k, v, out, lse, dq, dk, dv, stream=None):
        """dq, dk, dv from dout and the forward's inputs, output and lse (all physical order, bf16)."""
        _check(lib().hilberta_backward(dout.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                                       lse.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), self._h,
                                       _stream_ptr(stream)), "hilberta_backward")
        return dq, dk, dv

    def backward_static(self, dout, q, k, v, out, lse, dq, dk, dv, stream=None):
        """backward() with the scratch in the library's fixed array: no allocation in the call."""
        _check(lib().hilberta_backward_static(dout.data_ptr(), q.data_ptr(), k.data_ptr(), v.data_ptr(),
                                              out.data_ptr(), lse.data_ptr(), dq.data_ptr(), dk.data_ptr(),
                                              dv.data_ptr(), self._h, _stream_ptr(stream)),
               "hilberta_backward_static")
        return dq, dk, dv

    def forward_host(self, q, k, v, out, stream=None):
        """q, k, v, out: HOST tensors (pinned for asynchronous copies), original order."""
        for t in (q, k, v, out):
            if t.is_cuda or not t.is_contiguous():
                raise ValueError("forward_host wants contiguous host tensors")
        _check(lib().hilberta_forward_host(q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), self._h,
                                           _stream_ptr(stream)), "hilberta_forward_host")
        return out

    def _gather(self, fn, name, src, dst, stream):
        if src.shape != dst.shape or src.dtype != dst.dtype:
            raise ValueError("src and dst must match")
        if not (src.is_contiguous() and dst.is_contiguous()):
            raise ValueError("contiguous tensors only")
        if src.dim() < 2 or src.shape[-2] != self.S:
            raise ValueError("expected [..., S, row_elems]")
        batch = 1
        for s in src.shape[:-2]:
            batch *= int(s)
        _check(fn(src.data_ptr(), dst.data_ptr(), self._h, batch, int(src.shape[-1]), _dtype_code(src),
                  _stream_ptr(stream)), name)
        return dst

    def permute(self, src, dst, stream=None):
        return self._gather(lib().hilberta_permute, "hilberta_permute", src, dst, stream)

    def unpermute(self, src, dst, stream=None):
        return self._gather(lib().hilberta_unpermute, "hilberta_unpermute", src, dst, stream)

    def status(self) -> int:
        return int(lib().hilberta_plan_status(self._h))


def hilberta_plan(H, W, tile, layer_offset, shared_region, n_text) -> Plan:
    return Plan(H, W, tile, layer_offset, shared_region, n_text)


def hilberta_forward(q, k, v, out, plan: Plan, stream=None):
    return plan.forward(q, k, v, out, stream)


def hilberta_permute(src, dst, plan: Plan, stream=None):
    return plan.permute(src, dst, stream)


def hilberta_unpermute(src, dst, plan: Plan, stream=None):
    return plan.unpermute(src, dst, stream)


def launch_count() -> int:
    return int(lib().hilberta_launch_count())


def version() -> int:
    return int(lib().hilberta_version())
