"""ctypes binding of the batq C-ABI (include/batq.h, include/batq_debug.h): argument marshalling only.

Every function has the name of the C entry point it calls.  Tensors are
torch tensors used purely as device (or host) buffers; all arithmetic of the
path runs in the library's CUDA kernels.  There is no CPU fallback: loading
fails loudly when the shared library is missing.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

BATQ_OK = 0
SF_ROWMAJOR, SF_MMA = 0, 1
F32, BF16 = 0, 1
STATUS_NAMES = {0: "OK", 1: "ERR_NULL", 2: "ERR_SHAPE", 3: "ERR_ALIGN", 4: "ERR_UNSUPPORTED",
                5: "ERR_WORKSPACE", 6: "ERR_SINGULAR", 7: "ERR_CUDA", 8: "ERR_TIMEOUT"}

_LIB = None
_P, _I64, _I32, _SZ = C.c_void_p, C.c_int64, C.c_int32, C.c_size_t

# name -> (restype, argtypes); must list every symbol include/batq.h and include/batq_debug.h declare
SIGNATURES = {
    "batq_status_string": (C.c_char_p, [C.c_int]),
    "batq_version": (C.c_int, []),
    "batq_transform_create": (C.c_int, [C.POINTER(_P), _I32, _I32, _I32, _P, _I64, _P, _I64, _P, _P]),
    "batq_transform_destroy": (C.c_int, [_P]),
    "batq_transform_set_bf16_intermediates": (C.c_int, [_P, _I32]),
    "batq_sf_bytes": (_SZ, [_I64, _I64, _I32]),
    "batq_quantize_act": (C.c_int, [_P, _P, _I64, _I64, _I64, _P, _P, _I32, _P]),
    "batq_quantize_act_mxfp8": (C.c_int, [_P, _P, _I64, _I64, _I64, _P, _P, _I32, _P]),
    "batq_debug_transform_clip_f32": (C.c_int, [_P, _P, _I64, _I64, _I64, _P, _P]),
    "batq_weight_bytes": (_SZ, [_I64, _I64]),
    "batq_prepare_weight": (C.c_int, [_P, _P, _I64, _I64, _I64, _P, _P, _P, C.POINTER(_P), _P]),
    "batq_weight_destroy": (C.c_int, [_P]),
    "batq_weight_export": (C.c_int, [_P, _P, _P, _P]),
    "batq_weight_import": (C.c_int, [_P, _P, _I64, _I64, _P, C.POINTER(_P), _P]),
    "batq_gemm_mxfp4": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _I64, _P]),
    "batq_gemm_mxfp8_mxfp4": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _I64, _P]),
    "batq_linear_w4a8_workspace_bytes": (_SZ, [_P, _I64]),
    "batq_linear_w4a8": (C.c_int, [_P, _P, _P, _I64, _I64, _P, _I32, _I64, _P, _SZ, _P]),
    "batq_gemm_small_s_scratch_bytes": (_SZ, [_P, _I64]),
    "batq_gemm_mxfp4_small_s": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _I64, _P, _SZ, _P]),
    "batq_debug_force_small_s_splits": (None, [_I32]),
    "batq_debug_force_small_s_path": (None, [_I32]),
    "batq_debug_force_small_s_reduce": (None, [_I32]),
    "batq_debug_force_tile_width": (None, [_I32]),
    "batq_debug_force_prefill_path": (None, [_I32]),
    "batq_debug_force_gemm_kernel": (None, [_I32]),
    "batq_debug_force_quantizer": (None, [_I32]),
    "batq_linear_workspace_bytes": (_SZ, [_P, _I64]),
    "batq_linear_kernel_launches": (C.c_int32, [_P, _P, _I64]),
    "batq_debug_pair_schedule": (C.c_int32, [_I64, _I64, _I64, _I32, _I32, _P, _I32]),
    "batq_debug_wide_schedule": (C.c_int32, [_I64, _I64, _I64, _I32, _I32, _P, _I32]),
    "batq_linear_w4a4": (C.c_int, [_P, _P, _P, _I64, _I64, _P, _I32, _I64, _P, _SZ, _P]),
    "batq_linear_w4a4_host": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _P, _P, _P, _SZ, _P]),
    "batq_linear_w4a4_host_async": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _P, _P, _P, _SZ, _P]),
    "batq_linear_w4a8_host_async": (C.c_int, [_P, _P, _P, _I64, _P, _I32, _P, _P, _P, _SZ, _P]),
    "batq_host_drain": (C.c_int, [_P]),
    "batq_static_workspace_capacity": (_SZ, []),
    "batq_linear_w4a4_noalloc": (C.c_int, [_P, _P, _P, _I64, _I64, _P, _I32, _I64, _P]),
    "batq_last_device_status": (C.c_int, [_P]),
    "batq_debug_wait_timeout": (C.c_int, [_I64, _P]),
    "batq_debug_mma_peak": (C.c_int, [_I32, _I32, _I32, _I32, C.POINTER(C.c_double), _P]),
    "batq_debug_mma_peak_kind": (None, [_I32]),
    "batq_debug_mma_peak_second_width": (None, [_I32]),
    "batq_debug_mma_peak_gemm_loop": (None, [_I32]),
    "batq_debug_mma_peak_sf_column": (None, [_I32]),
    "batq_debug_mma_peak_load_stages": (None, [_I32]),
    "batq_debug_mma_peak_load_sharing": (None, [_I32]),
    "batq_debug_mma_peak_load_from_peer": (None, [_I32]),
    "batq_debug_mma_peak_with_loads": (C.c_int, [_P, _I32, _I32, _I32, _I32, _I32, C.POINTER(C.c_double),
                                                 C.POINTER(C.c_double), _P]),
}


class BatqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: BATQ_{STATUS_NAMES.get(status, status)}")


def lib_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbatq.so")


def load():
    """Loads libbatq.so (built in-tree by build.py); raises if it is missing."""
    global _LIB
    if _LIB is None:
        path = lib_path()
        if not os.path.exists(path):
            raise FileNotFoundError(f"{path} not found: run `python -m paper_2603_16590_b200.build`")
        lib = C.CDLL(path)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype, fn.argtypes = res, args
        _LIB = lib
    return _LIB


def _check(status: int, where: str):
    if status != BATQ_OK:
        raise BatqError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    return int(t)


def _stream():
    return torch.cuda.current_stream().cuda_stream


def _f32(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float32)


class Transform:
    """Owns a batq_transform handle."""

    def __init__(self, n, left, right, clip_lo=None, clip_hi=None, gr=4, gc=8):
        left, right, clip_lo, clip_hi = _f32(left), _f32(right), _f32(clip_lo), _f32(clip_hi)
        self._keep = (left, right, clip_lo, clip_hi)
        h = _P()
        ls = 0 if left.shape[0] == 1 else gr * gr
        rs = 0 if right.shape[0] == 1 else gc * gc
        st = load().batq_transform_create(
            C.byref(h), n, gr, gc, left.ctypes.data, ls, right.ctypes.data, rs,
            None if clip_lo is None else clip_lo.ctypes.data, None if clip_hi is None else clip_hi.ctypes.data)
        _check(st, "batq_transform_create")
        self.handle, self.n = h, n

    def close(self):
        if self.handle:
            load().batq_transform_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def batq_transform_create(n, left, right, clip_lo=None, clip_hi=None, gr=4, gc=8) -> Transform:
    return Transform(n, left, right, clip_lo, clip_hi, gr, gc)


def batq_transform_set_bf16_intermediates(t: Transform, on: bool):
    _check(load().batq_transform_set_bf16_intermediates(t.handle, 1 if on else 0), "batq_transform_set_bf16_intermediates")


def batq_sf_bytes(rows, n, layout) -> int:
    return load().batq_sf_bytes(rows, n, layout)


def batq_weight_bytes(m, n) -> int:
    return load().batq_weight_bytes(m, n)


def batq_quantize_act(t, x, codes, scales, scale_layout=SF_ROWMAJOR, ld=None, s=None, n=None):
    """x: bf16 (or int16 bit-pattern) CUDA tensor [s, n]; codes / scales: uint8 CUDA buffers."""
    s = x.shape[0] if s is None else s
    n = x.shape[1] if n is None else n
    ld = x.stride(0) if ld is None else ld
    st = load().batq_quantize_act(t.handle if t else None, _ptr(x), s, n, ld, _ptr(codes), _ptr(scales),
                                  scale_layout, _stream())
    _check(st, "batq_quantize_act")


def batq_quantize_act_mxfp8(t, x, codes, scales, scale_layout=SF_ROWMAJOR, ld=None, s=None, n=None):
    """As batq_quantize_act with E4M3 codes: codes is a uint8 CUDA buffer of s * n bytes."""
    s = x.shape[0] if s is None else s
    n = x.shape[1] if n is None else n
    ld = x.stride(0) if ld is None else ld
    st = load().batq_quantize_act_mxfp8(t.handle if t else None, _ptr(x), s, n, ld, _ptr(codes), _ptr(scales),
                                        scale_layout, _stream())
    _check(st, "batq_quantize_act_mxfp8")


def batq_debug_transform_clip_f32(t, x, out):
    st = load().batq_debug_transform_clip_f32(t.handle if t else None, _ptr(x), x.shape[0], x.shape[1],
                                              x.stride(0), _ptr(out), _stream())
    _check(st, "batq_debug_transform_clip_f32")


class Weight:
    """Owns a batq_weight handle and the device buffer behind it."""

    def __init__(self, t, w, clip_lo=None, clip_hi=None, stored=None):
        """From a bf16 weight w (offline fusion with the transform t), or from stored = (codes, scales)
        as batq_weight_export wrote them."""
        if stored is not None:
            codes, scales = stored
            m, n = codes.shape[0], codes.shape[1] * 2
            device = codes.device
        else:
            m, n = w.shape
            device = w.device
        self.m, self.n = m, n
        self.buf = torch.empty(batq_weight_bytes(m, n) + 1024, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 1024
        self._base = self.buf.data_ptr() + off
        h = _P()
        if stored is not None:
            st = load().batq_weight_import(_ptr(codes), _ptr(scales), m, n, self._base, C.byref(h), _stream())
            _check(st, "batq_weight_import")
        else:
            st = load().batq_prepare_weight(t.handle if t else None, _ptr(w), m, n, w.stride(0), _ptr(clip_lo),
                                            _ptr(clip_hi), self._base, C.byref(h), _stream())
            _check(st, "batq_prepare_weight")
        self.handle = h

    def close(self):
        if self.handle:
            load().batq_weight_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def batq_prepare_weight(t, w, clip_lo=None, clip_hi=None) -> Weight:
    return Weight(t, w, clip_lo, clip_hi)


def batq_weight_import(codes, scales) -> Weight:
    """A prepared weight from stored row-major codes [m x n/2] and scale bytes [m x n/32] (CUDA uint8)."""
    return Weight(None, None, stored=(codes.contiguous(), scales.contiguous()))


def batq_weight_export(w: Weight):
    codes = torch.empty((w.m, w.n // 2), dtype=torch.uint8, device=w.buf.device)
    scales = torch.empty((w.m, w.n // 32), dtype=torch.uint8, device=w.buf.device)
    _check(load().batq_weight_export(w.handle, _ptr(codes), _ptr(scales), _stream()), "batq_weight_export")
    return codes, scales


def batq_gemm_mxfp4(x_codes, x_scales_mma, w: Weight, s, y, ldy=None):
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_gemm_mxfp4(_ptr(x_codes), _ptr(x_scales_mma), w.handle, s, _ptr(y), dt,
                                y.stride(0) if ldy is None else ldy, _stream())
    _check(st, "batq_gemm_mxfp4")


def batq_gemm_mxfp8_mxfp4(x_codes8, x_scales_mma, w: Weight, s, y, ldy=None):
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_gemm_mxfp8_mxfp4(_ptr(x_codes8), _ptr(x_scales_mma), w.handle, s, _ptr(y), dt,
                                      y.stride(0) if ldy is None else ldy, _stream())
    _check(st, "batq_gemm_mxfp8_mxfp4")


def batq_linear_w4a8_workspace_bytes(w: Weight, s) -> int:
    return load().batq_linear_w4a8_workspace_bytes(w.handle, s)


def batq_linear_w4a8(t, w: Weight, x, y, workspace):
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a8(t.handle if t else None, w.handle, _ptr(x), x.shape[0], x.stride(0), _ptr(y), dt,
                                 y.stride(0), _ptr(workspace), workspace.numel(), _stream())
    _check(st, "batq_linear_w4a8")


def batq_gemm_small_s_scratch_bytes(w: Weight, s) -> int:
    return load().batq_gemm_small_s_scratch_bytes(w.handle, s)


def batq_gemm_mxfp4_small_s(x_codes, x_scales_mma, w: Weight, s, y, scratch, ldy=None):
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_gemm_mxfp4_small_s(_ptr(x_codes), _ptr(x_scales_mma), w.handle, s, _ptr(y), dt,
                                        y.stride(0) if ldy is None else ldy, _ptr(scratch), scratch.numel(), _stream())
    _check(st, "batq_gemm_mxfp4_small_s")


def batq_debug_force_small_s_splits(splits: int):
    load().batq_debug_force_small_s_splits(splits)


def batq_debug_force_small_s_reduce(which: int):
    load().batq_debug_force_small_s_reduce(which)


def batq_debug_force_small_s_path(which: int):
    load().batq_debug_force_small_s_path(which)


def batq_debug_force_prefill_path(which: int):
    load().batq_debug_force_prefill_path(which)


def batq_debug_force_tile_width(bn: int):
    load().batq_debug_force_tile_width(bn)


def batq_debug_force_gemm_kernel(which: int):
    load().batq_debug_force_gemm_kernel(which)


def batq_debug_force_quantizer(which: int):
    load().batq_debug_force_quantizer(which)


def batq_linear_workspace_bytes(w: Weight, s) -> int:
    return load().batq_linear_workspace_bytes(w.handle, s)


def _schedule(fn, s, m, n, sm_count):
    pairs = fn(s, m, n, sm_count, -1, None, 0)
    if pairs < 0:
        raise ValueError("bad shape")
    out = []
    for p in range(pairs):
        cnt = fn(s, m, n, sm_count, p, None, 0)
        buf = (C.c_int32 * (3 * max(cnt, 1)))()
        fn(s, m, n, sm_count, p, buf, cnt)
        out.append([(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(cnt)])
    return out


def batq_debug_pair_schedule(s, m, n, sm_count=148):
    """[[(row block, first feature, width), ...] per CTA pair] of the CTA-pair GEMM (host only)."""
    return _schedule(load().batq_debug_pair_schedule, s, m, n, sm_count)


def batq_debug_wide_schedule(s, m, n, sm_count=148):
    """The same for the wide-tile CTA-pair GEMM (host only)."""
    return _schedule(load().batq_debug_wide_schedule, s, m, n, sm_count)


def batq_linear_kernel_launches(t, w: Weight, s) -> int:
    return load().batq_linear_kernel_launches(t.handle if t is not None else None, w.handle, s)


def aligned_workspace(nbytes, device="cuda"):
    """A uint8 CUDA buffer whose returned view starts on a 1024-byte boundary."""
    buf = torch.empty(nbytes + 1024, dtype=torch.uint8, device=device)
    off = (-buf.data_ptr()) % 1024
    return buf[off:off + nbytes]


def batq_linear_w4a4(t, w: Weight, x, y, workspace):
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a4(t.handle if t else None, w.handle, _ptr(x), x.shape[0], x.stride(0), _ptr(y), dt,
                                 y.stride(0), _ptr(workspace), workspace.numel(), _stream())
    _check(st, "batq_linear_w4a4")


def batq_linear_w4a4_host(t, w: Weight, x_host, y_host, x_stage, y_stage, workspace):
    dt = F32 if y_host.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a4_host(t.handle if t else None, w.handle, _ptr(x_host), x_host.shape[0], _ptr(y_host),
                                      dt, _ptr(x_stage), _ptr(y_stage), _ptr(workspace), workspace.numel(), _stream())
    _check(st, "batq_linear_w4a4_host")


def batq_linear_w4a4_host_async(t, w: Weight, x_host, y_host, x_stage, y_stage, workspace):
    """Enqueues copy-in, layer and copy-out and returns; batq_host_drain() waits for them."""
    dt = F32 if y_host.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a4_host_async(t.handle if t else None, w.handle, _ptr(x_host), x_host.shape[0],
                                            _ptr(y_host), dt, _ptr(x_stage), _ptr(y_stage), _ptr(workspace),
                                            workspace.numel(), _stream())
    _check(st, "batq_linear_w4a4_host_async")


def batq_linear_w4a8_host_async(t, w: Weight, x_host, y_host, x_stage, y_stage, workspace):
    """The W4A8 layer with host buffers, enqueued only; batq_host_drain() waits."""
    dt = F32 if y_host.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a8_host_async(t.handle if t else None, w.handle, _ptr(x_host), x_host.shape[0],
                                            _ptr(y_host), dt, _ptr(x_stage), _ptr(y_stage), _ptr(workspace),
                                            workspace.numel(), _stream())
    _check(st, "batq_linear_w4a8_host_async")


def batq_host_drain():
    _check(load().batq_host_drain(_stream()), "batq_host_drain")


def batq_static_workspace_capacity() -> int:
    return load().batq_static_workspace_capacity()


def batq_linear_w4a4_noalloc(t, w: Weight, x, y):
    """The layer with the library's built-in scratch array instead of a caller
    workspace: for callers that cannot allocate device memory.  Calls on one
    device share that array, so keep them ordered on one stream."""
    dt = F32 if y.dtype == torch.float32 else BF16
    st = load().batq_linear_w4a4_noalloc(t.handle if t else None, w.handle, _ptr(x), x.shape[0], x.stride(0),
                                         _ptr(y), dt, y.stride(0), _stream())
    _check(st, "batq_linear_w4a4_noalloc")


def batq_last_device_status() -> int:
    return load().batq_last_device_status(_stream())


def batq_debug_wait_timeout(limit_ns: int):
    """Launches the one-warp kernel whose bounded wait runs out after limit_ns."""
    _check(load().batq_debug_wait_timeout(limit_ns, _stream()), "batq_debug_wait_timeout")


def batq_debug_mma_peak(pair: bool, bn: int, iters: int, sf_copies: bool = False) -> float:
    """Launches the MMA-only loop on the current stream; returns the flops of the launch."""
    flops = C.c_double(0.0)
    _check(load().batq_debug_mma_peak(1 if pair else 0, bn, iters, 1 if sf_copies else 0, C.byref(flops), _stream()),
           "batq_debug_mma_peak")
    return flops.value


def batq_debug_mma_peak_kind(a8: bool) -> None:
    load().batq_debug_mma_peak_kind(1 if a8 else 0)


def batq_debug_mma_peak_second_width(bn2: int) -> None:
    load().batq_debug_mma_peak_second_width(bn2)


def batq_debug_mma_peak_gemm_loop(on: bool) -> None:
    load().batq_debug_mma_peak_gemm_loop(1 if on else 0)


def batq_debug_mma_peak_sf_column(col: int) -> None:
    load().batq_debug_mma_peak_sf_column(col)


def batq_debug_mma_peak_load_stages(stages: int) -> None:
    load().batq_debug_mma_peak_load_stages(stages)


def batq_debug_mma_peak_load_sharing(ctas: int) -> None:
    load().batq_debug_mma_peak_load_sharing(ctas)


def batq_debug_mma_peak_load_from_peer(on: bool) -> None:
    load().batq_debug_mma_peak_load_from_peer(1 if on else 0)


def batq_debug_mma_peak_with_loads(w, pair: bool, bn: int, iters: int, load_iters: int, store_iters: int = 0):
    """Launches the MMA loop with an unsynchronised TMA load stream (and/or a stream of ordinary
    shared-memory stores) beside it on the current stream; returns (flops, loaded + stored bytes)."""
    flops, nbytes = C.c_double(0.0), C.c_double(0.0)
    _check(load().batq_debug_mma_peak_with_loads(w.handle if w is not None else None, 1 if pair else 0, bn, iters,
                                                 load_iters, store_iters, C.byref(flops),
                                                 C.byref(nbytes), _stream()), "batq_debug_mma_peak_with_loads")
    return flops.value, nbytes.value


def bits_to_cuda_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns (host) -> CUDA bf16 tensor (a copy, no arithmetic)."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
