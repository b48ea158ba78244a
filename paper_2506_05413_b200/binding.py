"""Thin Python binding over libsmoothrot.so (ctypes).

Argument marshalling only: every function checks the tensors it is handed,
passes raw device pointers, sizes and the current CUDA stream to the C entry
point of the same name, and raises on a non-zero status.  No arithmetic of the
method happens here, and there is no fallback: if the library is missing or a
tensor is not on a CUDA device the call fails.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsmoothrot.so")

_i64, _f32, _int, _vp, _sz = ctypes.c_int64, ctypes.c_float, ctypes.c_int, ctypes.c_void_p, ctypes.c_size_t

# name -> (restype, argtypes); mirrors include/smoothrot.h
SIGNATURES = {
    "smoothrot_status_string": (ctypes.c_char_p, [_int]),
    "smoothrot_calibrate": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _i64, _f32, _int, _vp, _vp, _vp, _vp, _vp, _vp]),
    "smoothrot_fuse_weights": (_int, [_vp, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _vp]),
    "smoothrot_fuse_weights_search_workspace_bytes": (_sz, [_i64, _i64]),
    "smoothrot_fuse_weights_search": (_int, [_vp, _i64, _i64, _i64, _vp, _f32, _int, _vp, _vp, _vp, _vp, _sz, _vp]),
    "smoothrot_quant_act": (_int, [_vp, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _vp]),
    "smoothrot_quant_act_glu": (_int, [_vp, _vp, _i64, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _vp]),
    "smoothrot_quant_act_heads": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _vp]),
    "smoothrot_quant_act_plain": (_int, [_vp, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _vp]),
    "smoothrot_kv_quant": (_int, [_vp, _i64, _i64, _i64, _f32, _vp, _vp, _vp, _vp]),
    "smoothrot_kv_dequant": (_int, [_vp, _vp, _vp, _i64, _i64, _vp, _i64, _vp]),
    "smoothrot_linear": (_int, [_vp, _vp, _i64, _vp, _vp, _i64, _i64, _vp, _i64, _vp, _sz, _vp]),
    "smoothrot_linear_static_scratch": (_int, [_vp, _vp, _i64, _vp, _vp, _i64, _i64, _vp, _i64, _vp]),
    "smoothrot_linear_decode_heads": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _f32, _vp, _vp, _i64, _vp, _i64, _vp, _vp, _vp]),
    "smoothrot_linear_decode": (_int, [_vp, _i64, _i64, _i64, _int, _vp, _f32, _vp, _vp, _i64, _vp, _i64, _vp, _vp, _vp]),
    "smoothrot_workspace_bytes": (_sz, [_i64, _i64, _i64]),
    "smoothrot_linear_plan_name": (ctypes.c_char_p, [_i64, _i64, _i64]),
    "smoothrot_debug_hadamard": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "smoothrot_debug_hadamard_heads": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _vp]),
    "smoothrot_debug_gemm_i32": (_int, [_vp, _i64, _vp, _i64, _i64, _vp, _vp, _sz, _vp]),
    "smoothrot_debug_set_wait_limit_ns": (_int, [ctypes.c_uint64]),
    "smoothrot_debug_wait_expiry": (_int, [_vp]),
    "smoothrot_paley28": (_int, [_vp]),
    "smoothrot_base_matrix": (_int, [_int, _vp]),
    "smoothrot_device_status": (_int, [ctypes.POINTER(_int), _int]),
    "smoothrot_launch_count": (_i64, []),
}

_lib = None


class SmoothRotError(RuntimeError):
    def __init__(self, status: int, text: str):
        super().__init__(f"libsmoothrot: {text} (status {status})")
        self.status = status


def load() -> ctypes.CDLL:
    """Loads libsmoothrot.so (once) and declares every entry point."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2506_05413_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().smoothrot_status_string(int(status)).decode()


def _check(status: int) -> None:
    if status != 0:
        raise SmoothRotError(status, status_string(status))


def _ptr(t, dtype=None, name="tensor"):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr() if t.numel() > 0 else None


def _rows(t, dtype, name):
    """A 2-D tensor whose rows are contiguous; returns (ptr, rows, cols, leading dim)."""
    if t.dim() != 2 or (t.shape[0] > 1 and t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name} must be 2-D with unit inner stride")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.shape[1], 1)
    return _ptr(t, dtype, name), t.shape[0], t.shape[1], ld


def _vec(t, n, name, dtype=torch.float32):
    if t is None:
        return None
    if t.dim() != 1 or t.shape[0] != n or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous vector of length {n}")
    return _ptr(t, dtype, name)


def _stream():
    return torch.cuda.current_stream().cuda_stream


def calibrate(X, amax, *, W=None, alpha=0.5, s_out=None, d=None, pre_w_out=None, pre_x_out=None):
    """smoothrot_calibrate: folds the batch X [T, K] (or None) into amax [K]; when W [N, K]
    is given, finalizes: writes s_out and, if d is given, pre_w_out = s*d, pre_x_out = d/s."""
    K = amax.shape[0]
    if X is not None:
        xp, T, Kx, ldx = _rows(X, torch.float16, "X")
        if Kx != K:
            raise ValueError("X and amax disagree on K")
    else:
        xp, T, ldx = None, 0, K
    finalize = W is not None
    if finalize:
        wp, N, Kw, ldw = _rows(W, torch.float16, "W")
        if Kw != K:
            raise ValueError("W and amax disagree on K")
        if s_out is None:
            raise ValueError("s_out is required to finalize")
    else:
        wp, N, ldw = None, 0, K
    _check(load().smoothrot_calibrate(xp, T, K, ldx, wp, N, ldw, float(alpha), int(finalize),
                                      _vec(amax, K, "amax"), _vec(s_out, K, "s_out"), _vec(d, K, "d"),
                                      _vec(pre_w_out, K, "pre_w_out"), _vec(pre_x_out, K, "pre_x_out"),
                                      _stream()))


def _quantize(fn, X, pre, clip, q_out, step_out, names):
    xp, R, K, ld = _rows(X, torch.float16, names[0])
    if q_out.dtype != torch.uint8 or tuple(q_out.shape) != (R, K // 2) or not q_out.is_contiguous():
        raise ValueError(f"{names[1]} must be a contiguous uint8 [{R}, {K // 2}] tensor")
    _check(fn(xp, R, K, ld, _vec(pre, K, "pre"), float(clip), _ptr(q_out, torch.uint8, names[1]),
              _vec(step_out, R, names[2]), _stream()))


def fuse_weights(W, pre, clip_w, Wq_out, dw_out):
    """smoothrot_fuse_weights: W [N, K] fp16 -> Wq_out [N, K/2] u8, dw_out [N] f32."""
    _quantize(load().smoothrot_fuse_weights, W, pre, clip_w, Wq_out, dw_out, ("W", "Wq_out", "dw_out"))


def fuse_weights_search(W, pre, lowest_ratio, ratio_count, Wq_out, dw_out, best_out=None, workspace=None):
    """smoothrot_fuse_weights_search: as fuse_weights, with the per-row clip ratio chosen from the grid
    1 .. lowest_ratio (ratio_count values) by least squared error.  best_out [N] int32 is optional;
    workspace (uint8) must hold at least one rotated fp32 row, ideally all N."""
    wp, N, K, ld = _rows(W, torch.float16, "W")
    if Wq_out.dtype != torch.uint8 or tuple(Wq_out.shape) != (N, K // 2) or not Wq_out.is_contiguous():
        raise ValueError(f"Wq_out must be a contiguous uint8 [{N}, {K // 2}] tensor")
    wsp = _ptr(workspace, None, "workspace")
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(load().smoothrot_fuse_weights_search(
        wp, N, K, ld, _vec(pre, K, "pre"), float(lowest_ratio), int(ratio_count),
        _ptr(Wq_out, torch.uint8, "Wq_out"), _vec(dw_out, N, "dw_out"),
        _vec(best_out, N, "best_out", torch.int32), wsp, wsb, _stream()))


def fuse_weights_search_workspace_bytes(N, K) -> int:
    return int(load().smoothrot_fuse_weights_search_workspace_bytes(int(N), int(K)))


def quant_act(X, pre, clip_a, Xq_out, dx_out):
    """smoothrot_quant_act: X [M, K] fp16 -> Xq_out [M, K/2] u8, dx_out [M] f32."""
    _quantize(load().smoothrot_quant_act, X, pre, clip_a, Xq_out, dx_out, ("X", "Xq_out", "dx_out"))


def quant_act_glu(gate, up, pre, clip_a, Xq_out, dx_out):
    """smoothrot_quant_act_glu: SiLU(gate) * up [M, K] (both fp16) -> Xq_out [M, K/2] u8, dx_out [M] f32."""
    gp, R, K, ldg = _rows(gate, torch.float16, "gate")
    up_p, Ru, Ku, ldu = _rows(up, torch.float16, "up")
    if (Ru, Ku) != (R, K):
        raise ValueError("gate and up must have the same shape")
    if Xq_out.dtype != torch.uint8 or tuple(Xq_out.shape) != (R, K // 2) or not Xq_out.is_contiguous():
        raise ValueError(f"Xq_out must be a contiguous uint8 [{R}, {K // 2}] tensor")
    _check(load().smoothrot_quant_act_glu(gp, up_p, R, K, ldg, ldu, _vec(pre, K, "pre"), float(clip_a),
                                          _ptr(Xq_out, torch.uint8, "Xq_out"), _vec(dx_out, R, "dx_out"),
                                          _stream()))


def quant_act_plain(X, pre, clip_a, Xq_out, dx_out):
    """smoothrot_quant_act_plain: X [M, K] fp16, no rotation -> Xq_out [M, K/2] u8, dx_out [M] f32."""
    _quantize(load().smoothrot_quant_act_plain, X, pre, clip_a, Xq_out, dx_out, ("X", "Xq_out", "dx_out"))


def quant_act_heads(X, n_heads, pre, clip_a, Xq_out, dx_out):
    """smoothrot_quant_act_heads: X [M, n_heads * head_dim] fp16, heads mixed by the Walsh-Hadamard matrix,
    -> Xq_out [M, K/2] u8, dx_out [M] f32."""
    xp, R, K, ld = _rows(X, torch.float16, "X")
    if n_heads <= 0 or K % n_heads:
        raise ValueError("the row length must be a multiple of n_heads")
    if Xq_out.dtype != torch.uint8 or tuple(Xq_out.shape) != (R, K // 2) or not Xq_out.is_contiguous():
        raise ValueError(f"Xq_out must be a contiguous uint8 [{R}, {K // 2}] tensor")
    _check(load().smoothrot_quant_act_heads(xp, R, int(n_heads), K // int(n_heads), ld, _vec(pre, K, "pre"),
                                            float(clip_a), _ptr(Xq_out, torch.uint8, "Xq_out"),
                                            _vec(dx_out, R, "dx_out"), _stream()))


KV_GROUP = 128


def kv_quant(X, clip, q_out, step_out, zero_out):
    """smoothrot_kv_quant: X [R, C] fp16 -> q_out [R, C/2] u8, step_out / zero_out [R, C/128] f32."""
    xp, R, C, ld = _rows(X, torch.float16, "X")
    if q_out.dtype != torch.uint8 or tuple(q_out.shape) != (R, C // 2) or not q_out.is_contiguous():
        raise ValueError(f"q_out must be a contiguous uint8 [{R}, {C // 2}] tensor")
    for t, name in ((step_out, "step_out"), (zero_out, "zero_out")):
        if t.dtype != torch.float32 or tuple(t.shape) != (R, C // KV_GROUP) or not t.is_contiguous():
            raise ValueError(f"{name} must be a contiguous float32 [{R}, {C // KV_GROUP}] tensor")
    _check(load().smoothrot_kv_quant(xp, R, C, ld, float(clip), _ptr(q_out, torch.uint8, "q_out"),
                                     _ptr(step_out, torch.float32, "step_out"),
                                     _ptr(zero_out, torch.float32, "zero_out"), _stream()))


def kv_dequant(q, step, zero, Y):
    """smoothrot_kv_dequant: Y [R, C] fp16 = (code - zero) * step."""
    yp, R, C, ld = _rows(Y, torch.float16, "Y")
    if q.dtype != torch.uint8 or tuple(q.shape) != (R, C // 2) or not q.is_contiguous():
        raise ValueError(f"q must be a contiguous uint8 [{R}, {C // 2}] tensor")
    _check(load().smoothrot_kv_dequant(_ptr(q, torch.uint8, "q"), _ptr(step, torch.float32, "step"),
                                       _ptr(zero, torch.float32, "zero"), R, C, yp, ld, _stream()))


def workspace_bytes(M, N, K) -> int:
    return int(load().smoothrot_workspace_bytes(int(M), int(N), int(K)))


def linear_plan_name(M, N, K) -> str:
    """Name of the kernel smoothrot_linear launches for this shape (host call, nothing runs)."""
    return load().smoothrot_linear_plan_name(int(M), int(N), int(K)).decode()


def _packed(t, name):
    if t.dim() != 2 or t.dtype != torch.uint8 or not t.is_contiguous():
        raise ValueError(f"{name} must be a contiguous 2-D uint8 tensor")
    return _ptr(t, torch.uint8, name), t.shape[0], t.shape[1] * 2


def linear(Xq, dx, Wq, dw, Y, workspace=None):
    """smoothrot_linear: Y [M, N] fp16 = dequant(Xq [M, K/2] . Wq [N, K/2]^T)."""
    xp, M, K = _packed(Xq, "Xq")
    wp, N, Kw = _packed(Wq, "Wq")
    if K != Kw:
        raise ValueError("Xq and Wq disagree on K")
    yp, My, Ny, ldy = _rows(Y, torch.float16, "Y")
    if (My, Ny) != (M, N):
        raise ValueError(f"Y must be [{M}, {N}]")
    wsp = _ptr(workspace, None, "workspace")
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(load().smoothrot_linear(xp, _vec(dx, M, "dx"), M, wp, _vec(dw, N, "dw"), N, K, yp, ldy,
                                   wsp, wsb, _stream()))


def linear_decode(X, pre, clip_a, Wq, dw, Y, Xq_out=None, dx_out=None, rotation=True):
    """smoothrot_linear_decode: the online activation path and linear in one kernel, for a few tokens
    (rotation=True: quant_act's path, K = 4096, M <= 4; rotation=False: quant_act_plain's, K <= 4096, M <= 8).
    X [M, K] fp16 -> Y [M, N] fp16; Xq_out [M, K/2] u8 and dx_out [M] f32 optionally receive the codes."""
    xp, M, K, ldx = _rows(X, torch.float16, "X")
    wp, N, Kw = _packed(Wq, "Wq")
    if K != Kw:
        raise ValueError("X and Wq disagree on K")
    yp, My, Ny, ldy = _rows(Y, torch.float16, "Y")
    if (My, Ny) != (M, N):
        raise ValueError(f"Y must be [{M}, {N}]")
    if Xq_out is not None and (Xq_out.dtype != torch.uint8 or tuple(Xq_out.shape) != (M, K // 2)
                               or not Xq_out.is_contiguous()):
        raise ValueError(f"Xq_out must be a contiguous uint8 [{M}, {K // 2}] tensor")
    _check(load().smoothrot_linear_decode(xp, M, K, ldx, 1 if rotation else 0, _vec(pre, K, "pre"), float(clip_a), wp, _vec(dw, N, "dw"), N,
                                          yp, ldy, _ptr(Xq_out, torch.uint8, "Xq_out"), _vec(dx_out, M, "dx_out"),
                                          _stream()))


def linear_decode_heads(X, n_heads, pre, clip_a, Wq, dw, Y, Xq_out=None, dx_out=None):
    """smoothrot_linear_decode_heads: quant_act_heads' path and linear in one kernel (32 heads of 128, M <= 4)."""
    xp, M, K, ldx = _rows(X, torch.float16, "X")
    wp, N, Kw = _packed(Wq, "Wq")
    if K != Kw or n_heads <= 0 or K % n_heads:
        raise ValueError("X, Wq and n_heads disagree on K")
    yp, My, Ny, ldy = _rows(Y, torch.float16, "Y")
    if (My, Ny) != (M, N):
        raise ValueError(f"Y must be [{M}, {N}]")
    if Xq_out is not None and (Xq_out.dtype != torch.uint8 or tuple(Xq_out.shape) != (M, K // 2)
                               or not Xq_out.is_contiguous()):
        raise ValueError(f"Xq_out must be a contiguous uint8 [{M}, {K // 2}] tensor")
    _check(load().smoothrot_linear_decode_heads(xp, M, int(n_heads), K // int(n_heads), ldx, _vec(pre, K, "pre"),
                                                float(clip_a), wp, _vec(dw, N, "dw"), N, yp, ldy,
                                                _ptr(Xq_out, torch.uint8, "Xq_out"), _vec(dx_out, M, "dx_out"),
                                                _stream()))


STATIC_SCRATCH_BYTES = 8 * 1024 * 1024   # SMOOTHROT_STATIC_SCRATCH_BYTES in the header


def linear_static_scratch(Xq, dx, Wq, dw, Y):
    """smoothrot_linear_static_scratch: same result as linear(), for callers that cannot
    hand over a workspace.  The split-K scratch is a fixed array inside the library (one per
    device, shared by all calls: do not let two calls overlap on the GPU).  Shapes that need
    more than STATIC_SCRATCH_BYTES raise SmoothRotError (status -7).  Allocates nothing."""
    xp, M, K = _packed(Xq, "Xq")
    wp, N, Kw = _packed(Wq, "Wq")
    if K != Kw:
        raise ValueError("Xq and Wq disagree on K")
    yp, My, Ny, ldy = _rows(Y, torch.float16, "Y")
    if (My, Ny) != (M, N):
        raise ValueError(f"Y must be [{M}, {N}]")
    _check(load().smoothrot_linear_static_scratch(xp, _vec(dx, M, "dx"), M, wp, _vec(dw, N, "dw"), N, K,
                                                  yp, ldy, _stream()))


def debug_hadamard(X, pre, Y):
    """smoothrot_debug_hadamard: Y [M, K] f32 = (X * pre) H / sqrt(K)."""
    xp, M, K, ld = _rows(X, torch.float16, "X")
    if Y.dtype != torch.float32 or tuple(Y.shape) != (M, K) or not Y.is_contiguous():
        raise ValueError("Y must be a contiguous float32 [M, K] tensor")
    _check(load().smoothrot_debug_hadamard(xp, M, K, ld, _vec(pre, K, "pre"), _ptr(Y, torch.float32, "Y"),
                                           _stream()))


def debug_hadamard_heads(X, n_heads, pre, Y):
    """smoothrot_debug_hadamard_heads: Y [M, K] f32 = (X * pre) (H_heads (x) I) / sqrt(n_heads)."""
    xp, M, K, ld = _rows(X, torch.float16, "X")
    if n_heads <= 0 or K % n_heads:
        raise ValueError("the row length must be a multiple of n_heads")
    if Y.dtype != torch.float32 or tuple(Y.shape) != (M, K) or not Y.is_contiguous():
        raise ValueError("Y must be a contiguous float32 [M, K] tensor")
    _check(load().smoothrot_debug_hadamard_heads(xp, M, int(n_heads), K // int(n_heads), ld, _vec(pre, K, "pre"),
                                                 _ptr(Y, torch.float32, "Y"), _stream()))


def debug_gemm_i32(Xq, Wq, acc, workspace=None):
    """smoothrot_debug_gemm_i32: acc [M, N] int32 = Xq . Wq^T on the codes."""
    xp, M, K = _packed(Xq, "Xq")
    wp, N, Kw = _packed(Wq, "Wq")
    if K != Kw:
        raise ValueError("Xq and Wq disagree on K")
    if acc.dtype != torch.int32 or tuple(acc.shape) != (M, N) or not acc.is_contiguous():
        raise ValueError("acc must be a contiguous int32 [M, N] tensor")
    wsp = _ptr(workspace, None, "workspace")
    wsb = workspace.numel() * workspace.element_size() if workspace is not None else 0
    _check(load().smoothrot_debug_gemm_i32(xp, M, wp, N, K, _ptr(acc, torch.int32, "acc"), wsp, wsb, _stream()))


def paley28():
    """The library's order-28 Paley matrix as a 28 x 28 list of +1/-1 (host call)."""
    buf = (ctypes.c_int8 * 784)()
    _check(load().smoothrot_paley28(ctypes.cast(buf, ctypes.c_void_p)))
    return [[int(buf[r * 28 + c]) for c in range(28)] for r in range(28)]


def base_matrix(order: int):
    """The library's Paley matrix of order 12, 20 or 28 as a list of rows of +1/-1 (host call)."""
    order = int(order)
    buf = (ctypes.c_int8 * (order * order))()
    _check(load().smoothrot_base_matrix(order, ctypes.cast(buf, ctypes.c_void_p)))
    return [[int(buf[r * order + c]) for c in range(order)] for r in range(order)]


def debug_set_wait_limit_ns(ns: int) -> None:
    """Limit of the kernels' bounded waits on the current device (0: back to two seconds)."""
    _check(load().smoothrot_debug_set_wait_limit_ns(int(ns)))


def debug_wait_expiry() -> None:
    """Enqueues the probe whose bounded wait is certain to run out (it returns normally)."""
    _check(load().smoothrot_debug_wait_expiry(_stream()))


def device_status(clear: bool = True) -> int:
    """0, or the code of the first bounded device-side wait that ran out (synchronises)."""
    out = _int(0)
    _check(load().smoothrot_device_status(ctypes.byref(out), int(clear)))
    return int(out.value)


def launch_count() -> int:
    return int(load().smoothrot_launch_count())
