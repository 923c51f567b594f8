"""ctypes binding of libflurka.so: the same names as include/flurka.h, argument marshalling only.

Every step of the forward pass runs inside the CUDA library.  If the library has not been built
(``python -m paper_2306_15799_b200.build``) loading raises; there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .configs import PERFORMER, RNN

IO_BF16 = 0x000
IO_FP32 = 0x100
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_STAGE1, PATH_TENSOR_STAGE3, PATH_TENSOR_STAGE23 = 0, 1, 2, 3, 4, 5

EXPORTS = [
    "flurka_forward", "flurka_forward_host", "flurka_workspace_bytes", "flurka_set_workspace",
    "flurka_set_path", "flurka_set_cta_limit", "flurka_last_path", "flurka_last_launches", "flurka_debug_copy",
    "flurka_last_status", "flurka_last_cuda_error", "flurka_set_stage_timing", "flurka_last_stage_ms",
    "flurka_strerror", "flurka_version", "flurka_forward_static_scratch", "flurka_static_scratch_need",
    "flurka_measure_ex2_rate", "flurka_forward_fused", "flurka_fused_workspace_bytes",
    "flurka_forward_partial", "flurka_partial_sums", "flurka_forward_finish",
    "flurka_backward", "flurka_backward_workspace_bytes", "flurka_set_stage1_pairs",
]

STATIC_SCRATCH_BYTES = 8 << 20

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libflurka.so")
_lib = None


class FlurkaError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        detail = ""
        if code == -6:
            detail = " (cudaError %d)" % load().flurka_last_cuda_error()
        super().__init__("%s failed: %d %s%s" % (what, code, strerror(code), detail))


def library_path() -> str:
    return _LIB_PATH


def load() -> ctypes.CDLL:
    """Loads libflurka.so and declares the prototypes. Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise FileNotFoundError(
            "%s not found: build it with `python -m paper_2306_15799_b200.build`" % _LIB_PATH)
    lib = ctypes.CDLL(_LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    fwd_args = [vp] * 6 + [ci] * 7 + [vp, vp]
    lib.flurka_forward.restype = ci
    lib.flurka_forward.argtypes = fwd_args
    lib.flurka_forward_host.restype = ci
    lib.flurka_forward_host.argtypes = fwd_args
    lib.flurka_forward_static_scratch.restype = ci
    lib.flurka_forward_static_scratch.argtypes = fwd_args
    lib.flurka_workspace_bytes.restype = sz
    lib.flurka_workspace_bytes.argtypes = [ci] * 7
    lib.flurka_static_scratch_need.restype = sz
    lib.flurka_static_scratch_need.argtypes = [ci] * 7
    lib.flurka_set_workspace.restype = ci
    lib.flurka_set_workspace.argtypes = [vp, sz]
    lib.flurka_set_path.restype = ci
    lib.flurka_set_path.argtypes = [ci]
    lib.flurka_set_cta_limit.restype = ci
    lib.flurka_set_cta_limit.argtypes = [ci]
    lib.flurka_last_path.restype = ci
    lib.flurka_last_launches.restype = ci
    lib.flurka_debug_copy.restype = ci
    lib.flurka_debug_copy.argtypes = [ci, vp, sz, vp]
    lib.flurka_last_status.restype = ci
    lib.flurka_last_cuda_error.restype = ci
    lib.flurka_set_stage_timing.restype = ci
    lib.flurka_set_stage_timing.argtypes = [ci]
    lib.flurka_last_stage_ms.restype = ci
    lib.flurka_last_stage_ms.argtypes = [ctypes.POINTER(ctypes.c_float)]
    lib.flurka_strerror.restype = ctypes.c_char_p
    lib.flurka_strerror.argtypes = [ci]
    lib.flurka_version.restype = ci
    lib.flurka_forward_fused.restype = ci
    lib.flurka_forward_fused.argtypes = [vp] * 9 + [ci] * 8 + [vp, vp]
    lib.flurka_fused_workspace_bytes.restype = sz
    lib.flurka_fused_workspace_bytes.argtypes = [ci] * 8
    lib.flurka_forward_partial.restype = ci
    lib.flurka_forward_partial.argtypes = [vp] * 4 + [ci] * 7 + [vp]
    lib.flurka_forward_finish.restype = ci
    lib.flurka_forward_finish.argtypes = [vp, vp] + [ci] * 7 + [vp, vp]
    lib.flurka_partial_sums.restype = ci
    lib.flurka_partial_sums.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(sz)]
    lib.flurka_backward.restype = ci
    lib.flurka_backward.argtypes = [vp] * 7 + [ci] * 7 + [vp] * 6
    lib.flurka_backward_workspace_bytes.restype = sz
    lib.flurka_backward_workspace_bytes.argtypes = [ci] * 7
    lib.flurka_set_stage1_pairs.restype = ci
    lib.flurka_set_stage1_pairs.argtypes = [ci]
    lib.flurka_measure_ex2_rate.restype = ci
    lib.flurka_measure_ex2_rate.argtypes = [ctypes.POINTER(ctypes.c_double)]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().flurka_strerror(code).decode()


def version() -> int:
    return load().flurka_version()


LAYOUT_BNHD = 0x200   # or-ed into the variant word: Q, K, V, out are [B,N,H,d]
EF_PER_HEAD = 0x400   # or-ed into the variant word: E, F are [H,k,N], one pair per head


def _variant_word(variant: int, dtype: torch.dtype, layout: str = "bhnd", ef_per_head: bool = False) -> int:
    if layout not in ("bhnd", "bnhd"):
        raise ValueError("flurka: layout must be 'bhnd' or 'bnhd'")
    word = variant | (LAYOUT_BNHD if layout == "bnhd" else 0) | (EF_PER_HEAD if ef_per_head else 0)
    if dtype == torch.bfloat16:
        return word | IO_BF16
    if dtype == torch.float32:
        return word | IO_FP32
    raise TypeError("flurka: tensors must be bfloat16 or float32, got %s" % dtype)


def _check(Q, K, V, E, F, W, variant, out, device_type, layout="bhnd"):
    for name, t in (("Q", Q), ("K", K), ("V", V), ("E", E), ("F", F), ("out", out)):
        if t.device.type != device_type:
            raise ValueError("flurka: %s must live on %s" % (name, device_type))
        if not t.is_contiguous():
            raise ValueError("flurka: %s must be contiguous" % name)
        if t.dtype != Q.dtype:
            raise TypeError("flurka: %s has dtype %s, Q has %s" % (name, t.dtype, Q.dtype))
    if Q.dim() != 4 or K.shape != Q.shape or V.shape != Q.shape or out.shape != Q.shape:
        raise ValueError("flurka: Q, K, V, out must all be [B,H,N,d] (or [B,N,H,d] with layout='bnhd')")
    if layout == "bnhd":
        B, N, H, d = Q.shape
    else:
        B, H, N, d = Q.shape
    if F.shape != E.shape or E.shape[-1] != N or not (E.dim() == 2 or (E.dim() == 3 and E.shape[0] == H)):
        raise ValueError("flurka: E, F must be [k,N], or [H,k,N] with one pair per head")
    k = E.shape[-2]
    m = 0
    if variant == PERFORMER:
        if W is None or W.dim() != 2 or W.shape[1] != d or W.dtype != Q.dtype or not W.is_contiguous() \
                or W.device.type != device_type:
            raise ValueError("flurka: W must be a contiguous [m,d] tensor like Q")
        m = W.shape[0]
    return B, H, N, d, k, m


def _stream_ptr(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def flurka_forward(Q, K, V, E, F, W, variant, out=None, stream=None, layout="bhnd"):
    """O = phi(Q)(phi(EK)^T FV) / phi(Q)(phi(EK)^T 1) on device tensors; asynchronous on `stream`.
    layout: 'bhnd' for [B,H,N,d] tensors, 'bnhd' for [B,N,H,d]."""
    if out is None:
        out = torch.empty_like(Q)
    B, H, N, d, k, m = _check(Q, K, V, E, F, W, variant, out, "cuda", layout)
    rc = load().flurka_forward(
        Q.data_ptr(), K.data_ptr(), V.data_ptr(), E.data_ptr(), F.data_ptr(),
        W.data_ptr() if W is not None else None, _variant_word(variant, Q.dtype, layout, E.dim() == 3),
        B, H, N, d, k, m, out.data_ptr(), _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward")
    return out


def flurka_forward_host(Q, K, V, E, F, W, variant, out=None, stream=None, layout="bhnd"):
    """The same on host (ideally pinned) tensors: copies in, computes, copies out, synchronises."""
    if out is None:
        out = torch.empty_like(Q, pin_memory=True)
    B, H, N, d, k, m = _check(Q, K, V, E, F, W, variant, out, "cpu", layout)
    rc = load().flurka_forward_host(
        Q.data_ptr(), K.data_ptr(), V.data_ptr(), E.data_ptr(), F.data_ptr(),
        W.data_ptr() if W is not None else None, _variant_word(variant, Q.dtype, layout, E.dim() == 3),
        B, H, N, d, k, m, out.data_ptr(), _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward_host")
    return out


def flurka_forward_fused(Xq, Xk, Xv, E, F, Wq, Wk, Wv, W, variant, H, out=None, stream=None):
    """Eq. (2) with its linear maps: Xq, Xk, Xv [B,N,dm] un-projected, Wq, Wk, Wv [dm,H*d]; out [B,N,H,d]."""
    B, N, dm = Xq.shape
    if Wq.dim() != 2 or Wq.shape[0] != dm or Wq.shape[1] % H:
        raise ValueError("flurka: Wq, Wk, Wv must be [dm, H*d]")
    d = Wq.shape[1] // H
    if out is None:
        out = torch.empty((B, N, H, d), dtype=Xq.dtype, device=Xq.device)
    for name, t in (("Xq", Xq), ("Xk", Xk), ("Xv", Xv), ("E", E), ("F", F), ("Wq", Wq), ("Wk", Wk), ("Wv", Wv),
                    ("out", out)):
        if t.device.type != "cuda" or not t.is_contiguous() or t.dtype != Xq.dtype:
            raise ValueError("flurka: %s must be a contiguous CUDA tensor of Xq's dtype" % name)
    if Xk.shape != Xq.shape or Xv.shape != Xq.shape or Wk.shape != Wq.shape or Wv.shape != Wq.shape:
        raise ValueError("flurka: Xq, Xk, Xv must be [B,N,dm] and Wq, Wk, Wv [dm,H*d]")
    if E.dim() != 2 or E.shape[1] != N or F.shape != E.shape or tuple(out.shape) != (B, N, H, d):
        raise ValueError("flurka: E, F must be [k,N] and out [B,N,H,d]")
    k, m = E.shape[0], 0
    if variant == PERFORMER:
        if W is None or W.dim() != 2 or W.shape[1] != d or W.dtype != Xq.dtype or not W.is_contiguous() \
                or W.device.type != "cuda":
            raise ValueError("flurka: W must be a contiguous [m,d] tensor like Xq")
        m = W.shape[0]
    rc = load().flurka_forward_fused(
        Xq.data_ptr(), Xk.data_ptr(), Xv.data_ptr(), E.data_ptr(), F.data_ptr(), Wq.data_ptr(), Wk.data_ptr(),
        Wv.data_ptr(), W.data_ptr() if W is not None else None, _variant_word(variant, Xq.dtype),
        B, H, N, dm, d, k, m, out.data_ptr(), _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward_fused")
    return out


class _DeviceBlock:
    """A block of library-owned device memory, presented through the CUDA array interface."""

    def __init__(self, ptr: int, n_floats: int):
        self.__cuda_array_interface__ = {"shape": (n_floats,), "typestr": "<f4", "data": (ptr, False), "version": 3,
                                         "strides": None}


def flurka_forward_partial(K, V, E, F, variant, m=0, stream=None, layout="bhnd"):
    """First half of a sequence-sharded forward: this shard's part of K' = E K, V' = F V.
    K, V: the shard's positions [B,H,n,d]; E, F: the matching columns [k,n] (dense)."""
    if layout == "bnhd":
        B, N, H, d = K.shape
    else:
        B, H, N, d = K.shape
    for name, t in (("K", K), ("V", V), ("E", E), ("F", F)):
        if t.device.type != "cuda" or not t.is_contiguous() or t.dtype != K.dtype:
            raise ValueError("flurka: %s must be a contiguous CUDA tensor of K's dtype" % name)
    if V.shape != K.shape or F.shape != E.shape or E.shape[-1] != N:
        raise ValueError("flurka: K, V must be alike and E, F [k,n] with n the slice length")
    rc = load().flurka_forward_partial(K.data_ptr(), V.data_ptr(), E.data_ptr(), F.data_ptr(),
                                       _variant_word(variant, K.dtype, layout, E.dim() == 3), B, H, N, d, E.shape[-2], m,
                                       _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward_partial")


def flurka_partial_sums():
    """The fp32 block [2][B*H][k][d] the last flurka_forward_partial left on this device, as a flat CUDA
    tensor that aliases the library's workspace (add it over the shards in place)."""
    ptr, n = ctypes.c_void_p(), ctypes.c_size_t()
    rc = load().flurka_partial_sums(ctypes.byref(ptr), ctypes.byref(n))
    if rc:
        raise FlurkaError(rc, "flurka_partial_sums")
    return torch.as_tensor(_DeviceBlock(ptr.value, n.value // 4), device="cuda")


def flurka_forward_finish(Q, W, variant, k, out=None, stream=None, layout="bhnd"):
    """Second half: key side and query side for this shard's queries on the summed K', V'."""
    if out is None:
        out = torch.empty_like(Q)
    if layout == "bnhd":
        B, N, H, d = Q.shape
    else:
        B, H, N, d = Q.shape
    if Q.device.type != "cuda" or not Q.is_contiguous() or out.shape != Q.shape or out.dtype != Q.dtype \
            or not out.is_contiguous():
        raise ValueError("flurka: Q and out must be contiguous CUDA tensors of one shape and dtype")
    m = 0
    if variant == PERFORMER:
        if W is None or W.dim() != 2 or W.shape[1] != d or W.dtype != Q.dtype or not W.is_contiguous():
            raise ValueError("flurka: W must be a contiguous [m,d] tensor like Q")
        m = W.shape[0]
    rc = load().flurka_forward_finish(Q.data_ptr(), W.data_ptr() if W is not None else None,
                                      _variant_word(variant, Q.dtype, layout), B, H, N, d, k, m, out.data_ptr(),
                                      _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward_finish")
    return out


def flurka_backward(Q, K, V, E, F, W, dO, variant, stream=None, layout="bhnd", out=None):
    """Gradients of the forward's output with respect to Q, K, V, E, F, given dO (device tensors).
    Returns (dQ, dK, dV, dE, dF), shaped and typed like the inputs (`out`: five such tensors to write into)."""
    B, H, N, d, k, m = _check(Q, K, V, E, F, W, variant, dO, "cuda", layout)
    grads = list(out) if out is not None else [torch.empty_like(t) for t in (Q, K, V, E, F)]
    for g, t in zip(grads, (Q, K, V, E, F)):
        if g.shape != t.shape or g.dtype != t.dtype or not g.is_cuda or not g.is_contiguous():
            raise ValueError("flurka_backward: `out` must hold five contiguous device tensors shaped like Q, K, V, E, F")
    rc = load().flurka_backward(
        Q.data_ptr(), K.data_ptr(), V.data_ptr(), E.data_ptr(), F.data_ptr(), W.data_ptr() if W is not None else None,
        dO.data_ptr(), _variant_word(variant, Q.dtype, layout, E.dim() == 3), B, H, N, d, k, m,
        *[g.data_ptr() for g in grads], _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_backward")
    return tuple(grads)


def flurka_backward_workspace_bytes(variant, io_dtype, B, H, N, d, k, m) -> int:
    return int(load().flurka_backward_workspace_bytes(_variant_word(variant, io_dtype), B, H, N, d, k, m))


def flurka_fused_workspace_bytes(variant, io_dtype, B, H, N, dm, d, k, m) -> int:
    return int(load().flurka_fused_workspace_bytes(_variant_word(variant, io_dtype), B, H, N, dm, d, k, m))


def flurka_workspace_bytes(variant, io_dtype, B, H, N, d, k, m) -> int:
    return int(load().flurka_workspace_bytes(_variant_word(variant, io_dtype), B, H, N, d, k, m))


def flurka_static_scratch_need(variant, io_dtype, B, H, N, d, k, m) -> int:
    """Bytes of the built-in scratch array flurka_forward_static_scratch would use (0: invalid arguments)."""
    return int(load().flurka_static_scratch_need(_variant_word(variant, io_dtype), B, H, N, d, k, m))


def flurka_set_workspace(buf) -> None:
    """buf: a uint8 CUDA tensor the caller keeps alive, or None for the library-owned workspace."""
    if buf is None:
        rc = load().flurka_set_workspace(None, 0)
    else:
        rc = load().flurka_set_workspace(buf.data_ptr(), buf.numel() * buf.element_size())
    if rc:
        raise FlurkaError(rc, "flurka_set_workspace")


def flurka_set_path(path: int) -> int:
    return int(load().flurka_set_path(path))


def flurka_set_stage1_pairs(on: bool) -> bool:
    return bool(load().flurka_set_stage1_pairs(1 if on else 0))


def flurka_set_cta_limit(max_ctas: int) -> int:
    return int(load().flurka_set_cta_limit(max_ctas))


def flurka_last_path() -> int:
    return int(load().flurka_last_path())


def flurka_last_launches() -> int:
    return int(load().flurka_last_launches())


def flurka_last_status() -> int:
    return int(load().flurka_last_status())


def flurka_debug_copy(which: int, shape, dtype=torch.float32, stream=None):
    """Returns a fresh CUDA tensor holding intermediate `which` of the last forward (see flurka.h)."""
    dst = torch.empty(shape, dtype=dtype, device="cuda")
    rc = load().flurka_debug_copy(which, dst.data_ptr(), dst.numel() * dst.element_size(), _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_debug_copy")
    return dst


def flurka_set_stage_timing(on: bool) -> None:
    rc = load().flurka_set_stage_timing(1 if on else 0)
    if rc:
        raise FlurkaError(rc, "flurka_set_stage_timing")


def flurka_last_stage_ms():
    """(down-projection, key side, query side) milliseconds of the last forward run with timing on."""
    ms = (ctypes.c_float * 3)()
    rc = load().flurka_last_stage_ms(ms)
    if rc:
        raise FlurkaError(rc, "flurka_last_stage_ms")
    return [float(x) for x in ms]


def flurka_measure_ex2_rate() -> float:
    """1e9 exponentials per second a bare ex2.approx loop reaches on the current GPU (synchronises)."""
    v = ctypes.c_double(0.0)
    rc = load().flurka_measure_ex2_rate(ctypes.byref(v))
    if rc:
        raise FlurkaError(rc, "flurka_measure_ex2_rate")
    return float(v.value)


def flurka_forward_static_scratch(Q, K, V, E, F, W, variant, out, stream=None):
    """flurka_forward without any allocation inside the library: scratch is a fixed device array.

    For callers that may not allocate device memory themselves (all memory owned by a framework
    allocator, latency-critical loops, plug-ins that only receive buffers).  `out` must be passed
    in; problems needing more than STATIC_SCRATCH_BYTES of scratch raise FlurkaError(-9).
    Calls share the array, so do not let two of them overlap on the GPU.
    """
    B, H, N, d, k, m = _check(Q, K, V, E, F, W, variant, out, "cuda")
    rc = load().flurka_forward_static_scratch(
        Q.data_ptr(), K.data_ptr(), V.data_ptr(), E.data_ptr(), F.data_ptr(),
        W.data_ptr() if W is not None else None, _variant_word(variant, Q.dtype, "bhnd", E.dim() == 3),
        B, H, N, d, k, m, out.data_ptr(), _stream_ptr(stream))
    if rc:
        raise FlurkaError(rc, "flurka_forward_static_scratch")
    return out
