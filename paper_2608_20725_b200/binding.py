"""Thin ctypes binding of libim2win.so: argument marshalling only.

Every function mirrors the C entry point of the same name (include/im2win.h)
on torch CUDA tensors; all arithmetic runs in the CUDA kernels behind the C
ABI.  Loading fails loudly when the library cannot be built or opened: there
is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

from . import build as _build

F32 = 0
F16 = 1

STATUS_NAMES = {
    0: "IM2WIN_OK", 1: "IM2WIN_ERR_INVALID_ARG", 2: "IM2WIN_ERR_NULL_POINTER", 3: "IM2WIN_ERR_MISALIGNED",
    4: "IM2WIN_ERR_WORKSPACE_TOO_SMALL", 5: "IM2WIN_ERR_UNSUPPORTED", 6: "IM2WIN_ERR_CUDA", 7: "IM2WIN_ERR_TIMEOUT",
}

EXPORTS = (
    "im2win_status_string", "im2win_workspace_size", "im2win_transform", "im2win_conv_f32", "im2win_conv_f16",
    "im2win_check_status", "im2win_layer_workspace_size", "im2win_layer_forward_host",
    "im2win_conv_f32_static", "im2win_pack_filter", "im2win_conv_packed", "im2win_conv_kernel_name", "im2win_nhwc_kernel_name",
    "im2win_nhwc_workspace_size", "im2win_transform_nhwc", "im2win_conv_f16_nhwc", "im2win_pack_filter_nhwc",
    "im2win_conv_packed_nhwc",
)

STATIC_SCRATCH_BYTES = 4 << 20


class Shape(ctypes.Structure):
    _fields_ = [(k, ctypes.c_int32) for k in ("N", "C", "H", "W", "Co", "Kh", "Kw", "stride", "pad")]


NCHW = 0
NHWC = 1


class Epilogue(ctypes.Structure):
    """im2win_epilogue: bias (device pointer or NULL), relu, out_dtype (F32/F16), out_layout (NCHW/NHWC)."""

    _fields_ = [("bias", ctypes.c_void_p), ("relu", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
                ("out_layout", ctypes.c_int32)]


class Im2winError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().im2win_status_string(code).decode()
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({msg})")


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Build (if stale) and load the shared library; raises on failure."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build_library()
    L = ctypes.CDLL(path)
    P = ctypes.POINTER
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
    L.im2win_status_string.argtypes = [ctypes.c_int]
    L.im2win_status_string.restype = ctypes.c_char_p
    L.im2win_workspace_size.argtypes = [P(Shape), ctypes.c_int, P(sz), P(sz), P(i32), P(i32)]
    L.im2win_transform.argtypes = [vp, vp, P(Shape), ctypes.c_int, vp]
    L.im2win_conv_f32.argtypes = [vp, vp, vp, vp, sz, P(Shape), vp]
    L.im2win_conv_f16.argtypes = [vp, vp, vp, vp, sz, P(Shape), vp]
    L.im2win_check_status.argtypes = [vp, vp]
    L.im2win_layer_workspace_size.argtypes = [P(Shape), ctypes.c_int, P(sz)]
    L.im2win_layer_forward_host.argtypes = [vp, vp, vp, vp, sz, P(Shape), ctypes.c_int, vp]
    L.im2win_conv_f32_static.argtypes = [vp, vp, vp, P(Shape), vp]
    L.im2win_pack_filter.argtypes = [vp, vp, sz, P(Shape), ctypes.c_int, vp]
    L.im2win_conv_packed.argtypes = [vp, vp, vp, sz, P(Shape), ctypes.c_int, vp]
    L.im2win_conv_kernel_name.argtypes = [P(Shape), ctypes.c_int]
    L.im2win_nhwc_workspace_size.argtypes = [P(Shape), P(sz), P(sz), P(i32), P(i32), P(i32)]
    L.im2win_transform_nhwc.argtypes = [vp, ctypes.c_int, vp, P(Shape), vp]
    L.im2win_conv_f16_nhwc.argtypes = [vp, vp, vp, P(Epilogue), vp, sz, P(Shape), vp]
    L.im2win_pack_filter_nhwc.argtypes = [vp, vp, sz, P(Shape), vp]
    L.im2win_conv_packed_nhwc.argtypes = [vp, vp, P(Epilogue), vp, sz, P(Shape), vp]
    for name in EXPORTS[1:]:
        getattr(L, name).restype = ctypes.c_int
    L.im2win_conv_kernel_name.restype = ctypes.c_char_p
    L.im2win_nhwc_kernel_name.argtypes = [P(Shape), P(Epilogue)]
    L.im2win_nhwc_kernel_name.restype = ctypes.c_char_p
    _lib = L
    return L


def make_shape(N, C, H, W, Co, Kh, Kw, stride, pad) -> Shape:
    return Shape(int(N), int(C), int(H), int(W), int(Co), int(Kh), int(Kw), int(stride), int(pad))


def as_shape(shape) -> Shape:
    if isinstance(shape, Shape):
        return shape
    if isinstance(shape, dict):
        return make_shape(**shape)
    if hasattr(shape, "dims"):
        return make_shape(**shape.dims())
    return make_shape(*shape)


def _check(code: int, where: str) -> None:
    if code != 0:
        raise Im2winError(code, where)


def _stream(stream) -> ctypes.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.float32:
        return F32
    if t == torch.float16:
        return F16
    raise TypeError(f"unsupported dtype {t}")


_size_cache: dict = {}


def im2win_workspace_size(shape, dtype: int) -> Tuple[int, int, int, int]:
    """Returns (window_bytes, scratch_bytes, Ho, Wo)."""
    s = as_shape(shape)
    if os.environ.get("IM2WIN_DEBUG"):           # the library's testing-aid switches may change the sizes
        return _workspace_size_uncached(s, dtype)
    key = (s.N, s.C, s.H, s.W, s.Co, s.Kh, s.Kw, s.stride, s.pad, dtype)
    hit = _size_cache.get(key)
    if hit is not None:
        return hit
    out = _workspace_size_uncached(s, dtype)
    _size_cache[key] = out
    return out


def _workspace_size_uncached(s: Shape, dtype: int) -> Tuple[int, int, int, int]:
    wb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    ho, wo = ctypes.c_int32(), ctypes.c_int32()
    _check(lib().im2win_workspace_size(ctypes.byref(s), dtype, ctypes.byref(wb), ctypes.byref(sb),
                                       ctypes.byref(ho), ctypes.byref(wo)), "im2win_workspace_size")
    return wb.value, sb.value, ho.value, wo.value


def im2win_conv_kernel_name(shape, dtype: int) -> str:
    """Name of the convolution kernel the library selects for the layer (for reports and tests)."""
    s = as_shape(shape)
    return lib().im2win_conv_kernel_name(ctypes.byref(s), dtype).decode()


def im2win_nhwc_kernel_name(shape, epilogue: Optional["Epilogue"] = None) -> str:
    """Name of the kernel im2win_conv_f16_nhwc selects for the layer and epilogue (for reports and tests)."""
    s = as_shape(shape)
    return lib().im2win_nhwc_kernel_name(ctypes.byref(s), None if epilogue is None else ctypes.byref(epilogue)).decode()


def im2win_transform(x: torch.Tensor, window: torch.Tensor, shape, stream=None) -> None:
    """x [N,C,H,W] -> window (flat tensor of window_bytes), both CUDA tensors of the same 2/4-byte dtype."""
    s = as_shape(shape)
    assert x.is_cuda and window.is_cuda and x.is_contiguous() and window.is_contiguous()
    assert x.dtype == window.dtype
    code = _dtype_code(x.dtype)
    wb, _, _, _ = im2win_workspace_size(s, code)
    assert x.numel() == s.N * s.C * s.H * s.W and window.numel() * window.element_size() >= wb
    _check(lib().im2win_transform(x.data_ptr(), window.data_ptr(), ctypes.byref(s), code, _stream(stream)),
           "im2win_transform")


def _conv(fn_name: str, dtype: torch.dtype, code: int, window, filt, y, scratch, shape, stream):
    s = as_shape(shape)
    for t in (window, filt, y, scratch):
        assert t.is_cuda and t.is_contiguous()
    assert window.dtype == dtype and filt.dtype == dtype and y.dtype == torch.float32
    wb, sb, ho, wo = im2win_workspace_size(s, code)
    assert window.numel() * window.element_size() >= wb
    assert filt.numel() == s.Co * s.C * s.Kh * s.Kw and y.numel() == s.N * s.Co * ho * wo
    _check(getattr(lib(), fn_name)(window.data_ptr(), filt.data_ptr(), y.data_ptr(), scratch.data_ptr(),
                                   scratch.numel() * scratch.element_size(), ctypes.byref(s), _stream(stream)),
           fn_name)


def im2win_conv_f32(window, filter_oihw, y, scratch, shape, stream=None) -> None:
    _conv("im2win_conv_f32", torch.float32, F32, window, filter_oihw, y, scratch, shape, stream)


def im2win_conv_f16(window, filter_oihw, y, scratch, shape, stream=None) -> None:
    _conv("im2win_conv_f16", torch.float16, F16, window, filter_oihw, y, scratch, shape, stream)


def im2win_conv_f32_static(window, filter_oihw, y, shape, stream=None) -> None:
    """fp32 convolution for callers that cannot allocate device memory: same as im2win_conv_f32
    but the scratch lives in a fixed array inside the library (layers needing more than
    STATIC_SCRATCH_BYTES are rejected).  Calls that may overlap on the GPU must be serialised."""
    s = as_shape(shape)
    for t in (window, filter_oihw, y):
        assert t.is_cuda and t.is_contiguous() and t.dtype == torch.float32
    _check(lib().im2win_conv_f32_static(window.data_ptr(), filter_oihw.data_ptr(), y.data_ptr(),
                                        ctypes.byref(s), _stream(stream)), "im2win_conv_f32_static")


def im2win_pack_filter(filter_oihw, scratch, shape, stream=None) -> None:
    """Packs the filter into `scratch` once (static weights); im2win_conv_packed then reuses it."""
    s = as_shape(shape)
    assert filter_oihw.is_cuda and filter_oihw.is_contiguous() and scratch.is_cuda
    _check(lib().im2win_pack_filter(filter_oihw.data_ptr(), scratch.data_ptr(), scratch.numel() * scratch.element_size(),
                                    ctypes.byref(s), _dtype_code(filter_oihw.dtype), _stream(stream)),
           "im2win_pack_filter")


def im2win_conv_packed(window, y, scratch, shape, stream=None) -> None:
    """Convolution with the filter that im2win_pack_filter left in `scratch` (same shape and dtype)."""
    s = as_shape(shape)
    assert window.is_cuda and window.is_contiguous() and y.is_cuda and y.dtype == torch.float32 and scratch.is_cuda
    _check(lib().im2win_conv_packed(window.data_ptr(), y.data_ptr(), scratch.data_ptr(),
                                    scratch.numel() * scratch.element_size(), ctypes.byref(s),
                                    _dtype_code(window.dtype), _stream(stream)),
           "im2win_conv_packed")


def im2win_check_status(scratch: torch.Tensor, stream=None) -> None:
    """Blocks until the stream is idle; raises if a bounded device wait gave up."""
    _check(lib().im2win_check_status(scratch.data_ptr(), _stream(stream)), "im2win_check_status")


def im2win_layer_workspace_size(shape, dtype: int) -> int:
    s = as_shape(shape)
    n = ctypes.c_size_t()
    _check(lib().im2win_layer_workspace_size(ctypes.byref(s), dtype, ctypes.byref(n)), "im2win_layer_workspace_size")
    return n.value


def im2win_layer_forward_host(x_host: torch.Tensor, filter_host: torch.Tensor, y_host: torch.Tensor,
                              device_workspace: torch.Tensor, shape, stream=None) -> None:
    """Whole layer from (pinned) host tensors; y_host is float32 on the host.  Asynchronous."""
    s = as_shape(shape)
    assert not x_host.is_cuda and not filter_host.is_cuda and not y_host.is_cuda and device_workspace.is_cuda
    assert x_host.is_contiguous() and filter_host.is_contiguous() and y_host.is_contiguous()
    assert x_host.dtype == filter_host.dtype and y_host.dtype == torch.float32
    code = _dtype_code(x_host.dtype)
    _check(lib().im2win_layer_forward_host(x_host.data_ptr(), filter_host.data_ptr(), y_host.data_ptr(),
                                           device_workspace.data_ptr(),
                                           device_workspace.numel() * device_workspace.element_size(),
                                           ctypes.byref(s), code, _stream(stream)),
           "im2win_layer_forward_host")


# ------------------------------------------------------- channel-innermost (NHWC) form
def make_epilogue(bias: Optional[torch.Tensor] = None, relu: bool = False, out_dtype: torch.dtype = torch.float32,
                  out_layout: int = NCHW) -> Epilogue:
    if bias is not None:
        assert bias.is_cuda and bias.dtype == torch.float32 and bias.is_contiguous()
    return Epilogue(None if bias is None else bias.data_ptr(), int(bool(relu)), _dtype_code(out_dtype), int(out_layout))


def im2win_nhwc_workspace_size(shape) -> Tuple[int, int, int, int, int]:
    """Returns (window_bytes, scratch_bytes, Ho, Wo, Cp) of the NHWC form."""
    s = as_shape(shape)
    wb, sb = ctypes.c_size_t(), ctypes.c_size_t()
    ho, wo, cp = ctypes.c_int32(), ctypes.c_int32(), ctypes.c_int32()
    _check(lib().im2win_nhwc_workspace_size(ctypes.byref(s), ctypes.byref(wb), ctypes.byref(sb), ctypes.byref(ho),
                                            ctypes.byref(wo), ctypes.byref(cp)), "im2win_nhwc_workspace_size")
    return wb.value, sb.value, ho.value, wo.value, cp.value


def im2win_transform_nhwc(x: torch.Tensor, x_layout: int, window: torch.Tensor, shape, stream=None) -> None:
    """x (float16, [N,C,H,W] for NCHW or [N,H,W,C] for NHWC) -> NHWC window tensor (flat float16)."""
    s = as_shape(shape)
    assert x.is_cuda and window.is_cuda and x.is_contiguous() and window.is_contiguous()
    assert x.dtype == torch.float16 and window.dtype == torch.float16
    wb = im2win_nhwc_workspace_size(s)[0]
    assert x.numel() == s.N * s.C * s.H * s.W and window.numel() * 2 >= wb
    _check(lib().im2win_transform_nhwc(x.data_ptr(), int(x_layout), window.data_ptr(), ctypes.byref(s), _stream(stream)),
           "im2win_transform_nhwc")


def _epi_ref(epilogue: Optional[Epilogue]):
    return None if epilogue is None else ctypes.byref(epilogue)


def im2win_conv_f16_nhwc(window, filter_oihw, y, scratch, shape, epilogue: Optional[Epilogue] = None, stream=None) -> None:
    s = as_shape(shape)
    for t in (window, filter_oihw, y, scratch):
        assert t.is_cuda and t.is_contiguous()
    assert window.dtype == torch.float16 and filter_oihw.dtype == torch.float16
    want = torch.float32 if epilogue is None or epilogue.out_dtype == F32 else torch.float16
    assert y.dtype == want
    _check(lib().im2win_conv_f16_nhwc(window.data_ptr(), filter_oihw.data_ptr(), y.data_ptr(), _epi_ref(epilogue),
                                      scratch.data_ptr(), scratch.numel() * scratch.element_size(), ctypes.byref(s),
                                      _stream(stream)), "im2win_conv_f16_nhwc")


def im2win_pack_filter_nhwc(filter_oihw, scratch, shape, stream=None) -> None:
    s = as_shape(shape)
    assert filter_oihw.is_cuda and filter_oihw.is_contiguous() and filter_oihw.dtype == torch.float16 and scratch.is_cuda
    _check(lib().im2win_pack_filter_nhwc(filter_oihw.data_ptr(), scratch.data_ptr(),
                                         scratch.numel() * scratch.element_size(), ctypes.byref(s), _stream(stream)),
           "im2win_pack_filter_nhwc")


def im2win_conv_packed_nhwc(window, y, scratch, shape, epilogue: Optional[Epilogue] = None, stream=None) -> None:
    s = as_shape(shape)
    assert window.is_cuda and window.dtype == torch.float16 and y.is_cuda and scratch.is_cuda
    _check(lib().im2win_conv_packed_nhwc(window.data_ptr(), y.data_ptr(), _epi_ref(epilogue), scratch.data_ptr(),
                                         scratch.numel() * scratch.element_size(), ctypes.byref(s), _stream(stream)),
           "im2win_conv_packed_nhwc")


def alloc_nhwc_buffers(shape, out_dtype: torch.dtype = torch.float32, out_layout: int = NCHW, device="cuda"):
    """Allocates (window, scratch, y) for one layer of the NHWC form with torch (device memory only)."""
    s = as_shape(shape)
    wb, sb, ho, wo, _ = im2win_nhwc_workspace_size(s)
    window = torch.empty(wb // 2, dtype=torch.float16, device=device)
    scratch = torch.empty(sb, dtype=torch.uint8, device=device)
    yshape = (s.N, s.Co, ho, wo) if out_layout == NCHW else (s.N, ho, wo, s.Co)
    y = torch.empty(yshape, dtype=out_dtype, device=device)
    return window, scratch, y


# ---------------------------------------------------------------- conveniences
def alloc_layer_buffers(shape, dtype: torch.dtype, device="cuda"):
    """Allocates (window, scratch, y) for one layer with torch (device memory only)."""
    s = as_shape(shape)
    code = _dtype_code(dtype)
    wb, sb, ho, wo = im2win_workspace_size(s, code)
    esize = 4 if code == F32 else 2
    window = torch.empty(max(wb // esize, 1), dtype=dtype, device=device)
    scratch = torch.empty(sb, dtype=torch.uint8, device=device)
    y = torch.empty((s.N, s.Co, ho, wo), dtype=torch.float32, device=device)
    return window, scratch, y


def conv2d_im2win(x: torch.Tensor, filter_oihw: torch.Tensor, stride: int, pad: int, stream=None) -> torch.Tensor:
    """Transform + convolution through the C ABI for CUDA tensors of float32 or float16; returns y (float32)."""
    N, C, H, W = x.shape
    Co, C2, Kh, Kw = filter_oihw.shape
    assert C == C2
    s = make_shape(N, C, H, W, Co, Kh, Kw, stride, pad)
    window, scratch, y = alloc_layer_buffers(s, x.dtype, x.device)
    x = x.contiguous()
    filter_oihw = filter_oihw.contiguous()
    im2win_transform(x, window, s, stream)
    if x.dtype == torch.float32:
        im2win_conv_f32(window, filter_oihw, y, scratch, s, stream)
    else:
        im2win_conv_f16(window, filter_oihw, y, scratch, s, stream)
    return y
