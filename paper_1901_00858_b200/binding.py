"""Thin ctypes binding of libhgc.so: argument marshalling only.

Every step of the path runs inside the CUDA library; torch is used for device memory and
streams.  The names mirror the C ABI (include/hgc.h).  If the compiled library is missing
this module raises on first use: there is no CPU or library fallback.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libhgc.so")
DEBUG_LIB_PATH = os.path.join(HERE, "libhgc_debug.so")   # the checked build (-DHGC_DEBUG)

HGC_OK, HGC_INVALID_ARG, HGC_UNSUPPORTED, HGC_BAD_ALIGNMENT, HGC_NO_WORKSPACE, HGC_CUDA_ERROR, \
    HGC_DEVICE_TIMEOUT = range(7)
HGC_PATH_DIRECT, HGC_PATH_DEPTHWISE, HGC_PATH_IGEMM = range(3)
HGC_FLAG_FORCE_DIRECT = 1
HGC_FLAG_X_NHWC = 2
HGC_FLAG_Y_NHWC = 4
HGC_FLAG_CTA_PAIRS = 8
HGC_FLAG_SHARED_TILES = 16
HGC_FLAG_FUSED_LAYOUT = 32
HGC_FLAG_WHOLE_TILES = 64
HGC_FLAG_GATHER_X = 128
PATH_NAMES = {HGC_PATH_DIRECT: "direct", HGC_PATH_DEPTHWISE: "depthwise", HGC_PATH_IGEMM: "igemm"}


class HgcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (hgc_status {status})")


class hgc_dwpw_params(ctypes.Structure):
    _fields_ = [(f, ctypes.c_int32) for f in ("n", "c", "h", "w", "k", "stride", "flags")]


class hgc_conv_params(ctypes.Structure):
    _fields_ = [(f, ctypes.c_int32) for f in (
        "n", "c", "h", "w", "k", "r", "s", "pad_h", "pad_w", "stride_h", "stride_w",
        "dil_h", "dil_w", "group", "flags")]


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libhgc.so (built in-tree by `python -m paper_1901_00858_b200.build`)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_1901_00858_b200.build` "
                "(nvcc, sm_100a). There is no fallback path.")
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i32p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_int32)
        szp = ctypes.POINTER(ctypes.c_size_t)
        L.hgc_conv_desc_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(hgc_conv_params)]
        L.hgc_conv_desc_destroy.argtypes = [vp]
        L.hgc_conv_forward.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int, vp]
        L.hgc_conv_forward_host.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int, vp]
        L.hgc_conv_forward_static.argtypes = [ctypes.POINTER(hgc_conv_params), vp, vp, vp, vp, ctypes.c_int, vp]
        L.hgc_inner_product_desc_create.argtypes = [ctypes.POINTER(ctypes.c_void_p), i32, i32, i32]
        L.hgc_cast_f32_to_f16.argtypes = [vp, vp, ctypes.c_int64, vp, vp]
        L.hgc_batchnorm_workspace_bytes.argtypes = [i32, i32, ctypes.c_int64]
        L.hgc_batchnorm_workspace_bytes.restype = ctypes.c_size_t
        L.hgc_batchnorm_forward.argtypes = [vp, vp, i32, i32, ctypes.c_int64, ctypes.c_float, i32, i32, vp, vp, vp, vp]
        L.hgc_bn_fold.argtypes = [vp, vp, vp, vp, vp, vp, ctypes.c_float, i32, ctypes.c_int64, vp, vp, vp]
        L.hgc_conv_output_dims.argtypes = [vp, i32p, i32p, i32p, i32p]
        L.hgc_conv_path.argtypes = [vp, i32p]
        L.hgc_conv_plan_info.argtypes = [vp, i32p, i32]
        L.hgc_conv_workspace_bytes.argtypes = [vp, szp]
        L.hgc_conv_host_workspace_bytes.argtypes = [vp, szp]
        L.hgc_conv_set_workspace.argtypes = [vp, vp, ctypes.c_size_t]
        L.hgc_conv_set_weights.argtypes = [vp, vp, vp]
        L.hgc_conv_last_device_status.argtypes = [vp, i32p]
        L.hgc_layout_nchw_to_nhwc.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp]
        L.hgc_layout_nhwc_to_nchw.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp]
        L.hgc_weights_repack.argtypes = [vp, vp, i32, i32, i32, i32, i32, i32, vp]
        L.hgc_kernel_launch_count.argtypes = [ctypes.POINTER(ctypes.c_uint64)]
        L.hgc_set_launch_overlap.argtypes = [ctypes.c_int]
        L.hgc_dwpw_desc_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(hgc_dwpw_params)]
        L.hgc_dwpw_set_weights.argtypes = [vp, vp, vp, vp]
        L.hgc_dwpw_forward.argtypes = [vp, vp, vp, vp, vp, vp, vp, ctypes.c_int, ctypes.c_int, vp]
        L.hgc_debug_set_wait_limit_ns.argtypes = [ctypes.c_uint64]
        L.hgc_debug_drop_copies.argtypes = [i32]
        L.hgc_debug_violations.argtypes = [i32p, i32p, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]
        L.hgc_debug_shrink_ranges.argtypes = [ctypes.c_int64]
        L.hgc_status_string.argtypes = [ctypes.c_int]
        L.hgc_status_string.restype = ctypes.c_char_p
        for name in ("hgc_conv_desc_create", "hgc_conv_desc_destroy", "hgc_conv_forward",
                     "hgc_conv_forward_host", "hgc_conv_forward_static", "hgc_conv_output_dims", "hgc_conv_path",
                     "hgc_conv_workspace_bytes", "hgc_conv_host_workspace_bytes", "hgc_conv_plan_info",
                     "hgc_conv_set_workspace", "hgc_conv_set_weights", "hgc_conv_last_device_status",
                     "hgc_layout_nchw_to_nhwc", "hgc_layout_nhwc_to_nchw", "hgc_weights_repack",
                     "hgc_kernel_launch_count", "hgc_inner_product_desc_create", "hgc_cast_f32_to_f16",
                     "hgc_set_launch_overlap", "hgc_batchnorm_forward", "hgc_bn_fold",
                     "hgc_debug_set_wait_limit_ns", "hgc_debug_drop_copies", "hgc_dwpw_desc_create",
                     "hgc_dwpw_set_weights", "hgc_dwpw_forward", "hgc_debug_checked_build", "hgc_debug_violations",
                     "hgc_debug_shrink_ranges"):
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().hgc_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != HGC_OK:
        raise HgcError(status, where)


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array / int / None."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if hasattr(t, "data_ptr"):
        return t.data_ptr()
    return t.ctypes.data


def _stream(stream) -> Optional[int]:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class ConvDesc:
    """Owns an hgc_conv_desc.  Keyword arguments are the fields of hgc_conv_params."""

    def __init__(self, n, c, h, w, k, r, s, pad_h=0, pad_w=0, stride_h=1, stride_w=1, dil_h=1,
                 dil_w=1, group=1, flags=0):
        self.params = hgc_conv_params(n, c, h, w, k, r, s, pad_h, pad_w, stride_h, stride_w,
                                      dil_h, dil_w, group, flags)
        self._h = ctypes.c_void_p()
        self._ws = None
        _check(lib().hgc_conv_desc_create(ctypes.byref(self._h), ctypes.byref(self.params)),
               "hgc_conv_desc_create")

    @classmethod
    def inner_product(cls, n, c, k):
        """hgc_inner_product_desc_create: the fully connected layer x[n][c] . w[k][c]^T + bias as
        the 1x1 convolution on a 1x1 plane; use with conv_forward (x, y may be 2-D tensors)."""
        self = cls.__new__(cls)
        self.params = hgc_conv_params(n, c, 1, 1, k, 1, 1, 0, 0, 1, 1, 1, 1, 1, 0)
        self._h = ctypes.c_void_p()
        self._ws = None
        _check(lib().hgc_inner_product_desc_create(ctypes.byref(self._h), n, c, k), "hgc_inner_product_desc_create")
        return self

    @property
    def handle(self):
        return self._h

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().hgc_conv_desc_destroy(self._h)
            self._h = ctypes.c_void_p()
            self._ws = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def output_dims(self):
        v = [ctypes.c_int32() for _ in range(4)]
        _check(lib().hgc_conv_output_dims(self._h, *[ctypes.byref(t) for t in v]), "hgc_conv_output_dims")
        return tuple(t.value for t in v)

    def path(self) -> int:
        v = ctypes.c_int32()
        _check(lib().hgc_conv_path(self._h, ctypes.byref(v)), "hgc_conv_path")
        return v.value

    def plan_info(self) -> dict:
        v = (ctypes.c_int32 * 19)()
        _check(lib().hgc_conv_plan_info(self._h, v, 19), "hgc_conv_plan_info")
        keys = ("path", "kb", "halo", "tn", "th", "pitch", "ncols", "tiles", "stages", "taps", "x_source",
                "k_slices", "grid", "shared_tiles", "pair", "fused_layout", "row_pairs", "replicas", "y_store")
        return dict(zip(keys, list(v)))

    def workspace_bytes(self) -> int:
        v = ctypes.c_size_t()
        _check(lib().hgc_conv_workspace_bytes(self._h, ctypes.byref(v)), "hgc_conv_workspace_bytes")
        return v.value

    def host_workspace_bytes(self) -> int:
        v = ctypes.c_size_t()
        _check(lib().hgc_conv_host_workspace_bytes(self._h, ctypes.byref(v)), "hgc_conv_host_workspace_bytes")
        return v.value

    def set_workspace(self, buf, nbytes: Optional[int] = None):
        """buf: a torch uint8 CUDA tensor (kept alive by this object) or None."""
        if buf is None:
            _check(lib().hgc_conv_set_workspace(self._h, None, 0), "hgc_conv_set_workspace")
            self._ws = None
            return
        nbytes = buf.numel() * buf.element_size() if nbytes is None else nbytes
        _check(lib().hgc_conv_set_workspace(self._h, _ptr(buf), nbytes), "hgc_conv_set_workspace")
        self._ws = buf

    def ensure_workspace(self, host: bool = False):
        """Allocates (with torch) and attaches a workspace of the needed size, if any."""
        import torch
        need = self.host_workspace_bytes() if host else self.workspace_bytes()
        have = 0 if self._ws is None else self._ws.numel()
        if need > have:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device="cuda"))

    def set_weights(self, w, stream=None):
        _check(lib().hgc_conv_set_weights(self._h, _ptr(w), _stream(stream)), "hgc_conv_set_weights")

    def last_device_status(self) -> int:
        v = ctypes.c_int32()
        _check(lib().hgc_conv_last_device_status(self._h, ctypes.byref(v)), "hgc_conv_last_device_status")
        return v.value


class DwPwDesc(ConvDesc):
    """hgc_dwpw_desc_create: a 3x3 depthwise layer (stride 1 or 2, pad 1) and the 1x1 pointwise layer
    behind it as one kernel; x channels-last.  Shares workspace / status / output_dims / close with
    ConvDesc."""

    def __init__(self, n, c, h, w, k, stride=1, flags=0):
        self.block_params = hgc_dwpw_params(n, c, h, w, k, stride, flags)
        self.params = hgc_conv_params(n, c, h, w, k, 1, 1, 0, 0, 1, 1, 1, 1, 1, flags)
        self._h = ctypes.c_void_p()
        self._ws = None
        _check(lib().hgc_dwpw_desc_create(ctypes.byref(self._h), ctypes.byref(self.block_params)),
               "hgc_dwpw_desc_create")

    def set_weights(self, w_dw, w_pw, stream=None):
        _check(lib().hgc_dwpw_set_weights(self._h, _ptr(w_dw), _ptr(w_pw), _stream(stream)), "hgc_dwpw_set_weights")


def dwpw_forward(desc: DwPwDesc, x, w_dw, bias_dw, w_pw, bias_pw, y, relu_dw: bool, relu_pw: bool, stream=None):
    """hgc_dwpw_forward: x [N,H,W,C] channels-last, w_dw [C,1,3,3], w_pw [K,C,1,1], y [N,K,P,Q] (or
    [N,P,Q,K] with HGC_FLAG_Y_NHWC): CUDA fp16 tensors; biases may be None."""
    _check(lib().hgc_dwpw_forward(desc.handle, _ptr(x), _ptr(w_dw), _ptr(bias_dw), _ptr(w_pw), _ptr(bias_pw), _ptr(y),
                                  int(bool(relu_dw)), int(bool(relu_pw)), _stream(stream)), "hgc_dwpw_forward")


def conv_forward(desc: ConvDesc, x, w, bias, y, relu: bool, stream=None):
    """hgc_conv_forward: x, w, bias (or None), y are CUDA fp16 tensors (or raw addresses)."""
    _check(lib().hgc_conv_forward(desc.handle, _ptr(x), _ptr(w), _ptr(bias), _ptr(y), int(bool(relu)),
                                  _stream(stream)), "hgc_conv_forward")


def conv_forward_host(desc: ConvDesc, x, w, bias, y, relu: bool, stream=None):
    """hgc_conv_forward_host: x, w, bias (or None), y are HOST fp16 buffers (pinned torch
    tensors or numpy arrays); copies are queued on the stream."""
    _check(lib().hgc_conv_forward_host(desc.handle, _ptr(x), _ptr(w), _ptr(bias), _ptr(y),
                                       int(bool(relu)), _stream(stream)), "hgc_conv_forward_host")


def conv_forward_static(params: hgc_conv_params, x, w, bias, y, relu: bool, stream=None):
    """hgc_conv_forward_static: the tensor-core layer with its scratch in the library's own fixed
    device array, for callers that may not allocate device memory.  `params` is an
    hgc_conv_params; x, w, bias (or None), y are CUDA fp16 tensors (or raw addresses)."""
    _check(lib().hgc_conv_forward_static(ctypes.byref(params), _ptr(x), _ptr(w), _ptr(bias), _ptr(y),
                                         int(bool(relu)), _stream(stream)), "hgc_conv_forward_static")


def cast_f32_to_f16(src, dst, count=None, overflow_count=None, stream=None):
    """hgc_cast_f32_to_f16: src float32 -> dst float16 CUDA tensors (round to nearest even);
    overflow_count: a 1-element int64 CUDA tensor that the kernel adds to, or None."""
    n = src.numel() if count is None else count
    _check(lib().hgc_cast_f32_to_f16(_ptr(src), _ptr(dst), n, _ptr(overflow_count), _stream(stream)),
           "hgc_cast_f32_to_f16")


def batchnorm_workspace_bytes(n: int, c: int, hw: int) -> int:
    return int(lib().hgc_batchnorm_workspace_bytes(n, c, hw))


def batchnorm_forward(x, y, eps, mean, var, workspace=None, shift_log2=0, use_stored=False, stream=None):
    """hgc_batchnorm_forward: x, y [N,C,...] float16 CUDA tensors; mean, var float32 [C] CUDA
    tensors (written, or read with use_stored); workspace: a CUDA tensor of at least
    batchnorm_workspace_bytes(...) bytes (not needed with use_stored)."""
    n, c = int(x.shape[0]), int(x.shape[1])
    hw = x.numel() // (n * c)
    _check(lib().hgc_batchnorm_forward(_ptr(x), _ptr(y), n, c, hw, float(eps), int(shift_log2), int(bool(use_stored)),
                                       _ptr(mean), _ptr(var), _ptr(workspace), _stream(stream)),
           "hgc_batchnorm_forward")


def bn_fold(w, bias, mean, var, eps, w_out, b_out, gamma=None, beta=None, stream=None):
    """hgc_bn_fold: stored statistics (float32 [K]) and optional gamma/beta folded into conv
    weights w [K,...] and bias [K] (or None); results in w_out, b_out (float16)."""
    k = int(w.shape[0])
    per_k = w.numel() // k
    _check(lib().hgc_bn_fold(_ptr(w), _ptr(bias), _ptr(mean), _ptr(var), _ptr(gamma), _ptr(beta), float(eps), k,
                             per_k, _ptr(w_out), _ptr(b_out), _stream(stream)), "hgc_bn_fold")


def layout_nchw_to_nhwc(src, dst, n, c, h, w, c_pad, stream=None):
    _check(lib().hgc_layout_nchw_to_nhwc(_ptr(src), _ptr(dst), n, c, h, w, c_pad, _stream(stream)),
           "hgc_layout_nchw_to_nhwc")


def layout_nhwc_to_nchw(src, dst, n, c, h, w, c_pad, stream=None):
    _check(lib().hgc_layout_nhwc_to_nchw(_ptr(src), _ptr(dst), n, c, h, w, c_pad, _stream(stream)),
           "hgc_layout_nhwc_to_nchw")


def weights_repack(src, dst, k, c_per_group, r, s, group, c_pad, stream=None):
    _check(lib().hgc_weights_repack(_ptr(src), _ptr(dst), k, c_per_group, r, s, group, c_pad,
                                    _stream(stream)), "hgc_weights_repack")


def set_launch_overlap(enabled: bool) -> None:
    """hgc_set_launch_overlap: programmatic dependent launch of the library's kernels on/off."""
    _check(lib().hgc_set_launch_overlap(int(bool(enabled))), "hgc_set_launch_overlap")


def debug_set_wait_limit_ns(ns: int) -> None:
    """hgc_debug_set_wait_limit_ns: limit of the device-side waits (0 = the default of 2 s)."""
    _check(lib().hgc_debug_set_wait_limit_ns(int(ns)), "hgc_debug_set_wait_limit_ns")


def debug_drop_copies(index: int) -> None:
    """hgc_debug_drop_copies: the first CTA of later launches never issues its index-th copy (-1: off)."""
    _check(lib().hgc_debug_drop_copies(int(index)), "hgc_debug_drop_copies")


def use_checked_build() -> None:
    """Makes this process load libhgc_debug.so (the -DHGC_DEBUG build) instead of libhgc.so; call it
    before anything else touches the library."""
    global LIB_PATH
    if _lib is not None:
        raise RuntimeError("the library is loaded already")
    LIB_PATH = DEBUG_LIB_PATH


def debug_checked_build() -> bool:
    """hgc_debug_checked_build: True when the loaded library tests its hand-addressed accesses."""
    return bool(lib().hgc_debug_checked_build())


def debug_violations() -> dict:
    """hgc_debug_violations: accesses outside the call's tensors since the last call, and the first
    one's source line, address and size; clears the record (synchronises the device)."""
    count, line = ctypes.c_int32(), ctypes.c_int32()
    addr, nbytes = ctypes.c_uint64(), ctypes.c_uint64()
    _check(lib().hgc_debug_violations(ctypes.byref(count), ctypes.byref(line), ctypes.byref(addr), ctypes.byref(nbytes)),
           "hgc_debug_violations")
    return {"count": count.value, "line": line.value, "addr": addr.value, "bytes": nbytes.value}


def debug_shrink_ranges(nbytes: int) -> None:
    """hgc_debug_shrink_ranges: later calls register their tensors `nbytes` short (test hook; 0 = off)."""
    _check(lib().hgc_debug_shrink_ranges(int(nbytes)), "hgc_debug_shrink_ranges")


def kernel_launch_count() -> int:
    v = ctypes.c_uint64()
    _check(lib().hgc_kernel_launch_count(ctypes.byref(v)), "hgc_kernel_launch_count")
    return v.value
