"""Thin ctypes binding of libwtconv_b200.so (include/wtconv.h).

Argument marshalling only: every step of the operator runs in the CUDA library.  Tensors
are torch CUDA tensors (torch supplies device memory and streams); the functions below pass
their raw pointers through the C ABI.  There is no CPU fallback: if the shared library is
missing or fails to load, importing the symbols raises.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwtconv_b200.so")

F32, F16, BF16 = 0, 1, 2
FLAG_TILED_ONLY = 1
FLAG_TEST_NO_COPY = 2
FLAG_NO_TEAM = 4
FLAG_NO_WINDOW = 64
FLAG_PREFER_WINDOW = 128
FLAG_REFERENCE_CHAIN = 8            # comparator: the layer as separate operators with every intermediate in HBM
FLAG_ABLATE_FUSED_ANALYSIS = 16     # (with FLAG_REFERENCE_CHAIN, forward) butterfly on chip in the level conv kernel
FLAG_ABLATE_COLLAPSED_SYNTHESIS = 32  # (with FLAG_REFERENCE_CHAIN, forward) one closed-form synthesis pass
ARITHMETIC_DTYPE = "f32"  # every kernel multiplies and accumulates in float32, whatever the storage type
_DTYPES = {torch.float32: F32, torch.float16: F16, torch.bfloat16: BF16}
DTYPE_NAMES = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}

EXPORTS = ["wtconv_status_string", "wtconv_level_shape", "wtconv_workspace_bytes", "wtconv_plan_name", "wtconv_plan_describe",
           "wtconv_launch_count", "wtconv_forward", "wtconv_backward", "wtconv_read_status", "wtconv_backward_static",
           "wtconv_step_host_workspace_bytes", "wtconv_step_host"]


class Desc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("C", ctypes.c_int32), ("H", ctypes.c_int32), ("W", ctypes.c_int32),
                ("k", ctypes.c_int32), ("L", ctypes.c_int32), ("dtype", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class WTConvError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("wtconv status %d: %s" % (code, msg))
        self.code = code


_lib = None


def lib():
    """Load the shared library (raises OSError if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OSError("%s not found: build it with `python -m paper_2608_10805_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, sz, i32p = ctypes.c_void_p, ctypes.c_size_t, ctypes.POINTER(ctypes.c_int32)
        dp = ctypes.POINTER(Desc)
        L.wtconv_status_string.restype = ctypes.c_char_p
        L.wtconv_status_string.argtypes = [ctypes.c_int]
        L.wtconv_plan_name.restype = ctypes.c_char_p
        L.wtconv_plan_name.argtypes = [dp]
        L.wtconv_plan_describe.argtypes = [dp, ctypes.c_char_p, sz]
        L.wtconv_level_shape.argtypes = [dp, ctypes.c_int, i32p, i32p]
        L.wtconv_workspace_bytes.argtypes = [dp, ctypes.POINTER(sz), ctypes.POINTER(sz)]
        L.wtconv_launch_count.argtypes = [dp, i32p, i32p]
        L.wtconv_forward.argtypes = [dp] + [vp] * 7 + [vp, sz, vp]
        L.wtconv_backward.argtypes = [dp] + [vp] * 13 + [vp, sz, vp]
        L.wtconv_backward_static.argtypes = [dp] + [vp] * 13 + [vp]
        L.wtconv_read_status.argtypes = [dp, vp, vp, vp]
        L.wtconv_step_host_workspace_bytes.argtypes = [dp, ctypes.POINTER(sz)]
        L.wtconv_step_host.argtypes = [dp] + [vp] * 14 + [vp, sz, vp]
        _lib = L
    return _lib


def _check(code):
    if code != 0:
        raise WTConvError(code, lib().wtconv_status_string(code).decode())


def make_desc(B, C, H, W, k, L, dtype, flags=0):
    if isinstance(dtype, str):
        dtype = DTYPE_NAMES[dtype]
    return Desc(B, C, H, W, k, L, _DTYPES[dtype] if not isinstance(dtype, int) else dtype, flags)


def wtconv_level_shape(desc, level):
    h, w = ctypes.c_int32(), ctypes.c_int32()
    _check(lib().wtconv_level_shape(ctypes.byref(desc), level, ctypes.byref(h), ctypes.byref(w)))
    return h.value, w.value


def wtconv_workspace_bytes(desc):
    f, b = ctypes.c_size_t(), ctypes.c_size_t()
    _check(lib().wtconv_workspace_bytes(ctypes.byref(desc), ctypes.byref(f), ctypes.byref(b)))
    return f.value, b.value


def wtconv_plan_name(desc):
    r = lib().wtconv_plan_name(ctypes.byref(desc))
    return None if r is None else r.decode()


def wtconv_plan_describe(desc):
    buf = ctypes.create_string_buffer(256)
    _check(lib().wtconv_plan_describe(ctypes.byref(desc), buf, 256))
    return buf.value.decode()


def wtconv_launch_count(desc):
    f, b = ctypes.c_int32(), ctypes.c_int32()
    _check(lib().wtconv_launch_count(ctypes.byref(desc), ctypes.byref(f), ctypes.byref(b)))
    return f.value, b.value


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _need_cuda(*ts):
    for t in ts:
        if t is not None and not (t.is_cuda and t.is_contiguous()):
            raise ValueError("expected contiguous CUDA tensors")


def wtconv_forward(desc, x, w0, s0, b0, wl, sl, out, workspace, stream=None):
    """out <- WTConv(x) (Algorithm 1).  All tensors CUDA, contiguous; `workspace` a uint8 CUDA tensor."""
    _need_cuda(x, w0, s0, b0, wl, sl, out, workspace)
    _check(lib().wtconv_forward(ctypes.byref(desc), _ptr(x), _ptr(w0), _ptr(s0), _ptr(b0), _ptr(wl), _ptr(sl),
                                _ptr(out), _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                _stream(stream)))
    return out


def wtconv_backward(desc, x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl,
                    workspace, stream=None):
    _need_cuda(x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl, workspace)
    _check(lib().wtconv_backward(ctypes.byref(desc), _ptr(x), _ptr(grad_out), _ptr(w0), _ptr(s0), _ptr(b0), _ptr(wl),
                                 _ptr(sl), _ptr(grad_x), _ptr(grad_w0), _ptr(grad_s0), _ptr(grad_b0), _ptr(grad_wl),
                                 _ptr(grad_sl), _ptr(workspace), workspace.numel(), _stream(stream)))


def wtconv_read_status(desc, workspace, h_flag, stream=None):
    """Enqueue a copy of the workspace's device status word into the host int32 tensor `h_flag` (pin it).
    `workspace=None` reads the array built into the library (the one wtconv_backward_static uses)."""
    _need_cuda(workspace)
    if h_flag.is_cuda or h_flag.dtype != torch.int32 or h_flag.numel() < 1:
        raise ValueError("h_flag must be a host int32 tensor")
    _check(lib().wtconv_read_status(ctypes.byref(desc), _ptr(workspace), _ptr(h_flag), _stream(stream)))


STATIC_SCRATCH_BYTES = 8 << 20


def wtconv_backward_static(desc, x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl,
                           stream=None):
    """wtconv_backward without a workspace argument, for callers that must not allocate device memory:
    the scratch is an array built into the library (see include/wtconv.h for its limits)."""
    _need_cuda(x, grad_out, w0, s0, b0, wl, sl, grad_x, grad_w0, grad_s0, grad_b0, grad_wl, grad_sl)
    _check(lib().wtconv_backward_static(ctypes.byref(desc), _ptr(x), _ptr(grad_out), _ptr(w0), _ptr(s0), _ptr(b0),
                                        _ptr(wl), _ptr(sl), _ptr(grad_x), _ptr(grad_w0), _ptr(grad_s0), _ptr(grad_b0),
                                        _ptr(grad_wl), _ptr(grad_sl), _stream(stream)))


def wtconv_step_host_workspace_bytes(desc):
    n = ctypes.c_size_t()
    _check(lib().wtconv_step_host_workspace_bytes(ctypes.byref(desc), ctypes.byref(n)))
    return n.value


def wtconv_step_host(desc, h_x, h_g, h_w0, h_s0, h_b0, h_wl, h_sl, h_out, h_gx, h_gw0, h_gs0, h_gb0, h_gwl, h_gsl,
                     workspace, stream=None):
    """Forward+backward from (pinned) HOST tensors; `workspace` is a uint8 CUDA tensor."""
    for t in (h_x, h_g, h_w0, h_s0, h_b0, h_wl, h_sl, h_out, h_gx, h_gw0, h_gs0, h_gb0, h_gwl, h_gsl):
        if t is not None and (t.is_cuda or not t.is_contiguous()):
            raise ValueError("expected contiguous host tensors")
    _need_cuda(workspace)
    _check(lib().wtconv_step_host(ctypes.byref(desc), _ptr(h_x), _ptr(h_g), _ptr(h_w0), _ptr(h_s0), _ptr(h_b0),
                                  _ptr(h_wl), _ptr(h_sl), _ptr(h_out), _ptr(h_gx), _ptr(h_gw0), _ptr(h_gs0),
                                  _ptr(h_gb0), _ptr(h_gwl), _ptr(h_gsl), _ptr(workspace), workspace.numel(),
                                  _stream(stream)))


# ----------------------------------------------------------------------------- convenience
def alloc_workspace(desc, device="cuda"):
    f, b = wtconv_workspace_bytes(desc)
    return torch.empty(max(f, b, 256), dtype=torch.uint8, device=device)


def forward_backward(desc, x, g, w0, s0, b0, wl, sl, workspace=None, stream=None):
    """Allocate outputs, run forward and backward, return (out, grads dict).  Marshalling only."""
    dev = x.device
    ws = workspace if workspace is not None else alloc_workspace(desc, dev)
    out = torch.empty_like(x)
    gx = torch.empty_like(x)
    gw0, gs0 = torch.empty_like(w0), torch.empty_like(s0)
    gb0 = torch.empty_like(b0) if b0 is not None else None
    if desc.L > 0:
        gwl, gsl = torch.empty_like(wl), torch.empty_like(sl)
    else:
        gwl = gsl = None
    flags = torch.zeros(2, dtype=torch.int32).pin_memory()
    wtconv_forward(desc, x, w0, s0, b0, wl, sl, out, ws, stream)
    wtconv_read_status(desc, ws, flags[0:1], stream)
    wtconv_backward(desc, x, g, w0, s0, b0, wl, sl, gx, gw0, gs0, gb0, gwl, gsl, ws, stream)
    wtconv_read_status(desc, ws, flags[1:2], stream)
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    if int(flags[0]) or int(flags[1]):  # a bounded device-side wait ran out: the outputs are not valid
        raise WTConvError(11, lib().wtconv_status_string(11).decode())
    return out, dict(dx=gx, dw0=gw0, ds0=gs0, db0=gb0, dwl=gwl, dsl=gsl)
