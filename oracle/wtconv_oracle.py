"""ctypes front end of the fp64 CPU oracle (oracle/wtconv_oracle.c).

TEST INFRASTRUCTURE ONLY: the test suite, the smoke check and the benchmark's
CPU-baseline leg are the only callers.  Nothing here imports, or is imported by,
the CUDA package.  All arithmetic is in the C file; this module only marshals
numpy arrays (C-contiguous float64) and compiles the C file on first use.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wtconv_oracle.c")
_LIB = os.path.join(_HERE, "libwtconv_oracle.so")
_lib = None


def build(force=False):
    """Compile the oracle with gcc (no fast-math: fp64 IEEE arithmetic in source order)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        i = ctypes.c_int
        lib.wtoracle_num_threads.restype = i
        lib.wtoracle_level_shape.argtypes = [i, i, i, ctypes.POINTER(i), ctypes.POINTER(i)]
        lib.wtoracle_haar_analysis.argtypes = [dp, i, i, dp]
        lib.wtoracle_haar_synthesis.argtypes = [dp, i, i, dp]
        lib.wtoracle_corr2d_same.argtypes = [dp, i, i, dp, i, dp]
        lib.wtoracle_synthesis_cascade.argtypes = [ctypes.POINTER(dp), i, i, i, dp]
        lib.wtoracle_forward.argtypes = [i] * 6 + [dp] * 7
        lib.wtoracle_backward.argtypes = [i] * 6 + [dp] * 13
        _lib = lib
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _c(a):
    return None if a is None else np.ascontiguousarray(a, dtype=np.float64)


def num_threads():
    return int(_load().wtoracle_num_threads())


def level_shape(H, W, level):
    h, w = ctypes.c_int(), ctypes.c_int()
    _load().wtoracle_level_shape(H, W, level, ctypes.byref(h), ctypes.byref(w))
    return h.value, w.value


def haar_analysis(X):
    """X [H,W] -> Y [4,ceil(H/2),ceil(W/2)] (LL,LH,HL,HH), zero pad bottom/right."""
    X = _c(X)
    H, W = X.shape
    Y = np.empty((4, (H + 1) // 2, (W + 1) // 2))
    _load().wtoracle_haar_analysis(_p(X), H, W, _p(Y))
    return Y


def haar_synthesis(T, H, W):
    """T [4,ceil(H/2),ceil(W/2)] -> [H,W] (cropped)."""
    T = _c(T)
    assert T.shape == (4, (H + 1) // 2, (W + 1) // 2)
    R = np.empty((H, W))
    _load().wtoracle_haar_synthesis(_p(T), H, W, _p(R))
    return R


def corr2d_same(X, w):
    X, w = _c(X), _c(w)
    H, W = X.shape
    k = w.shape[0]
    out = np.empty((H, W))
    _load().wtoracle_corr2d_same(_p(X), H, W, _p(w), k, _p(out))
    return out


def synthesis_cascade(Z, H, W):
    """Z: list of L arrays, Z[l-1] of shape [4,H_l,W_l]. Returns R^1 [H,W] (upward loop of Algorithm 1)."""
    Zc = [_c(z) for z in Z]
    L = len(Zc)
    for l, z in enumerate(Zc, 1):
        assert z.shape == (4,) + level_shape(H, W, l), (z.shape, level_shape(H, W, l))
    arr = (ctypes.POINTER(ctypes.c_double) * max(L, 1))(*[_p(z) for z in Zc])
    R = np.empty((H, W))
    _load().wtoracle_synthesis_cascade(arr, H, W, L, _p(R))
    return R


def _params(C, k, L, w0, s0, b0, wl, sl):
    w0, s0, b0 = _c(w0), _c(s0), _c(b0)
    assert w0.shape == (C, k, k) and s0.shape == (C,)
    assert b0 is None or b0.shape == (C,)
    if L > 0:
        wl, sl = _c(wl), _c(sl)
        assert wl.shape == (L, C, 4, k, k) and sl.shape == (L, C, 4)
    else:
        wl = sl = None
    return w0, s0, b0, wl, sl


def forward(x, w0, s0, b0, wl, sl, L):
    """WTConv forward (Algorithm 1). x [B,C,H,W]; returns out [B,C,H,W] float64."""
    x = _c(x)
    B, C, H, W = x.shape
    k = np.asarray(w0).shape[-1]
    w0, s0, b0, wl, sl = _params(C, k, L, w0, s0, b0, wl, sl)
    out = np.empty_like(x)
    _load().wtoracle_forward(B, C, H, W, k, L, _p(x), _p(w0), _p(s0), _p(b0), _p(wl), _p(sl), _p(out))
    return out


def backward(x, g, w0, s0, b0, wl, sl, L):
    """Gradients of sum(out * g). Returns dict dx, dw0, ds0, db0 (None without bias), dwl, dsl."""
    x, g = _c(x), _c(g)
    B, C, H, W = x.shape
    assert g.shape == x.shape
    k = np.asarray(w0).shape[-1]
    w0, s0, b0, wl, sl = _params(C, k, L, w0, s0, b0, wl, sl)
    dx = np.empty_like(x)
    dw0 = np.empty((C, k, k))
    ds0 = np.empty((C,))
    db0 = np.empty((C,)) if b0 is not None else None
    dwl = np.empty((L, C, 4, k, k))
    dsl = np.empty((L, C, 4))
    _load().wtoracle_backward(B, C, H, W, k, L, _p(x), _p(g), _p(w0), _p(s0), _p(b0), _p(wl), _p(sl),
                              _p(dx), _p(dw0), _p(ds0), _p(db0), _p(dwl), _p(dsl))
    return dict(dx=dx, dw0=dw0, ds0=ds0, db0=db0, dwl=dwl, dsl=dsl)
