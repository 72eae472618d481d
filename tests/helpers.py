"""Shared helpers of the parity tests: run the CUDA library through its C ABI binding and the
fp64 oracle on the same seeded inputs, and compare tensor by tensor."""
import numpy as np
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import wtconv as wt

# Tolerances of the benchmark spec: max |gpu - oracle| / max |oracle| per tensor.
TOL = {"f32": 1e-5, "f16": 2e-2, "bf16": 2e-2}
GRAD_NAMES = ("dx", "dw0", "ds0", "db0", "dwl", "dsl")


def to_dev(a, dtype=torch.float32):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(dtype).contiguous()


def run_gpu(wl, I, flags=0, pad_alloc=True):
    """Returns (out, grads) as float64 numpy arrays computed by the CUDA library."""
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags)
    x, g = to_dev(I["x"], tdt), to_dev(I["g"], tdt)
    w0, s0, b0 = to_dev(I["w0"]), to_dev(I["s0"]), to_dev(I["b0"])
    wl_, sl = (to_dev(I["wl"]), to_dev(I["sl"])) if wl.L > 0 else (None, None)
    out, gr = wt.forward_backward(desc, x, g, w0, s0, b0, wl_, sl)
    torch.cuda.synchronize()
    f = lambda t: None if t is None else t.double().cpu().numpy()
    return f(out), {k: f(v) for k, v in gr.items()}


def run_oracle(wl, I):
    out = O.forward(I["x"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    gr = O.backward(I["x"], I["g"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    return out, gr


def rel_err(a, ref):
    m = np.max(np.abs(ref))
    return float(np.max(np.abs(a - ref)) / (m if m > 0 else 1.0))


def assert_close(wl, got, ref, tol=None, what=""):
    """got/ref = (out, grads). Every tensor is compared on its own against the tolerance."""
    tol = TOL[wl.dtype] if tol is None else tol
    errs = {"out": rel_err(got[0], ref[0])}
    for n in GRAD_NAMES:
        r = ref[1].get(n)
        if r is None or r.size == 0:
            continue
        errs[n] = rel_err(got[1][n], r)
    bad = {k: v for k, v in errs.items() if not (v <= tol)}
    assert not bad, "%s %s: rel err over %g: %s (all: %s)" % (wl.name, what, tol, bad, errs)
    return errs
