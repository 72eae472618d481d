"""Shared helpers of the parity tests: run the CUDA library through its C ABI binding and the
fp64 oracle on the same seeded inputs, and compare tensor by tensor.

Every output and the workspace of a guarded run sit between guard bands filled with a byte pattern; outputs are
filled with NaN before the call.  After the call the bands must be intact (nothing was written outside a buffer)
and no NaN may be left (every element was written).  This stands in for a memory checker."""
import numpy as np
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import wtconv as wt

# Tolerances of the benchmark spec: max |gpu - oracle| / max |oracle| per tensor.
TOL = {"f32": 1e-5, "f16": 2e-2, "bf16": 2e-2}
GRAD_NAMES = ("dx", "dw0", "ds0", "db0", "dwl", "dsl")
GUARD = 4096          # bytes of guard band on each side of a guarded buffer
GUARD_BYTE = 0xA5


def to_dev(a, dtype=torch.float32):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to("cuda").to(dtype).contiguous()


class Guarded:
    """A device buffer of `nbytes` between two guard bands; `.view(dtype, shape)` gives the tensor in between."""

    def __init__(self, nbytes, device="cuda"):
        self.nbytes = int(nbytes)
        pad = (-self.nbytes) % 256
        self.raw = torch.full((GUARD + self.nbytes + pad + GUARD,), GUARD_BYTE, dtype=torch.uint8, device=device)
        assert self.raw.data_ptr() % 256 == 0
        self.body = self.raw[GUARD:GUARD + self.nbytes]

    def view(self, dtype, shape):
        return self.body.view(dtype).view(shape)

    def intact(self):
        lo, hi = self.raw[:GUARD], self.raw[GUARD + self.nbytes:]
        return bool((lo == GUARD_BYTE).all()) and bool((hi == GUARD_BYTE).all())


def guarded_like(t, fill=float("nan")):
    g = Guarded(t.numel() * t.element_size(), t.device)
    v = g.view(t.dtype, t.shape)
    v.fill_(fill)
    return g, v


def run_gpu(wl, I, flags=0, guarded=True):
    """Returns (out, grads) as float64 numpy arrays computed by the CUDA library (outputs NaN-filled and guarded)."""
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags)
    x, g = to_dev(I["x"], tdt), to_dev(I["g"], tdt)
    w0, s0, b0 = to_dev(I["w0"]), to_dev(I["s0"]), to_dev(I["b0"])
    wl_, sl = (to_dev(I["wl"]), to_dev(I["sl"])) if wl.L > 0 else (None, None)
    f = lambda t: None if t is None else t.double().cpu().numpy()
    if not guarded:
        out, gr = wt.forward_backward(desc, x, g, w0, s0, b0, wl_, sl)
        torch.cuda.synchronize()
        return f(out), {k: f(v) for k, v in gr.items()}
    bands = []

    def mk(t):
        if t is None:
            return None
        gb, v = guarded_like(t)
        bands.append(gb)
        return v
    out, gx, gw0, gs0, gb0, gwl, gsl = mk(x), mk(x), mk(w0), mk(s0), mk(b0), mk(wl_), mk(sl)
    fb, bb = wt.wtconv_workspace_bytes(desc)
    wsg = Guarded(max(fb, bb, 256))
    bands.append(wsg)
    ws = wsg.body
    ws.fill_(0xFF)  # NaN as floats, -1 as words: a call that depends on what it finds in its workspace shows
    flags_h = torch.zeros(2, dtype=torch.int32).pin_memory()
    wt.wtconv_forward(desc, x, w0, s0, b0, wl_, sl, out, ws)
    wt.wtconv_read_status(desc, ws, flags_h[0:1])
    wt.wtconv_backward(desc, x, g, w0, s0, b0, wl_, sl, gx, gw0, gs0, gb0, gwl, gsl, ws)
    wt.wtconv_read_status(desc, ws, flags_h[1:2])
    torch.cuda.synchronize()
    assert int(flags_h[0]) == 0 and int(flags_h[1]) == 0, "a bounded device-side wait ran out"
    assert all(b.intact() for b in bands), "%s: a guard band was overwritten" % wl.name
    gr = dict(dx=gx, dw0=gw0, ds0=gs0, db0=gb0, dwl=gwl, dsl=gsl)
    for n, t in [("out", out)] + list(gr.items()):
        assert t is None or not bool(torch.isnan(t).any()), "%s: %s has elements the library never wrote" % (wl.name, n)
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
