"""The workspace-free backward entry point (wtconv_backward_static), through the C ABI.

It exists for callers that are not allowed to allocate device memory when they call the backward pass (a
runtime with a frozen memory plan, a plug-in that only receives input/output buffers, a latency-critical
loop where cudaMalloc may stall or fail): its scratch is an array built into the library.  The test calls it
twice in a row - the second call finds the first call's leftovers in the shared array - and compares every
gradient with the ordinary entry point's and with the fp64 oracle.  This file is
named so that pytest collects it last: a run that stops at the first failure has then run every other test.
"""
import ctypes

import pytest
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

pytestmark = pytest.mark.gpu


def _tensors(wl, seed_shift=0):
    I = inputs.make_inputs(wl.with_(seed=wl.seed + seed_shift), bias=True)
    tdt = wt.DTYPE_NAMES[wl.dtype]
    dev = lambda a, dt=torch.float32: torch.from_numpy(a).cuda().to(dt).contiguous()
    return I, (dev(I["x"], tdt), dev(I["g"], tdt), dev(I["w0"]), dev(I["s0"]), dev(I["b0"]), dev(I["wl"]), dev(I["sl"]))


def _grads_like(x, w0, s0, b0, wl_, sl):
    return (torch.full_like(x, float("nan")), torch.full_like(w0, float("nan")), torch.full_like(s0, float("nan")),
            torch.full_like(b0, float("nan")), torch.full_like(wl_, float("nan")), torch.full_like(sl, float("nan")))


@pytest.mark.parametrize("wl", [Workload("na_stage1", 8, 6, 56, 56, 5, 3, "f32", 41),      # block-per-plane kernels
                                Workload("na_odd", 3, 5, 7, 7, 5, 2, "bf16", 42),
                                Workload("na_team", 6, 16, 7, 7, 5, 1, "bf16", 43),         # team kernels
                                Workload("na_tiled", 1, 3, 90, 75, 5, 3, "f32", 44)],      # tiled path: Z^l and carriers in the array
                         ids=lambda w: w.name)
def test_static_scratch_backward_matches_workspace_backward_twice(wl):
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt)
    assert wt.wtconv_workspace_bytes(desc)[1] <= wt.STATIC_SCRATCH_BYTES
    tol = 1e-5 if wl.dtype == "f32" else 2e-2
    for call in range(2):  # second call: the shared array still holds the first call's contents
        I, (x, g, w0, s0, b0, wl_, sl) = _tensors(wl, seed_shift=call)
        oracle = O.backward(I["x"], I["g"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
        ref = _grads_like(x, w0, s0, b0, wl_, sl)
        ws = wt.alloc_workspace(desc)
        wt.wtconv_backward(desc, x, g, w0, s0, b0, wl_, sl, *ref, ws)
        got = _grads_like(x, w0, s0, b0, wl_, sl)
        wt.wtconv_backward_static(desc, x, g, w0, s0, b0, wl_, sl, *got)
        torch.cuda.synchronize()
        for name, a, r in zip(("dx", "dw0", "ds0", "db0", "dwl", "dsl"), got, ref):
            a, r = a.double(), r.double()
            assert torch.isfinite(a).all(), name
            err = float((a - r).abs().max() / r.abs().max().clamp_min(1e-30))
            assert err <= tol, (wl.name, call, name, err)
            o = torch.from_numpy(oracle[name]).cuda()
            assert float((a - o).abs().max() / o.abs().max().clamp_min(1e-30)) <= tol, (wl.name, call, name, "vs oracle")
    # the status word of the built-in array is readable too (workspace = None) and clean after these calls
    flag = torch.ones(1, dtype=torch.int32).pin_memory()
    wt.wtconv_read_status(desc, None, flag)
    torch.cuda.synchronize()
    assert int(flag[0]) == 0


def test_static_scratch_rejects_shapes_that_need_more_than_it_holds():
    # large planes take the tiled path, whose scratch is far beyond the built-in array: refused before any launch
    desc = wt.make_desc(16, 256, 256, 256, 5, 5, torch.float16)
    assert wt.wtconv_workspace_bytes(desc)[1] > wt.STATIC_SCRATCH_BYTES
    P = ctypes.c_void_p
    a = P(256)  # never dereferenced: the size check comes first
    code = wt.lib().wtconv_backward_static(ctypes.byref(desc), a, a, a, a, None, a, a, a, a, a, None, a, a, None)
    assert code == 7  # WTCONV_ERR_WORKSPACE
