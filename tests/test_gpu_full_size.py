"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.  The CUDA library
runs on the whole tensor; the fp64 oracle recomputes a sample of channels (every plane of those channels,
so the batch-summed parameter gradients of the sampled channels are complete) and the corresponding slices
are compared element by element.  The small benchmark configuration is compared in full."""
import numpy as np
import pytest
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt

from helpers import TOL, rel_err

pytestmark = pytest.mark.gpu


def _run_full_and_compare(wl, channels):
    I = inputs.make_inputs(wl)
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt)
    dev = lambda a, dt=torch.float32: torch.from_numpy(a).cuda().to(dt).contiguous()
    x, g = dev(I["x"], tdt), dev(I["g"], tdt)
    w0, s0, wl_, sl = dev(I["w0"]), dev(I["s0"]), dev(I["wl"]), dev(I["sl"])
    out, gr = wt.forward_backward(desc, x, g, w0, s0, None, wl_, sl)
    torch.cuda.synchronize()
    ch = list(channels)
    sub = lambda a, axis: np.ascontiguousarray(np.take(a, ch, axis=axis))
    xs, gs = sub(I["x"], 1), sub(I["g"], 1)
    w0s, s0s, wls, sls = sub(I["w0"], 0), sub(I["s0"], 0), sub(I["wl"], 1), sub(I["sl"], 1)
    rout = O.forward(xs, w0s, s0s, None, wls, sls, wl.L)
    rgr = O.backward(xs, gs, w0s, s0s, None, wls, sls, wl.L)
    idx = torch.tensor(ch, device="cuda")
    got = {
        "out": out.index_select(1, idx).double().cpu().numpy(),
        "dx": gr["dx"].index_select(1, idx).double().cpu().numpy(),
        "dw0": gr["dw0"].index_select(0, idx).double().cpu().numpy(),
        "ds0": gr["ds0"].index_select(0, idx).double().cpu().numpy(),
        "dwl": gr["dwl"].index_select(1, idx).double().cpu().numpy(),
        "dsl": gr["dsl"].index_select(1, idx).double().cpu().numpy(),
    }
    ref = dict(out=rout, dx=rgr["dx"], dw0=rgr["dw0"], ds0=rgr["ds0"], dwl=rgr["dwl"], dsl=rgr["dsl"])
    errs = {n: rel_err(got[n], ref[n]) for n in ref}
    tol = TOL[wl.dtype]
    bad = {n: e for n, e in errs.items() if not e <= tol}
    assert not bad, "%s [%s]: %s (all %s)" % (wl.name, wt.wtconv_plan_name(desc), bad, errs)
    # nothing may be left unwritten anywhere in the full tensors
    assert torch.isfinite(out).all() and torch.isfinite(gr["dx"]).all()
    return errs


def test_tiny_config_in_full():
    wl = inputs.WORKLOADS["tiny"]
    _run_full_and_compare(wl, range(wl.C))


def test_stage1_f32_bench_config_in_full():
    wl = inputs.WORKLOADS["stage1_f32"]  # the configuration bench.py times
    _run_full_and_compare(wl, range(wl.C))


@pytest.mark.parametrize("name", ["stage1_bf16", "stage2_bf16", "stage3_bf16", "stage4_bf16"])
def test_wtconvnext_stage_set_bf16(name):
    wl = inputs.WORKLOADS[name]
    _run_full_and_compare(wl, [0, 1, wl.C // 2, wl.C - 2, wl.C - 1])


@pytest.mark.parametrize("name", ["convnext_s1_bf16", "convnext_s2_bf16", "convnext_s3_bf16", "convnext_s4_bf16"])
def test_wtconvnext_depth_schedule_bf16(name):
    wl = inputs.WORKLOADS[name]  # L = (5, 4, 3, 2): grids shrink through odd sizes (7 -> 4 -> 2, 14 -> 7 -> 4 -> 2)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wt.DTYPE_NAMES[wl.dtype])) in ("plane", "team")
    _run_full_and_compare(wl, [0, 1, wl.C // 2, wl.C - 1])


@pytest.mark.parametrize("name", ["stage1_k3_f32", "stage1_k7_f32"])
def test_kernel_size_variants(name):
    wl = inputs.WORKLOADS[name]
    _run_full_and_compare(wl, [0, wl.C // 2, wl.C - 1])


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("L", [1, 2, 3, 4, 5])
def test_level_sweep(L, dtype):
    wl = inputs.WORKLOADS["sweep_L%d_%s" % (L, dtype)]
    _run_full_and_compare(wl, [0, 63, wl.C - 1])


@pytest.mark.parametrize("name", ["large_f16", "large_odd_f16"])
def test_large_planes(name):
    wl = inputs.WORKLOADS[name]
    _run_full_and_compare(wl, [0, wl.C - 1])
