"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.  The CUDA library runs
on the whole tensor (outputs NaN-filled and between guard bands); the fp64 oracle recomputes EVERY channel, one
channel group at a time (every plane of those channels, so their batch-summed parameter gradients are complete),
and the corresponding slices are compared element by element.  Only the two 0.2-0.27 G-element shapes are compared
on a sample of channel groups (the oracle would need minutes for all of them)."""
import numpy as np
import pytest
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt

from helpers import TOL, guarded_like, rel_err

pytestmark = pytest.mark.gpu


def _run_full_and_compare(wl, groups=None, group=None, flags=0):
    """groups: iterable of first channels of the channel groups to compare (None = all), group = channels per group."""
    I = inputs.make_inputs(wl)
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags)
    dev = lambda a, dt=torch.float32: torch.from_numpy(a).cuda().to(dt).contiguous()
    x, g = dev(I["x"], tdt), dev(I["g"], tdt)
    w0, s0, wl_, sl = dev(I["w0"]), dev(I["s0"]), dev(I["wl"]), dev(I["sl"])
    bands, outs = [], []
    for t in (x, x, w0, s0, wl_, sl):
        gb, v = guarded_like(t)
        bands.append(gb); outs.append(v)
    out, gx, gw0, gs0, gwl, gsl = outs
    ws = wt.alloc_workspace(desc)
    wt.wtconv_forward(desc, x, w0, s0, None, wl_, sl, out, ws)
    wt.wtconv_backward(desc, x, g, w0, s0, None, wl_, sl, gx, gw0, gs0, None, gwl, gsl, ws)
    torch.cuda.synchronize()
    assert all(b.intact() for b in bands), "a guard band was overwritten"
    for n, t in zip(("out", "dx", "dw0", "ds0", "dwl", "dsl"), outs):  # outputs were NaN before the calls
        assert not bool(torch.isnan(t).any()), "%s has elements the library never wrote" % n
    if group is None:  # bound the oracle's working set: about 8 M elements per chunk
        group = max(1, min(wl.C, (8 << 20) // (wl.B * wl.H * wl.W)))
    firsts = list(range(0, wl.C, group)) if groups is None else list(groups)
    worst = {}
    for c0 in firsts:
        ch = slice(c0, min(wl.C, c0 + group))
        xs, gs = np.ascontiguousarray(I["x"][:, ch]), np.ascontiguousarray(I["g"][:, ch])
        w0s, s0s = np.ascontiguousarray(I["w0"][ch]), np.ascontiguousarray(I["s0"][ch])
        wls, sls = np.ascontiguousarray(I["wl"][:, ch]), np.ascontiguousarray(I["sl"][:, ch])
        rout = O.forward(xs, w0s, s0s, None, wls, sls, wl.L)
        rgr = O.backward(xs, gs, w0s, s0s, None, wls, sls, wl.L)
        got = {"out": out[:, ch], "dx": gx[:, ch], "dw0": gw0[ch], "ds0": gs0[ch], "dwl": gwl[:, ch], "dsl": gsl[:, ch]}
        ref = dict(out=rout, dx=rgr["dx"], dw0=rgr["dw0"], ds0=rgr["ds0"], dwl=rgr["dwl"], dsl=rgr["dsl"])
        for n in ref:
            if ref[n].size:
                worst[n] = max(worst.get(n, 0.0), rel_err(got[n].double().cpu().numpy(), ref[n]))
    tol = TOL[wl.dtype]
    bad = {n: e for n, e in worst.items() if not e <= tol}
    assert not bad, "%s [%s]: %s (all %s)" % (wl.name, wt.wtconv_plan_describe(desc), bad, worst)
    return worst


def test_tiny_config_in_full():
    _run_full_and_compare(inputs.WORKLOADS["tiny"])


def test_stage1_f32_bench_config_in_full():
    _run_full_and_compare(inputs.WORKLOADS["stage1_f32"])


@pytest.mark.parametrize("name", ["stage1_bf16", "stage2_bf16", "stage3_bf16", "stage4_bf16"])
def test_wtconvnext_stage_set_bf16(name):
    _run_full_and_compare(inputs.WORKLOADS[name])  # the configuration bench.py times, every channel


@pytest.mark.parametrize("name", ["convnext_s1_bf16", "convnext_s2_bf16", "convnext_s3_bf16", "convnext_s4_bf16"])
def test_wtconvnext_depth_schedule_bf16(name):
    wl = inputs.WORKLOADS[name]  # L = (5, 4, 3, 2): grids shrink through odd sizes (7 -> 4 -> 2, 14 -> 7 -> 4 -> 2)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wt.DTYPE_NAMES[wl.dtype])) in ("plane", "team")
    _run_full_and_compare(wl)


@pytest.mark.parametrize("name,flags", [("stage1_k3_f32", 0), ("stage1_k3_f32", wt.FLAG_TILED_ONLY), ("stage1_k7_f32", 0)],
                         ids=["k3_in_5x5_tables", "k3_per_level_kernels", "k7"])
def test_kernel_size_variants(name, flags):
    wl = inputs.WORKLOADS[name]
    plan = wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wt.DTYPE_NAMES[wl.dtype], flags))
    assert plan == ("plane" if (wl.k == 3 and flags == 0) else "tiled")  # 3 x 3 kernels ride the k = 5 kernels by default
    _run_full_and_compare(wl, flags=flags)


@pytest.mark.parametrize("dtype", ["f32", "f16"])
@pytest.mark.parametrize("L", [1, 2, 3, 4, 5])
def test_level_sweep(L, dtype):
    _run_full_and_compare(inputs.WORKLOADS["sweep_L%d_%s" % (L, dtype)])


@pytest.mark.parametrize("name", ["large_f16", "large_odd_f16"])
def test_large_planes(name):
    wl = inputs.WORKLOADS[name]  # 16 x 256 planes of 256 x 256 / 225 x 225: six channels spread over the tensor
    _run_full_and_compare(wl, groups=[0, 1, 77, 128, wl.C - 2, wl.C - 1], group=1)
