"""The reference-style comparator (the layer as the chain of separate operators of Sec. 3.1, every intermediate in
HBM) and the cumulative ablation steps of Table 8, through the C ABI, against the fp64 oracle: the comparator is a
measuring stick, so it has to compute the same operator as everything else."""
import numpy as np
import pytest
import torch

from oracle import wtconv_oracle as O
from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import TOL, assert_close, rel_err, run_gpu, run_oracle, to_dev

pytestmark = pytest.mark.gpu

REF = wt.FLAG_REFERENCE_CHAIN
SHAPES = [
    Workload("tiny", 1, 8, 16, 16, 5, 2, "f32", 0),
    Workload("ragged_multi_tile", 2, 3, 37, 45, 5, 3, "f32", 11),
    Workload("k3", 2, 2, 20, 33, 3, 2, "f32", 12),
    Workload("k7", 1, 3, 40, 24, 7, 2, "f32", 13),
    Workload("odd7", 3, 5, 7, 7, 5, 2, "f32", 14),
    Workload("base_only", 2, 3, 9, 12, 5, 0, "f32", 17),
    Workload("deep", 1, 2, 70, 66, 5, 6, "f32", 18),
    Workload("many_images", 11, 3, 28, 28, 5, 2, "f32", 31),   # more images than batch splits of the gradient kernels
    Workload("big_plane", 1, 2, 150, 131, 5, 4, "f32", 24),
]


@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_reference_chain_forward_backward(wl):
    I = inputs.make_inputs(wl, bias=True)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "f32", REF)) == "reference-chain"
    assert_close(wl, run_gpu(wl, I, REF), run_oracle(wl, I))


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_reference_chain_16bit(dtype):
    wl = SHAPES[1].with_(dtype=dtype)
    I = inputs.make_inputs(wl)
    assert_close(wl, run_gpu(wl, I, REF), run_oracle(wl, I))


@pytest.mark.parametrize("extra", [wt.FLAG_ABLATE_FUSED_ANALYSIS,
                                   wt.FLAG_ABLATE_FUSED_ANALYSIS | wt.FLAG_ABLATE_COLLAPSED_SYNTHESIS,
                                   wt.FLAG_ABLATE_COLLAPSED_SYNTHESIS], ids=["fused_analysis", "plus_collapsed", "collapsed_only"])
@pytest.mark.parametrize("wl", [SHAPES[0], SHAPES[1], SHAPES[3], SHAPES[4], SHAPES[5]], ids=lambda w: w.name)
def test_ablation_steps_forward(wl, extra):
    I = inputs.make_inputs(wl, bias=True)
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "f32", REF | extra)
    x = to_dev(I["x"])
    out = torch.full_like(x, float("nan"))
    ws = wt.alloc_workspace(desc)
    wt.wtconv_forward(desc, x, to_dev(I["w0"]), to_dev(I["s0"]), to_dev(I["b0"]),
                      to_dev(I["wl"]) if wl.L else None, to_dev(I["sl"]) if wl.L else None, out, ws)
    torch.cuda.synchronize()
    ref = O.forward(I["x"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    assert rel_err(out.double().cpu().numpy(), ref) <= TOL["f32"]


def test_reference_chain_on_the_level_sweep_config():
    """Full size of the sweep configuration (B=32, C=128, 64 x 64, L=3, fp32), a sample of channels against the oracle."""
    wl = inputs.WORKLOADS["sweep_L3_f32"]
    I = inputs.make_inputs(wl)
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "f32", REF)
    dev = lambda a: torch.from_numpy(a).cuda().contiguous()
    out, gr = wt.forward_backward(desc, dev(I["x"]), dev(I["g"]), dev(I["w0"]), dev(I["s0"]), None, dev(I["wl"]), dev(I["sl"]))
    torch.cuda.synchronize()
    ch = [0, 63, wl.C - 1]
    sub = lambda a, axis: np.ascontiguousarray(np.take(a, ch, axis=axis))
    rout = O.forward(sub(I["x"], 1), sub(I["w0"], 0), sub(I["s0"], 0), None, sub(I["wl"], 1), sub(I["sl"], 1), wl.L)
    rgr = O.backward(sub(I["x"], 1), sub(I["g"], 1), sub(I["w0"], 0), sub(I["s0"], 0), None, sub(I["wl"], 1), sub(I["sl"], 1), wl.L)
    idx = torch.tensor(ch, device="cuda")
    got = {"out": out.index_select(1, idx), "dx": gr["dx"].index_select(1, idx), "dw0": gr["dw0"].index_select(0, idx),
           "ds0": gr["ds0"].index_select(0, idx), "dwl": gr["dwl"].index_select(1, idx), "dsl": gr["dsl"].index_select(1, idx)}
    ref = dict(out=rout, dx=rgr["dx"], dw0=rgr["dw0"], ds0=rgr["ds0"], dwl=rgr["dwl"], dsl=rgr["dsl"])
    errs = {n: rel_err(got[n].double().cpu().numpy(), ref[n]) for n in ref}
    assert all(e <= TOL["f32"] for e in errs.values()), errs
