"""The library neither allocates nor synchronises, so a forward+backward step can be captured into a CUDA
graph (what one does with the launch-bound small stages) and replayed on new data in the same buffers."""
import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import TOL, rel_err, to_dev
from oracle import wtconv_oracle as O

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl", [
    Workload("graph_stage4", 4, 16, 7, 7, 5, 2, "bf16", 41),     # team kernels
    Workload("graph_stage2", 2, 8, 28, 28, 5, 2, "f32", 42),
    Workload("graph_tiled", 1, 3, 90, 75, 5, 3, "f32", 43),      # tiled path (several launches per call)
], ids=lambda w: w.name)
def test_step_replays_from_a_cuda_graph(wl):
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt)
    I1 = inputs.make_inputs(wl)
    I2 = inputs.make_inputs(wl.with_(seed=wl.seed + 100))
    w0, s0, wl_, sl = (to_dev(I1[n]) for n in ("w0", "s0", "wl", "sl"))
    x, g = to_dev(I1["x"], tdt), to_dev(I1["g"], tdt)
    out, gx = torch.empty_like(x), torch.empty_like(x)
    gw0, gs0, gwl, gsl = (torch.empty_like(t) for t in (w0, s0, wl_, sl))
    ws = wt.alloc_workspace(desc)

    def step(stream=None):
        wt.wtconv_forward(desc, x, w0, s0, None, wl_, sl, out, ws, stream=stream)
        wt.wtconv_backward(desc, x, g, w0, s0, None, wl_, sl, gx, gw0, gs0, None, gwl, gsl, ws, stream=stream)

    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in (out, gx, gw0, gs0, gwl, gsl)]

    step()  # first call outside capture (function attributes, lazy module loading)
    eager1 = snapshot()
    x.copy_(to_dev(I2["x"], tdt)); g.copy_(to_dev(I2["g"], tdt))
    step()
    eager2 = snapshot()

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    x.copy_(to_dev(I1["x"], tdt)); g.copy_(to_dev(I1["g"], tdt))
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        step(stream=side)
    for t in (out, gx, gw0, gs0, gwl, gsl):
        t.fill_(float("nan"))
    graph.replay()
    for got, want in zip(snapshot(), eager1):
        assert torch.equal(got, want)  # same kernels, same order: bit-identical (the reductions are fixed-order)
    x.copy_(to_dev(I2["x"], tdt)); g.copy_(to_dev(I2["g"], tdt))
    graph.replay()
    replayed = snapshot()
    for got, want in zip(replayed, eager2):
        assert torch.equal(got, want)
    # and the replayed step is the operator itself: every tensor against the fp64 oracle on the second input set
    ref_out = O.forward(I2["x"], I1["w0"], I1["s0"], None, I1["wl"], I1["sl"], wl.L)
    ref = O.backward(I2["x"], I2["g"], I1["w0"], I1["s0"], None, I1["wl"], I1["sl"], wl.L)
    for got, want in zip(replayed, (ref_out, ref["dx"], ref["dw0"], ref["ds0"], ref["dwl"], ref["dsl"])):
        assert rel_err(got.double().cpu().numpy(), want) <= TOL[wl.dtype]
