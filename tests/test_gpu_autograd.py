"""The torch.autograd front end against the fp64 oracle: gradients reach x and every parameter through
`loss.backward()` and equal the oracle's analytic backward."""
import numpy as np
import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200.inputs import Workload

from helpers import TOL, rel_err, run_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl,bias", [
    (Workload("ag_plane", 2, 4, 28, 28, 5, 2, "f32", 31), True),
    (Workload("ag_odd_bf16", 3, 5, 7, 7, 5, 2, "bf16", 32), False),
    (Workload("ag_tiled_k3", 2, 3, 20, 33, 3, 2, "f32", 33), True),
    (Workload("ag_base_only", 2, 3, 9, 12, 5, 0, "f32", 34), False),
], ids=lambda v: v.name if isinstance(v, Workload) else str(v))
def test_module_gradients_match_oracle(wl, bias):
    from paper_2608_10805_b200.autograd import WTConv2d
    from paper_2608_10805_b200 import wtconv as wt
    I = inputs.make_inputs(wl, bias=bias)
    tdt = wt.DTYPE_NAMES[wl.dtype]
    layer = WTConv2d(wl.C, wl.k, wl.L, bias=bias)
    with torch.no_grad():
        layer.w0.copy_(torch.from_numpy(I["w0"]))
        layer.s0.copy_(torch.from_numpy(I["s0"]))
        layer.wl.copy_(torch.from_numpy(I["wl"]))
        layer.sl.copy_(torch.from_numpy(I["sl"]))
        if bias:
            layer.b0.copy_(torch.from_numpy(I["b0"]))
    x = torch.from_numpy(I["x"]).cuda().to(tdt).requires_grad_(True)
    g = torch.from_numpy(I["g"]).cuda().to(tdt)
    out = layer(x)
    (out.float() * g.float()).sum().backward()
    ref_out, ref = run_oracle(wl, I)
    tol = TOL[wl.dtype]
    got = {"out": out, "dx": x.grad, "dw0": layer.w0.grad, "ds0": layer.s0.grad, "dwl": layer.wl.grad,
           "dsl": layer.sl.grad}
    want = {"out": ref_out, "dx": ref["dx"], "dw0": ref["dw0"], "ds0": ref["ds0"], "dwl": ref["dwl"], "dsl": ref["dsl"]}
    if bias:
        got["db0"], want["db0"] = layer.b0.grad, ref["db0"]
    for n in want:
        if want[n].size == 0:
            continue
        e = rel_err(got[n].detach().double().cpu().numpy(), want[n])
        assert e <= tol, "%s %s: %g" % (wl.name, n, e)


def test_cpu_tensor_is_refused():
    from paper_2608_10805_b200.autograd import WTConv2d
    layer = WTConv2d(2, 5, 1)
    with pytest.raises(RuntimeError):
        layer(torch.zeros(1, 2, 8, 8))
