"""wtconv_step_host (host buffers in, host buffers out, copies inside) against the fp64 oracle, and twice in
a row on the same buffers: the internal copy stream is joined before the caller's stream reaches the end."""
import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import TOL, rel_err, run_oracle

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wl,bias", [
    (Workload("host_plane", 3, 4, 28, 28, 5, 2, "f32", 51), True),
    (Workload("host_bf16", 4, 6, 14, 14, 5, 1, "bf16", 52), False),
    (Workload("host_tiled", 1, 2, 90, 75, 3, 2, "f32", 53), False),
    (Workload("host_chunked", 64, 16, 56, 56, 5, 3, "f32", 54), True),   # large enough for the chunked pipeline
], ids=lambda v: v.name if isinstance(v, Workload) else str(v))
def test_host_step_matches_oracle(wl, bias):
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt)
    pin = lambda a, dt=torch.float32: torch.from_numpy(a).to(dt).contiguous().pin_memory()
    ws = torch.empty(wt.wtconv_step_host_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.Stream()
    for seed_shift in (0, 100):  # second round: new data through the same buffers and the same internal stream
        I = inputs.make_inputs(wl.with_(seed=wl.seed + seed_shift), bias=bias)
        hx, hg = pin(I["x"], tdt), pin(I["g"], tdt)
        hw0, hs0, hwl, hsl = pin(I["w0"]), pin(I["s0"]), pin(I["wl"]), pin(I["sl"])
        hb0 = pin(I["b0"]) if bias else None
        hout, hgx = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()
        hgw0, hgs0, hgwl, hgsl = (torch.empty_like(t).pin_memory() for t in (hw0, hs0, hwl, hsl))
        hgb0 = torch.empty_like(hb0).pin_memory() if bias else None
        for t in (hout, hgx):
            t.fill_(float("nan"))
        wt.wtconv_step_host(desc, hx, hg, hw0, hs0, hb0, hwl, hsl, hout, hgx, hgw0, hgs0, hgb0, hgwl, hgsl, ws, stream)
        stream.synchronize()  # the caller's stream alone: the internal stream must have been joined
        ref_out, ref = run_oracle(wl, I)
        got = {"out": hout, "dx": hgx, "dw0": hgw0, "ds0": hgs0, "dwl": hgwl, "dsl": hgsl}
        want = {"out": ref_out, "dx": ref["dx"], "dw0": ref["dw0"], "ds0": ref["ds0"], "dwl": ref["dwl"], "dsl": ref["dsl"]}
        if bias:
            got["db0"], want["db0"] = hgb0, ref["db0"]
        for n in want:
            e = rel_err(got[n].double().numpy(), want[n])
            assert e <= TOL[wl.dtype], "%s %s: %g" % (wl.name, n, e)
