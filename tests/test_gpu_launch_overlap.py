"""Calls that follow one another on a stream without anything between them: the persistent kernels start their
set-up behind the tail of the kernel before them and nothing clears a workspace between calls.  A training loop
that runs several layers of different shapes through ONE shared workspace must still get every layer's results
right: each backward call's partial sums and status words are overwritten by the next layer's calls only after the
epilogue that reads them has finished."""
import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_oracle, to_dev

pytestmark = pytest.mark.gpu

LAYERS = [Workload("ov_plane_28", 6, 24, 28, 28, 5, 2, "bf16", 81),   # fused backward
          Workload("ov_team_7", 12, 32, 7, 7, 5, 1, "bf16", 82),      # team kernels
          Workload("ov_split_40", 3, 10, 40, 36, 5, 3, "f32", 83),    # split backward (weight-gradient + input-gradient kernels)
          Workload("ov_plane_14", 8, 40, 14, 14, 5, 1, "f16", 84),
          Workload("ov_tiled_k7", 2, 6, 20, 24, 7, 2, "f32", 85)]     # per-level kernels between the persistent ones


def test_layers_share_one_workspace_back_to_back():
    descs = [wt.make_desc(w.B, w.C, w.H, w.W, w.k, w.L, wt.DTYPE_NAMES[w.dtype], 0) for w in LAYERS]
    plans = [wt.wtconv_plan_name(d) for d in descs]
    assert {"plane", "team", "tiled"} <= set(plans), plans
    nbytes = max(max(wt.wtconv_workspace_bytes(d)) for d in descs)
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")
    Is = [inputs.make_inputs(w) for w in LAYERS]
    dev = []
    for w, I in zip(LAYERS, Is):
        tdt = wt.DTYPE_NAMES[w.dtype]
        x, g = to_dev(I["x"], tdt), to_dev(I["g"], tdt)
        p = [to_dev(I[k]) for k in ("w0", "s0", "wl", "sl")]
        dev.append((x, g, p))
    nan = float("nan")
    results = []
    flags = torch.zeros(2 * len(LAYERS) * 2, dtype=torch.int32).pin_memory()
    k = 0
    for rep in range(2):  # the second pass finds every layer's stale sums and tags in the workspace
        results = []
        for d, (x, g, p) in zip(descs, dev):
            out, gx = torch.full_like(x, nan), torch.full_like(x, nan)
            gp = [torch.full_like(t, nan) for t in p]
            wt.wtconv_forward(d, x, p[0], p[1], None, p[2], p[3], out, ws)
            results.append((out, gx, gp))
        for d, (x, g, p), (out, gx, gp) in reversed(list(zip(descs, dev, results))):  # backward in reverse layer order
            wt.wtconv_backward(d, x, g, p[0], p[1], None, p[2], p[3], gx, gp[0], gp[1], None, gp[2], gp[3], ws)
        wt.wtconv_read_status(descs[0], ws, flags[k:k + 1])
        k += 1
    torch.cuda.synchronize()
    assert not bool(flags.any())
    f = lambda t: t.double().cpu().numpy()
    for w, I, (out, gx, gp) in zip(LAYERS, Is, results):
        got = (f(out), dict(dx=f(gx), dw0=f(gp[0]), ds0=f(gp[1]), db0=None, dwl=f(gp[2]), dsl=f(gp[3])))
        assert_close(w, got, run_oracle(w, I), what="shared workspace")
