"""The timeout path of the kernels' bounded waits, exercised without hanging or faulting anything: under
WTCONV_FLAG_TEST_NO_COPY no bulk copy is ever issued and the wait limit is tiny, so every wait for a copy runs out;
the kernels must then record it in the status word and return normally (nothing is in flight), the context must
stay usable, and the Python layers must surface the condition as WTCONV_ERR_TIMEOUT."""
import re

import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_gpu, run_oracle, to_dev

pytestmark = pytest.mark.gpu

CASES = [(Workload("plane_28", 8, 12, 28, 28, 5, 2, "bf16", 71), wt.FLAG_NO_TEAM),   # block-per-plane kernels with a prefetch ring
         (Workload("team_7", 16, 16, 7, 7, 5, 1, "bf16", 72), 0)]                  # team kernels


@pytest.mark.parametrize("wl,flags", CASES, ids=lambda v: v.name if hasattr(v, "name") else None)
def test_waits_run_out_status_is_set_and_context_survives(wl, flags):
    tdt = wt.DTYPE_NAMES[wl.dtype]
    good = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags)
    text = wt.wtconv_plan_describe(good)
    rings = [int(v) for v in re.findall(r"ring=(\d+)", text)]
    assert len(rings) == 2 and min(rings) >= 1, "pick a shape whose plans prefetch by bulk copy: " + text
    bad = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags | wt.FLAG_TEST_NO_COPY)
    I = inputs.make_inputs(wl)
    x, g = to_dev(I["x"], tdt), to_dev(I["g"], tdt)
    w0, s0, wl_, sl = to_dev(I["w0"]), to_dev(I["s0"]), to_dev(I["wl"]), to_dev(I["sl"])
    out, gx = torch.empty_like(x), torch.empty_like(x)
    gw0, gs0, gwl, gsl = (torch.empty_like(t) for t in (w0, s0, wl_, sl))
    ws = wt.alloc_workspace(bad)
    flag = torch.zeros(2, dtype=torch.int32).pin_memory()
    wt.wtconv_forward(bad, x, w0, s0, None, wl_, sl, out, ws)
    wt.wtconv_read_status(bad, ws, flag[0:1])
    wt.wtconv_backward(bad, x, g, w0, s0, None, wl_, sl, gx, gw0, gs0, None, gwl, gsl, ws)
    wt.wtconv_read_status(bad, ws, flag[1:2])
    torch.cuda.synchronize()  # returns: no kernel spins, no fault
    assert int(flag[0]) != 0 and int(flag[1]) != 0
    with pytest.raises(wt.WTConvError) as e:  # the convenience layer reports it as WTCONV_ERR_TIMEOUT
        wt.forward_backward(bad, x, g, w0, s0, None, wl_, sl)
    assert e.value.code == 11
    # the context is intact: the same shape without the test flag gives oracle-exact results and a clean status
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))


def test_autograd_layer_reports_an_earlier_timeout():
    from paper_2608_10805_b200 import autograd as ag
    wl = CASES[1][0]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, torch.bfloat16, wt.FLAG_TEST_NO_COPY)
    I = inputs.make_inputs(wl)
    x = to_dev(I["x"], torch.bfloat16)
    out = torch.empty_like(x)
    ws = wt.alloc_workspace(desc)
    ag.status_watch.drain()
    wt.wtconv_forward(desc, x, to_dev(I["w0"]), to_dev(I["s0"]), None, to_dev(I["wl"]), to_dev(I["sl"]), out, ws)
    with pytest.raises(wt.WTConvError):
        ag.status_watch.after_call(desc, ws)
        ag.status_watch.drain()
    ag.status_watch.drain()  # nothing is left pending


def test_a_workspace_carries_nothing_from_one_call_to_the_next():
    """No call clears its workspace.  A call that timed out leaves its tag in the status words and its partial
    sums (of another shape) in the workspace; a later call of a different shape on the same workspace must read as
    clean and give the oracle's results."""
    first, flags1 = CASES[0]
    second = Workload("plane_14_after", 4, 24, 14, 14, 5, 2, "f32", 73)
    tdt1, tdt2 = wt.DTYPE_NAMES[first.dtype], wt.DTYPE_NAMES[second.dtype]
    bad = wt.make_desc(first.B, first.C, first.H, first.W, first.k, first.L, tdt1, flags1 | wt.FLAG_TEST_NO_COPY)
    good = wt.make_desc(second.B, second.C, second.H, second.W, second.k, second.L, tdt2, wt.FLAG_NO_TEAM)
    assert wt.wtconv_plan_name(good) == "plane"
    nbytes = max(max(wt.wtconv_workspace_bytes(bad)), max(wt.wtconv_workspace_bytes(good)))
    ws = torch.full((nbytes,), 0xFF, dtype=torch.uint8, device="cuda")
    flag = torch.zeros(3, dtype=torch.int32).pin_memory()
    I1, I2 = inputs.make_inputs(first), inputs.make_inputs(second)
    x1, g1 = to_dev(I1["x"], tdt1), to_dev(I1["g"], tdt1)
    p1 = [to_dev(I1[k]) for k in ("w0", "s0", "wl", "sl")]
    gx1 = torch.empty_like(x1)
    gp1 = [torch.empty_like(t) for t in p1]
    wt.wtconv_backward(bad, x1, g1, p1[0], p1[1], None, p1[2], p1[3], gx1, gp1[0], gp1[1], None, gp1[2], gp1[3], ws)
    wt.wtconv_read_status(bad, ws, flag[0:1])
    x2, g2 = to_dev(I2["x"], tdt2), to_dev(I2["g"], tdt2)
    p2 = [to_dev(I2[k]) for k in ("w0", "s0", "wl", "sl")]
    out2, gx2 = torch.full_like(x2, float("nan")), torch.full_like(x2, float("nan"))
    gp2 = [torch.full_like(t, float("nan")) for t in p2]
    wt.wtconv_forward(good, x2, p2[0], p2[1], None, p2[2], p2[3], out2, ws)
    wt.wtconv_read_status(good, ws, flag[1:2])
    wt.wtconv_backward(good, x2, g2, p2[0], p2[1], None, p2[2], p2[3], gx2, gp2[0], gp2[1], None, gp2[2], gp2[3], ws)
    wt.wtconv_read_status(good, ws, flag[2:3])
    torch.cuda.synchronize()
    assert int(flag[0]) != 0 and int(flag[1]) == 0 and int(flag[2]) == 0
    f = lambda t: t.double().cpu().numpy()
    got = (f(out2), dict(dx=f(gx2), dw0=f(gp2[0]), ds0=f(gp2[1]), db0=None, dwl=f(gp2[2]), dsl=f(gp2[3])))
    assert_close(second, got, run_oracle(second, I2))
