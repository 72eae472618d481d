"""Calls on distinct streams with distinct workspaces may overlap (the header's contract), also when issued from
several host threads at once (the plan cache and the lazily created per-device state are shared)."""
import threading

import pytest
import torch

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import to_dev

pytestmark = pytest.mark.gpu

CASES = [
    Workload("conc_a", 4, 8, 28, 28, 5, 2, "f32", 61),
    Workload("conc_b", 2, 6, 56, 56, 5, 3, "bf16", 62),
    Workload("conc_c", 1, 3, 90, 75, 5, 3, "f32", 63),   # tiled path
    Workload("conc_d", 6, 16, 7, 7, 5, 2, "f16", 64),
]


def _setup(wl):
    tdt = wt.DTYPE_NAMES[wl.dtype]
    I = inputs.make_inputs(wl)
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt)
    t = dict(x=to_dev(I["x"], tdt), g=to_dev(I["g"], tdt), w0=to_dev(I["w0"]), s0=to_dev(I["s0"]), wl=to_dev(I["wl"]),
             sl=to_dev(I["sl"]))
    return desc, t


def _run(desc, t, stream):
    ws = wt.alloc_workspace(desc)
    with torch.cuda.stream(stream):
        out, gr = wt.forward_backward(desc, t["x"], t["g"], t["w0"], t["s0"], None, t["wl"], t["sl"], ws, stream)
    return out, gr, ws


def test_overlapping_calls_from_several_threads_match_serial_results():
    setups = [_setup(wl) for wl in CASES]
    serial = []
    for desc, t in setups:
        out, gr, _ = _run(desc, t, torch.cuda.current_stream())
        torch.cuda.synchronize()
        serial.append((out.clone(), {k: v.clone() for k, v in gr.items() if v is not None}))
    results = [None] * len(setups)
    errors = []

    def worker(i):
        try:
            torch.cuda.set_device(0)
            s = torch.cuda.Stream()
            for _ in range(5):  # several rounds so that the calls of different threads really interleave
                results[i] = _run(setups[i][0], setups[i][1], s)
            s.synchronize()
        except Exception as e:  # surfaced in the main thread below
            errors.append((i, repr(e)))

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(len(setups))]
    for th in threads:
        th.start()
    for th in threads:
        th.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for (out, gr, _), (sout, sgr) in zip(results, serial):
        assert torch.equal(out, sout)  # same kernels on the same data: bit-identical
        for k, v in sgr.items():
            assert torch.equal(gr[k], v), k


@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_status_word_reads_zero_after_a_normal_step(wl):
    desc, t = _setup(wl)
    s = torch.cuda.Stream()
    out, gr, ws = _run(desc, t, s)
    flag = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    wt.wtconv_read_status(desc, ws, flag, s)
    s.synchronize()
    assert int(flag[0]) == 0 and bool(torch.isfinite(out.float()).all())
