"""The batch-sharded (data-parallel) path on CPU ranks: two gloo processes each take their share of the batch
(paper_2608_10805_b200.dp.shard_batch), compute the operator with the fp64 oracle standing in for the per-rank GPU
library, write their parameter gradients through the views of ONE flat buffer (dp.FlatGrads - the object bench.py
and a trainer use) and sum that buffer with a single all-reduce, the only exchange the sharded operator has.  The
result must equal the single-process result on the full batch; activations need no exchange at all."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from oracle import wtconv_oracle as O
    from paper_2608_10805_b200 import dp, inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.Workload("dp", 5, 3, 14, 10, 5, 2, "f32", 77)  # 5 images over 2 ranks: uneven shares
    I = inputs.make_inputs(wl, bias=True)
    lo, hi = dp.shard_batch(wl.B, rank, world)
    x, g = I["x"][lo:hi], I["g"][lo:hi]
    out = O.forward(x, I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    gr = O.backward(x, g, I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    flat = dp.FlatGrads(wl.C, wl.k, wl.L, bias=True, device="cpu")
    for n in flat.views:  # the library would write these views directly
        flat[n].copy_(torch.from_numpy(gr[n]).float())
    calls = {"n": 0}
    real = dist.all_reduce

    def counting(*a, **kw):
        calls["n"] += 1
        return real(*a, **kw)
    dist.all_reduce = counting
    flat.all_reduce()  # the data-parallel exchange: exactly one collective over the flat buffer
    dist.all_reduce = real
    tmax = torch.tensor([float(rank + 1)])
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)  # timing convention of the benchmark: max over ranks
    q.put((rank, (lo, hi), out, gr["dx"], {n: v.numpy().copy() for n, v in flat.views.items()}, calls["n"], float(tmax.item())))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_batch_sharded_two_ranks_match_single_process():
    sys.path.insert(0, ROOT)
    from oracle import wtconv_oracle as O
    from paper_2608_10805_b200 import dp, inputs
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted([q.get(timeout=100) for _ in procs], key=lambda t: t[0])
    for p in procs:
        p.join(timeout=30)
        assert p.exitcode == 0
    wl = inputs.Workload("dp", 5, 3, 14, 10, 5, 2, "f32", 77)
    I = inputs.make_inputs(wl, bias=True)
    out = O.forward(I["x"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    gr = O.backward(I["x"], I["g"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    assert [r[1] for r in res] == [(0, 2), (2, 5)]  # contiguous shares that cover the batch
    np.testing.assert_allclose(np.concatenate([res[0][2], res[1][2]]), out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([res[0][3], res[1][3]]), gr["dx"], rtol=0, atol=1e-12)
    for n in ("dw0", "ds0", "db0", "dwl", "dsl"):  # both ranks hold the full-batch sums (float32 buffer)
        scale = np.abs(gr[n]).max()
        np.testing.assert_allclose(res[0][4][n], gr[n], rtol=0, atol=2e-6 * scale)
        np.testing.assert_array_equal(res[0][4][n], res[1][4][n])
    assert res[0][5] == res[1][5] == 1  # one collective per step
    assert res[0][6] == res[1][6] == 2.0


def test_flat_gradient_buffer_layout():
    sys.path.insert(0, ROOT)
    from paper_2608_10805_b200 import dp
    f = dp.FlatGrads(6, 5, 3, bias=True, device="cpu")
    assert list(f.views) == ["dw0", "ds0", "db0", "dwl", "dsl"]
    assert f["dwl"].shape == (3, 6, 4, 5, 5) and f["dsl"].shape == (3, 6, 4) and f["dw0"].is_contiguous()
    base = f.flat.data_ptr()
    for v in f.views.values():  # every view starts on a 16-byte boundary inside the one buffer
        assert (v.data_ptr() - base) % 16 == 0 and base <= v.data_ptr() < base + f.flat.numel() * 4
    g = dp.FlatGrads(4, 3, 0, bias=False, device="cpu")
    assert list(g.views) == ["dw0", "ds0"] and g["dwl"] is None
    assert [dp.shard_batch(7, r, 3) for r in range(3)] == [(0, 2), (2, 4), (4, 7)]
