"""The batch-sharded (data-parallel) path on CPU ranks: two gloo processes each take half of the batch,
compute the operator with the fp64 oracle standing in for the per-rank GPU library, and sum the parameter
gradients with one all-reduce - the only exchange the sharded operator has.  The result must equal the
single-process result on the full batch; activations need no exchange at all."""
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
    from paper_2608_10805_b200 import inputs
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = inputs.Workload("dp", 4, 3, 14, 10, 5, 2, "f32", 77)
    I = inputs.make_inputs(wl, bias=True)
    per = wl.B // world
    sl = slice(rank * per, (rank + 1) * per)
    x, g = I["x"][sl], I["g"][sl]
    out = O.forward(x, I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    gr = O.backward(x, g, I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    for n in ("dw0", "ds0", "db0", "dwl", "dsl"):  # the data-parallel exchange: sum of parameter gradients
        t = torch.from_numpy(gr[n])
        dist.all_reduce(t)
        gr[n] = t.numpy()
    # timing convention of the benchmark: max over ranks
    tmax = torch.tensor([float(rank + 1)])
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    q.put((rank, out, gr, float(tmax.item())))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_batch_sharded_two_ranks_match_single_process():
    sys.path.insert(0, ROOT)
    from oracle import wtconv_oracle as O
    from paper_2608_10805_b200 import inputs
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
    wl = inputs.Workload("dp", 4, 3, 14, 10, 5, 2, "f32", 77)
    I = inputs.make_inputs(wl, bias=True)
    out = O.forward(I["x"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    gr = O.backward(I["x"], I["g"], I["w0"], I["s0"], I["b0"], I["wl"], I["sl"], wl.L)
    np.testing.assert_allclose(np.concatenate([res[0][1], res[1][1]]), out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(np.concatenate([res[0][2]["dx"], res[1][2]["dx"]]), gr["dx"], rtol=0, atol=1e-12)
    for n in ("dw0", "ds0", "db0", "dwl", "dsl"):
        np.testing.assert_allclose(res[0][2][n], gr[n], rtol=0, atol=1e-10)
        np.testing.assert_allclose(res[1][2][n], gr[n], rtol=0, atol=1e-10)
    assert res[0][3] == res[1][3] == 2.0
