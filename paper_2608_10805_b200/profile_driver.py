"""Small driver for profiler captures: runs forward+backward of a named workload (optionally with a smaller
batch) a few times through the C ABI on random tensors.  Usage:
    python -m paper_2608_10805_b200.profile_driver <workload> [batch] [repeats] [flags]
"""
import sys

import torch

from . import inputs
from . import wtconv as wt


def main():
    name = sys.argv[1]
    wl = inputs.WORKLOADS[name]
    if len(sys.argv) > 2:
        wl = wl.with_(B=int(sys.argv[2]))
    reps = int(sys.argv[3]) if len(sys.argv) > 3 else 2
    flags = int(sys.argv[4], 0) if len(sys.argv) > 4 else 0
    tdt = wt.DTYPE_NAMES[wl.dtype]
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, tdt, flags)
    x = torch.randn(wl.B, wl.C, wl.H, wl.W, device="cuda").to(tdt)
    g = torch.randn_like(x)
    w0 = torch.randn(wl.C, wl.k, wl.k, device="cuda") * 0.1
    s0 = torch.rand(wl.C, device="cuda") + 0.5
    wl_ = torch.randn(wl.L, wl.C, 4, wl.k, wl.k, device="cuda") * 0.1
    sl = torch.rand(wl.L, wl.C, 4, device="cuda") + 0.5
    for _ in range(reps):
        wt.forward_backward(desc, x, g, w0, s0, None, wl_, sl)
    torch.cuda.synchronize()
    print("ok", wt.wtconv_plan_name(desc), wt.wtconv_launch_count(desc))


if __name__ == "__main__":
    main()
