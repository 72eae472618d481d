"""Data-parallel plumbing of the batch-sharded WTConv step.

The operator shards by batch with no activation exchange: every (image, channel) plane is independent in the
forward pass and for grad_x; only the parameter gradients sum over the batch.  So one rank's step is the
library's forward + backward on its own images, followed by ONE all-reduce (sum) over a single flat buffer that
holds every parameter gradient.  This module owns that buffer layout; it contains no WTConv arithmetic.
"""
from collections import OrderedDict

import torch


def grad_shapes(C, k, L, bias=False):
    """Shapes of the parameter gradients, in the order they sit in the flat buffer."""
    s = OrderedDict()
    s["dw0"] = (C, k, k)
    s["ds0"] = (C,)
    if bias:
        s["db0"] = (C,)
    if L > 0:
        s["dwl"] = (L, C, 4, k, k)
        s["dsl"] = (L, C, 4)
    return s


class FlatGrads:
    """One contiguous float32 buffer with a named view per parameter gradient.

    The library writes the gradients through the views (they are ordinary contiguous tensors); the data-parallel
    exchange is a single all-reduce of `flat`."""

    def __init__(self, C, k, L, bias=False, device="cuda"):
        self.shapes = grad_shapes(C, k, L, bias)
        sizes = [int(torch.Size(s).numel()) for s in self.shapes.values()]
        # every view starts on a 16-byte boundary (4 floats)
        offs, total = [], 0
        for n in sizes:
            offs.append(total)
            total += (n + 3) // 4 * 4
        self.flat = torch.zeros(total, dtype=torch.float32, device=device)
        self.views = OrderedDict((name, self.flat[o:o + n].view(shape))
                                 for (name, shape), o, n in zip(self.shapes.items(), offs, sizes))

    def __getitem__(self, name):
        return self.views.get(name)

    def all_reduce(self, group=None):
        """Sum the parameter gradients over the ranks of `group` (the step's only exchange)."""
        import torch.distributed as dist
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(self.flat, op=dist.ReduceOp.SUM, group=group)
        return self.flat


def shard_batch(B, rank, world):
    """Images [lo, hi) of a global batch of B that rank `rank` of `world` owns (contiguous, sizes differ by <= 1)."""
    lo = B * rank // world
    hi = B * (rank + 1) // world
    return lo, hi
