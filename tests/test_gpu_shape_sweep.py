"""Seeded sweep over irregular shapes, level counts and storage types through whatever kernel family the dispatcher
picks (team, plane, window, tiled), against the fp64 oracle, with guard bands and NaN-filled outputs.  The shapes are
drawn once from a fixed seed; degenerate ones (single rows and columns, one pixel, more levels than the plane has
bits) are added by hand."""
import numpy as np
import pytest

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_gpu, run_oracle

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.Generator(np.random.Philox(key=20260810))
    out = []
    for i in range(48):
        H, W = int(rng.integers(1, 150)), int(rng.integers(1, 150))
        if i % 3 == 0:  # the tiny-plane kernels need small planes and channel groups
            H, W = int(rng.integers(3, 11)), int(rng.integers(3, 11))
        B, C = int(rng.integers(1, 6)), int(rng.choice([1, 2, 3, 4, 8, 16]))
        while B * C * H * W > 300000:
            B, C = max(1, B // 2), max(1, C // 2)
        L = int(rng.integers(0, 7))
        k = 5 if i % 8 else int(rng.choice([3, 7]))
        dt = ["f32", "f32", "f16", "bf16"][i % 4]
        out.append(Workload("sweep%02d_%dx%dx%dx%d_k%d_L%d_%s" % (i, B, C, H, W, k, L, dt), B, C, H, W, k, L, dt, 300 + i))
    extra = [(1, 2, 1000, 1, 5, 3, "f32"), (1, 2, 1, 1000, 5, 2, "f16"), (1, 1, 71, 71, 5, 8, "f32"), (2, 2, 80, 80, 5, 5, "bf16"),
             (1, 2, 500, 3, 5, 8, "f32"), (1, 8, 2, 2, 5, 4, "f32"), (3, 16, 1, 7, 5, 1, "bf16"), (1, 1, 260, 260, 5, 8, "f16"),
             (2, 4, 139, 72, 5, 3, "f32"), (1, 3, 288, 40, 5, 0, "f32")]
    for j, (B, C, H, W, k, L, dt) in enumerate(extra):
        out.append(Workload("edge%02d_%dx%dx%dx%d_L%d_%s" % (j, B, C, H, W, L, dt), B, C, H, W, k, L, dt, 400 + j))
    return out


@pytest.mark.parametrize("wl", _cases(), ids=lambda w: w.name)
def test_dispatcher_choice_matches_the_oracle(wl):
    I = inputs.make_inputs(wl, bias=(wl.seed % 2 == 0))
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wl.dtype)) in ("team", "plane", "window", "tiled")
    assert_close(wl, run_gpu(wl, I), run_oracle(wl, I))
