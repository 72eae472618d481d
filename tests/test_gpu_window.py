"""Large planes on the window kernels (levels 1-2 on chip per window, levels >= 3 through the level-2 carrier on the
whole-plane kernels), against the fp64 oracle: aligned and unaligned rows, planes that are not multiples of the
window, every level count from 0 levels on the carrier to several, all storage types, and bit-exact index math."""
import numpy as np
import pytest

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

PW = wt.FLAG_PREFER_WINDOW  # aligned rows go to the tiled kernels by default: ask for the window kernels

SHAPES = [
    Workload("w_aligned_L2", 2, 3, 128, 96, 5, 2, "f32", 81),        # no carrier
    Workload("w_aligned_L5", 2, 3, 128, 128, 5, 5, "f32", 82),       # carrier 32 x 32 with three levels
    Workload("w_ragged_L4", 1, 2, 150, 131, 5, 4, "f32", 83),        # odd width: rows start at any 4-byte offset
    Workload("w_225_L5", 1, 2, 225, 225, 5, 5, "f32", 84),           # 225 -> 113 -> 57 -> 29 -> 15 -> 8
    Workload("w_L1", 1, 2, 100, 100, 5, 1, "f32", 85),
    Workload("w_L3_many", 5, 4, 136, 120, 5, 3, "f32", 86),            # several images and channels: gradient flushes
    Workload("w_tall", 1, 2, 300, 72, 5, 3, "f32", 87),
    Workload("w_wide", 1, 2, 76, 290, 5, 6, "f32", 88),
]


@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_window_kernels_fp32(wl):
    I = inputs.make_inputs(wl, bias=True)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "f32", PW)) == "window"
    assert_close(wl, run_gpu(wl, I, PW), run_oracle(wl, I))


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("wl", [SHAPES[1], SHAPES[2], SHAPES[3], SHAPES[5]], ids=lambda w: w.name)
def test_window_kernels_16bit(wl, dtype):
    wl = wl.with_(dtype=dtype)
    I = inputs.make_inputs(wl)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, dtype, PW)) == "window"
    assert_close(wl, run_gpu(wl, I, PW), run_oracle(wl, I))


@pytest.mark.parametrize("shape", [(128, 128, 3), (130, 77, 4), (225, 225, 5), (99, 201, 2)])
def test_window_index_and_padding_math_bit_exact(shape):
    H, W, L = shape
    wl = Workload("dyadic_window", 2, 3, H, W, 5, L, "f32", 90)
    I = inputs.make_dyadic_inputs(wl, bias=True)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, H, W, 5, L, "f32", PW)) == "window"
    out, gr = run_gpu(wl, I, PW)
    rout, rgr = run_oracle(wl, I)
    assert np.array_equal(out, rout)
    assert np.array_equal(gr["dx"], rgr["dx"])
    for n in ("dw0", "ds0", "db0", "dwl", "dsl"):
        assert np.array_equal(gr[n], rgr[n]), n


def test_default_dispatch_by_row_alignment():
    """Unaligned rows -> window kernels; 16-byte aligned rows -> tiled kernels unless the window kernels are asked for."""
    assert wt.wtconv_plan_name(wt.make_desc(16, 256, 225, 225, 5, 5, "f16")) == "window"
    assert wt.wtconv_plan_name(wt.make_desc(16, 256, 256, 256, 5, 5, "f16")) == "tiled"
    assert wt.wtconv_plan_name(wt.make_desc(16, 256, 256, 256, 5, 5, "f16", PW)) == "window"
    assert wt.wtconv_plan_name(wt.make_desc(1, 2, 150, 131, 5, 4, "f32")) == "window"


def test_tiled_path_still_serves_large_planes_when_asked():
    wl = SHAPES[2]
    I = inputs.make_inputs(wl, bias=True)
    assert wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, "f32", wt.FLAG_NO_WINDOW)) == "tiled"
    assert_close(wl, run_gpu(wl, I, wt.FLAG_NO_WINDOW), run_oracle(wl, I))
