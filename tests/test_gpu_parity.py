"""GPU parity: the CUDA library, called through the C ABI, against the fp64 oracle on the same
seeded inputs, element by element.  fp32: rel err <= 1e-5; fp16/bf16 storage (fp32 arithmetic):
<= 2e-2; index / padding math: bit-exact on dyadic inputs."""
import numpy as np
import pytest

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

PATHS = [pytest.param(0, id="auto"), pytest.param(wt.FLAG_TILED_ONLY, id="tiled")]

SMALL = [
    Workload("tiny", 1, 8, 16, 16, 5, 2, "f32", 0),                 # benchmark config 1
    Workload("ragged_multi_tile", 2, 3, 37, 45, 5, 3, "f32", 11),   # several tiles + ragged tails, odd sizes
    Workload("k3", 2, 2, 20, 33, 3, 2, "f32", 12),
    Workload("k7", 1, 3, 40, 24, 7, 2, "f32", 13),
    Workload("odd7", 3, 5, 7, 7, 5, 2, "f32", 14),                  # 7 -> 4 -> 2, padded at both levels
    Workload("one_pixel", 2, 2, 1, 1, 5, 2, "f32", 15),             # degenerate: every level grid is 1x1
    Workload("row", 1, 2, 1, 19, 5, 3, "f32", 16),
    Workload("base_only", 2, 3, 9, 12, 5, 0, "f32", 17),            # L = 0
    Workload("deep", 1, 2, 70, 66, 5, 8, "f32", 18),                # maximum level count, grids shrink to 1x1
    Workload("stage1_small", 2, 4, 56, 56, 5, 3, "f32", 19),
    Workload("stage2_small", 2, 4, 28, 28, 5, 2, "f32", 20),
    Workload("stage3_small", 2, 4, 14, 14, 5, 1, "f32", 21),
    Workload("stage4_small", 3, 5, 7, 7, 5, 1, "f32", 22),
    Workload("sweep_small_L5", 1, 3, 64, 64, 5, 5, "f32", 23),
    Workload("big_plane", 1, 2, 225, 225, 5, 5, "f32", 24),
    Workload("convnext_s1_small", 2, 3, 56, 56, 5, 5, "f32", 25),   # the network's depth schedule L = (5, 4, 3, 2)
    Workload("convnext_s2_small", 2, 3, 28, 28, 5, 4, "f32", 26),
    Workload("convnext_s3_small", 3, 5, 14, 14, 5, 3, "f32", 27),
]


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("wl", SMALL, ids=lambda w: w.name)
def test_small_fp32(wl, flags):
    I = inputs.make_inputs(wl)
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))


# Tiny planes with a channel count the team kernels can group (several planes per thread team); the same
# shapes also run on the block-per-plane kernels (FLAG_NO_TEAM) and on the tiled path.
TEAM_SHAPES = [
    Workload("team_7x7", 5, 16, 7, 7, 5, 1, "f32", 51),
    Workload("team_7x7_L2", 3, 8, 7, 7, 5, 2, "f32", 52),          # 7 -> 4 -> 2
    Workload("team_8x8_L3", 2, 8, 8, 8, 5, 3, "f32", 53),          # grids shrink to 1 x 1
    Workload("team_9x9_L2", 4, 8, 9, 9, 5, 2, "f32", 54),          # 9 -> 5 -> 3, odd at every level
    Workload("team_5x10", 3, 8, 5, 10, 5, 1, "f32", 55),           # non-square
    Workload("team_base_only", 2, 8, 6, 6, 5, 0, "f32", 56),
    Workload("team_many_groups", 37, 24, 7, 7, 5, 1, "f32", 57),   # several channel groups per block, ragged unit ranges
]
TEAM_PATHS = [pytest.param(0, id="team"), pytest.param(wt.FLAG_NO_TEAM, id="plane"), pytest.param(wt.FLAG_TILED_ONLY, id="tiled")]


@pytest.mark.parametrize("flags", TEAM_PATHS)
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
@pytest.mark.parametrize("wl", TEAM_SHAPES, ids=lambda w: w.name)
def test_tiny_planes(wl, dtype, flags):
    wl = wl.with_(dtype=dtype)
    I = inputs.make_inputs(wl, bias=True)
    name = wt.wtconv_plan_name(wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, dtype, flags))
    if flags == 0:  # a group of planes must be a 16-byte multiple: not every 16-bit shape qualifies
        assert name == "team" or (dtype != "f32" and name == "plane")
    else:
        assert name == {wt.FLAG_NO_TEAM: "plane", wt.FLAG_TILED_ONLY: "tiled"}[flags]
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("wl", [SMALL[1], SMALL[4], SMALL[9]], ids=lambda w: w.name)
def test_bias(wl, flags):
    I = inputs.make_inputs(wl, bias=True)
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("wl", [SMALL[1], SMALL[4], SMALL[9], SMALL[10], SMALL[11], SMALL[13]], ids=lambda w: w.name)
def test_small_16bit(wl, dtype, flags):
    wl = wl.with_(dtype=dtype)
    I = inputs.make_inputs(wl)  # x, g already rounded to the storage type
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))


@pytest.mark.parametrize("flags", PATHS)
@pytest.mark.parametrize("shape", [(7, 7, 2), (29, 29, 4), (57, 33, 3), (56, 56, 3), (14, 14, 1), (28, 28, 2), (7, 7, 1, 8),
                                   (9, 9, 3, 4)])
def test_index_and_padding_math_bit_exact(shape, flags):
    """Dyadic inputs make every intermediate exact in fp32, so out and grad_x must equal the
    oracle bit for bit whatever the summation order; any difference is an index/sign/padding bug."""
    H, W, L = shape[:3]
    wl = Workload("dyadic", 2, shape[3] if len(shape) > 3 else 3, H, W, 5, L, "f32", 30)  # 8 / 4 channels: the team kernels' groups
    I = inputs.make_dyadic_inputs(wl, bias=True)
    out, gr = run_gpu(wl, I, flags)
    rout, rgr = run_oracle(wl, I)
    assert np.array_equal(out, rout)
    assert np.array_equal(gr["dx"], rgr["dx"])
    for n in ("dw0", "ds0", "db0", "dwl", "dsl"):  # sums of a few thousand exact terms stay exact here too
        assert np.array_equal(gr[n], rgr[n]), n


def test_level_shape_export_matches_ceil():
    for H, W in [(56, 56), (7, 7), (225, 225), (13, 9), (1, 1)]:
        d = wt.make_desc(1, 1, H, W, 5, 0, "f32")
        for l in range(0, 9):
            assert wt.wtconv_level_shape(d, l) == (-(-H // 2 ** l), -(-W // 2 ** l))
