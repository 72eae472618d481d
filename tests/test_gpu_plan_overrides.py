"""Launch-plan overrides of the block-per-plane kernels (WTCONV_TUNE* bits of desc.flags): every alternative plan -
split backward instead of the fused one, no bulk-copy prefetch, 4- or 8-row register tiles - must compute the same
operator as the planner's own choice, so each is compared with the fp64 oracle on the network's plane sizes."""
import pytest

from paper_2608_10805_b200 import inputs
from paper_2608_10805_b200 import wtconv as wt
from paper_2608_10805_b200.inputs import Workload

from helpers import assert_close, run_gpu, run_oracle

pytestmark = pytest.mark.gpu

NO_BULK, NO_FUSED_BWD, TILE_8, TILE_4 = 1 << 28, 1 << 29, 1 << 30, 1 << 31
SHAPES = [Workload("s56", 3, 4, 56, 56, 5, 3, "f32", 61), Workload("s28", 3, 6, 28, 28, 5, 2, "bf16", 62),
          Workload("s7", 5, 16, 7, 7, 5, 1, "bf16", 63), Workload("s64", 2, 3, 64, 64, 5, 5, "f16", 64)]
OVERRIDES = [NO_BULK, NO_FUSED_BWD, TILE_8, TILE_4, NO_BULK | NO_FUSED_BWD, TILE_4 | NO_FUSED_BWD, TILE_8 | NO_BULK]


@pytest.mark.parametrize("tune", OVERRIDES, ids=lambda t: "tune_%08x" % t)
@pytest.mark.parametrize("wl", SHAPES, ids=lambda w: w.name)
def test_overridden_plans_match_the_oracle(wl, tune):
    flags = tune | wt.FLAG_NO_TEAM  # the overrides address the block-per-plane kernels
    desc = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wl.dtype, flags)
    assert wt.wtconv_plan_name(desc) == "plane"
    text = wt.wtconv_plan_describe(desc)
    if tune & NO_FUSED_BWD:
        assert "split" in text, text
    if tune & NO_BULK:
        assert "ring=0" in text and "ring=1" not in text, text
    if tune & TILE_4:
        assert "th=4" in text and "th=8" not in text, text
    if tune & TILE_8:
        assert "th=8" in text and "th=4" not in text, text
    I = inputs.make_inputs(wl, bias=True)
    assert_close(wl, run_gpu(wl, I, flags), run_oracle(wl, I))
