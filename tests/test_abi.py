"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, and rejects bad arguments with the documented status codes before any launch."""
import ctypes
import os
import re

import pytest

from paper_2608_10805_b200 import build as wbuild
from paper_2608_10805_b200 import wtconv as wt

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    wbuild.build()
    return wt.lib()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "wtconv.h")).read()
    declared = set(re.findall(r"\b(wtconv_[a-z_0-9]+)\s*\(", hdr))
    assert declared == set(wt.EXPORTS), declared ^ set(wt.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    for code in range(0, 12):
        s = lib.wtconv_status_string(code)
        assert s and s != b"unknown status"
    assert lib.wtconv_status_string(99) == b"unknown status"


def test_level_shape_and_errors(lib):
    d = wt.make_desc(1, 1, 225, 225, 5, 5, "f16")
    assert [wt.wtconv_level_shape(d, l) for l in range(6)] == [(225, 225), (113, 113), (57, 57), (29, 29), (15, 15), (8, 8)]
    with pytest.raises(wt.WTConvError) as e:
        wt.wtconv_level_shape(d, 9)
    assert e.value.code == 4


@pytest.mark.parametrize("kw,code", [(dict(B=0), 2), (dict(H=0), 2), (dict(k=4), 3), (dict(k=9), 3), (dict(L=-1), 4),
                                     (dict(L=9), 4), (dict(dtype=7), 5)])
def test_descriptor_validation(lib, kw, code):
    base = dict(B=2, C=3, H=8, W=8, k=5, L=2, dtype=0, flags=0)
    base.update(kw)
    d = wt.Desc(**base)
    f, b = ctypes.c_size_t(), ctypes.c_size_t()
    assert lib.wtconv_workspace_bytes(ctypes.byref(d), ctypes.byref(f), ctypes.byref(b)) == code
    assert wt.wtconv_plan_name(d) is None


def test_argument_validation_happens_before_any_cuda_call(lib):
    d = wt.make_desc(2, 3, 8, 8, 5, 2, "f32")
    fb, bb = wt.wtconv_workspace_bytes(d)
    assert fb > 0 and bb >= fb
    buf = (ctypes.c_char * 4096)()
    a = ctypes.addressof(buf)
    a = (a + 255) // 256 * 256
    P = ctypes.c_void_p
    # NULL x
    assert lib.wtconv_forward(ctypes.byref(d), None, P(a), P(a), None, P(a), P(a), P(a + 1024), P(a), fb, None) == 1
    # misaligned activation pointer
    assert lib.wtconv_forward(ctypes.byref(d), P(a + 4), P(a), P(a), None, P(a), P(a), P(a + 2048), P(a), fb, None) == 6
    # workspace too small
    assert lib.wtconv_forward(ctypes.byref(d), P(a), P(a), P(a), None, P(a), P(a), P(a + 2048), P(a), fb - 1, None) == 7
    # out overlaps x
    assert lib.wtconv_forward(ctypes.byref(d), P(a), P(a), P(a), None, P(a), P(a), P(a + 16), P(a), fb, None) == 8
    # backward: bias and its gradient must come together
    args = [P(a), P(a), P(a), P(a), P(a), P(a), P(a), P(a + 2048), P(a), P(a), None, P(a), P(a)]
    assert lib.wtconv_backward(ctypes.byref(d), *args, P(a), bb, None) == 1


def test_plan_and_launch_count(lib):
    d = wt.make_desc(2, 3, 301, 301, 5, 3, "f32")  # rows that are not 16-byte multiples: window kernels
    assert wt.wtconv_plan_name(d) == "window"
    assert wt.wtconv_launch_count(d) == (4, 7)
    assert wt.wtconv_launch_count(wt.make_desc(2, 3, 301, 301, 5, 2, "f32")) == (1, 2)
    assert wt.wtconv_plan_name(wt.make_desc(2, 3, 300, 300, 5, 3, "f32")) == "tiled"
    assert wt.wtconv_plan_name(wt.make_desc(2, 3, 300, 300, 5, 3, "f32", wt.FLAG_PREFER_WINDOW)) == "window"
    dn = wt.make_desc(2, 3, 300, 300, 5, 3, "f32", wt.FLAG_NO_WINDOW)
    assert wt.wtconv_plan_name(dn) == "tiled"
    assert wt.wtconv_launch_count(dn) == (4, 5)
    dt = wt.make_desc(2, 3, 56, 56, 5, 3, "f32", wt.FLAG_TILED_ONLY)
    assert wt.wtconv_plan_name(dt) == "tiled"
    assert wt.wtconv_plan_name(wt.make_desc(2, 3, 56, 56, 7, 3, "f32")) == "tiled"  # k = 7: per-level kernels
    # k = 3 rides the k = 5 kernels (filters in zero-bordered 5 x 5 tables: one launch more forward, two backward,
    # the tables at the head of the workspace) unless the per-level kernels are asked for
    d3, d5 = wt.make_desc(2, 8, 56, 56, 3, 3, "f32"), wt.make_desc(2, 8, 56, 56, 5, 3, "f32")
    assert wt.wtconv_plan_name(d3) == wt.wtconv_plan_name(d5) == "plane"
    f5, b5 = wt.wtconv_launch_count(d5)
    assert wt.wtconv_launch_count(d3) == (f5 + 1, b5 + 2)
    tables = 2 * (8 * 25 * 4 + 3 * 8 * 4 * 25 * 4)  # parameters and their gradients, before 256-byte rounding
    w3, w5 = wt.wtconv_workspace_bytes(d3), wt.wtconv_workspace_bytes(d5)
    assert tables <= w3[0] - w5[0] <= tables + 4 * 256 and w3[1] - w5[1] == w3[0] - w5[0]
    assert wt.wtconv_plan_describe(d3).startswith("3x3 kernels in 5x5 tables: plane")
    d3t = wt.make_desc(2, 8, 56, 56, 3, 3, "f32", wt.FLAG_TILED_ONLY)
    assert wt.wtconv_plan_name(d3t) == "tiled" and wt.wtconv_launch_count(d3t) == (4, 5)


def test_scratch_memory_accounting(lib):
    """Device memory the layer needs beyond its inputs and outputs.  Whole-plane kernels keep every intermediate
    on chip: the forward needs only a status word and the backward its per-block gradient partials, a few
    MiB at most on every stage of the network (they fit the library's built-in scratch).  The tiled path keeps
    Z^l and the raw carriers in HBM: 4 + 1 float32 per level-l coefficient and plane (the carrier of the last level is not needed)."""
    from paper_2608_10805_b200 import inputs
    for name in ("stage1_f32", "stage1_bf16", "stage2_bf16", "stage3_bf16", "stage4_bf16",
                 "convnext_s1_bf16", "convnext_s2_bf16", "convnext_s3_bf16", "convnext_s4_bf16"):
        wl = inputs.WORKLOADS[name]
        d = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wl.dtype)
        assert wt.wtconv_plan_name(d) in ("plane", "team")
        fb, bb = wt.wtconv_workspace_bytes(d)
        assert fb == 256 and bb < (8 << 20), (name, fb, bb)
    wl = inputs.WORKLOADS["large_f16"]
    d = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wl.dtype, wt.FLAG_PREFER_WINDOW)
    assert wt.wtconv_plan_name(d) == "window"
    fb, bb = wt.wtconv_workspace_bytes(d)
    n16 = wl.N // 16 * 4  # one fp32 carrier-sized tensor (a sixteenth of the elements)
    assert 3 * n16 <= fb <= 3 * n16 + (8 << 20) and fb <= bb <= 3 * n16 + (16 << 20)  # X2, R3, G2: 0.75 B per element
    d = wt.make_desc(wl.B, wl.C, wl.H, wl.W, wl.k, wl.L, wl.dtype, wt.FLAG_NO_WINDOW)
    fb, _ = wt.wtconv_workspace_bytes(d)
    P, coeffs = wl.B * wl.C, 0
    for l in range(1, wl.L + 1):
        Hl, Wl = wt.wtconv_level_shape(d, l)
        coeffs += (4 + (1 if l < wl.L else 0)) * Hl * Wl
    assert abs(fb - 4 * P * coeffs) <= 4096 * (wl.L + 2), (fb, 4 * P * coeffs)


def test_host_planning_over_a_shape_sweep(lib):
    """The host-side planners (pure integer code) give a plan, a launch count and a workspace size for every
    shape in a sweep that crosses the plane / tiled boundary, odd sizes, L = 0 and grids that shrink to 1 x 1."""
    seen = set()
    for H, W in [(1, 1), (1, 19), (7, 7), (9, 12), (13, 9), (14, 14), (28, 28), (29, 29), (56, 56), (57, 33), (64, 64),
                 (70, 66), (71, 71), (96, 40), (128, 128), (225, 225)]:
        for L in (0, 1, 2, 3, 5, 8):
            for dt in ("f32", "bf16"):
                for B, C in ((1, 1), (2, 3), (64, 96), (128, 768)):
                    d = wt.make_desc(B, C, H, W, 5, L, dt)
                    name = wt.wtconv_plan_name(d)
                    assert name in ("team", "plane", "window", "tiled"), (H, W, L, dt, B, C, name)
                    seen.add(name)
                    nf, nb = wt.wtconv_launch_count(d)
                    if name == "team":
                        assert nf == 1 and nb == 2
                    elif name == "plane":
                        assert nf == 1 and nb in (2, 3)
                    elif name == "window":
                        assert (nf, nb) == ((4, 7) if L > 2 else (1, 2))
                    else:
                        assert nf == L + 1 and nb == L + 2
                    assert wt.wtconv_plan_describe(d).startswith(name)
                    fb, bb = wt.wtconv_workspace_bytes(d)
                    assert fb >= (256 if name != "tiled" else 0) and bb >= fb and bb > 0 and fb % 256 == 0 and bb % 256 == 0, (H, W, L, dt, B, C, fb, bb)
                    for lvl in range(L + 1):
                        assert wt.wtconv_level_shape(d, lvl) == (-(-H // (1 << lvl)), -(-W // (1 << lvl)))
    assert seen == {"team", "plane", "window", "tiled"}


def test_host_step_workspace_covers_its_batch_chunks(lib):
    """wtconv_step_host runs the kernels chunk by chunk on B / n images (n up to 8); the scratch a chunk needs is not
    monotone in B (the gradient partial slots depend on how blocks split the units), so the reported size must
    cover the chunk descriptor as well as the whole batch."""
    from paper_2608_10805_b200 import inputs
    shapes = [(96, 56, 56, 3), (192, 28, 28, 2), (384, 14, 14, 1), (768, 7, 7, 1), (512, 7, 7, 1), (128, 64, 64, 3)]
    for C, H, W, L in shapes:
        for dt, esz in (("f32", 4), ("bf16", 2)):
            for B in (8, 16, 32, 64, 96, 128, 192, 256, 384):
                d = wt.make_desc(B, C, H, W, 5, L, dt)
                total = wt.wtconv_step_host_workspace_bytes(d)
                act = -(-B * C * H * W * esz // 256) * 256
                par = sum(-(-n * 4 // 256) * 256 for n in (C * 25, C, C, L * C * 100, L * C * 4))
                scratch = total - 4 * act - 10 * par
                per_image = C * H * W * esz
                for n in (8, 4, 2):  # the library's chunking rule
                    if B % n == 0 and B // n >= 4 and (B // n * per_image) % 16 == 0 and B // n * per_image >= (4 << 20):
                        fb, bb = wt.wtconv_workspace_bytes(wt.make_desc(B // n, C, H, W, 5, L, dt))
                        assert max(fb, bb) <= scratch, (C, H, W, L, dt, B, n, max(fb, bb), scratch)
                        break
                fb, bb = wt.wtconv_workspace_bytes(d)
                assert max(fb, bb) <= scratch


def test_binding_refuses_to_run_without_the_library(monkeypatch):
    monkeypatch.setattr(wt, "_lib", None)
    monkeypatch.setattr(wt, "LIB_PATH", "/nonexistent/libwtconv_b200.so")
    with pytest.raises(OSError):
        wt.lib()
