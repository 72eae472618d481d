"""Seeded synthetic inputs and the named workloads.

This module holds no WTConv arithmetic: it only draws random tensors and lists
shapes, so that the CUDA library and the CPU oracle can be fed the very same
values.  Distributions follow the benchmark's recipe: activations and upstream
gradients ~ N(0,1); depthwise weights ~ N(0, std 0.1); per-channel scales ~
U(0.5, 1.5); no bias unless asked for.  Every tensor has its own Philox stream,
keyed by (workload seed, tensor index), so changing one shape never shifts
another tensor's values.
"""
from dataclasses import dataclass, replace

import numpy as np

_TENSOR_INDEX = {"x": 0, "g": 1, "w0": 2, "s0": 3, "wl": 4, "sl": 5, "b0": 6}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    C: int
    H: int
    W: int
    k: int
    L: int
    dtype: str  # "f32" | "f16" | "bf16"  (activation storage type; arithmetic is fp32)
    seed: int

    @property
    def N(self):
        return self.B * self.C * self.H * self.W

    def with_(self, **kw):
        return replace(self, **kw)


# The benchmark's configurations (WTConvNeXt-T stage shapes and the level sweep).
WORKLOADS = {
    "tiny": Workload("tiny", 1, 8, 16, 16, 5, 2, "f32", 0),
    "stage1_f32": Workload("stage1_f32", 64, 96, 56, 56, 5, 3, "f32", 1),
    **{"sweep_L%d_%s" % (L, dt): Workload("sweep_L%d_%s" % (L, dt), 32, 128, 64, 64, 5, L, dt, 2)
       for L in (1, 2, 3, 4, 5) for dt in ("f32", "f16")},
    "stage1_bf16": Workload("stage1_bf16", 128, 96, 56, 56, 5, 3, "bf16", 3),
    "stage2_bf16": Workload("stage2_bf16", 128, 192, 28, 28, 5, 2, "bf16", 3),
    "stage3_bf16": Workload("stage3_bf16", 128, 384, 14, 14, 5, 1, "bf16", 3),
    "stage4_bf16": Workload("stage4_bf16", 128, 768, 7, 7, 5, 1, "bf16", 3),
    # the network's own depth schedule, L = (5, 4, 3, 2) on the four stages: repeated odd padding 7 -> 4 -> 2
    "convnext_s1_bf16": Workload("convnext_s1_bf16", 64, 96, 56, 56, 5, 5, "bf16", 5),
    "convnext_s2_bf16": Workload("convnext_s2_bf16", 64, 192, 28, 28, 5, 4, "bf16", 5),
    "convnext_s3_bf16": Workload("convnext_s3_bf16", 64, 384, 14, 14, 5, 3, "bf16", 5),
    "convnext_s4_bf16": Workload("convnext_s4_bf16", 64, 768, 7, 7, 5, 2, "bf16", 5),
    # kernel-size variants of the stage-1 layer
    "stage1_k3_f32": Workload("stage1_k3_f32", 16, 96, 56, 56, 3, 3, "f32", 6),
    "stage1_k7_f32": Workload("stage1_k7_f32", 16, 96, 56, 56, 7, 3, "f32", 6),
    # the paper's traffic-validation shape (C = 128, 128 x 128, k = 5) at a batch that makes one tensor (268 MB) larger
    # than the 126 MB L2, so that DRAM counters see what the I/O model counts
    **{"traffic_L%d_f32" % L: Workload("traffic_L%d_f32" % L, 32, 128, 128, 128, 5, L, "f32", 7) for L in (1, 3, 5)},
    "large_f16": Workload("large_f16", 16, 256, 256, 256, 5, 5, "f16", 4),
    "large_odd_f16": Workload("large_odd_f16", 16, 256, 225, 225, 5, 5, "f16", 4),
}


def _rng(seed, tensor):
    return np.random.Generator(np.random.Philox(key=int(seed) * 16 + _TENSOR_INDEX[tensor]))


def round_to_dtype(a, dtype):
    """Round a float32 array to the activation dtype and widen back to float32 (exactly)."""
    if dtype == "f32":
        return a
    import torch
    td = {"f16": torch.float16, "bf16": torch.bfloat16}[dtype]
    return torch.from_numpy(a).to(td).to(torch.float32).numpy()


def make_inputs(wl, bias=False, channels=None):
    """Draw the tensors of a workload as float32 numpy arrays.

    x and g are already rounded to the workload's activation dtype (so a 16-bit
    run and the fp64 oracle consume identical values).  ``channels`` (a slice or
    index list) keeps only those channels of every tensor *after* drawing, so a
    channel subset has the same values as in the full tensor.
    """
    B, C, H, W, k, L = wl.B, wl.C, wl.H, wl.W, wl.k, wl.L
    x = _rng(wl.seed, "x").standard_normal((B, C, H, W), dtype=np.float32)
    g = _rng(wl.seed, "g").standard_normal((B, C, H, W), dtype=np.float32)
    w0 = (0.1 * _rng(wl.seed, "w0").standard_normal((C, k, k))).astype(np.float32)
    s0 = _rng(wl.seed, "s0").uniform(0.5, 1.5, (C,)).astype(np.float32)
    wl_ = (0.1 * _rng(wl.seed, "wl").standard_normal((L, C, 4, k, k))).astype(np.float32)
    sl = _rng(wl.seed, "sl").uniform(0.5, 1.5, (L, C, 4)).astype(np.float32)
    b0 = (0.1 * _rng(wl.seed, "b0").standard_normal((C,))).astype(np.float32) if bias else None
    x = round_to_dtype(x, wl.dtype)
    g = round_to_dtype(g, wl.dtype)
    if channels is not None:
        x, g = np.ascontiguousarray(x[:, channels]), np.ascontiguousarray(g[:, channels])
        w0, s0 = np.ascontiguousarray(w0[channels]), np.ascontiguousarray(s0[channels])
        wl_, sl = np.ascontiguousarray(wl_[:, channels]), np.ascontiguousarray(sl[:, channels])
        b0 = None if b0 is None else np.ascontiguousarray(b0[channels])
    return dict(x=x, g=g, w0=w0, s0=s0, b0=b0, wl=wl_, sl=sl)


def make_dyadic_inputs(wl, bias=False):
    """Inputs on which every intermediate is exactly representable in fp32.

    Activations and gradients are small integers, weights lie in {0, +-1/2, +-1, +-2}
    and scales in {1/2, 1, 2}; all Haar factors are powers of two.  Any summation
    order then gives the same bits, so a result that differs from the oracle at all
    exposes an index, padding or sign error rather than rounding.
    """
    B, C, H, W, k, L = wl.B, wl.C, wl.H, wl.W, wl.k, wl.L
    r = _rng(wl.seed + 1000, "x")
    x = r.integers(-4, 5, (B, C, H, W)).astype(np.float32)
    g = _rng(wl.seed + 1000, "g").integers(-4, 5, (B, C, H, W)).astype(np.float32)
    vals = np.array([0.0, 0.5, -0.5, 1.0, -1.0, 2.0, -2.0], dtype=np.float32)
    w0 = vals[_rng(wl.seed + 1000, "w0").integers(0, len(vals), (C, k, k))]
    wl_ = vals[_rng(wl.seed + 1000, "wl").integers(0, len(vals), (L, C, 4, k, k))]
    sv = np.array([0.5, 1.0, 2.0], dtype=np.float32)
    s0 = sv[_rng(wl.seed + 1000, "s0").integers(0, 3, (C,))]
    sl = sv[_rng(wl.seed + 1000, "sl").integers(0, 3, (L, C, 4))]
    b0 = vals[_rng(wl.seed + 1000, "b0").integers(0, len(vals), (C,))] if bias else None
    return dict(x=x, g=g, w0=w0, s0=s0, b0=b0, wl=wl_, sl=sl)
