"""torch.autograd front end of the WTConv library: an autograd Function and an nn.Module.

Marshalling only: forward calls `wtconv_forward`, backward calls `wtconv_backward` (which recomputes
everything it needs from x, so nothing but x and the parameters is kept between the two calls — the
on-chip recomputation of Sec. 4.1 applied to training memory).  Parameters are float32 in every
activation dtype.  The layer is Algorithm 1 of the paper: base depthwise conv with scale (and optional
bias) plus L Haar levels with their own depthwise convs and scales.
"""
import collections

import torch

from . import wtconv as wt


class _StatusWatch:
    """Deferred check of the kernels' device status word, without synchronising.

    After every library call the status word of its workspace is copied (asynchronously, on the same stream) into
    a pinned host integer and an event is recorded.  Later calls look at the copies whose events have completed
    and raise if one is non-zero: a bounded device-side wait ran out in that earlier call and its outputs were not
    valid.  `drain()` waits for everything outstanding (call it before trusting results at the end of a run)."""

    def __init__(self):
        self.pending = collections.deque()
        self.free = []

    def after_call(self, desc, ws):
        flag = self.free.pop() if self.free else torch.zeros(1, dtype=torch.int32).pin_memory()
        wt.wtconv_read_status(desc, ws, flag)
        ev = torch.cuda.Event()
        ev.record()
        self.pending.append((ev, flag))
        self.poll()

    def poll(self, wait=False):
        while self.pending and (wait or self.pending[0][0].query()):
            ev, flag = self.pending.popleft()
            if wait:
                ev.synchronize()
            bad = int(flag[0]) != 0
            self.free.append(flag)
            if bad:
                raise wt.WTConvError(11, "a bounded device-side wait ran out in an earlier WTConv call; its outputs are not valid")

    def drain(self):
        self.poll(wait=True)


status_watch = _StatusWatch()


class WTConvFunction(torch.autograd.Function):
    """out = WTConv(x; w0, s0, b0, wl, sl).  b0 may be None.  k and L are read from wl's shape."""

    @staticmethod
    def forward(ctx, x, w0, s0, b0, wl, sl):
        if not x.is_cuda:
            raise RuntimeError("WTConvFunction runs on CUDA tensors only (there is no CPU path)")
        x = x.contiguous()
        B, C, H, W = x.shape
        k, L = w0.shape[-1], wl.shape[0]
        desc = wt.make_desc(B, C, H, W, k, L, x.dtype)
        params = [p.detach().float().contiguous() for p in (w0, s0, wl, sl)]
        b0c = None if b0 is None else b0.detach().float().contiguous()
        out = torch.empty_like(x)
        ws = wt.alloc_workspace(desc, x.device)
        wt.wtconv_forward(desc, x, params[0], params[1], b0c, params[2], params[3], out, ws)
        status_watch.after_call(desc, ws)
        ctx.desc, ctx.ws, ctx.has_bias = desc, ws, b0 is not None
        ctx.save_for_backward(x, params[0], params[1], b0c if b0c is not None else x.new_empty(0), params[2], params[3])
        return out

    @staticmethod
    def backward(ctx, grad_out):
        x, w0, s0, b0, wl, sl = ctx.saved_tensors
        b0 = b0 if ctx.has_bias else None
        g = grad_out.contiguous()
        gx = torch.empty_like(x)
        gw0, gs0, gwl, gsl = (torch.empty_like(t) for t in (w0, s0, wl, sl))
        gb0 = torch.empty_like(b0) if b0 is not None else None
        wt.wtconv_backward(ctx.desc, x, g, w0, s0, b0, wl, sl, gx, gw0, gs0, gb0, gwl, gsl, ctx.ws)
        status_watch.after_call(ctx.desc, ctx.ws)
        return gx, gw0, gs0, gb0, gwl, gsl


class WTConv2d(torch.nn.Module):
    """Depthwise wavelet convolution layer (Algorithm 1): `channels` planes, kernel size k in {3, 5, 7},
    `levels` Haar levels.  Initialisation follows the benchmark's recipe: weights N(0, 0.1), level scales
    0.1, base scale 1 — any other initialisation can be written into the parameters afterwards."""

    def __init__(self, channels, kernel_size=5, levels=1, bias=True, device="cuda"):
        super().__init__()
        k, C, L = kernel_size, channels, levels
        self.channels, self.kernel_size, self.levels = C, k, L
        P = torch.nn.Parameter
        self.w0 = P(0.1 * torch.randn(C, k, k, device=device))
        self.s0 = P(torch.ones(C, device=device))
        self.b0 = P(torch.zeros(C, device=device)) if bias else None
        self.wl = P(0.1 * torch.randn(L, C, 4, k, k, device=device))
        self.sl = P(torch.full((L, C, 4), 0.1, device=device))

    def forward(self, x):
        return WTConvFunction.apply(x, self.w0, self.s0, self.b0, self.wl, self.sl)
