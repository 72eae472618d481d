"""Pins for the fp64 CPU oracle: every check here compares the oracle with something
that is NOT the oracle's own code - the Haar matrix of Proposition 1, a brute-force
evaluator built from explicit Haar basis functions, perfect-reconstruction closed
forms, Proposition 2's bit-indexed sum, Eq. 8/9 (scale folding), Algorithm 1 restated
with torch's fp64 library convolutions + autograd, central finite differences and the
adjoint identity.  A dropped term, wrong sign, wrong index or transposed operand in
the oracle fails at least one of them.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import wtconv_oracle as O

HAAR = 0.5 * np.array([[1, 1, 1, 1], [1, 1, -1, -1], [1, -1, 1, -1], [1, -1, -1, 1]], dtype=np.float64)  # Prop. 1


def rand_params(rng, C, k, L, bias=False):
    w0 = rng.normal(0, 0.1, (C, k, k))
    s0 = rng.uniform(0.5, 1.5, (C,))
    wl = rng.normal(0, 0.1, (L, C, 4, k, k))
    sl = rng.uniform(0.5, 1.5, (L, C, 4))
    b0 = rng.normal(0, 0.1, (C,)) if bias else None
    return w0, s0, b0, wl, sl


# ----------------------------------------------------------------------------- Haar pair
def test_haar_matrix_symmetric_self_inverse():
    assert np.array_equal(HAAR, HAAR.T)
    assert np.array_equal(HAAR @ HAAR, np.eye(4))


def test_analysis_is_haar_matrix_per_block():
    rng = np.random.default_rng(0)
    X = rng.integers(-8, 9, (6, 10)).astype(np.float64)
    Y = O.haar_analysis(X)
    for i in range(3):
        for j in range(5):
            blk = np.array([X[2 * i, 2 * j], X[2 * i, 2 * j + 1], X[2 * i + 1, 2 * j], X[2 * i + 1, 2 * j + 1]])
            assert np.array_equal(Y[:, i, j], HAAR @ blk)


def test_synthesis_follows_sign_table():
    # Appendix A sign table: rows (ry,rx) -> signs of (LH, HL, HH)
    table = {(0, 0): (1, 1, 1), (0, 1): (1, -1, -1), (1, 0): (-1, 1, -1), (1, 1): (-1, -1, 1)}
    T = np.array([3.0, 5.0, 7.0, 11.0]).reshape(4, 1, 1)
    R = O.haar_synthesis(T, 2, 2)
    for (ry, rx), (a, b, c) in table.items():
        assert R[ry, rx] == 0.5 * (3.0 + a * 5.0 + b * 7.0 + c * 11.0)


@pytest.mark.parametrize("H,W", [(8, 8), (7, 7), (13, 9), (1, 1), (2, 5)])
def test_single_level_perfect_reconstruction_exact(H, W):
    rng = np.random.default_rng(1)
    X = rng.integers(-100, 101, (H, W)).astype(np.float64)
    assert np.array_equal(O.haar_synthesis(O.haar_analysis(X), H, W), X)


@pytest.mark.parametrize("H,W,l", [(56, 56, 3), (7, 7, 2), (225, 225, 5), (13, 9, 3), (5, 1, 4)])
def test_level_shape_is_ceil(H, W, l):
    assert O.level_shape(H, W, l) == (-(-H // 2 ** l), -(-W // 2 ** l))


def test_odd_edge_coefficients_are_not_zero():
    # last row of an odd plane pads c=d=0: LL = LH = (a+b)/2, HL = HH = (a-b)/2
    X = np.arange(15, dtype=np.float64).reshape(3, 5)
    Y = O.haar_analysis(X)
    a, b = X[2, 0], X[2, 1]
    assert Y[0, 1, 0] == 0.5 * (a + b) and Y[1, 1, 0] == 0.5 * (a + b)
    assert Y[2, 1, 0] == 0.5 * (a - b) and Y[3, 1, 0] == 0.5 * (a - b)


# ----------------------------------------------------------------------------- conv
def test_corr2d_is_cross_correlation_not_convolution():
    X = np.zeros((5, 5)); X[2, 2] = 1.0
    w = np.arange(9, dtype=np.float64).reshape(3, 3)
    out = O.corr2d_same(X, w)
    # impulse response of a cross-correlation is the 180-degree rotated kernel
    assert np.array_equal(out[1:4, 1:4], w[::-1, ::-1])


@pytest.mark.parametrize("k", [3, 5, 7])
def test_corr2d_matches_torch_conv2d(k):
    rng = np.random.default_rng(2)
    X = rng.normal(size=(9, 12)); w = rng.normal(size=(k, k))
    ref = F.conv2d(torch.from_numpy(X)[None, None], torch.from_numpy(w)[None, None], padding=k // 2)[0, 0].numpy()
    np.testing.assert_allclose(O.corr2d_same(X, w), ref, rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------- brute force
def _sigma(sub, l, y, x):
    sy = -1.0 if (y >> (l - 1)) & 1 else 1.0
    sx = -1.0 if (x >> (l - 1)) & 1 else 1.0
    return (1.0, sy, sx, sy * sx)[sub]


def brute_force_forward(x, w0, s0, b0, wl, sl, L):
    """Direct evaluation from explicit Haar basis functions psi_{l,sub,i,j} = 2^-l * sigma_sub on
    the 2^l x 2^l block (i,j) (zero outside the image); no cascade anywhere."""
    B, C, H, W = x.shape
    k = w0.shape[-1]; R = k // 2
    out = np.zeros_like(x)
    for b in range(B):
        for c in range(C):
            xp = x[b, c]
            acc = np.zeros((H, W))
            for y in range(H):
                for xx in range(W):
                    t = 0.0
                    for u in range(k):
                        for v in range(k):
                            yy, xv = y + u - R, xx + v - R
                            if 0 <= yy < H and 0 <= xv < W:
                                t += w0[c, u, v] * xp[yy, xv]
                    acc[y, xx] = s0[c] * (t + (b0[c] if b0 is not None else 0.0))
            for l in range(1, L + 1):
                Hl, Wl = -(-H // 2 ** l), -(-W // 2 ** l)
                Y = np.zeros((4, Hl, Wl))
                for sub in range(4):
                    for y in range(H):
                        for xx in range(W):
                            Y[sub, y >> l, xx >> l] += 2.0 ** -l * _sigma(sub, l, y, xx) * xp[y, xx]
                Z = np.zeros((4, Hl, Wl))
                for sub in range(4):
                    for i in range(Hl):
                        for j in range(Wl):
                            t = 0.0
                            for u in range(k):
                                for v in range(k):
                                    ii, jj = i + u - R, j + v - R
                                    if 0 <= ii < Hl and 0 <= jj < Wl:
                                        t += wl[l - 1, c, sub, u, v] * Y[sub, ii, jj]
                            Z[sub, i, j] = sl[l - 1, c, sub] * t
                for y in range(H):
                    for xx in range(W):
                        for sub in range(4):
                            acc[y, xx] += 2.0 ** -l * _sigma(sub, l, y, xx) * Z[sub, y >> l, xx >> l]
            out[b, c] = acc
    return out


@pytest.mark.parametrize("shape,k,L,bias", [((1, 2, 16, 16), 5, 2, False), ((1, 2, 7, 7), 5, 2, True),
                                            ((2, 1, 13, 9), 3, 3, False), ((1, 1, 6, 10), 7, 1, True),
                                            ((1, 1, 5, 3), 5, 3, False)])
def test_forward_matches_basis_function_brute_force(shape, k, L, bias):
    rng = np.random.default_rng(3)
    x = rng.normal(size=shape)
    w0, s0, b0, wl, sl = rand_params(rng, shape[1], k, L, bias)
    np.testing.assert_allclose(O.forward(x, w0, s0, b0, wl, sl, L), brute_force_forward(x, w0, s0, b0, wl, sl, L),
                               rtol=0, atol=1e-13)


# ----------------------------------------------------------------------------- identity-conv closed forms
def _delta(k):
    d = np.zeros((k, k)); d[k // 2, k // 2] = 1.0
    return d


@pytest.mark.parametrize("H,W", [(8, 8), (7, 9)])
def test_identity_conv_single_level_returns_input(H, W):
    rng = np.random.default_rng(4)
    C, k = 2, 5
    x = rng.integers(-50, 51, (1, C, H, W)).astype(np.float64)
    w0 = np.zeros((C, k, k)); s0 = np.ones(C)
    wl = np.broadcast_to(_delta(k), (1, C, 4, k, k)).copy(); sl = np.ones((1, C, 4))
    assert np.array_equal(O.forward(x, w0, s0, None, wl, sl, 1), x)


@pytest.mark.parametrize("H,W,L", [(16, 16, 3), (13, 9, 3), (7, 7, 2)])
def test_multilevel_haar_perfect_reconstruction(H, W, L):
    # delta on every high band, delta on LL of the deepest level only: standard multi-level Haar PR
    rng = np.random.default_rng(5)
    C, k = 1, 3
    x = rng.integers(-50, 51, (1, C, H, W)).astype(np.float64)
    wl = np.zeros((L, C, 4, k, k)); wl[:, :, 1:] = _delta(k); wl[L - 1, :, 0] = _delta(k)
    out = O.forward(x, np.zeros((C, k, k)), np.ones(C), None, wl, np.ones((L, C, 4)), L)
    assert np.array_equal(out, x)


@pytest.mark.parametrize("H,W,L", [(16, 16, 3), (13, 9, 3)])
def test_identity_everywhere_adds_block_means(H, W, L):
    # delta on every band: out = x + sum_{l=1}^{L-1} 2^-l * X^l[y>>l, x>>l], X^l = 2^-l * (zero-padded block sum)
    rng = np.random.default_rng(6)
    C, k = 1, 5
    x = rng.integers(-50, 51, (1, C, H, W)).astype(np.float64)
    wl = np.broadcast_to(_delta(k), (L, C, 4, k, k)).copy()
    out = O.forward(x, np.zeros((C, k, k)), np.ones(C), None, wl, np.ones((L, C, 4)), L)
    expect = x.copy()
    for l in range(1, L):
        s = 2 ** l
        Hp, Wp = -(-H // s) * s, -(-W // s) * s
        xp = np.zeros((Hp, Wp)); xp[:H, :W] = x[0, 0]
        bs = xp.reshape(Hp // s, s, Wp // s, s).sum(axis=(1, 3))  # block sums
        expect[0, 0] += (4.0 ** -l) * np.kron(bs, np.ones((s, s)))[:H, :W]
    assert np.array_equal(out, expect)


# ----------------------------------------------------------------------------- Prop. 2: closed form = cascade
def closed_form_synthesis(Z, H, W):
    y = np.arange(H)[:, None]; x = np.arange(W)[None, :]
    R = np.zeros((H, W))
    for l, z in enumerate(Z, 1):
        sy = 1.0 - 2.0 * ((y >> (l - 1)) & 1); sx = 1.0 - 2.0 * ((x >> (l - 1)) & 1)
        i, j = y >> l, x >> l
        R += 2.0 ** -l * (z[0][i, j] + sy * z[1][i, j] + sx * z[2][i, j] + sy * sx * z[3][i, j])
    return R


@pytest.mark.parametrize("H,W,L", [(16, 16, 4), (7, 7, 2), (13, 9, 4), (25, 25, 5), (10, 6, 3), (56, 56, 3)])
def test_cascade_equals_bit_indexed_closed_form(H, W, L):
    rng = np.random.default_rng(7)
    Z = [rng.normal(size=(4,) + O.level_shape(H, W, l)) for l in range(1, L + 1)]
    np.testing.assert_allclose(O.synthesis_cascade(Z, H, W), closed_form_synthesis(Z, H, W), rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- Eq. 8 / Eq. 9
def test_scale_folding_forward_and_gradients():
    rng = np.random.default_rng(8)
    B, C, H, W, k, L = 2, 3, 10, 7, 5, 2
    x = rng.normal(size=(B, C, H, W)); g = rng.normal(size=(B, C, H, W))
    w0, s0, b0, wl, sl = rand_params(rng, C, k, L, bias=True)
    out = O.forward(x, w0, s0, b0, wl, sl, L)
    w0f, b0f, wlf = w0 * s0[:, None, None], b0 * s0, wl * sl[..., None, None]
    one0, onel = np.ones_like(s0), np.ones_like(sl)
    np.testing.assert_allclose(O.forward(x, w0f, one0, b0f, wlf, onel, L), out, rtol=0, atol=1e-13)
    gr = O.backward(x, g, w0, s0, b0, wl, sl, L)
    gf = O.backward(x, g, w0f, one0, b0f, wlf, onel, L)  # gradients w.r.t. the folded parameters
    np.testing.assert_allclose(gr["dx"], gf["dx"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(gr["dw0"], s0[:, None, None] * gf["dw0"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(gr["db0"], s0 * gf["db0"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(gr["ds0"], (gf["dw0"] * w0).sum((1, 2)) + gf["db0"] * b0, rtol=0, atol=1e-12)
    np.testing.assert_allclose(gr["dwl"], sl[..., None, None] * gf["dwl"], rtol=0, atol=1e-12)
    np.testing.assert_allclose(gr["dsl"], (gf["dwl"] * wl).sum((3, 4)), rtol=0, atol=1e-12)


# ----------------------------------------------------------------------------- Algorithm 1 with library convolutions
def torch_reference(x, w0, s0, b0, wl, sl, L):
    """Algorithm 1 the way Sec. 3.1 says the reference runs it: Haar analysis as a grouped
    stride-2 conv2d against +-1/2 filters, depthwise conv2d, scale multiply, slice, add, cat,
    grouped conv_transpose2d; odd sizes zero-padded bottom/right and cropped after synthesis."""
    B, C, H, W = x.shape
    k = w0.shape[-1]
    filt = torch.tensor(HAAR, dtype=torch.float64).reshape(4, 1, 2, 2).repeat(C, 1, 1, 1)  # [4C,1,2,2], channel-major
    carrier, Zs, shapes = x, [], []
    for l in range(L):
        h, w = carrier.shape[-2:]
        shapes.append((h, w))
        xp = F.pad(carrier, (0, w % 2, 0, h % 2))
        Y = F.conv2d(xp, filt, stride=2, groups=C)                        # [B,4C,h/2,w/2]
        Zc = F.conv2d(Y, wl[l].reshape(4 * C, 1, k, k), padding=k // 2, groups=4 * C)
        Zs.append(Zc * sl[l].reshape(1, 4 * C, 1, 1))
        carrier = Y.reshape(B, C, 4, *Y.shape[-2:])[:, :, 0]
    Rn = None
    for l in reversed(range(L)):
        Z = Zs[l].reshape(B, C, 4, *Zs[l].shape[-2:])
        ll = Z[:, :, 0] + (Rn if Rn is not None else 0.0)
        T = torch.cat([ll[:, :, None], Z[:, :, 1:]], dim=2).reshape(B, 4 * C, *Z.shape[-2:])
        Rn = F.conv_transpose2d(T, filt, stride=2, groups=C)[..., :shapes[l][0], :shapes[l][1]]
    base = F.conv2d(x, w0.reshape(C, 1, k, k), padding=k // 2, groups=C)
    if b0 is not None:
        base = base + b0.reshape(1, C, 1, 1)
    out = base * s0.reshape(1, C, 1, 1)
    return out + Rn if Rn is not None else out


@pytest.mark.parametrize("shape,k,L,bias", [((2, 3, 16, 16), 5, 2, False), ((2, 3, 7, 7), 5, 2, True),
                                            ((1, 2, 13, 9), 3, 3, True), ((2, 2, 12, 20), 7, 2, False),
                                            ((1, 2, 29, 29), 5, 5, False), ((2, 2, 8, 8), 5, 0, True)])
def test_forward_and_all_gradients_match_torch_autograd(shape, k, L, bias):
    rng = np.random.default_rng(9)
    x = rng.normal(size=shape); g = rng.normal(size=shape)
    w0, s0, b0, wl, sl = rand_params(rng, shape[1], k, L, bias)
    t = {n: torch.tensor(v, dtype=torch.float64, requires_grad=True)
         for n, v in dict(x=x, w0=w0, s0=s0, wl=wl, sl=sl).items()}
    tb = torch.tensor(b0, dtype=torch.float64, requires_grad=True) if bias else None
    out = torch_reference(t["x"], t["w0"], t["s0"], tb, t["wl"], t["sl"], L)
    (out * torch.from_numpy(g)).sum().backward()
    np.testing.assert_allclose(O.forward(x, w0, s0, b0, wl, sl, L), out.detach().numpy(), rtol=0, atol=1e-12)
    gr = O.backward(x, g, w0, s0, b0, wl, sl, L)
    np.testing.assert_allclose(gr["dx"], t["x"].grad.numpy(), rtol=0, atol=1e-11)
    np.testing.assert_allclose(gr["dw0"], t["w0"].grad.numpy(), rtol=0, atol=1e-10)
    np.testing.assert_allclose(gr["ds0"], t["s0"].grad.numpy(), rtol=0, atol=1e-10)
    if bias:
        np.testing.assert_allclose(gr["db0"], tb.grad.numpy(), rtol=0, atol=1e-10)
    else:
        assert gr["db0"] is None
    if L > 0:
        np.testing.assert_allclose(gr["dwl"], t["wl"].grad.numpy(), rtol=0, atol=1e-10)
        np.testing.assert_allclose(gr["dsl"], t["sl"].grad.numpy(), rtol=0, atol=1e-10)


# ----------------------------------------------------------------------------- finite differences / adjoint
def test_gradients_match_central_finite_differences():
    rng = np.random.default_rng(10)
    B, C, H, W, k, L = 2, 2, 9, 6, 5, 3
    x = rng.normal(size=(B, C, H, W)); g = rng.normal(size=(B, C, H, W))
    w0, s0, b0, wl, sl = rand_params(rng, C, k, L, bias=True)
    P = dict(x=x, w0=w0, s0=s0, b0=b0, wl=wl, sl=sl)
    gr = O.backward(x, g, w0, s0, b0, wl, sl, L)

    def loss(**kw):
        q = dict(P); q.update(kw)
        return float((O.forward(q["x"], q["w0"], q["s0"], q["b0"], q["wl"], q["sl"], L) * g).sum())

    eps = 1e-3  # the map is linear in each argument: central differences are exact up to rounding
    for name, gname in [("x", "dx"), ("w0", "dw0"), ("s0", "ds0"), ("b0", "db0"), ("wl", "dwl"), ("sl", "dsl")]:
        a = P[name]
        idxs = [tuple(rng.integers(0, s) for s in a.shape) for _ in range(12)]
        for idx in idxs:
            ap, am = a.copy(), a.copy()
            ap[idx] += eps; am[idx] -= eps
            fd = (loss(**{name: ap}) - loss(**{name: am})) / (2 * eps)
            assert abs(fd - gr[gname][idx]) < 1e-8 * max(1.0, abs(fd)), (name, idx, fd, gr[gname][idx])


def test_adjoint_identity_in_x():
    # <g, J v> = <J^T g, v> where J = d out / d x (bias-free forward is linear in x)
    rng = np.random.default_rng(11)
    B, C, H, W, k, L = 1, 2, 11, 14, 5, 3
    v = rng.normal(size=(B, C, H, W)); g = rng.normal(size=(B, C, H, W))
    w0, s0, _, wl, sl = rand_params(rng, C, k, L)
    lhs = (g * O.forward(v, w0, s0, None, wl, sl, L)).sum()
    rhs = (O.backward(v, g, w0, s0, None, wl, sl, L)["dx"] * v).sum()
    assert abs(lhs - rhs) < 1e-10 * max(1.0, abs(lhs))


def test_grad_wrt_level_output_is_analysis_cascade_of_g():
    # with s=1 and W=delta the level conv is the identity, so dL/dZ^l = dL/dY^l(conv part); check via dsl:
    # dsl[l,c,sub] = <dZ^l, corr(Y^l, W)> = <analysis-cascade(g)^l, Y^l> when W = delta
    rng = np.random.default_rng(12)
    C, H, W, k, L = 1, 12, 8, 3, 2
    x = rng.normal(size=(1, C, H, W)); g = rng.normal(size=(1, C, H, W))
    wl = np.broadcast_to(_delta(k), (L, C, 4, k, k)).copy()
    gr = O.backward(x, g, np.zeros((C, k, k)), np.ones(C), None, wl, np.ones((L, C, 4)), L)
    cx, cg = x[0, 0], g[0, 0]
    for l in range(L):
        Y, D = O.haar_analysis(cx), O.haar_analysis(cg)
        np.testing.assert_allclose(gr["dsl"][l, 0], (Y * D).sum((1, 2)), rtol=0, atol=1e-12)
        cx, cg = Y[0], D[0]
