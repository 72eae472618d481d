"""The paper's I/O and arithmetic cost model, in units of N = B*C*H*W elements.

These are reporting formulas (the benchmark prints measured traffic next to them);
they are not used by any kernel.
  q_ref    Eq. 2  : HBM elements moved by the reference chain of framework primitives
  q_fused  Eq. 10 : HBM elements moved by the paper's fused design
  mac      Eq. 3  : multiply-accumulates of the reference (analysis and synthesis as 2x2 convs)
The exact per-shape counts below (conv_macs, compulsory_bytes) are this library's own
roofline inputs: they count the real level grids ceil(H/2^l) x ceil(W/2^l), so odd
sizes are handled, and only the k*k convolution taps.
"""


def level_sum(L):
    """sum_{l=1..L} N_l / N with N_l = N / 4^(l-1)  =  4/3 (1 - 4^-L)."""
    return 4.0 / 3.0 * (1.0 - 4.0 ** -L)


def q_ref(L):
    return 7.0 + (6.0 + 19.0 / 4.0) * level_sum(L)


def q_fused(L):
    return 4.0 + 13.0 / 3.0 * (1.0 - 4.0 ** -L) - 4.0 ** -L


def traffic_ratio(L):
    return q_ref(L) / q_fused(L)


def mac(k, L):
    return k * k + (k * k + 8) * level_sum(L)


def intensity_ref(k, L, elem_bytes=4):
    """FLOP per byte of the reference implementation (Eq. 4)."""
    return 2.0 * mac(k, L) / (elem_bytes * q_ref(L))


def level_shapes(H, W, L):
    """[(H_0,W_0), (H_1,W_1), ...]: H_l = ceil(H_{l-1} / 2)."""
    out = [(H, W)]
    for _ in range(L):
        H, W = (H + 1) // 2, (W + 1) // 2
        out.append((H, W))
    return out


def conv_macs(B, C, H, W, k, L):
    """k*k taps on the base grid and on the four subbands of every level grid (forward)."""
    shp = level_shapes(H, W, L)
    return B * C * k * k * (H * W + sum(4 * h * w for h, w in shp[1:]))


def algorithmic_flops(B, C, H, W, k, L, direction):
    """2 FLOP per tap MAC; backward repeats the forward taps twice (input gradient and
    weight gradient), so forward+backward is three times forward."""
    f = 2 * conv_macs(B, C, H, W, k, L)
    return {"fwd": f, "bwd": 2 * f, "fwd+bwd": 3 * f}[direction]


def compulsory_bytes(N, elem_bytes, direction):
    """Bytes the operator must move whatever the design: forward reads x and writes out;
    backward reads x and grad_out and writes grad_x (parameters are O(L*C*k^2))."""
    return {"fwd": 2, "bwd": 3, "fwd+bwd": 5}[direction] * N * elem_bytes
