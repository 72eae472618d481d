"""The I/O-model calculator against the numbers the paper prints (Table 1, Sec. 1, Sec. 3)."""
import os

import pytest

from paper_2608_10805_b200 import io_model as M

G = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    for line in open(os.path.join(G, name)):
        line = line.split("#")[0].split()
        if line:
            out.append(line)
    return out


def test_table1_traffic():
    for L, qr, qf, ratio in _rows("paper_table1_traffic.txt"):
        L = int(L)
        assert abs(M.q_ref(L) - float(qr)) <= 0.0051
        assert abs(M.q_fused(L) - float(qf)) <= 0.0051
        assert abs(M.traffic_ratio(L) - float(ratio)) <= 0.0051


def test_printed_constants():
    c = {n: (float(v), float(t)) for n, v, t in _rows("paper_arithmetic_constants.txt")}
    chk = lambda name, val: abs(val - c[name][0]) <= c[name][1] + 1e-12 or pytest.fail("%s: %r vs %r" % (name, val, c[name]))
    chk("mac_k5_L1", M.mac(5, 1))
    chk("mac_k5_L5", M.mac(5, 5))
    chk("flop_k5_L5", 2 * M.mac(5, 5))
    chk("bytes_fp32_L5", 4 * M.q_ref(5))
    chk("intensity_k5_L5", M.intensity_ref(5, 5))
    chk("q_ref_limit", M.q_ref(60))
    chk("ratio_limit", M.traffic_ratio(60))
    chk("dw7_mac", 7 * 7)
    N = 8 * 64 * 256 * 256
    chk("example_N_millions", N / 1e6)
    chk("example_GB_moved", 4 * M.q_ref(5) * N / 1e9)


def test_exact_counts_reduce_to_model_on_power_of_two_shapes():
    B, C, H, W, k, L = 2, 3, 64, 64, 5, 4
    N = B * C * H * W
    assert M.conv_macs(B, C, H, W, k, L) == pytest.approx(N * k * k * (1 + M.level_sum(L)))
    assert M.level_shapes(225, 225, 5) == [(225, 225), (113, 113), (57, 57), (29, 29), (15, 15), (8, 8)]
    assert M.compulsory_bytes(N, 2, "fwd+bwd") == 10 * N
