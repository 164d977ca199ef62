"""Pins for the CPU oracle: hand-worked fixtures, closed forms, reductions to library routines,
brute-force structure identities and invariants.  None of these re-types the oracle's formula."""
import numpy as np
import pytest
import scipy.signal
import torch

import oracle
from paper_2006_09791_b200 import synth
from paper_2006_09791_b200.workloads import Layer

from golden_io import load_case, load_numbers

GOLDEN_CASES = ["fig3_shape_index_valued.txt", "delta_no_flip.txt", "ones_zero_padding.txt",
                "stride2_pad1.txt", "dilation2.txt", "two_groups_asymmetric.txt", "per_axis_stride_pad.txt",
                "per_axis_dilation.txt"]


def _axes(p, key):
    """A fixture gives one value for both axes (`stride 2`) or one per axis (`stride_h 2 stride_w 3`)."""
    return p[key] if key in p else (p[key + "_h"], p[key + "_w"])


@pytest.mark.parametrize("name", GOLDEN_CASES)
def test_hand_worked(name):
    x, w, p, y = load_case(name)
    got, macs = oracle.gconv_ref(x, w, _axes(p, "stride"), _axes(p, "pad"), _axes(p, "dilation"), p["groups"], return_macs=True)
    assert got.shape == y.shape
    np.testing.assert_array_equal(got, y)  # small integers: exact in fp64
    assert macs == y.size * w.shape[1] * w.shape[2] * w.shape[3]


def _rand(shape, seed, tid):
    return synth.uniform(shape, seed, tid)


def test_block_diagonal_equivalence():
    """A grouped convolution equals a standard one whose weight is block-diagonal, zero elsewhere.
    Adding exact zeros does not change an fp64 sum, so the two agree exactly."""
    for seed, (N, C_in, C_out, g, H, W, KH, KW, s, p, d) in enumerate([
            (2, 6, 4, 2, 5, 7, 3, 3, 1, 1, 1), (1, 8, 8, 4, 6, 5, 3, 2, 2, 1, 1), (1, 6, 9, 3, 7, 7, 3, 3, 1, 2, 2)]):
        Cg, Kg = C_in // g, C_out // g
        x = _rand((N, C_in, H, W), seed, 0)
        w = _rand((C_out, Cg, KH, KW), seed, 1)
        wbd = np.zeros((C_out, C_in, KH, KW), dtype=np.float32)
        for j in range(g):
            wbd[j * Kg:(j + 1) * Kg, j * Cg:(j + 1) * Cg] = w[j * Kg:(j + 1) * Kg]
        np.testing.assert_array_equal(oracle.gconv_ref(x, w, s, p, d, g), oracle.gconv_ref(x, wbd, s, p, d, 1))


def test_groups1_is_standard_convolution_scipy():
    """groups = 1, stride 1: each output plane is the sum over input channels of a 2-D 'valid'
    cross-correlation of the zero-padded plane (scipy.signal.correlate2d, a library routine)."""
    N, C_in, C_out, H, W, K, pad = 2, 3, 4, 6, 5, 3, 1
    x = _rand((N, C_in, H, W), 11, 0)
    w = _rand((C_out, C_in, K, K), 11, 1)
    xp = np.pad(x.astype(np.float64), ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    want = np.zeros((N, C_out, H, W))
    for n in range(N):
        for k in range(C_out):
            for c in range(C_in):
                want[n, k] += scipy.signal.correlate2d(xp[n, c], w[k, c].astype(np.float64), mode="valid")
    np.testing.assert_allclose(oracle.gconv_ref(x, w, 1, pad, 1, 1), want, rtol=0, atol=1e-13)


def test_depthwise_is_per_channel_correlation():
    """groups = C: channel c of y is the 2-D correlation of channel c of x with its own 3x3 filter."""
    N, C, H, W = 2, 5, 7, 6
    x = _rand((N, C, H, W), 12, 0)
    w = _rand((C, 1, 3, 3), 12, 1)
    got = oracle.gconv_ref(x, w, 1, 1, 1, C)
    for n in range(N):
        for c in range(C):
            want = scipy.signal.correlate2d(x[n, c].astype(np.float64), w[c, 0].astype(np.float64), mode="same")
            np.testing.assert_allclose(got[n, c], want, rtol=0, atol=1e-13)


def test_pointwise_is_per_group_matmul():
    """A 1x1 grouped convolution is one [Kg x Cg] . [Cg x HW] matrix product per (image, group)."""
    N, C_in, C_out, g, H, W = 2, 12, 8, 4, 5, 3
    Cg, Kg = C_in // g, C_out // g
    x = _rand((N, C_in, H, W), 13, 0)
    w = _rand((C_out, Cg, 1, 1), 13, 1)
    got = oracle.gconv_ref(x, w, 1, 0, 1, g)
    for n in range(N):
        for j in range(g):
            Xg = x[n, j * Cg:(j + 1) * Cg].reshape(Cg, H * W).astype(np.float64)
            Wg = w[j * Kg:(j + 1) * Kg, :, 0, 0].astype(np.float64)
            np.testing.assert_allclose(got[n, j * Kg:(j + 1) * Kg].reshape(Kg, H * W), Wg @ Xg, rtol=0, atol=1e-13)


@pytest.mark.parametrize("cfg", [
    (2, 8, 12, 2, 9, 7, 3, 3, 1, 1, 1), (1, 8, 8, 8, 8, 8, 3, 3, 2, 1, 1), (3, 4, 6, 2, 10, 11, 5, 3, 2, 2, 1),
    (1, 6, 6, 3, 9, 9, 3, 3, 1, 2, 2), (2, 16, 16, 1, 7, 7, 1, 1, 2, 0, 1), (1, 4, 8, 4, 12, 5, 3, 3, 3, 1, 1)])
def test_matches_torch_conv2d_float64(cfg):
    """General (stride, pad, dilation, groups): agreement with a library convolution run in fp64."""
    N, C_in, C_out, g, H, W, KH, KW, s, p, d = cfg
    x = _rand((N, C_in, H, W), 21, 0)
    w = _rand((C_out, C_in // g, KH, KW), 21, 1)
    want = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), None, s, p, d, g)
    got = oracle.gconv_ref(x, w, s, p, d, g)
    assert got.shape == tuple(want.shape)
    np.testing.assert_allclose(got, want.numpy(), rtol=0, atol=1e-12)


@pytest.mark.parametrize("cfg", [
    (2, 8, 12, 2, 9, 7, 3, 3, (2, 1), (1, 0), (1, 1)), (1, 6, 6, 3, 11, 8, 3, 2, (1, 3), (2, 1), (2, 1)),
    (2, 4, 8, 4, 7, 12, 1, 5, (1, 2), (0, 2), (1, 2)), (1, 8, 4, 1, 10, 6, 5, 1, (3, 1), (1, 0), (1, 1))])
def test_per_axis_parameters_match_torch_conv2d_float64(cfg):
    """stride, padding and dilation given per axis (S_h, S_w of Algorithm 1): agreement with a library convolution
    in fp64, and the transposed problem (x and w transposed, every pair swapped) gives the transposed result."""
    N, C_in, C_out, g, H, W, KH, KW, s, p, d = cfg
    x = _rand((N, C_in, H, W), 23, 0)
    w = _rand((C_out, C_in // g, KH, KW), 23, 1)
    want = torch.nn.functional.conv2d(torch.from_numpy(x).double(), torch.from_numpy(w).double(), None, s, p, d, g)
    got, macs = oracle.gconv_ref(x, w, s, p, d, g, return_macs=True)
    assert got.shape == tuple(want.shape)
    np.testing.assert_allclose(got, want.numpy(), rtol=0, atol=1e-12)
    assert macs == got.size * (C_in // g) * KH * KW
    swapped = oracle.gconv_ref(x.transpose(0, 1, 3, 2), w.transpose(0, 1, 3, 2), s[::-1], p[::-1], d[::-1], g)
    np.testing.assert_array_equal(swapped, got.transpose(0, 1, 3, 2))


def _im2col_matmul(x, w, stride, pad, dilation, groups):
    """A formulation that shares nothing with the oracle's loop nest: per group, the zero-padded input is unfolded
    into a [Cg*KH*KW, H_out*W_out] matrix with numpy slicing and multiplied by the [Kg, Cg*KH*KW] filter matrix."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w, np.float64)
    N, C_in, H, W = x.shape
    C_out, Cg, KH, KW = w.shape
    Kg = C_out // groups
    xp = np.pad(x, ((0, 0), (0, 0), (pad, pad), (pad, pad)))
    Ho = (H + 2 * pad - dilation * (KH - 1) - 1) // stride + 1
    Wo = (W + 2 * pad - dilation * (KW - 1) - 1) // stride + 1
    y = np.empty((N, C_out, Ho, Wo))
    for n in range(N):
        for g in range(groups):
            cols = np.stack([xp[n, g * Cg + c, r * dilation:r * dilation + (Ho - 1) * stride + 1:stride,
                                s * dilation:s * dilation + (Wo - 1) * stride + 1:stride].reshape(-1)
                             for c in range(Cg) for r in range(KH) for s in range(KW)])
            y[n, g * Kg:(g + 1) * Kg] = (w[g * Kg:(g + 1) * Kg].reshape(Kg, -1) @ cols).reshape(Kg, Ho, Wo)
    return y


def test_unfold_and_matmul_agrees():
    """The oracle against the im2col + matrix-product formulation of the same definition (Section II), over strides,
    paddings, dilations, unequal Cg and Kg and non-square kernels."""
    for seed, (N, C_in, C_out, g, H, W, KH, KW, s, p, d) in enumerate([
            (2, 8, 12, 2, 6, 5, 3, 2, 2, 1, 1), (1, 6, 6, 6, 9, 9, 3, 3, 1, 1, 1), (2, 4, 8, 1, 7, 10, 3, 3, 1, 2, 2),
            (1, 12, 6, 3, 11, 8, 5, 3, 3, 2, 1), (3, 16, 16, 4, 8, 8, 1, 1, 2, 0, 1)]):
        x = _rand((N, C_in, H, W), 131 + seed, 0)
        w = _rand((C_out, C_in // g, KH, KW), 131 + seed, 1)
        np.testing.assert_allclose(oracle.gconv_ref(x, w, s, p, d, g), _im2col_matmul(x, w, s, p, d, g), rtol=0, atol=1e-12)


def test_gspc_baseline_is_pinned_to_the_oracle():
    """The float32 CPU program of the paper's method (Algorithm 1, Section III-B: four stages, tiles T_I and T_O) that
    the benchmark times as its second CPU baseline computes the oracle's tensor, for tile pairs from (1, 1) up to the
    bounds of Eq. (1) (T_I = CPG, T_O = KPG); tile sizes that do not divide are rejected."""
    cases = [(2, 8, 12, 2, 6, 5, 3, 2, 2, 1, 1, [(1, 1), (2, 3), (4, 6), (4, 2)]),
             (1, 16, 16, 4, 14, 14, 3, 3, 1, 1, 1, [(1, 4), (4, 4), (2, 1)]),
             (3, 6, 6, 6, 8, 9, 3, 3, 2, 1, 1, [(1, 1)]),                      # depthwise: both tiles can only be 1
             (1, 32, 64, 1, 9, 9, 3, 3, 1, 2, 2, [(8, 16), (32, 64), (1, 8)])]
    for seed, (N, C_in, C_out, g, H, W, KH, KW, s, p, d, tiles) in enumerate(cases):
        x = _rand((N, C_in, H, W), 31 + seed, 0)
        w = _rand((C_out, C_in // g, KH, KW), 31 + seed, 1)
        want = oracle.gconv_ref(x, w, s, p, d, g)
        for T_I, T_O in tiles:
            wp = oracle.gspc_pack_kernels(w, g, T_I, T_O)
            for threads in (1, 3):
                got = oracle.gspc_forward(x, wp, w.shape, s, p, d, g, T_I, T_O, threads=threads)
                assert np.max(np.abs(got - want)) <= 1e-5 * np.max(np.abs(want)), (seed, T_I, T_O)
    with pytest.raises(ValueError):
        oracle.gspc_pack_kernels(np.zeros((12, 4, 3, 3), np.float32), 2, 3, 4)     # T_I = 3 does not divide CPG = 4
    # the Fig. 3 shape with its stated tile sizes T_I = T_O = 2 (small integers: exact in float32)
    x = np.arange(16, dtype=np.float32).reshape(1, 4, 2, 2)
    w = np.arange(32, dtype=np.float32).reshape(4, 2, 2, 2)
    got = oracle.gspc_forward(x, oracle.gspc_pack_kernels(w, 2, 2, 2), w.shape, 1, 0, 1, 2, 2, 2)
    np.testing.assert_array_equal(got.ravel(), [140, 364, 1836, 2572])


def test_mac_counter_closed_form_and_table1():
    """Eq. (2): the counter equals N*C_in*C_out*KH*KW*H_out*W_out/g, and Eq. (2) applied to a
    WRN-40-2 whose 3x3 convs are grouped C_in->C_in reproduces the row differences of the MAC
    column of Table I (the g-independent layers cancel)."""
    # (C, H_in, stride, count) of the grouped 3x3 layers of WRN-40-2 with every conv(Ci->Co)
    # replaced by grouped(Ci->Ci) + pointwise(Ci->Co): 6 blocks x 2 convs per stage.
    shapes = [(16, 32, 1, 1), (32, 32, 1, 11), (32, 32, 2, 1), (64, 16, 1, 11), (64, 16, 2, 1), (128, 8, 1, 11)]
    for C, HW, s, _ in shapes:  # counter vs closed form, on real runs at the cheapest group count
        L = Layer("t", 1, C, HW, HW, C, stride=s, groups=16)
        x = np.zeros((1, C, HW, HW), np.float32)
        w = np.zeros((C, C // 16, 3, 3), np.float32)
        _, macs = oracle.gconv_ref(x, w, s, 1, 1, 16, threads=4, return_macs=True)
        assert macs == L.macs == 1 * C * C * 9 * L.H_out * L.W_out // 16
    total = lambda g: sum(Layer("t", 1, C, HW, HW, C, stride=s, groups=g).macs * cnt for C, HW, s, cnt in shapes)
    printed = load_numbers("wrn_table1_macs.txt", "macs_millions")  # S, G2, G4, G8, G16
    for (ga, a), (gb, b) in zip([(2, printed[1]), (4, printed[2]), (8, printed[3])],
                                [(4, printed[2]), (8, printed[3]), (16, printed[4])]):
        assert abs((total(ga) - total(gb)) / 1e6 - (a - b)) < 0.011  # table is rounded to 0.01 M
    # S row: standard 3x3 convs Ci->Co without the pointwise layers G models add
    std = [(16, 32, 32, 1, 1), (32, 32, 32, 1, 11), (32, 64, 32, 2, 1), (64, 64, 16, 1, 11), (64, 128, 16, 2, 1),
           (128, 128, 8, 1, 11)]
    s_macs = sum(Layer("t", 1, ci, hw, hw, co, stride=s).macs * cnt for ci, co, hw, s, cnt in std)
    pw_macs = sum(Layer("t", 1, ci, hw // s, hw // s, co, KH=1, KW=1, pad=0).macs * cnt for ci, co, hw, s, cnt in std)
    assert abs((s_macs - total(2) - pw_macs) / 1e6 - (printed[0] - printed[1])) < 0.011


def test_invariants():
    N, C_in, C_out, g, H, W = 2, 8, 12, 4, 7, 6
    Cg, Kg = C_in // g, C_out // g
    x1, x2 = _rand((N, C_in, H, W), 41, 0), _rand((N, C_in, H, W), 42, 0)
    w1, w2 = _rand((C_out, Cg, 3, 3), 41, 1), _rand((C_out, Cg, 3, 3), 42, 1)
    f = lambda x, w: oracle.gconv_ref(x, w, 1, 1, 1, g)
    # linear in x and in w (values chosen so that the fp32 sums are exact: multiples of 2^-24 in [-2,2))
    np.testing.assert_allclose(f((x1 + x2) / 2, w1), (f(x1, w1) + f(x2, w1)) / 2, rtol=0, atol=1e-12)
    np.testing.assert_allclose(f(x1, (w1 + w2) / 2), (f(x1, w1) + f(x1, w2)) / 2, rtol=0, atol=1e-12)
    # batch independence
    np.testing.assert_array_equal(f(x1, w1)[1:2], f(x1[1:2], w1))
    # group independence: zeroing one group's filters zeroes exactly its output channels
    wz = w1.copy()
    wz[Kg:2 * Kg] = 0
    yz, y = f(x1, wz), f(x1, w1)
    assert np.all(yz[:, Kg:2 * Kg] == 0)
    np.testing.assert_array_equal(np.delete(yz, np.s_[Kg:2 * Kg], axis=1), np.delete(y, np.s_[Kg:2 * Kg], axis=1))
    # changing group 0's input channels changes only group 0's outputs
    xm = x1.copy()
    xm[:, :Cg] = x2[:, :Cg]
    np.testing.assert_array_equal(f(xm, w1)[:, Kg:], y[:, Kg:])
    assert np.any(f(xm, w1)[:, :Kg] != y[:, :Kg])
    # permuting the groups of x and w together permutes y's channel blocks
    perm = [2, 0, 3, 1]
    xp = np.concatenate([x1[:, j * Cg:(j + 1) * Cg] for j in perm], axis=1)
    wp = np.concatenate([w1[j * Kg:(j + 1) * Kg] for j in perm], axis=0)
    np.testing.assert_array_equal(f(xp, wp), np.concatenate([y[:, j * Kg:(j + 1) * Kg] for j in perm], axis=1))
    # all ones, no padding: every output is the tap count Cg*KH*KW
    ones = oracle.gconv_ref(np.ones((1, C_in, 5, 5), np.float32), np.ones((C_out, Cg, 3, 3), np.float32), 1, 0, 1, g)
    assert np.all(ones == Cg * 9)
    # shift equivariance in the interior (stride 1, no padding)
    xs = np.roll(x1, (1, 2), axis=(2, 3))
    a = oracle.gconv_ref(x1, w1, 1, 0, 1, g)
    b = oracle.gconv_ref(xs, w1, 1, 0, 1, g)
    np.testing.assert_array_equal(b[:, :, 1:, 2:], a[:, :, :-1, :-2])


def test_threads_do_not_change_the_result():
    x = _rand((3, 8, 9, 9), 51, 0)
    w = _rand((8, 2, 3, 3), 51, 1)
    np.testing.assert_array_equal(oracle.gconv_ref(x, w, 1, 1, 1, 4, threads=1), oracle.gconv_ref(x, w, 1, 1, 1, 4, threads=8))


def test_rejects_bad_problems():
    x = np.zeros((1, 6, 4, 4), np.float32)
    with pytest.raises(ValueError):
        oracle.gconv_ref(x, np.zeros((4, 2, 3, 3), np.float32), groups=4)  # 6 % 4 != 0
    with pytest.raises(ValueError):
        oracle.gconv_ref(x, np.zeros((6, 2, 5, 5), np.float32), groups=3)  # window larger than image
    assert oracle.out_dim(56, 3, 2, 1) == 28 and oracle.out_dim(7, 3, 1, 1) == 7 and oracle.out_dim(4, 3, 2, 1) == 2
