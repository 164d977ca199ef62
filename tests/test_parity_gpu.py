"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same seeded
inputs, element by element over the whole tensor.  Bar: max|y-y_ref|/max|y_ref| <= 1e-5 for the
FP32 variants and <= 5e-3 for the TF32 variant."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_09791_b200 import build as gbuild
from paper_2006_09791_b200 import gconv, synth
from paper_2006_09791_b200.torch_util import attach_workspace
from paper_2006_09791_b200.workloads import (Layer, config0, depthwise5x5_layers, mobilenetv2_dw_layers, resnet34_layers, resnext_layers,
                                             sweep_layers, wrn_stack)

from golden_io import load_case
from gpu_util import check_layer, rel_err, run_layer

pytestmark = pytest.mark.gpu

ALL_VARIANTS = [gconv.GCONV_VARIANT_DIRECT_GENERIC, gconv.GCONV_VARIANT_DIRECT_TILED, gconv.GCONV_VARIANT_IGEMM_TF32]


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _supported(L, v):
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        return gconv.gconv_variant_supported(d, v)
    finally:
        gconv.gconv_desc_destroy(d)


@pytest.mark.parametrize("name", ["fig3_shape_index_valued.txt", "delta_no_flip.txt", "ones_zero_padding.txt",
                                  "stride2_pad1.txt", "dilation2.txt", "two_groups_asymmetric.txt"])
def test_hand_worked_cases_on_gpu(name):
    x, w, p, y_want = load_case(name)
    N, C_in, H, W = x.shape
    C_out, _, KH, KW = w.shape
    L = Layer(name, N, C_in, H, W, C_out, KH, KW, p["stride"], p["pad"], p["dilation"], p["groups"])
    for v in ALL_VARIANTS:
        if _supported(L, v):
            y, _ = run_layer(L, x, w, v)
            np.testing.assert_allclose(y, y_want, rtol=1e-6, atol=0)


PER_AXIS = [  # N, C_in, H, W, C_out, KH, KW, (stride), (pad), (dilation), groups
    (2, 16, 19, 33, 32, 3, 3, (2, 1), (1, 1), (1, 1), 4), (3, 8, 14, 40, 8, 3, 3, (1, 2), (0, 1), (1, 1), 8),
    (1, 32, 28, 28, 64, 1, 7, (1, 1), (0, 3), (1, 1), 2), (2, 32, 28, 28, 32, 7, 1, (2, 1), (3, 0), (1, 1), 1),
    (2, 12, 23, 17, 18, 3, 5, (3, 2), (2, 1), (2, 1), 3), (1, 64, 56, 56, 64, 3, 3, (1, 1), (2, 1), (2, 1), 16),
    (65, 4, 9, 130, 4, 3, 3, (1, 3), (1, 0), (1, 2), 1)]


@pytest.mark.parametrize("cfg", PER_AXIS)
def test_per_axis_stride_padding_dilation(cfg):
    """gconv_desc_create_2d (S_h and S_w of Algorithm 1 given separately) against the oracle's per-axis sum, whole
    tensor, FP32 tolerance; the hand-worked per-axis fixtures exactly."""
    N, C_in, H, W, C_out, KH, KW, st, pd, dl, g = cfg
    x, w = synth.make_layer_tensors(N, C_in, H, W, C_out, KH, KW, g, synth.layer_seed(3, N, C_in, H, g))
    y, used = _run_2d(x, w, st, pd, dl, g)
    assert used == gconv.GCONV_VARIANT_DIRECT_GENERIC
    y_ref = oracle.gconv_ref(x, w, st, pd, dl, g, threads=8)
    assert y.shape == y_ref.shape
    assert rel_err(y, y_ref) <= gconv.VARIANT_TOLERANCE[used]


PER_AXIS_STRIDE_TC = [  # N, C_in, H, W, C_out, (stride), groups: 3x3, pad 1, a stride of 2 on one axis, planes the tensor-core tilings address
    (4, 32, 32, 32, 64, (2, 1), 2), (3, 64, 56, 56, 64, (1, 2), 4), (2, 128, 28, 28, 128, (2, 1), 8), (5, 64, 16, 16, 64, (1, 2), 1),
    (6, 128, 8, 8, 128, (2, 1), 4), (2, 64, 64, 64, 64, (2, 1), 1), (3, 16, 20, 24, 32, (1, 2), 2), (1, 8, 12, 128, 8, (2, 1), 1),
    (2, 64, 56, 56, 128, (1, 2), 1), (9, 32, 15, 32, 32, (2, 1), 8), (40, 256, 56, 56, 256, (1, 2), 1)]


@pytest.mark.parametrize("cfg", PER_AXIS_STRIDE_TC)
def test_per_axis_stride_on_the_tensor_core_variant(cfg):
    """S_h != S_w (Algorithm 1) with strides of 1 and 2: the tensor-core variant computes the stride-1 layer and stores its
    even rows or columns; whole tensor against the per-axis oracle at the TF32 tolerance."""
    N, C_in, H, W, C_out, st, g = cfg
    x, w = synth.make_layer_tensors(N, C_in, H, W, C_out, 3, 3, g, synth.layer_seed(4, N, C_in, H, g))
    y, used = _run_2d(x, w, st, (1, 1), (1, 1), g)
    assert used == gconv.GCONV_VARIANT_IGEMM_TF32
    y_ref = oracle.gconv_ref(x, w, st, (1, 1), (1, 1), g, threads=16)
    assert y.shape == y_ref.shape and np.all(np.isfinite(y))
    assert rel_err(y, y_ref) <= gconv.VARIANT_TOLERANCE[used]


@pytest.mark.parametrize("name", ["per_axis_stride_pad.txt", "per_axis_dilation.txt"])
def test_per_axis_hand_worked_cases_on_gpu(name):
    x, w, p, y_want = load_case(name)
    y, _ = _run_2d(x, w, (p["stride_h"], p["stride_w"]), (p["pad_h"], p["pad_w"]), (p["dilation_h"], p["dilation_w"]), p["groups"])
    np.testing.assert_allclose(y, y_want, rtol=1e-6, atol=0)


def _run_2d(x_np, w_np, st, pd, dl, g):
    dev = torch.device("cuda:0")
    N, C_in, H, W = x_np.shape
    C_out, _, KH, KW = w_np.shape
    d = gconv.gconv_desc_create_2d(N, C_in, H, W, C_out, KH, KW, st[0], st[1], pd[0], pd[1], dl[0], dl[1], g)
    try:
        Ho, Wo = gconv.gconv_out_shape(d)
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        y = torch.full((N, C_out, Ho, Wo), float("nan"), dtype=torch.float32, device=dev)
        gconv.gconv_pack_weights(d, torch.from_numpy(w_np).to(dev), wp, None)
        gconv.gconv_forward(d, torch.from_numpy(x_np).to(dev), wp, y, None)
        assert gconv.gconv_last_status(d, None) == gconv.GCONV_OK
        return y.cpu().numpy(), gconv.gconv_variant(d)
    finally:
        gconv.gconv_desc_destroy(d)


def test_config0_every_variant():
    (L,) = config0()
    ran = 0
    for v in ALL_VARIANTS:
        if _supported(L, v):
            check_layer(L, v)
            ran += 1
    assert ran >= 1
    check_layer(L)


ODD_SHAPES = [
    # N, C_in, H, W, C_out, KH, KW, stride, pad, dil, groups
    (2, 6, 13, 11, 9, 3, 3, 1, 1, 1, 3), (1, 8, 17, 19, 8, 3, 3, 2, 1, 1, 8), (3, 4, 9, 33, 12, 3, 3, 1, 1, 1, 2),
    (1, 10, 7, 7, 10, 3, 3, 1, 1, 1, 10), (2, 12, 21, 5, 6, 5, 3, 2, 2, 1, 3), (1, 16, 12, 12, 32, 1, 1, 1, 0, 1, 4),
    (1, 6, 15, 15, 6, 3, 3, 1, 2, 2, 2), (2, 32, 16, 16, 32, 3, 3, 1, 1, 1, 2), (1, 48, 20, 24, 96, 3, 3, 1, 1, 1, 3),
    (2, 64, 14, 14, 64, 3, 3, 1, 1, 1, 1), (1, 32, 7, 7, 32, 3, 3, 1, 1, 1, 1), (1, 24, 56, 56, 24, 3, 3, 2, 1, 1, 24),
    (5, 3, 37, 41, 3, 3, 3, 1, 1, 1, 3), (1, 4, 64, 130, 4, 3, 3, 1, 1, 1, 4), (2, 16, 33, 35, 16, 3, 3, 2, 1, 1, 4),
    (2, 16, 33, 36, 24, 3, 3, 2, 1, 1, 2), (1, 32, 31, 32, 32, 3, 3, 2, 1, 1, 1), (3, 8, 16, 16, 16, 3, 3, 2, 1, 1, 1),
    (1, 64, 9, 64, 64, 3, 3, 2, 1, 1, 4), (2, 96, 10, 8, 96, 3, 3, 1, 1, 1, 1), (1, 128, 6, 128, 128, 3, 3, 1, 1, 1, 2),
    (2, 12, 13, 12, 12, 3, 3, 2, 1, 1, 12), (1, 8, 9, 128, 8, 3, 3, 1, 1, 1, 8), (3, 20, 57, 56, 20, 3, 3, 1, 1, 1, 20),
    (2, 6, 30, 28, 6, 3, 3, 2, 1, 1, 6), (1, 40, 5, 4, 40, 3, 3, 1, 1, 1, 40), (2, 7, 3, 8, 7, 3, 3, 2, 1, 1, 7),
    (3, 16, 14, 14, 32, 3, 3, 2, 1, 1, 2), (2, 8, 7, 7, 8, 3, 3, 1, 1, 1, 1), (1, 32, 9, 30, 32, 3, 3, 1, 1, 1, 4),
    (2, 24, 5, 6, 24, 3, 3, 1, 1, 1, 3), (1, 16, 21, 50, 16, 3, 3, 2, 1, 1, 2), (2, 8, 3, 126, 8, 3, 3, 1, 1, 1, 1),
    (2, 9, 14, 14, 9, 3, 3, 1, 1, 1, 9), (1, 5, 7, 7, 5, 3, 3, 1, 1, 1, 5), (2, 6, 15, 13, 6, 3, 3, 2, 1, 1, 6),
    (1, 4, 9, 250, 4, 3, 3, 2, 1, 1, 4), (1, 3, 6, 127, 3, 3, 3, 1, 1, 1, 3),
    (2, 40, 12, 16, 72, 3, 3, 1, 1, 1, 1), (1, 24, 28, 28, 88, 3, 3, 1, 1, 1, 1), (2, 48, 8, 8, 120, 3, 3, 2, 1, 1, 3),
    (1, 160, 16, 32, 160, 3, 3, 1, 1, 1, 5), (3, 36, 6, 44, 36, 3, 3, 1, 1, 1, 9), (1, 12, 64, 64, 12, 3, 3, 1, 1, 1, 6),
    (1, 1, 1, 1, 1, 1, 1, 1, 0, 1, 1), (1, 2, 3, 3, 2, 3, 3, 1, 0, 1, 2), (1, 16, 8, 8, 16, 3, 3, 1, 1, 1, 16),
    # stride 2 on tall planes of odd width that take the padded copy
    (2, 32, 48, 15, 32, 3, 3, 2, 1, 1, 2), (1, 128, 57, 29, 128, 3, 3, 2, 1, 1, 4), (2, 16, 70, 27, 32, 3, 3, 2, 1, 1, 1),
    # degenerate planes: one pixel, one row, one column, an output of one pixel
    (2, 8, 1, 1, 8, 3, 3, 1, 1, 1, 2), (1, 8, 1, 9, 16, 3, 3, 1, 1, 1, 1), (1, 16, 2, 2, 16, 3, 3, 2, 1, 1, 4), (3, 8, 1, 7, 8, 3, 3, 1, 1, 1, 8),
    (2, 8, 9, 1, 8, 3, 3, 1, 1, 1, 8), (1, 32, 1, 32, 32, 3, 3, 1, 1, 1, 2), (2, 6, 2, 14, 6, 5, 5, 2, 2, 1, 6), (1, 4, 28, 28, 4, 5, 5, 1, 2, 1, 4),
]


@pytest.mark.parametrize("cfg", ODD_SHAPES)
def test_odd_shapes_every_variant(cfg):
    L = Layer("odd", *cfg)
    for v in [gconv.GCONV_VARIANT_AUTO] + ALL_VARIANTS:
        if v == gconv.GCONV_VARIANT_AUTO or _supported(L, v):
            check_layer(L, v, seed=7)


# Larger row-box layers (several tiles per CTA, ragged last row block, odd number of row blocks, width 56 with two
# segments per row, stride 2): narrow merged groups, a 64-wide group with one big resident filter bank, streamed filter
# banks with two and four filter tiles.
LARGE_ROWBOX_SHAPES = [
    (12, 128, 56, 56, 128, 3, 3, 1, 1, 1, 4), (44, 64, 56, 56, 64, 3, 3, 1, 1, 1, 1), (40, 256, 30, 28, 256, 3, 3, 1, 1, 1, 2),
    (24, 64, 54, 56, 64, 3, 3, 2, 1, 1, 8), (90, 32, 28, 40, 32, 3, 3, 1, 1, 1, 2), (11, 128, 56, 52, 256, 3, 3, 1, 1, 1, 1),
]


@pytest.mark.parametrize("cfg", LARGE_ROWBOX_SHAPES)
def test_large_rowbox_shapes(cfg):
    check_layer(Layer("rowbox", *cfg), seed=11)


# Pair tiles (filter banks too large to stay resident, streamed once per two pixel tiles): an odd number of pixel tiles
# (the last pair's second tile is empty), two and four filter tiles, 28-wide rows (one segment) and 56-/40-wide rows (two
# segments), a group width that is a multiple of 16 but not of 32, a padded width (54 -> 56), two groups, an even count.
PAIR_TILE_SHAPES = [
    (23, 128, 26, 56, 128, 3, 3, 1, 1, 1, 1), (23, 128, 28, 28, 256, 3, 3, 1, 1, 1, 1), (61, 144, 10, 40, 128, 3, 3, 1, 1, 1, 1),
    (61, 128, 10, 54, 128, 3, 3, 1, 1, 1, 1), (12, 256, 56, 56, 256, 3, 3, 1, 1, 1, 2), (24, 128, 26, 56, 128, 3, 3, 1, 1, 1, 1),
]


@pytest.mark.parametrize("cfg", PAIR_TILE_SHAPES)
def test_pair_tile_shapes(cfg):
    err, used = check_layer(Layer("pair", *cfg), seed=3)
    assert used == gconv.GCONV_VARIANT_IGEMM_TF32


# Widths whose rows are not a multiple of 16 bytes, where the gather producer builds the stages (raw rows by bulk copy,
# copy warps shared memory to shared memory): even widths (8-byte accesses) and odd ones, planes that end inside a tile,
# batches that end inside a tile, many tiles per CTA, several groups per CTA, stride 2 on 7x7 planes.
COPY_WARP_SHAPES = [
    (5, 32, 14, 14, 32, 3, 3, 1, 1, 1, 4), (9, 64, 7, 7, 64, 3, 3, 1, 1, 1, 2), (2, 16, 17, 30, 16, 3, 3, 1, 1, 1, 2),
    (3, 24, 10, 6, 24, 3, 3, 1, 1, 1, 3), (4, 32, 15, 15, 32, 3, 3, 1, 1, 1, 1), (2, 8, 9, 31, 16, 3, 3, 1, 1, 1, 1),
    (7, 32, 7, 7, 32, 3, 3, 2, 1, 1, 4), (300, 64, 14, 14, 64, 3, 3, 1, 1, 1, 2), (40, 512, 14, 14, 512, 3, 3, 1, 1, 1, 32),
    (33, 256, 7, 7, 256, 3, 3, 1, 1, 1, 8), (1, 8, 5, 7, 8, 3, 3, 1, 1, 1, 1), (6, 48, 13, 14, 96, 3, 3, 1, 1, 1, 6),
    (3, 512, 56, 30, 512, 3, 3, 1, 1, 1, 64), (5, 32, 28, 31, 32, 3, 3, 1, 1, 1, 2), (2, 16, 8, 29, 16, 3, 3, 1, 1, 1, 1),   # halo stages
]


# More of the gather producer: stride 2 (even/odd column blocks) on 14x14, 7x7, 15x15, 30-wide and 13x9 planes, tiles
# made of two and of four whole images, a tile that is the short last one of its image, whole-plane bulk copies (planes
# that are not a multiple of 16 bytes) and boxes of a row range, two filter tiles per group, dilation, 8- and
# 16-channel stages, pointwise layers (centre tap only) with both strides, a batch that ends inside a tile.
GATHER_SHAPES = [
    (64, 256, 14, 14, 512, 3, 3, 2, 1, 1, 16), (9, 64, 14, 14, 128, 3, 3, 2, 1, 1, 2), (7, 32, 7, 7, 32, 3, 3, 2, 1, 1, 1),
    (5, 32, 15, 15, 64, 3, 3, 2, 1, 1, 2), (3, 16, 11, 30, 32, 3, 3, 2, 1, 1, 1), (6, 48, 13, 9, 96, 3, 3, 2, 1, 1, 6),
    (11, 32, 7, 6, 32, 3, 3, 2, 1, 1, 1), (4, 32, 19, 18, 32, 3, 3, 2, 1, 1, 1), (3, 24, 22, 22, 24, 3, 3, 1, 1, 1, 1),
    (2, 32, 30, 30, 32, 3, 3, 1, 1, 1, 2), (13, 8, 6, 6, 16, 3, 3, 1, 1, 1, 1), (3, 32, 14, 14, 128, 3, 3, 1, 1, 1, 1),
    (4, 32, 14, 14, 32, 3, 3, 1, 3, 3, 2), (3, 16, 15, 30, 64, 1, 1, 2, 0, 1, 1), (5, 24, 7, 7, 40, 1, 1, 1, 0, 1, 1),
    (2, 192, 15, 30, 1024, 1, 1, 2, 0, 1, 8), (33, 256, 14, 14, 512, 3, 3, 2, 1, 1, 8),
    # wide groups (one CTA per SM, eight copy warps): a resident bank, streamed banks shared by a pair of pixel tiles with an
    # odd and an even number of tiles, two filter tiles, stride 2 (8-channel stages), 7x7 planes (two images per tile)
    (300, 64, 14, 14, 64, 3, 3, 1, 1, 1, 1), (5, 128, 14, 14, 128, 3, 3, 1, 1, 1, 1), (6, 256, 14, 14, 128, 3, 3, 1, 1, 1, 2),
    (7, 128, 14, 14, 256, 3, 3, 2, 1, 1, 1), (9, 192, 7, 7, 64, 3, 3, 1, 1, 1, 1), (4, 64, 18, 18, 64, 3, 3, 1, 1, 1, 1),
    (3, 128, 15, 15, 64, 3, 3, 2, 1, 1, 1), (10, 64, 30, 30, 128, 3, 3, 1, 1, 1, 1),
    # stride 2 on tall planes of odd width: the raw part of a tile comes in several pieces, rows start at odd flat pixels, and an
    # (even, odd) column pair can straddle two pieces (narrow and wide groups)
    (2, 64, 64, 31, 64, 3, 3, 2, 1, 1, 1), (3, 32, 64, 31, 64, 3, 3, 2, 1, 1, 1), (3, 512, 64, 31, 512, 3, 3, 2, 1, 1, 4),
]


@pytest.mark.parametrize("cfg", GATHER_SHAPES)
def test_gather_producer_shapes(cfg):
    L = Layer("gather", *cfg)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32
        assert gconv.gconv_forward_launches(d) == 1 and gconv.gconv_workspace_bytes(d) == 0
    finally:
        gconv.gconv_desc_destroy(d)
    check_layer(L, seed=27)
    check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC, seed=27)


@pytest.mark.parametrize("cfg", COPY_WARP_SHAPES)
def test_copy_warp_producer_shapes(cfg):
    L = Layer("copywarp", *cfg)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32
        assert gconv.gconv_forward_launches(d) == 1          # no padding pass: the copy warps read the real rows
    finally:
        gconv.gconv_desc_destroy(d)
    check_layer(L, seed=23)


# Two filter tiles per group (80 filters: two tiles of 40) in the two-CTA launch shape, alone and with several groups,
# on segment tilings, row boxes and stride-2 row tiles.
TWO_FILTER_TILE_SHAPES = [
    (4, 16, 16, 16, 80, 3, 3, 1, 1, 1, 1), (40, 32, 16, 16, 160, 3, 3, 1, 1, 1, 2), (3, 16, 32, 32, 80, 3, 3, 1, 1, 1, 1),
    (130, 16, 8, 8, 80, 3, 3, 1, 1, 1, 1), (5, 16, 28, 28, 80, 3, 3, 1, 1, 1, 1), (6, 16, 32, 32, 80, 3, 3, 2, 1, 1, 1),
    (128, 64, 16, 16, 320, 3, 3, 2, 1, 1, 4),
]


@pytest.mark.parametrize("cfg", TWO_FILTER_TILE_SHAPES)
def test_two_filter_tiles_per_group(cfg):
    check_layer(Layer("nt2", *cfg), seed=37)


# Pointwise (1x1, pad 0) convolutions: the tensor-core variant runs them as the centre tap of a 3x3 filter.
POINTWISE_SHAPES = [
    (8, 64, 16, 16, 64, 1, 1, 1, 0, 1, 1), (3, 32, 32, 32, 128, 1, 1, 1, 0, 1, 1), (5, 256, 14, 14, 256, 1, 1, 1, 0, 1, 1),
    (4, 64, 16, 16, 128, 1, 1, 2, 0, 1, 1), (2, 256, 28, 28, 256, 1, 1, 1, 0, 1, 1), (130, 32, 32, 32, 32, 1, 1, 1, 0, 1, 4),
    (7, 128, 7, 7, 64, 1, 1, 1, 0, 1, 2), (2, 64, 56, 56, 256, 1, 1, 1, 0, 1, 1), (3, 48, 20, 24, 96, 1, 1, 2, 0, 1, 3),
]


@pytest.mark.parametrize("cfg", POINTWISE_SHAPES)
def test_pointwise_on_the_tensor_core_variant(cfg):
    L = Layer("pointwise", *cfg)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32
    finally:
        gconv.gconv_desc_destroy(d)
    check_layer(L, seed=41)
    check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC, seed=41)


def test_seeded_random_pointwise_shapes():
    """Pointwise layers drawn over plane sizes (re-cut planes, odd sizes, one-pixel rows), both strides, groups, narrow and
    wide filter tiles."""
    import random
    rng = random.Random(4242)
    done = 0
    while done < 40:
        g = rng.choice([1, 1, 1, 2, 4, 8])
        cg = rng.choice([8, 16, 24, 32, 64, 128, 256])
        kg = rng.choice([8, 16, 32, 40, 64, 80, 128, 256])
        C, K = g * cg, g * kg
        if C > 1024 or K > 1024:
            continue
        H = rng.choice([1, 4, 7, 8, 9, 14, 15, 16, 17, 28, 31, 32, 33, 56, 57])
        W = rng.choice([4, 6, 7, 8, 12, 14, 15, 16, 20, 28, 30, 32, 36, 56, 60, 64, 100, 128])
        stride = rng.choice([1, 1, 2])
        N = rng.choice([1, 2, 3, 5, 8, 33, 128])
        while N > 1 and (N * C * H * W > 8e6 or N * K * H * W > 8e6 or N * H * W * C * K > 4e9):
            N //= 2
        check_layer(Layer("randpw%d" % done, N, C, H, W, K, 1, 1, stride, 0, 1, g), seed=500 + done)
        done += 1


# Dilated 3x3 (pad = dilation) on the tensor-core variant: vertical taps become shifts by `dilation` rows, horizontal
# ones lane shifts by `dilation` columns inside a 32-pixel segment, so only planes whose rows divide 32 pixels
# (after padding the width to a multiple of 4) are taken: 32, 16 and 8 wide, 14 (copy warps) and 7.
DILATED_SHAPES = [
    (2, 32, 32, 32, 32, 3, 3, 1, 2, 2, 4), (3, 64, 16, 16, 64, 3, 3, 1, 2, 2, 2), (4, 128, 8, 8, 128, 3, 3, 1, 3, 3, 8),
    (5, 32, 14, 14, 32, 3, 3, 1, 2, 2, 4), (2, 64, 16, 16, 128, 3, 3, 1, 4, 4, 1), (2, 32, 7, 7, 32, 3, 3, 1, 2, 2, 1),
    (1, 16, 32, 32, 16, 3, 3, 1, 5, 5, 2), (130, 64, 32, 32, 64, 3, 3, 1, 2, 2, 8), (9, 32, 24, 16, 48, 3, 3, 1, 6, 6, 1),
    (3, 256, 14, 14, 256, 3, 3, 1, 2, 2, 1), (2, 16, 40, 8, 16, 3, 3, 1, 9, 9, 2),
]


@pytest.mark.parametrize("cfg", DILATED_SHAPES)
def test_dilated_shapes_on_the_tensor_core_variant(cfg):
    L = Layer("dilated", *cfg)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32
    finally:
        gconv.gconv_desc_destroy(d)
    check_layer(L, seed=29)
    check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC, seed=29)


def test_dilation_the_tensor_core_variant_does_not_take():
    """Rows that do not divide a segment, pad != dilation, stride 2: the selector falls back and the result still agrees."""
    for cfg in ((1, 16, 28, 28, 16, 3, 3, 1, 2, 2, 2), (1, 16, 16, 16, 16, 3, 3, 1, 1, 2, 2), (1, 16, 16, 16, 16, 3, 3, 2, 2, 2, 2)):
        L = Layer("dilated_fallback", *cfg)
        d = gconv.gconv_desc_create(*L.desc_args())
        try:
            assert gconv.gconv_variant(d) != gconv.GCONV_VARIANT_IGEMM_TF32
            assert not gconv.gconv_variant_supported(d, gconv.GCONV_VARIANT_IGEMM_TF32)
        finally:
            gconv.gconv_desc_destroy(d)
        check_layer(L, seed=30)


@pytest.mark.parametrize("groups", [1, 2, 4, 8, 16])
def test_wrn_stack_small_batch(groups):
    """Every distinct layer of the WRN-40-2-shaped stack at N = 1 and a ragged N = 3, all variants."""
    for N in (1, 3):
        for L in wrn_stack(groups, N):
            check_layer(L)
            for v in ALL_VARIANTS[1:]:
                if _supported(L, v):
                    check_layer(L, v)


@pytest.mark.parametrize("groups", [1, 2, 4, 8, 16, 32])
def test_resnet34_shapes(groups):
    for L in resnet34_layers(groups, 2):
        check_layer(L)


def test_resnext_shapes():
    for L in resnext_layers(N=1):
        check_layer(L)


def test_sweep_to_depthwise_small_batch():
    for L in sweep_layers(N=1):
        check_layer(L)


def test_mobilenetv2_depthwise_shapes():
    for L in mobilenetv2_dw_layers(N=2):
        check_layer(L)
        check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC)


def _seeded_random_shapes(seed, count):
    """3x3, pad = dilation layers drawn from the sizes the selector, the tilings and the kernel families branch on (plane
    sizes around the 32-pixel segment and the 128-pixel tile, widths that need padding or copy warps, narrow and wide
    groups, unequal Cg and Kg, both strides, dilation 1 to 3, ragged batches), each small enough for the oracle."""
    import random
    rng = random.Random(seed)
    out = []
    while len(out) < count:
        g = rng.choice([1, 1, 2, 2, 4, 4, 8, 16, 32, 64])
        cg = rng.choice([1, 2, 4, 8, 8, 16, 16, 32, 32, 64, 128])
        kg = rng.choice([cg, cg, cg, 2 * cg, max(1, cg // 2), 3 * cg // 2 if cg % 2 == 0 else cg])
        C, K = g * cg, g * kg
        if C > 512 or K > 512:
            continue
        H = rng.choice([3, 5, 7, 8, 9, 14, 15, 16, 17, 27, 28, 30, 31, 32, 33, 40, 55, 56, 57, 64, 75, 96, 113])
        W = rng.choice([3, 5, 6, 7, 8, 9, 11, 12, 13, 14, 15, 16, 17, 19, 20, 21, 23, 24, 25, 27, 28, 29, 30, 31, 32, 33, 35, 36, 40, 48, 52, 54,
                        56, 57, 60, 63, 64, 96, 127, 128])
        stride = rng.choice([1, 1, 1, 2])
        dil = rng.choice([1, 1, 1, 1, 2, 3])
        if H <= 2 * dil or W <= 2 * dil:
            dil = 1
        macs_per_image = C // g * K * 9 * ((H - 1) // stride + 1) * ((W - 1) // stride + 1)
        N = min(rng.choice([1, 2, 3, 5, 8, 13, 32, 64, 128, 200]), max(1, int(1.5e9 // macs_per_image)))
        if N * C * H * W > 40e6:
            continue
        out.append((N, C, H, W, K, 3, 3, stride, dil, dil, g))
    return out


@pytest.mark.parametrize("chunk", range(10))
def test_seeded_random_shapes(chunk):
    for i, cfg in enumerate(_seeded_random_shapes(20260 + chunk, 25)):
        check_layer(Layer("rand%d_%d" % (chunk, i), *cfg), seed=100 * chunk + i)


DW5_SHAPES = [
    # N, C, H, W, C_out, 5, 5, stride, pad 2, dilation 1, groups = C: widths around the 4- and 8-column strips, odd sizes
    (2, 8, 9, 7, 8, 5, 5, 1, 2, 1, 8), (1, 5, 13, 13, 5, 5, 5, 2, 2, 1, 5), (3, 16, 20, 24, 16, 5, 5, 1, 2, 1, 16),
    (2, 12, 17, 33, 12, 5, 5, 2, 2, 1, 12), (1, 4, 6, 128, 4, 5, 5, 1, 2, 1, 4), (2, 6, 5, 5, 6, 5, 5, 1, 2, 1, 6),
    (1, 3, 31, 64, 3, 5, 5, 2, 2, 1, 3), (2, 10, 12, 10, 10, 5, 5, 2, 2, 1, 10), (1, 7, 40, 36, 7, 5, 5, 1, 2, 1, 7),
]


@pytest.mark.parametrize("cfg", DW5_SHAPES)
def test_depthwise_5x5_shapes(cfg):
    L = Layer("dw5", *cfg)
    err, used = check_layer(L, seed=5)
    assert used == gconv.GCONV_VARIANT_DIRECT_TILED           # the stream kernel, not the generic fallback
    check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC, seed=5)


DW_PLANE_SHAPES = [
    # N, C, H, W, K, stride: depthwise on planes 7, 14 and 28 pixels wide (batches of whole planes through shared memory):
    # plane counts that are not a multiple of four or of the batch (a short last batch, or nothing but one), heights that
    # differ from the width, odd output heights, both filter sizes and strides
    (3, 5, 7, 7, 3, 1), (1, 3, 7, 7, 5, 1), (2, 6, 9, 14, 5, 2), (5, 7, 20, 28, 3, 2), (9, 33, 14, 14, 3, 1), (4, 9, 5, 7, 3, 2),
    (3, 4, 28, 28, 5, 2), (2, 64, 13, 14, 5, 1), (1, 2, 30, 28, 5, 1), (7, 11, 28, 28, 5, 1), (2, 50, 7, 7, 5, 2), (6, 96, 14, 14, 5, 2),
    (1, 1, 7, 7, 3, 1), (13, 20, 3, 14, 3, 1), (2, 130, 27, 28, 3, 2),
]


@pytest.mark.parametrize("cfg", DW_PLANE_SHAPES)
def test_depthwise_small_planes(cfg):
    N, C, H, W, K, stride = cfg
    L = Layer("dwp", N, C, H, W, C, K, K, stride, K // 2, 1, C)
    err, used = check_layer(L, seed=9)
    assert used == gconv.GCONV_VARIANT_DIRECT_TILED
    check_layer(L, gconv.GCONV_VARIANT_DIRECT_GENERIC, seed=9)


def test_depthwise_5x5_network_shapes():
    for L in depthwise5x5_layers(N=2):
        check_layer(L)


@pytest.mark.parametrize("shape", [(16, 32, 32, 32, 4), (8, 64, 16, 16, 2), (24, 128, 8, 8, 8), (6, 64, 28, 28, 1), (4, 16, 56, 56, 16),
                                   (4, 32, 14, 14, 4), (8, 32, 28, 28, 32), (3, 256, 14, 14, 1), (20, 64, 7, 7, 2)])
def test_dependent_chain_back_to_back(shape):
    """Five layers launched back to back on one stream, each reading the previous layer's output (the kernels start
    their set-up, weight fetch and an L2 prefetch before the previous kernel has finished, so this is the case that
    must not read early): once eagerly and once as a CUDA-graph replay over NaN-filled buffers.  Every layer's output
    is compared with the oracle applied to the input that layer actually saw on the GPU."""
    N, C, H, W, groups = shape
    L = Layer("chain", N, C, H, W, C, groups=groups)
    dev = torch.device("cuda:0")
    depth = 5
    x0, _ = synth.make_layer_tensors(N, C, H, W, C, 3, 3, groups, synth.layer_seed(31, N, C, groups))
    ws = [synth.make_layer_tensors(1, C, H, W, C, 3, 3, groups, synth.layer_seed(32, k, C, groups))[1] for k in range(depth)]
    descs = [gconv.gconv_desc_create(*L.desc_args()) for _ in range(depth)]
    try:
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            wss = [attach_workspace(d, dev) for d in descs]
            bufs = [torch.from_numpy(x0).to(dev)] + [torch.empty(L.y_elems, dtype=torch.float32, device=dev) for _ in range(depth)]
            wps = []
            for d, w in zip(descs, ws):
                wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
                gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp, stream)
                wps.append(wp)

            def run_chain():
                for k in range(depth):
                    gconv.gconv_forward(descs[k], bufs[k], wps[k], bufs[k + 1], stream)

            for use_graph in (False, True):
                for b in bufs[1:]:
                    b.fill_(float("nan"))
                if use_graph:
                    stream.synchronize()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        run_chain()
                    for b in bufs[1:]:
                        b.fill_(float("nan"))
                    graph.replay()
                else:
                    run_chain()
                stream.synchronize()
                for d in descs:
                    assert gconv.gconv_last_status(d, stream) == gconv.GCONV_OK
                outs = [bufs[0].cpu().numpy()] + [b.cpu().numpy().reshape(N, C, H, W) for b in bufs[1:]]
                for k in range(depth):
                    assert np.all(np.isfinite(outs[k + 1])), "layer %d wrote a non-finite value or skipped one" % k
                    ref = oracle.gconv_ref(outs[k].reshape(N, C, H, W), ws[k], 1, 1, 1, groups, threads=8)
                    err = rel_err(outs[k + 1], ref)
                    assert err <= gconv.VARIANT_TOLERANCE[gconv.gconv_variant(descs[k])], (k, use_graph, err)
    finally:
        for d in descs:
            gconv.gconv_desc_destroy(d)


def _stack_chain(layers, groups, seed, batches_checked):
    """Runs `layers` as a real chain (layer k reads layer k-1's output) on one stream, eagerly and as a CUDA-graph replay
    over NaN-filled buffers, and compares every layer's output with the oracle applied to the input that layer saw."""
    dev = torch.device("cuda:0")
    L0 = layers[0]
    x0, _ = synth.make_layer_tensors(L0.N, L0.C_in, L0.H, L0.W, L0.C_out, 3, 3, groups, synth.layer_seed(seed, L0.N, groups))
    ws = [synth.make_layer_tensors(1, L.C_in, L.H, L.W, L.C_out, 3, 3, groups, synth.layer_seed(seed + 1, k, groups))[1]
          for k, L in enumerate(layers)]
    descs = [gconv.gconv_desc_create(*L.desc_args()) for L in layers]
    try:
        stream = torch.cuda.Stream()
        with torch.cuda.stream(stream):
            wss = [attach_workspace(d, dev) for d in descs]
            bufs = [torch.from_numpy(x0).to(dev)] + [torch.empty(L.y_elems, dtype=torch.float32, device=dev) for L in layers]
            wps = []
            for d, w in zip(descs, ws):
                wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
                gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp, stream)
                wps.append(wp)

            def run_chain():
                for k, d in enumerate(descs):
                    gconv.gconv_forward(d, bufs[k], wps[k], bufs[k + 1], stream)

            for use_graph in batches_checked:
                for b in bufs[1:]:
                    b.fill_(float("nan"))
                if use_graph:
                    stream.synchronize()
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(graph, stream=stream):
                        run_chain()
                    for b in bufs[1:]:
                        b.fill_(float("nan"))
                    graph.replay()
                else:
                    run_chain()
                stream.synchronize()
                for d in descs:
                    assert gconv.gconv_last_status(d, stream) == gconv.GCONV_OK
                seen = bufs[0].cpu().numpy().reshape(L0.N, L0.C_in, L0.H, L0.W)
                for k, L in enumerate(layers):
                    got = bufs[k + 1].cpu().numpy().reshape(L.N, L.C_out, L.H_out, L.W_out)
                    assert np.all(np.isfinite(got)), "layer %d (%s) wrote a non-finite value or skipped one" % (k, L.name)
                    ref = oracle.gconv_ref(seen, ws[k], L.stride, L.pad, L.dilation, groups, threads=oracle.max_threads())
                    err = rel_err(got, ref)
                    assert err <= gconv.VARIANT_TOLERANCE[gconv.gconv_variant(descs[k])], (k, L.name, use_graph, err)
                    seen = got
    finally:
        for d in descs:
            gconv.gconv_desc_destroy(d)


@pytest.mark.parametrize("groups,N", [(1, 1), (2, 3), (4, 128), (8, 5), (16, 1), (1, 128)])
def test_wrn_stack_as_a_real_chain(groups, N):
    """The 18 layers of the WRN-40-2-shaped stack in network order -- six 32-channel layers at 32x32, the stride-2
    transition to 64 channels, five layers at 16x16, the stride-2 transition to 128 channels, five layers at 8x8 --
    each reading its predecessor's output.  This is the chain the bench replays at batch 1."""
    layers = []
    for L in wrn_stack(groups, N):
        layers.extend([L] * L.repeat)
    assert len(layers) == 18 and layers[6].stride == 2 and layers[12].stride == 2
    _stack_chain(layers, groups, 51, (False, True))


@pytest.mark.parametrize("groups,N", [(1, 1), (4, 2), (32, 1)])
def test_resnet34_stack_as_a_real_chain(groups, N):
    """The ResNet-34-shaped layers in network order (56x56 down to 7x7 through three stride-2 transitions), chained."""
    _stack_chain(resnet34_layers(groups, N), groups, 53, (False, True))


BLOCK_SHAPES = [
    # N, C_in of the grouped 3x3, H, W, groups, C2 (pointwise outputs) [, C_out of the grouped 3x3 if not C_in]
    (2, 32, 32, 32, 4, 32), (40, 32, 32, 32, 4, 32), (130, 32, 32, 32, 16, 48), (3, 64, 16, 16, 2, 64), (96, 64, 16, 16, 8, 128),
    (64, 128, 8, 8, 8, 128), (9, 64, 56, 56, 16, 64), (20, 128, 28, 28, 32, 64), (33, 96, 20, 24, 3, 80), (7, 64, 30, 60, 8, 16),
    (5, 32, 12, 56, 1, 32, 64), (1, 32, 8, 8, 32, 256), (12, 64, 16, 16, 2, 96, 128),
]


@pytest.mark.parametrize("cfg", BLOCK_SHAPES)
def test_fused_grouped_pointwise_block(cfg):
    """The paper's G(g) block in one kernel: grouped 3x3 then pointwise.  Compared with the oracle's grouped convolution
    (its fp64 result rounded to fp32, as the kernel keeps the intermediate in fp32) followed by its 1x1 convolution."""
    N, Cin, H, W, groups, C2 = cfg[:6]
    C = cfg[6] if len(cfg) > 6 else Cin                    # channels between the two convolutions
    L = Layer("block", N, Cin, H, W, C, groups=groups)
    dev = torch.device("cuda:0")
    x, w = synth.make_layer_tensors(N, Cin, H, W, C, 3, 3, groups, synth.layer_seed(41, N, C, groups))
    _, w2 = synth.make_layer_tensors(1, C, 1, 1, C2, 1, 1, 1, synth.layer_seed(42, C, C2))
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_block_supported(d, C2)
        guard, sentinel = 64, float(np.float32(-1.2345678e30))
        pb = gconv.gconv_block_packed_bytes(d, C2)
        wp_full = torch.full((pb // 4 + 2 * guard,), sentinel, dtype=torch.float32, device=dev)
        y_full = torch.full((N * C2 * H * W + 2 * guard,), sentinel, dtype=torch.float32, device=dev)
        wp, y2 = wp_full[guard:guard + pb // 4], y_full[guard:guard + N * C2 * H * W]
        gconv.gconv_block_pack_weights(d, C2, torch.from_numpy(w).to(dev), torch.from_numpy(w2.reshape(C2, C)).to(dev), wp)
        xd = torch.from_numpy(x).to(dev)
        gconv.gconv_block_forward(d, C2, xd, wp, y2)
        gconv.gconv_block_forward(d, C2, xd, wp, y2)          # back to back: the second starts before the first ends
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK
        for band in (wp_full[:guard], wp_full[-guard:], y_full[:guard], y_full[-guard:]):
            assert bool((band == sentinel).all()), "guard band overwritten"
        got = y2.cpu().numpy().reshape(N, C2, H, W)
        y1 = oracle.gconv_ref(x, w, 1, 1, 1, groups, threads=8)
        ref = oracle.gconv_ref(y1.astype(np.float32), w2, 1, 0, 1, 1, threads=8)
        assert np.all(np.isfinite(got))
        assert rel_err(got, ref) <= 5e-3
    finally:
        gconv.gconv_desc_destroy(d)


def test_fused_block_rejects_what_it_cannot_run():
    for cfg, C2 in (((1, 32, 32, 32, 32, 3, 3, 2, 1, 1, 4), 32), ((1, 32, 14, 14, 32, 3, 3, 1, 1, 1, 4), 32),
                    ((1, 32, 32, 32, 32, 3, 3, 1, 1, 1, 4), 24), ((1, 256, 28, 28, 256, 3, 3, 1, 1, 1, 32), 256),
                    ((1, 32, 32, 32, 32, 5, 5, 1, 2, 1, 32), 32), ((1, 32, 8, 8, 32, 3, 3, 1, 1, 1, 32), 272)):
        d = gconv.gconv_desc_create(*cfg)
        try:
            assert not gconv.gconv_block_supported(d, C2)
            assert gconv.gconv_block_packed_bytes(d, C2) == 0
        finally:
            gconv.gconv_desc_destroy(d)


def test_pack_mismatch_is_reported_not_fatal():
    (L,) = config0()
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, 5)
    dev = torch.device("cuda:0")
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        wp = torch.zeros(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)  # never packed
        y = torch.full((L.y_elems,), 7.0, dtype=torch.float32, device=dev)
        gconv.gconv_forward(d, torch.from_numpy(x).to(dev), wp, y)
        assert gconv.gconv_last_status(d) == gconv.GCONV_ERR_PACK_MISMATCH
        assert bool((y == 7.0).all())
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK  # reading clears it
        gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
        gconv.gconv_forward(d, torch.from_numpy(x).to(dev), wp, y)
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK
        y_ref = oracle.gconv_ref(x, w, 1, 1, 1, L.groups)
        assert rel_err(y.cpu().numpy().reshape(y_ref.shape), y_ref) <= gconv.VARIANT_TOLERANCE[gconv.gconv_variant(d)]
    finally:
        gconv.gconv_desc_destroy(d)


def test_weights_packed_under_another_batch_plane_or_stride():
    """The tensor-core variant's packed layout follows more than the filter shape (merge width and filter tile depend on
    the stride, the batch and the plane size).  Weights packed under a descriptor with the same filters but another
    batch, plane or stride must give either the right y or GCONV_ERR_PACK_MISMATCH with y untouched -- never a wrong y."""
    dev = torch.device("cuda:0")
    pairs = [
        # (descriptor the weights are packed under, descriptor that runs them)
        (Layer("pw_n1", 1, 128, 8, 8, 128, 1, 1, 1, 0, 1, 1), Layer("pw_n1024", 1024, 128, 8, 8, 128, 1, 1, 1, 0, 1, 1)),
        (Layer("g8_s1", 4, 64, 32, 32, 128, groups=8), Layer("g8_s2", 4, 64, 32, 32, 128, stride=2, groups=8)),
        (Layer("wide_n2", 2, 256, 56, 56, 256), Layer("wide_n32", 32, 256, 56, 56, 256)),
        (Layer("same_a", 2, 32, 32, 32, 32, groups=4), Layer("same_b", 7, 32, 16, 16, 32, groups=4)),
    ]
    outcomes = set()
    for La, Lb in pairs:
        x, w = synth.make_layer_tensors(Lb.N, Lb.C_in, Lb.H, Lb.W, Lb.C_out, Lb.KH, Lb.KW, Lb.groups, synth.layer_seed(61, Lb.N, Lb.H))
        da, db = gconv.gconv_desc_create(*La.desc_args()), gconv.gconv_desc_create(*Lb.desc_args())
        try:
            assert gconv.gconv_variant(da) == gconv.gconv_variant(db) == gconv.GCONV_VARIANT_IGEMM_TF32
            nb = max(gconv.gconv_packed_bytes(da), gconv.gconv_packed_bytes(db))
            wp = torch.zeros(nb // 4, dtype=torch.float32, device=dev)
            gconv.gconv_pack_weights(da, torch.from_numpy(w).to(dev), wp)
            y = torch.full((Lb.y_elems,), 7.0, dtype=torch.float32, device=dev)
            gconv.gconv_forward(db, torch.from_numpy(x).to(dev), wp, y)
            st = gconv.gconv_last_status(db)
            if st == gconv.GCONV_ERR_PACK_MISMATCH:
                assert bool((y == 7.0).all())
            else:
                assert st == gconv.GCONV_OK
                ref = oracle.gconv_ref(x, w, Lb.stride, Lb.pad, Lb.dilation, Lb.groups, threads=oracle.max_threads())
                assert rel_err(y.cpu().numpy().reshape(ref.shape), ref) <= gconv.VARIANT_TOLERANCE[gconv.GCONV_VARIANT_IGEMM_TF32]
            outcomes.add(st)
        finally:
            gconv.gconv_desc_destroy(da)
            gconv.gconv_desc_destroy(db)
    assert outcomes == {gconv.GCONV_OK, gconv.GCONV_ERR_PACK_MISMATCH}     # both outcomes occur among the pairs


def test_bounded_wait_runs_out_and_the_context_survives():
    """Failure path of the tensor-core kernel.  The test hook makes the first thread block's producer leave out one
    stage fill (nothing is issued, the barrier is never armed); the consumer's wait on it must give up after the time
    limit, the kernel must return with GCONV_ERR_TIMEOUT recorded, and the next ordinary forward of the same
    descriptor must be correct (tensor memory was freed, the context is intact).  Nothing faults, traps or hangs."""
    dev = torch.device("cuda:0")
    for L, skip in ((Layer("to_a", 8, 32, 32, 32, 32, groups=4), 0), (Layer("to_b", 6, 128, 28, 28, 128), 3)):
        x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, synth.layer_seed(63, L.N))
        d = gconv.gconv_desc_create(*L.desc_args())
        try:
            assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            xd = torch.from_numpy(x).to(dev)
            y = torch.zeros(L.y_elems, dtype=torch.float32, device=dev)
            gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
            gconv.gconv_desc_set_debug(d, wait_limit_us=2000, skip_stage=skip)
            t0 = torch.cuda.Event(enable_timing=True)
            t1 = torch.cuda.Event(enable_timing=True)
            t0.record()
            gconv.gconv_forward(d, xd, wp, y)
            t1.record()
            assert gconv.gconv_last_status(d) == gconv.GCONV_ERR_TIMEOUT
            assert t0.elapsed_time(t1) < 500.0            # a handful of 2 ms waits, not the default second, not forever
            assert gconv.gconv_last_status(d) == gconv.GCONV_OK       # reading clears it
            gconv.gconv_desc_set_debug(d, 0, -1)
            for _ in range(2):
                y.fill_(float("nan"))
                gconv.gconv_forward(d, xd, wp, y)
                assert gconv.gconv_last_status(d) == gconv.GCONV_OK
                ref = oracle.gconv_ref(x, w, 1, 1, 1, L.groups, threads=oracle.max_threads())
                assert rel_err(y.cpu().numpy().reshape(ref.shape), ref) <= gconv.VARIANT_TOLERANCE[gconv.GCONV_VARIANT_IGEMM_TF32]
        finally:
            gconv.gconv_desc_destroy(d)


def test_padded_copy_layers_need_an_attached_workspace():
    """Widths the bulk tensor copies cannot address that are too wide for the gather producer (more than 32 output columns):
    gconv_forward allocates nothing, it refuses to run until the caller attaches the workspace, then runs in two launches."""
    dev = torch.device("cuda:0")
    L = Layer("w54", 3, 128, 10, 54, 128, groups=1)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        need = gconv.gconv_workspace_bytes(d)
        if need == 0:
            pytest.skip("this build serves the shape without a workspace")
        x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, 71)
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        xd = torch.from_numpy(x).to(dev)
        y = torch.full((L.y_elems,), 7.0, dtype=torch.float32, device=dev)
        gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
        free0 = torch.cuda.mem_get_info()[0]
        with pytest.raises(gconv.GconvError) as e:
            gconv.gconv_forward(d, xd, wp, y)
        assert e.value.status == gconv.GCONV_ERR_WORKSPACE and bool((y == 7.0).all())
        ws = attach_workspace(d, dev)
        assert ws is not None and ws.numel() * 4 >= need
        free1 = torch.cuda.mem_get_info()[0]
        gconv.gconv_forward(d, xd, wp, y)
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK
        assert torch.cuda.mem_get_info()[0] == free1 and free1 <= free0     # the forward itself allocated nothing
        ref = oracle.gconv_ref(x, w, 1, 1, 1, L.groups, threads=oracle.max_threads())
        assert rel_err(y.cpu().numpy().reshape(ref.shape), ref) <= gconv.VARIANT_TOLERANCE[gconv.gconv_variant(d)]
    finally:
        gconv.gconv_desc_destroy(d)


def test_forward_host_and_second_stream():
    L = Layer("host", 2, 16, 20, 20, 16, groups=4)
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, 9)
    dev = torch.device("cuda:0")
    s = torch.cuda.Stream()
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        with torch.cuda.stream(s):
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            w_d = torch.from_numpy(w).to(dev)
            xs = torch.empty(L.x_elems, dtype=torch.float32, device=dev)
            ys = torch.empty(L.y_elems, dtype=torch.float32, device=dev)
        xh = torch.from_numpy(x).pin_memory()
        yh = torch.empty(L.y_elems, dtype=torch.float32).pin_memory()
        gconv.gconv_pack_weights(d, w_d, wp, s)
        gconv.gconv_forward_host(d, xh, wp, yh, xs, ys, s)
        assert gconv.gconv_last_status(d, s) == gconv.GCONV_OK
        y_ref = oracle.gconv_ref(x, w, 1, 1, 1, L.groups)
        assert rel_err(yh.numpy().reshape(y_ref.shape), y_ref) <= gconv.VARIANT_TOLERANCE[gconv.gconv_variant(d)]
    finally:
        gconv.gconv_desc_destroy(d)
