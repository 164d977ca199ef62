"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol the
header declares, validates descriptors and reports shapes/MACs."""
import os
import re

import pytest

from paper_2006_09791_b200 import build as gbuild
from paper_2006_09791_b200 import gconv
from paper_2006_09791_b200.workloads import (R34_GROUPS, Layer, config0, mobilenetv2_dw_layers, resnet34_layers, resnext_layers, sweep_layers,
                                             wrn_stack)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "gconv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gconv_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol():
    lib = gconv.load()
    names = _declared_symbols()
    assert "gconv_desc_create" in names and "gconv_pack_weights" in names and "gconv_forward" in names
    for n in names:
        assert hasattr(lib, n), n
    assert set(names) == set(gconv._SIGNATURES), set(names) ^ set(gconv._SIGNATURES)


def test_descriptor_queries():
    for L in config0() + wrn_stack(4, 128) + resnet34_layers(32, 64):
        d = gconv.gconv_desc_create(*L.desc_args())
        try:
            assert gconv.gconv_out_shape(d) == (L.H_out, L.W_out)
            assert gconv.gconv_macs(d) == L.macs
            v = gconv.gconv_variant(d)
            assert v in gconv.VARIANT_TOLERANCE and gconv.gconv_variant_supported(d, v)
            assert gconv.gconv_packed_bytes(d) >= 4 * L.w_elems
            assert gconv.gconv_forward_launches(d) >= 1
        finally:
            gconv.gconv_desc_destroy(d)


@pytest.mark.parametrize("args", [
    (0, 8, 8, 8, 8, 3, 3, 1, 1, 1, 1), (1, 6, 8, 8, 8, 3, 3, 1, 1, 1, 4), (1, 8, 8, 8, 6, 3, 3, 1, 1, 1, 4),
    (1, 8, 8, 8, 8, 3, 3, 0, 1, 1, 1), (1, 8, 8, 8, 8, 3, 3, 1, -1, 1, 1), (1, 8, 8, 8, 8, 3, 3, 1, 1, 0, 1),
    (1, 8, 2, 2, 8, 5, 5, 1, 0, 1, 1), (1, 8, 8, 8, 8, 3, 3, 1, 1, 1, 0), (1, 8, 4, 4, 8, 3, 3, 1, 0, 2, 1)])
def test_rejects_invalid_descriptors(args):
    with pytest.raises(gconv.GconvError) as e:
        gconv.gconv_desc_create(*args)
    assert e.value.status == gconv.GCONV_ERR_INVALID_ARG


def test_per_axis_descriptor():
    """One stride, padding and dilation per axis (S_h and S_w of Algorithm 1): output size by the floor formula per
    axis; equal axes are the square descriptor; unequal axes leave only the generic FP32 variant."""
    d = gconv.gconv_desc_create_2d(2, 8, 9, 14, 16, 3, 5, 2, 3, 1, 0, 1, 2, 4)
    try:
        assert gconv.gconv_out_shape(d) == ((9 + 2 - 2 - 1) // 2 + 1, (14 + 0 - 2 * 4 - 1) // 3 + 1) == (5, 2)
        assert gconv.gconv_macs(d) == 2 * 16 * 5 * 2 * 2 * 3 * 5
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_DIRECT_GENERIC
        assert not gconv.gconv_variant_supported(d, gconv.GCONV_VARIANT_IGEMM_TF32)
        assert not gconv.gconv_variant_supported(d, gconv.GCONV_VARIANT_DIRECT_TILED)
        with pytest.raises(gconv.GconvError) as e:
            gconv.gconv_desc_set_variant(d, gconv.GCONV_VARIANT_IGEMM_TF32)
        assert e.value.status == gconv.GCONV_ERR_UNSUPPORTED
    finally:
        gconv.gconv_desc_destroy(d)
    # strides of 1 and 2 that differ per axis (3x3, pad 1, width a multiple of 4) run on the tensor-core variant
    d = gconv.gconv_desc_create_2d(4, 64, 28, 28, 64, 3, 3, 2, 1, 1, 1, 1, 1, 4)
    try:
        assert gconv.gconv_out_shape(d) == (14, 28)
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32 and gconv.gconv_workspace_bytes(d) == 0
        assert not gconv.gconv_block_supported(d, 64)
    finally:
        gconv.gconv_desc_destroy(d)
    for L in config0() + wrn_stack(4, 128)[:3]:
        a = gconv.gconv_desc_create(*L.desc_args())
        b = gconv.gconv_desc_create_2d(L.N, L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.stride, L.stride, L.pad, L.pad,
                                       L.dilation, L.dilation, L.groups)
        try:
            assert gconv.gconv_variant(a) == gconv.gconv_variant(b) and gconv.gconv_packed_bytes(a) == gconv.gconv_packed_bytes(b)
            assert gconv.gconv_out_shape(a) == gconv.gconv_out_shape(b)
        finally:
            gconv.gconv_desc_destroy(a)
            gconv.gconv_desc_destroy(b)
    for bad in [(1, 8, 8, 8, 8, 3, 3, 1, 0, 1, 1, 1, 1, 1), (1, 8, 8, 8, 8, 3, 3, 1, 1, 1, -1, 1, 1, 1),
                (1, 8, 8, 8, 8, 3, 3, 1, 1, 1, 1, 1, 0, 1), (1, 8, 8, 4, 8, 3, 3, 1, 1, 1, 0, 1, 2, 1)]:
        with pytest.raises(gconv.GconvError) as e:
            gconv.gconv_desc_create_2d(*bad)
        assert e.value.status == gconv.GCONV_ERR_INVALID_ARG


def test_null_and_variant_errors():
    lib = gconv.load()
    assert lib.gconv_desc_create(None, 1, 8, 8, 8, 8, 3, 3, 1, 1, 1, 1) == gconv.GCONV_ERR_NULL
    assert lib.gconv_desc_destroy(None) == gconv.GCONV_OK
    assert lib.gconv_packed_bytes(None) == 0 and lib.gconv_variant(None) == -1 and lib.gconv_macs(None) == -1
    d = gconv.gconv_desc_create(1, 8, 8, 8, 8, 5, 5, 1, 2, 1, 2)
    try:
        assert lib.gconv_pack_weights(d, None, None, None) == gconv.GCONV_ERR_NULL
        assert lib.gconv_forward(d, None, None, None, None) == gconv.GCONV_ERR_NULL
        assert lib.gconv_pack_weights(d, 4, 16, None) == gconv.GCONV_ERR_ALIGNMENT
        assert lib.gconv_forward(d, 16, 16, 8, None) == gconv.GCONV_ERR_ALIGNMENT
        assert lib.gconv_desc_set_variant(d, 99) == gconv.GCONV_ERR_INVALID_ARG
        # a 5x5 kernel is outside what the tiled and tensor-core variants accept
        assert lib.gconv_desc_set_variant(d, gconv.GCONV_VARIANT_IGEMM_TF32) == gconv.GCONV_ERR_UNSUPPORTED
        assert gconv.gconv_variant(d) == gconv.GCONV_VARIANT_DIRECT_GENERIC
        gconv.gconv_desc_set_variant(d, gconv.GCONV_VARIANT_DIRECT_GENERIC)
        gconv.gconv_desc_set_variant(d, gconv.GCONV_VARIANT_AUTO)
    finally:
        gconv.gconv_desc_destroy(d)
    assert gconv.status_string(gconv.GCONV_ERR_TIMEOUT) and gconv.variant_name(3) == "igemm_tf32"


def test_workspace_is_caller_owned_and_rarely_needed():
    """gconv_forward allocates nothing: the few layers that compute on a zero-padded copy of x report the bytes they
    need and refuse to run without an attached workspace; no layer of the benchmark families needs one (one launch each)."""
    lib = gconv.load()
    assert lib.gconv_workspace_bytes(None) == 0
    bench_layers = config0() + wrn_stack(1, 128) + wrn_stack(16, 128) + sweep_layers(32) + resnext_layers(64) + mobilenetv2_dw_layers(64)
    for g in R34_GROUPS:
        bench_layers += resnet34_layers(g, 64)
    for L in bench_layers:
        d = gconv.gconv_desc_create(*L.desc_args())
        try:
            assert gconv.gconv_workspace_bytes(d) == 0, (L.name, L.groups)
            assert gconv.gconv_forward_launches(d) == 1, (L.name, L.groups)
        finally:
            gconv.gconv_desc_destroy(d)
    # a width the bulk tensor copies cannot address and too wide for the gather producer's 32-lane segments: padded copy of x
    L = Layer("w54", 4, 128, 10, 54, 128, groups=1)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        if gconv.gconv_variant(d) == gconv.GCONV_VARIANT_IGEMM_TF32 and gconv.gconv_workspace_bytes(d) > 0:
            assert gconv.gconv_workspace_bytes(d) == 4 * L.N * L.C_in * 10 * 56       # rows padded from 54 to 56 columns
            assert gconv.gconv_forward_launches(d) == 2
            # no workspace attached: nothing is enqueued (the pointers are never touched), and no device is needed
            assert lib.gconv_forward(d, 16, 16, 32, None) in (gconv.GCONV_ERR_WORKSPACE, gconv.GCONV_ERR_CUDA)
            assert lib.gconv_desc_set_workspace(d, 8, 1 << 20) == gconv.GCONV_ERR_ALIGNMENT
            assert lib.gconv_desc_set_workspace(d, 0, 0) == gconv.GCONV_OK
        gconv.gconv_desc_set_variant(d, gconv.GCONV_VARIANT_DIRECT_GENERIC)
        assert gconv.gconv_workspace_bytes(d) == 0
    finally:
        gconv.gconv_desc_destroy(d)
    assert lib.gconv_desc_set_workspace(None, 0, 0) == gconv.GCONV_ERR_NULL
    assert lib.gconv_desc_set_debug(None, 0, -1) == gconv.GCONV_ERR_NULL
    assert "workspace" in gconv.status_string(gconv.GCONV_ERR_WORKSPACE)
