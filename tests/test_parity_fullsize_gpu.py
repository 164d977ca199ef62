"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (selector's variant, same
batch, including a CUDA-graph replay).  The WHOLE output tensor is compared with the oracle, element by element, for
every group count of every benchmark family: max|y - y_ref| / max|y_ref| over the full tensor within the tolerance of
the variant that ran.  Only the >2^31-element case is sampled: there the oracle would need hours, so slices the
oracle can compute one by one are compared in full."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_09791_b200 import build as gbuild
from paper_2006_09791_b200 import gconv, synth
from paper_2006_09791_b200.torch_util import attach_workspace
from paper_2006_09791_b200.workloads import (R34_GROUPS, SWEEP_GROUPS, WRN_GROUPS, config0, depthwise5x5_layers, mobilenetv2_dw_layers,
                                             pointwise_layers, resnet34_layers, resnext_layers, sweep_layers, wrn_stack)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    gbuild.build()


def _run_full(L, x, w, use_graph):
    dev = torch.device("cuda:0")
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            xd = torch.from_numpy(x).to(dev)
            wd = torch.from_numpy(w).to(dev)
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            y = torch.full((L.y_elems,), float("nan"), dtype=torch.float32, device=dev)
            ws = attach_workspace(d, dev)
            gconv.gconv_pack_weights(d, wd, wp, s)
            gconv.gconv_forward(d, xd, wp, y, s)
            if use_graph:
                s.synchronize()
                y.fill_(float("nan"))
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=s):
                    gconv.gconv_forward(d, xd, wp, y, s)
                graph.replay()
            s.synchronize()
        assert gconv.gconv_last_status(d, s) == gconv.GCONV_OK
        return y.cpu().numpy().reshape(L.N, L.C_out, L.H_out, L.W_out), gconv.gconv_variant(d)
    finally:
        gconv.gconv_desc_destroy(d)


def _check_full(L, y, x, w, variant):
    """Element by element over the whole tensor, the acceptance metric of the paper's problem statement."""
    tol = gconv.VARIANT_TOLERANCE[variant]
    assert np.all(np.isfinite(y)), "non-finite output (an element was never written?)"
    ref = oracle.gconv_ref(x, w, L.stride, L.pad, L.dilation, L.groups, threads=oracle.max_threads())
    assert ref.shape == y.shape
    rel = float(np.max(np.abs(y.astype(np.float64) - ref)) / np.max(np.abs(ref)))
    assert rel <= tol, "%s groups=%d variant %s: rel err %.3e > %.1e" % (L.name, L.groups, gconv.variant_name(variant), rel, tol)


def test_config0_single_layer():
    (L,) = config0()
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, synth.layer_seed(76), L.x_dist)
    y, v = _run_full(L, x, w, use_graph=True)
    _check_full(L, y, x, w, v)


@pytest.mark.parametrize("groups", WRN_GROUPS)
def test_wrn_stack_at_batch_128(groups):
    """Every distinct layer of the bench step (batch 128), every group count, the whole tensor."""
    for i, L in enumerate(wrn_stack(groups, 128)):
        x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, groups, synth.layer_seed(77, i, groups), L.x_dist)
        y, v = _run_full(L, x, w, use_graph=(i % 2 == 0))
        _check_full(L, y, x, w, v)


@pytest.mark.parametrize("idx", range(len(SWEEP_GROUPS)))     # every group count of the sweep to depthwise
def test_group_sweep_at_batch_32(idx):
    L = sweep_layers(32)[idx]
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, synth.layer_seed(78, idx), L.x_dist)
    y, v = _run_full(L, x, w, use_graph=True)
    _check_full(L, y, x, w, v)


@pytest.mark.parametrize("groups", R34_GROUPS)
def test_resnet34_layers_at_batch_64(groups):
    """The ResNet-34-shaped rows at the batch the bench times them at, every group count, the whole tensor: pair tiles
    and streamed filter banks (groups 1 and 2), 14x14 and 7x7 planes, stride-2 tiles with wide and narrow groups."""
    for i, L in enumerate(resnet34_layers(groups, 64)):
        x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, groups, synth.layer_seed(83, i, groups), L.x_dist)
        y, v = _run_full(L, x, w, use_graph=(i % 2 == 1))
        _check_full(L, y, x, w, v)


def _sweep_row_families():
    """The other rows of the bench's tables at the batch it times them at: ResNeXt-shaped grouped layers (stride-2
    tiles, 14x14 and 7x7 planes, tap blocks), MobileNetV2-shaped depthwise 3x3 and depthwise 5x5 layers, pointwise layers."""
    return resnext_layers(64) + mobilenetv2_dw_layers(64) + depthwise5x5_layers(64) + pointwise_layers(64)


@pytest.mark.parametrize("idx", range(len(_sweep_row_families())))
def test_sweep_table_rows_at_batch_64(idx):
    L = _sweep_row_families()[idx]
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups, synth.layer_seed(80, idx), L.x_dist)
    y, v = _run_full(L, x, w, use_graph=(idx % 2 == 1))
    _check_full(L, y, x, w, v)


def test_more_than_2_to_31_elements():
    """Maximum sizes: x and y each hold more than 2^31 elements, so every 32-bit index in the path would wrap.
    The batch is a two-image block repeated on the device; slices are checked against the oracle on that block."""
    from paper_2006_09791_b200.workloads import Layer
    for groups, C in ((2, 128), (128, 128)):          # tensor-core variant and depthwise stream kernel
        N = 4100 if groups == 2 else 4400
        L = Layer("huge_g%d" % groups, N, C, 64, 64, C, groups=groups)
        assert L.x_elems > 2 ** 31 and L.y_elems > 2 ** 31
        dev = torch.device("cuda:0")
        xb, w = synth.make_layer_tensors(2, L.C_in, L.H, L.W, L.C_out, 3, 3, groups, synth.layer_seed(79, groups))
        d = gconv.gconv_desc_create(*L.desc_args())
        try:
            x = torch.from_numpy(xb).to(dev).repeat(N // 2, 1, 1, 1)
            wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
            y = torch.full((L.y_elems,), float("nan"), dtype=torch.float32, device=dev)
            gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
            gconv.gconv_forward(d, x, wp, y)
            st = gconv.gconv_last_status(d)
            assert st == gconv.GCONV_OK, (gconv.status_string(st), gconv.gconv_last_status_detail(d))
            v = gconv.gconv_variant(d)
            tol = gconv.VARIANT_TOLERANCE[v]
            yv = y.view(N, L.C_out, L.H_out, L.W_out)
            assert bool(torch.isfinite(yv[::97]).all()) and bool(torch.isfinite(yv[-3:]).all())
            for n, g in [(0, 0), (N - 1, groups - 1), (N // 2 + 1, groups // 2), (2049, 1), (N - 2, 0)]:
                ref = oracle.gconv_ref(xb[n % 2:n % 2 + 1, g * L.Cg:(g + 1) * L.Cg], w[g * L.Kg:(g + 1) * L.Kg], 1, 1, 1, 1, threads=16)[0]
                got = yv[n, g * L.Kg:(g + 1) * L.Kg].cpu().numpy().astype(np.float64)
                assert np.max(np.abs(got - ref)) <= tol * max(np.max(np.abs(ref)), 1e-30), (L.name, n, g)
            del x, y, yv
            torch.cuda.empty_cache()
        finally:
            gconv.gconv_desc_destroy(d)


def _fused_blocks():
    from paper_2006_09791_b200.workloads import fused_blocks
    return fused_blocks()


@pytest.mark.parametrize("idx", range(len(_fused_blocks())))
def test_fused_blocks_at_bench_batch(idx):
    """The fused grouped 3x3 + pointwise blocks the bench times, at its batch, back to back (two launches, the second a
    CUDA-graph replay on odd rows).  The whole output is checked: the oracle's grouped convolution, rounded to fp32 (the
    kernel keeps the intermediate in fp32), then its 1x1 convolution."""
    L, C2 = _fused_blocks()[idx]
    dev = torch.device("cuda:0")
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, synth.layer_seed(81, idx), L.x_dist)
    _, w2 = synth.make_layer_tensors(1, L.C_out, 1, 1, C2, 1, 1, 1, synth.layer_seed(82, idx))
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        assert gconv.gconv_block_supported(d, C2)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            xd = torch.from_numpy(x).to(dev)
            wp = torch.empty(gconv.gconv_block_packed_bytes(d, C2) // 4, dtype=torch.float32, device=dev)
            y2 = torch.full((L.N * C2 * L.H * L.W,), float("nan"), dtype=torch.float32, device=dev)
            scratch = torch.empty_like(y2)
            gconv.gconv_block_pack_weights(d, C2, torch.from_numpy(w).to(dev), torch.from_numpy(w2.reshape(C2, L.C_out)).to(dev), wp, s)
            gconv.gconv_block_forward(d, C2, xd, wp, scratch, s)
            if idx % 2 == 1:
                s.synchronize()
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(graph, stream=s):
                    gconv.gconv_block_forward(d, C2, xd, wp, scratch, s)
                    gconv.gconv_block_forward(d, C2, xd, wp, y2, s)
                graph.replay()
            else:
                gconv.gconv_block_forward(d, C2, xd, wp, y2, s)
            s.synchronize()
        assert gconv.gconv_last_status(d, s) == gconv.GCONV_OK
        got = y2.cpu().numpy().reshape(L.N, C2, L.H, L.W)
        assert np.all(np.isfinite(got))
        tol = gconv.VARIANT_TOLERANCE[gconv.GCONV_VARIANT_IGEMM_TF32]
        y1 = oracle.gconv_ref(x, w, 1, 1, 1, L.groups, threads=oracle.max_threads()).astype(np.float32)
        ref = oracle.gconv_ref(y1, w2, 1, 0, 1, 1, threads=oracle.max_threads())
        err = np.max(np.abs(got.astype(np.float64) - ref)) / np.max(np.abs(ref))
        assert err <= tol, (L.name, L.groups, C2, err)
    finally:
        gconv.gconv_desc_destroy(d)
