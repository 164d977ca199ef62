"""The allocation-free entry point, gconv_forward_host_static, against the ordinary host-buffer entry point and
against the oracle.  Some callers (a plugin under a foreign allocator, a service whose device memory is fixed at
start-up, a loop that cannot take the device-wide synchronisation of an allocation) may not allocate device memory;
for them the library keeps its scratch -- status block, staging for x and y, the workspace of the layers that need
one -- in a static device array.  The file name sorts last on purpose: if this test fails, a run that stops at the
first failure has already run everything else."""
import numpy as np
import pytest
import torch

import oracle
from paper_2006_09791_b200 import build as gbuild
from paper_2006_09791_b200 import gconv, synth
from paper_2006_09791_b200.torch_util import attach_workspace
from paper_2006_09791_b200.workloads import Layer

pytestmark = pytest.mark.gpu


def _both_ways(L, seed):
    """y from gconv_forward_host (caller-allocated staging), y from the static-scratch entry point, the oracle's y."""
    dev = torch.device("cuda:0")
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups, seed)
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        gconv.gconv_pack_weights(d, torch.from_numpy(w).to(dev), wp)
        xh = torch.from_numpy(x).pin_memory()
        y_ref = torch.empty(L.y_elems, dtype=torch.float32).pin_memory()
        xs = torch.empty(L.x_elems, dtype=torch.float32, device=dev)
        ys = torch.empty(L.y_elems, dtype=torch.float32, device=dev)
        ws = attach_workspace(d, dev)                       # the ordinary entry point's workspace, if the layer needs one
        gconv.gconv_forward_host(d, xh, wp, y_ref, xs, ys)
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK
        gconv.gconv_desc_set_workspace(d, None, 0)          # the static entry point brings its own
        y_new = torch.full((L.y_elems,), float("nan"), dtype=torch.float32).pin_memory()
        # The first call in a process makes the driver load the library's device image (the static array with it), which
        # shows up in the free-memory figure once; from then on a call must leave that figure exactly as it found it.
        gconv.gconv_forward_host_static(d, xh, wp, y_new)   # synchronous: y_new is complete on return
        y_new.fill_(float("nan"))
        torch.cuda.synchronize()
        free0 = torch.cuda.mem_get_info()[0]
        gconv.gconv_forward_host_static(d, xh, wp, y_new)
        assert torch.cuda.mem_get_info()[0] == free0, "the static entry point changed the amount of free device memory"
        tol = gconv.VARIANT_TOLERANCE[gconv.gconv_variant(d)]
        y_orc = oracle.gconv_ref(x, w, L.stride, L.pad, L.dilation, L.groups, threads=8)
        return y_ref.numpy().copy(), y_new.numpy().copy(), y_orc.reshape(-1), tol
    finally:
        gconv.gconv_desc_destroy(d)


def test_static_scratch_matches_on_two_calls_in_a_row():
    gbuild.build()
    # different layers back to back (tensor-core and CUDA-core variants, the second smaller than the first so it runs
    # over the first call's leftovers in the shared scratch; the third needs the padded-copy workspace where the
    # build still uses one; the last repeats the first)
    for L, seed in [(Layer("a", 4, 64, 32, 32, 64, groups=2), 11), (Layer("b", 3, 24, 20, 28, 24, stride=2, groups=24), 12),
                    (Layer("c", 3, 128, 10, 54, 128), 14), (Layer("a", 4, 64, 32, 32, 64, groups=2), 13)]:
        y_ref, y_new, y_orc, tol = _both_ways(L, seed)
        assert np.all(np.isfinite(y_new))
        scale = float(np.max(np.abs(y_orc)))
        assert float(np.max(np.abs(y_new.astype(np.float64) - y_orc))) / scale <= tol, L.name      # against the oracle
        assert float(np.max(np.abs(y_new.astype(np.float64) - y_ref))) / scale <= tol, L.name      # against the existing entry point


def test_static_scratch_rejects_layers_beyond_its_size():
    gbuild.build()
    L = Layer("big", 128, 32, 32, 32, 32)   # x alone is 16 MiB
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        rc = gconv.load().gconv_forward_host_static(d, 16, 16, 16, None)   # pointers are never touched
        assert rc == gconv.GCONV_ERR_TOO_LARGE
        assert "16 MiB" in gconv.status_string(rc)
    finally:
        gconv.gconv_desc_destroy(d)
