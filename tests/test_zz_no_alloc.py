"""The allocation-free entry point, gconv_forward_host_static, against the ordinary host-buffer
entry point.  Some callers (a plugin under a foreign allocator, a service with memory fixed at
start-up, code inside a stream capture) may not allocate device memory; for them the library keeps
its scratch in a static device array.  The file name sorts last on purpose: if this test fails, a
run that stops at the first failure has already run everything else."""
import numpy as np
import pytest
import torch

from paper_2006_09791_b200 import build as gbuild
from paper_2006_09791_b200 import gconv, synth
from paper_2006_09791_b200.workloads import Layer

pytestmark = pytest.mark.gpu


def _both_ways(L, seed):
    """y from gconv_forward_host (caller-allocated staging) and from the static-scratch entry point."""
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
        gconv.gconv_forward_host(d, xh, wp, y_ref, xs, ys)
        assert gconv.gconv_last_status(d) == gconv.GCONV_OK
        y_new = torch.full((L.y_elems,), float("nan"), dtype=torch.float32).pin_memory()
        gconv.gconv_forward_host_static(d, xh, wp, y_new)   # synchronous: y_new is complete on return
        tol = gconv.VARIANT_TOLERANCE[gconv.gconv_variant(d)]
        return y_ref.numpy().copy(), y_new.numpy().copy(), tol
    finally:
        gconv.gconv_desc_destroy(d)


def test_static_scratch_matches_on_two_calls_in_a_row():
    gbuild.build()
    # two different layers back to back (tensor-core and CUDA-core variants, the second smaller than
    # the first so it runs over the first call's leftovers in the shared scratch)
    for L, seed in [(Layer("a", 4, 64, 32, 32, 64, groups=2), 11), (Layer("b", 3, 24, 20, 28, 24, stride=2, groups=24), 12),
                    (Layer("a", 4, 64, 32, 32, 64, groups=2), 13)]:
        y_ref, y_new, tol = _both_ways(L, seed)
        assert np.all(np.isfinite(y_new))
        err = float(np.max(np.abs(y_new.astype(np.float64) - y_ref)) / np.max(np.abs(y_ref)))
        assert err <= tol, (L.name, err)


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
