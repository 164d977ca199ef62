"""Helpers for the GPU parity tests: run one layer through the C ABI and compare with the oracle."""
import numpy as np
import torch

import oracle
from paper_2006_09791_b200 import gconv, synth
from paper_2006_09791_b200.torch_util import attach_workspace


def run_layer(L, x_np, w_np, variant=gconv.GCONV_VARIANT_AUTO, stream=None, guard=64):
    """Returns (y as numpy float32, variant used).  y and w_packed are surrounded by sentinel guard
    bands that must survive the launches."""
    dev = torch.device("cuda:0")
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        if variant != gconv.GCONV_VARIANT_AUTO:
            gconv.gconv_desc_set_variant(d, variant)
        used = gconv.gconv_variant(d)
        ws = attach_workspace(d, dev)    # None for most layers
        x = torch.from_numpy(x_np).to(dev)
        w = torch.from_numpy(w_np).to(dev)
        pb = gconv.gconv_packed_bytes(d)
        assert pb % 4 == 0
        sentinel = float(np.float32(-1.2345678e30))
        wp_full = torch.full((pb // 4 + 2 * guard,), sentinel, dtype=torch.float32, device=dev)
        y_elems = L.y_elems
        y_full = torch.full((y_elems + 2 * guard,), sentinel, dtype=torch.float32, device=dev)
        wp = wp_full[guard:guard + pb // 4]
        y = y_full[guard:guard + y_elems]
        gconv.gconv_pack_weights(d, w, wp, stream)
        gconv.gconv_forward(d, x, wp, y, stream)
        st = gconv.gconv_last_status(d, stream)
        assert st == gconv.GCONV_OK, gconv.status_string(st)
        torch.cuda.synchronize()
        for band in (wp_full[:guard], wp_full[-guard:], y_full[:guard], y_full[-guard:]):
            assert bool((band == sentinel).all()), "guard band overwritten"
        return y.cpu().numpy().reshape(L.N, L.C_out, L.H_out, L.W_out), used
    finally:
        gconv.gconv_desc_destroy(d)


def rel_err(y, y_ref):
    """max|y - y_ref| / max|y_ref| over the whole tensor (the acceptance metric)."""
    return float(np.max(np.abs(y.astype(np.float64) - y_ref)) / max(np.max(np.abs(y_ref)), 1e-300))


def check_layer(L, variant=gconv.GCONV_VARIANT_AUTO, seed=0, threads=8):
    x, w = synth.make_layer_tensors(L.N, L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups,
                                    synth.layer_seed(seed, L.N, L.C_in, L.H, L.groups), L.x_dist)
    y, used = run_layer(L, x, w, variant)
    y_ref = oracle.gconv_ref(x, w, L.stride, L.pad, L.dilation, L.groups, threads=threads)
    err = rel_err(y, y_ref)
    tol = gconv.VARIANT_TOLERANCE[used]
    assert np.all(np.isfinite(y)), "non-finite output"
    assert err <= tol, "%s variant %s: rel err %.3e > %.1e" % (L.name, gconv.variant_name(used), err, tol)
    return err, used
