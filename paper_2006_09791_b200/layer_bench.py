"""Time one grouped-convolution layer through the C ABI (also the entry used for ncu captures).

    python -m paper_2006_09791_b200.layer_bench --cin 32 --cout 32 --hw 32 --groups 1 --n 128 \
        [--stride 1] [--k 3] [--variant auto|generic|tiled|igemm] [--reps 20] [--bufs 0] [--c2 C2]

With --c2 the fused block runs instead (this grouped 3x3 followed by a pointwise convolution to C2 channels,
gconv_block_forward); bytes and FLOPs then count x, y2 and both contractions.

Prints one JSON line: ms per launch (CUDA events around `reps` back-to-back launches that rotate
over `bufs` distinct x/y buffer pairs; bufs = 0 picks enough pairs to cycle more than twice the L2),
GFLOP/s from Eq. (2) of the paper, GB/s on the compulsory bytes.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import build as gbuild
from . import gconv, synth
from .torch_util import attach_workspace
from .workloads import Layer

VARIANTS = {"auto": gconv.GCONV_VARIANT_AUTO, "generic": gconv.GCONV_VARIANT_DIRECT_GENERIC,
            "tiled": gconv.GCONV_VARIANT_DIRECT_TILED, "igemm": gconv.GCONV_VARIANT_IGEMM_TF32}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--cin", type=int, required=True)
    ap.add_argument("--cout", type=int, default=0)
    ap.add_argument("--hw", type=int, required=True)
    ap.add_argument("--w", type=int, default=0)
    ap.add_argument("--groups", type=int, default=1)
    ap.add_argument("--n", type=int, default=1)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--k", type=int, default=3, help="square filter size, pad = k // 2")
    ap.add_argument("--variant", default="auto", choices=sorted(VARIANTS))
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--bufs", type=int, default=0)
    ap.add_argument("--c2", type=int, default=0)
    a = ap.parse_args()
    gbuild.build()
    L = Layer("layer", a.n, a.cin, a.hw, a.w or a.hw, a.cout or a.cin, a.k, a.k, a.stride, a.k // 2, 1, a.groups)
    dev = torch.device("cuda:0")
    y_elems = L.N * a.c2 * L.H_out * L.W_out if a.c2 else L.y_elems
    per = 4 * (L.x_elems + y_elems)
    nbuf = a.bufs or max(2, -(-(2 * 126 * 2 ** 20 + (64 << 20)) // per))
    x0, w0 = synth.make_layer_tensors(min(L.N, 2), L.C_in, L.H, L.W, L.C_out, L.KH, L.KW, L.groups, 7)
    xs = [torch.from_numpy(x0).to(dev).repeat(-(-L.N // x0.shape[0]), 1, 1, 1)[:L.N].contiguous() for _ in range(nbuf)]
    ys = [torch.empty(y_elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
    d = gconv.gconv_desc_create(*L.desc_args())
    if VARIANTS[a.variant]:
        gconv.gconv_desc_set_variant(d, VARIANTS[a.variant])
    ws = attach_workspace(d, dev)
    s = torch.cuda.Stream()
    torch.cuda.synchronize()
    if a.c2:
        if not gconv.gconv_block_supported(d, a.c2):
            raise SystemExit("the fused block does not take this shape")
        _, w2 = synth.make_layer_tensors(1, L.C_out, 1, 1, a.c2, 1, 1, 1, 8)
        wp = torch.empty(gconv.gconv_block_packed_bytes(d, a.c2) // 4, dtype=torch.float32, device=dev)
        gconv.gconv_block_pack_weights(d, a.c2, torch.from_numpy(w0).to(dev), torch.from_numpy(w2.reshape(a.c2, L.C_out)).to(dev), wp, s)
        forward = lambda x, y: gconv.gconv_block_forward(d, a.c2, x, wp, y, s)
        flops = L.flops + 2 * L.N * L.H_out * L.W_out * L.C_out * a.c2
        nbytes = per + 4 * (L.w_elems + L.C_out * a.c2)
    else:
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        gconv.gconv_pack_weights(d, torch.from_numpy(w0).to(dev), wp, s)
        forward = lambda x, y: gconv.gconv_forward(d, x, wp, y, s)
        flops, nbytes = L.flops, L.compulsory_bytes
    with torch.cuda.stream(s):
        for i in range(a.warmup):
            forward(xs[i % nbuf], ys[i % nbuf])
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.synchronize()
        e0.record(s)
        for i in range(a.reps):
            forward(xs[i % nbuf], ys[i % nbuf])
        e1.record(s)
        s.synchronize()
    st = gconv.gconv_last_status(d, s)
    ms = e0.elapsed_time(e1) / a.reps
    print(json.dumps({"layer": L.desc_args(), "variant": gconv.variant_name(gconv.gconv_variant(d)), "status": st,
                      "c2": a.c2, "ms": ms, "gflops": flops / ms / 1e6, "gbs": nbytes / ms / 1e6, "bufs": nbuf,
                      "device_bytes": nbuf * per}))
    gconv.gconv_desc_destroy(d)


if __name__ == "__main__":
    main()
