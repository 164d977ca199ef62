"""Times every supported kernel variant on a grid of layers; the table it prints is what the
selector's rule in csrc/gconv_api.cu (select_variant) is derived from.

    python -m paper_2006_09791_b200.selector_sweep [--quick] > table.txt

Each cell is the median per-launch time (µs, cold L2: launches rotate over buffers that cycle more
than twice the L2) of gconv_forward with that variant forced; `auto` names the selector's choice.
"""
from __future__ import annotations

import argparse
import statistics

import torch

from . import build as gbuild
from . import gconv, synth
from .torch_util import attach_workspace
from .workloads import Layer, resnet34_layers, resnext_layers, sweep_layers, wrn_stack

VARIANTS = [(gconv.GCONV_VARIANT_DIRECT_GENERIC, "generic"), (gconv.GCONV_VARIANT_DIRECT_TILED, "tiled"),
            (gconv.GCONV_VARIANT_IGEMM_TF32, "igemm")]


def time_variant(L, variant, reps=20):
    dev = torch.device("cuda:0")
    d = gconv.gconv_desc_create(*L.desc_args())
    try:
        if not gconv.gconv_variant_supported(d, variant):
            return None
        gconv.gconv_desc_set_variant(d, variant)
        ws = attach_workspace(d, dev)
        per = 4 * (L.x_elems + L.y_elems)
        nbuf = max(2, min(64, -(-(2 * 126 * 2 ** 20 + (64 << 20)) // per)))
        x0, w0 = synth.make_layer_tensors(min(L.N, 2), L.C_in, L.H, L.W, L.C_out, 3, 3, L.groups, 5, L.x_dist)
        xs = [torch.from_numpy(x0).to(dev).repeat(-(-L.N // x0.shape[0]), 1, 1, 1)[:L.N].contiguous() for _ in range(nbuf)]
        ys = [torch.empty(L.y_elems, dtype=torch.float32, device=dev) for _ in range(nbuf)]
        wp = torch.empty(gconv.gconv_packed_bytes(d) // 4, dtype=torch.float32, device=dev)
        s = torch.cuda.Stream()
        times = []
        with torch.cuda.stream(s):
            gconv.gconv_pack_weights(d, torch.from_numpy(w0).to(dev), wp, s)
            for i in range(3):
                gconv.gconv_forward(d, xs[i % nbuf], wp, ys[i % nbuf], s)
            s.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=s):
                for i in range(reps):
                    gconv.gconv_forward(d, xs[i % nbuf], wp, ys[i % nbuf], s)
            graph.replay()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for _ in range(5):
                e0.record(s)
                graph.replay()
                e1.record(s)
                s.synchronize()
                times.append(1e3 * e0.elapsed_time(e1) / reps)
        assert gconv.gconv_last_status(d, s) == 0
        return statistics.median(times)
    finally:
        gconv.gconv_desc_destroy(d)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--quick", action="store_true")
    a = ap.parse_args()
    gbuild.build()
    layers = []
    for g in (1, 4, 16):
        layers += wrn_stack(g, 128)
    layers += [L.with_(N=1) for L in wrn_stack(1, 1)] + [L.with_(N=1) for L in wrn_stack(16, 1)]
    layers += sweep_layers(32)
    if not a.quick:
        layers += resnext_layers(64) + resnet34_layers(1, 64) + resnet34_layers(32, 64)
        layers += [Layer("dw_32@32", 128, 32, 32, 32, 32, groups=32), Layer("dw_128@8", 128, 128, 8, 8, 128, groups=128),
                   Layer("dw_64@112", 16, 64, 112, 112, 64, groups=64), Layer("dw_64@112s2", 16, 64, 112, 112, 64, stride=2, groups=64)]
    print("| layer | N | groups | Cg | Kg | H·W | " + " | ".join(n + " µs" for _, n in VARIANTS) + " | auto | best |")
    print("|---|---|---|---|---|---|" + "---|" * (len(VARIANTS) + 2))
    for L in layers:
        d = gconv.gconv_desc_create(*L.desc_args())
        auto = gconv.variant_name(gconv.gconv_variant(d))
        gconv.gconv_desc_destroy(d)
        ts = [time_variant(L, v, reps=6 if (v == gconv.GCONV_VARIANT_DIRECT_GENERIC and L.macs > 2e9) else 20) for v, _ in VARIANTS]
        best = min((t, n) for t, (_, n) in zip(ts, VARIANTS) if t is not None)[1]
        cells = " | ".join("%.1f" % t if t is not None else "–" for t in ts)
        print("| %s | %d | %d | %d | %d | %d | %s | %s | %s |" % (L.name, L.N, L.groups, L.Cg, L.Kg, L.H * L.W, cells, auto, best), flush=True)


if __name__ == "__main__":
    main()
