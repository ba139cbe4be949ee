"""Run one layer shape through the library a few times: the small, self-ending program that
`ncu` captures are taken from (and a quick way to time a single shape with CUDA events).

    python -m paper_1908_05460_b200.profile_layer --c 16 --k 16 --hw 32 --n 128 --dtype bf16 --method exact

Inputs are seeded synthetic tensors as in the benchmark; every launch uses its own copy of the
inputs (`--copies`, default enough to exceed twice the L2 capacity) so that data comes from HBM."""
from __future__ import annotations

import argparse
import statistics

import torch

from . import binding as B
from . import build as build_mod
from . import inputs as I
from .layers import ConvLayer


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--n", type=int, default=128)
    ap.add_argument("--c", type=int, required=True)
    ap.add_argument("--k", type=int, required=True)
    ap.add_argument("--hw", type=int, required=True)
    ap.add_argument("--r", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--pad", type=int, default=None)
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f32"])
    ap.add_argument("--method", default="exact", choices=["exact", "top1", "zero", "random"])
    ap.add_argument("--algo", default="auto", choices=["auto", "direct", "tensor"])
    ap.add_argument("--copies", type=int, default=0)
    ap.add_argument("--iters", type=int, default=3, help="timed passes over all copies")
    args = ap.parse_args()

    build_mod.build()
    B.load()
    pad = args.r // 2 if args.pad is None else args.pad
    layer = ConvLayer("profile", args.n, args.c, args.hw, args.hw, args.k, args.r, args.r, args.stride, pad)
    dt = torch.bfloat16 if args.dtype == "bf16" else torch.float32
    eb = 2 if args.dtype == "bf16" else 4
    x, dy = I.make_layer_inputs(layer, dt, 0, 0)
    xg, dyg = I.to_nhwc(x).cuda(), dy.cuda()
    nbytes = (xg.numel() + dyg.numel()) * eb
    copies = args.copies or max(2, min(64, -(-280_000_000 // nbytes)))
    bufs = [(xg, dyg)] + [(xg.clone(), dyg.clone()) for _ in range(copies - 1)]
    dw = torch.empty(layer.k, layer.r, layer.s, layer.c, dtype=torch.float32, device="cuda")
    desc = B.make_desc(layer, dt, alpha=1.0 / layer.n, algo={"auto": 0, "direct": 1, "tensor": 2}[args.algo])
    ws = B.attach_workspace(desc)
    method = {"exact": B.METHOD_EXACT, "top1": B.METHOD_TOP1, "zero": B.METHOD_ZERO, "random": B.METHOD_RANDOM}[args.method]

    def one(xb, dyb):
        if method == B.METHOD_EXACT:
            B.gaconv_dw_exact(xb, dyb, dw, desc)
        else:
            B.gaconv_dw_approx(method, xb, dyb, dw, desc, 1)

    one(*bufs[0])
    torch.cuda.synchronize()
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(args.iters):
        es.record()
        for xb, dyb in bufs:
            one(xb, dyb)
        ee.record()
        ee.synchronize()
        ts.append(es.elapsed_time(ee) * 1e3 / copies)
    status = B.gaconv_poll_async_status(desc)
    print("layer n=%d c=%d k=%d hw=%d r=%d stride=%d %s %s: %.2f us per call (median of %d passes over %d copies, "
          "host-launched), status %d, launches so far %d"
          % (layer.n, layer.c, layer.k, layer.h, layer.r, layer.stride, args.dtype, args.method, statistics.median(ts),
             args.iters, copies, status, B.gaconv_launch_count()))
    del ws


if __name__ == "__main__":
    main()
