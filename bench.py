#!/usr/bin/env python
"""Benchmark of the filter-gradient (dW) hot path on B200.

One "step" is one pass of the whole path over one synthetic batch of the paper's three CIFAR-10
layer sets at batch 128 (default: VGG-19 in bf16 -- the largest single-GPU workload -- with ResNet-20
and the two-layer CNN in bf16 and fp32 beside it): for every layer the exact dW, the top-1
approximation (Algorithm 1), the zero gradient and the random gradient, each dispatched by the
approximation-schedule driver.  The step is captured once in a CUDA graph and replayed; it is ordered
method-major so that a buffer is touched again only after more than twice the L2 capacity of other
data has streamed through (cold-L2 protocol).

Prints ONE JSON line (rank 0).  `value` is microseconds per layer pass (all four methods of one
layer in one dtype), aggregated over GPUs: step time / (layer passes per step * n_gpus).

Other modes: --config 2|3|4 restricts the step to one layer set; --sweep runs the approximation-
schedule sweep at batch 256; --layer n,c,k,hw[,r[,stride]] times one layer shape (the small,
self-ending program the ncu captures under profiles/ are taken from).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "dW-conv us/layer"
UNIT = "us/layer"
WORKLOADS = {0: "vgg19+resnet20+cnn2_cifar10_n128", 2: "resnet20_cifar10_n128", 3: "cnn2_cifar10_n128", 4: "vgg19_cifar10_n128"}
ORACLE_SAMPLE_IMAGES = 128    # images per distinct layer shape that both oracle legs time (the whole batch at N = 128): ~6 s of CPU work


def workload_sets(config: int, batch: int, dtypes=None):
    """[(config id, layers, dtype names)] of the step: config 0 = all three layer sets."""
    from paper_1908_05460_b200.layers import layer_set
    sets = []
    for cfg in ((4, 2, 3) if config == 0 else (config,)):
        names = dtypes if dtypes else (["bf16"] if cfg == 4 else ["bf16", "f32"])
        sets.append((cfg, layer_set(cfg, batch), names))
    return sets


def traffic_from_profiles(kernel: str, family: str):
    """DRAM bytes of one captured launch of `kernel` on a layer of `family`, from the table in profiles/dram_traffic.md
    (rows: | kernel | family | layer | dram read B | dram write B | algorithmic B | source |).  None when no row matches."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    if not os.path.exists(path):
        return None
    for line in open(path):
        cells = [c.strip() for c in line.strip().strip("|").split("|")]
        if len(cells) >= 7 and cells[0] == kernel and cells[1] == family:
            try:
                rd, wr, alg = int(cells[3]), int(cells[4]), int(cells[5])
            except ValueError:
                continue
            return {"bytes_per_launch": rd + wr, "dram_read": rd, "dram_write": wr, "algorithmic_bytes": alg, "layer": cells[2],
                    "source": "profiles/dram_traffic.md (" + cells[6] + "): one ncu capture of that layer, not this run"}
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------------
# clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx = float(parts[1])
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.path)
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = mx
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ------------------------------------------------------------------------------------------------
# CPU oracle legs
def oracle_sample_us_per_layer(layers, imgs: int = ORACLE_SAMPLE_IMAGES):
    """Times the oracle (exact + top-1 + zero + random) on `imgs` images of every distinct layer shape
    and extrapolates linearly in the batch size.  Returns (us per layer pass, seconds spent, threads)."""
    import numpy as np
    from oracle import oracle
    from paper_1908_05460_b200 import inputs as I
    import torch
    seen, total_us, spent = {}, 0.0, 0.0
    for li, l in enumerate(layers):
        key = (l.c, l.k, l.h, l.r, l.stride)
        if key not in seen:
            ls = l.with_batch(min(imgs, l.n))
            x, dy = I.make_layer_inputs(ls, torch.float32, 2, li)
            xd, dyd = x.double().numpy(), dy.double().numpy()
            sh = oracle.Shape(ls.n, ls.c, ls.h, ls.w, ls.k, ls.r, ls.s, ls.stride, ls.stride, ls.pad, ls.pad)
            t0 = time.perf_counter()
            oracle.dw_exact(xd, dyd, sh)
            oracle.dw_top1(xd, dyd, sh)
            t1 = time.perf_counter()
            cnt = l.k * l.c * l.r * l.s
            oracle.dw_zero(cnt); oracle.dw_random(cnt, 1, 1.0 / 128)
            t2 = time.perf_counter()
            seen[key] = ((t1 - t0) * (l.n / ls.n) + (t2 - t1)) * 1e6
            spent += t2 - t0
        total_us += seen[key]
    return total_us / len(layers), spent, oracle.num_threads()


def run_reference(args, layers):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    for _ in range(args.warmup):
        oracle_sample_us_per_layer(layers)
    vals, t0 = [], time.perf_counter()
    threads = 1
    for _ in range(args.steps):
        v, _, threads = oracle_sample_us_per_layer(layers)
        vals.append(v)
    wall = time.perf_counter() - t0
    value = statistics.mean(vals)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": wall / args.steps * 1e3,
            "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOADS[args.config], "note": "CPU oracle; each step times %d of %d images per "
                       "distinct layer shape and scales by the batch size" % (ORACLE_SAMPLE_IMAGES, args.batch)},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": "%d of %d images per distinct layer shape (exact+top1+zero+random, fp64), scaled to the "
                                       "full batch" % (ORACLE_SAMPLE_IMAGES, args.batch)},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------
def layer_sm_budget(layer, eb, peaks, args):
    """SMs a layer is sized for when the layers of a step run next to one another on several lanes: a share that
    grows with the layer's roofline time (the minimum for the latency-bound layers, up to the maximum)."""
    if args.lanes == 1:
        return 0
    t_roof = max(layer.flops_exact() / (peaks["bf16_tflops"] * 1e12 * (1.0 if eb == 2 else 0.5)),
                 layer.bytes_exact(eb) / (peaks["hbm_gbs"] * 1e9)) * 1e6
    return max(args.budget_min, min(args.budget_max, int(148 * t_roof / args.budget_div)))


def run_sweep(args):
    """Approximation-schedule sweep: ResNet-20 and VGG-19 layer sets at batch 256, bf16.  A seeded mask
    approximates a fraction f of the layers (top-1 method) on odd steps; even steps are all exact.
    Reports the summed dW time per simulated training step (8 steps: 4 exact, 4 masked)."""
    import torch
    from paper_1908_05460_b200 import binding as B
    from paper_1908_05460_b200 import inputs as I
    from paper_1908_05460_b200 import build as build_mod
    from paper_1908_05460_b200.layers import layer_set
    build_mod.build()
    B.load()
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    out = {"workload": "schedule sweep, N=%d, bf16, seeded mask on odd steps, top-1 method, %d lanes" % (args.sweep_batch, args.lanes), "nets": {}}
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for cfg, name in ((2, "resnet20"), (4, "vgg19")):
        layers = layer_set(cfg, args.sweep_batch)
        L = len(layers)
        slots = []
        for li, l in enumerate(layers):
            x, dy = I.make_layer_inputs(l, torch.bfloat16, 5, li + 100 * cfg)
            d = B.make_desc(l, torch.bfloat16, alpha=1.0 / l.n, sm_budget=layer_sm_budget(l, 2, peaks, args))
            slots.append((I.to_nhwc(x).cuda(), dy.cuda(),
                          torch.empty(l.k, l.r, l.s, l.c, dtype=torch.float32, device="cuda"), d, B.attach_workspace(d)))
        rows = []
        for f in (0.0, 0.25, 0.5, 0.75, 1.0):
            sched = B.Schedule(L, B.SCHED_SEEDED_FRACTION_ALT_BATCH, B.METHOD_TOP1, f, 20260101)
            graphs = {}
            packed = sched.pack_step([sl[0] for sl in slots], [sl[1] for sl in slots], [sl[2] for sl in slots], [sl[3] for sl in slots])
            for parity in (0, 1):                       # one CUDA graph per step parity: the switch costs nothing
                def one_step(t=parity):
                    sched.run_step(t, packed, lanes=args.lanes)
                one_step(); torch.cuda.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    one_step()
                graphs[parity] = g
            times = {0: [], 1: []}
            for rep in range(3 + args.warmup):
                for t in range(8):
                    es.record(); graphs[t % 2].replay(); ee.record(); ee.synchronize()
                    if rep >= args.warmup:
                        times[t % 2].append(es.elapsed_time(ee) * 1e3)
            ev, od = statistics.median(times[0]), statistics.median(times[1])
            rows.append({"fraction": f, "approximated_layers": sum(sched.method(l, 1) != B.METHOD_EXACT for l in range(L)),
                         "exact_step_us": ev, "masked_step_us": od, "mean_step_us": 0.5 * (ev + od),
                         "saving_vs_all_exact": 1.0 - 0.5 * (ev + od) / ev})
            sched.close()
        out["nets"][name] = rows
        del slots
    out["note"] = ("paper context: with dW a third of a layer's time and a quarter of layer-batches approximated the "
                   "paper's bound on the training speedup is ~8%; here only the dW time itself is measured")
    print(json.dumps(out))


def run_one_layer(args):
    """--layer: one layer shape through the library a few times, each launch on its own copy of the inputs
    (enough copies to exceed twice the L2 capacity unless --copies says otherwise).  Prints one line."""
    import torch
    from paper_1908_05460_b200 import binding as B
    from paper_1908_05460_b200 import inputs as I
    from paper_1908_05460_b200 import build as build_mod
    from paper_1908_05460_b200.layers import ConvLayer
    build_mod.build()
    B.load()
    v = [int(t) for t in args.layer.split(",")]
    n, c, k, hw = v[:4]
    r = v[4] if len(v) > 4 else 3
    stride = v[5] if len(v) > 5 else 1
    layer = ConvLayer("layer", n, c, hw, hw, k, r, r, stride, r // 2)
    dname = (args.dtypes or "bf16").split(",")[0]
    dt = torch.bfloat16 if dname == "bf16" else torch.float32
    eb = 2 if dname == "bf16" else 4
    x, dy = I.make_layer_inputs(layer, dt, 0, 0)
    xg, dyg = I.to_nhwc(x).cuda(), dy.cuda()
    nbytes = (xg.numel() + dyg.numel()) * eb
    copies = args.copies or max(2, min(64, -(-280_000_000 // nbytes)))
    bufs = [(xg, dyg)] + [(xg.clone(), dyg.clone()) for _ in range(copies - 1)]
    dw = torch.empty(layer.k, layer.r, layer.s, layer.c, dtype=torch.float32, device="cuda")
    desc = B.make_desc(layer, dt, alpha=1.0 / layer.n, topk=args.topk)
    ws = B.attach_workspace(desc)
    method = {"exact": B.METHOD_EXACT, "top1": B.METHOD_TOP1, "zero": B.METHOD_ZERO, "random": B.METHOD_RANDOM,
              "topk": B.METHOD_TOPK}[args.method]

    def one(xb, dyb):
        if method == B.METHOD_EXACT:
            B.gaconv_dw_exact(xb, dyb, dw, desc)
        else:
            B.gaconv_dw_approx(method, xb, dyb, dw, desc, 1)

    one(*bufs[0])
    torch.cuda.synchronize()
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ts = []
    for _ in range(max(1, args.layer_iters)):
        es.record()
        for xb, dyb in bufs:
            one(xb, dyb)
        ee.record()
        ee.synchronize()
        ts.append(es.elapsed_time(ee) * 1e3 / copies)
    launches = B.gaconv_launch_count()
    # the same burst replayed from a CUDA graph: launch cost off the host, as inside a captured training step
    graph_us = None
    if not args.no_graph:
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            for xb, dyb in bufs:
                one(xb, dyb)
        gr.replay()
        torch.cuda.synchronize()
        tg = []
        for _ in range(max(1, args.layer_iters)):
            es.record()
            gr.replay()
            ee.record()
            ee.synchronize()
            tg.append(es.elapsed_time(ee) * 1e3 / copies)
        graph_us = statistics.median(tg)
    print(json.dumps({"layer": args.layer, "dtype": dname, "method": args.method, "us_per_call_host_launched": statistics.median(ts),
                      "us_per_call_graph": graph_us, "copies": copies, "status": B.gaconv_poll_async_status(desc), "launches": launches}))
    del ws


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=0, choices=[0, 2, 3, 4],
                    help="layer sets of the step: 0 all three (default), 2 ResNet-20, 3 two-layer CNN, 4 VGG-19")
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--dtypes", default=None, help="comma list of bf16,f32 (default: the workload's)")
    ap.add_argument("--layer-iters", type=int, default=5, help="per-layer timing repetitions (median)")
    ap.add_argument("--lanes", type=int, default=12, help="streams on which the layers of a step run next to one another (1..16)")
    ap.add_argument("--budget-div", type=float, default=12.0, help="SM share of a layer in the step: 148 * roofline us / this")
    ap.add_argument("--budget-min", type=int, default=18)
    ap.add_argument("--budget-max", type=int, default=74)
    ap.add_argument("--allreduce", action="store_true",
                    help="N > 1: treat the ranks' batches as shards of one batch and sum the exact / top-1 filter gradients of the "
                         "layer set over the ranks in one bucketed all-reduce per step (inside the timed region)")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--detail", default=None, help="write the per-layer table to this JSON file")
    ap.add_argument("--sweep", action="store_true", help="run the approximation-schedule sweep instead of the step benchmark")
    ap.add_argument("--sweep-batch", type=int, default=256)
    ap.add_argument("--layer", default=None, help="n,c,k,hw[,r[,stride]]: time one layer shape and exit")
    ap.add_argument("--method", default="exact", choices=["exact", "top1", "zero", "random", "topk"], help="method of --layer")
    ap.add_argument("--topk", type=int, default=4, help="entries per map of --method topk")
    ap.add_argument("--copies", type=int, default=0, help="input copies of --layer (0: enough to exceed twice the L2)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    sets = workload_sets(args.config, args.batch, args.dtypes.split(",") if args.dtypes else None)
    if args.impl == "reference":
        run_reference(args, [l for _, ls, _ in sets for l in ls])
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.layer:
        run_one_layer(args)
        return

    import torch
    import torch.distributed as dist
    from paper_1908_05460_b200 import binding as B
    from paper_1908_05460_b200 import inputs as I
    from paper_1908_05460_b200 import build as build_mod

    from paper_1908_05460_b200 import dist_util
    rank, world, local = dist_util.env_rank()
    if rank == 0:
        build_mod.build()
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    B.load()
    peaks = measured_peaks()
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32}

    # ---- inputs: generated on the host (seeded), resident in HBM before any timed region ----
    class Slot:
        pass
    slots = []
    h2d = d2h = 0
    for cfg, layers, dtype_names in sets:
        for dname in dtype_names:
            for li, l in enumerate(layers):
                s = Slot()
                s.layer, s.li, s.dtype, s.dname, s.cfg = l, len([t for t in slots if t.cfg == cfg and t.dname == dname]), tdt[dname], dname, cfg
                s.net = {2: "resnet20", 3: "cnn2", 4: "vgg19"}[cfg]
                x, dy = I.make_layer_inputs(l, s.dtype, cfg, li + 1000 * rank)
                s.x_host = I.to_nhwc(x).pin_memory(); s.dy_host = dy.contiguous().pin_memory()
                s.x = s.x_host.cuda(); s.dy = s.dy_host.cuda()
                s.dw = torch.empty(l.k, l.r, l.s, l.c, dtype=torch.float32, device="cuda")
                s.dw_host = torch.empty(l.k, l.r, l.s, l.c, dtype=torch.float32).pin_memory()
                s.eb = 2 if s.dtype == torch.bfloat16 else 4
                s.desc = B.make_desc(l, s.dtype, alpha=1.0 / l.n)            # per-layer timings: the whole GPU for one layer
                s.ws = B.attach_workspace(s.desc)
                # the step runs layers next to one another on several lanes: each layer is sized for a share of the SMs
                # that grows with its roofline time (18 SMs for the latency-bound layers, up to half the GPU)
                s.budget = layer_sm_budget(l, s.eb, peaks, args)
                s.step_desc = B.make_desc(l, s.dtype, alpha=1.0 / l.n, sm_budget=s.budget)
                s.step_ws = B.attach_workspace(s.step_desc)
                h2d += (s.x_host.numel() + s.dy_host.numel()) * s.eb          # a layer's inputs are copied once per step
                d2h += 4 * s.dw.numel() * 4
                slots.append(s)
    L = len(slots)
    for i, s in enumerate(slots):
        s.sid = i                      # layer index within the step's schedule
    input_bytes = sum((s.x.numel() + s.dy.numel()) * s.eb for s in slots)

    methods = [("exact", B.METHOD_EXACT), ("top1", B.METHOD_TOP1), ("zero", B.METHOD_ZERO), ("random", B.METHOD_RANDOM)]
    # schedule 3 of the paper (all layers every 4th batch): step 4t+3 approximates, others are exact
    scheds = {m: B.Schedule(L, B.SCHED_ALL_LAYERS_EVERY_4TH_BATCH, m if m >= 0 else B.METHOD_TOP1, 0.0, 1234)
              for _, m in methods}

    def run_one(s, m, t):
        scheds[m].run_layer(s.sid, 4 * t + (3 if m >= 0 else 0), s.x, s.dy, s.dw, s.desc)

    packed = {m: scheds[m].pack_step([s.x for s in slots], [s.dy for s in slots], [s.dw for s in slots], [s.step_desc for s in slots])
              for _, m in methods}

    def step(t):
        for _, m in methods:                # method-major: a buffer is reused only after a full input pass
            scheds[m].run_step(4 * t + (3 if m >= 0 else 0), packed[m], lanes=args.lanes)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, graph capture ----
    c0 = B.gaconv_launch_count()
    step(0)
    launches_per_step = B.gaconv_launch_count() - c0
    torch.cuda.synchronize()
    graph = None
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step(1)
    base_step = (lambda t: graph.replay()) if graph is not None else step
    if args.allreduce and world > 1:
        # data-parallel filter gradient: after the step every rank holds the gradient of its shard; one bucket, one sum
        def run_step(t):
            base_step(t)
            dist_util.allreduce_dw_bucket([s.dw for s in slots], [B.METHOD_EXACT] * len(slots))
    else:
        run_step = base_step
    for t in range(args.warmup):
        run_step(t)
    # the inputs were generated on the host for seconds while the GPU sat idle: keep it busy for a quarter of a second
    # more, so that the clocks are up when the timed region starts (extra untimed steps, beyond the W asked for)
    extra_warm, t_spin = 0, time.perf_counter()
    torch.cuda.synchronize()
    while time.perf_counter() - t_spin < 0.25:
        run_step(args.warmup + extra_warm)
        extra_warm += 1
        if extra_warm % 8 == 0:
            torch.cuda.synchronize()
    barrier()

    # ---- timed region: exactly K steps ----
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for t in range(args.steps):
        run_step(t)
    ev1.record()
    barrier()
    ms_total = ev0.elapsed_time(ev1)
    if rank == 0:
        time.sleep(0.2)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = dist_util.max_over_ranks(ms_total, "cuda") / args.steps      # slowest rank decides
    passes = len(slots)
    value = dist_util.us_per_layer(ms_step, passes, world)

    # ---- the step, method by method: one graph per method, replayed over cold inputs (another method's pass in between) ----
    es0, ee0 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_by_method = {}
    if not args.no_graph and args.layer_iters > 0:
        gm = {}
        for name, m in methods:
            gm[name] = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gm[name]):
                scheds[m].run_step(4 * 1 + (3 if m >= 0 else 0), packed[m], lanes=args.lanes)
        order = [n for n, _ in methods]
        ts = {n: [] for n in order}
        for rep in range(4):
            for i, name in enumerate(order):
                gm[order[(i + 1) % 2]].replay()            # stream the other input-reading method's data through L2 first
                es0.record(); gm[name].replay(); ee0.record(); ee0.synchronize()
                if rep > 0:
                    ts[name].append(es0.elapsed_time(ee0) * 1e3)
        step_by_method = {n: statistics.median(v) for n, v in ts.items()}
        del gm

    # ---- per-layer timing on the launching stream ----
    # streamed: a CUDA graph of back-to-back launches of one layer, each on its own copy of the inputs,
    #   enough copies that a buffer is touched again only after > 2.5x the L2 capacity has streamed by
    #   (cold data, launch latency amortised as inside the step);
    # isolated: one launch after a 256 MB L2-flushing write, event to event (includes launch latency).
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    es, ee = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def isolated_us(fn, iters):
        ts = []
        for _ in range(iters):
            flush.fill_(1)
            es.record(); fn(); ee.record()
            ee.synchronize()
            ts.append(es.elapsed_time(ee) * 1e3)
        return statistics.median(ts)

    def streamed_us(s, m, iters):
        nbytes = (s.x.numel() + s.dy.numel()) * s.eb
        copies = 48 if m in (B.METHOD_ZERO, B.METHOD_RANDOM) else max(2, min(400, -(-330_000_000 // nbytes)))
        if m in (B.METHOD_ZERO, B.METHOD_RANDOM):
            bufs = [(s.x, s.dy)] * copies
        else:
            bufs = [(s.x, s.dy)] + [(s.x.clone(), s.dy.clone()) for _ in range(copies - 1)]
        step_no = 4 * 2 + (3 if m >= 0 else 0)

        def burst():
            for xb, dyb in bufs:
                scheds[m].run_layer(s.sid, step_no, xb, dyb, s.dw, s.desc)
        burst()
        torch.cuda.synchronize()
        gr = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gr):
            burst()
        gr.replay()
        torch.cuda.synchronize()
        ts = []
        for _ in range(iters):
            es.record(); gr.replay(); ee.record()
            ee.synchronize()
            ts.append(es.elapsed_time(ee) * 1e3 / copies)
        del gr, bufs
        return statistics.median(ts)

    empty_pair_us = isolated_us(lambda: None, 20)
    table, seen = [], {}
    for s in (slots if args.layer_iters > 0 else []):
        l = s.layer
        key = (s.dname, l.c, l.k, l.h, l.r, l.stride)       # layers of one shape share one measurement
        if key not in seen:
            row = {}
            for name, m in methods:
                row[name + "_us"] = streamed_us(s, m, args.layer_iters)
            for name, m in methods[:2]:
                row[name + "_isolated_us"] = isolated_us(lambda: run_one(s, m, 2), 5)
            seen[key] = row
        row = dict(seen[key])
        row.update({"layer": l.name, "net": s.net, "index": s.li, "dtype": s.dname})
        fl, be, bt = l.flops_exact(), l.bytes_exact(s.eb), l.bytes_top1(s.eb)
        t_tensor = fl / (peaks["bf16_tflops"] * 1e12 * (1.0 if s.eb == 2 else 0.5)) * 1e6   # tf32 nominal ratio 1/2
        t_hbm = be / (peaks["hbm_gbs"] * 1e9) * 1e6
        row.update({"gflop": fl / 1e9, "exact_bytes": be, "top1_bytes": bt,
                    "exact_tflops": fl / row["exact_us"] / 1e6, "exact_gbs": be / row["exact_us"] / 1e3,
                    "exact_roof_us": max(t_tensor, t_hbm), "exact_bound": "tensor" if t_tensor > t_hbm else "hbm",
                    "exact_frac": max(t_tensor, t_hbm) / row["exact_us"],
                    "top1_gbs": bt / row["top1_us"] / 1e3, "top1_frac": bt / (peaks["hbm_gbs"] * 1e3) / row["top1_us"],
                    "top1_speedup": row["exact_us"] / row["top1_us"]})
        table.append(row)
    sum_us = {name: sum(r[name + "_us"] for r in table) for name, _ in methods}

    # ---- roofline per kernel family: exact dW on tensor-bound layers, exact dW on HBM-bound layers, top-1 ----
    # a family's fraction = sum of the layers' roofline times / sum of their measured times
    roof = {"bound": None, "achieved": None, "peak": None, "unit": None, "kernel": None, "frac": None, "traffic": None}
    if table:
        tb = [r for r in table if r["exact_bound"] == "tensor"]; hb = [r for r in table if r["exact_bound"] == "hbm"]
        fams = {}
        if tb:
            t = sum(r["exact_us"] for r in tb)
            # fp32 layers count at the TF32 peak (half the bf16 peak): FLOPs scaled to bf16-equivalents
            eq = sum(r["gflop"] * (1.0 if r["dtype"] == "bf16" else 2.0) for r in tb)
            fams["exact_tensor_bound"] = {"bound": "tensor", "achieved": eq / t * 1e3, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                          "frac": sum(r["exact_roof_us"] for r in tb) / t, "layers": len(tb), "sum_us": t,
                                          "note": "bf16-equivalent TFLOP/s (fp32 layers counted at the TF32 peak, half the bf16 peak)"}
        if hb:
            t = sum(r["exact_us"] for r in hb)
            fams["exact_hbm_bound"] = {"bound": "hbm", "achieved": sum(r["exact_bytes"] for r in hb) / t / 1e3, "peak": peaks["hbm_gbs"],
                                       "unit": "GB/s", "frac": sum(r["exact_roof_us"] for r in hb) / t, "layers": len(hb), "sum_us": t}
        t = sum_us["top1"]
        fams["top1"] = {"bound": "hbm", "achieved": sum(r["top1_bytes"] for r in table) / t / 1e3, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": sum(r["top1_bytes"] for r in table) / (peaks["hbm_gbs"] * 1e3) / t, "layers": len(table), "sum_us": t}
        # the dominant kernel first (the exact families are both mostly exact_tc_kernel launches, as in the ncu launch
        # list of the step), then that kernel's larger family
        kernel_of = {"exact_tensor_bound": "exact_tc_kernel", "exact_hbm_bound": "exact_tc_kernel", "top1": "top1_fused_kernel"}
        per_kernel = {}
        for f, v in fams.items():
            per_kernel[kernel_of[f]] = per_kernel.get(kernel_of[f], 0.0) + v["sum_us"]
        kernel = max(per_kernel, key=per_kernel.get)
        dom = max((f for f in fams if kernel_of[f] == kernel), key=lambda f: fams[f]["sum_us"])
        roof = {k: fams[dom][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
        roof.update({"kernel": kernel, "family": dom, "peak_source": peaks["source"], "families": fams,
                     "traffic": traffic_from_profiles(kernel, dom)})
        # the same ratio for the layers as they run in the step (sized for their SM share, overlapping on the lanes):
        # sum of the layers' roofline times / the method's share of the replayed step
        if step_by_method:
            roof["in_step"] = {
                "exact": {"sum_roof_us": sum(r["exact_roof_us"] for r in table), "step_us": step_by_method["exact"],
                          "frac": sum(r["exact_roof_us"] for r in table) / step_by_method["exact"]},
                "top1": {"sum_roof_us": sum(r["top1_bytes"] for r in table) / (peaks["hbm_gbs"] * 1e3), "step_us": step_by_method["top1"],
                         "frac": sum(r["top1_bytes"] for r in table) / (peaks["hbm_gbs"] * 1e3) / step_by_method["top1"]},
                "note": "layers overlap in the step, so these are throughput fractions of the whole GPU, not per-launch ones"}

    # ---- end to end through the host-buffer entry point (H2D and D2H inside the timed region) ----
    e2e = None
    if not args.no_e2e:
        # a layer's inputs cross the link once per step (with its exact gradient); the other three gradients of the layer
        # reuse the device copies; every result is read back to the host
        # Layers alternate between two streams (all calls of a layer on the same one), so that one layer's results go back
        # to the host while the next layer's inputs come in; the host waits once, at the end of the step.  Each method's
        # result has its own pinned host buffer.
        e2e_streams = [torch.cuda.Stream(), torch.cuda.Stream()]
        for s in slots:
            s.dw_hosts = [s.dw_host] + [torch.empty_like(s.dw_host).pin_memory() for _ in range(len(methods) - 1)]

        def e2e_step(t):
            main = torch.cuda.current_stream()
            for st in e2e_streams:
                st.wait_stream(main)
            for i, s in enumerate(slots):
                for j, (_, m) in enumerate(methods):
                    first = m == B.METHOD_EXACT
                    B.gaconv_dw_from_host_async(m, s.x_host if first else None, s.dy_host if first else None, s.dw_hosts[j], s.x, s.dy,
                                                s.dw, s.desc, seed=t, stream=e2e_streams[i & 1])
            for st in e2e_streams:
                main.wait_stream(st)
            main.synchronize()          # the step's results are on the host
        e2e_step(0)
        barrier()
        k2 = max(1, min(args.steps, 3))
        ev0.record()
        for t in range(k2):
            e2e_step(t)
        ev1.record()
        barrier()
        ms_e = dist_util.max_over_ranks(ev0.elapsed_time(ev1) / k2, "cuda")
        e2e = {"value": dist_util.us_per_layer(ms_e, passes, world), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": k2}

    # bounded device waits that gave up leave a flag in the layer's workspace: none may be set after a clean run
    timeouts = sum(1 for s in slots for d in (s.desc, s.step_desc) if B.gaconv_poll_async_status(d) != B.OK)
    if timeouts:
        print("warning: %d workspace status words report a device wait that gave up" % timeouts, file=sys.stderr)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    cpu = None
    if not args.no_cpu:
        v, spent, threads = oracle_sample_us_per_layer([s.layer for s in slots])
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle",
               "sample": "%d of %d images per distinct layer shape (exact+top1+zero+random, fp64), scaled to the "
                         "full batch; %.1f s of CPU work" % (ORACLE_SAMPLE_IMAGES, args.batch, spent)}

    nets = {}
    for r in table:
        d = nets.setdefault(r["net"] + "/" + r["dtype"], {"layers": 0, "exact_us": 0.0, "top1_us": 0.0, "exact_roof_us": 0.0})
        d["layers"] += 1; d["exact_us"] += r["exact_us"]; d["top1_us"] += r["top1_us"]; d["exact_roof_us"] += r["exact_roof_us"]
    dnames = sorted({s.dname for s in slots})
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "+".join(dnames) + " inputs, f32 accumulate", "data": "synthetic",
        "config": {"workload": "%s (%d layer passes x {exact, top1, zero, random}; sets: %s)"
                               % (WORKLOADS[args.config].replace("n128", "n%d" % args.batch), passes,
                                  ", ".join("%s %s" % ({2: "resnet20", 3: "cnn2", 4: "vgg19"}[c], "/".join(dn)) for c, _, dn in sets)),
                   "layer_passes_per_step": passes, "extra_warmup_steps": extra_warm, "cuda_graph": graph is not None, "lanes": args.lanes,
                   "parallelism": ("dp%d, one dW all-reduce per step" % world) if (args.allreduce and world > 1) else ("%d independent replicas" % world if world > 1 else "1 GPU"),
                   "sm_budget": "per layer min(%d, max(%d, 148 * roofline us / %g)) SMs in the step; whole GPU in the per-layer timings"
                                % (args.budget_max, args.budget_min, args.budget_div),
                   "l2": "inputs larger than L2: %.0f MB stream through between two uses of a buffer (method-major "
                         "order); per-layer timings stream over rotating input copies > 2.5x L2" % (input_bytes / 1e6)},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
        "device_wait_timeouts": timeouts,
        "roofline": roof, "cpu_baseline": cpu,
        "breakdown_us": {"step_by_method": step_by_method, "streamed_sum_per_step": sum_us, "event_pair_overhead_us": empty_pair_us,
                         "exact_us_per_layer": sum_us["exact"] / passes, "top1_us_per_layer": sum_us["top1"] / passes,
                         "top1_speedup_over_exact": (sum_us["exact"] / sum_us["top1"]) if table else None,
                         "per_set": nets},
        "paper_context": "paper reports >7% training wall-clock speedup (ResNet-20/VGG-19, Titan Xp, TF 1.13, cuDNN 7.4.2)",
    }
    if args.detail:
        os.makedirs(os.path.dirname(os.path.abspath(args.detail)), exist_ok=True)
        json.dump({"summary": line, "layers": table}, open(args.detail, "w"), indent=1)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
