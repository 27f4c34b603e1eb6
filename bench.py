#!/usr/bin/env python
"""Benchmark of the splatting training step (forward + backward, 8 views of a 1M-Gaussian scene).

`python bench.py --gpus N --steps K --warmup W` prints ONE JSON line on rank 0.
A "step" is one pass of the whole hot path over one batch: for each of the 8 orbit cameras,
gs_preprocess -> gs_render_forward -> gs_render_backward on the 1M-Gaussian clustered scene
(the 1M configuration of the benchmark list) with the neural appearance model; the SH model and
the appearance-decode sweep are timed beside it and reported in extra keys.

`--impl reference` times the CPU oracle (the plain double-precision restatement of the method) on
the host cores on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "fwd+bwd rasterizer ms/iter @1M Gaussians; appearance-decode GB/s vs HBM peak"
N_GAUSS, WIDTH, HEIGHT, VIEWS = 1_000_000, 1256, 828, 8

# Algorithmic cost per unit: flops per evaluated list entry of the blend kernels and bytes per Gaussian of
# the per-Gaussian kernels.
# Blend kernels (fp32 ALU bound): flops per list entry evaluated for a pixel (the alpha test) and per
# pair composited, counted from the kernels' arithmetic.
BLEND_FLOPS_PER_EVALUATED = 8.0       # 3.5 (quad falloff, shared by 4 pixels) + ex2 + mul + min + compare
BLEND_FWD_FLOPS_PER_COMPOSITED = 10.0  # 1-a, T(1-a), compare, aT, three FMAs
BLEND_BWD_FLOPS_PER_COMPOSITED = 45.0  # reciprocal, T and S recovery, d/d alpha, nine gradient FMAs
FP32_LANES_PER_SM, NUM_SMS = 128, 148


def cache_note(config):
    if config in (3, 4):
        return "inputs_larger_than_L2 (per-view working set > 126 MB; every view another camera)"
    return "working set smaller than L2 and not flushed: a small parity case, bound by launch latency, not a bench line"
FP32_ALU_PEAK_TFLOPS = NUM_SMS * FP32_LANES_PER_SM * 2 * 1965e6 / 1e12   # 74.4 at the maximum SM clock


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), sm_max_mhz=float(p.get("sm_max_mhz", 1965.0)), source="measured")
    return dict(hbm_gbs=6650.0, sm_max_mhz=1965.0, source="fallback")


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples during the timed region."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in open(self.path):
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        os.unlink(self.path)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(args):
    from paper_2609_05255_b200 import replicas
    return replicas.rank_env()


def workload_of(args, scenes):
    """The seeded synthetic workload of --config: name, sizes, cameras, a scene factory per appearance model
    and the arms timed (the first one carries the headline numbers)."""
    c = args.config
    if c == 3:
        n, views = args.n or N_GAUSS, args.views or VIEWS
        return dict(name=f"config3: {n} Gaussians (64 clusters + shell), {WIDTH}x{HEIGHT}, {views} orbit views, "
                         "neural appearance (8 fp16 features + shared 32-16-16-3 MLP), with SH degree 3 and Spherical Voronoi beside it, fwd+bwd",
                    n=n, views=views, width=WIDTH, height=HEIGHT, cams=scenes.orbit_cameras(WIDTH, HEIGHT, views),
                    scene=lambda app: scenes.config3(app, n=n, width=WIDTH, height=HEIGHT, views=views).scene,
                    arms=[(scenes.APP_NEURAL, "neural"), (scenes.APP_SH, "sh"), (scenes.APP_SV, "sv")])
    if c == 1:
        w = scenes.config1()
        return dict(name="config1: 1000 Gaussians in a box, 64x64, identity camera, SH degree 3, fwd+bwd",
                    n=w.scene.n, views=1, width=64, height=64, cams=w.cameras, scene=lambda app: w.scene,
                    arms=[(scenes.APP_SH, "sh")])
    if c == 2:
        w = scenes.config2()
        return dict(name="config2: 100k Gaussians in a box, 512x512, identity camera, neural appearance, fwd+bwd",
                    n=w.scene.n, views=1, width=512, height=512, cams=w.cameras, scene=lambda app: w.scene,
                    arms=[(scenes.APP_NEURAL, "neural")])
    views = args.views or 16
    w = scenes.config4(views=views)
    return dict(name=f"config4: 3M Gaussians (256 clusters, depths 1-50, + shell), 1920x1080, {views} orbit views, "
                     "neural appearance, fwd+bwd",
                n=w.scene.n, views=views, width=1920, height=1080, cams=w.cameras, scene=lambda app: w.scene,
                arms=[(scenes.APP_NEURAL, "neural")])


# ---------------------------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    from paper_2609_05255_b200 import api, replicas, scenes

    rank, world, local = dist_setup(args)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = replicas.init_process_group("nccl", world, dev)
    peaks = measured_peaks()
    ctx = api.Context(local)
    wl = workload_of(args, scenes)
    n, views, WIDTH, HEIGHT, cams_host = wl["n"], wl["views"], wl["width"], wl["height"], wl["cams"]
    cams = [api.make_camera(c) for c in cams_host]

    def make_arm(app):
        host = wl["scene"](app)
        ds = api.upload_scene(host, dev)
        probe = api.alloc_projected(ds.n, dev, with_extent=False)
        pairs = [api.gs_preprocess(ctx, ds, c, probe) for c in cams]
        cap = int(max(pairs) * 1.02) + 1024
        r = api.Renderer(ctx, ds.n, WIDTH, HEIGHT, app, pair_capacity=cap)
        return host, ds, r, pairs

    gen = torch.Generator(device=dev); gen.manual_seed(4242 + rank)
    G = torch.randn((views, 3, HEIGHT, WIDTH), device=dev, generator=gen)
    head = wl["arms"][0][1]                     # the arm the headline numbers are quoted on

    def step(ds, r):
        for v in range(views):
            r.forward(ds, cams[v])
            r.backward(ds, cams[v], G[v])

    # Two views in flight: the views of an iteration are independent, so they alternate between two
    # streams, each with its own context and buffers.  The latency-bound binning of one view then
    # runs beside the ALU-bound blending of the other.
    n_lanes = 1 if args.single_stream else max(1, args.streams)
    lane_ctx = [ctx] + [api.Context(local) for _ in range(n_lanes - 1)]
    lanes = [torch.cuda.Stream(dev) for _ in range(n_lanes)]

    def step_two_streams(ds, pair):   # pair: one Renderer per lane
        main = torch.cuda.current_stream(dev)
        for s in lanes:
            s.wait_stream(main)
        for v in range(views):
            r, s = pair[v % n_lanes], lanes[v % n_lanes]
            r.forward_async(ds, cams[v], stream=s)      # no host wait: the instance count stays on the device
            r.backward(ds, cams[v], G[v], stream=s)
        for s in lanes:
            main.wait_stream(s)

    def barrier():
        torch.cuda.synchronize()
        replicas.barrier(dist)
        torch.cuda.synchronize()

    def timed(fn, steps, warmup, drain=None):
        for _ in range(warmup):
            fn()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        if drain:
            drain()          # work the steps left on other streams ends inside the timed region
        e1.record()
        barrier()
        return replicas.max_over_ranks(e0.elapsed_time(e1) / steps, dist, dev)

    def profile(fn, steps):
        api.gs_profile_enable(ctx, True)
        api.gs_profile_collect(ctx)
        tot_ms, tot_l = {}, {}
        for _ in range(steps):
            fn()
            ms, launches = api.gs_profile_collect(ctx)
            for k in ms:
                tot_ms[k] = tot_ms.get(k, 0.0) + ms[k]; tot_l[k] = tot_l.get(k, 0) + launches[k]
        api.gs_profile_enable(ctx, False)
        return {k: v / steps for k, v in tot_ms.items()}, {k: v / steps for k, v in tot_l.items()}

    results = {}
    sampler = ClockSampler(local)
    clocks = None
    arms = [a for a in wl["arms"] if not (args.skip_sh and a[1] != head)]
    for app, tag in arms:
        host, ds, r, pairs = make_arm(app)
        if tag == head:
            sampler.start()
        ms_one = timed(lambda: step(ds, r), args.steps, args.warmup)
        ms = ms_streams = ms_one
        graph_note = None
        if views > 1 and n_lanes > 1:
            rs = [r] + [api.Renderer(c, ds.n, WIDTH, HEIGHT, app, pair_capacity=r.pair_capacity) for c in lane_ctx[1:]]
            ms = timed(lambda: step_two_streams(ds, rs), args.steps, args.warmup)
            for c, s_ in zip(lane_ctx, lanes):
                api.gs_async_status(c, s_)              # raises if a view had outgrown its pair capacity
            ms_streams = ms
            if not args.no_graph:
                # The same iteration captured once as a CUDA graph (nothing in it waits for the host) and replayed:
                # the kernels, their order and their arguments are unchanged, only the launching is.
                try:
                    cap = torch.cuda.Stream(dev)
                    cap.wait_stream(torch.cuda.current_stream(dev))
                    graph = torch.cuda.CUDAGraph()
                    with torch.cuda.stream(cap):
                        step_two_streams(ds, rs)            # once more outside the capture, on the capture stream
                        torch.cuda.synchronize()
                        with torch.cuda.graph(graph, stream=cap):
                            step_two_streams(ds, rs)
                    torch.cuda.current_stream(dev).wait_stream(cap)
                    ms_graph = timed(graph.replay, args.steps, args.warmup)
                    for c, s_ in zip(lane_ctx, lanes):
                        api.gs_async_status(c, s_)
                    graph_note = {"ms_per_step": ms_graph, "captured": True}
                    ms = min(ms, ms_graph)
                    del graph
                except Exception as e:                      # capture is an optimisation of the launching only
                    graph_note = {"captured": False, "why": str(e)[:200]}
                    torch.cuda.synchronize()
            half_streams = None
            if tag == "neural" and args.config == 3 and not args.skip_decode:
                ds.decoder_precision = 1                    # plain fp16 operands, the paper's precision
                half_streams = timed(lambda: step_two_streams(ds, rs), args.steps, args.warmup)
                for c, s_ in zip(lane_ctx, lanes):
                    api.gs_async_status(c, s_)
                ds.decoder_precision = 0
            del rs
        else:
            half_streams = None
        stage_ms, stage_launches = profile(lambda: step(ds, r), max(1, min(args.steps, 3)))
        if tag == head:
            # keep the GPU under the same load until the sampler has a few readings (100 ms apart)
            t_end = time.perf_counter() + max(0.0, 1.0 - args.steps * ms * 1e-3)
            while time.perf_counter() < t_end:
                step(ds, r)
                torch.cuda.synchronize()
            clocks = sampler.stop()
        # units of the blend kernels: list entries up to each pixel's last composited one, over the views
        entries = 0
        visible = records = with_gradient = 0
        evaluated = composited = warp_steps = warp_steps_idle = 0
        for v in range(views):
            r.forward(ds, cams[v])
            torch.cuda.synchronize()
            entries += int(r.n_contrib.sum(dtype=torch.int64).item())
            ev, co, ws_, wi = api.gs_profile_blend_counts(ctx, r.proj, r.binning, cams[v])
            evaluated += ev; composited += co; warp_steps += ws_; warp_steps_idle += wi
            rect = r.proj.rect.to(torch.int32) & 0xFFFF
            vis_rows = (rect[:, 2] > rect[:, 0]) & (rect[:, 3] > rect[:, 1])
            visible += int(vis_rows.sum().item())
            # Gaussians that receive a gradient in this view (the backward leaves the 2D gradients [n,12] at the start of
            # the workspace): the others are hidden behind saturated pixels and the preprocess backward skips them
            r.backward(ds, cams[v], G[v])
            torch.cuda.synchronize()
            g2d = r.workspace[: ds.n * 48].view(torch.float32).reshape(ds.n, 12)
            with_gradient += int(((g2d[:, :9] != 0).any(1) & vis_rows).sum().item())
            records += int((r.proj.cell_count.to(torch.int64) & 0x7FFFFFFF).sum().item())
        # the same step through the unfused reference path (App. D "Fusion"): appearance as passes of its own
        unfused = None
        if args.config == 3 and not args.skip_decode:
            ds.separate_pass = 1
            u_one = timed(lambda: step(ds, r), args.steps, args.warmup)
            u_stage, _ = profile(lambda: step(ds, r), max(1, min(args.steps, 3)))
            ds.separate_pass = 0
            unfused = {"ms_per_step_single_stream": u_one, "fused_ms_per_step_single_stream": ms_one,
                       "stages_ms_per_step": {k: round(v, 4) for k, v in u_stage.items() if v > 0}}
        half = None
        if tag == "neural" and args.config == 3 and not args.skip_decode:
            ds.decoder_precision = 1
            h_one = timed(lambda: step(ds, r), args.steps, args.warmup)
            h_stage, _ = profile(lambda: step(ds, r), max(1, min(args.steps, 3)))
            ds.decoder_precision = 0
            half = {"ms_per_step": half_streams, "ms_per_step_single_stream": h_one,
                    "split_ms_per_step": ms_streams, "split_ms_per_step_single_stream": ms_one,
                    "stages_ms_per_step": {k: round(v, 4) for k, v in h_stage.items() if v > 0},
                    "what": "the decoder's products on plain fp16 operands (GS_DECODER_HALF, the paper's precision) instead of "
                            "split ones; colours within 2e-3 of the oracle instead of 2e-5 (tests/test_gpu_half_precision.py)"}
        # the architecture table's other decoders (App. D) through the same step: they run unfused, their appearance
        # passes on the tcgen05 kernels, the backward on the Gaussians that received a gradient only
        variants_step = None
        if tag == "neural" and args.config == 3 and not args.skip_decode:
            variants_step = {"default_decoder_fused_ms_per_step": ms_streams, "default_decoder_fused_ms_per_step_single_stream": ms_one}
            keep = (ds.features, ds.mlp_weights, ds.mlp_hidden, ds.mlp_layers, ds.num_features, r.grads)
            gen_v = torch.Generator(device=dev); gen_v.manual_seed(909)
            rs_v = ([r] + [api.Renderer(c, ds.n, WIDTH, HEIGHT, app, pair_capacity=r.pair_capacity) for c in lane_ctx[1:]]
                    if views > 1 and n_lanes > 1 else None)
            for hidden, layers, nfeat in ((16, 1, 8), (16, 3, 8), (32, 2, 8), (16, 2, 16)):
                nw = api.decoder_num_weights(hidden, layers)
                ds.features = (0.5 * torch.randn((ds.n, nfeat), device=dev, generator=gen_v)).half()
                ds.mlp_weights = ((torch.rand((nw,), device=dev, generator=gen_v) - 0.5) * (16.0 / hidden) ** 0.5).half()
                ds.mlp_hidden, ds.mlp_layers, ds.num_features = hidden, layers, nfeat
                r.grads = api.alloc_grads(ds.n, 1, dev, nfeat, nw)
                v_one = timed(lambda: step(ds, r), args.steps, args.warmup)
                v_stage, _ = profile(lambda: step(ds, r), max(1, min(args.steps, 3)))
                v_streams = None
                if rs_v:                                               # the views on the lanes' streams, as the headline runs
                    for rr in rs_v[1:]:
                        rr.grads = api.alloc_grads(ds.n, 1, dev, nfeat, nw)
                    v_streams = timed(lambda: step_two_streams(ds, rs_v), args.steps, args.warmup)
                    for c, s_ in zip(lane_ctx, lanes):
                        api.gs_async_status(c, s_)
                api.gs_set_decoder_engine(ctx, api.GS_ENGINE_WARP_MMA)   # the fp32 kernels, dense over all Gaussians
                v_fma = timed(lambda: step(ds, r), args.steps, args.warmup)
                api.gs_set_decoder_engine(ctx, api.GS_ENGINE_AUTO)
                variants_step[f"h{hidden}_l{layers}_f{nfeat}"] = {
                    "weights": nw, "ms_per_step": v_streams, "ms_per_step_single_stream": v_one,
                    "ms_per_step_single_stream_fp32_fma_dense": v_fma,
                    "stages_ms_per_step": {k: round(v, 4) for k, v in v_stage.items() if v > 0}}
            ds.features, ds.mlp_weights, ds.mlp_hidden, ds.mlp_layers, ds.num_features, r.grads = keep
            del rs_v
        results[tag] = dict(ms=ms, ms_one=ms_one, ms_streams=ms_streams, graph=graph_note, unfused=unfused, half=half, variants_step=variants_step,
                            stage_ms=stage_ms, stage_launches=stage_launches, pairs=pairs,
                            entries=entries, visible=visible, records=records, with_gradient=with_gradient, evaluated=evaluated, composited=composited,
                            warp_steps=warp_steps, warp_steps_idle=warp_steps_idle,
                            host=host, ds=ds, r=r, app=tag)

    # ---- end to end through the public API with host buffers (neural arm)
    e2e_host = None if args.skip_e2e else measure_e2e(api, torch, ctx, results[head], cams, G, views, args, timed, dev)
    e2e = None if args.skip_e2e else measure_e2e_training(api, torch, lane_ctx, lanes, results[head], cams, G, views, args,
                                                           timed, dev, WIDTH, HEIGHT)

    # ---- appearance-decode sweep (separate-pass kernels, HBM resident)
    decode = None if (args.skip_decode or args.config != 3) else decode_sweep(api, torch, ctx, dev, peaks, args)
    adam = None if (args.skip_decode or args.config != 3) else adam_sweep(api, torch, ctx, dev, peaks, n)
    prepass = None if (args.skip_decode or args.config != 3) else prepass_sweep(api, torch, ctx, dev, peaks, args, scenes)
    sort_ref = None if (args.skip_decode or args.config != 3) else sort_reference(torch, results[head], cams, views, dev)

    if rank != 0:
        return
    neural = results[head]
    ms = neural["ms"]
    stage_ms = neural["stage_ms"]
    total_stage = sum(stage_ms.values()) or 1.0
    dominant = max(stage_ms, key=stage_ms.get)
    launches_per_step = int(round(sum(neural["stage_launches"].values())))
    clock_mhz = peaks["sm_max_mhz"]
    alu_peak = NUM_SMS * FP32_LANES_PER_SM * 2 * clock_mhz * 1e6 / 1e12   # TFLOP/s
    roof = stage_roofline(dominant, neural, views, n, peaks, alu_peak)
    # which run the fraction refers to: the stage times come from the single-stream pass, not from `value`
    roof["ms_per_step_single_stream"] = neural["ms_one"]
    roof["stage_sum_ms_per_step_single_stream"] = total_stage
    roof["stage_ms_per_step_single_stream"] = stage_ms[dominant]
    roof["launches_of_the_stage_per_step"] = views
    roof["note"] = ("achieved = algorithmic work of one launch / (stage_ms_per_step_single_stream / launches); `value` is the "
                    "same step with several views in flight on streams of their own, where stages overlap")
    if e2e is not None:
        e2e["what"] = ("e2e = a training iteration: " + e2e["what"] + ".  e2e_gradients_to_host = the other reading, every "
                       "input from the host and every output to it: scene parameters and upstream gradients start in pinned host "
                       "memory each step, the image and all per-Gaussian gradients of every view end there")
    if e2e_host is not None:
        e2e_host["what"] = ("scene parameters and upstream gradients start in pinned host memory each step; the image and all "
                            "per-Gaussian gradient buffers of every view end there (no optimiser step); the other reading of "
                            "'end to end' beside `e2e`")
    out = {
        "metric": METRIC, "value": replicas.job_ms_per_iteration(ms, 1, world), "unit": f"ms/iter ({views} views, fwd+bwd)", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": False,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl["name"], "appearance": head,
                   "n": n, "width": WIDTH, "height": HEIGHT, "views": views,
                   "cache": cache_note(args.config),
                   "multi_gpu": "replicas only"},
        "gprimitives_per_s": world * n * views / (ms * 1e-3) / 1e9,
        "ms_per_step_single_stream": neural["ms_one"], "ms_per_step_streams_no_graph": neural["ms_streams"],
        "cuda_graph": neural["graph"],
        "streams": 1 if views == 1 else n_lanes,
        "clocks": clocks, "e2e": e2e, "e2e_gradients_to_host": e2e_host, "gpu_launches": launches_per_step,
        "roofline": roof,
        "rooflines": {k: stage_roofline(k, neural, views, n, peaks, alu_peak)
                      for k in ("preprocess_fwd", "depth_sort", "keygen", "tile_sort", "tile_ranges", "blend_fwd",
                                "blend_bwd", "preprocess_bwd") if stage_ms.get(k, 0) > 0},
        "stages_ms_per_step": {k: round(v, 4) for k, v in stage_ms.items() if v > 0},
        "stage_share": {k: round(v / total_stage, 4) for k, v in stage_ms.items() if v > 0},
        "pairs_per_view": neural["pairs"], "visible_per_view": neural["visible"] / views,
        "with_gradient_per_view": neural["with_gradient"] / views,
        "blend_warp_steps_per_view": neural["warp_steps"] / views,
        "blend_warp_steps_without_a_taker_per_view": neural["warp_steps_idle"] / views,
        "sh": None if "sh" not in results or head == "sh" else {
            "ms_per_step": results["sh"]["ms"], "ms_per_step_single_stream": results["sh"]["ms_one"],
            "stages_ms_per_step": {k: round(v, 4) for k, v in results["sh"]["stage_ms"].items() if v > 0}},
        "sv": None if "sv" not in results or head == "sv" else {
            "ms_per_step": results["sv"]["ms"], "ms_per_step_single_stream": results["sv"]["ms_one"],
            "stages_ms_per_step": {k: round(v, 4) for k, v in results["sv"]["stage_ms"].items() if v > 0}},
        "neural_half_precision": results[head].get("half") if head == "neural" else None,
        "separate_pass_step": {t: results[t]["unfused"] for t in results if results[t].get("unfused")} or None,
        "decoder_variants_step": results[head].get("variants_step") if head == "neural" else None,
        "appearance_decode": decode,
        "adam_update": adam,
        "viewer_prepass": prepass,
        "sort_reference": sort_ref,
        "peaks": peaks,
    }
    if not args.skip_cpu:
        out["cpu_baseline"] = cpu_baseline(neural["host"], cams_host, n)
    print(json.dumps(out))


# Figures read from ncu captures of single launches (orbit view 0 of the default workload) live in
# profiles/ncu_constants.json, each with the command that produced it and the commit it was taken at:
#   dram_bytes    dram__bytes_read.sum + dram__bytes_write.sum of the launch
#   issue_active  smsp__issue_active.avg.pct_of_peak_sustained_active / 100: the share of issue slots the kernel
#                 fills while it runs.  For the ALU-bound blend kernels this, not the flop rate, says how close to
#                 the machine they are: the flop count is the method's minimum arithmetic, the issue slots also
#                 carry loads, predicates, shuffles and loop control.
def ncu_constants():
    path = os.path.join(ROOT, "profiles", "ncu_constants.json")
    if not os.path.exists(path):
        return None
    return json.load(open(path))


# Names of the timed stages (the C ABI's stage enumeration) and the kernels behind them.
STAGE_KERNELS = {
    "preprocess_fwd": "k_preprocess_fwd (projection, fused appearance, cell records of 4x4 tiles)",
    "depth_sort": "4 x (k_radix_hist, k_radix_scan_rows, k_radix_scatter<8>) on the 32-bit depth keys of all Gaussians",
    "keygen": "k_emit_records: (cell id, 16-bit tile mask) records in depth order",
    "tile_sort": "k_radix_hist, k_radix_scan_rows, k_radix_scatter<9>: one stable pass on the cell id",
    "tile_ranges": "k_cell_chunks, k_chunk_counts, k_cell_prefix, k_tile_scan, k_expand: records -> per-tile lists",
    "blend_fwd": "k_blend_fwd", "blend_bwd": "k_blend_bwd",
    "preprocess_bwd": "k_preprocess_bwd_sparse (zero rows at once, the Gaussians with a gradient in full batches) + k_wgrad_reduce"}


def stage_roofline(stage, arm, views, n, peaks, alu_peak):
    out = _stage_roofline(stage, arm, views, n, peaks, alu_peak)
    out["kernels"] = STAGE_KERNELS.get(stage)
    out["ms_per_launch"] = arm["stage_ms"][stage] / views
    out["timed_as"] = "single stream, views one after another (CUDA events around the stage's launches)"
    out["traffic_source"] = None
    consts = ncu_constants()
    if consts and n == consts.get("n") and arm.get("app") == consts.get("appearance"):
        e = consts["entries"].get(stage)
        if e:
            out["traffic"] = e.get("dram_bytes")
            out["issue_active_frac_ncu"] = e.get("issue_active")
            out["fma_pipe_active_frac_ncu"] = e.get("fma_pipe_cycles_active")
            out["alu_pipe_active_frac_ncu"] = e.get("alu_pipe_cycles_active")
            out["traffic_source"] = (f"profiles/ncu_constants.json: {e.get('kernel')} ({e.get('launch')}), "
                                     f"captured at commit {e.get('commit') or consts.get('commit')}")
    return out


def _stage_roofline(stage, arm, views, n, peaks, alu_peak):
    ms = arm["stage_ms"][stage] / views          # average duration of one launch of the stage
    if stage in ("blend_fwd", "blend_bwd"):
        if stage == "blend_fwd":
            ev, per_c = arm["evaluated"] / views, BLEND_FWD_FLOPS_PER_COMPOSITED
        else:   # the backward walks each pixel's list only up to its last composited entry
            ev, per_c = arm["entries"] / views, BLEND_BWD_FLOPS_PER_COMPOSITED
        co = arm["composited"] / views
        flops = BLEND_FLOPS_PER_EVALUATED * ev + per_c * co
        achieved = flops / (ms * 1e-3) / 1e12
        return {"kernel": stage, "bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "TFLOP/s",
                "frac": achieved / alu_peak, "traffic": None, "peak_source": "148 SMs x 128 lanes x 2 x max SM clock",
                "evaluated_per_launch": ev, "composited_per_launch": co,
                "flops_per_evaluated": BLEND_FLOPS_PER_EVALUATED, "flops_per_composited": per_c}
    vis = arm["visible"] / views
    P = sum(arm["pairs"]) / views                # (Gaussian, tile) instances of a view
    R = arm["records"] / views                   # (Gaussian, cell of 4 x 4 tiles) records of a view
    app_bytes = 28.0
    per_launch = {"preprocess_fwd": 44.0 * n + 12.0 * n + (app_bytes + 48.0) * vis + 4.0 * R,
                  # rectangle of every Gaussian, 2D gradients of the visible ones, a gradient row for every Gaussian;
                  # parameters and 2D gradients again for the ones that received a gradient
                  "preprocess_bwd": 8.0 * n + 48.0 * vis + 88.0 * n + (44.0 + 48.0 + app_bytes) * (arm["with_gradient"] / views),
                  "depth_sort": (4 * 20.0 - 4.0) * n,     # per pass: keys read twice, values once, both written
                  "keygen": 8.0 * n + 12.0 * R,           # id + count per Gaussian; record read, key + value written
                  "tile_sort": 20.0 * R,                  # one pass: keys read twice, values once, both written
                  "tile_ranges": 12.0 * R + 4.0 * P}.get(stage, 0.0)   # keys twice + values read, ids written
    achieved = per_launch / (ms * 1e-3) / 1e9
    return {"kernel": stage, "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peaks["source"],
            "algorithmic_bytes_per_launch": per_launch, "visible": vis, "instances": P, "records": R}


def measure_e2e(api, torch, ctx, arm, cams, G, views, args, timed, dev):
    """Same step, but the scene parameters and upstream gradients start in pinned host memory and the
    image and every gradient buffer of every view end there: the host<->device copies are inside the
    timed region.  The copies run on their own streams (one per direction) against double-buffered
    device buffers, so that view v's results travel while view v+1 is computed; the step ends when the
    last copy has landed."""
    host, ds, r = arm["host"], arm["ds"], arm["r"]
    pin = lambda t: t.cpu().pin_memory()
    app_names = ["features", "mlp_weights"] if arm["app"] == "neural" else ["sh_rest"]
    names = ["means", "log_scales", "quats", "opacity_logits", "base_color"] + app_names
    h_scene = {k: pin(getattr(ds, k)) for k in names}
    h_G = pin(G)
    grads = [r.grads, api.alloc_grads(ds.n, r.app, dev)]
    images = [r.image, torch.empty_like(r.image)]
    h_grads = {k: torch.empty_like(getattr(grads[0], k), device="cpu").pin_memory() for k in names}
    h_image = torch.empty_like(r.image, device="cpu").pin_memory()
    d_G = [torch.empty_like(G[0]), torch.empty_like(G[0])]
    h2d = sum(t.numel() * t.element_size() for t in h_scene.values()) + views * d_G[0].numel() * 4
    d2h = views * (sum(t.numel() * t.element_size() for t in h_grads.values()) + h_image.numel() * 4)
    main = torch.cuda.current_stream(dev)
    up, down = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_up = [torch.cuda.Event(), torch.cuda.Event()]
    ev_down = [torch.cuda.Event(), torch.cuda.Event()]
    ev_done = [torch.cuda.Event() for _ in range(views)]

    def step():
        up.wait_stream(main)                       # the previous step no longer reads the scene
        with torch.cuda.stream(up):
            for k in names:
                getattr(ds, k).copy_(h_scene[k], non_blocking=True)
            d_G[0].copy_(h_G[0], non_blocking=True)
            ev_up[0].record(up)
        for v in range(views):
            b = v & 1
            if v + 1 < views:
                with torch.cuda.stream(up):
                    if v >= 1:
                        up.wait_event(ev_done[v - 1])   # d_G[1 - b] was the input of view v - 1
                    d_G[1 - b].copy_(h_G[v + 1], non_blocking=True)
                    ev_up[1 - b].record(up)
            main.wait_event(ev_up[b])
            if v >= 2:
                main.wait_event(ev_down[b])         # view v - 2 has left buffer set b
            r.image, r.grads = images[b], grads[b]
            r.forward(ds, cams[v])
            r.backward(ds, cams[v], d_G[b])
            ev_done[v].record(main)
            with torch.cuda.stream(down):
                down.wait_event(ev_done[v])
                h_image.copy_(images[b], non_blocking=True)
                for k in names:
                    h_grads[k].copy_(getattr(grads[b], k), non_blocking=True)
                ev_down[b].record(down)
        main.wait_stream(down)

    ms = timed(step, max(2, args.steps // 2), 2)
    r.image, r.grads = images[0], grads[0]
    return {"value": ms, "unit": f"ms/iter ({views} views, fwd+bwd)", "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "overlap": "copies on their own streams, double-buffered"}


def measure_e2e_training(api, torch, lane_ctx, lanes, arm, cams, G, views, args, timed, dev, WIDTH, HEIGHT):
    """One training iteration end to end, as a trainer would run it: the scene lives on the device; every step
    the upstream gradients of the views come from pinned host memory, the views are rendered forward and
    backward (each into gradient buffers of its own, on the lanes' streams, without host waits), ONE fused Adam
    launch sums the views' gradients and updates all parameters (fp32 masters, half copies for the next step),
    and the rendered images go back to pinned host memory.  Copies run on streams of their own."""
    ds, r0 = arm["ds"], arm["r"]
    neural = arm["app"] == "neural"
    n = ds.n
    rs = [r0] + [api.Renderer(c, n, WIDTH, HEIGHT, r0.app, pair_capacity=r0.pair_capacity) for c in lane_ctx[1:]]
    group = min(views, 8)              # views per Adam update: one launch sums at most eight gradient sets
    grads = [r0.grads] + [api.alloc_grads(n, r0.app, dev) for _ in range(group - 1)]
    # two sets of image and upstream-gradient buffers: the copies of one step overlap the kernels of the next
    images2 = [[r0.image] + [torch.empty_like(r0.image) for _ in range(group - 1)],
               [torch.empty_like(r0.image) for _ in range(group)]]
    h_G = G.cpu().pin_memory()
    d_G2 = [torch.empty_like(G), torch.empty_like(G)]
    h_images = torch.empty((views,) + tuple(r0.image.shape), dtype=torch.float32).pin_memory()
    y0 = 0.28209479177387814
    spec = [("means", 3, 1.6e-6), ("log_scales", 3, 5e-5), ("quats", 4, 1e-5), ("opacity_logits", 1, 5e-4)]
    spec += [("base_color", 3, 0.00025), ("features", 8, 0.008e-2), ("mlp_weights", 1, 0.003e-2)] if neural else \
            [("base_color", 3, 0.0025 * y0 * 1e-2), ("sh_rest", 45, 0.000125e-2)]
    masters, moments = {}, {}
    for name, cols, lr in spec:        # rates scaled down: random upstream gradients must not wreck the synthetic scene
        stored = getattr(ds, name)
        masters[name] = stored.float().contiguous() if stored.dtype != torch.float32 else stored
        moments[name] = (torch.zeros_like(masters[name]), torch.zeros_like(masters[name]))

    def adam_tensors(count):           # the update that sums the first `count` gradient sets
        out = []
        for name, cols, lr in spec:
            stored = getattr(ds, name)
            out.append(api.AdamTensor(masters[name], getattr(grads[0], name), moments[name][0], moments[name][1], [lr] * cols,
                                      0.9, 0.99 if name == "mlp_weights" else 0.999, 1e-15,
                                      half_copy=stored if stored.dtype == torch.float16 else None,
                                      more_grads=[getattr(g, name) for g in grads[1:count]]))
        return out

    tensors_for = {c: adam_tensors(c) for c in {min(group, views - b) for b in range(0, views, group)}}
    main = torch.cuda.current_stream(dev)
    up, down = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_up = [torch.cuda.Event() for _ in range(views)]
    ev_done = [torch.cuda.Event() for _ in range(views)]
    state = {"step": 0, "iter": 0}
    ev_kernels_done = [torch.cuda.Event(), torch.cuda.Event()]   # the kernels of the last step that used buffer set p
    ev_images_out = [torch.cuda.Event(), torch.cuda.Event()]     # ... and its image downloads
    used = [False, False]
    L = len(lanes)

    def step():
        p = state["iter"] % 2
        state["iter"] += 1
        d_G, images = d_G2[p], images2[p]
        if used[p]:
            up.wait_event(ev_kernels_done[p])      # the step before last has read this set's upstream gradients
        with torch.cuda.stream(up):
            for v in range(views):
                d_G[v].copy_(h_G[v], non_blocking=True)
                ev_up[v].record(up)
        for b in range(0, views, group):
            for s in lanes:
                s.wait_stream(main)                # the parameters of this group are in place
                if used[p] and b == 0:
                    s.wait_event(ev_images_out[p])  # this set's images have left for the host
            count = min(group, views - b)
            for k in range(count):
                v = b + k
                r, s = rs[v % L], lanes[v % L]
                s.wait_event(ev_up[v])
                r.image, r.grads = images[k], grads[k]
                r.forward_async(ds, cams[v], stream=s)
                r.backward(ds, cams[v], d_G[v], stream=s)
                ev_done[v].record(s)
                with torch.cuda.stream(down):
                    down.wait_event(ev_done[v])
                    h_images[v].copy_(images[k], non_blocking=True)
            for s in lanes:
                main.wait_stream(s)
            if b + group < views:
                main.wait_stream(down)             # the next group renders into the same image buffers
            state["step"] += 1
            api.gs_adam_step(lane_ctx[0], tensors_for[count], state["step"])
        ev_kernels_done[p].record(main)
        ev_images_out[p].record(down)
        used[p] = True

    ms = timed(step, max(2, args.steps // 2), 3, drain=lambda: main.wait_stream(down))
    for c, s_ in zip(lane_ctx, lanes):
        api.gs_async_status(c, s_)
    finite = all(bool(torch.isfinite(m).all()) for m in masters.values())
    r0.image, r0.grads = images2[0][0], grads[0]
    return {"value": ms, "unit": f"ms/iter ({views} views, fwd+bwd, + one fused Adam update per {group} views)",
            "h2d_bytes_per_step": int(h_G.numel() * 4), "d2h_bytes_per_step": int(h_images.numel() * 4),
            "what": "upstream gradients in, rendered images out, parameters stay on the device and are updated by Adam; "
                    "two buffer sets, so one step's copies overlap the next step's kernels",
            "streams": L, "parameters_finite_after_run": finite}


def sort_reference(torch, arm, cams, views, dev):
    """Context for the ordering stages: the library's stable sort of one view's instance list as 64-bit
    (tile, depth bits) keys with the Gaussian ids as values - the one-key formulation - timed as a library
    call beside this library's ordering (depth sort of the Gaussians, then records per cell of 4 x 4 tiles sorted by
    cell and expanded into the per-tile lists)."""
    r = arm["r"]
    r.forward(arm["ds"], cams[0])      # view 0's lists, with the host-side count
    torch.cuda.synchronize()
    P = int(r.num_pairs)
    tiles = r.binning.sorted_tiles[:P].to(torch.int64)
    vals = r.binning.sorted_vals[:P].to(torch.int64)
    depth = r.proj.depth_key.view(torch.int32).to(torch.int64) & 0xffffffff
    keys = (tiles << 32) | depth[vals]
    gen = torch.Generator(device=dev); gen.manual_seed(9)
    perm = torch.randperm(P, device=dev, generator=gen)
    keys, vals = keys[perm].contiguous(), vals[perm].to(torch.int32).contiguous()
    ts = []
    for i in range(8):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        sk, order = torch.sort(keys, stable=True)
        sv = vals[order]
        e1.record()
        torch.cuda.synchronize()
        if i >= 3:
            ts.append(e0.elapsed_time(e1))
    ts.sort()
    ours = sum(arm["stage_ms"][k] for k in ("depth_sort", "keygen", "tile_sort", "tile_ranges")) / views
    return {"instances": P, "library_sort_64bit_keys_ms": round(ts[len(ts) // 2], 4),
            "this_library_ordering_ms_per_view": round(ours, 4),
            "what": "torch.sort(stable) of (tile << 32 | depth bits) keys + gather of the ids (the one-key formulation, keys already "
                    "emitted), against this library's whole ordering of one view: depth sort of the Gaussians, record emission, "
                    "record sort by cell and expansion into the per-tile lists"}


def adam_sweep(api, torch, ctx, dev, peaks, n):
    """The step that follows the rendering path: one fused Adam update of every parameter of a model, SH
    (59 floats per Gaussian) against neural (22 floats + 816 weights), one launch each.  The tensors are far
    larger than L2 (16 B of state per element), so the stream is measured from HBM."""
    y0 = 0.28209479177387814
    geo = [("means", 3, 1.6e-4), ("log_scales", 3, 5e-3), ("quats", 4, 1e-3), ("opacity_logits", 1, 5e-2)]
    sv_rates = ([0.0008] * 3 + [0.002] * 3 + [0.006]) * 7      # per site: colour, site direction, temperature (App. B)
    sets = {"sh": geo + [("base_color", 3, 0.0025 * y0), ("sh_rest", 45, 0.000125)],
            "neural": geo + [("base_color", 3, 0.00025), ("features", 8, 0.008), ("mlp_weights", 1, 0.003)],
            "sv": geo + [("base_color", 3, 0.0008), ("sv_sites", 49, sv_rates)]}
    out = {}
    for tag, spec in sets.items():
        gen = torch.Generator(device=dev); gen.manual_seed(77)
        tensors, nbytes = [], 0
        for name, cols, lr in spec:
            rows = 816 if name == "mlp_weights" else n
            p = torch.randn((rows, cols), device=dev, generator=gen)
            g = torch.randn((rows, cols), device=dev, generator=gen) * 1e-3
            m, v = torch.zeros_like(p), torch.zeros_like(p)
            half = torch.empty((rows, cols), device=dev, dtype=torch.float16) if name in ("features", "mlp_weights") else None
            tensors.append(api.AdamTensor(p, g, m, v, lr if isinstance(lr, list) else [lr] * cols, 0.9,
                                          0.99 if name == "mlp_weights" else 0.999, 1e-15, half_copy=half))
            nbytes += rows * cols * (28 + (2 if half is not None else 0))
        for it in range(3):
            api.gs_adam_step(ctx, tensors, it + 1)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 20
        e0.record()
        for it in range(reps):
            api.gs_adam_step(ctx, tensors, it + 4)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[tag] = {"ms": round(ms, 4), "bytes_per_gaussian": round(nbytes / n, 1), "GBps": round(gbs, 1),
                    "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4), "launches_per_update": 1}
        del tensors
    out["n"] = n
    out["cache"] = "tensors larger than L2 (352 MB neural, 944 MB SH at 1M)"
    return out


def prepass_sweep(api, torch, ctx, dev, peaks, args, scenes):
    """The viewer's per-frame colour prepass of the neural model (560 MAC per Gaussian on tensor cores, one RGBA8
    texel out) and its one-off export fold, at 1M / 3M / 10M Gaussians.  64 B move per Gaussian and frame."""
    out = {}
    sizes = [1_000_000, 3_000_000, 10_000_000] if not args.quick else [1_000_000]
    cam = api.make_camera(scenes.orbit_cameras(WIDTH, HEIGHT, 8)[1])
    flush = torch.empty(64 * 1024 * 1024, device=dev, dtype=torch.float32)
    for n in sizes:
        sc, _, _ = scenes.config5(n, scenes.APP_NEURAL)
        ds = api.upload_scene(sc, dev)
        pre = torch.empty((n, 16), device=dev, dtype=torch.float16)
        rgba = torch.empty((n, 4), device=dev, dtype=torch.uint8)
        api.gs_neural_fold(ctx, ds, pre)
        for _ in range(3):
            api.gs_neural_prepass(ctx, ds, pre, cam, rgba)
        torch.cuda.synchronize()
        t_fold = t_pre = 0.0
        reps = 10
        for _ in range(reps):
            flush.zero_()
            e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
            e0.record(); api.gs_neural_fold(ctx, ds, pre); e1.record()
            flush.zero_()
            e0b = torch.cuda.Event(enable_timing=True); e0b.record()
            api.gs_neural_prepass(ctx, ds, pre, cam, rgba); e2.record()
            torch.cuda.synchronize()
            t_fold += e0.elapsed_time(e1); t_pre += e0b.elapsed_time(e2)
        ms = t_pre / reps
        gbs = 64.0 * n / (ms * 1e-3) / 1e9
        out[f"{n // 1_000_000}M"] = {"prepass_ms": round(ms, 4), "fold_ms": round(t_fold / reps, 4), "bytes_per_gaussian": 64,
                                      "GBps": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
                                      "Ggaussians_per_s": round(n / (ms * 1e-3) / 1e9, 3), "mac_per_gaussian": 560}
        del ds, pre, rgba
    out["cache"] = "L2 flushed between iterations (256 MiB write)"
    return out


def decode_sweep(api, torch, ctx, dev, peaks, args):
    """Separate-pass colour decode forward + backward at 1M / 3M / 10M Gaussians: SH, neural, Spherical Voronoi."""
    out = {}
    sizes = [1_000_000, 3_000_000, 10_000_000] if not args.quick else [1_000_000]
    for n in sizes:
        gen = torch.Generator(device=dev); gen.manual_seed(5000 + n % 997)
        dirs = torch.randn((n, 3), device=dev, generator=gen)
        dirs = (dirs / dirs.norm(dim=1, keepdim=True)).contiguous()
        gcol = torch.randn((n, 3), device=dev, generator=gen)
        base = 0.14 + 0.03 * torch.randn((n, 3), device=dev, generator=gen)
        z = torch.zeros((1, 4), device=dev)
        for app, tag in ((0, "sh"), (1, "neural"), (2, "sv")):
            if app == 2:     # Spherical Voronoi: 7 sites x 7 raw parameters = 196 B per primitive
                sites = torch.randn((n, 7, 7), device=dev, generator=gen)
                sites[:, :, 0:3] *= 0.15
                sc = api.DeviceScene(z, z, z, z[0], base, 2, 3, sv_sites=sites.contiguous())
                bytes_fwd, bytes_bwd = 196 + 12 + 12, 12 + 196 + 12 + 196 + 12 + 12
            elif app == 0:
                sc = api.DeviceScene(z, z, z, z[0], base, 0, 3, sh_rest=0.05 * torch.randn((n, 15, 3), device=dev, generator=gen))
                bytes_fwd, bytes_bwd = 192 + 12 + 12, 12 + 192 + 12 + 192 + 12 + 12
            else:
                w = (torch.rand((816,), device=dev, generator=gen) - 0.5).half()
                sc = api.DeviceScene(z, z, z, z[0], base, 1, 3,
                                     features=(0.1 * torch.randn((n, 8), device=dev, generator=gen)).half(), mlp_weights=w)
                bytes_fwd, bytes_bwd = 28 + 12 + 12, 12 + 12 + 28 + 12 + 32 + 12
            color = torch.empty((n, 3), device=dev)
            grads = api.alloc_grads(n, app, dev)
            gd = torch.empty((n, 3), device=dev)
            flush = torch.empty((256 << 20,), device=dev, dtype=torch.uint8)

            def run(fn, reps=10):
                ts = []
                for i in range(reps + 3):
                    flush.zero_()                      # evict L2 between iterations
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(); fn(); e1.record()
                    torch.cuda.synchronize()
                    if i >= 3:
                        ts.append(e0.elapsed_time(e1))
                ts.sort()
                return ts[len(ts) // 2]
            for precision in ((0, 1) if app == 1 else (0,)):
              sc.decoder_precision = precision
              row = f"{tag}{'_half' if precision else ''}_{n // 1_000_000}M"
              f_ms = run(lambda: api.gs_appearance_forward(ctx, sc, dirs, color))
              b_ms = run(lambda: api.gs_appearance_backward(ctx, sc, dirs, gcol, grads, gd))
              gbs = (bytes_fwd + bytes_bwd) * n / ((f_ms + b_ms) * 1e-3) / 1e9
              out[row] = {
                "fwd_ms": round(f_ms, 4), "bwd_ms": round(b_ms, 4), "bytes_per_primitive": bytes_fwd + bytes_bwd,
                "GBps": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
                "fwd_GBps": round(bytes_fwd * n / (f_ms * 1e-3) / 1e9, 1),
                "bwd_GBps": round(bytes_bwd * n / (b_ms * 1e-3) / 1e9, 1),
                "Gprimitives_per_s": round(n / ((f_ms + b_ms) * 1e-3) / 1e9, 3)}
              if app == 1:      # the row above is the default engine (per kernel the faster); both engines on their own
                for eng, name in ((api.GS_ENGINE_WARP_MMA, "warp_mma"), (api.GS_ENGINE_TCGEN05, "tcgen05")):
                    api.gs_set_decoder_engine(ctx, eng)
                    out[row]["fwd_ms_" + name] = round(run(lambda: api.gs_appearance_forward(ctx, sc, dirs, color)), 4)
                    out[row]["bwd_ms_" + name] = round(run(lambda: api.gs_appearance_backward(ctx, sc, dirs, gcol, grads, gd)), 4)
                api.gs_set_decoder_engine(ctx, api.GS_ENGINE_AUTO)
            del sc, color, grads, gd, flush
        # the decoder variants of the architecture table (App. D): 1M only; the default engine runs them on tcgen05,
        # GS_ENGINE_WARP_MMA selects the fp32 CUDA-core kernels they were first built on
        for hidden, layers, nfeat in (((16, 1, 8), (16, 3, 8), (32, 2, 8), (16, 2, 16)) if n == 1_000_000 else ()):
            nw = api.decoder_num_weights(hidden, layers)
            w = ((torch.rand((nw,), device=dev, generator=gen) - 0.5) * (16.0 / hidden) ** 0.5).half()
            sc = api.DeviceScene(z, z, z, z[0], base, 1, 3,
                                 features=(0.1 * torch.randn((n, nfeat), device=dev, generator=gen)).half(), mlp_weights=w,
                                 mlp_hidden=hidden, mlp_layers=layers, num_features=nfeat)
            fb = 2 * nfeat
            bytes_fwd, bytes_bwd = fb + 12 + 12 + 12, 12 + 12 + fb + 12 + 12 + 4 * nfeat + 12
            color = torch.empty((n, 3), device=dev)
            grads = api.alloc_grads(n, 1, dev, nfeat, nw)
            gd = torch.empty((n, 3), device=dev)
            flush = torch.empty((256 << 20,), device=dev, dtype=torch.uint8)

            def run_v(fn, reps=10):
                ts = []
                for i in range(reps + 3):
                    flush.zero_()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(); fn(); e1.record()
                    torch.cuda.synchronize()
                    if i >= 3:
                        ts.append(e0.elapsed_time(e1))
                ts.sort()
                return ts[len(ts) // 2]
            f_ms = run_v(lambda: api.gs_appearance_forward(ctx, sc, dirs, color))
            b_ms = run_v(lambda: api.gs_appearance_backward(ctx, sc, dirs, gcol, grads, gd))
            api.gs_set_decoder_engine(ctx, api.GS_ENGINE_WARP_MMA)
            f_fma = run_v(lambda: api.gs_appearance_forward(ctx, sc, dirs, color))
            b_fma = run_v(lambda: api.gs_appearance_backward(ctx, sc, dirs, gcol, grads, gd))
            api.gs_set_decoder_engine(ctx, api.GS_ENGINE_AUTO)
            # forward: one pass over the weights; backward: the forward again, the transposed pass and the weight gradient
            flop_fwd, flop_bwd = 2 * nw * n, 6 * nw * n
            gbs = (bytes_fwd + bytes_bwd) * n / ((f_ms + b_ms) * 1e-3) / 1e9
            dflt = out[f"neural_{n // 1_000_000}M"]          # the default decoder (816 weights) on the same Gaussians
            out[f"neural_h{hidden}_l{layers}_f{nfeat}_{n // 1_000_000}M"] = {
                "weights": nw, "engine": "tcgen05", "fwd_ms": round(f_ms, 4), "bwd_ms": round(b_ms, 4),
                "fwd_ms_fp32_fma": round(f_fma, 4), "bwd_ms_fp32_fma": round(b_fma, 4),
                "bytes_per_primitive": bytes_fwd + bytes_bwd,
                "GBps": round(gbs, 1), "frac_of_hbm_peak": round(gbs / peaks["hbm_gbs"], 4),
                "fwd_TFLOPs": round(flop_fwd / (f_ms * 1e-3) / 1e12, 2),
                "bwd_TFLOPs": round(flop_bwd / (b_ms * 1e-3) / 1e12, 2),
                "fp32_fma_frac_of_fp32_alu_peak": round((flop_fwd + flop_bwd) / ((f_fma + b_fma) * 1e-3) / 1e12 / FP32_ALU_PEAK_TFLOPS, 4),
                "time_per_weight_over_default_decoder": {
                    "fwd": round((f_ms / nw) / (dflt["fwd_ms"] / 816), 3), "bwd": round((b_ms / nw) / (dflt["bwd_ms"] / 816), 3)},
                "Gprimitives_per_s": round(n / ((f_ms + b_ms) * 1e-3) / 1e9, 3)}
            del sc, color, grads, gd, flush
        del dirs, gcol, base
        torch.cuda.empty_cache()
    out["cache"] = "L2 flushed between iterations (256 MiB write)"
    return out


# ---------------------------------------------------------------------------------------------
# the oracle on the host cores (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_view_ms(host_scene, cam, G):
    from oracle import gs_oracle
    t0 = time.perf_counter()
    gs_oracle.render(host_scene, cam, G)
    return (time.perf_counter() - t0) * 1e3


def cpu_baseline(host_scene, cams, n):
    from oracle import gs_oracle
    from paper_2609_05255_b200 import scenes
    gs_oracle.build()
    views = len(cams)
    G = scenes.upstream_gradient(cams[0], 4242)
    sample = min(views, 4 if n <= 1_500_000 else 2)          # about 10 s of host time at the headline size
    ms = sum(oracle_view_ms(host_scene, cams[v], G) for v in range(sample)) / sample
    return {"value": ms * views, "unit": f"ms/iter ({views} views, fwd+bwd)", "cores": gs_oracle.num_threads(),
            "kind": "oracle",
            "sample": f"{sample} of {views} views of the full {n}-Gaussian scene, fwd+bwd, mean per view scaled x{views}"}


def run_reference(args):
    rank, world, _ = dist_setup(args)
    if rank != 0:
        return
    from oracle import gs_oracle
    from paper_2609_05255_b200 import scenes
    gs_oracle.build()
    wl = workload_of(args, scenes)
    views, n, WIDTH, HEIGHT, cams = wl["views"], wl["n"], wl["width"], wl["height"], wl["cams"]
    host = wl["scene"](wl["arms"][0][0])
    Gs = [scenes.upstream_gradient(cams[0], 4242)]
    for _ in range(args.warmup):
        oracle_view_ms(host, cams[0], Gs[0])
    t = [oracle_view_ms(host, cams[k % views], Gs[0]) for k in range(args.steps)]
    ms = sum(t) / len(t) * views
    sample = f"each step = 1 of {views} views of the full {n}-Gaussian scene, fwd+bwd, scaled x{views}"
    out = {"impl": "reference", "metric": METRIC, "value": ms, "unit": f"ms/iter ({views} views, fwd+bwd)",
           "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
           "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           # the same keys and values as the other arm's line: it is the same workload
           "config": {"workload": wl["name"], "appearance": wl["arms"][0][1], "n": n, "width": WIDTH,
                      "height": HEIGHT, "views": views, "cache": cache_note(args.config), "multi_gpu": "replicas only"},
           "cpu_baseline": {"value": ms, "unit": f"ms/iter ({views} views, fwd+bwd)", "cores": gs_oracle.num_threads(),
                            "kind": "oracle", "sample": sample},
           "e2e": {"value": ms, "unit": f"ms/iter ({views} views, fwd+bwd)", "h2d_bytes_per_step": 0,
                   "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3, choices=[1, 2, 3, 4],
                    help="workload (3 = the headline: 1M Gaussians, 8 views; the others fill the results table)")
    ap.add_argument("--n", type=int, default=None, help="override the Gaussian count of config 3")
    ap.add_argument("--views", type=int, default=None, help="override the number of views of configs 3 and 4")
    ap.add_argument("--quick", action="store_true", help="decode sweep at 1M only")
    ap.add_argument("--skip-decode", action="store_true")
    ap.add_argument("--skip-cpu", action="store_true")
    ap.add_argument("--skip-sh", action="store_true", help="time the neural arm only (profiling runs)")
    ap.add_argument("--skip-e2e", action="store_true")
    ap.add_argument("--single-stream", action="store_true", help="time the views one after another on one stream only")
    ap.add_argument("--no-graph", action="store_true", help="do not try the CUDA-graph replay of the multi-stream iteration")
    ap.add_argument("--streams", type=int, default=4, help="views in flight (each on its own stream, context and buffers)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
