#!/usr/bin/env python
"""Benchmark of the ViT pipeline-stage forward on B200.

One step = one pass of the whole hot path over one batch of synthetic images: patch embed,
every stage of the partition, classification head.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload huge14|large16|base16]
  python bench.py --impl reference ...     # times the CPU oracle instead (bounded sample per step)

With N > 1 (launched under torchrun) every rank runs an independent replica on its own GPU
(images are independent, there is no data-path collective); the value is the aggregate.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import vitgen  # noqa: E402

WORKLOADS = {
    # name: (preset, batch, microbatch, stages) -- the single-GPU configurations of the metric
    "huge14": ("huge14", 128, 128, 1),
    "large16": ("large16", 128, 8, 16),
    "base16": ("base16", 64, 16, 4),
    "small16": ("small16", 64, 16, 4),
    # the compressed (distilled) family, 198 tokens
    "deit_base16": ("deit_base16", 64, 16, 4),
    "deit_small16": ("deit_small16", 64, 16, 4),
    "deit_tiny16": ("deit_tiny16", 64, 16, 4),
}
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the fc1 GEMM, from the ncu capture
# whose summary is kept under profiles/ (same kernel build); None = not captured
NCU_TRAFFIC = {"huge14": 384.4e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL_BF16_TFLOPS = 2250.0   # datasheet dense bf16 figure of the B200 (context; the measured peaks are the denominators)


def max_over_ranks(ms, dist=None, device=None):
    """Slowest rank's time: the job is as fast as its slowest replica.  `dist` is torch.distributed
    (initialised) or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_images_per_s(world, batch_per_rank, ms_per_step):
    """Whole-job throughput of `world` independent replicas that each process `batch_per_rank`
    images per step (weak scaling, no data-path collective)."""
    return world * batch_per_rank / (ms_per_step / 1e3)


def rank_pixel_seed(rank):
    """Each replica gets its own images."""
    return rank


def flops_per_image(s):
    T, H, F = s.tokens, s.hidden, s.mlp_dim
    gemm = {
        "qkv": 2 * T * 3 * H * H, "outproj": 2 * T * H * H, "fc1": 2 * T * H * F, "fc2": 2 * T * H * F,
    }
    attn = 4 * T * T * H
    embed = 2 * s.n_patches * s.patch_k * H
    head = 2 * H * s.num_classes
    total = s.layers * (sum(gemm.values()) + attn) + embed + head
    return total, gemm, attn, embed


def stage_counts(shape, n_stages, seed=0):
    if n_stages == 1:
        return [shape.layers]
    if shape.layers % n_stages == 0 and n_stages != 16:
        return [shape.layers // n_stages] * n_stages
    return [b - a for a, b in vitgen.uneven_partition(n_stages, shape.layers, seed)]


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            self.t.join(timeout=2)

    def summary(self):
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": max(mx), "power_w": float(np.median(pw)),
                "reasons": sorted(reasons), "samples": len(sm)}


def oracle_images_per_s(shape, n_images, seed=0, params=None):
    """Times the CPU oracle, as it stands, on `n_images` images of the workload."""
    from oracle import vit_oracle as O
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        cores = os.cpu_count() or 1
    if params is None:
        params, _ = vitgen.make_params(shape, seed=seed)
    pix = vitgen.make_pixels(shape, n_images, seed=seed)
    t0 = time.perf_counter()
    O.forward(params, shape, pix)
    dt = time.perf_counter() - t0
    return n_images / dt, cores, dt


def microbatch_sweep(vit, model, shape, dev, torch, total=256, sizes=(1, 2, 4, 8, 16, 32, 64, 128, 256)):
    """Microbatch sizes through an equal 4-stage partition: `total` images split into microbatches
    issued round-robin on min(4, total/mb) streams (throughput), and one microbatch alone on one
    stream (latency per image).  Needs max_microbatch >= the largest size that is run."""
    counts = stage_counts(shape, 4)
    out = []
    pix = torch.from_numpy(vitgen.make_pixels(shape, total, seed=1)).to(dev)
    logits = torch.empty((total, shape.num_classes), dtype=torch.float32, device=dev)
    for mb in sizes:
        if mb > model.cfg.max_microbatch:
            continue
        ns = max(1, min(4, total // mb))
        wss, streams, wsb = model.make_pipeline_buffers(mb, ns)

        def run_all():
            model.run_pipeline(counts, mb, pix, logits, wss, streams, wsb)

        def run_one():
            model.run_pipeline(counts, mb, pix[:mb], logits[:mb], wss[:1], streams[:1], wsb)

        res = {"microbatch": mb, "streams": ns}
        for fn, key, imgs, reps in ((run_all, "images_per_s", total, 3), (run_one, "latency_ms_per_image", mb, 5)):
            for _ in range(2):
                fn()
            torch.cuda.synchronize(dev)
            t0 = time.perf_counter()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(streams[0])
            for s in streams[1:]:
                s.wait_event(e0)
            for _ in range(reps):
                fn()
            for s in streams[1:]:
                e = torch.cuda.Event()
                e.record(s)
                streams[0].wait_event(e)
            e1.record(streams[0])
            torch.cuda.synchronize(dev)
            ms = e0.elapsed_time(e1) / reps
            res[key] = imgs / (ms / 1e3) if key == "images_per_s" else ms / imgs
            if key == "latency_ms_per_image":
                res["latency_ms_per_microbatch"] = ms
        for s in streams:
            model.check(s)
        out.append(res)
        del wss
    return out


def measure_workload(vit, torch, dev, name, steps=5, warmup=3, group=1):
    """Device-timed images/s of one of the named workloads (inputs resident), used for the extra
    workloads reported beside the headline one.  `group` > 1 carries that many microbatches through
    every launch together."""
    preset, batch, mb, n_stages = WORKLOADS[name]
    shape = vitgen.preset(preset)
    counts = stage_counts(shape, n_stages)
    _, blob = vitgen.make_params(shape, seed=0)
    model = vit.VitModel(shape, blob, vit.VIT_BF16, mb * group, device=dev)
    del blob
    pix = torch.from_numpy(vitgen.make_pixels(shape, batch, seed=0)).to(dev)
    logits = torch.empty((batch, shape.num_classes), dtype=torch.float32, device=dev)
    n_streams = max(1, min(4, batch // (mb * group)))
    wss, streams, wsb = model.make_pipeline_buffers(mb * group, n_streams)

    def step():
        model.run_pipeline(counts, mb, pix, logits, wss, streams, wsb, group=group)

    for _ in range(warmup):
        step()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(streams[0])
    for s_ in streams[1:]:
        s_.wait_event(e0)
    for _ in range(steps):
        step()
    for s_ in streams[1:]:
        e = torch.cuda.Event()
        e.record(s_)
        streams[0].wait_event(e)
    e1.record(streams[0])
    torch.cuda.synchronize(dev)
    for s_ in streams:
        model.check(s_)
    ms = e0.elapsed_time(e1) / steps
    total_flops = flops_per_image(shape)[0]
    model.close()
    value = batch / (ms / 1e3)
    return {"workload": f"ViT-{preset}, batch {batch}, microbatch {mb}, {n_stages} stages, {n_streams} streams"
                        + (f", {group} microbatches per launch" if group > 1 else ""),
            "value": value, "unit": "images/s", "ms_per_step": ms, "tflops": value * total_flops / 1e12}


def workload_config(preset, shape, batch, mb, counts, world, n_streams):
    return {
        "workload": f"ViT-{preset} forward, batch {batch}, microbatch {mb}, stages {counts}, "
                    f"{shape.tokens} tokens, {shape.layers} layers, hidden {shape.hidden}",
        "global_batch": world * batch, "streams": n_streams,
        "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
        "l2": "activations and weights per layer exceed L2 (no flush needed)",
    }


def run_reference(args, rank):
    if rank != 0:
        return
    preset, batch, mb, n_stages = WORKLOADS[args.workload]
    shape = vitgen.preset(preset)
    params, _ = vitgen.make_params(shape, seed=0)
    per_step = 1
    times = []
    cores = 1
    for i in range(args.warmup + args.steps):
        ips, cores, dt = oracle_images_per_s(shape, per_step, params=params)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = per_step / (ms / 1e3)
    line = {
        "impl": "reference", "metric": "images/sec", "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(preset, shape, batch, mb, stage_counts(shape, n_stages), 1,
                                  max(1, min(4, batch // mb))) | {"reference_images_per_step": per_step},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": cores, "kind": "oracle",
                         "sample": f"{per_step} image per step of the {preset} workload, numpy fp64"},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_stage_per_gpu(args, vit, torch, dist, dev, rank, world):
    """One pipeline stage per GPU (strong scaling: the batch is fixed, the layers are spread).
    Every rank holds the whole parameter set and runs its own layer range; activations travel
    rank to rank by NCCL send/receive into the receiver's own buffers."""
    from paper_2110_14895_b200 import pipeline as PL
    preset, batch, mb, _ = WORKLOADS[args.workload]
    mb = min(mb, 32)
    shape = vitgen.preset(preset)
    if world > shape.layers:
        raise SystemExit("more GPUs than layers")
    _, layers = PL.plan_stages([1.0] * shape.layers, world, act_bytes=1.0, link_bytes_per_s=1e30)
    if len(layers) != world:
        raise SystemExit("the partitioner used fewer stages than GPUs")
    lb, le = PL.stage_ranges(layers)[rank]
    _, blob = vitgen.make_params(shape, seed=0)
    model = vit.VitModel(shape, blob, vit.VIT_BF16, mb, device=dev)
    del blob
    pipe = PL.StagePipeline(PL.VitStageExecutor(model, lb, le, rank == 0, rank == world - 1), dist, mb)
    pix = torch.from_numpy(vitgen.make_pixels(shape, batch, seed=0)).to(dev) if rank == 0 else None
    logits = torch.empty((batch, shape.num_classes), dtype=torch.float32, device=dev) if rank == world - 1 else None
    for _ in range(args.warmup):
        pipe.run(batch, mb, pixels=pix, logits=logits)
    torch.cuda.synchronize(dev)
    dist.barrier()
    torch.cuda.synchronize(dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        pipe.run(batch, mb, pixels=pix, logits=logits)
    e1.record()
    torch.cuda.synchronize(dev)
    dist.barrier()
    ms = max_over_ranks(e0.elapsed_time(e1), dist, dev) / args.steps
    model.check()
    if rank == 0:
        total_flops = flops_per_image(shape)[0]
        value = batch / (ms / 1e3)
        print(json.dumps({
            "metric": "images/sec", "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"ViT-{preset} forward, batch {batch}, microbatch {mb}, one stage per GPU, "
                                   f"layers per stage {layers}", "global_batch": batch,
                       "parallelism": f"pipeline pp{world}", "l2": "activations and weights per layer exceed L2"},
            "tflops": value * total_flops / 1e12}), flush=True)
    model.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default="huge14", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra-workloads", action="store_true",
                    help="skip the brief ViT-L/16 and ViT-B/16 measurements reported under 'workloads'")
    ap.add_argument("--streams", type=int, default=0, help="streams for the stage runner (0 = min(4, microbatches))")
    ap.add_argument("--mode", default="replicas", choices=["replicas", "pipeline"],
                    help="N > 1 only: independent replicas (default), or one pipeline stage per GPU with "
                         "point-to-point hand-off of the activations (the paper's runtime)")
    ap.add_argument("--e2e-microbatch", type=int, default=64,
                    help="microbatch of the host-buffer (end to end) leg: copies of one microbatch overlap the compute of others")
    ap.add_argument("--sweep", action="store_true",
                    help="run the microbatch sweep (sizes 1..256, 4 stages, streams; key 'sweep') also for workloads other than the default")
    ap.add_argument("--no-sweep", action="store_true", help="skip the microbatch sweep of the default run")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist
    import paper_2110_14895_b200 as vit

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    if args.mode == "pipeline" and world > 1:
        run_stage_per_gpu(args, vit, torch, dist, dev, rank, world)
        dist.destroy_process_group()
        return

    preset, batch, mb, n_stages = WORKLOADS[args.workload]
    shape = vitgen.preset(preset)
    counts = stage_counts(shape, n_stages)
    _, blob = vitgen.make_params(shape, seed=0)
    model = vit.VitModel(shape, blob, vit.VIT_BF16, mb, device=dev)
    pix_host = torch.from_numpy(vitgen.make_pixels(shape, batch, seed=rank_pixel_seed(rank))).pin_memory()
    pix = pix_host.to(dev)
    logits = torch.empty((batch, shape.num_classes), dtype=torch.float32, device=dev)
    n_streams = args.streams if args.streams > 0 else max(1, min(4, batch // mb))   # microbatches round-robin on streams
    wss, streams, wsb = model.make_pipeline_buffers(mb, n_streams)

    def step():
        model.run_pipeline(counts, mb, pix, logits, wss, streams, wsb)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(fn, steps, stream_list):
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream_list[0])
        for s in stream_list[1:]:
            s.wait_event(ev0)
        for _ in range(steps):
            fn()
        for s in stream_list[1:]:
            e = torch.cuda.Event()
            e.record(s)
            stream_list[0].wait_event(e)
        ev1.record(stream_list[0])
        barrier()
        return max_over_ranks(ev0.elapsed_time(ev1), dist if world > 1 else None, dev)

    for _ in range(args.warmup):
        step()
    for s_ in streams:
        model.check(s_)

    launches0 = model.launches
    with ClockSampler(local) as clk:
        ms_total = timed(step, args.steps, streams)
    launches = model.launches - launches0
    model.check(streams[0])
    ms_step = ms_total / args.steps
    value = aggregate_images_per_s(world, batch, ms_step)

    # per-kernel timing over the same steps (event pairs around every launch, same stream)
    vit.vit_profile_enable(model.h, True)
    prof_steps = min(args.steps, 5)
    # one stream for this pass, so that the event pairs of different microbatches do not overlap
    timed(lambda: model.run_pipeline(counts, mb, pix, logits, wss[:1], streams[:1], wsb), prof_steps, streams[:1])
    prof = vit.vit_profile_collect(model.h)
    vit.vit_profile_enable(model.h, False)

    # end to end: host pixels in, host logits out, through the host-buffer entry point
    e2e_mb = min(mb, args.e2e_microbatch)
    e2e_streams_n = min(4, max(1, batch // e2e_mb))
    e_wss, e_streams, e_wsb = model.make_pipeline_buffers(e2e_mb, e2e_streams_n)
    logits_host = torch.empty((batch, shape.num_classes), dtype=torch.float32).pin_memory()

    def step_host():
        model.run_pipeline(counts, e2e_mb, pix_host, logits_host, e_wss, e_streams, e_wsb, host=True)

    for _ in range(2):
        step_host()
    e2e_steps = max(3, min(args.steps, 10))
    ms_e2e = timed(step_host, e2e_steps, e_streams) / e2e_steps
    for s in e_streams:
        model.check(s)
    e2e_value = aggregate_images_per_s(world, batch, ms_e2e)

    # microbatch sweep (ViT-H/14 by default): a handle of its own with room for microbatches of 256,
    # after the headline measurements so that they are not affected
    sweep = None
    if world == 1 and not args.no_sweep and (args.sweep or args.workload == "huge14"):
        sweep_model = vit.VitModel(shape, blob, vit.VIT_BF16, 256, device=dev)
        sweep = microbatch_sweep(vit, sweep_model, shape, dev, torch)
        sweep_model.close()
    del blob

    # the other single-GPU configurations of the metric, briefly (rank 0 of a single-GPU run only)
    extra = {}
    if world == 1 and not args.no_extra_workloads and args.workload == "huge14":
        extra["large16"] = measure_workload(vit, torch, dev, "large16")
        extra["large16_grouped"] = measure_workload(vit, torch, dev, "large16", group=4)
        extra["base16"] = measure_workload(vit, torch, dev, "base16")

    if rank == 0:
        pk = peaks()
        total_flops, gemm, attn, embed = flops_per_image(shape)
        gemm_ms = sum(prof[k][0] for k in ("qkv", "outproj", "fc1", "fc2"))
        gemm_launches = sum(prof[k][1] for k in ("qkv", "outproj", "fc1", "fc2"))
        gemm_flops = sum(gemm.values()) * shape.layers * batch * prof_steps
        gemm_all = gemm_flops / (gemm_ms / 1e3) / 1e12 if gemm_ms > 0 else None
        # the dominant kernel: the fc1 GEMM (bias + GELU epilogue), the largest single share of the step
        top_ms, top_n = prof["fc1"]
        achieved = gemm["fc1"] * shape.layers * batch * prof_steps / (top_ms / 1e3) / 1e12 if top_ms > 0 else None
        peak = pk["bf16_tflops_sustained"]
        per_class = {}
        M = batch * shape.tokens
        for k, (ms, n) in prof.items():
            if n == 0:
                continue
            per_class[k] = {"ms_per_step": ms / prof_steps, "launches_per_step": n // prof_steps}
            if k in gemm:
                per_class[k]["tflops"] = gemm[k] * shape.layers * batch * prof_steps / (ms / 1e3) / 1e12
            if k == "attention":
                per_class[k]["tflops"] = attn * shape.layers * batch * prof_steps / (ms / 1e3) / 1e12
            if k == "layernorm":
                # the LayerNorm statistics kernel (the normalisation itself is applied in the QKV and
                # fc1 epilogues): reads every row once, writes 8 bytes per row
                per_class[k]["gbs"] = 2 * shape.layers * prof_steps * (M * shape.hidden * 2 + M * 8) / (ms / 1e3) / 1e9
                per_class[k]["what"] = "row statistics; normalisation folded into the QKV and fc1 GEMMs"
        line = {
            "metric": "images/sec", "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": workload_config(preset, shape, batch, mb, counts, world, n_streams),
            "tflops": value * total_flops / 1e12,
            "frac_of_bf16_peak": {"burst": value * total_flops / 1e12 / world / pk["bf16_tflops"],
                                  "sustained": value * total_flops / 1e12 / world / pk["bf16_tflops_sustained"],
                                  "nominal": value * total_flops / 1e12 / world / NOMINAL_BF16_TFLOPS,
                                  "peaks": pk["source"], "burst_tflops": pk["bf16_tflops"],
                                  "sustained_tflops": pk["bf16_tflops_sustained"], "nominal_tflops": NOMINAL_BF16_TFLOPS},
            "e2e": {"value": e2e_value, "unit": "images/s",
                    "h2d_bytes_per_step": int(pix_host.numel() * 4), "d2h_bytes_per_step": int(logits_host.numel() * 4),
                    "microbatch": e2e_mb, "streams": e2e_streams_n},
            "gpu_launches": int(launches),
            "clocks": clk.summary(),
            "roofline": {
                "kernel": "linear_tc_kernel<256, GELU> (fc1 GEMM)", "bound": "tensor",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None,
                "peak_kind": f"{pk['source']} sustained bf16 (kernel timed inside a long step)",
                "frac_of_burst": achieved / pk["bf16_tflops"] if achieved else None,
                "launches": top_n, "traffic": NCU_TRAFFIC.get(args.workload),
                "all_gemms": {"achieved": gemm_all, "frac": gemm_all / peak if gemm_all else None,
                              "frac_of_burst": gemm_all / pk["bf16_tflops"] if gemm_all else None,
                              "frac_of_nominal": gemm_all / NOMINAL_BF16_TFLOPS if gemm_all else None,
                              "launches": gemm_launches},
            },
            "kernels": per_class,
        }
        if extra:
            for w in extra.values():
                w["frac_of_bf16_peak"] = {"burst": w["tflops"] / pk["bf16_tflops"],
                                          "sustained": w["tflops"] / pk["bf16_tflops_sustained"],
                                          "nominal": w["tflops"] / NOMINAL_BF16_TFLOPS}
            line["workloads"] = extra
        if sweep is not None:
            line["sweep"] = sweep
        if not args.no_cpu_baseline and world == 1:
            n_img = 6 if preset == "huge14" else 16      # about 10-15 s of host work
            ips, cores, dt = oracle_images_per_s(shape, n_img)
            line["cpu_baseline"] = {"value": ips, "unit": "images/s", "cores": cores, "kind": "oracle",
                                    "sample": f"{n_img} images of the same workload, numpy fp64, {dt:.1f} s"}
        print(json.dumps(line), flush=True)
    model.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
