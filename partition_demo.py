"""Per-layer stage times measured on this GPU (the analogue of the paper's per-layer timing
figure) fed to the pipeline partitioner:  python partition_demo.py
The devices are this GPU at the given relative speeds; links carry `--gbs` GB/s."""
import argparse
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import vitgen  # noqa: E402
import paper_2110_14895_b200 as vit  # noqa: E402


def measure_layer_times(model, shape, mb, reps=5):
    x = torch.randn((mb, model.T, shape.hidden), device="cuda").to(torch.bfloat16)
    out = torch.empty_like(x)
    times = []
    for l in range(shape.layers):
        model.run_stage(l, l + 1, x, out=out)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            model.run_stage(l, l + 1, x, out=out)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1) / reps * 1e-3)
    model.check()
    return np.array(times)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--model", default="base16", choices=sorted(vitgen.PRESETS))
    ap.add_argument("--microbatch", type=int, default=16)
    ap.add_argument("--speeds", default="1,1,0.5,0.25", help="relative speed of each device")
    ap.add_argument("--gbs", type=float, default=770.0, help="link bandwidth, GB/s")
    ap.add_argument("--mem-layers", type=float, default=1e9, help="layers a device can hold")
    a = ap.parse_args()
    shape = vitgen.preset(a.model)
    _, blob = vitgen.make_params(shape, seed=0)
    model = vit.VitModel(shape, blob, vit.VIT_BF16, a.microbatch)
    t = measure_layer_times(model, shape, a.microbatch)
    print("per-layer time on this GPU (us):", " ".join(f"{v * 1e6:.1f}" for v in t))
    speeds = np.array([float(s) for s in a.speeds.split(",")])
    D, L = len(speeds), shape.layers
    act_bytes = a.microbatch * model.T * shape.hidden * 2.0
    t_opt, stages = vit.vit_partition(t[None, :] / speeds[:, None], np.full(L, act_bytes), np.ones(L),
                                      np.full(D, a.mem_layers), np.full((D, D), a.gbs * 1e9))
    print(f"T_opt = {t_opt * 1e6:.1f} us per microbatch -> {a.microbatch / t_opt:.0f} images/s pipelined")
    for n, u in stages:
        print(f"  {n:2d} layers on device {u} (speed {speeds[u]:g})")
    model.close()


if __name__ == "__main__":
    main()
