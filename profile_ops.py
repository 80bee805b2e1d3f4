"""Runs one kernel of the library a few times on random device data, for ncu captures and
quick timing:  python profile_ops.py --op linear --M 32896 --N 5120 --K 1280 --epilogue 1
Prints the mean CUDA-event time per launch."""
import argparse

import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import paper_2110_14895_b200 as vit  # noqa: E402


class _Shape:
    image_size, patch_size, channels, hidden, layers, heads, mlp_dim, num_classes, ln_eps = 32, 16, 3, 64, 1, 1, 64, 8, 1e-6


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--op", required=True, choices=["linear", "linear_ln", "attention", "layernorm", "rowstats"])
    ap.add_argument("--M", type=int, default=32896)
    ap.add_argument("--N", type=int, default=1280)
    ap.add_argument("--K", type=int, default=1280)
    ap.add_argument("--epilogue", type=int, default=0)
    ap.add_argument("--images", type=int, default=128)
    ap.add_argument("--T", type=int, default=257)
    ap.add_argument("--heads", type=int, default=16)
    ap.add_argument("--d", type=int, default=80)
    ap.add_argument("--reps", type=int, default=5)
    a = ap.parse_args()
    cfg = vit.make_config(_Shape, vit.VIT_BF16, 1)
    blob = np.zeros(vit.vit_param_count(cfg), dtype=np.float32)
    h = vit.vit_create(cfg, blob)
    bf = torch.bfloat16
    if a.op == "linear":
        x = torch.randn(a.M, a.K, device="cuda").to(bf)
        w = (torch.randn(a.N, a.K, device="cuda") / a.K ** 0.5).to(bf)
        b = torch.randn(a.N, device="cuda")
        out = torch.randn(a.M, a.N, device="cuda").to(bf)
        res = out.data_ptr() if a.epilogue == 2 else 0
        run = lambda: vit.vit_op_linear(h, vit.VIT_BF16, a.M, a.N, a.K, x.data_ptr(), w.data_ptr(), b.data_ptr(),
                                        a.epilogue, res, out.data_ptr())
        work = 2.0 * a.M * a.N * a.K
        unit = "TFLOP/s"
    elif a.op == "linear_ln":
        # the QKV / fc1 product with the LayerNorm folded in (epilogue 0 = plain, 1 = GELU)
        x = torch.randn(a.M, a.K, device="cuda").to(bf)
        w = (torch.randn(a.N, a.K, device="cuda") / a.K ** 0.5).to(bf)
        c1 = w.float().sum(-1).contiguous()
        c0 = torch.randn(a.N, device="cuda")
        stats = torch.empty(a.M, 2, device="cuda")
        out = torch.empty(a.M, a.N, device="cuda", dtype=bf)
        vit.vit_op_rowstats(h, a.M, a.K, x.data_ptr(), 1e-6, stats.data_ptr())
        run = lambda: vit.vit_op_linear_ln(h, a.M, a.N, a.K, x.data_ptr(), stats.data_ptr(), w.data_ptr(), c1.data_ptr(),
                                           c0.data_ptr(), a.epilogue, out.data_ptr())
        work = 2.0 * a.M * a.N * a.K
        unit = "TFLOP/s"
    elif a.op == "rowstats":
        x = torch.randn(a.M, a.N, device="cuda").to(bf)
        stats = torch.empty(a.M, 2, device="cuda")
        run = lambda: vit.vit_op_rowstats(h, a.M, a.N, x.data_ptr(), 1e-6, stats.data_ptr())
        work = (a.M * a.N * 2 + a.M * 8) / 1e-3     # bytes, scaled so the print below reads GB/s
        unit = "GB/s"
    elif a.op == "attention":
        H = a.heads * a.d
        qkv = torch.randn(a.images * a.T, 3 * H, device="cuda").to(bf)
        out = torch.empty(a.images * a.T, H, device="cuda", dtype=bf)
        run = lambda: vit.vit_op_attention(h, vit.VIT_BF16, a.images, a.T, a.heads, a.d, qkv.data_ptr(), out.data_ptr())
        work = 4.0 * a.images * a.T * a.T * H
        unit = "TFLOP/s"
    else:
        x = torch.randn(a.M, a.N, device="cuda").to(bf)
        y = torch.empty_like(x)
        g = torch.ones(a.N, device="cuda")
        b = torch.zeros(a.N, device="cuda")
        run = lambda: vit.vit_op_layernorm(h, vit.VIT_BF16, a.M, a.N, x.data_ptr(), g.data_ptr(), b.data_ptr(), 1e-6, y.data_ptr())
        work = 2.0 * a.M * a.N * 2 / 1e-3   # bytes, scaled so the print below reads GB/s
        unit = "GB/s"
    run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.reps):
        run()
    e1.record()
    torch.cuda.synchronize()
    vit.vit_check_status(h)
    ms = e0.elapsed_time(e1) / a.reps
    print(f"{a.op}: {ms * 1e3:.1f} us per launch, {work / (ms * 1e-3) / 1e12:.1f} {unit}")
    vit.vit_destroy(h)


if __name__ == "__main__":
    main()
