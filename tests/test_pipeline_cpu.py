"""One stage per process with point-to-point hand-off (the paper's runtime, Section 3.1): the
schedule, the double buffering, a ragged last microbatch and the behaviour when a rank has left,
on CPU with gloo ranks.  The stage arithmetic here is the CPU oracle behind the runner's executor
interface; on GPUs the same runner drives the CUDA library (not exercised here)."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import vitgen  # noqa: E402
from oracle import vit_oracle as O  # noqa: E402

CFG = vitgen.ViTConfig(image_size=8, patch_size=4, channels=3, hidden=16, layers=4, heads=2, mlp_dim=32,
                       num_classes=7)


class OracleExecutor:
    """The runner's executor interface on CPU tensors, computed by the oracle (test side only)."""

    def __init__(self, params, cfg, lb, le):
        self.p, self.cfg, self.lb, self.le = params, cfg, lb, le

    def empty_activation(self, mb):
        return torch.full((mb, self.cfg.tokens, self.cfg.hidden), float("nan"), dtype=torch.float64)

    def empty_logits(self, mb):
        return torch.empty((mb, self.cfg.num_classes), dtype=torch.float64)

    def embed(self, pixels, out):
        out.copy_(torch.from_numpy(O.patch_embed(self.p, self.cfg, pixels.numpy())))

    def stage(self, x, out):
        out.copy_(torch.from_numpy(O.run_stage(self.p, self.cfg, self.lb, self.le, x.numpy())))

    def head(self, x, logits):
        logits.copy_(torch.from_numpy(O.head(self.p, self.cfg, x.numpy())))


def _init(rank, world, port, timeout_s=30):
    import datetime
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world, timeout=datetime.timedelta(seconds=timeout_s))


def _pipeline_worker(rank, world, port, stage_layers, batches, microbatch, q):
    from paper_2110_14895_b200 import pipeline as PL
    _init(rank, world, port)
    params, _ = vitgen.make_params(CFG, seed=3, bf16=False, ln_affine=True)
    lb, le = PL.stage_ranges(stage_layers)[rank]
    pipe = PL.StagePipeline(OracleExecutor(params, CFG, lb, le), dist, max_microbatch=microbatch)
    results = []
    for step, batch in enumerate(batches):
        pix = torch.from_numpy(vitgen.make_pixels(CFG, batch, seed=10 + step).astype(np.float64)) if rank == 0 else None
        logits = torch.full((batch, CFG.num_classes), float("nan"), dtype=torch.float64) if rank == world - 1 else None
        pipe.run(batch, microbatch, pixels=pix, logits=logits)
        results.append(None if logits is None else logits.numpy())
    q.put((rank, results, list(pipe.log)))
    dist.barrier()
    dist.destroy_process_group()


def _spawn(target, world, args):
    port = 29500 + (os.getpid() * 7 + np.random.randint(0, 1000)) % 3000
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=target, args=(r, world, port) + args + (q,)) for r in range(world)]
    for p in procs:
        p.start()
    return procs, q


@pytest.mark.parametrize("stage_layers", [[1, 3], [2, 1, 1]])
def test_stage_per_rank_pipeline_matches_single_process_forward(stage_layers):
    world, microbatch, batches = len(stage_layers), 2, [5, 4]     # 5 = 2 + 2 + 1: ragged last microbatch
    procs, q = _spawn(_pipeline_worker, world, (stage_layers, batches, microbatch))
    res = {r: (out, log) for r, out, log in (q.get(timeout=180) for _ in range(world))}
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    params, _ = vitgen.make_params(CFG, seed=3, bf16=False, ln_affine=True)
    for step, batch in enumerate(batches):
        want = O.forward(params, CFG, vitgen.make_pixels(CFG, batch, seed=10 + step).astype(np.float64))
        got = res[world - 1][0][step]
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)   # same arithmetic, same order: no rounding at a boundary
    # schedule of a middle / last rank in the first batch (three microbatches): the receive of
    # microbatch m + 1 is posted before the stage of microbatch m runs, alternating buffers
    log = res[1][1]
    first_batch = log[:log.index(("irecv", 0), 1)] if ("irecv", 0) in log[1:] else log
    order = [e for e in first_batch if e[0] in ("irecv", "stage")]
    assert order[:6] == [("irecv", 0), ("irecv", 1), ("stage", 0), ("irecv", 2), ("stage", 1), ("stage", 2)]
    sends = [e for e in res[0][1] if e[0] == "isend"]
    assert sends[:3] == [("isend", 0), ("isend", 1), ("isend", 2)]


def _leaver_worker(rank, world, port, leaver, q):
    from paper_2110_14895_b200 import pipeline as PL
    _init(rank, world, port, timeout_s=5)
    params, _ = vitgen.make_params(CFG, seed=3, bf16=False)
    lb, le = PL.stage_ranges([2, 2])[rank]
    pipe = PL.StagePipeline(OracleExecutor(params, CFG, lb, le), dist, max_microbatch=2, roll_call_timeout_s=2.0)
    pix = torch.from_numpy(vitgen.make_pixels(CFG, 2, seed=1).astype(np.float64))
    logits = torch.empty((2, CFG.num_classes), dtype=torch.float64)
    pipe.run(2, 2, pixels=pix, logits=logits)                 # step 0: everybody is there
    dist.barrier()
    if rank == leaver:                                        # leaves between steps, nothing in flight
        q.put((rank, "left"))
        return
    try:
        pipe.run(2, 2, pixels=pix, logits=logits)             # step 1: the neighbour is gone
        q.put((rank, "no error"))
    except PL.PipelineError as e:
        q.put((rank, f"error: {e}"))


def test_a_rank_that_left_between_steps_is_reported_not_waited_for():
    import time
    t0 = time.time()
    procs, q = _spawn(_leaver_worker, 2, (1,))
    res = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
    assert res[1] == "left"
    assert res[0].startswith("error:") and "did not join step 1" in res[0], res[0]
    assert time.time() - t0 < 90


def test_microbatch_sizes_stage_ranges_and_plan():
    from paper_2110_14895_b200 import pipeline as PL
    import paper_2110_14895_b200 as vit
    from paper_2110_14895_b200 import build as b
    b.build()
    vit.lib()
    assert PL.microbatch_sizes(5, 2) == [2, 2, 1] and PL.microbatch_sizes(8, 8) == [8] and PL.microbatch_sizes(3, 8) == [3]
    assert PL.stage_ranges([2, 1, 3]) == [(0, 2), (2, 3), (3, 6)]
    with pytest.raises(ValueError):
        PL.stage_ranges([2, 0])
    # equal layers, four devices, fast links: the most even split; a slow link keeps everything on one device
    t, stages = PL.plan_stages([1e-3] * 12, 4, act_bytes=1e6)
    assert stages == [3, 3, 3, 3] and t == pytest.approx(3e-3)
    t, stages = PL.plan_stages([1e-3] * 12, 4, act_bytes=1e6, link_bytes_per_s=1e3)
    assert stages == [12] and t == pytest.approx(12e-3)
