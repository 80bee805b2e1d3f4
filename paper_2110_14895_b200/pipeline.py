"""One pipeline stage per device, point-to-point hand-off of the stage output to the next stage.

This is the runtime of the paper (Section 3.1, Fig. 2): the model is split into parts T_1 ... T_k
of consecutive layers, part i runs on the i-th device, a device works on one microbatch at a time
and sends its intermediate output only to the device of the next stage; the last stage produces
the result.  Section 3.3 (Eq. 2) assumes that sending overlaps computing; here every boundary
has two buffers per direction, so the transfer of microbatch m is in flight while microbatch
m + 1 is computed.

One process per device, `torch.distributed` for the transport (NCCL between GPUs: the activation
[microbatch, T, H] lands in the receiving GPU's own memory before any kernel reads it; gloo for
the CPU tests of the schedule).  The arithmetic of a stage is an *executor* object:
`VitStageExecutor` runs the CUDA library (vit_patch_embed / vit_run_stage / vit_head); there is
no CPU stand-in in this package.

A rank that is gone is noticed on the host, before anything is launched: every step starts with a
roll call through the process group's key-value store with a time limit, and the point-to-point
operations carry the process group's own timeout.
"""
import time
from dataclasses import dataclass

import numpy as np


class PipelineError(RuntimeError):
    pass


def microbatch_sizes(batch: int, microbatch: int):
    """Equal microbatches, the last one possibly smaller (Section 2.1: the minibatch is split
    into microbatches that flow through the stages one after the other)."""
    if batch < 1 or microbatch < 1:
        raise ValueError("batch and microbatch must be positive")
    full, rest = divmod(batch, microbatch)
    return [microbatch] * full + ([rest] if rest else [])


def stage_ranges(stage_layers):
    """[(begin, end)] of the stages from their layer counts."""
    out, lb = [], 0
    for n in stage_layers:
        if n < 1:
            raise ValueError("every stage needs at least one layer")
        out.append((lb, lb + n))
        lb += n
    return out


def plan_stages(layer_time, world, act_bytes, link_bytes_per_s=770e9, layer_mem=None, device_mem=None):
    """Layer counts per rank from the library's partitioner (Section 3.3) for `world` identical
    devices joined by links of `link_bytes_per_s`: layer_time [L] seconds per layer on one device,
    act_bytes the size of one microbatch of activations.  Returns (T_opt, [layers of rank 0, ...]);
    fewer stages than ranks are possible when sending costs more than it saves."""
    from . import binding
    lt = np.asarray(layer_time, dtype=np.float64)
    L = lt.shape[0]
    t_opt, stages = binding.vit_partition_categories(
        lt[None, :], np.full(L, float(act_bytes)), np.ones(L) if layer_mem is None else layer_mem,
        np.array([float(L) if device_mem is None else device_mem]), np.array([[float(link_bytes_per_s)]]),
        [int(world)])
    return t_opt, [n for n, _ in stages]


class VitStageExecutor:
    """Runs a rank's share of the model on its GPU through the CUDA library."""

    def __init__(self, model, layer_begin, layer_end, first, last):
        import torch
        self.torch, self.model = torch, model
        self.lb, self.le, self.first, self.last = layer_begin, layer_end, first, last
        self.hidden, self.tokens, self.classes = model.shape.hidden, model.T, model.shape.num_classes
        self.act_dtype, self.device = model.act_dtype, model.device

    def empty_activation(self, mb):
        return self.torch.empty((mb, self.tokens, self.hidden), dtype=self.act_dtype, device=self.device)

    def empty_logits(self, mb):
        return self.torch.empty((mb, self.classes), dtype=self.torch.float32, device=self.device)

    def embed(self, pixels, out):
        mb = pixels.shape[0]
        ws = self.model.workspace(mb)
        from . import binding as B
        B.vit_patch_embed(self.model.h, mb, pixels.data_ptr(), out.data_ptr(), ws.data_ptr(), ws.numel(),
                          self.model._stream(None))

    def stage(self, x, out):
        self.model.run_stage(self.lb, self.le, x, out=out)

    def head(self, x, logits):
        mb = x.shape[0]
        ws = self.model.workspace(mb)
        from . import binding as B
        B.vit_head(self.model.h, mb, x.data_ptr(), logits.data_ptr(), ws.data_ptr(), ws.numel(),
                   self.model._stream(None))


@dataclass
class _Slot:
    buf: object = None      # tensor
    work: object = None     # outstanding send or receive on it


class StagePipeline:
    """Rank r of `world` runs stage r.  Rank 0 embeds the images, the last rank classifies.

    `executor` provides empty_activation(mb), empty_logits(mb), embed(pixels, out), stage(x, out),
    head(x, logits).  `dist` is torch.distributed with an initialised default group.
    """

    def __init__(self, executor, dist, max_microbatch, roll_call_timeout_s=10.0):
        self.ex, self.dist = executor, dist
        self.rank, self.world = dist.get_rank(), dist.get_world_size()
        self.first, self.last = self.rank == 0, self.rank == self.world - 1
        self.max_mb = max_microbatch
        self.timeout = roll_call_timeout_s
        self.step = 0
        # two buffers towards each neighbour: a transfer is in flight on one while the other is in use
        self.recv = [_Slot(executor.empty_activation(max_microbatch)) for _ in range(2)] if not self.first else []
        self.send = [_Slot(executor.empty_activation(max_microbatch)) for _ in range(2)] if not self.last else []
        self.local = executor.empty_activation(max_microbatch) if self.last else None
        self.log = []           # (event, microbatch) in issue order, for inspection and tests

    # ---- failure detection on the host ---------------------------------------------------------
    def roll_call(self):
        """Every rank announces the step it is about to run and waits, with a time limit, until all
        others have done the same.  A rank that has left never answers, and the others raise
        instead of queueing work that would wait for it."""
        store = self.dist.distributed_c10d._get_default_store()
        store.set(f"pipeline/step{self.step}/rank{self.rank}", "1")
        deadline = time.monotonic() + self.timeout
        for r in range(self.world):
            key = f"pipeline/step{self.step}/rank{r}"
            while True:
                try:
                    if store.check([key]):
                        break
                except Exception as e:          # the store itself is gone (rank 0 hosts it)
                    raise PipelineError(f"rank {self.rank}: store unreachable at step {self.step}: {e}") from e
                if time.monotonic() > deadline:
                    raise PipelineError(f"rank {self.rank}: rank {r} did not join step {self.step} "
                                        f"within {self.timeout:g} s")
                time.sleep(0.01)

    def _wait(self, slot, what):
        if slot.work is not None:
            try:
                slot.work.wait()
            except Exception as e:
                raise PipelineError(f"rank {self.rank}: {what} failed: {e}") from e
            slot.work = None

    # ---- one batch -------------------------------------------------------------------------------
    def run(self, batch, microbatch, pixels=None, logits=None):
        """Pushes `batch` images through the pipeline in microbatches.  `pixels` [batch, C, S, S] is
        needed on rank 0, `logits` [batch, classes] is filled on the last rank.  Returns when this
        rank's share is issued and its transfers have completed."""
        if microbatch > self.max_mb:
            raise ValueError("microbatch above max_microbatch")
        if self.first and pixels is None:
            raise ValueError("rank 0 needs the pixels")
        if self.last and logits is None:
            raise ValueError("the last rank needs a logits buffer")
        self.roll_call()
        sizes = microbatch_sizes(batch, microbatch)
        dist, ex = self.dist, self.ex
        if not self.first:                                   # the first activation can already travel
            self.recv[0].work = dist.irecv(self.recv[0].buf[:sizes[0]], src=self.rank - 1)
            self.log.append(("irecv", 0))
        first_image = 0
        for m, n in enumerate(sizes):
            if self.first:
                x_in = None
            else:
                slot = self.recv[m % 2]
                self._wait(slot, f"receive of microbatch {m}")
                self.log.append(("recv_done", m))
                x_in = slot.buf[:n]
                if m + 1 < len(sizes):
                    # the other buffer was read by the stage of microbatch m - 1, which has been
                    # issued before this call: stream order (GPU) or program order (CPU) keeps them apart
                    nxt = self.recv[(m + 1) % 2]
                    nxt.work = dist.irecv(nxt.buf[:sizes[m + 1]], src=self.rank - 1)
                    self.log.append(("irecv", m + 1))
            if self.last:
                out = self.local[:n]
            else:
                oslot = self.send[m % 2]
                self._wait(oslot, f"send of microbatch {m - 2}")   # the buffer's previous transfer
                out = oslot.buf[:n]
            if self.first:
                ex.embed(pixels[first_image:first_image + n], out)
                ex.stage(out, out)
            else:
                ex.stage(x_in, out)
            self.log.append(("stage", m))
            if self.last:
                ex.head(out, logits[first_image:first_image + n])
                self.log.append(("head", m))
            else:
                oslot.work = dist.isend(out, dst=self.rank + 1)
                self.log.append(("isend", m))
            first_image += n
        for slot in self.send:
            self._wait(slot, "send")
        self.step += 1
