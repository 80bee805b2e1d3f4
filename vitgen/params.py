"""Parameter inventory, seeded generation and the flat fp32 blob layout.

Blob layout (fp32, tensors back to back in this order, matrices [out, in] row-major):

    patch.W [H, C*P*P]   column index = c*P*P + i*P + j  (channel, row, column inside the patch)
    patch.b [H]    cls [H]    (dist [H] when the model has a distillation token)    pos [T, H]
    for each layer l:  l{l}.ln1.g [H]  l{l}.ln1.b [H]
                       l{l}.Wqkv [3H, H]  l{l}.bqkv [3H]     rows [0,H) Q, [H,2H) K, [2H,3H) V; head h owns rows h*d..(h+1)*d of each
                       l{l}.Wo [H, H]     l{l}.bo [H]
                       l{l}.ln2.g [H]     l{l}.ln2.b [H]
                       l{l}.W1 [F, H]     l{l}.b1 [F]
                       l{l}.W2 [H, F]     l{l}.b2 [H]
    lnf.g [H]  lnf.b [H]  head.W [classes, H]  head.b [classes]
    (head_dist.W [classes, H]  head_dist.b [classes] when the model has a distillation token)
"""
from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np

from .config import ViTConfig

_CHUNK = 1 << 20   # elements per independently keyed generator chunk
_STD = 0.02


def param_specs(cfg: ViTConfig):
    """List of (name, shape, kind) in blob order; kind is 'normal', 'gain' or 'shift'."""
    H, F, T, C = cfg.hidden, cfg.mlp_dim, cfg.tokens, cfg.num_classes
    specs = [
        ("patch.W", (H, cfg.patch_k), "normal"),
        ("patch.b", (H,), "normal"),
        ("cls", (H,), "normal"),
    ]
    if cfg.extra_tokens:
        specs.append(("dist", (H,), "normal"))
    specs.append(("pos", (T, H), "normal"))
    for l in range(cfg.layers):
        p = f"l{l}."
        specs += [
            (p + "ln1.g", (H,), "gain"), (p + "ln1.b", (H,), "shift"),
            (p + "Wqkv", (3 * H, H), "normal"), (p + "bqkv", (3 * H,), "normal"),
            (p + "Wo", (H, H), "normal"), (p + "bo", (H,), "normal"),
            (p + "ln2.g", (H,), "gain"), (p + "ln2.b", (H,), "shift"),
            (p + "W1", (F, H), "normal"), (p + "b1", (F,), "normal"),
            (p + "W2", (H, F), "normal"), (p + "b2", (H,), "normal"),
        ]
    specs += [
        ("lnf.g", (H,), "gain"), ("lnf.b", (H,), "shift"),
        ("head.W", (C, H), "normal"), ("head.b", (C,), "normal"),
    ]
    if cfg.extra_tokens:
        specs += [("head_dist.W", (C, H), "normal"), ("head_dist.b", (C,), "normal")]
    return specs


def param_count(cfg: ViTConfig) -> int:
    return sum(int(np.prod(s)) for _, s, _ in param_specs(cfg))


def round_to_bf16_inplace(a: np.ndarray) -> None:
    """Round fp32 values to the nearest bf16-representable value, ties to even, in place."""
    u = a.reshape(-1).view(np.uint32)
    for s in range(0, u.size, _CHUNK):
        v = u[s:s + _CHUNK]
        t = (v >> np.uint32(16)) & np.uint32(1)
        t += np.uint32(0x7FFF)
        v += t
        v &= np.uint32(0xFFFF0000)


def _fill_normal(out: np.ndarray, seed: int, stream: int, chunk: int, mean: float, bf16: bool):
    g = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ stream, chunk]))
    g.standard_normal(out.size, dtype=np.float32, out=out)
    out *= np.float32(_STD)
    if mean != 0.0:
        out += np.float32(mean)
    if bf16:
        round_to_bf16_inplace(out)


def make_params(cfg: ViTConfig, seed: int = 0, bf16: bool = True, ln_affine: bool = False,
                blob: np.ndarray | None = None):
    """Draw every parameter.  Returns (dict name -> fp32 array view, flat fp32 blob).

    The dict entries are views into the blob, so the two always hold the same bits.
    """
    specs = param_specs(cfg)
    total = sum(int(np.prod(s)) for _, s, _ in specs)
    if blob is None:
        blob = np.empty(total, dtype=np.float32)
    assert blob.size == total and blob.dtype == np.float32
    views, jobs, off = {}, [], 0
    for tid, (name, shape, kind) in enumerate(specs):
        n = int(np.prod(shape))
        flat = blob[off:off + n]
        views[name] = flat.reshape(shape)
        off += n
        if kind == "normal" or ln_affine:
            mean = 1.0 if kind == "gain" else 0.0
            for c, s in enumerate(range(0, n, _CHUNK)):
                jobs.append((flat[s:s + _CHUNK], seed, tid, c, mean, bf16))
        else:
            flat[:] = 1.0 if kind == "gain" else 0.0
    with ThreadPoolExecutor(max_workers=min(32, os.cpu_count() or 1)) as ex:
        list(ex.map(lambda j: _fill_normal(*j), jobs))
    return views, blob


def pack_blob(cfg: ViTConfig, params: dict) -> np.ndarray:
    """Concatenate named tensors into the flat layout (for hand-built test parameters)."""
    parts = []
    for name, shape, _ in param_specs(cfg):
        a = np.asarray(params[name], dtype=np.float32)
        assert a.shape == tuple(shape), (name, a.shape, shape)
        parts.append(a.reshape(-1))
    return np.ascontiguousarray(np.concatenate(parts))


def unpack_blob(cfg: ViTConfig, blob: np.ndarray) -> dict:
    views, off = {}, 0
    for name, shape, _ in param_specs(cfg):
        n = int(np.prod(shape))
        views[name] = blob[off:off + n].reshape(shape)
        off += n
    assert off == blob.size
    return views
