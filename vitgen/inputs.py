"""Seeded pixels and stage partitions."""
import numpy as np

from .config import ViTConfig

_PIXEL_STREAM = 0xF00D


def make_pixels(cfg: ViTConfig, batch: int, seed: int = 0, first: int = 0) -> np.ndarray:
    """fp32 [batch, C, S, S], uniform in [-1, 1).  Image index `first + b` has its own key, so
    an image is the same bits whatever batch it is generated in."""
    out = np.empty((batch, cfg.channels, cfg.image_size, cfg.image_size), dtype=np.float32)
    for b in range(batch):
        g = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ _PIXEL_STREAM, first + b]))
        flat = out[b].reshape(-1)
        g.random(flat.size, dtype=np.float32, out=flat)
        flat *= np.float32(2.0)
        flat -= np.float32(1.0)
    return out


def equal_partition(n_stages: int, layers: int):
    """Stage boundaries [(begin, end)] for an even split (layers % n_stages == 0)."""
    assert layers % n_stages == 0
    k = layers // n_stages
    return [(i * k, (i + 1) * k) for i in range(n_stages)]


def uneven_partition(n_stages: int, layers: int, seed: int = 0):
    """Seeded uneven split: every stage gets one layer, the remaining layers are dealt out at
    random.  Returns [(begin, end)] with the counts summing to `layers`."""
    assert 1 <= n_stages <= layers
    counts = np.ones(n_stages, dtype=np.int64)
    g = np.random.Generator(np.random.Philox(key=[(seed << 20) ^ 0x57A6E, n_stages]))
    for s in g.integers(0, n_stages, size=layers - n_stages):
        counts[s] += 1
    bounds, b = [], 0
    for c in counts:
        bounds.append((b, b + int(c)))
        b += int(c)
    return bounds
