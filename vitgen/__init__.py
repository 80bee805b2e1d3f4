"""Seeded synthetic inputs for a pre-LN Vision Transformer: configuration presets,
parameters, pixels and stage partitions.

This package only produces data.  It holds none of the model's arithmetic (no
LayerNorm, GEMM, attention, GELU), so both the CPU oracle and the CUDA library
can be fed from it without sharing any computation.

Recipe (stands in for pretrained weights and dataset images, which the paper's
experimental setup uses but which carry no information the forward pass needs):
  * every weight, bias, the class token and the position table: N(0, 0.02^2);
  * LayerNorm gain 1 / shift 0 (or, for tests of the affine path, 1+N(0,0.02^2)
    and N(0,0.02^2));
  * pixels: uniform [-1, 1) fp32, NCHW;
  * optional rounding of every parameter to the nearest bf16 value (ties to
    even), still stored as fp32, so that weight quantisation is common to every
    consumer.
Numbers come from numpy's Philox counter-based bit generator keyed by
(seed, stream id, chunk index); the streams are frozen by checksums kept with
the tests.
"""
from .config import ViTConfig, PRESETS, preset
from .params import (param_specs, param_count, make_params, pack_blob, unpack_blob,
                     round_to_bf16_inplace)
from .inputs import make_pixels, uneven_partition, equal_partition

__all__ = [
    "ViTConfig", "PRESETS", "preset", "param_specs", "param_count", "make_params",
    "pack_blob", "unpack_blob", "round_to_bf16_inplace", "make_pixels",
    "uneven_partition", "equal_partition",
]
