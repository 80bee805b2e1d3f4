"""Writes tests/golden/vitgen_checksums.txt: SHA-256 of the seeded parameter blob and pixels.

Calls only the input generator (no oracle, no CUDA).  Re-run after a deliberate change of
the recipe:  python tests/golden/make_golden.py
"""
import hashlib
import os
import sys

HERE = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, os.path.dirname(os.path.dirname(HERE)))
import vitgen  # noqa: E402


def digests():
    out = {}
    cfg = vitgen.preset("tiny16")
    for tag, kw in (("tiny16_seed0_fp32", dict(bf16=False)), ("tiny16_seed0_bf16", dict(bf16=True)),
                    ("tiny16_seed0_bf16_affine", dict(bf16=True, ln_affine=True))):
        _, blob = vitgen.make_params(cfg, seed=0, **kw)
        out[tag] = hashlib.sha256(blob.tobytes()).hexdigest()
    out["tiny16_pixels_seed0_b2"] = hashlib.sha256(vitgen.make_pixels(cfg, 2, seed=0).tobytes()).hexdigest()
    out["partition_16_24_seed0"] = ",".join(f"{a}-{b}" for a, b in vitgen.uneven_partition(16, 24, 0))
    return out


if __name__ == "__main__":
    with open(os.path.join(HERE, "vitgen_checksums.txt"), "w") as f:
        f.write("# input-generator checksums (numpy Philox streams); written by make_golden.py\n")
        for k, v in digests().items():
            f.write(f"{k} {v}\n")
