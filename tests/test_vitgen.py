"""The seeded input generator: frozen streams, layout, bf16 rounding, partitions."""
import importlib.util
import os

import numpy as np

import vitgen

HERE = os.path.dirname(os.path.abspath(__file__))


def test_streams_match_committed_checksums():
    spec = importlib.util.spec_from_file_location("make_golden", os.path.join(HERE, "golden", "make_golden.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    want = {}
    for line in open(os.path.join(HERE, "golden", "vitgen_checksums.txt")):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        want[k] = v
    assert mod.digests() == want


def test_param_counts():
    assert vitgen.param_count(vitgen.preset("tiny16")) == 5_717_416
    assert vitgen.param_count(vitgen.preset("base16")) == 86_567_656
    assert vitgen.param_count(vitgen.preset("large16")) == 304_326_632
    assert vitgen.param_count(vitgen.preset("huge14")) == 632_045_800
    assert vitgen.param_count(vitgen.preset("small16")) == 22_050_664


def test_blob_views_and_pack_roundtrip():
    cfg = vitgen.preset("tiny16").with_(layers=2)
    p, blob = vitgen.make_params(cfg, seed=1)
    assert blob.size == vitgen.param_count(cfg)
    assert np.shares_memory(p["pos"], blob)
    np.testing.assert_array_equal(vitgen.pack_blob(cfg, p), blob)
    q = vitgen.unpack_blob(cfg, blob)
    assert all(np.array_equal(p[k], q[k]) for k in p)
    assert (p["l0.ln1.g"] == 1).all() and (p["l1.ln2.b"] == 0).all()
    w = p["l0.W1"]
    assert abs(float(w.std()) - 0.02) < 5e-4 and abs(float(w.mean())) < 5e-4


def test_bf16_rounding_is_nearest_even():
    a = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, 1.0 + 2.0 ** -9, -(1.0 + 2.0 ** -7 + 2.0 ** -9)],
                 dtype=np.float32)
    vitgen.round_to_bf16_inplace(a)
    # ties go to the even bf16 mantissa; everything else to nearest
    np.testing.assert_array_equal(a, np.array([1.0, 1.0, 1.0 + 2.0 ** -6, 1.0, -(1.0 + 2.0 ** -7)], dtype=np.float32))
    _, blob = vitgen.make_params(vitgen.preset("tiny16").with_(layers=1), seed=0, bf16=True)
    assert (blob.view(np.uint32) & 0xFFFF == 0).all()


def test_pixels_are_per_image_streams():
    cfg = vitgen.preset("tiny16")
    a = vitgen.make_pixels(cfg, 3, seed=5)
    b = vitgen.make_pixels(cfg, 1, seed=5, first=2)
    assert a.dtype == np.float32 and a.shape == (3, 3, 224, 224)
    np.testing.assert_array_equal(a[2:], b)
    assert a.min() >= -1.0 and a.max() < 1.0 and abs(float(a.mean())) < 5e-3


def test_partitions():
    p = vitgen.uneven_partition(16, 24, 0)
    assert len(p) == 16 and p[0][0] == 0 and p[-1][1] == 24
    assert all(b > a for a, b in p) and all(p[i][1] == p[i + 1][0] for i in range(15))
    assert len({b - a for a, b in p}) > 1
    assert vitgen.equal_partition(4, 12) == [(0, 3), (3, 6), (6, 9), (9, 12)]
