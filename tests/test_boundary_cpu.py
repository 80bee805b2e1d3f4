"""Host-side checks of the C boundary that need no GPU: the library loads, exports every
symbol the header declares, and its size queries and argument checks behave."""
import os
import re

import numpy as np
import pytest

import vitgen
import paper_2110_14895_b200 as vit
from paper_2110_14895_b200 import build as vit_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    vit_build.build()
    return vit.lib()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "vit.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vit_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(L):
    names = _declared_functions()
    assert len(names) >= 16
    for n in names:
        assert hasattr(L, n), n
    assert sorted(vit.EXPORTS) == names


def test_param_count_matches_generator(L):
    for name in vitgen.PRESETS:
        shape = vitgen.preset(name)
        for dt in (vit.VIT_BF16, vit.VIT_FP32):
            assert vit.vit_param_count(vit.make_config(shape, dt, 4)) == vitgen.param_count(shape)


def test_invalid_configs_give_zero_sizes(L):
    good = vitgen.preset("tiny16")
    bad = [good.with_(patch_size=15), good.with_(heads=5), good.with_(hidden=200, heads=4),
           good.with_(mlp_dim=100), good.with_(layers=0), good.with_(image_size=1024, patch_size=16)]
    for shape in bad:
        cfg = vit.make_config(shape, vit.VIT_BF16, 1)
        assert vit.vit_param_count(cfg) == 0
        assert vit.vit_workspace_bytes(cfg, 1) == 0
    cfg = vit.make_config(good, 7, 1)
    assert vit.vit_param_count(cfg) == 0
    cfg = vit.make_config(good, vit.VIT_BF16, 0)
    assert vit.vit_param_count(cfg) == 0


def test_workspace_sizes(L):
    shape = vitgen.preset("huge14")
    cfg = vit.make_config(shape, vit.VIT_BF16, 128)
    M = 128 * 257
    stage = M * 1280 * 2 + M * 5120 * 2 + M * 8      # attention output, QKV / MLP hidden, LayerNorm statistics
    assert vit.vit_workspace_bytes(cfg, 128) >= stage
    assert vit.vit_workspace_bytes(cfg, 128) < stage + 4096
    assert vit.vit_workspace_bytes(cfg, 0) == 0
    pipe = vit.vit_pipeline_workspace_bytes(cfg, 8)
    assert pipe >= vit.vit_workspace_bytes(cfg, 8) + 8 * 3 * 224 * 224 * 4 + 8 * 257 * 1280 * 2
    cfg32 = vit.make_config(shape, vit.VIT_FP32, 128)
    # twice the activation buffers of the bf16 mode (the statistics buffer has the same size in both)
    assert vit.vit_workspace_bytes(cfg32, 4) >= 2 * (vit.vit_workspace_bytes(cfg, 4) - 768 - 4 * 257 * 8)


def test_status_strings(L):
    seen = set()
    for s in range(0, -8, -1):
        t = vit.status_string(s)
        assert t and t != "unknown status"
        seen.add(t)
    assert len(seen) == 8
    assert vit.status_string(-99) == "unknown status"


def test_create_rejects_bad_arguments_before_touching_a_device(L):
    shape = vitgen.preset("tiny16").with_(layers=1)
    cfg = vit.make_config(shape, vit.VIT_BF16, 1)
    blob = np.zeros(vitgen.param_count(shape) - 1, dtype=np.float32)
    with pytest.raises(vit.VitError) as e:
        vit.vit_create(cfg, blob)
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    badcfg = vit.make_config(shape.with_(heads=5), vit.VIT_BF16, 1)
    with pytest.raises(vit.VitError) as e:
        vit.vit_create(badcfg, blob)
    assert e.value.status == vit.VIT_ERR_CONFIG


def test_missing_library_fails_loudly(monkeypatch):
    import paper_2110_14895_b200.binding as b
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", "/nonexistent/libvit_b200.so")
    with pytest.raises(RuntimeError):
        b.lib()
