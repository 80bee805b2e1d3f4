"""vit_head_static: the classification head for callers that cannot allocate device memory
(real-time loops that must stay out of the allocator, plugins whose host owns every byte of
device memory).  Its scratch is a fixed array inside the library, so the caller passes only the
tokens and the logits buffer.

The file name sorts last on purpose: a run that stops at the first failure has then already
been through every other test.  The test also passes on its own in a fresh process.
"""
import numpy as np
import pytest

import vitgen

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _model(shape, max_mb, dtype=None):
    import paper_2110_14895_b200 as vit
    _, blob = vitgen.make_params(shape, seed=11, ln_affine=True)
    return vit, vit.VitModel(shape, blob, vit.VIT_BF16 if dtype is None else dtype, max_mb)


def test_head_static_matches_head_on_two_calls_in_a_row():
    shape = vitgen.preset("tiny16").with_(layers=1)
    vit, m = _model(shape, 8)
    gen = torch.Generator(device="cuda").manual_seed(3)
    for call, mb in enumerate((8, 5)):          # second call reuses the array with other contents
        tokens = (2.0 * torch.randn((mb, m.T, shape.hidden), device="cuda", generator=gen)).to(torch.bfloat16)
        want = m.head(tokens)                   # existing entry point, caller-provided scratch
        got = torch.full_like(want, float("nan"))
        vit.vit_head_static(m.h, mb, tokens.data_ptr(), got.data_ptr())
        m.check()
        assert torch.isfinite(got).all(), call
        # same kernels, same inputs: the tolerance of the other head tests (2e-2 of max |logit|)
        # is met with room to spare; in fact the two results are identical
        err = (got - want).abs().max().item()
        assert err <= 2e-2 * want.abs().max().item(), (call, err)
        assert torch.equal(got, want), call
    m.close()


def test_head_static_with_distillation_token_matches_head():
    """Two feature rows per image (class and distillation token) go through the fixed array."""
    shape = vitgen.preset("deit_tiny16").with_(layers=1)
    vit, m = _model(shape, 6)
    tokens = torch.randn((6, m.T, shape.hidden), device="cuda").to(torch.bfloat16)
    want = m.head(tokens)
    for _ in range(2):
        got = torch.full_like(want, float("nan"))
        vit.vit_head_static(m.h, 6, tokens.data_ptr(), got.data_ptr())
        m.check()
        assert torch.equal(got, want)
    m.close()


def test_head_static_fp32_mode_matches_head():
    shape = vitgen.preset("tiny16").with_(layers=1)
    vit, m = _model(shape, 3, dtype=1)
    tokens = torch.randn((3, m.T, shape.hidden), device="cuda")
    want = m.head(tokens)
    got = torch.empty_like(want)
    for _ in range(2):
        got.fill_(float("nan"))
        vit.vit_head_static(m.h, 3, tokens.data_ptr(), got.data_ptr())
        m.check()
        assert (got - want).abs().max().item() <= 1e-3 * want.abs().max().item()
    m.close()


def test_head_static_rejects_sizes_beyond_its_array():
    # microbatch * hidden = 257 * 2048 floats is just over the 512 Ki limit
    shape = vitgen.ViTConfig(image_size=32, patch_size=16, hidden=2048, layers=1, heads=16, mlp_dim=64,
                             num_classes=16)
    vit, m = _model(shape, 257)
    assert 257 * shape.hidden > vit.VIT_HEAD_STATIC_MAX_FLOATS >= 256 * shape.hidden
    tokens = torch.zeros((257, m.T, shape.hidden), dtype=torch.bfloat16, device="cuda")
    logits = torch.zeros((257, shape.num_classes), device="cuda")
    before = m.launches
    with pytest.raises(vit.VitError) as e:
        vit.vit_head_static(m.h, 257, tokens.data_ptr(), logits.data_ptr())
    assert e.value.status == vit.VIT_ERR_TOO_LARGE
    assert "scratch" in str(e.value)
    assert m.launches == before                  # nothing was launched
    vit.vit_head_static(m.h, 256, tokens.data_ptr(), logits.data_ptr())   # the largest allowed size
    m.check()
    want = m.head(tokens[:256].contiguous())
    assert torch.equal(logits[:256], want)
    with pytest.raises(vit.VitError) as e:
        vit.vit_head_static(m.h, 0, tokens.data_ptr(), logits.data_ptr())
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    m.close()
