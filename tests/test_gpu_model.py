"""End-to-end parity of the CUDA path with the CPU oracle on the same seeded inputs, and the
stage-composition invariant on the GPU.  Everything goes through the C boundary."""
import os

import numpy as np
import pytest

import vitgen
from oracle import vit_oracle as O

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def _vit():
    import paper_2110_14895_b200 as vit
    return vit


def logits_within_tolerance(got, want, rel_max, min_cos=None):
    """max |dlogit| <= rel_max * max |logit| over the whole array; cosine per image."""
    got = np.asarray(got, dtype=np.float64)
    scale = np.abs(want).max()
    err = np.abs(got - want).max()
    cos = (got * want).sum(-1) / (np.linalg.norm(got, axis=-1) * np.linalg.norm(want, axis=-1))
    ok = err <= rel_max * scale and (min_cos is None or cos.min() >= min_cos)
    return ok, f"max|d|={err:.3e} ({err / scale:.3e} of max|logit|), min cos={cos.min():.6f}"


def _model(shape, dtype, max_mb, seed=0, bf16_weights=True, ln_affine=False):
    vit = _vit()
    params, blob = vitgen.make_params(shape, seed=seed, bf16=bf16_weights, ln_affine=ln_affine)
    return vit, vit.VitModel(shape, blob, dtype, max_mb), params


# ---------------------------------------------------------------------------------------------
# ViT-Tiny/16, batch 1, fp32 mode, two stages [0,6)+[6,12): within 1e-3 of the oracle.
def test_tiny_fp32_two_stages_matches_oracle():
    shape = vitgen.preset("tiny16")
    vit, m, params = _model(shape, _vit().VIT_FP32, 2, bf16_weights=False)
    pix = vitgen.make_pixels(shape, 1, seed=0)
    got = m.forward(torch.from_numpy(pix).cuda(), stages=[(0, 6), (6, 12)])
    m.check()
    want = O.forward(params, shape, pix, [(0, 6), (6, 12)])
    ok, msg = logits_within_tolerance(got.cpu().numpy(), want, 1e-3)
    assert ok, msg
    m.close()


@pytest.mark.parametrize("dtype_name", ["bf16", "fp32"])
def test_tiny_intermediate_tensors_match_oracle(dtype_name):
    vit = _vit()
    dtype = vit.VIT_BF16 if dtype_name == "bf16" else vit.VIT_FP32
    shape = vitgen.preset("tiny16").with_(layers=2)
    vit, m, params = _model(shape, dtype, 3, seed=5, ln_affine=True)
    pix = vitgen.make_pixels(shape, 3, seed=5)
    x = m.patch_embed(torch.from_numpy(pix).cuda())
    m.check()
    want = O.patch_embed(params, shape, pix)
    tol = 1e-5 if dtype_name == "fp32" else 2.0 ** -8
    got = x.float().cpu().numpy()
    assert np.abs(got - want).max() <= tol * np.abs(want).max() + (3e-3 if dtype_name == "bf16" else 0)
    y = m.run_stage(0, 2, x)
    m.check()
    want2 = O.run_stage(params, shape, 0, 2, want)
    rel = np.abs(y.float().cpu().numpy() - want2).max() / np.abs(want2).max()
    assert rel <= (1e-4 if dtype_name == "fp32" else 2e-2), rel
    m.close()


def test_tiny_bf16_matches_oracle_and_composes_bit_exactly():
    shape = vitgen.preset("tiny16")
    vit, m, params = _model(shape, _vit().VIT_BF16, 4)
    pix = vitgen.make_pixels(shape, 4, seed=0)
    dpix = torch.from_numpy(pix).cuda()
    whole = m.forward(dpix)
    want = O.forward(params, shape, pix)
    ok, msg = logits_within_tolerance(whole.cpu().numpy(), want, 2e-2, 0.9995)
    assert ok, msg
    x0 = m.patch_embed(dpix)
    ref = m.run_stage(0, shape.layers, x0)
    for k in range(1, shape.layers):
        a = m.run_stage(0, k, x0)
        b = m.run_stage(k, shape.layers, a, out=a)       # second stage in place
        assert torch.equal(ref, b), k
    m.check()
    m.close()


def test_stage_argument_errors():
    shape = vitgen.preset("tiny16").with_(layers=3)
    vit, m, _ = _model(shape, _vit().VIT_BF16, 2)
    x = torch.zeros((2, m.T, shape.hidden), dtype=torch.bfloat16, device="cuda")
    ws = m.workspace(2)
    def run(lb, le, mb=2, inp=None, out=None, wsb=None):
        vit.vit_run_stage(m.h, lb, le, mb, (inp or x.data_ptr()), (out or x.data_ptr()), ws.data_ptr(),
                          ws.numel() if wsb is None else wsb)
    for lb, le in [(0, 0), (2, 1), (-1, 2), (0, 4), (3, 3)]:
        with pytest.raises(vit.VitError) as e:
            run(lb, le)
        assert e.value.status == vit.VIT_ERR_RANGE
    with pytest.raises(vit.VitError) as e:
        run(0, 1, mb=3)
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    with pytest.raises(vit.VitError) as e:
        run(0, 1, wsb=1024)
    assert e.value.status == vit.VIT_ERR_WORKSPACE
    with pytest.raises(vit.VitError) as e:
        run(0, 1, out=x.data_ptr() + 256)            # partial overlap
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    before = m.launches
    with pytest.raises(vit.VitError):
        run(0, 9)
    assert m.launches == before                       # a failed call launches nothing
    m.close()


# ---------------------------------------------------------------------------------------------
def _pipeline_vs_oracle(name, batch, mb, stages, n_streams, sample, host=False):
    """Runs the stage runner on the full batch; the oracle evaluates the sampled images only
    (images are independent, so that is the same function)."""
    shape = vitgen.preset(name)
    vit, m, params = _model(shape, _vit().VIT_BF16, mb)
    pix = vitgen.make_pixels(shape, batch, seed=0)
    wss, streams, wsb = m.make_pipeline_buffers(mb, n_streams)
    counts = [le - lb for lb, le in stages]
    if host:
        hp = torch.from_numpy(pix).pin_memory()
        logits = torch.empty((batch, shape.num_classes), dtype=torch.float32).pin_memory()
        torch.cuda.synchronize()
        m.run_pipeline(counts, mb, hp, logits, wss, streams, wsb, host=True)
    else:
        dp = torch.from_numpy(pix).cuda()
        logits = torch.full((batch, shape.num_classes), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        m.run_pipeline(counts, mb, dp, logits, wss, streams, wsb)
    for s in streams:
        m.check(s)
    got = logits.cpu().numpy()
    assert np.isfinite(got).all()
    want = O.forward(params, shape, pix[sample])
    ok, msg = logits_within_tolerance(got[sample], want, 2e-2, 0.9995)
    assert ok, msg
    return vit, m, pix, got


def test_base16_batch64_four_microbatches_four_stages():
    sample = [0, 15, 16, 31, 47, 48, 62, 63]
    vit, m, pix, got = _pipeline_vs_oracle("base16", 64, 16, vitgen.equal_partition(4, 12), 4, sample)
    # the single-call result on one microbatch is bit-identical to the staged pipeline result
    one = m.forward(torch.from_numpy(pix[16:32]).cuda())
    assert np.array_equal(one.cpu().numpy(), got[16:32])
    m.close()


def test_small16_batch32_two_microbatches_three_stages():
    _, m, _, _ = _pipeline_vs_oracle("small16", 32, 16, [(0, 5), (5, 6), (6, 12)], 2, [0, 15, 16, 31])
    m.close()


# ---------------------------------------------------------------------------------------------
# The compressed (distilled) family: a distillation token after the class token (198 tokens) and a
# second classifier; tiny / small / base dimensions.
@pytest.mark.parametrize("dtype_name", ["bf16", "fp32"])
def test_distilled_tiny_intermediate_tensors_and_logits_match_oracle(dtype_name):
    vit = _vit()
    dtype = vit.VIT_BF16 if dtype_name == "bf16" else vit.VIT_FP32
    shape = vitgen.preset("deit_tiny16").with_(layers=2)
    vit, m, params = _model(shape, dtype, 3, seed=7, ln_affine=True, bf16_weights=dtype_name == "bf16")
    assert m.T == 198
    pix = vitgen.make_pixels(shape, 3, seed=7)
    x = m.patch_embed(torch.from_numpy(pix).cuda())
    m.check()
    want = O.patch_embed(params, shape, pix)
    got = x.float().cpu().numpy()
    tol = 1e-5 if dtype_name == "fp32" else 2.0 ** -8
    assert np.abs(got - want).max() <= tol * np.abs(want).max() + (3e-3 if dtype_name == "bf16" else 0)
    # the two special rows exactly as defined
    assert np.abs(got[:, :2] - want[:, :2]).max() <= tol * np.abs(want[:, :2]).max()
    y = m.run_stage(0, 2, x)
    logits = m.head(y)
    m.check()
    want_y = O.run_stage(params, shape, 0, 2, want)
    want_l = O.head(params, shape, want_y)
    ok, msg = logits_within_tolerance(logits.cpu().numpy(), want_l, 1e-3 if dtype_name == "fp32" else 2e-2)
    assert ok, msg
    # the head on the oracle's own tokens isolates the two-classifier mean from upstream error
    yt = torch.from_numpy(want_y.astype(np.float32)).cuda().to(m.act_dtype)
    l2 = m.head(yt).cpu().numpy()
    want_l2 = O.head(params, shape, yt.float().cpu().numpy().astype(np.float64))
    assert np.abs(l2 - want_l2).max() <= 1e-4 * max(1.0, np.abs(want_l2).max())
    m.close()


@pytest.mark.parametrize("name,batch,mb", [("deit_tiny16", 8, 4), ("deit_small16", 32, 16), ("deit_base16", 32, 16)])
def test_distilled_models_pipeline_matches_oracle(name, batch, mb):
    sample = [0, mb - 1, mb, batch - 1]
    _, m, pix, got = _pipeline_vs_oracle(name, batch, mb, vitgen.equal_partition(4, 12), 2, sample)
    one = m.forward(torch.from_numpy(pix[mb:2 * mb]).cuda())
    assert np.array_equal(one.cpu().numpy(), got[mb:2 * mb])       # staged == single call, bit for bit
    m.close()


def test_base16_host_buffers_pipeline():
    _, m, _, _ = _pipeline_vs_oracle("base16", 8, 4, vitgen.equal_partition(4, 12), 2, [0, 3, 4, 7], host=True)
    m.close()


def test_large16_batch128_microbatch8_uneven_16_stages():
    stages = vitgen.uneven_partition(16, 24, seed=0)
    sample = [0, 7, 8, 64, 71, 120, 127]
    vit, m, pix, got = _pipeline_vs_oracle("large16", 128, 8, stages, 1, sample)
    one = m.forward(torch.from_numpy(pix[64:72]).cuda())
    assert np.array_equal(one.cpu().numpy(), got[64:72])
    m.close()


def test_large16_grouped_microbatches_match_ungrouped_and_oracle():
    """Several microbatches carried through every launch together: the same function of every
    image as microbatch by microbatch, bit for bit (rows of a GEMM, rows of LayerNorm and heads of
    attention do not depend on what else is in the launch, and the K order is fixed), and within
    the bf16 tolerance of the oracle."""
    shape = vitgen.preset("large16")
    vit, m, params = _model(shape, _vit().VIT_BF16, 32)
    B, mb = 40, 8                                   # five microbatches: a full group of four and a ragged one
    pix = vitgen.make_pixels(shape, B, seed=3)
    dp = torch.from_numpy(pix).cuda()
    stages = [le - lb for lb, le in vitgen.uneven_partition(16, 24, seed=0)]
    outs = []
    for group in (1, 4):
        wss, streams, wsb = m.make_pipeline_buffers(mb * group, 2)
        logits = torch.full((B, shape.num_classes), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        m.run_pipeline(stages, mb, dp, logits, wss, streams, wsb, group=group)
        for s in streams:
            m.check(s)
        outs.append(logits.cpu().numpy())
    sample = [0, 7, 8, 31, 32, 39]
    want = O.forward(params, shape, pix[sample])
    for got in outs:
        assert np.isfinite(got).all()
        ok, msg = logits_within_tolerance(got[sample], want, 2e-2, 0.9995)
        assert ok, msg
    assert np.array_equal(outs[0], outs[1])
    with pytest.raises(vit.VitError) as e:          # group * microbatch beyond max_microbatch
        m.run_pipeline(stages, mb, dp, logits, wss, streams, wsb, group=5)
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    m.close()


def test_huge14_batch128_single_stage_equals_eight_stages_and_oracle():
    shape = vitgen.preset("huge14")
    vit, m, params = _model(shape, _vit().VIT_BF16, 128)
    B = 128
    pix = vitgen.make_pixels(shape, B, seed=0)
    dp = torch.from_numpy(pix).cuda()
    x0 = m.patch_embed(dp)
    a = m.run_stage(0, 32, x0)
    la = m.head(a)
    b = x0.clone()
    for lb, le in vitgen.equal_partition(8, 32):
        m.run_stage(lb, le, b, out=b)
    lb_ = m.head(b)
    m.check()
    assert torch.equal(a, b)
    assert torch.equal(la, lb_)
    sample = [0, 1, 63, 64, 100, 127]
    want = O.forward(params, shape, pix[sample])
    ok, msg = logits_within_tolerance(la.cpu().numpy()[sample], want, 2e-2, 0.9995)
    assert ok, msg
    m.close()


def test_huge14_microbatch_sweep_every_size_matches_oracle():
    """The microbatch sweep in full: 256 images of ViT-H/14 through four stages of eight layers,
    microbatch sizes 1 ... 256 on min(4, 256/size) streams.  Every size is compared with the
    oracle on images that are the first or the last of a microbatch at that size (image 0 and
    255 at every size, 63|64 and 127|128 at sizes up to 64 and 128).  Tile shapes differ between
    sizes, so the sizes are not required to agree bit for bit; their largest mutual difference is
    printed."""
    shape = vitgen.preset("huge14")
    vit, m, params = _model(shape, _vit().VIT_BF16, 256)
    B = 256
    pix = vitgen.make_pixels(shape, B, seed=0)
    dp = torch.from_numpy(pix).cuda()
    sample = [0, 63, 64, 127, 128, 255]
    want = O.forward(params, shape, pix[sample])
    first = None
    for mb in (1, 2, 4, 8, 16, 32, 64, 128, 256):
        ns = min(4, B // mb)
        wss, streams, wsb = m.make_pipeline_buffers(mb, ns)
        logits = torch.full((B, shape.num_classes), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        m.run_pipeline([8, 8, 8, 8], mb, dp, logits, wss, streams, wsb)
        for s in streams:
            m.check(s)
        got = logits.cpu().numpy()
        assert np.isfinite(got).all(), mb
        ok, msg = logits_within_tolerance(got[sample], want, 2e-2, 0.9995)
        assert ok, (mb, msg)
        if first is None:
            first = got
        else:
            print(f"microbatch {mb}: max |logit - logit at microbatch 1| = {np.abs(got - first).max():.3e}")
        del wss, logits
        torch.cuda.empty_cache()
    m.close()


def test_bounded_wait_raises_status_and_leaves_the_handle_usable():
    """A wait nothing satisfies expires after its (short) limit: the status word reports it once,
    nothing hangs, and the same handle then runs a stage correctly."""
    shape = vitgen.preset("tiny16").with_(layers=2)
    vit, m, _ = _model(shape, _vit().VIT_BF16, 1)
    x = torch.randn((1, m.T, shape.hidden), device="cuda").to(torch.bfloat16)
    ref = m.run_stage(0, 2, x)
    m.check()
    vit.vit_debug_wait_probe(m.h, 2_000_000)          # about a millisecond
    with pytest.raises(vit.VitError) as e:
        m.check()
    assert e.value.status == vit.VIT_ERR_TIMEOUT
    m.check()                                          # the word was cleared by the read
    again = m.run_stage(0, 2, x)
    m.check()
    assert torch.equal(ref, again)
    m.close()


def test_pipeline_ragged_last_microbatch_and_argument_errors():
    """Batch 5 in microbatches of 2 leaves a last microbatch of one image; stage counts must sum
    to the layer count; a failed call launches nothing."""
    shape = vitgen.preset("tiny16").with_(layers=4)
    vit, m, params = _model(shape, _vit().VIT_BF16, 2)
    pix = vitgen.make_pixels(shape, 5, seed=2)
    dp = torch.from_numpy(pix).cuda()
    wss, streams, wsb = m.make_pipeline_buffers(2, 2)
    logits = torch.full((5, shape.num_classes), float("nan"), dtype=torch.float32, device="cuda")
    torch.cuda.synchronize()
    m.run_pipeline([1, 3], 2, dp, logits, wss, streams, wsb)
    for s in streams:
        m.check(s)
    want = O.forward(params, shape, pix)
    ok, msg = logits_within_tolerance(logits.cpu().numpy(), want, 2e-2, 0.9995)
    assert ok, msg
    one = m.forward(dp[4:5])                      # the ragged microbatch equals a batch-of-one call
    assert torch.equal(one, logits[4:5])
    before = m.launches
    for counts, status in (([1, 2], vit.VIT_ERR_RANGE), ([4, 0], vit.VIT_ERR_RANGE), ([], vit.VIT_ERR_INVALID_ARG)):
        with pytest.raises(vit.VitError) as e:
            m.run_pipeline(counts, 2, dp, logits, wss, streams, wsb)
        assert e.value.status == status
    with pytest.raises(vit.VitError) as e:
        m.run_pipeline([4], 3, dp, logits, wss, streams, wsb)      # microbatch above max_microbatch
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    with pytest.raises(vit.VitError) as e:
        m.run_pipeline([4], 2, dp, logits, wss, streams, 1024)     # workspace too small
    assert e.value.status == vit.VIT_ERR_WORKSPACE
    assert m.launches == before
    m.close()


def test_stage_pipeline_executor_on_the_gpu_single_rank():
    """The stage-per-device runner with the CUDA executor on one rank (first and last stage at
    once, so nothing is sent): embeds, runs the stage and classifies microbatch by microbatch, with
    a ragged last microbatch, and gives the bits of a direct forward call."""
    import torch.distributed as dist
    from paper_2110_14895_b200 import pipeline as PL
    shape = vitgen.preset("tiny16").with_(layers=3)
    vit, m, params = _model(shape, _vit().VIT_BF16, 2)
    port = 29000 + (os.getpid() % 500)
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1)
    try:
        pipe = PL.StagePipeline(PL.VitStageExecutor(m, 0, shape.layers, True, True), dist, max_microbatch=2)
        pix = torch.from_numpy(vitgen.make_pixels(shape, 5, seed=4)).cuda()
        logits = torch.full((5, shape.num_classes), float("nan"), dtype=torch.float32, device="cuda")
        for _ in range(2):                                   # two steps: the roll call advances
            pipe.run(5, 2, pixels=pix, logits=logits)
        torch.cuda.synchronize()
        m.check()
        assert [e for e in pipe.log if e[0] == "stage"][:3] == [("stage", 0), ("stage", 1), ("stage", 2)]
        want = torch.cat([m.forward(pix[i:i + 2]) for i in (0, 2, 4)])
        assert torch.equal(logits, want)
        ok, msg = logits_within_tolerance(logits.cpu().numpy(), O.forward(params, shape, pix.cpu().numpy()), 2e-2, 0.9995)
        assert ok, msg
    finally:
        dist.destroy_process_group()
    m.close()


@pytest.mark.parametrize("name,mb", [("tiny16", 3), ("deit_tiny16", 2), ("huge14", 2)])
def test_kernels_stay_inside_their_buffers(name, mb):
    """Workspace, activations and logits are carved out of one allocation with guard bands of a
    known pattern on both sides of each; after patch embed, two stages and the head every guard
    byte is still in place (with exactly the workspace size the library asks for)."""
    shape = vitgen.preset(name).with_(layers=2)
    vit, m, _ = _model(shape, _vit().VIT_BF16, mb)
    G = 4096                                                     # guard bytes, keeps 256-byte alignment
    sizes = {"ws": vit.vit_workspace_bytes(m.cfg, mb), "tok": mb * m.T * shape.hidden * 2,
             "out": mb * m.T * shape.hidden * 2, "logits": mb * shape.num_classes * 4}
    off, total = {}, G
    for k, n in sizes.items():
        off[k] = total
        total += (n + 255) // 256 * 256 + G
    buf = torch.full((total,), 0xA5, dtype=torch.uint8, device="cuda")
    base = buf.data_ptr()
    assert base % 256 == 0
    pix = torch.from_numpy(vitgen.make_pixels(shape, mb, seed=1)).cuda()
    ptr = {k: base + o for k, o in off.items()}
    vit.vit_patch_embed(m.h, mb, pix.data_ptr(), ptr["tok"], ptr["ws"], sizes["ws"])
    vit.vit_run_stage(m.h, 0, 1, mb, ptr["tok"], ptr["out"], ptr["ws"], sizes["ws"])
    vit.vit_run_stage(m.h, 1, 2, mb, ptr["out"], ptr["out"], ptr["ws"], sizes["ws"])
    vit.vit_head(m.h, mb, ptr["out"], ptr["logits"], ptr["ws"], sizes["ws"])
    m.check()
    host = buf.cpu().numpy()
    guards = np.ones(total, dtype=bool)
    for k, n in sizes.items():
        guards[off[k]:off[k] + n] = False
    assert (host[guards] == 0xA5).all(), {k: int((host[off[k] + sizes[k]:off[k] + sizes[k] + G] != 0xA5).sum()) for k in sizes}
    logits = host[off["logits"]:off["logits"] + sizes["logits"]].copy().view(np.float32)
    assert np.isfinite(logits).all()
    m.close()
