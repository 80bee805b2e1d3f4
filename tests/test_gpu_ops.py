"""Each CUDA kernel on its own against the CPU oracle's definition of the same operation,
called through the C boundary (vit_op_*)."""
import numpy as np
import pytest

import vitgen
from oracle import vit_oracle as O

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2110_14895_b200 as vit
    shape = vitgen.preset("tiny16").with_(layers=1)
    _, blob = vitgen.make_params(shape, seed=0)
    m = vit.VitModel(shape, blob, vit.VIT_BF16, 1)
    yield vit, m
    m.check()
    m.close()


def _bf16(a):
    """numpy fp32/fp64 -> (cuda bf16 tensor, the rounded values as fp64 numpy)."""
    t = torch.from_numpy(np.asarray(a, dtype=np.float32)).to(torch.bfloat16).cuda()
    return t, t.float().cpu().numpy().astype(np.float64)


def _f32(a):
    t = torch.from_numpy(np.asarray(a, dtype=np.float32)).cuda()
    return t, t.cpu().numpy().astype(np.float64)


BF16_EPS = 2.0 ** -8      # half an ulp of bf16, relative


# ------------------------------------------------------------------------------- LayerNorm
@pytest.mark.parametrize("rows,cols", [(1, 192), (5, 768), (197, 1024), (1031, 1280), (64, 2048), (33, 64)])
def test_layernorm_bf16(ctx, rows, cols):
    vit, m = ctx
    rng = np.random.default_rng(rows * 7 + cols)
    x, xr = _bf16(rng.normal(0.3, 2.0, size=(rows, cols)))
    g, gr = _f32(1 + 0.1 * rng.normal(size=cols))
    b, br = _f32(0.1 * rng.normal(size=cols))
    y = torch.full_like(x, float("nan"))
    vit.vit_op_layernorm(m.h, vit.VIT_BF16, rows, cols, x.data_ptr(), g.data_ptr(), b.data_ptr(), 1e-6, y.data_ptr())
    torch.cuda.synchronize()
    want = O.layernorm(xr, gr, br, 1e-6)
    got = y.float().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= BF16_EPS * np.abs(want).max() + 1e-5


@pytest.mark.parametrize("rows,cols", [(1, 192), (5, 768), (1031, 1280), (33, 64)])
def test_rowstats_bf16(ctx, rows, cols):
    vit, m = ctx
    rng = np.random.default_rng(rows + 3 * cols)
    x, xr = _bf16(rng.normal(0.7, 1.5, size=(rows, cols)))
    stats = torch.full((rows, 2), float("nan"), dtype=torch.float32, device="cuda")
    vit.vit_op_rowstats(m.h, rows, cols, x.data_ptr(), 1e-6, stats.data_ptr())
    torch.cuda.synchronize()
    got = stats.cpu().numpy()
    mean = xr.mean(-1)
    rstd = 1.0 / np.sqrt(((xr - mean[:, None]) ** 2).mean(-1) + 1e-6)     # the two quantities of the oracle's layernorm
    np.testing.assert_allclose(got[:, 0], mean, rtol=0, atol=2e-6 * np.abs(xr).max())
    np.testing.assert_allclose(got[:, 1], rstd, rtol=2e-6)


# LayerNorm folded into the product: compared with the oracle's layernorm -> linear (-> gelu) on
# the same rows, every tiling; the test folds gain and shift into the operands the way vit_create does
@pytest.mark.parametrize("M,N,K", [(300, 1000 // 8 * 8, 328), (257 * 16, 3840, 1280), (257 * 16, 5120, 1280)])
@pytest.mark.parametrize("tiling", [1, 2, 3])
@pytest.mark.parametrize("gelu", [0, 1])
def test_linear_with_folded_layernorm(ctx, M, N, K, gelu, tiling):
    vit, m = ctx
    rng = np.random.default_rng(M + N + K + gelu)
    x, xr = _bf16(rng.normal(0.3, 2.0, size=(M, K)))
    g = 1 + 0.2 * rng.normal(size=K)
    b = 0.3 * rng.normal(size=K)
    w = rng.normal(size=(N, K)) / np.sqrt(K)
    wq = torch.from_numpy(w.astype(np.float32)).to(torch.bfloat16).float().numpy().astype(np.float64)   # weight as the model holds it
    bias = rng.normal(size=N)
    wg, wgr = _bf16(wq * g[None, :])
    c1, _ = _f32(wgr.sum(-1))
    c0, _ = _f32(bias + wq @ b)
    stats = torch.empty((M, 2), dtype=torch.float32, device="cuda")
    out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    vit.vit_op_rowstats(m.h, M, K, x.data_ptr(), 1e-6, stats.data_ptr())
    vit.vit_op_linear_ln(m.h, M, N, K, x.data_ptr(), stats.data_ptr(), wg.data_ptr(), c1.data_ptr(), c0.data_ptr(),
                         gelu, out.data_ptr(), tiling)
    m.check()
    pre = O.linear(O.layernorm(xr, g, b, 1e-6), wq, bias)
    want = O.gelu(pre) if gelu else pre
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    # output rounding to bf16; the bf16 rounding of gain * weight (uniform within 2^-9 relative per
    # term, K random terms: standard deviation 2^-9 / sqrt(3) of the outputs' scale, bounded here at
    # seven standard deviations); fp32 accumulation
    scale = np.sqrt((pre ** 2).mean())               # of the product before the activation (|gelu'| <= 1.13)
    tol = BF16_EPS * np.abs(want) + 1.13 * 7 * 2.0 ** -9 / np.sqrt(3) * scale + 4e-6 * np.sqrt(K)
    bad = err > tol
    where = np.argwhere(bad)[:3]
    assert not bad.any(), (int(bad.sum()), float(err.max()), where.tolist(),
                           [(float(want[i, j]), float(got[i, j]), float(pre[i, j])) for i, j in where])


@pytest.mark.parametrize("rows,cols", [(3, 192), (200, 1280), (7, 100)])
def test_layernorm_fp32(ctx, rows, cols):
    vit, m = ctx
    rng = np.random.default_rng(rows + cols)
    x, xr = _f32(rng.normal(0.3, 2.0, size=(rows, cols)))
    g, gr = _f32(1 + 0.1 * rng.normal(size=cols))
    b, br = _f32(0.1 * rng.normal(size=cols))
    y = torch.full_like(x, float("nan"))
    vit.vit_op_layernorm(m.h, vit.VIT_FP32, rows, cols, x.data_ptr(), g.data_ptr(), b.data_ptr(), 1e-6, y.data_ptr())
    torch.cuda.synchronize()
    want = O.layernorm(xr, gr, br, 1e-6)
    assert np.abs(y.cpu().numpy() - want).max() <= 1e-5 * np.abs(want).max()


# ------------------------------------------------------------------------------- linear
LINEAR_SHAPES = [
    # M, N, K: single tile, ragged rows, several tiles, both tile widths, N not a tile multiple
    (128, 256, 64), (128, 128, 128), (1, 192, 192), (127, 576, 192), (129, 192, 768),
    (197, 768, 192), (300, 1000 // 8 * 8, 320), (1576, 1024, 1024), (3152, 2304, 768),
    (257 * 40, 1280, 640), (257 * 24, 3840, 1280), (2000, 1280, 5120),
]


@pytest.mark.parametrize("M,N,K", LINEAR_SHAPES)
@pytest.mark.parametrize("epi", [0, 1, 2])
def test_linear_bf16(ctx, M, N, K, epi):
    _linear_case(ctx, M, N, K, epi, 0)


# every tiling of the tensor-core kernel (128x128, 128x256, CTA pair 256x256) with every epilogue:
# a ragged shape (partial tiles in M and N, K not a multiple of 64), a shape of several rounds of
# the static schedule with an odd number of row tiles, and the fc1 / fc2 shapes of ViT-H at a
# quarter batch (pair tiling is what the cost model picks there)
TILED_SHAPES = [(300, 1000 // 8 * 8, 328), (129 * 37, 1280, 1280), (257 * 32, 5120, 1280), (257 * 32, 1280, 5120)]


@pytest.mark.parametrize("M,N,K", TILED_SHAPES)
@pytest.mark.parametrize("tiling", [1, 2, 3])
@pytest.mark.parametrize("epi", [0, 1, 2])
def test_linear_bf16_every_tiling(ctx, M, N, K, epi, tiling):
    _linear_case(ctx, M, N, K, epi, tiling)


def _linear_case(ctx, M, N, K, epi, tiling):
    vit, m = ctx
    rng = np.random.default_rng(M + 3 * N + 7 * K + epi)
    a, ar = _bf16(rng.normal(size=(M, K)))
    w, wr = _bf16(rng.normal(size=(N, K)) / np.sqrt(K))
    bias, br = _f32(rng.normal(size=N))
    res, rr = _bf16(rng.normal(size=(M, N)))
    out = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")
    if epi == 2:                       # in place, as the stage does it
        out.copy_(res)
        resp = out.data_ptr()
    else:
        resp = 0
    if tiling == 0:
        vit.vit_op_linear(m.h, vit.VIT_BF16, M, N, K, a.data_ptr(), w.data_ptr(), bias.data_ptr(), epi, resp, out.data_ptr())
    else:
        vit.vit_op_linear_tiled(m.h, vit.VIT_BF16, M, N, K, a.data_ptr(), w.data_ptr(), bias.data_ptr(), epi, resp,
                                out.data_ptr(), tiling)
    m.check()
    want = O.linear(ar, wr, br)
    if epi == 1:
        want = O.gelu(want)
    elif epi == 2:
        want = want + rr
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - want)
    # output rounding to bf16 (relative) + fp32 accumulation over K terms of size ~1/sqrt(K)
    tol = BF16_EPS * np.abs(want) + 2e-6 * np.sqrt(K) + 1e-6
    bad = err > tol
    assert not bad.any(), (int(bad.sum()), float(err.max()), np.argwhere(bad)[:5].tolist())


@pytest.mark.parametrize("M,N,K", [(1, 10, 8), (70, 130, 33), (197, 576, 192), (300, 192, 768)])
@pytest.mark.parametrize("epi", [0, 1, 2])
def test_linear_fp32(ctx, M, N, K, epi):
    vit, m = ctx
    rng = np.random.default_rng(M + N + K + epi)
    a, ar = _f32(rng.normal(size=(M, K)))
    w, wr = _f32(rng.normal(size=(N, K)) / np.sqrt(K))
    bias, br = _f32(rng.normal(size=N))
    res, rr = _f32(rng.normal(size=(M, N)))
    out = torch.full((M, N), float("nan"), dtype=torch.float32, device="cuda")
    vit.vit_op_linear(m.h, vit.VIT_FP32, M, N, K, a.data_ptr(), w.data_ptr(), bias.data_ptr(), epi,
                      res.data_ptr() if epi == 2 else 0, out.data_ptr())
    m.check()
    want = O.linear(ar, wr, br)
    if epi == 1:
        want = O.gelu(want)
    elif epi == 2:
        want = want + rr
    assert np.abs(out.cpu().numpy() - want).max() <= 2e-5 * max(1.0, np.abs(want).max())


# ------------------------------------------------------------------------------- attention
def _oracle_attention(qkv, images, T, heads):
    return np.concatenate([O.attention(qkv[i * T:(i + 1) * T], heads) for i in range(images)], 0)


@pytest.mark.parametrize("images,T,heads,d", [(1, 5, 2, 16), (2, 197, 3, 64), (3, 257, 2, 80), (1, 32, 1, 128),
                                              (2, 33, 2, 64), (1, 16, 1, 32), (1, 300, 1, 96), (1, 70, 2, 112),
                                              (2, 258, 1, 64), (1, 260, 2, 80), (2, 193, 2, 80), (1, 208, 1, 64),
                                              (1, 241, 1, 80), (1, 256, 2, 64)])
@pytest.mark.parametrize("spread", [0.5, 4.0])
def test_attention_bf16(ctx, images, T, heads, d, spread):
    vit, m = ctx
    rng = np.random.default_rng(T * 31 + d + int(spread * 10))
    H = heads * d
    raw = rng.normal(size=(images * T, 3 * H))
    raw[:, :2 * H] *= np.sqrt(spread)          # q.k/sqrt(d) then has standard deviation ~ spread
    qkv, qr = _bf16(raw)
    out = torch.full((images * T, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    vit.vit_op_attention(m.h, vit.VIT_BF16, images, T, heads, d, qkv.data_ptr(), out.data_ptr())
    m.check()
    want = _oracle_attention(qr, images, T, heads)
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    # P is rounded to bf16 before PV and the output is bf16.  With near-uniform attention the
    # rounding errors of P average out, so the bound scales with the outputs, not with |V|max:
    # two bf16 half-ulps of the largest output plus a small share of |V|max.
    vmax = np.abs(qr[:, 2 * H:]).max()
    assert np.abs(got - want).max() <= 2 * BF16_EPS * np.abs(want).max() + 5e-4 * vmax


def test_attention_bf16_identical_keys_gives_mean_of_values(ctx):
    vit, m = ctx
    rng = np.random.default_rng(99)
    T, heads, d = 257, 2, 80
    H = heads * d
    raw = rng.normal(size=(T, 3 * H))
    raw[:, H:2 * H] = raw[0, H:2 * H]
    qkv, qr = _bf16(raw)
    out = torch.empty((T, H), dtype=torch.bfloat16, device="cuda")
    vit.vit_op_attention(m.h, vit.VIT_BF16, 1, T, heads, d, qkv.data_ptr(), out.data_ptr())
    m.check()
    mean = qr[:, 2 * H:].mean(0)
    assert np.abs(out.float().cpu().numpy() - mean).max() <= 2 * BF16_EPS * np.abs(qr[:, 2 * H:]).max()


@pytest.mark.parametrize("images,T,heads,d", [(1, 5, 2, 4), (2, 197, 3, 64), (1, 257, 2, 80)])
def test_attention_fp32(ctx, images, T, heads, d):
    vit, m = ctx
    rng = np.random.default_rng(T + d)
    H = heads * d
    qkv, qr = _f32(rng.normal(size=(images * T, 3 * H)))
    out = torch.full((images * T, H), float("nan"), dtype=torch.float32, device="cuda")
    vit.vit_op_attention(m.h, vit.VIT_FP32, images, T, heads, d, qkv.data_ptr(), out.data_ptr())
    m.check()
    want = _oracle_attention(qr, images, T, heads)
    assert np.abs(out.cpu().numpy() - want).max() <= 2e-5


# ------------------------------------------------------------------------------- degenerate and extreme sizes
def test_empty_inputs_launch_nothing_and_succeed(ctx):
    """Zero rows / zero images are valid calls that do nothing (a ragged split can leave them)."""
    vit, m = ctx
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(64, dtype=torch.float32, device="cuda")
    before = m.launches
    vit.vit_op_linear(m.h, vit.VIT_BF16, 0, 64, 64, x.data_ptr(), x.data_ptr(), f.data_ptr(), 0, 0, x.data_ptr())
    vit.vit_op_layernorm(m.h, vit.VIT_BF16, 0, 64, x.data_ptr(), f.data_ptr(), f.data_ptr(), 1e-6, x.data_ptr())
    vit.vit_op_rowstats(m.h, 0, 64, x.data_ptr(), 1e-6, f.data_ptr())
    vit.vit_op_attention(m.h, vit.VIT_BF16, 0, 197, 1, 64, x.data_ptr(), x.data_ptr())
    m.check()
    assert (x == 0).all() and (f == 0).all()
    assert m.launches - before <= 4          # counted as calls; no kernel had anything to do


@pytest.mark.parametrize("M,N,K", [(1, 8, 8), (3, 16, 24), (130, 8, 4096)])
def test_linear_bf16_smallest_and_longest_shapes(ctx, M, N, K):
    _linear_case(ctx, M, N, K, 0, 0)
    _linear_case(ctx, M, N, K, 2, 0)


def test_attention_bf16_longest_sequence(ctx):
    """T = 512 is the longest sequence a configuration may have (warp-level kernel)."""
    vit, m = ctx
    rng = np.random.default_rng(512)
    T, heads, d = 512, 2, 64
    H = heads * d
    qkv, qr = _bf16(rng.normal(size=(T, 3 * H)))
    out = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device="cuda")
    vit.vit_op_attention(m.h, vit.VIT_BF16, 1, T, heads, d, qkv.data_ptr(), out.data_ptr())
    m.check()
    want = _oracle_attention(qr, 1, T, heads)
    got = out.float().cpu().numpy()
    assert np.isfinite(got).all()
    assert np.abs(got - want).max() <= 2 * BF16_EPS * np.abs(want).max() + 5e-4 * np.abs(qr[:, 2 * H:]).max()


# ------------------------------------------------------------------------------- argument checks
def test_op_argument_errors(ctx):
    vit, m = ctx
    x = torch.zeros(64, 64, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(64, dtype=torch.float32, device="cuda")
    with pytest.raises(vit.VitError) as e:
        vit.vit_op_linear(m.h, vit.VIT_BF16, 64, 60, 64, x.data_ptr(), x.data_ptr(), f.data_ptr(), 0, 0, x.data_ptr())
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    with pytest.raises(vit.VitError):
        vit.vit_op_linear(m.h, vit.VIT_BF16, 64, 64, 64, x.data_ptr() + 2, x.data_ptr(), f.data_ptr(), 0, 0, x.data_ptr())
    with pytest.raises(vit.VitError):
        vit.vit_op_linear(m.h, vit.VIT_BF16, 64, 64, 64, x.data_ptr(), x.data_ptr(), f.data_ptr(), 2, 0, x.data_ptr())
    with pytest.raises(vit.VitError):
        vit.vit_op_attention(m.h, vit.VIT_BF16, 1, 16, 1, 24, x.data_ptr(), x.data_ptr())
    with pytest.raises(vit.VitError):
        vit.vit_op_layernorm(m.h, 5, 1, 64, x.data_ptr(), f.data_ptr(), f.data_ptr(), 1e-6, x.data_ptr())
