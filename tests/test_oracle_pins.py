"""Pins for the CPU oracle: closed forms, invariants and a scalar brute-force model.

Each test is chosen so that a plausible slip in the oracle (dropped term, wrong sign or
index, transposed operand, wrong flatten order) fails at least one of them.
"""
import math

import numpy as np
import pytest

import vitgen
from oracle import vit_oracle as O

TINY = vitgen.ViTConfig(image_size=4, patch_size=2, channels=3, hidden=8, layers=2, heads=2,
                        mlp_dim=16, num_classes=10, ln_eps=1e-6)


def _rand_params(cfg, seed, std=0.5):
    rng = np.random.default_rng(seed)
    p = {}
    for name, shape, kind in vitgen.param_specs(cfg):
        a = rng.normal(0.0, std, size=shape)
        if kind == "gain":
            a = 1.0 + 0.3 * a
        p[name] = a
    return p


# ----------------------------------------------------------------------------- inventory
def test_parameter_inventory_matches_paper_count():
    # Section 1 of the paper: ViT-Base has 86.6M parameters.
    n = vitgen.param_count(vitgen.preset("base16"))
    assert n == 86_567_656
    assert round(n / 1e6, 1) == 86.6


# ----------------------------------------------------------------------------- LayerNorm
def test_layernorm_closed_form():
    x = np.array([[1.0, 2.0, 3.0, 4.0]])
    y = O.layernorm(x, np.ones(4), np.zeros(4), 0.0)
    np.testing.assert_allclose(y[0], [-1.3416407865, -0.4472135955, 0.4472135955, 1.3416407865],
                               rtol=0, atol=1e-9)


def test_layernorm_moments_and_invariances():
    rng = np.random.default_rng(1)
    x = rng.normal(3.0, 2.0, size=(7, 64))
    eps = 1e-6
    y = O.layernorm(x, np.ones(64), np.zeros(64), eps)
    assert np.abs(y.mean(-1)).max() < 1e-12
    var = x.var(-1)
    np.testing.assert_allclose(y.var(-1), var / (var + eps), rtol=1e-12)
    # shift and positive scale of the input leave the output unchanged (eps -> 0)
    y0 = O.layernorm(x, np.ones(64), np.zeros(64), 0.0)
    y1 = O.layernorm(5.0 * x + 11.0, np.ones(64), np.zeros(64), 0.0)
    np.testing.assert_allclose(y0, y1, atol=1e-10)
    # affine part: gain multiplies, shift adds, per feature
    g, b = rng.normal(size=64), rng.normal(size=64)
    np.testing.assert_allclose(O.layernorm(x, g, b, 0.0), y0 * g + b, atol=1e-12)


def test_layernorm_eps_sits_inside_sqrt():
    x = np.array([[0.0, 2.0]])            # mean 1, biased variance 1
    y = O.layernorm(x, np.ones(2), np.zeros(2), 3.0)
    np.testing.assert_allclose(y[0], [-0.5, 0.5], atol=1e-15)   # 1/sqrt(1+3)


# ----------------------------------------------------------------------------- softmax
def test_softmax_closed_form_and_invariants():
    s = np.array([[0.0, math.log(2.0), math.log(3.0)]])
    np.testing.assert_allclose(O.softmax_rows(s)[0], [1 / 6, 2 / 6, 3 / 6], atol=1e-15)
    rng = np.random.default_rng(2)
    s = rng.normal(0, 10, size=(9, 33))
    p = O.softmax_rows(s)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
    np.testing.assert_allclose(O.softmax_rows(s + 1234.5), p, atol=1e-12)
    assert np.isfinite(O.softmax_rows(s * 1e3)).all()           # no overflow


# ----------------------------------------------------------------------------- GELU
def test_gelu_values():
    v = np.array([0.0, 1.0, -1.0, 2.0, 8.0, -8.0])
    want = [0.0, 0.8413447460685429, -0.15865525393145707, 1.9544997361036416, 8.0, 0.0]
    np.testing.assert_allclose(O.gelu(v), want, atol=1e-12)
    grid = np.linspace(-6, 6, 2401)
    ref = np.array([0.5 * t * (1.0 + math.erf(t / math.sqrt(2.0))) for t in grid])
    np.testing.assert_allclose(O.gelu(grid), ref, atol=1e-14)


# ----------------------------------------------------------------------------- linear
def test_linear_orientation_and_bias():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(5, 4))
    W = np.zeros((3, 4))
    W[0, 1] = 1.0                          # output 0 reads input 1
    W[2, 3] = -2.0                         # output 2 reads input 3
    b = np.array([10.0, 20.0, 30.0])
    y = O.linear(x, W, b)
    np.testing.assert_allclose(y[:, 0], x[:, 1] + 10.0)
    np.testing.assert_allclose(y[:, 1], 20.0)
    np.testing.assert_allclose(y[:, 2], -2.0 * x[:, 3] + 30.0)
    np.testing.assert_allclose(O.linear(x, np.eye(4), np.zeros(4)), x)


# ----------------------------------------------------------------------------- attention
def test_attention_identical_keys_gives_mean_of_values():
    rng = np.random.default_rng(4)
    T, d = 11, 4
    q = rng.normal(size=(T, d))
    k = np.tile(rng.normal(size=(1, d)), (T, 1))
    v = rng.normal(size=(T, d))
    out = O.attention_head(q, k, v)
    np.testing.assert_allclose(out, np.tile(v.mean(0), (T, 1)), atol=1e-12)


def test_attention_one_hot_selects_value_row_and_single_token():
    rng = np.random.default_rng(5)
    T, d = 6, 8
    k = np.eye(T, d)
    sel = np.array([3, 0, 5, 1, 1, 2])
    q = 1e4 * np.eye(T, d)[sel]
    v = rng.normal(size=(T, d))
    np.testing.assert_allclose(O.attention_head(q, k, v), v[sel], atol=1e-9)
    one = rng.normal(size=(1, d))
    np.testing.assert_allclose(O.attention_head(one, one, v[:1]), v[:1], atol=1e-15)


def test_attention_scale_is_one_over_sqrt_d():
    # two keys, logits differ by q.(k0-k1)/sqrt(d) = ln 3  ->  weights 3/4, 1/4
    d = 16
    q = np.zeros((1, d)); q[0, 0] = 1.0
    k = np.zeros((2, d)); k[0, 0] = math.log(3.0) * math.sqrt(d)
    v = np.array([[1.0] + [0.0] * (d - 1), [0.0] * d])
    out = O.attention_head(q, k, v)
    assert abs(out[0, 0] - 0.75) < 1e-12


def test_multihead_column_layout():
    # Q, K, V blocks and per-head column ownership: make head 1's V the only non-zero input.
    T, H, heads = 5, 8, 2
    d = H // heads
    rng = np.random.default_rng(6)
    qkv = np.zeros((T, 3 * H))
    vals = rng.normal(size=(T, d))
    qkv[:, 2 * H + d:2 * H + 2 * d] = vals            # V, head 1
    out = O.attention(qkv, heads)
    np.testing.assert_allclose(out[:, :d], 0.0)
    np.testing.assert_allclose(out[:, d:], np.tile(vals.mean(0), (T, 1)), atol=1e-12)


# ----------------------------------------------------------------------------- layer / stage
def test_layer_is_identity_when_output_projections_vanish():
    cfg = TINY
    p = _rand_params(cfg, 7)
    for l in range(cfg.layers):
        for n in ("Wo", "bo", "W2", "b2"):
            p[f"l{l}.{n}"] = np.zeros_like(p[f"l{l}.{n}"])
    x = np.random.default_rng(8).normal(size=(3, cfg.tokens, cfg.hidden))
    np.testing.assert_array_equal(O.run_stage(p, cfg, 0, cfg.layers, x), x)


def test_stage_range_errors():
    cfg = TINY
    p = _rand_params(cfg, 7)
    x = np.zeros((1, cfg.tokens, cfg.hidden))
    for lb, le in [(0, 0), (1, 1), (-1, 1), (0, 3), (2, 1)]:
        with pytest.raises(ValueError):
            O.run_stage(p, cfg, lb, le, x)


@pytest.mark.parametrize("dtype", [np.float64, np.float32])
def test_stage_composition_is_bit_exact_for_every_split(dtype):
    # Section 3.1: Y = T_k(...T_1(X)), sum l_i = L, for any partition.
    cfg = vitgen.ViTConfig(image_size=32, patch_size=8, hidden=32, layers=6, heads=4, mlp_dim=64,
                           num_classes=10)
    p, _ = vitgen.make_params(cfg, seed=3, bf16=False, ln_affine=True)
    pix = vitgen.make_pixels(cfg, 2, seed=3)
    x0 = O.patch_embed(p, cfg, pix, dtype)
    whole = O.run_stage(p, cfg, 0, cfg.layers, x0, dtype)
    assert whole.dtype == dtype
    for k in range(1, cfg.layers):
        a = O.run_stage(p, cfg, 0, k, x0, dtype)
        b = O.run_stage(p, cfg, k, cfg.layers, a, dtype)
        assert np.array_equal(whole, b), k
    parts = [(0, 1), (1, 2), (2, 4), (4, 5), (5, 6)]
    np.testing.assert_array_equal(O.forward(p, cfg, pix, parts, dtype), O.head(p, cfg, whole, dtype))


def test_image_result_is_independent_of_its_batch():
    cfg = vitgen.ViTConfig(image_size=32, patch_size=8, hidden=32, layers=2, heads=4, mlp_dim=64,
                           num_classes=10)
    p, _ = vitgen.make_params(cfg, seed=4, bf16=False)
    pix = vitgen.make_pixels(cfg, 3, seed=4)
    full = O.forward(p, cfg, pix)
    for b in range(3):
        assert np.array_equal(full[b:b + 1], O.forward(p, cfg, pix[b:b + 1]))


def test_float32_oracle_agrees_with_float64():
    cfg = vitgen.preset("tiny16").with_(layers=3)
    p, _ = vitgen.make_params(cfg, seed=0, bf16=False)
    pix = vitgen.make_pixels(cfg, 1, seed=0)
    a = O.forward(p, cfg, pix, dtype=np.float64)
    b = O.forward(p, cfg, pix, dtype=np.float32)
    assert np.abs(a - b).max() <= 1e-5 * np.abs(a).max()


# ----------------------------------------------------------------------------- patch embed
def test_patch_embed_flatten_and_token_order():
    cfg = vitgen.ViTConfig(image_size=6, patch_size=2, channels=3, hidden=4, layers=1, heads=1,
                           mlp_dim=4, num_classes=2)
    G, P = cfg.grid, cfg.patch_size
    # pixel value encodes its own coordinates
    img = np.zeros((1, 3, 6, 6))
    for c in range(3):
        for yy in range(6):
            for xx in range(6):
                img[0, c, yy, xx] = 100 * c + 10 * yy + xx
    p = _rand_params(cfg, 9)
    p["patch.W"] = np.zeros_like(p["patch.W"])
    probes = [(0, 0, 0), (1, 1, 0), (2, 0, 1), (1, 1, 1)]       # (c, i, j) per output feature
    for o, (c, i, j) in enumerate(probes):
        p["patch.W"][o, c * P * P + i * P + j] = 1.0
    x = O.patch_embed(p, cfg, img)
    np.testing.assert_allclose(x[0, 0], p["cls"] + p["pos"][0])
    for py in range(G):
        for px in range(G):
            t = 1 + py * G + px
            for o, (c, i, j) in enumerate(probes):
                want = 100 * c + 10 * (py * P + i) + (px * P + j) + p["patch.b"][o] + p["pos"][t, o]
                assert abs(x[0, t, o] - want) < 1e-12
    # zero weights: tokens are bias + position only
    p["patch.W"][:] = 0
    x = O.patch_embed(p, cfg, img)
    np.testing.assert_allclose(x[0, 1:], p["patch.b"] + p["pos"][1:], atol=1e-15)


def test_head_reads_class_token_only():
    cfg = TINY
    p = _rand_params(cfg, 10)
    rng = np.random.default_rng(11)
    x = rng.normal(size=(2, cfg.tokens, cfg.hidden))
    a = O.head(p, cfg, x)
    x2 = x.copy()
    x2[:, 1:] = rng.normal(size=x2[:, 1:].shape)
    np.testing.assert_array_equal(a, O.head(p, cfg, x2))
    f = O.layernorm(x[:, 0], p["lnf.g"], p["lnf.b"], cfg.ln_eps)
    np.testing.assert_allclose(a, f @ p["head.W"].T + p["head.b"], atol=1e-12)


# ----------------------------------------------------------------------------- brute force
def _scalar_vit(p, cfg, img):
    """Literal index-by-index evaluation in Python floats, written separately from the oracle."""
    P, G, H, F, T = cfg.patch_size, cfg.grid, cfg.hidden, cfg.mlp_dim, cfg.tokens
    nh, d, eps = cfg.heads, cfg.head_dim, cfg.ln_eps
    x = [[0.0] * H for _ in range(T)]
    for o in range(H):
        x[0][o] = float(p["cls"][o] + p["pos"][0][o])
    first = 1
    if cfg.extra_tokens:                       # distillation token right after the class token
        first = 2
        for o in range(H):
            x[1][o] = float(p["dist"][o] + p["pos"][1][o])
    for py in range(G):
        for px in range(G):
            t = first + py * G + px
            for o in range(H):
                acc = 0.0
                for c in range(cfg.channels):
                    for i in range(P):
                        for j in range(P):
                            acc += float(p["patch.W"][o][c * P * P + i * P + j]) * float(img[c][py * P + i][px * P + j])
                x[t][o] = acc + float(p["patch.b"][o]) + float(p["pos"][t][o])

    def ln(row, g, b):
        mu = sum(row) / len(row)
        var = sum((r - mu) ** 2 for r in row) / len(row)
        return [(r - mu) / math.sqrt(var + eps) * float(g[i]) + float(b[i]) for i, r in enumerate(row)]

    def lin(row, W, b):
        return [sum(float(W[o][i]) * row[i] for i in range(len(row))) + float(b[o]) for o in range(len(b))]

    for l in range(cfg.layers):
        q = lambda n: p[f"l{l}.{n}"]
        qkv = [lin(ln(x[t], q("ln1.g"), q("ln1.b")), q("Wqkv"), q("bqkv")) for t in range(T)]
        a = [[0.0] * H for _ in range(T)]
        for h in range(nh):
            for t in range(T):
                s = [sum(qkv[t][h * d + e] * qkv[u][H + h * d + e] for e in range(d)) / math.sqrt(d)
                     for u in range(T)]
                m = max(s)
                w = [math.exp(v - m) for v in s]
                z = sum(w)
                for e in range(d):
                    a[t][h * d + e] = sum(w[u] / z * qkv[u][2 * H + h * d + e] for u in range(T))
        for t in range(T):
            o = lin(a[t], q("Wo"), q("bo"))
            x[t] = [x[t][i] + o[i] for i in range(H)]
        for t in range(T):
            u1 = lin(ln(x[t], q("ln2.g"), q("ln2.b")), q("W1"), q("b1"))
            u1 = [0.5 * v * (1.0 + math.erf(v / math.sqrt(2.0))) for v in u1]
            o = lin(u1, q("W2"), q("b2"))
            x[t] = [x[t][i] + o[i] for i in range(H)]
    f = ln(x[0], p["lnf.g"], p["lnf.b"])
    logits = lin(f, p["head.W"], p["head.b"])
    if cfg.extra_tokens:                       # mean of the class-token and distillation-token classifiers
        fd = ln(x[1], p["lnf.g"], p["lnf.b"])
        ld = lin(fd, p["head_dist.W"], p["head_dist.b"])
        logits = [(u + v) / 2.0 for u, v in zip(logits, ld)]
    return logits, x


def test_brute_force_scalar_model_2_layers_5_tokens():
    cfg = TINY
    assert cfg.tokens == 5 and cfg.layers == 2
    p = _rand_params(cfg, 12)
    pix = np.random.default_rng(13).uniform(-1, 1, size=(2, 3, 4, 4))
    got = O.forward(p, cfg, pix)
    tokens = O.run_stage(p, cfg, 0, 2, O.patch_embed(p, cfg, pix))
    for n in range(2):
        logits, x = _scalar_vit(p, cfg, pix[n])
        np.testing.assert_allclose(got[n], logits, rtol=0, atol=1e-5 * max(abs(v) for v in logits))
        np.testing.assert_allclose(tokens[n], np.array(x), rtol=0, atol=1e-10)


# ----------------------------------------------------------------------------- distillation token
DIST = TINY.with_(extra_tokens=1)


def test_distillation_token_inventory_and_count():
    # one more token, one more position row, a second classifier
    assert DIST.tokens == TINY.tokens + 1 and DIST.first_patch_token == 2
    H, C = DIST.hidden, DIST.num_classes
    assert vitgen.param_count(DIST) - vitgen.param_count(TINY) == H + H + C * H + C
    names = [n for n, _, _ in vitgen.param_specs(DIST)]
    assert names.index("dist") == names.index("cls") + 1 and names[-2:] == ["head_dist.W", "head_dist.b"]
    # the distilled small / base shapes: 198 tokens
    assert vitgen.preset("deit_small16").tokens == 198 and vitgen.preset("deit_base16").tokens == 198


def test_distillation_token_order_and_special_rows():
    """Zero patch weights: token 0 = cls + pos[0], token 1 = dist + pos[1], patch tokens start at 2
    and carry patch.b + pos[t].  A one-hot patch weight reads back the pixel that encodes its own
    (patch, channel, row, column), which pins the flatten and token order with the extra token."""
    cfg = DIST
    p = _rand_params(cfg, 3)
    p["patch.W"] = np.zeros_like(p["patch.W"])
    pix = np.random.default_rng(4).uniform(-1, 1, size=(1, 3, 4, 4))
    x = O.patch_embed(p, cfg, pix)[0]
    np.testing.assert_allclose(x[0], p["cls"] + p["pos"][0], atol=1e-12)
    np.testing.assert_allclose(x[1], p["dist"] + p["pos"][1], atol=1e-12)
    for t in range(2, cfg.tokens):
        np.testing.assert_allclose(x[t], p["patch.b"] + p["pos"][t], atol=1e-12)
    P, G = cfg.patch_size, cfg.grid
    img = np.zeros((1, 3, 4, 4))
    for c in range(3):
        for r in range(4):
            for q in range(4):
                img[0, c, r, q] = 1000 * ((r // P) * G + q // P) + 100 * c + 10 * (r % P) + (q % P)
    c, i, j = 2, 1, 0
    p["patch.W"][5, c * P * P + i * P + j] = 1.0
    p["patch.b"] = np.zeros_like(p["patch.b"])
    p["pos"] = np.zeros_like(p["pos"])
    x = O.patch_embed(p, cfg, img)[0]
    for patch in range(G * G):
        assert x[2 + patch, 5] == 1000 * patch + 100 * c + 10 * i + j


def test_distillation_head_is_the_mean_of_two_classifiers():
    cfg = DIST
    p = _rand_params(cfg, 5)
    rng = np.random.default_rng(6)
    x = rng.normal(size=(2, cfg.tokens, cfg.hidden))
    plain = TINY
    on_cls = O.head({k: p[k] for k in ("lnf.g", "lnf.b", "head.W", "head.b")}, plain, x[:, [0] + list(range(2, cfg.tokens))])
    swapped = dict(p)
    q = {"lnf.g": p["lnf.g"], "lnf.b": p["lnf.b"], "head.W": p["head_dist.W"], "head.b": p["head_dist.b"]}
    on_dist = O.head(q, plain, x[:, 1:])            # row 1 presented as "row 0" to the plain head
    np.testing.assert_allclose(O.head(p, cfg, x), (on_cls + on_dist) / 2, atol=1e-12)
    # rows other than 0 and 1 do not matter
    y = x.copy()
    y[:, 2:] = rng.normal(size=y[:, 2:].shape)
    np.testing.assert_allclose(O.head(p, cfg, y), O.head(p, cfg, x), atol=0)


def test_brute_force_scalar_model_with_distillation_token():
    cfg = DIST
    assert cfg.tokens == 6
    p = _rand_params(cfg, 21)
    pix = np.random.default_rng(22).uniform(-1, 1, size=(2, 3, 4, 4))
    got = O.forward(p, cfg, pix)
    tokens = O.run_stage(p, cfg, 0, 2, O.patch_embed(p, cfg, pix))
    for n in range(2):
        logits, x = _scalar_vit(p, cfg, pix[n])
        np.testing.assert_allclose(got[n], logits, rtol=0, atol=1e-5 * max(abs(v) for v in logits))
        np.testing.assert_allclose(tokens[n], np.array(x), rtol=0, atol=1e-10)
