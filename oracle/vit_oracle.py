"""CPU oracle: the forward pass of a pre-LN Vision Transformer, written out plainly.

TEST INFRASTRUCTURE ONLY.  Nothing on the product path imports this file; it exists so that
the CUDA library can be compared against an independent statement of the same function.
It shares no code with the CUDA path.  Parity status: every function below is pinned by the
CPU tests (closed forms, invariants, and a scalar brute-force model), none is unpinned.

What is computed, and where the paper states it:
  * A transformer layer = multi-head self-attention + MLP + two layer normalisations +
    residual connections (Section 2.1, "Transformer-based Models").
  * A pipeline stage T_i = l_i consecutive layers; the model output is
    T_k(...T_2(T_1(X))) with sum(l_i) = L (Section 3.1).  `run_stage(lb, le)` is T_i.
  * An embedding layer precedes the transformer layers and gives every input a uniform
    dimension; the task is image classification, the last stage produces the final result
    (Sections 3.1 and 4).  `patch_embed` and `head` are these two book-ends.
  * The compressed models of Section 5.5 are distilled transformers of the same structure: they
    carry a distillation token beside the class token (cfg.extra_tokens = 1) and a second
    classifier on it; the prediction is the mean of the two classifiers' outputs.
The paper gives no formula for the individual operations; the ones used are the textbook
definitions for a pre-LN ViT and are spelled out in each docstring.

Precision: `dtype` selects the arithmetic (np.float64 by default, np.float32 available).
Images are processed one at a time so that an image's result does not depend on the batch it
is in, and no value is rounded at a stage boundary, so any split of [0, L) into stages gives
bit-identical results to a single call.

Activations are [mb, T, H]; parameters are a dict name -> array, matrices [out, in].
"""
import numpy as np
from scipy.special import erf as _erf


def layernorm(x, g, b, eps):
    """LN(x)_i = (x_i - mu) / sqrt(var + eps) * g_i + b_i over the last axis,
    mu = mean(x), var = mean((x - mu)^2) (biased)."""
    mu = x.mean(axis=-1, keepdims=True)
    xc = x - mu
    var = (xc * xc).mean(axis=-1, keepdims=True)
    return xc / np.sqrt(var + x.dtype.type(eps)) * g + b


def softmax_rows(s):
    """softmax over the last axis: exp(s - rowmax) / sum(exp(s - rowmax))."""
    e = np.exp(s - s.max(axis=-1, keepdims=True))
    return e / e.sum(axis=-1, keepdims=True)


def gelu(v):
    """gelu(v) = 0.5 v (1 + erf(v / sqrt(2)))."""
    return v.dtype.type(0.5) * v * (v.dtype.type(1.0) + _erf(v / np.sqrt(v.dtype.type(2.0))))


def linear(x, W, b):
    """x [rows, in] times W [out, in] transposed, plus b [out]."""
    return x @ W.T + b


def attention_head(q, k, v):
    """One head: S = q k^T / sqrt(d); P = softmax_rows(S); returns P v.  q, k, v are [T, d]."""
    d = q.shape[-1]
    s = (q @ k.T) / np.sqrt(q.dtype.type(d))
    return softmax_rows(s) @ v


def attention(qkv, heads):
    """Multi-head self-attention on one image.  qkv is [T, 3H] with column blocks Q, K, V and,
    inside each block, head h in columns h*d..(h+1)*d.  Returns the concatenated heads [T, H]."""
    T, H3 = qkv.shape
    H = H3 // 3
    d = H // heads
    out = np.empty((T, H), dtype=qkv.dtype)
    for h in range(heads):
        c = slice(h * d, (h + 1) * d)
        out[:, c] = attention_head(qkv[:, :H][:, c], qkv[:, H:2 * H][:, c], qkv[:, 2 * H:][:, c])
    return out


def _cast(params, dtype):
    return {k: np.asarray(v, dtype=dtype) for k, v in params.items()}


def patch_embed(params, cfg, pixels, dtype=np.float64):
    """Embedding book-end.  pixels [mb, C, S, S].  Token t = t0 + py*(S/P) + px is
    patch.W . vec(patch) + patch.b + pos[t], vec ordered (channel, row, column);
    token 0 is cls + pos[0]; with a distillation token, token 1 is dist + pos[1] and t0 = 2
    (otherwise t0 = 1).  Returns [mb, T, H]."""
    names = ("patch.W", "patch.b", "cls", "pos") + (("dist",) if cfg.extra_tokens else ())
    p = _cast({k: params[k] for k in names}, dtype)
    t0 = 1 + cfg.extra_tokens
    P, G = cfg.patch_size, cfg.grid
    mb = pixels.shape[0]
    x = np.empty((mb, cfg.tokens, cfg.hidden), dtype=dtype)
    for n in range(mb):
        img = np.asarray(pixels[n], dtype=dtype)
        x[n, 0] = p["cls"] + p["pos"][0]
        if cfg.extra_tokens:
            x[n, 1] = p["dist"] + p["pos"][1]
        for py in range(G):
            for px in range(G):
                vec = img[:, py * P:(py + 1) * P, px * P:(px + 1) * P].reshape(-1)
                t = t0 + py * G + px
                x[n, t] = p["patch.W"] @ vec + p["patch.b"] + p["pos"][t]
    return x


def layer(params, cfg, l, x):
    """One pre-LN transformer layer on one image, x [T, H]:
       x = x + Wo.attention(LN1(x).Wqkv^T + bqkv) + bo ;  x = x + W2.gelu(W1.LN2(x) + b1) + b2."""
    g = lambda name: params[f"l{l}.{name}"]
    y = layernorm(x, g("ln1.g"), g("ln1.b"), cfg.ln_eps)
    qkv = linear(y, g("Wqkv"), g("bqkv"))
    a = attention(qkv, cfg.heads)
    x = x + linear(a, g("Wo"), g("bo"))
    z = layernorm(x, g("ln2.g"), g("ln2.b"), cfg.ln_eps)
    u = gelu(linear(z, g("W1"), g("b1")))
    return x + linear(u, g("W2"), g("b2"))


def run_stage(params, cfg, layer_begin, layer_end, x, dtype=np.float64):
    """Pipeline stage T_i: layers [layer_begin, layer_end) applied to x [mb, T, H]."""
    if not (0 <= layer_begin < layer_end <= cfg.layers):
        raise ValueError("stage must satisfy 0 <= begin < end <= L")
    x = np.asarray(x, dtype=dtype)
    out = np.empty_like(x)
    for l in range(layer_begin, layer_end):
        pl = _cast({k: v for k, v in params.items() if k.startswith(f"l{l}.")}, dtype)
        src = x if l == layer_begin else out
        for n in range(x.shape[0]):
            out[n] = layer(pl, cfg, l, src[n])
    return out


def head(params, cfg, x, dtype=np.float64):
    """Classification book-end: final LayerNorm of the class token (row 0 of each image),
    then logits = f . head.W^T + head.b.  With a distillation token, row 1 goes through the same
    LayerNorm and its own classifier head_dist, and the result is the mean of the two logit
    vectors.  Returns [mb, classes]."""
    names = ("lnf.g", "lnf.b", "head.W", "head.b") + (("head_dist.W", "head_dist.b") if cfg.extra_tokens else ())
    p = _cast({k: params[k] for k in names}, dtype)
    x = np.asarray(x, dtype=dtype)
    out = np.empty((x.shape[0], cfg.num_classes), dtype=dtype)
    for n in range(x.shape[0]):
        f = layernorm(x[n, 0], p["lnf.g"], p["lnf.b"], cfg.ln_eps)
        out[n] = p["head.W"] @ f + p["head.b"]
        if cfg.extra_tokens:
            fd = layernorm(x[n, 1], p["lnf.g"], p["lnf.b"], cfg.ln_eps)
            out[n] = (out[n] + p["head_dist.W"] @ fd + p["head_dist.b"]) / dtype(2)
    return out


def forward(params, cfg, pixels, stages=None, dtype=np.float64):
    """Whole model: embed, every stage in order, head.  `stages` is [(begin, end)] covering
    [0, L) (default: one stage)."""
    stages = stages or [(0, cfg.layers)]
    x = patch_embed(params, cfg, pixels, dtype)
    for lb, le in stages:
        x = run_stage(params, cfg, lb, le, x, dtype)
    return head(params, cfg, x, dtype)
