"""Decoder-only LM forward with int4 linears and perturbed scales (oracle, fp64).

The paper treats the model as a black-box loss L(Delta (.) theta_bar; B)
(Eq. 5, Algorithm 1) whose de-quantisation is part of the ordinary forward
pass (Sec. 3.2.1).  The two model families below are the textbook definitions
of the architectures the paper fine-tunes (Llama-2 and OPT, Sec. 4.1); only the
decoder-block linears are int4 with trainable scales, which is what reproduces
the trainable-parameter counts of Table 2 (block linear weights / 128);
embeddings, lm_head, norms and biases are 16-bit and frozen.

Full-model loss values: parity unpinned by the paper (it prints no worked
example).  What is pinned here: zero block weights give loss = ln(V); S = 1
attention is the identity on V; RoPE keeps norms and is relative; the scale
inventory matches Table 2.

A model is a dict:
  cfg     dict(arch='llama'|'opt', n_layers, d_model, n_heads, d_ffn, vocab,
               max_seq, norm_eps, rope_theta)
  embed   [V][d]            pos_embed [max_seq][d] (opt only)
  layers  list of dict(norm1_w, norm2_w [, norm1_b, norm2_b],
                       lin = {name: dict(q int8[K][N], s [G][N] [, bias [N]])})
  final_norm_w [, final_norm_b],  lm_head [V][d]
"""
import numpy as np
from .int4 import GROUP, num_groups
from .linear import perturbed_linear

LINEAR_ORDER = {
    "llama": ("q", "k", "v", "o", "gate", "up", "down"),
    "opt": ("q", "k", "v", "o", "fc1", "fc2"),
}
IGNORE_INDEX = -100


def linear_shapes(cfg):
    """(name, K, N) of the int4 linears of one decoder block, in index order."""
    d, f = cfg["d_model"], cfg["d_ffn"]
    if cfg["arch"] == "llama":
        return [("q", d, d), ("k", d, d), ("v", d, d), ("o", d, d),
                ("gate", d, f), ("up", d, f), ("down", f, d)]
    return [("q", d, d), ("k", d, d), ("v", d, d), ("o", d, d),
            ("fc1", d, f), ("fc2", f, d)]


def scale_index_bases(cfg):
    """Global logical scale index of the first scale of every linear.

    Linears are enumerated layer by layer in LINEAR_ORDER; each occupies
    G*N consecutive indices (row-major [G][N]); bases are rounded up to a
    multiple of 8.  Returns (bases[layer][name], total).
    """
    bases, run = [], 0
    for _ in range(cfg["n_layers"]):
        row = {}
        for name, K, N in linear_shapes(cfg):
            run = (run + 7) // 8 * 8
            row[name] = run
            run += num_groups(K) * N
        bases.append(row)
    return bases, run


def num_trainable_scales(cfg):
    return sum(num_groups(K) * N for _, K, N in linear_shapes(cfg)) * cfg["n_layers"]


def rmsnorm(x, w, eps):
    return x / np.sqrt(np.mean(x * x, axis=-1, keepdims=True) + eps) * w


def layernorm(x, w, b, eps):
    mu = np.mean(x, axis=-1, keepdims=True)
    var = np.mean((x - mu) ** 2, axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * w + b


def rope(x, theta):
    """x [B][S][H][dh]; rotate pairs (i, i + dh/2) by pos * theta**(-2i/dh)."""
    B, S, H, dh = x.shape
    half = dh // 2
    inv = theta ** (-np.arange(half, dtype=np.float64) * 2.0 / dh)
    ang = np.arange(S, dtype=np.float64)[:, None] * inv[None, :]
    c, s = np.cos(ang)[None, :, None, :], np.sin(ang)[None, :, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def causal_attention(q, k, v):
    """softmax(q k^T / sqrt(dh) + causal mask) v on [B][S][H][dh]."""
    B, S, H, dh = q.shape
    sc = np.einsum("bshd,bthd->bhst", q, k) / np.sqrt(dh)
    mask = np.triu(np.ones((S, S), dtype=bool), k=1)
    sc = np.where(mask[None, None], -np.inf, sc)
    sc = sc - sc.max(axis=-1, keepdims=True)
    p = np.exp(sc)
    p /= p.sum(axis=-1, keepdims=True)
    return np.einsum("bhst,bthd->bshd", p, v)


def cross_entropy(logits, labels):
    """mean over labels != -100 of logsumexp(logits) - logits[label]."""
    labels = np.asarray(labels).reshape(-1)
    logits = logits.reshape(labels.size, -1)
    keep = labels != IGNORE_INDEX
    m = logits.max(axis=-1, keepdims=True)
    lse = (m + np.log(np.exp(logits - m).sum(axis=-1, keepdims=True)))[:, 0]
    picked = logits[np.arange(labels.size), np.where(keep, labels, 0)]
    return float(np.sum((lse - picked)[keep]) / max(int(keep.sum()), 1))


def forward_loss(model, tokens, labels, seed, sign, eps, capture=None):
    """L(Delta' (.) theta_bar; B) with Delta' = Delta + sign*eps*z(seed).

    capture: optional dict filled with 'hidden' (list, output of every block,
    [T][d]) and 'logits' ([T][V]) for per-layer parity checks.
    """
    cfg = model["cfg"]
    tokens = np.asarray(tokens)
    B, S = tokens.shape
    d, H = cfg["d_model"], cfg["n_heads"]
    dh = d // H
    bases, _ = scale_index_bases(cfg)
    x = np.asarray(model["embed"], dtype=np.float64)[tokens.reshape(-1)]
    if cfg["arch"] == "opt":
        pos = np.asarray(model["pos_embed"], dtype=np.float64)[:S]
        x = (x.reshape(B, S, d) + pos[None]).reshape(B * S, d)

    def lin(layer, li, name, inp):
        p = layer["lin"][name]
        return perturbed_linear(inp, p["q"], p["s"], seed, bases[li][name], sign, eps,
                                p.get("bias"))

    for li, layer in enumerate(model["layers"]):
        if cfg["arch"] == "llama":
            n1 = rmsnorm(x, np.asarray(layer["norm1_w"], np.float64), cfg["norm_eps"])
        else:
            n1 = layernorm(x, np.asarray(layer["norm1_w"], np.float64),
                           np.asarray(layer["norm1_b"], np.float64), cfg["norm_eps"])
        qh = lin(layer, li, "q", n1).reshape(B, S, H, dh)
        kh = lin(layer, li, "k", n1).reshape(B, S, H, dh)
        vh = lin(layer, li, "v", n1).reshape(B, S, H, dh)
        if cfg["arch"] == "llama":
            qh, kh = rope(qh, cfg["rope_theta"]), rope(kh, cfg["rope_theta"])
        att = causal_attention(qh, kh, vh).reshape(B * S, d)
        h = x + lin(layer, li, "o", att)
        if cfg["arch"] == "llama":
            n2 = rmsnorm(h, np.asarray(layer["norm2_w"], np.float64), cfg["norm_eps"])
            g = lin(layer, li, "gate", n2)
            u = lin(layer, li, "up", n2)
            act = g / (1.0 + np.exp(-g)) * u
            x = h + lin(layer, li, "down", act)
        else:
            n2 = layernorm(h, np.asarray(layer["norm2_w"], np.float64),
                           np.asarray(layer["norm2_b"], np.float64), cfg["norm_eps"])
            act = np.maximum(lin(layer, li, "fc1", n2), 0.0)
            x = h + lin(layer, li, "fc2", act)
        if capture is not None:
            capture.setdefault("hidden", []).append(x.copy())
    if cfg["arch"] == "llama":
        xn = rmsnorm(x, np.asarray(model["final_norm_w"], np.float64), cfg["norm_eps"])
    else:
        xn = layernorm(x, np.asarray(model["final_norm_w"], np.float64),
                       np.asarray(model["final_norm_b"], np.float64), cfg["norm_eps"])
    logits = xn @ np.asarray(model["lm_head"], dtype=np.float64).T
    if capture is not None:
        capture["logits"] = logits
    return cross_entropy(logits, labels)
