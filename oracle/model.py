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


def dense_tensor_names(cfg):
    """The un-quantised tensors that joint SPSA also perturbs and updates, in index order:
    (key, layer or None).  Embedding and lm_head matrices, then every norm gain (and norm bias, OPT)."""
    opt = cfg["arch"] == "opt"
    names = [("embed", None), ("lm_head", None)]
    for li in range(cfg["n_layers"]):
        names.append(("norm1_w", li))
        if opt:
            names.append(("norm1_b", li))
        names.append(("norm2_w", li))
        if opt:
            names.append(("norm2_b", li))
    names.append(("final_norm_w", None))
    if opt:
        names.append(("final_norm_b", None))
    return names


def dense_tensor(model, key, layer):
    return model[key] if layer is None else model["layers"][layer][key]


def dense_index_bases(cfg):
    """Logical indices of the un-quantised tensors under joint SPSA: they follow the scales in the same
    z(seed, index) stream (so one seed still regenerates every direction), each base rounded up to a
    multiple of 8.  Returns ({(key, layer): base}, total)."""
    _, run = scale_index_bases(cfg)
    d, V = cfg["d_model"], cfg["vocab"]
    out = {}
    for key, layer in dense_tensor_names(cfg):
        run = (run + 7) // 8 * 8
        out[(key, layer)] = run
        run += V * d if key in ("embed", "lm_head") else d
    return out, run


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


def forward_loss(model, tokens, labels, seed, sign, eps, capture=None, perturb_scales=True,
                 perturb_dense=False):
    """L(Delta' (.) theta_bar; B) with Delta' = Delta + sign*eps*z(seed).

    perturb_dense: joint mode (Sec. 3.2.1, closing remark; Sec. 4.1): the un-quantised tensors
    of dense_tensor_names are perturbed as well, theta' = theta + sign*eps*z (plain SPSA,
    Def. 3.1), with z from the same seed at the indices of dense_index_bases.
    perturb_scales=False leaves the scales alone (used to pin the dense part by itself).

    capture: optional dict filled with 'hidden' (list, output of every block,
    [T][d]) and 'logits' ([T][V]) for per-layer parity checks.
    """
    from . import philox
    cfg = model["cfg"]
    tokens = np.asarray(tokens)
    B, S = tokens.shape
    d, H = cfg["d_model"], cfg["n_heads"]
    dh = d // H
    bases, _ = scale_index_bases(cfg)
    dbases, _ = dense_index_bases(cfg)
    scale_sign = sign if perturb_scales else 0

    def dense(key, layer=None):
        """theta or theta + sign*eps*z of one un-quantised tensor, fp64."""
        t = np.asarray(dense_tensor(model, key, layer), dtype=np.float64)
        if not perturb_dense or sign == 0:
            return t
        z = philox.normal_range(seed, dbases[(key, layer)], t.size).astype(np.float64).reshape(t.shape)
        return t + float(sign) * float(eps) * z          # Def. 3.1 (same as qzo.spsa_perturbed)

    x = dense("embed")[tokens.reshape(-1)]
    if cfg["arch"] == "opt":
        pos = np.asarray(model["pos_embed"], dtype=np.float64)[:S]
        x = (x.reshape(B, S, d) + pos[None]).reshape(B * S, d)

    def lin(layer, li, name, inp):
        p = layer["lin"][name]
        return perturbed_linear(inp, p["q"], p["s"], seed, bases[li][name], scale_sign, eps,
                                p.get("bias"))

    for li, layer in enumerate(model["layers"]):
        if cfg["arch"] == "llama":
            n1 = rmsnorm(x, dense("norm1_w", li), cfg["norm_eps"])
        else:
            n1 = layernorm(x, dense("norm1_w", li), dense("norm1_b", li), cfg["norm_eps"])
        qh = lin(layer, li, "q", n1).reshape(B, S, H, dh)
        kh = lin(layer, li, "k", n1).reshape(B, S, H, dh)
        vh = lin(layer, li, "v", n1).reshape(B, S, H, dh)
        if cfg["arch"] == "llama":
            qh, kh = rope(qh, cfg["rope_theta"]), rope(kh, cfg["rope_theta"])
        att = causal_attention(qh, kh, vh).reshape(B * S, d)
        h = x + lin(layer, li, "o", att)
        if cfg["arch"] == "llama":
            n2 = rmsnorm(h, dense("norm2_w", li), cfg["norm_eps"])
            g = lin(layer, li, "gate", n2)
            u = lin(layer, li, "up", n2)
            act = g / (1.0 + np.exp(-g)) * u
            x = h + lin(layer, li, "down", act)
        else:
            n2 = layernorm(h, dense("norm2_w", li), dense("norm2_b", li), cfg["norm_eps"])
            act = np.maximum(lin(layer, li, "fc1", n2), 0.0)
            x = h + lin(layer, li, "fc2", act)
        if capture is not None:
            capture.setdefault("hidden", []).append(x.copy())
    if cfg["arch"] == "llama":
        xn = rmsnorm(x, dense("final_norm_w"), cfg["norm_eps"])
    else:
        xn = layernorm(x, dense("final_norm_w"), dense("final_norm_b"), cfg["norm_eps"])
    logits = xn @ dense("lm_head").T
    if capture is not None:
        capture["logits"] = logits
    return cross_entropy(logits, labels)
