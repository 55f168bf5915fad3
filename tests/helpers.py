"""Test-side glue: turn the seeded raw tensors into an oracle model (numpy)."""
import copy

import numpy as np

from oracle import int4, linear as olinear, model as omodel


def f32(t):
    return t.float().numpy() if hasattr(t, "numpy") else np.asarray(t, dtype=np.float32)


def build_oracle_model(raw):
    """Quantise every block linear with the oracle's quantiser (Eq. 3)."""
    m = {"cfg": dict(raw["cfg"]), "embed": f32(raw["embed"]), "lm_head": f32(raw["lm_head"]),
         "final_norm_w": f32(raw["final_norm_w"])}
    if "pos_embed" in raw:
        m["pos_embed"] = f32(raw["pos_embed"])
    if "final_norm_b" in raw:
        m["final_norm_b"] = f32(raw["final_norm_b"])
    layers = []
    for layer in raw["layers"]:
        out = {k: f32(v) for k, v in layer.items() if k != "lin"}
        out["lin"] = {}
        for name, ent in layer["lin"].items():
            q, s = int4.quantize_int4(f32(ent["w"]))
            o = {"q": q, "s": s}
            if "bias" in ent:
                o["bias"] = f32(ent["bias"])
            out["lin"][name] = o
        layers.append(out)
    m["layers"] = layers
    return m


def clone_model(m):
    return copy.deepcopy(m)


def llama_forward_with_bf16_storage(model, tokens, seed, sign, eps):
    """The oracle's Llama forward (fp64 arithmetic, same functions) with every tensor that a 16-bit
    implementation keeps in memory rounded to bf16 where it is stored: the de-quantised weight s' q, the
    norm outputs, every linear's output, the rotated q and k, the attention output, the activation and the
    residual stream.  It answers one question: how far does bf16 STORAGE alone move a block's output away
    from the un-rounded oracle?  Where that already exceeds the 2e-2 bound (strongly non-linear models),
    the parity test bounds the GPU by this figure instead.  Returns (hidden per block, logits)."""
    cfg = model["cfg"]
    assert cfg["arch"] == "llama"
    B, S = tokens.shape
    d, H = cfg["d_model"], cfg["n_heads"]
    dh = d // H
    bases, _ = omodel.scale_index_bases(cfg)
    bf = lambda a: int4.bf16_round(np.asarray(a, dtype=np.float32)).astype(np.float64)
    x = np.asarray(model["embed"], np.float64)[tokens.reshape(-1)]

    def lin(layer, li, name, inp):
        p = layer["lin"][name]
        sp = olinear.perturbed_scales(p["s"], seed, bases[li][name], sign, eps)
        w = bf(sp[np.arange(p["q"].shape[0]) // int4.GROUP] * p["q"].astype(np.float64))
        return bf(inp @ w)

    hidden = []
    for li, layer in enumerate(model["layers"]):
        n1 = bf(omodel.rmsnorm(x, np.asarray(layer["norm1_w"], np.float64), cfg["norm_eps"]))
        qh = bf(omodel.rope(lin(layer, li, "q", n1).reshape(B, S, H, dh), cfg["rope_theta"]))
        kh = bf(omodel.rope(lin(layer, li, "k", n1).reshape(B, S, H, dh), cfg["rope_theta"]))
        vh = lin(layer, li, "v", n1).reshape(B, S, H, dh)
        att = bf(omodel.causal_attention(qh, kh, vh).reshape(B * S, d))
        h = bf(x + lin(layer, li, "o", att))
        n2 = bf(omodel.rmsnorm(h, np.asarray(layer["norm2_w"], np.float64), cfg["norm_eps"]))
        g, u = lin(layer, li, "gate", n2), lin(layer, li, "up", n2)
        act = bf(g / (1.0 + np.exp(-g)) * u)
        x = bf(h + lin(layer, li, "down", act))
        hidden.append(x.copy())
    xn = bf(omodel.rmsnorm(x, np.asarray(model["final_norm_w"], np.float64), cfg["norm_eps"]))
    return hidden, xn @ np.asarray(model["lm_head"], dtype=np.float64).T


def loss_tolerance(kept_tokens):
    """Bound on |L_gpu - L_oracle| for a mean over `kept_tokens` positions.  The 1e-3 of the method's
    configurations is stated for their batches (the smallest keeps 188 positions), where the bf16 rounding
    errors of the single tokens' losses (a few 1e-3 each, independent from token to token) average out; a
    mean over fewer positions averages fewer of them, so the bound widens by sqrt(188 / kept)."""
    return 1e-3 * max(1.0, (188.0 / max(int(kept_tokens), 1)) ** 0.5)
