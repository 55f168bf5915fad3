"""Test-side glue: turn the seeded raw tensors into an oracle model (numpy)."""
import copy

import numpy as np

from oracle import int4


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
