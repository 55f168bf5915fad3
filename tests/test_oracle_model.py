"""Pins for oracle/model.py: textbook special cases, library routines as independent
implementations (torch / transformers on CPU in fp64), and the scale inventory of Table 2."""
import os

import numpy as np
import pytest
import torch

from oracle import int4, model as omodel
from paper_2505_13430_b200 import inputs
from tests.helpers import build_oracle_model

GOLD = os.path.join(os.path.dirname(__file__), "golden", "table2_trainable_params.txt")


def test_table2_scale_inventory():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    for name, printed, exact in rows:
        n = omodel.num_trainable_scales(inputs.model_cfg(name))
        assert n == int(exact)
        assert f"{n:.2e}".replace("e+0", "e") == printed
    assert omodel.num_trainable_scales(inputs.model_cfg("llama13b")) == 99_123_200
    assert omodel.num_trainable_scales(inputs.model_cfg("tiny")) == 12_672
    bases, total = omodel.scale_index_bases(inputs.model_cfg("tiny"))
    assert total == 12_672 and bases[0]["q"] == 0 and bases[0]["k"] == 512
    assert all(b % 8 == 0 for row in bases for b in row.values())


def test_norms_against_torch():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((7, 48))
    w, b = rng.standard_normal(48), rng.standard_normal(48)
    tx = torch.from_numpy(x)
    ref = torch.nn.functional.layer_norm(tx, (48,), torch.from_numpy(w), torch.from_numpy(b), 1e-5)
    np.testing.assert_allclose(omodel.layernorm(x, w, b, 1e-5), ref.numpy(), rtol=1e-12, atol=1e-12)
    ref = torch.nn.functional.rms_norm(tx, (48,), torch.from_numpy(w), 1e-5)
    np.testing.assert_allclose(omodel.rmsnorm(x, w, 1e-5), ref.numpy(), rtol=1e-12, atol=1e-12)
    y = omodel.rmsnorm(x, np.ones(48), 0.0)
    np.testing.assert_allclose((y * y).mean(-1), 1.0, rtol=1e-12)


def test_attention_against_torch_and_special_cases():
    rng = np.random.default_rng(1)
    q, k, v = (rng.standard_normal((2, 9, 3, 16)) for _ in range(3))
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(omodel.causal_attention(q, k, v), ref.permute(0, 2, 1, 3).numpy(),
                               rtol=1e-10, atol=1e-12)
    # S = 1: identity on V; first position of any sequence: its own V
    np.testing.assert_allclose(omodel.causal_attention(q[:, :1], k[:, :1], v[:, :1]), v[:, :1])
    np.testing.assert_allclose(omodel.causal_attention(q, k, v)[:, 0], v[:, 0], rtol=1e-12)
    # causality: a change in the last key/value leaves earlier outputs alone
    k2, v2 = k.copy(), v.copy()
    k2[:, -1] += 1.0
    v2[:, -1] -= 2.0
    a, b = omodel.causal_attention(q, k, v), omodel.causal_attention(q, k2, v2)
    assert np.array_equal(a[:, :-1], b[:, :-1]) and not np.allclose(a[:, -1], b[:, -1])


def test_rope_properties():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((1, 12, 2, 8))
    y = omodel.rope(x, 10000.0)
    np.testing.assert_allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    np.testing.assert_allclose(y[:, 0], x[:, 0])                  # position 0 unrotated
    # relative: <rope(q)_m, rope(k)_n> depends on m - n only
    qv, kv = rng.standard_normal(8), rng.standard_normal(8)
    qs = omodel.rope(np.broadcast_to(qv, (1, 12, 1, 8)).copy(), 10000.0)[0, :, 0]
    ks = omodel.rope(np.broadcast_to(kv, (1, 12, 1, 8)).copy(), 10000.0)[0, :, 0]
    assert abs(qs[5] @ ks[3] - qs[9] @ ks[7]) < 1e-12
    assert abs(qs[5] @ ks[3] - qs[5] @ ks[4]) > 1e-6
    # pair (i, i + dh/2), first pair rotates by pos * 1 rad
    e = np.zeros((1, 3, 1, 8)); e[..., 0] = 1.0
    r = omodel.rope(e, 10000.0)[0, :, 0]
    np.testing.assert_allclose(r[2, 0], np.cos(2.0)); np.testing.assert_allclose(r[2, 4], np.sin(2.0))


def test_cross_entropy_against_torch_and_ln_v():
    rng = np.random.default_rng(3)
    logits = rng.standard_normal((10, 33)) * 3
    labels = rng.integers(0, 33, size=10); labels[[2, 7]] = -100
    ref = torch.nn.functional.cross_entropy(torch.from_numpy(logits), torch.from_numpy(labels).long(),
                                            ignore_index=-100)
    assert abs(omodel.cross_entropy(logits, labels) - float(ref)) < 1e-12
    assert abs(omodel.cross_entropy(np.zeros((4, 1024)), np.array([1, 2, 3, 4])) - np.log(1024)) < 1e-14


def _tiny_raw(arch):
    name = "tiny" if arch == "llama" else "tiny_opt"
    cfg = inputs.model_cfg(name, n_layers=2, d_model=64, n_heads=4,
                           d_ffn=176 if arch == "llama" else 256, vocab=128, max_seq=16)
    raw = inputs.raw_model_tensors(cfg, seed=11)
    # make norms non-trivial so a dropped gain/bias would show
    g = torch.Generator().manual_seed(5)
    for layer in raw["layers"]:
        for k in list(layer):
            if k.startswith("norm"):
                layer[k] = layer[k] + 0.1 * torch.randn(layer[k].shape, generator=g)
    raw["final_norm_w"] = raw["final_norm_w"] + 0.1 * torch.randn(64, generator=g)
    if "final_norm_b" in raw:
        raw["final_norm_b"] = raw["final_norm_b"] + 0.1 * torch.randn(64, generator=g)
    # larger weights so attention and the MLP are far from their linear regime
    for layer in raw["layers"]:
        for ent in layer["lin"].values():
            ent["w"] = ent["w"] * 8.0
    return cfg, raw


def test_zero_head_gives_ln_vocab():
    cfg, raw = _tiny_raw("llama")
    m = build_oracle_model(raw)
    m["lm_head"] = np.zeros_like(m["lm_head"])
    tok, lab = inputs.tokens_and_labels(cfg, 2, 16)
    assert abs(omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, +1, 1e-3) - np.log(128)) < 1e-13


def test_llama_forward_matches_transformers_fp64():
    from transformers import LlamaConfig, LlamaForCausalLM
    cfg, raw = _tiny_raw("llama")
    m = build_oracle_model(raw)
    hc = LlamaConfig(vocab_size=128, hidden_size=64, intermediate_size=176, num_hidden_layers=2,
                     num_attention_heads=4, num_key_value_heads=4, max_position_embeddings=16,
                     rms_norm_eps=cfg["norm_eps"], rope_theta=cfg["rope_theta"], attention_bias=False,
                     tie_word_embeddings=False, attn_implementation="eager")
    hf = LlamaForCausalLM(hc).double().eval()
    sd = {"model.embed_tokens.weight": m["embed"], "lm_head.weight": m["lm_head"],
          "model.norm.weight": m["final_norm_w"]}
    names = {"q": "self_attn.q_proj", "k": "self_attn.k_proj", "v": "self_attn.v_proj",
             "o": "self_attn.o_proj", "gate": "mlp.gate_proj", "up": "mlp.up_proj", "down": "mlp.down_proj"}
    for li, layer in enumerate(m["layers"]):
        sd[f"model.layers.{li}.input_layernorm.weight"] = layer["norm1_w"]
        sd[f"model.layers.{li}.post_attention_layernorm.weight"] = layer["norm2_w"]
        for k, hfname in names.items():
            sd[f"model.layers.{li}.{hfname}.weight"] = int4.dequantize(layer["lin"][k]["q"], layer["lin"][k]["s"]).T
    hf.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)).double() for k, v in sd.items()})
    tok, lab = inputs.tokens_and_labels(cfg, 3, 16)
    cap = {}
    loss = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, 0, 1e-3, capture=cap)
    with torch.no_grad():
        out = hf(input_ids=tok.long(), output_hidden_states=True)
    # the library builds its rotary tables in fp32, hence 1e-6 rather than fp64 rounding
    np.testing.assert_allclose(cap["logits"], out.logits.reshape(-1, 128).numpy(), rtol=2e-6, atol=2e-6)
    np.testing.assert_allclose(cap["hidden"][0], out.hidden_states[1].reshape(-1, 64).numpy(), rtol=2e-6, atol=2e-6)
    ref = torch.nn.functional.cross_entropy(out.logits.reshape(-1, 128), lab.long().reshape(-1), ignore_index=-100)
    assert abs(loss - float(ref)) < 1e-6
    assert abs(loss - np.log(128)) > 1e-3       # the case is not degenerate
    assert np.abs(cap["logits"]).max() > 0.1


def test_opt_forward_matches_transformers_fp64():
    from transformers import OPTConfig, OPTForCausalLM
    cfg, raw = _tiny_raw("opt")
    m = build_oracle_model(raw)
    hc = OPTConfig(vocab_size=128, hidden_size=64, ffn_dim=256, num_hidden_layers=2, num_attention_heads=4,
                   max_position_embeddings=16, word_embed_proj_dim=64, do_layer_norm_before=True,
                   tie_word_embeddings=False, activation_function="relu", dropout=0.0,
                   attn_implementation="eager")
    hf = OPTForCausalLM(hc).double().eval()
    pos = np.zeros((18, 64)); pos[2:] = m["pos_embed"]          # the library keeps two unused leading rows
    sd = {"model.decoder.embed_tokens.weight": m["embed"], "lm_head.weight": m["lm_head"],
          "model.decoder.embed_positions.weight": pos,
          "model.decoder.final_layer_norm.weight": m["final_norm_w"],
          "model.decoder.final_layer_norm.bias": m["final_norm_b"]}
    names = {"q": "self_attn.q_proj", "k": "self_attn.k_proj", "v": "self_attn.v_proj",
             "o": "self_attn.out_proj", "fc1": "fc1", "fc2": "fc2"}
    for li, layer in enumerate(m["layers"]):
        p = f"model.decoder.layers.{li}."
        sd[p + "self_attn_layer_norm.weight"] = layer["norm1_w"]; sd[p + "self_attn_layer_norm.bias"] = layer["norm1_b"]
        sd[p + "final_layer_norm.weight"] = layer["norm2_w"]; sd[p + "final_layer_norm.bias"] = layer["norm2_b"]
        for k, hfname in names.items():
            sd[p + hfname + ".weight"] = int4.dequantize(layer["lin"][k]["q"], layer["lin"][k]["s"]).T
            sd[p + hfname + ".bias"] = layer["lin"][k]["bias"]
    hf.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)).double() for k, v in sd.items()})
    tok, lab = inputs.tokens_and_labels(cfg, 3, 16)
    cap = {}
    loss = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, 0, 1e-3, capture=cap)
    with torch.no_grad():
        out = hf(input_ids=tok.long())
    # the library's eager attention takes its softmax in fp32, hence 1e-6
    np.testing.assert_allclose(cap["logits"], out.logits.reshape(-1, 128).numpy(), rtol=2e-6, atol=2e-6)
    ref = torch.nn.functional.cross_entropy(out.logits.reshape(-1, 128), lab.long().reshape(-1), ignore_index=-100)
    assert abs(loss - float(ref)) < 1e-6
    assert np.abs(cap["logits"]).max() > 0.1


def test_perturbation_changes_loss_and_sign_zero_ignores_seed():
    cfg, raw = _tiny_raw("llama")
    m = build_oracle_model(raw)
    tok, lab = inputs.tokens_and_labels(cfg, 2, 16)
    l0a = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, 0, 1e-3)
    l0b = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 2, 0, 1e-3)
    lp = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, +1, 1e-3)
    lm = omodel.forward_loss(m, tok.numpy(), lab.numpy(), 1, -1, 1e-3)
    assert l0a == l0b and lp != lm and abs(0.5 * (lp + lm) - l0a) < 1e-3
