"""Pins for the oracle's joint mode (Q-SPSA on the scales combined with plain SPSA on the
un-quantised tensors; Sec. 3.2.1 closing remark, Def. 3.1, Def. 3.2): the exact finite difference on
a quadratic loss, the model's directional derivative against reverse-mode gradients of an
independent implementation, index ranges, and the update's invariants."""
import numpy as np
import torch

from oracle import int4, model as omodel, philox, qzo
from paper_2505_13430_b200 import inputs
from tests.helpers import build_oracle_model, clone_model
from tests.test_oracle_model import _tiny_raw


def test_spsa_finite_difference_is_exact_on_quadratic_loss():
    # Def. 3.1 on Y = X W, L = 0.5 ||Y - T||^2: L is quadratic in W, so the central difference equals
    # z . dL/dW for any eps.
    rng = np.random.default_rng(5)
    x, w, tgt = rng.standard_normal((7, 24)), rng.standard_normal((24, 5)), rng.standard_normal((7, 5))
    seed, base = 31, 40

    def loss(sign, eps):
        return 0.5 * np.sum((x @ qzo.spsa_perturbed(w, seed, base, sign, eps) - tgt) ** 2)

    grad = x.T @ (x @ w - tgt)
    z = philox.normal_range(seed, base, w.size).astype(np.float64).reshape(w.shape)
    want = float(np.sum(z * grad))
    for eps in (1e-3, 1e-2, 0.5):
        assert abs(qzo.directional_derivative(loss(+1, eps), loss(-1, eps), eps) - want) <= 1e-9 * abs(want)
    assert np.array_equal(qzo.spsa_perturbed(w, seed, base, 0, 1e-3), w)


def test_dense_index_ranges_follow_the_scales_and_do_not_overlap():
    for name in ("tiny", "tiny_opt", "llama7b"):
        cfg = inputs.model_cfg(name)
        _, scales_total = omodel.scale_index_bases(cfg)
        bases, total = omodel.dense_index_bases(cfg)
        names = omodel.dense_tensor_names(cfg)
        assert list(bases) == names and names[0] == ("embed", None) and names[1] == ("lm_head", None)
        d, V = cfg["d_model"], cfg["vocab"]
        end = scales_total
        count = 0
        for key in names:
            size = V * d if key[0] in ("embed", "lm_head") else d
            assert bases[key] % 8 == 0 and end <= bases[key] < end + 8
            end = bases[key] + size
            count += size
        assert end == total
        n_vec = (2 * cfg["n_layers"] + 1) * (2 if cfg["arch"] == "opt" else 1)
        assert count == 2 * V * d + n_vec * d


def _hf_llama(m, cfg):
    from transformers import LlamaConfig, LlamaForCausalLM
    hc = LlamaConfig(vocab_size=128, hidden_size=64, intermediate_size=176, num_hidden_layers=2,
                     num_attention_heads=4, num_key_value_heads=4, max_position_embeddings=16,
                     rms_norm_eps=cfg["norm_eps"], rope_theta=cfg["rope_theta"], attention_bias=False,
                     tie_word_embeddings=False, attn_implementation="eager")
    hf = LlamaForCausalLM(hc).double()
    sd = {"model.embed_tokens.weight": m["embed"], "lm_head.weight": m["lm_head"], "model.norm.weight": m["final_norm_w"]}
    names = {"q": "self_attn.q_proj", "k": "self_attn.k_proj", "v": "self_attn.v_proj",
             "o": "self_attn.o_proj", "gate": "mlp.gate_proj", "up": "mlp.up_proj", "down": "mlp.down_proj"}
    for li, layer in enumerate(m["layers"]):
        sd[f"model.layers.{li}.input_layernorm.weight"] = layer["norm1_w"]
        sd[f"model.layers.{li}.post_attention_layernorm.weight"] = layer["norm2_w"]
        for k, hfname in names.items():
            sd[f"model.layers.{li}.{hfname}.weight"] = int4.dequantize(layer["lin"][k]["q"], layer["lin"][k]["s"]).T
    hf.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)).double() for k, v in sd.items()})
    return hf


def test_dense_directional_derivative_matches_reverse_mode_gradients():
    # d/d eps L(theta + eps z) at 0 = z . grad L: the gradient comes from autograd on an independent
    # implementation of the same architecture, z from the oracle's index ranges.  A wrong base, a swapped
    # tensor or a sign error in the joint mode breaks the agreement.
    cfg, raw = _tiny_raw("llama")
    m = build_oracle_model(raw)
    tok, lab = inputs.tokens_and_labels(cfg, 3, 16)
    hf = _hf_llama(m, cfg)
    out = hf(input_ids=tok.long())
    loss = torch.nn.functional.cross_entropy(out.logits.reshape(-1, 128), lab.long().reshape(-1), ignore_index=-100)
    loss.backward()
    grads = {("embed", None): hf.model.embed_tokens.weight.grad, ("lm_head", None): hf.lm_head.weight.grad,
             ("final_norm_w", None): hf.model.norm.weight.grad}
    for li in range(2):
        grads[("norm1_w", li)] = hf.model.layers[li].input_layernorm.weight.grad
        grads[("norm2_w", li)] = hf.model.layers[li].post_attention_layernorm.weight.grad
    seed = 9
    bases, _ = omodel.dense_index_bases(cfg)
    want = 0.0
    for key, g in grads.items():
        z = philox.normal_range(seed, bases[key], g.numel()).astype(np.float64).reshape(tuple(g.shape))
        want += float(np.sum(z * g.numpy()))
    terms = {}
    errs = []
    for eps in (1e-4, 2e-5):
        lp = omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, +1, eps, perturb_scales=False, perturb_dense=True)
        lm = omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, -1, eps, perturb_scales=False, perturb_dense=True)
        errs.append(abs(qzo.directional_derivative(lp, lm, eps) - want))
    # O(eps^2) away (the embeddings are N(0, 0.02), so eps must be small against that), shrinking with eps;
    # the bound is far below the smallest single tensor's share (6e-3), so a tensor perturbed with another
    # one's z does not pass
    assert abs(want) > 1.0
    assert errs[1] <= 5e-4 and 10.0 < errs[0] / errs[1] < 40.0
    # joint = scales part + dense part to first order (one z stream, disjoint index ranges)
    eps = 1e-4
    def dd(**kw):
        return qzo.directional_derivative(omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, +1, eps, **kw),
                                          omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, -1, eps, **kw), eps)
    d_s, d_d, d_j = dd(), dd(perturb_scales=False, perturb_dense=True), dd(perturb_dense=True)
    assert abs(d_j - (d_s + d_d)) <= 1e-3 * (abs(d_s) + abs(d_d))
    # sign 0 ignores the mode
    assert omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, 0, eps, perturb_dense=True) == \
        omodel.forward_loss(m, tok.numpy(), lab.numpy(), seed, 0, eps)


def test_dense_update_invariants():
    cfg, raw = _tiny_raw("opt")
    m = build_oracle_model(raw)
    before = clone_model(m)
    qzo.update_model_dense(m, 7, 1e-3, 0.0)                           # d' = 0: bit-unchanged
    for key, layer in omodel.dense_tensor_names(cfg):
        assert np.array_equal(omodel.dense_tensor(m, key, layer), omodel.dense_tensor(before, key, layer))
    qzo.update_model_dense(m, 7, 1e-3, 2.5)
    bases, _ = omodel.dense_index_bases(cfg)
    moved = 0
    for key, layer in omodel.dense_tensor_names(cfg):
        old = np.asarray(omodel.dense_tensor(before, key, layer), dtype=np.float64)
        new = np.asarray(omodel.dense_tensor(m, key, layer), dtype=np.float64)
        z = philox.normal_range(7, bases[(key, layer)], old.size).astype(np.float64).reshape(old.shape)
        exact = old - 1e-3 * 2.5 * z                                  # Eq. 2 with the estimate d' z; no clamp
        ulp = 2.0 ** -8 if key in ("embed", "lm_head") else 2.0 ** -23
        assert np.all(np.abs(new - exact) <= ulp * np.maximum(np.abs(exact), 1e-3) + 1e-9)
        if key in ("embed", "lm_head"):
            assert np.array_equal(int4.bf16_round(new.astype(np.float32)), new.astype(np.float32))
        moved += int(np.sum(new != old))
    assert moved > 0
    # the in-place form of the two perturbations and the restore returns to the start (fp64 rounding)
    w = np.asarray(before["lm_head"], dtype=np.float64)
    a = qzo.spsa_perturbed(w, 3, 64, +1, 1e-3)
    b = a - 2e-3 * philox.normal_range(3, 64, w.size).astype(np.float64).reshape(w.shape)
    c = b + 1e-3 * philox.normal_range(3, 64, w.size).astype(np.float64).reshape(w.shape)
    assert np.allclose(b, qzo.spsa_perturbed(w, 3, 64, -1, 1e-3), rtol=0, atol=1e-15)
    assert np.allclose(c, w, rtol=0, atol=1e-15)


def test_joint_step_updates_scales_and_dense_tensors_from_one_clipped_derivative():
    cfg, raw = _tiny_raw("llama")
    m = build_oracle_model(raw)
    tok, lab = inputs.tokens_and_labels(cfg, 2, 16)
    a = clone_model(m)
    lp, lm, d, dc = qzo.step_functional(a, tok.numpy(), lab.numpy(), 11, 1e-3, 1e-3, 0.05, joint=True, lr_dense=1e-2)
    assert abs(dc) == 0.05 and abs(d) > 0.05                          # the clip branch of Eq. 6 is the active one
    b = clone_model(m)
    qzo.update_model_scales(b, 11, 1e-3, dc)
    qzo.update_model_dense(b, 11, 1e-2, dc)
    for li in range(2):
        for nm in omodel.LINEAR_ORDER["llama"]:
            assert np.array_equal(a["layers"][li]["lin"][nm]["s"], b["layers"][li]["lin"][nm]["s"])
        assert np.array_equal(a["layers"][li]["norm1_w"], b["layers"][li]["norm1_w"])
    assert np.array_equal(a["embed"], b["embed"]) and not np.array_equal(a["embed"], m["embed"])
