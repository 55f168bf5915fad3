"""GPU parity of the joint mode (Q-SPSA on the scales combined with SPSA on the un-quantised tensors)
against the oracle on the tiny configurations: perturbed forwards, losses, and the seeded update of
the scales, of the embedding / lm_head matrices and of the norm vectors from one clipped d'."""
import numpy as np
import pytest
import torch

from oracle import model as omodel, qzo as oqzo
from paper_2505_13430_b200 import inputs
from tests.helpers import build_oracle_model, clone_model

pytestmark = pytest.mark.gpu


def _relerr(got, ref):
    got = got.float().cpu().numpy().astype(np.float64)
    return np.abs(got - ref).max() / np.abs(ref).max()


def _bf16_ulp_diff(a, b):
    def key(t):
        i = t.view(torch.int16).to(torch.int32) & 0xFFFF
        return torch.where(i >= 0x8000, 0x8000 - i, i)
    return (key(a) - key(b)).abs()


def _gpu_name(key, layer):
    return key if layer is None else f"L{layer}.{key}"


@pytest.mark.parametrize("name", ["tiny", "tiny_opt"])
def test_joint_forward_step_and_update_match_oracle(name):
    from paper_2505_13430_b200 import qzo as lib
    cfg = inputs.model_cfg(name)
    c = inputs.CONFIGS[name]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    g = torch.Generator().manual_seed(3)
    for layer in raw["layers"]:                          # norm vectors away from 1 / 0, so that a mix-up shows
        for k in ("norm1_w", "norm2_w", "norm1_b", "norm2_b"):
            if k in layer:
                layer[k] = layer[k] + 0.1 * torch.randn(layer[k].shape, generator=g)
        for ent in layer["lin"].values():
            ent["w"] = ent["w"] * 3.0
    om = build_oracle_model(raw)
    T = c["batch"] * c["seq"]
    gm = lib.build_model_from_raw(raw, T)
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    tok_d, lab_d = tok.cuda(), lab.cuda()
    # eps four times the configuration's, so that what the un-quantised tensors add to the losses is well
    # above the loss tolerance and a forward that left them unperturbed could not pass
    seed, eps, lr, clip, lr_dense = 42, 4 * c["eps"], c["lr"] * 50, c["clip"], 2e-3

    plain = {s: gm.qzo_forward_loss(tok_d, lab_d, seed, s, eps).cpu().clone() for s in (+1, -1)}
    gm.qzo_enable_joint_spsa(lr_dense)
    losses = {}
    for sign in (+1, -1, 0):
        cap = {}
        ref = omodel.forward_loss(om, tok.numpy(), lab.numpy(), seed, sign, eps, capture=cap, perturb_dense=True)
        for li in range(cfg["n_layers"]):
            gm.qzo_debug_set_capture(li)
            loss = gm.qzo_forward_loss(tok_d, lab_d, seed, sign, eps).cpu().clone()
            assert _relerr(gm.qzo_debug_layer_output(li, 0, T), cap["hidden"][li]) <= 2e-2, (sign, li)
        assert _relerr(gm.qzo_debug_layer_output(0, 1, T), cap["logits"]) <= 2e-2
        assert abs(float(loss[0]) - ref) <= 1e-3, (sign, float(loss[0]), ref)
        losses[sign] = (loss, ref)
    # the mode really perturbs more than the scales: the losses moved away from the plain ones, by what the
    # oracle says (the oracle's own two modes differ by far more than the tolerance)
    ref_plain = omodel.forward_loss(om, tok.numpy(), lab.numpy(), seed, +1, eps)
    assert abs(ref_plain - losses[+1][1]) > 3e-3 and abs(float(plain[+1][0]) - float(losses[+1][0][0])) > 3e-3

    # whole step: both signs in one pass; the losses are those of the single-sign calls, bit for bit
    before = {k: gm.tensor(k).clone() for k in ["embed", "lm_head", "scales"] +
              [_gpu_name(*kl) for kl in omodel.dense_tensor_names(cfg)[2:]]}
    lp, lm, d, dc = gm.qzo_step(tok_d, lab_d, seed, eps, lr, clip)
    assert np.float32(lp) == np.float32(losses[+1][0][0]) and np.float32(lm) == np.float32(losses[-1][0][0])
    assert abs(lp - losses[+1][1]) <= 1e-3 and abs(lm - losses[-1][1]) <= 1e-3
    assert gm.qzo_device_status() == 0
    # the update, from the device's own clipped d': scales and matrices within one bf16 ulp, vectors to fp32 rounding
    om2 = clone_model(om)
    oqzo.update_model_scales(om2, seed, lr, dc)
    oqzo.update_model_dense(om2, seed, lr_dense, dc)
    order = omodel.LINEAR_ORDER[cfg["arch"]]
    for li in range(cfg["n_layers"]):
        for i, nm in enumerate(order):
            ref = torch.from_numpy(om2["layers"][li]["lin"][nm]["s"]).bfloat16()
            assert int(_bf16_ulp_diff(gm.scales_of(li, i).cpu(), ref).max()) <= 1
    moved = 0
    for key, layer in omodel.dense_tensor_names(cfg):
        got = gm.tensor(_gpu_name(key, layer)).cpu()
        ref = torch.from_numpy(np.asarray(omodel.dense_tensor(om2, key, layer), dtype=np.float32))
        # the device's z agrees with the oracle's to 5e-6, so theta - coef z agrees to 5e-6 |coef| before storage;
        # the matrices are then rounded to bf16 (one ulp = 2^-7 relative at most; counting ulps would be
        # meaningless for the entries that the update leaves next to zero)
        floor = 5e-6 * abs(lr_dense * dc) + 1e-9
        if key in ("embed", "lm_head"):
            err = (got.float() - ref).abs() - 2.0 ** -7 * ref.abs()
            assert float(err.max()) <= floor, key
        else:
            assert float((got - ref).abs().max()) <= floor + 2.0 ** -22 * float(ref.abs().max()), (key, layer)
        moved += int((got != before[_gpu_name(key, layer)].cpu()).sum())
    assert moved > 0 and dc != 0.0
    # switched off again, the path is the plain one
    for k, v in before.items():
        gm.tensor(k).copy_(v)
    gm.qzo_enable_joint_spsa(0.0, on=False)
    again = gm.qzo_forward_loss(tok_d, lab_d, seed, +1, eps).cpu()
    assert torch.equal(again.view(torch.int32), plain[+1].view(torch.int32))
    gm.close()
