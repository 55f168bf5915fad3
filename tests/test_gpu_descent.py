"""End to end: repeated QZO steps on one batch lower that batch's loss, and the same steps with the sign of
the learning rate flipped raise it.  Nothing here comes from the oracle: the check is the method's purpose
(Algorithm 1 is ZO-SGD on the scales; E[d z] is the gradient of the smoothed loss, Sec. 3.1), so a wrong sign
anywhere on the path from the perturbation to the update fails it."""
import pytest
import torch

from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["tiny", "tiny_opt"])
def test_qzo_steps_descend(name):
    from paper_2505_13430_b200 import qzo
    cfg = inputs.model_cfg(name)
    c = inputs.CONFIGS[name]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    t, l = tok.cuda(), lab.cuda()
    end = {}
    for sgn in (+1.0, -1.0):
        gm = qzo.build_model_from_raw(raw, c["batch"] * c["seq"])
        start = float(gm.qzo_forward_loss(t, l, 0, 0, c["eps"]).cpu()[0])
        for step in range(600):
            gm.qzo_step(t, l, 1000 + step, c["eps"], sgn * c["lr"], c["clip"], read_back=(step % 100 == 99))
        end[sgn] = float(gm.qzo_forward_loss(t, l, 0, 0, c["eps"]).cpu()[0])
        assert gm.qzo_device_status() == 0
        assert bool((gm.scales >= 0).all())                   # the update clamps at zero (Algorithm 1, last loop)
        gm.close()
    print(f"{name}: loss {start:.4f} -> {end[+1.0]:.4f} with lr = {c['lr']:g}, -> {end[-1.0]:.4f} with lr = {-c['lr']:g}")
    # measured: 7.006 -> 6.81 / 7.19 (tiny), 6.968 -> 6.82 / 7.11 (tiny_opt) after 600 steps
    assert end[+1.0] < start - 0.08 and end[-1.0] > start + 0.08


@pytest.mark.parametrize("name", ["tiny", "tiny_opt"])
def test_joint_spsa_steps_descend_on_the_unquantised_tensors(name):
    # Joint mode with lr = 0: the scales stay where they are and only the embedding, the lm_head and the norm
    # vectors move (ZO-SGD with the same d', Def. 3.2); the batch's loss must fall, and rise with -lr_dense.
    from paper_2505_13430_b200 import qzo
    cfg = inputs.model_cfg(name)
    c = inputs.CONFIGS[name]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    t, l = tok.cuda(), lab.cuda()
    end = {}
    for sgn in (+1.0, -1.0):
        gm = qzo.build_model_from_raw(raw, c["batch"] * c["seq"])
        gm.qzo_enable_joint_spsa(sgn * 1e-4)
        before = gm.scales.clone()
        start = float(gm.qzo_forward_loss(t, l, 0, 0, c["eps"]).cpu()[0])
        for step in range(600):
            gm.qzo_step(t, l, 1000 + step, c["eps"], 0.0, c["clip"], read_back=(step % 100 == 99))
        end[sgn] = float(gm.qzo_forward_loss(t, l, 0, 0, c["eps"]).cpu()[0])
        assert gm.qzo_device_status() == 0
        assert torch.equal(gm.scales.view(torch.int16), before.view(torch.int16))
        gm.close()
    print(f"{name} (joint, scales frozen): loss {start:.4f} -> {end[+1.0]:.4f} with lr_dense = 1e-4, -> {end[-1.0]:.4f} with -1e-4")
    # measured: 7.006 -> 6.918 / 7.157 (tiny), 6.968 -> 6.897 / 7.084 (tiny_opt)
    assert end[+1.0] < start - 0.03 and end[-1.0] > start + 0.03
