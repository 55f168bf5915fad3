"""With one rank the data-parallel step is Algorithm 1 on the whole batch: same losses, same d, and
bit-identical scales as qzo_step (d formed on the host here, on the device there)."""
import pytest
import torch

from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


def test_single_rank_dp_step_equals_qzo_step():
    from paper_2505_13430_b200 import qzo, data_parallel as dp
    cfg = inputs.model_cfg("tiny")
    c = inputs.CONFIGS["tiny"]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    gm = qzo.build_model_from_raw(raw, c["batch"] * c["seq"])
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    tok_d, lab_d = tok.cuda(), lab.cuda()
    before = gm.scales.clone()
    ref = gm.qzo_step(tok_d, lab_d, 42, c["eps"], c["lr"] * 50, c["clip"])
    after_ref = gm.scales.clone()
    gm.scales.copy_(before)
    got = dp.dp_step(gm, tok_d, lab_d, 42, c["eps"], c["lr"] * 50, c["clip"])
    assert got[0] == ref[0] and got[1] == ref[1]
    assert abs(got[2] - ref[2]) <= 1e-6 * max(1.0, abs(ref[2])) and got[3] == ref[3]
    assert torch.equal(gm.scales.view(torch.int16), after_ref.view(torch.int16))
    assert not torch.equal(after_ref.view(torch.int16), before.view(torch.int16))
    assert dp.kept_tokens(lab) == c["batch"] * (c["seq"] - 1)
    gm.close()
