"""With one rank the data-parallel step (begin, exchange, finish) is Algorithm 1 on the whole batch:
same losses, same d and bit-identical scales as qzo_step; and splitting the batch over two model
replicas whose loss sums are added (what two ranks' all-reduce does) gives the whole-batch step."""
import pytest
import torch

from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


def _tiny():
    from paper_2505_13430_b200 import qzo
    cfg = inputs.model_cfg("tiny")
    c = inputs.CONFIGS["tiny"]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    return qzo, cfg, c, raw, tok, lab


def test_single_rank_dp_step_equals_qzo_step():
    from paper_2505_13430_b200 import data_parallel as dp
    qzo, cfg, c, raw, tok, lab = _tiny()
    gm = qzo.build_model_from_raw(raw, c["batch"] * c["seq"])
    tok_d, lab_d = tok.cuda(), lab.cuda()
    before = gm.scales.clone()
    ref = gm.qzo_step(tok_d, lab_d, 42, c["eps"], c["lr"] * 50, c["clip"])
    after_ref = gm.scales.clone()
    gm.scales.copy_(before)
    # three times: the first data-parallel step of the shape replays what qzo_step left recorded or records
    # itself; every one of them must reproduce the direct step
    for _ in range(3):
        gm.scales.copy_(before)
        got = dp.dp_step(gm, tok_d, lab_d, 42, c["eps"], c["lr"] * 50, c["clip"])
        assert got == ref
        assert torch.equal(gm.scales.view(torch.int16), after_ref.view(torch.int16))
    assert gm.qzo_recorded_step_count() == 1
    assert not torch.equal(after_ref.view(torch.int16), before.view(torch.int16))
    gm.close()


def test_two_replicas_with_added_loss_sums_follow_the_whole_batch_step():
    # Two "ranks" emulated one after the other on one GPU (nothing waits on anything): each runs the begin
    # half on its half of the batch, the sums are added as an all-reduce would, both finish with the total.
    qzo, cfg, c, raw, tok, lab = _tiny()
    T = c["batch"] * c["seq"]
    whole = qzo.build_model_from_raw(raw, T)
    ranks = [qzo.build_model_from_raw(raw, T) for _ in range(2)]
    seed, eps, lr, clip = 9, c["eps"], c["lr"] * 50, c["clip"]
    ref = whole.qzo_step(tok.cuda(), lab.cuda(), seed, eps, lr, clip)
    half = c["batch"] // 2
    sums = [ranks[r].qzo_step_begin(tok[r * half:(r + 1) * half].contiguous().cuda(),
                                    lab[r * half:(r + 1) * half].contiguous().cuda(), seed, eps) for r in range(2)]
    total = sums[0] + sums[1]
    assert float(total[2]) == float(total[3]) == c["batch"] * (c["seq"] - 1)
    outs = [ranks[r].qzo_step_finish(total, seed, eps, lr, clip) for r in range(2)]
    assert outs[0] == outs[1]
    # the token-weighted mean of the halves is the whole batch's mean up to fp32 summation order
    assert abs(outs[0][0] - ref[0]) <= 2e-6 * abs(ref[0]) and abs(outs[0][1] - ref[1]) <= 2e-6 * abs(ref[1])
    assert torch.equal(ranks[0].scales.view(torch.int16), ranks[1].scales.view(torch.int16))
    if outs[0][3] == ref[3]:             # same clipped d' (both clipped, or bit-equal d): same update as the whole batch
        assert torch.equal(ranks[0].scales.view(torch.int16), whole.scales.view(torch.int16))
    for m in ranks + [whole]:
        m.close()


def test_seed_per_rank_step_matches_the_oracle_and_keeps_replicas_identical():
    # Two "ranks" emulated one after the other on one GPU (nothing waits on anything): rank r perturbs with
    # seed base + r on its half of the batch; both then apply rank 0's update and rank 1's update in that order,
    # each from that rank's own loss sums.  Both replicas must end bit-identical, the losses must be the
    # oracle's for (half, seed), and the scales must be the oracle's after the same two updates.
    import numpy as np
    from oracle import model as omodel, qzo as oqzo
    from tests.helpers import build_oracle_model, loss_tolerance
    qzo, cfg, c, raw, tok, lab = _tiny()
    om = build_oracle_model(raw)
    T = c["batch"] * c["seq"]
    ranks = [qzo.build_model_from_raw(raw, T) for _ in range(2)]
    base, eps, lr_each, clip = 300, c["eps"], c["lr"] * 25, c["clip"]
    half = c["batch"] // 2
    halves = [(tok[r * half:(r + 1) * half].contiguous(), lab[r * half:(r + 1) * half].contiguous()) for r in range(2)]
    sums = [ranks[r].qzo_step_begin(halves[r][0].cuda(), halves[r][1].cuda(), base + r, eps).clone() for r in range(2)]
    outs = [[ranks[k].qzo_step_finish(sums[r], base + r, eps, lr_each, clip) for r in range(2)] for k in range(2)]
    assert outs[0] == outs[1]
    assert torch.equal(ranks[0].scales.view(torch.int16), ranks[1].scales.view(torch.int16))
    order = omodel.LINEAR_ORDER[cfg["arch"]]
    for r in range(2):
        t, l = halves[r][0].numpy(), halves[r][1].numpy()
        tol = loss_tolerance(int((l >= 0).sum()))
        assert abs(outs[0][r][0] - omodel.forward_loss(om, t, l, base + r, +1, eps)) <= tol
        assert abs(outs[0][r][1] - omodel.forward_loss(om, t, l, base + r, -1, eps)) <= tol
    for r in range(2):                                       # the oracle's updates with the device's own d'
        oqzo.update_model_scales(om, base + r, lr_each, outs[0][r][3])
    for li in range(cfg["n_layers"]):
        for i, nm in enumerate(order):
            got = ranks[0].scales_of(li, i).float().cpu().numpy()
            ref = om["layers"][li]["lin"][nm]["s"].astype(np.float32)
            # two updates, each rounded to bf16: within one ulp each
            assert np.all(np.abs(got - ref) <= 2.0 ** -6 * np.abs(ref) + 1e-12)
    assert outs[0][0][3] != 0.0 or outs[0][1][3] != 0.0
    for m in ranks:
        m.close()
