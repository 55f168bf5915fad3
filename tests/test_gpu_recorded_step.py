"""qzo_step with its two forwards replayed from a recorded launch sequence (a CUDA graph per batch shape, its
GEMMs reading seed and eps from device memory) against the same steps issued launch by launch: losses, d, d' and the
scales must agree bit for bit, step after step, across seeds, step sizes and batch shapes."""
import pytest
import torch

from paper_2505_13430_b200 import inputs

pytestmark = pytest.mark.gpu


def _models(name):
    from paper_2505_13430_b200 import qzo
    cfg = inputs.model_cfg(name)
    c = inputs.CONFIGS[name]
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    T = c["batch"] * c["seq"]
    recorded = qzo.build_model_from_raw(raw, T)
    direct = qzo.build_model_from_raw(raw, T)
    direct.qzo_use_recorded_steps(False)
    tok, lab = inputs.tokens_and_labels(cfg, c["batch"], c["seq"], seed=7)
    return qzo, c, recorded, direct, tok, lab


@pytest.mark.parametrize("name", ["tiny", "tiny_opt"])
def test_replayed_steps_equal_direct_steps(name):
    qzo, c, recorded, direct, tok, lab = _models(name)
    shapes = [(c["batch"], c["seq"]), (1, 16), (c["batch"] - 1, c["seq"])]       # paired, paired small, two passes
    schedule = []
    for rep in range(3):                                   # every shape: first step direct, then recorded, then replayed
        for si, (nb, ns) in enumerate(shapes):
            schedule.append((nb, ns, 100 + 7 * rep + si, c["eps"] * (1 + rep), c["lr"] * 50 * (1 + si), c["clip"] / (1 + rep)))
    for nb, ns, seed, eps, lr, clip in schedule:
        t, l = tok[:nb, :ns].contiguous().cuda(), lab[:nb, :ns].contiguous().cuda()
        n0 = qzo.qzo_launch_count()
        a = recorded.qzo_step(t, l, seed, eps, lr, clip)
        n1 = qzo.qzo_launch_count()
        b = direct.qzo_step(t, l, seed, eps, lr, clip)
        n2 = qzo.qzo_launch_count()
        assert a == b, (nb, ns, seed)
        assert torch.equal(recorded.scales.view(torch.int16), direct.scales.view(torch.int16)), (nb, ns, seed)
        # a replay accounts for the kernels it runs (plus the one that writes the step's parameters)
        assert n1 - n0 in (n2 - n1, n2 - n1 + 1), (n1 - n0, n2 - n1)
        # the logits both models keep from the step's forward (both signs' rows when they ran as one pass)
        rows = nb * ns * (2 if nb * ns in (16, 32, 64, 128) or (nb * ns) % 256 == 0 else 1)
        la = recorded.qzo_debug_layer_output(0, 1, rows)
        lb = direct.qzo_debug_layer_output(0, 1, rows)
        assert torch.equal(la.view(torch.int32), lb.view(torch.int32)), (nb, ns, seed)
        with pytest.raises(qzo.QzoError):
            recorded.qzo_debug_layer_output(0, 1, rows - 1)           # the buffer must hold every row of the last forward
    # every shape was recorded on one model and none on the other; the host-token entry point takes the same route
    assert recorded.qzo_recorded_step_count() == len(shapes) and direct.qzo_recorded_step_count() == -1
    assert recorded.qzo_device_status() == 0 and direct.qzo_device_status() == 0
    nb, ns = shapes[0]
    a = recorded.qzo_step_host(tok[:nb, :ns].contiguous(), lab[:nb, :ns].contiguous(), 5, c["eps"], c["lr"] * 50, c["clip"])
    b = direct.qzo_step_host(tok[:nb, :ns].contiguous(), lab[:nb, :ns].contiguous(), 5, c["eps"], c["lr"] * 50, c["clip"])
    assert a == b and torch.equal(recorded.scales.view(torch.int16), direct.scales.view(torch.int16))
    recorded.close()
    direct.close()


def test_replayed_step_reports_failures_and_leaves_the_scales_untouched():
    # The failure is made on the host (the status word is written with a copy, a scale is set to NaN); the
    # replayed step must report it like the direct one and change nothing.
    qzo, c, recorded, direct, tok, lab = _models("tiny")
    t, l = tok.cuda(), lab.cuda()
    for seed in (1, 2, 3):                                  # direct, recorded, replayed
        recorded.qzo_step(t, l, seed, c["eps"], c["lr"] * 50, c["clip"])
    assert recorded.qzo_recorded_step_count() == 1
    before = recorded.scales.clone()
    recorded.qzo_debug_set_status(1)
    with pytest.raises(qzo.QzoError) as e:
        recorded.qzo_step(t, l, 4, c["eps"], c["lr"] * 50, c["clip"])
    assert e.value.status == qzo.ERR_DEVICE_TIMEOUT
    assert torch.equal(recorded.scales.view(torch.int16), before.view(torch.int16))
    recorded.qzo_debug_set_status(0)
    recorded.scales[5] = float("nan")
    before = recorded.scales.clone()
    with pytest.raises(qzo.QzoError) as e:
        recorded.qzo_step(t, l, 5, c["eps"], c["lr"] * 50, c["clip"])
    assert e.value.status == qzo.ERR_NONFINITE
    torch.cuda.synchronize()
    assert bool((recorded.scales.view(torch.int16) == before.view(torch.int16)).all())
    recorded.close()
    direct.close()


def test_shapes_beyond_the_recording_limit_run_directly():
    # A model records at most 16 batch shapes; the shapes it meets after that keep running launch by launch,
    # with the same results.
    qzo, c, recorded, direct, tok, lab = _models("tiny")
    shapes = [(nb, ns) for nb in (1, 2, 3) for ns in (8, 16, 24, 32, 40, 48)]           # 18 shapes
    for rep in range(2):
        for i, (nb, ns) in enumerate(shapes):
            t, l = tok[:nb, :ns].contiguous().cuda(), lab[:nb, :ns].contiguous().cuda()
            a = recorded.qzo_step(t, l, 50 + i, c["eps"], c["lr"] * 50, c["clip"])
            b = direct.qzo_step(t, l, 50 + i, c["eps"], c["lr"] * 50, c["clip"])
            assert a == b, (nb, ns)
    assert recorded.qzo_recorded_step_count() == 16
    assert torch.equal(recorded.scales.view(torch.int16), direct.scales.view(torch.int16))
    recorded.close()
    direct.close()
