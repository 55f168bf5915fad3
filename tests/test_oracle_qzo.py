"""Pins for oracle/qzo.py: Eq. 6 cases, the exact finite difference on a quadratic loss,
Algorithm 1's in-place perturbations against the functional form, and the update's invariants."""
import numpy as np

from oracle import int4, linear, philox, qzo, model as omodel
from paper_2505_13430_b200 import inputs
from tests.helpers import build_oracle_model, clone_model


def test_ddc_three_cases_and_bounds():
    assert qzo.ddc_clip(250.0, 100.0) == 100.0
    assert qzo.ddc_clip(-250.0, 100.0) == -100.0
    assert qzo.ddc_clip(3.5, 100.0) == 3.5
    assert qzo.ddc_clip(100.0, 100.0) == 100.0 and qzo.ddc_clip(-100.0, 100.0) == -100.0
    assert qzo.ddc_clip(5.0, 0.0) == 0.0 and qzo.ddc_clip(-5.0, 0.0) == 0.0
    rng = np.random.default_rng(0)
    for d in rng.standard_normal(100) * 300:
        dc = qzo.ddc_clip(d, 100.0)
        assert abs(dc) <= min(abs(d), 100.0) and dc * d >= 0
    assert qzo.directional_derivative(2.0, 1.0, 0.25) == 2.0


def test_finite_difference_is_exact_on_quadratic_loss():
    # Y = X (s (.) q), L = 0.5 ||Y - T||^2 is quadratic in s, so the central difference
    # equals z . dL/ds for any eps (Eq. 5's approximation becomes an identity).
    rng = np.random.default_rng(4)
    M, K, N = 6, 256, 5
    x = rng.standard_normal((M, K))
    q = rng.integers(-8, 8, size=(K, N)).astype(np.int8)
    s = int4.bf16_round(rng.uniform(0.005, 0.02, size=(2, N)).astype(np.float32))
    tgt = rng.standard_normal((M, N))
    seed, base = 17, 24

    def loss(sign, eps):
        y = linear.perturbed_linear(x, q, s, seed, base, sign, eps)
        return 0.5 * np.sum((y - tgt) ** 2)

    y0 = linear.perturbed_linear(x, q, s, seed, base, 0, 0.0)
    grad = np.zeros((2, N))
    for g in range(2):
        xq = x[:, g * 128:(g + 1) * 128] @ q[g * 128:(g + 1) * 128].astype(np.float64)   # [M][N]
        grad[g] = np.sum((y0 - tgt) * xq, axis=0)
    z = philox.normal_range(seed, base, 2 * N).astype(np.float64).reshape(2, N)
    want = float(np.sum(z * grad))
    for eps in (1e-3, 1e-2, 0.3):
        d = qzo.directional_derivative(loss(+1, eps), loss(-1, eps), eps)
        assert abs(d - want) <= 1e-9 * abs(want)


def _setup():
    cfg = inputs.model_cfg("tiny", n_layers=2, d_model=64, n_heads=4, d_ffn=176, vocab=96, max_seq=16)
    raw = inputs.raw_model_tensors(cfg, seed=21)
    for layer in raw["layers"]:
        for ent in layer["lin"].values():
            ent["w"] = ent["w"] * 6.0
    m = build_oracle_model(raw)
    tok, lab = inputs.tokens_and_labels(cfg, 2, 16)
    return cfg, m, tok.numpy(), lab.numpy()


def test_cross_entropy_difference_converges_quadratically():
    cfg, m, tok, lab = _setup()
    ds = []
    for eps in (4e-3, 2e-3, 1e-3, 5e-4):
        lp = omodel.forward_loss(m, tok, lab, 3, +1, eps)
        lm = omodel.forward_loss(m, tok, lab, 3, -1, eps)
        ds.append(qzo.directional_derivative(lp, lm, eps))
    e1, e2, e3 = abs(ds[0] - ds[3]), abs(ds[1] - ds[3]), abs(ds[2] - ds[3])
    # error ~ c eps^2: halving eps divides it by ~4
    assert e1 > 0 and 2.5 < e1 / e2 < 6.5 and e3 < e2


def test_in_place_perturbation_equals_functional_form():
    # Algorithm 1 moves the scales in place; the oracle (and the library) evaluate Delta + sign*eps*z from the
    # untouched scales.  The two readings agree: a forward on scales moved by +eps z (then by -2 eps z) is the
    # forward with sign +1 (-1), and the third move restores the scales to fp64 rounding.
    cfg, m, tok, lab = _setup()
    seed, eps = 42, 1e-3
    a, b = clone_model(m), clone_model(m)
    lp = omodel.forward_loss(a, tok, lab, seed, +1, eps)
    lm = omodel.forward_loss(a, tok, lab, seed, -1, eps)
    qzo.perturb_scales_in_place(b, +eps, seed)
    assert abs(omodel.forward_loss(b, tok, lab, seed, 0, eps) - lp) < 1e-12
    qzo.perturb_scales_in_place(b, -2.0 * eps, seed)
    assert abs(omodel.forward_loss(b, tok, lab, seed, 0, eps) - lm) < 1e-12
    qzo.perturb_scales_in_place(b, +eps, seed)
    moved = False
    for la, lb in zip(a["layers"], b["layers"]):
        for name in la["lin"]:
            sa, sb = np.asarray(la["lin"][name]["s"], dtype=np.float64), lb["lin"][name]["s"]
            assert np.all(np.abs(sa - sb) <= 1e-15)
            moved = moved or sb.dtype == np.float64
    assert moved and lp != lm
    # the step built on the functional form: d from those two losses, d' clipped, scales updated and non-negative
    out = qzo.step_functional(a, tok, lab, seed, eps, 1e-3, 100.0)
    assert out[0] == lp and out[1] == lm and out[2] == qzo.directional_derivative(lp, lm, eps)
    for la in a["layers"]:
        for name in la["lin"]:
            assert np.all(la["lin"][name]["s"] >= 0)


def test_update_invariants():
    rng = np.random.default_rng(5)
    s = int4.bf16_round(rng.uniform(0.005, 0.02, size=(4, 64)).astype(np.float32))
    same = qzo.update_scales_flat(s, 9, 16, 1e-5, 0.0)
    assert np.array_equal(same.view(np.uint32), s.view(np.uint32))          # d' = 0: bit-unchanged
    # C = 0 clips every d to 0: model unchanged (the zero-shot point of the clipping sweep)
    assert qzo.ddc_clip(123.0, 0.0) == 0.0
    up = qzo.update_scales_flat(s, 9, 16, 1e-5, 100.0)
    assert np.all(up >= 0) and np.array_equal(int4.bf16_round(up), up)
    z = philox.normal_range(9, 16, s.size).reshape(s.shape).astype(np.float64)
    exact = np.maximum(s.astype(np.float64) - 1e-5 * 100.0 * z, 0.0)
    assert np.all(np.abs(up - exact) <= 2.0 ** -8 * exact + 1e-9)
    # max(., 0) fires for a large step; sign of the move follows -d' z
    big = qzo.update_scales_flat(s, 9, 16, 1e-2, 100.0)
    assert (big == 0).any() and np.all(big >= 0)
    moved = up.astype(np.float64) - s
    strong = np.abs(1e-3 * z) > 2.0 ** -7 * s
    assert np.all(np.sign(moved[strong]) == -np.sign(z[strong]))
    # same seed -> same z in perturbation and update; other seed -> other z
    assert not np.array_equal(qzo.update_scales_flat(s, 10, 16, 1e-5, 100.0), up)


def test_step_uses_same_batch_and_seed_for_both_forwards():
    cfg, m, tok, lab = _setup()
    lp, lm, d, dc = qzo.step_functional(clone_model(m), tok, lab, 8, 1e-3, 1e-5, 100.0, update=False)
    assert lp == omodel.forward_loss(m, tok, lab, 8, +1, 1e-3)
    assert lm == omodel.forward_loss(m, tok, lab, 8, -1, 1e-3)
    assert d == (lp - lm) / 2e-3 and abs(dc) <= 100.0
