"""Pins for the optimizer oracle (Section 4.1's recipe: AdamW, maximum gradient norm 0.3):
closed forms, a library routine on the same inputs, invariants, and planted mistakes."""
import numpy as np
import pytest
import torch

from oracle import optimizer_oracle as P


def _state(rng, shapes):
    params = [rng.standard_normal(s) * 0.02 for s in shapes]
    grads = [rng.standard_normal(s) * 0.5 for s in shapes]
    zeros = [np.zeros(s) for s in shapes]
    return params, grads, zeros, [z.copy() for z in zeros]


def test_norm_is_joint_over_all_arrays_and_clip_bounds_it():
    # 3-4-12 Pythagorean quadruple: the joint norm of (3, 4) and (12,) is 13, not 5 or 12
    assert P.grad_norm([np.array([3.0, 4.0]), np.array([[12.0]])]) == pytest.approx(13.0, abs=1e-12)
    assert P.clip_coefficient(13.0, 0.3) == pytest.approx(0.3 / (13.0 + 1e-6), rel=1e-15)
    assert P.clip_coefficient(0.1, 0.3) == 1.0          # below the bound: untouched
    assert P.clip_coefficient(13.0, 0.0) == 1.0         # disabled
    rng = np.random.default_rng(0)
    g = [rng.standard_normal((7, 5)), rng.standard_normal(11)]
    c = P.clip_coefficient(P.grad_norm(g), 0.3)
    assert P.grad_norm([c * t for t in g]) == pytest.approx(0.3, rel=1e-5)
    assert P.grad_norm([c * t for t in g]) <= 0.3


def test_first_step_closed_form():
    # with zero moments and t = 1 the bias corrections cancel: m_hat = g, v_hat = g^2
    rng = np.random.default_rng(1)
    params, grads, m, v = _state(rng, [(6, 4), (4, 10)])
    lr, eps = 2e-5, 1e-8
    new_p, new_m, new_v, norm, coef = P.adamw_step(params, grads, m, v, 1, lr, eps=eps, max_norm=0.3)
    assert coef < 1.0 and norm == pytest.approx(np.sqrt(sum((g * g).sum() for g in grads)))
    for p0, g, p1, m1, v1 in zip(params, grads, new_p, new_m, new_v):
        gc = coef * g
        np.testing.assert_allclose(p1, p0 - lr * gc / (np.abs(gc) + eps), rtol=0, atol=1e-15)
        np.testing.assert_allclose(m1, 0.1 * gc, rtol=1e-12)
        np.testing.assert_allclose(v1, 0.001 * gc * gc, rtol=1e-12)


def test_constant_gradient_moves_lr_per_step():
    # a gradient that never changes keeps m_hat = g and v_hat = g^2 at every step, so each step
    # moves every parameter by lr * g / (|g| + eps) whatever the betas are
    g = [np.array([0.2, -0.05, 0.01])]
    p, m, v = [np.zeros(3)], [np.zeros(3)], [np.zeros(3)]
    lr, eps, steps = 1e-3, 1e-8, 25
    for t in range(1, steps + 1):
        p, m, v, _, coef = P.adamw_step(p, g, m, v, t, lr, beta1=0.8, beta2=0.95, eps=eps, max_norm=0.0)
        assert coef == 1.0
    np.testing.assert_allclose(p[0], -steps * lr * g[0] / (np.abs(g[0]) + eps), rtol=1e-10)


def test_weight_decay_is_decoupled():
    # zero gradient: the moments stay zero and only the multiplicative decay acts.  A decay that
    # went through the gradient (L2 form) would instead move every parameter by about lr.
    p0 = [np.array([1.0, -2.0, 0.5])]
    z = [np.zeros(3)]
    lr, wd = 1e-2, 0.1
    p1, m1, v1, norm, coef = P.adamw_step(p0, z, z, z, 1, lr, weight_decay=wd)
    np.testing.assert_allclose(p1[0], p0[0] * (1 - lr * wd), rtol=1e-15)
    assert norm == 0.0 and coef == 1.0 and not m1[0].any() and not v1[0].any()


@pytest.mark.parametrize("wd,max_norm", [(0.0, 0.3), (0.05, 0.3), (0.0, 0.0)])
def test_matches_library_adamw_with_library_clipping(wd, max_norm):
    rng = np.random.default_rng(2)
    shapes = [(16, 8), (8, 24), (5,)]
    params, _, m, v = _state(rng, shapes)
    tp = [torch.tensor(p, dtype=torch.float64, requires_grad=True) for p in params]
    lr = 2e-5
    opt = torch.optim.AdamW(tp, lr=lr, betas=(0.9, 0.999), eps=1e-8, weight_decay=wd)
    for t in range(1, 7):
        grads = [rng.standard_normal(s) * (0.01 if t % 2 else 2.0) for s in shapes]   # below and above the bound
        for q, g in zip(tp, grads):
            q.grad = torch.tensor(g, dtype=torch.float64)
        if max_norm > 0:
            lib_norm = float(torch.nn.utils.clip_grad_norm_(tp, max_norm))
        opt.step()
        params, m, v, norm, coef = P.adamw_step(params, grads, m, v, t, lr, weight_decay=wd, max_norm=max_norm)
        if max_norm > 0:
            assert norm == pytest.approx(lib_norm, rel=1e-12)
        for q, p in zip(tp, params):
            np.testing.assert_allclose(q.detach().numpy(), p, rtol=0, atol=1e-14)


def test_update_is_invariant_to_gradient_scale_up_to_eps():
    # Adam normalises the gradient, so clipping changes the first step only through eps
    rng = np.random.default_rng(3)
    params, grads, m, v = _state(rng, [(9, 3)])
    a = P.adamw_step(params, grads, m, v, 1, 1e-3, eps=0.0, max_norm=0.3)[0][0]
    b = P.adamw_step(params, grads, m, v, 1, 1e-3, eps=0.0, max_norm=0.0)[0][0]
    np.testing.assert_allclose(a, b, rtol=0, atol=1e-15)


def test_rejects_bad_arguments():
    z = [np.zeros(2)]
    with pytest.raises(ValueError):
        P.adamw_step(z, z, z, z, 0, 1e-3)
    with pytest.raises(ValueError):
        P.adamw_step(z, z, z, z, 1, 1e-3, beta1=1.0)
    with pytest.raises(ValueError):
        P.adamw_step(z, [np.zeros(3)], z, z, 1, 1e-3)
    with pytest.raises(ValueError):
        P.adamw_step(z, z + z, z, z, 1, 1e-3)
