"""CPU oracle for the adapter update of a QA-LoRA fine-tuning step (arXiv 2309.14717).

TEST INFRASTRUCTURE ONLY.  Plain, slow definition of what the CUDA library's
optimizer entry point computes; only the tests and the benchmark's CPU legs may
import it, the product path never does, and this module imports nothing from the
CUDA package.  Everything is numpy in fp64.

Section 4.1 (training details) fixes the recipe: AdamW, a maximum gradient norm of
0.3, a constant learning rate (2e-5 for 7B/13B, 1e-5 for 33B/65B).  Only the
adapter factors A and B are trained; the quantized weights are frozen (Section 3.3).
The "paged" attribute of the optimizer in that section concerns where its state
lives, not what it computes.

Readings taken where the paper is silent (each is exercised by a pin in
tests/test_optimizer_pins.py):
  * The gradient norm is the Euclidean norm over ALL trained parameters of the step
    taken together, and gradients are multiplied by min(1, max_norm / (norm + 1e-6))
    (the usual clipping convention, small constant included).
  * AdamW is the decoupled-weight-decay form: the decay multiplies the parameter by
    (1 - lr * weight_decay) and does not enter the moment estimates.
  * Bias-corrected moments; the step is lr * m_hat / (sqrt(v_hat) + eps).
  * beta1 = 0.9, beta2 = 0.999, eps = 1e-8, weight_decay = 0 are defaults of the
    caller, not constants of this module.

parity: every function below has at least one pin; none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

__all__ = ["grad_norm", "clip_coefficient", "adamw_step"]


def grad_norm(grads) -> float:
    """Euclidean norm over every element of every array in `grads` (Section 4.1:
    the quantity bounded by the maximum gradient norm)."""
    total = 0.0
    for g in grads:
        g = np.asarray(g, dtype=np.float64)
        total += float(np.sum(g * g))
    return float(np.sqrt(total))


def clip_coefficient(norm: float, max_norm: float) -> float:
    """Factor applied to all gradients so that their joint norm does not exceed
    `max_norm` (Section 4.1: maximum gradient norm 0.3).  max_norm <= 0 disables
    clipping."""
    if max_norm <= 0.0:
        return 1.0
    return min(1.0, max_norm / (norm + 1e-6))


def adamw_step(params, grads, exp_avg, exp_avg_sq, step: int, lr: float, beta1: float = 0.9,
               beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.0,
               max_norm: float = 0.3):
    """One clipped AdamW update (Section 4.1) of the arrays in `params`.

    `step` counts from 1.  Returns (new_params, new_exp_avg, new_exp_avg_sq, norm,
    coefficient); nothing is modified in place.
    """
    if step < 1:
        raise ValueError("step counts from 1")
    if not (0.0 <= beta1 < 1.0 and 0.0 <= beta2 < 1.0):
        raise ValueError("beta1 and beta2 must lie in [0, 1)")
    if not (len(params) == len(grads) == len(exp_avg) == len(exp_avg_sq)):
        raise ValueError("one gradient and one pair of moments per parameter array")
    norm = grad_norm(grads)
    coef = clip_coefficient(norm, max_norm)
    new_p, new_m, new_v = [], [], []
    for p, g, m, v in zip(params, grads, exp_avg, exp_avg_sq):
        p, g, m, v = (np.asarray(t, dtype=np.float64) for t in (p, g, m, v))
        if not (p.shape == g.shape == m.shape == v.shape):
            raise ValueError("shapes of parameter, gradient and moments differ")
        g = coef * g
        p = p * (1.0 - lr * weight_decay)
        m = beta1 * m + (1.0 - beta1) * g
        v = beta2 * v + (1.0 - beta2) * g * g
        m_hat = m / (1.0 - beta1 ** step)
        v_hat = v / (1.0 - beta2 ** step)
        p = p - lr * m_hat / (np.sqrt(v_hat) + eps)
        new_p.append(p); new_m.append(m); new_v.append(v)
    return new_p, new_m, new_v, norm, coef
