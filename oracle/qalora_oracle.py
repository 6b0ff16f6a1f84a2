"""CPU oracle for the QA-LoRA linear layer (arXiv 2309.14717).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain definition of what the
CUDA library computes.  Only the tests, the smoke check and the benchmark's CPU
baseline leg may import it; the product path never does, and this module
imports nothing from the CUDA package.  Everything is numpy.  Floating point is
fp64, except the quantizer's rounding decision, which is taken in IEEE fp32
(the precision the library's quantize kernel uses), with an fp64 shadow beside
it.

Notation (the paper's symbol L is the NUMBER of groups; here it is never used
bare):
    K = D_in, N = D_out, M = tokens, g = group size, G = K // g groups,
    r = D_int (adapter rank), b = bit width, s = adapter coefficient,
    alpha[G, N], beta[G, N] = scaling and zero factors per (group, column),
    c[K, N] = integer codes in {0 .. 2^b - 1},
    A[G, r], B[r, N] = adapter factors (Section 3.3: A is "L x D_int").

Readings taken where the paper is silent (each is exercised by a pin in
tests/test_oracle_pins.py):
  * Eq. 1 is the normative quantizer: W~ = alpha*c + beta with beta the group
    minimum (an additive zero), applied per group of g consecutive input
    channels and per output column (Section 3.3).
  * The integer rounding is round-half-to-even.
  * A constant group (max == min) takes alpha = 1, codes 0, beta = min.
  * Codes are clamped to [0, 2^b - 1] after rounding.
  * The pooling is a plain sum over g consecutive channels (Appendix B Eq. 3;
    Algorithm 1 multiplies an average pool by the window length).
  * Merge, in additive-zero form: beta' = beta + s * (A @ B).  Appendix B /
    Algorithm 1 state the same update for a zero POINT z (W~ = alpha*(c - z)):
    z' = z - s*(A @ B)/alpha; the two agree under z = -beta/alpha.

parity: every function below has at least one pin; none is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "levels", "quantize", "quantize_fp64_shadow", "dequantize", "pool",
    "forward", "backward", "backward_adapter", "merge", "merge_zero_point", "zero_point_from_beta",
    "beta_from_zero_point", "dequantize_zero_point", "words_per_unit",
    "pack", "unpack", "adapter_param_count",
]


def levels(bits: int) -> int:
    """Largest code, 2^b - 1 (Eq. 1)."""
    if bits not in (2, 3, 4):
        raise ValueError("bits must be 2, 3 or 4")
    return (1 << bits) - 1


def _check_group(K: int, g: int) -> int:
    if g <= 0 or K % g != 0:
        raise ValueError("group size must divide D_in")
    return K // g


# ----------------------------------------------------------------------------
# Quantizer: Eq. 1 applied per group (Section 3.3)
# ----------------------------------------------------------------------------
def _quantize_in(W: np.ndarray, g: int, bits: int, ftype):
    """Eq. 1 per (group, column), every operation in `ftype`, one at a time."""
    W = np.asarray(W)
    if W.ndim != 2:
        raise ValueError("W must be [K, N]")
    if not np.all(np.isfinite(W)):
        raise ValueError("W must be finite")
    K, N = W.shape
    G = _check_group(K, g)
    qmax = ftype(levels(bits))
    Wg = W.astype(ftype).reshape(G, g, N)
    lo = Wg.min(axis=1)                       # beta = min           (Eq. 1)
    hi = Wg.max(axis=1)
    d = (hi - lo).astype(ftype)
    alpha = (d / qmax).astype(ftype)          # (max - min)/(2^b - 1) (Eq. 1)
    alpha = np.where(hi == lo, ftype(1), alpha).astype(ftype)
    beta = lo.astype(ftype)
    t = ((Wg - beta[:, None, :]).astype(ftype) / alpha[:, None, :]).astype(ftype)
    c = np.rint(t)                            # round half to even
    c = np.clip(c, 0, levels(bits))
    codes = c.astype(np.uint8).reshape(K, N)
    return codes, alpha, beta


def quantize(W: np.ndarray, g: int, bits: int):
    """Group-wise min-max quantization, the fp32 normative sequence.

    Eq. 1 with (alpha, beta) taken per group of g consecutive rows of W and per
    column (Section 3.3).  d = hi - lo; alpha = d / (2^b - 1); t = (w - beta) /
    alpha; c = clamp(rint(t)): four IEEE fp32 operations, no fused multiply-add
    and no reciprocal, so that a GPU kernel can reproduce the integer decision
    bit for bit.  Returns (codes uint8 [K, N], alpha fp32 [G, N], beta fp32
    [G, N]).
    """
    return _quantize_in(np.asarray(W, dtype=np.float32), g, bits, np.float32)


def quantize_fp64_shadow(W: np.ndarray, g: int, bits: int):
    """The same rule evaluated in fp64 on the same stored fp32 weights."""
    return _quantize_in(np.asarray(W, dtype=np.float32), g, bits, np.float64)


def dequantize(codes: np.ndarray, alpha: np.ndarray, beta: np.ndarray, g: int) -> np.ndarray:
    """W~[k, n] = alpha[k // g, n] * c[k, n] + beta[k // g, n] in fp64 (Eq. 1)."""
    K, N = codes.shape
    G = _check_group(K, g)
    a = np.asarray(alpha, dtype=np.float64).reshape(G, 1, N)
    z = np.asarray(beta, dtype=np.float64).reshape(G, 1, N)
    c = codes.astype(np.float64).reshape(G, g, N)
    return (a * c + z).reshape(K, N)


# ----------------------------------------------------------------------------
# The layer: Algorithm 1 (qalora_forward), Appendix B Eq. 3 and Eq. 4
# ----------------------------------------------------------------------------
def pool(x: np.ndarray, g: int) -> np.ndarray:
    """xp[m, q] = sum of x[m, k] over the g channels of group q (Appendix B Eq. 3)."""
    x = np.asarray(x, dtype=np.float64)
    M, K = x.shape
    G = _check_group(K, g)
    return x.reshape(M, G, g).sum(axis=2)


def forward(x, codes, alpha, beta, g, A=None, B=None, s=0.0) -> np.ndarray:
    """y = x @ W~ + s * ((pool(x) @ A) @ B)   (Algorithm 1; Appendix B Eq. 4).

    With A or B absent (rank 0) this is the deployed, plain quantized layer.
    """
    x = np.asarray(x, dtype=np.float64)
    y = x @ dequantize(codes, alpha, beta, g)
    if A is not None and B is not None and np.asarray(A).shape[1] > 0:
        A = np.asarray(A, dtype=np.float64)
        B = np.asarray(B, dtype=np.float64)
        y = y + float(s) * ((pool(x, g) @ A) @ B)
    return y


def backward_adapter(x, dy, g, A, B, s):
    """The adapter gradients alone (they do not involve W):
        dT = s * dy @ B^T;  dA = pool(x)^T @ dT;  dB = s * (pool(x) @ A)^T @ dy.
    Both are sums over token rows, so row blocks can be processed separately and added."""
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    s = float(s)
    xp = pool(x, g)
    dT = s * (dy @ B.T)
    dA = xp.T @ dT
    dB = s * ((xp @ A).T @ dy)
    return dA, dB


def backward(x, dy, codes, alpha, beta, g, A, B, s):
    """Gradients of l = sum(dy * y) with the base weights frozen (Section 3.1).

    y is linear in x and bilinear in (A, B):
        dT = s * dy @ B^T                                  [M, r]
        dX = dy @ W~^T + repeat_g(dT @ A^T)                [M, K]
        dA = pool(x)^T @ dT                                [G, r]
        dB = s * (pool(x) @ A)^T @ dy                      [r, N]
    Returns (dX, dA, dB) in fp64.
    """
    x = np.asarray(x, dtype=np.float64)
    dy = np.asarray(dy, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    s = float(s)
    dT = s * (dy @ B.T)
    dXp = dT @ A.T                                        # [M, G]
    dX = dy @ dequantize(codes, alpha, beta, g).T + np.repeat(dXp, g, axis=1)
    dA, dB = backward_adapter(x, dy, g, A, B, s)
    return dX, dA, dB


def merge(beta, A, B, s) -> np.ndarray:
    """beta'[q, n] = beta[q, n] + s * sum_i A[q, i] * B[i, n]   (Appendix B Eq. 7).

    The paper folds s*A@B into the zero factors; written for its zero point z
    (W~ = alpha*(c - z)) the update is z' = z - s*A@B/alpha; for the additive
    zero of Eq. 1 (z = -beta/alpha) that is the line above, with no division.
    """
    beta = np.asarray(beta, dtype=np.float64)
    A = np.asarray(A, dtype=np.float64)
    B = np.asarray(B, dtype=np.float64)
    return beta + float(s) * (A @ B)


def merge_zero_point(z, alpha, A, B, s) -> np.ndarray:
    """Algorithm 1's merge as printed: z' = z - s * (A @ B) / alpha (zero-point form)."""
    z = np.asarray(z, dtype=np.float64)
    alpha = np.asarray(alpha, dtype=np.float64)
    P = np.asarray(A, dtype=np.float64) @ np.asarray(B, dtype=np.float64)
    return z - float(s) * P / alpha


def zero_point_from_beta(alpha, beta) -> np.ndarray:
    """z = -beta / alpha: the zero POINT of Algorithm 1's form W~ = alpha * (c - z) that
    describes the same weights as Eq. 1's additive zero beta (W~ = alpha * c + beta)."""
    alpha = np.asarray(alpha, dtype=np.float64)
    if np.any(alpha == 0):
        raise ValueError("alpha must be non-zero")
    return -np.asarray(beta, dtype=np.float64) / alpha


def beta_from_zero_point(alpha, z) -> np.ndarray:
    """beta = -alpha * z: Eq. 1's additive zero for a layer stored in Algorithm 1's
    zero-point form (an integer z from an asymmetric integer quantizer, or the real z'
    left by Algorithm 1's merge)."""
    return -np.asarray(alpha, dtype=np.float64) * np.asarray(z, dtype=np.float64)


def dequantize_zero_point(codes: np.ndarray, alpha: np.ndarray, z: np.ndarray, g: int) -> np.ndarray:
    """W~[k, n] = alpha[k // g, n] * (c[k, n] - z[k // g, n])  (Algorithm 1, pre_quantization)."""
    K, N = codes.shape
    G = _check_group(K, g)
    a = np.asarray(alpha, dtype=np.float64).reshape(G, 1, N)
    zz = np.asarray(z, dtype=np.float64).reshape(G, 1, N)
    c = codes.astype(np.float64).reshape(G, g, N)
    return (a * (c - zz)).reshape(K, N)


# ----------------------------------------------------------------------------
# Packed code layout (the library's own; this is an independent implementation
# of the layout's prose specification)
# ----------------------------------------------------------------------------
# A pack unit is 32 consecutive input channels (k-block kb = k // 32) of one
# output column n; j = k % 32 is the position inside the unit.  The packed
# array is little-endian uint32 [K/32][N][words]:
#   INT4, 4 words: word j // 8;  e = j % 8;  the code sits at bit 16*(e & 1) + 4*(e >> 1).
#   INT2, 2 words: word j // 16; e = j % 16; the code sits at bit 16*(e & 1) + 2*(e >> 1).
#   INT3, 3 words: words 0..1 hold (c & 3) in the INT2 arrangement; word 2
#                  holds (c >> 2) of position j at bit 16*(j & 1) + (j >> 1).
# (Even positions fill the low half-word and odd positions the high half-word,
# so one shift and one mask pull out a pair of neighbouring channels.)
def words_per_unit(bits: int) -> int:
    levels(bits)
    return {4: 4, 3: 3, 2: 2}[bits]


def pack(codes: np.ndarray, bits: int) -> np.ndarray:
    """codes uint8 [K, N] -> uint32 [K/32, N, words]."""
    K, N = codes.shape
    if K % 32 != 0:
        raise ValueError("D_in must be a multiple of 32")
    if codes.max(initial=0) > levels(bits):
        raise ValueError("code out of range")
    c = codes.astype(np.uint32).reshape(K // 32, 32, N)
    out = np.zeros((K // 32, N, words_per_unit(bits)), dtype=np.uint32)
    for j in range(32):
        cj = c[:, j, :]
        if bits == 4:
            e = j % 8
            out[:, :, j // 8] |= cj << np.uint32(16 * (e & 1) + 4 * (e >> 1))
        elif bits == 2:
            e = j % 16
            out[:, :, j // 16] |= cj << np.uint32(16 * (e & 1) + 2 * (e >> 1))
        else:
            e = j % 16
            out[:, :, j // 16] |= (cj & np.uint32(3)) << np.uint32(16 * (e & 1) + 2 * (e >> 1))
            out[:, :, 2] |= (cj >> np.uint32(2)) << np.uint32(16 * (j & 1) + (j >> 1))
    return out


def unpack(packed: np.ndarray, bits: int) -> np.ndarray:
    """uint32 [K/32, N, words] -> codes uint8 [K, N]."""
    KB, N, words = packed.shape
    if words != words_per_unit(bits):
        raise ValueError("wrong number of words per unit")
    p = packed.astype(np.uint32)
    c = np.zeros((KB, 32, N), dtype=np.uint32)
    for j in range(32):
        if bits == 4:
            e = j % 8
            c[:, j, :] = (p[:, :, j // 8] >> np.uint32(16 * (e & 1) + 4 * (e >> 1))) & np.uint32(15)
        elif bits == 2:
            e = j % 16
            c[:, j, :] = (p[:, :, j // 16] >> np.uint32(16 * (e & 1) + 2 * (e >> 1))) & np.uint32(3)
        else:
            e = j % 16
            lo = (p[:, :, j // 16] >> np.uint32(16 * (e & 1) + 2 * (e >> 1))) & np.uint32(3)
            hi = (p[:, :, 2] >> np.uint32(16 * (j & 1) + (j >> 1))) & np.uint32(1)
            c[:, j, :] = lo | (hi << np.uint32(2))
    return c.reshape(KB * 32, N).astype(np.uint8)


# ----------------------------------------------------------------------------
# Storage bookkeeping (Section 3.3; Table 2)
# ----------------------------------------------------------------------------
def adapter_param_count(K: int, N: int, g: int, r: int) -> int:
    """Learnable parameters of one layer: A is [K/g, r], B is [r, N] (Section 3.3)."""
    return (_check_group(K, g) + N) * r
