"""Pins for the CPU oracle: each check ties an oracle function to something
other than itself (hand-worked examples of Eq. 1, brute force, closed forms,
library routines on special cases, finite differences, the paper's Table 2)."""
import itertools
import os

import numpy as np
import pytest

from oracle import qalora_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                yield [p.strip() for p in line.split("|")]


def _rand_layer(rng, K, N, g, bits, r, M):
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float32)
    codes, alpha, beta = O.quantize(W, g, bits)
    x = rng.standard_normal((M, K))
    A = rng.standard_normal((K // g, r)) * 0.3
    B = rng.standard_normal((r, N)) * 0.3
    dy = rng.standard_normal((M, N))
    return W, codes, alpha, beta, x, A, B, dy


# ---------------------------------------------------------------- quantizer --
@pytest.mark.parametrize("row", list(_rows("eq1_worked_examples.txt")))
def test_eq1_worked_examples(row):
    bits, w, alpha, beta, codes = row
    w = np.array([float(v) for v in w.split()], dtype=np.float32).reshape(-1, 1)
    want = np.array([int(v) for v in codes.split()], dtype=np.uint8).reshape(-1, 1)
    for fn in (O.quantize, O.quantize_fp64_shadow):
        c, a, b = fn(w, w.shape[0], int(bits))
        assert a.shape == (1, 1) and float(a[0, 0]) == float(alpha)
        assert float(b[0, 0]) == float(beta)
        assert np.array_equal(c, want)


@pytest.mark.parametrize("bits", [2, 3, 4])
@pytest.mark.parametrize("g", [4, 8, 32])
def test_quantizer_is_nearest_level_brute_force(bits, g):
    rng = np.random.default_rng(100 + bits * 10 + g)
    K, N = 4 * g, 7
    W = (rng.standard_normal((K, N)) * 0.02).astype(np.float32)
    W[rng.random((K, N)) < 0.05] *= 10
    codes, alpha, beta = O.quantize(W, g, bits)
    G = K // g
    Wg = W.astype(np.float64).reshape(G, g, N)
    # alpha and beta against a direct scan of each group
    for q, n in itertools.product(range(G), range(N)):
        col = [float(W[q * g + i, n]) for i in range(g)]
        assert float(beta[q, n]) == min(col)
        assert abs(float(alpha[q, n]) - (max(col) - min(col)) / (2 ** bits - 1)) <= 2e-7 * (max(col) - min(col))
    # each code is the arg-min over ALL levels of |w - (alpha*c + beta)|
    lv = np.arange(2 ** bits, dtype=np.float64)
    a64 = alpha.astype(np.float64)[:, None, :, None]
    b64 = beta.astype(np.float64)[:, None, :, None]
    dist = np.abs(Wg[..., None] - (a64 * lv + b64))            # [G, g, N, levels]
    best = dist.min(axis=-1)
    chosen = np.take_along_axis(dist, codes.reshape(G, g, N, 1).astype(np.int64), axis=-1)[..., 0]
    assert np.all(chosen <= best + 1e-6 * a64[..., 0])
    # the extreme codes are attained in every (non-constant) group
    cg = codes.reshape(G, g, N)
    assert np.all(cg.min(axis=1) == 0) and np.all(cg.max(axis=1) == 2 ** bits - 1)
    # rounding error bound of Eq. 1
    Wt = O.dequantize(codes, alpha, beta, g)
    assert np.all(np.abs(W - Wt) <= np.repeat(alpha, g, axis=0) * 0.5 * (1 + 1e-5))


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_fp32_and_fp64_rounding_decisions_agree(bits):
    rng = np.random.default_rng(7)
    W = (rng.standard_normal((256, 64)) * 0.02).astype(np.float32)
    c32, a32, b32 = O.quantize(W, 32, bits)
    c64, a64, b64 = O.quantize_fp64_shadow(W, 32, bits)
    assert np.array_equal(b32.astype(np.float64), b64)
    assert np.allclose(a32, a64, rtol=1e-6, atol=0)
    differ = int((c32 != c64).sum())
    assert differ <= 2                       # only possible within ~1e-6 of a half
    assert np.all(np.abs(c32.astype(int) - c64.astype(int)) <= 1)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_requantizing_dequantized_weights_reproduces_codes(bits):
    rng = np.random.default_rng(11 + bits)
    W = (rng.standard_normal((128, 24)) * 0.02).astype(np.float32)
    codes, alpha, beta = O.quantize(W, 32, bits)
    Wt = O.dequantize(codes, alpha, beta, 32).astype(np.float32)
    codes2, alpha2, beta2 = O.quantize(Wt, 32, bits)
    assert np.array_equal(codes, codes2)
    assert np.array_equal(beta, beta2)
    assert np.all(np.abs(alpha2 - alpha) <= 2 * np.spacing(alpha))


def test_constant_group_and_column_wise_special_cases():
    W = np.full((64, 3), 0.125, dtype=np.float32)
    W[32:, 1] = np.linspace(-1, 1, 32, dtype=np.float32)
    codes, alpha, beta = O.quantize(W, 32, 4)
    assert np.all(codes[:32] == 0) and np.all(alpha[0] == 1) and np.all(beta[0] == 0.125)
    assert np.array_equal(O.dequantize(codes, alpha, beta, 32)[:32], W[:32].astype(np.float64))
    # g = K is the paper's column-wise quantization (Section 3.1): one pair per column
    rng = np.random.default_rng(5)
    W = rng.standard_normal((96, 5)).astype(np.float32)
    codes, alpha, beta = O.quantize(W, 96, 3)
    assert alpha.shape == (1, 5)
    assert np.array_equal(beta[0], W.min(axis=0))
    assert np.allclose(alpha[0], (W.max(axis=0) - W.min(axis=0)) / 7, rtol=1e-6)


def test_rejects_bad_arguments():
    W = np.zeros((64, 4), dtype=np.float32)
    with pytest.raises(ValueError):
        O.quantize(W, 48, 4)
    with pytest.raises(ValueError):
        O.quantize(W, 32, 5)
    Wn = W.copy()
    Wn[3, 1] = np.inf
    with pytest.raises(ValueError):
        O.quantize(Wn, 32, 4)


# ------------------------------------------------------------------- layer ---
def test_pool_is_a_plain_group_sum():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 24))
    xp = O.pool(x, 8)
    for m in range(5):
        for q in range(3):
            assert abs(xp[m, q] - sum(x[m, 8 * q + i] for i in range(8))) < 1e-12
    # Algorithm 1 writes it as an average pool times the window length
    assert np.allclose(xp, x.reshape(5, 3, 8).mean(axis=2) * 8, rtol=1e-13)


@pytest.mark.parametrize("bits,g", [(4, 32), (3, 32), (2, 64), (4, 128)])
def test_merge_invariant(bits, g):
    """The merged plain quantized layer reproduces the unmerged QA-LoRA output
    (Appendix B Eq. 7), and the zero-point form printed in Algorithm 1 is the
    same update."""
    rng = np.random.default_rng(21 + bits + g)
    K, N, r, M = 2 * g if g >= 64 else 4 * g, 20, 6, 9
    W, codes, alpha, beta, x, A, B, _ = _rand_layer(rng, K, N, g, bits, r, M)
    s = 1.7
    y = O.forward(x, codes, alpha, beta, g, A, B, s)
    beta2 = O.merge(beta, A, B, s)
    y2 = O.forward(x, codes, alpha, beta2, g)            # rank 0: plain quantized layer
    assert np.max(np.abs(y - y2)) <= 1e-12 * np.max(np.abs(y))
    assert np.max(np.abs(y - O.forward(x, codes, alpha, beta, g))) > 1e-3   # adapter is not a no-op
    # zero-point form: W~ = alpha*(c - z), z = -beta/alpha, z' = z - s*A@B/alpha
    a64 = alpha.astype(np.float64)
    z2 = O.merge_zero_point(-beta.astype(np.float64) / a64, a64, A, B, s)
    assert np.allclose(-z2 * a64, beta2, rtol=1e-12, atol=1e-15)
    Wz = np.repeat(a64, g, axis=0) * (codes.astype(np.float64) - np.repeat(z2, g, axis=0))
    assert np.max(np.abs(x @ Wz - y)) <= 1e-11 * np.max(np.abs(y))


def test_effective_update_structure_and_rank_bound():
    rng = np.random.default_rng(33)
    K, N, g, r, M = 48, 10, 8, 4, 6
    W, codes, alpha, beta, x, A, B, _ = _rand_layer(rng, K, N, g, 4, r, M)
    s = 0.5
    E = np.zeros((K, K // g))
    for k in range(K):
        E[k, k // g] = 1.0
    dW = s * E @ A @ B                                   # dense effective update
    y_lora = O.forward(x, codes, alpha, beta, g, A, B, s) - O.forward(x, codes, alpha, beta, g)
    assert np.allclose(y_lora, x @ dW, rtol=1e-11, atol=1e-12)
    for k in range(K):                                   # rows equal inside a group
        assert np.array_equal(dW[k], dW[(k // g) * g])
    assert np.linalg.matrix_rank(dW) <= min(r, K // g)
    # one group per column: every row of the update is the same vector, rank <= 1 (Section 3.3)
    A1 = rng.standard_normal((1, r))
    dW1 = s * np.ones((K, 1)) @ A1 @ B
    c1, a1, b1 = O.quantize(W, K, 4)
    y1 = O.forward(x, c1, a1, b1, K, A1, B, s) - O.forward(x, c1, a1, b1, K)
    assert np.allclose(y1, x @ dW1, rtol=1e-11, atol=1e-12)
    assert np.linalg.matrix_rank(dW1) <= 1


def test_group_size_one_is_plain_lora():
    """g = 1: every group is constant, W~ = W exactly, the pool is the identity,
    and the layer is y = x W + s x A B (Section 3.1)."""
    rng = np.random.default_rng(44)
    K, N, r, M = 12, 7, 3, 5
    W = rng.standard_normal((K, N)).astype(np.float32)
    codes, alpha, beta = O.quantize(W, 1, 4)
    assert np.all(codes == 0)
    x = rng.standard_normal((M, K)); A = rng.standard_normal((K, r)); B = rng.standard_normal((r, N))
    y = O.forward(x, codes, alpha, beta, 1, A, B, 0.3)
    assert np.allclose(y, x @ W.astype(np.float64) + 0.3 * x @ A @ B, rtol=1e-12, atol=1e-12)
    # s = 0 and A = 0 both give the plain quantized layer
    c2, a2, b2 = O.quantize(W, 4, 4)
    A2 = rng.standard_normal((3, r))
    base = x @ O.dequantize(c2, a2, b2, 4)
    assert np.array_equal(O.forward(x, c2, a2, b2, 4, A2, B, 0.0), base)
    assert np.array_equal(O.forward(x, c2, a2, b2, 4, np.zeros_like(A2), B, 2.0), base)


def test_forward_backward_equal_dense_matmul_with_effective_weight():
    rng = np.random.default_rng(55)
    K, N, g, r, M = 64, 12, 16, 5, 7
    W, codes, alpha, beta, x, A, B, dy = _rand_layer(rng, K, N, g, 3, r, M)
    s = 1.3
    Weff = O.dequantize(codes, alpha, beta, g) + s * np.repeat(A @ B, g, axis=0)
    assert np.allclose(O.forward(x, codes, alpha, beta, g, A, B, s), x @ Weff, rtol=1e-12, atol=1e-12)
    dX, dA, dB = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    assert np.allclose(dX, dy @ Weff.T, rtol=1e-12, atol=1e-12)
    dP = s * O.pool(x, g).T @ dy                          # gradient w.r.t. P = A @ B
    assert np.allclose(dA, dP @ B.T, rtol=1e-12, atol=1e-12)
    assert np.allclose(dB, A.T @ dP, rtol=1e-12, atol=1e-12)


def test_backward_by_finite_differences_and_adjoint():
    rng = np.random.default_rng(66)
    K, N, g, r, M = 32, 6, 8, 3, 4
    W, codes, alpha, beta, x, A, B, dy = _rand_layer(rng, K, N, g, 4, r, M)
    s = 0.7

    def loss(x_, A_, B_):
        return float(np.sum(dy * O.forward(x_, codes, alpha, beta, g, A_, B_, s)))

    dX, dA, dB = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    h = 1e-3                                             # l is linear in each argument: differences are exact
    for arr, grad, which in ((x, dX, 0), (A, dA, 1), (B, dB, 2)):
        for idx in itertools.product(*(range(n) for n in arr.shape)):
            p = arr.copy(); p[idx] += h
            m = arr.copy(); m[idx] -= h
            args_p = [x, A, B]; args_p[which] = p
            args_m = [x, A, B]; args_m[which] = m
            fd = (loss(*args_p) - loss(*args_m)) / (2 * h)
            assert abs(fd - grad[idx]) <= 1e-8 * max(1.0, abs(grad[idx])), (which, idx)
    # adjoint identity <dy, J u> = <J^T dy, u> for the map x -> y
    u = rng.standard_normal(x.shape)
    Ju = O.forward(u, codes, alpha, beta, g, A, B, s)
    assert abs(np.sum(dy * Ju) - np.sum(dX * u)) <= 1e-10 * abs(np.sum(dy * Ju))


def test_a_planted_transpose_or_sign_error_would_be_caught():
    """The pins above are only useful if plausible mistakes fail them: plant three."""
    rng = np.random.default_rng(77)
    K, N, g, r, M = 32, 6, 8, 3, 4
    W, codes, alpha, beta, x, A, B, dy = _rand_layer(rng, K, N, g, 4, r, M)
    s = 0.9
    y = O.forward(x, codes, alpha, beta, g, A, B, s)
    wrong_sign = O.forward(x, codes, alpha, O.merge(beta, A, B, -s), g)
    assert np.max(np.abs(y - wrong_sign)) > 1e-3
    mean_pool = x @ O.dequantize(codes, alpha, beta, g) + s * (O.pool(x, g) / g) @ A @ B
    assert np.max(np.abs(y - mean_pool)) > 1e-3
    dX, dA, dB = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    assert np.max(np.abs(dB - (O.pool(x, g) @ A).T @ dy)) > 1e-3        # dropped s


# ------------------------------------------------------------------ packing --
@pytest.mark.parametrize("row", list(_rows("pack_words.txt")))
def test_pack_hand_written_words(row):
    bits, rule, words = row
    codes = np.array([eval(rule, {"j": j}) for j in range(32)], dtype=np.uint8).reshape(32, 1)
    want = np.array([int(w, 16) for w in words.split()], dtype=np.uint32)
    got = O.pack(codes, int(bits))
    assert got.shape == (1, 1, O.words_per_unit(int(bits)))
    assert np.array_equal(got[0, 0], want)
    assert np.array_equal(O.unpack(got, int(bits)), codes)


@pytest.mark.parametrize("bits", [2, 3, 4])
def test_pack_round_trip_and_independence_of_positions(bits):
    rng = np.random.default_rng(bits)
    codes = rng.integers(0, 2 ** bits, size=(96, 5), dtype=np.uint8)
    packed = O.pack(codes, bits)
    assert packed.dtype == np.uint32 and packed.shape == (3, 5, O.words_per_unit(bits))
    assert np.array_equal(O.unpack(packed, bits), codes)
    # every (position, bit) lands on its own packed bit: one-hot codes give
    # one-hot words, all distinct
    seen = set()
    for j in range(32):
        for bit in range(bits):
            c = np.zeros((32, 1), dtype=np.uint8); c[j, 0] = 1 << bit
            w = O.pack(c, bits)[0, 0]
            nz = [(i, int(v)) for i, v in enumerate(w) if v]
            assert len(nz) == 1 and bin(nz[0][1]).count("1") == 1
            seen.add(nz[0])
    assert len(seen) == 32 * bits
    with pytest.raises(ValueError):
        O.pack(np.full((32, 1), 2 ** bits, dtype=np.uint8), bits)


# ------------------------------------------------------------------ Table 2 --
@pytest.mark.parametrize("row", list(_rows("table2_params.txt")))
def test_param_counts_reproduce_table_2(row):
    model, layers, hidden, mlp, qlora_m, qalora_m = row
    layers, h, f = int(layers), int(hidden), int(mlp)
    linears = [(h, h)] * 4 + [(h, f), (h, f), (f, h)]     # q k v o gate up down
    qalora = layers * sum(O.adapter_param_count(K, N, 32, 64) for K, N in linears)
    qlora = layers * sum(O.adapter_param_count(K, N, 1, 64) for K, N in linears)
    assert round(qalora / 1e6) == int(qalora_m)
    assert round(qlora / 1e6) == int(qlora_m)


def test_zero_point_form_of_algorithm_1():
    """Algorithm 1 writes the layer as alpha * (c - z); Eq. 1 as alpha * c + beta.  A hand-worked
    asymmetric INT4 example with an integer zero point, the conversion in both directions, and
    a sign error that must be caught."""
    # scale 0.5, integer zero point 6: codes 0, 6, 15 stand for -3, 0 and 4.5
    codes = np.array([[0], [6], [15], [8]], dtype=np.uint8)
    alpha, z = np.array([[0.5]]), np.array([[6.0]])
    np.testing.assert_array_equal(O.dequantize_zero_point(codes, alpha, z, 4).ravel(), [-3.0, 0.0, 4.5, 1.0])
    beta = O.beta_from_zero_point(alpha, z)
    assert beta[0, 0] == -3.0                                  # the weight that code 0 stands for
    np.testing.assert_array_equal(O.dequantize(codes, alpha, beta, 4).ravel(), [-3.0, 0.0, 4.5, 1.0])
    assert O.zero_point_from_beta(alpha, beta)[0, 0] == 6.0
    # random layers: both forms give the same weights, and the round trip is the identity
    rng = np.random.default_rng(77)
    W, codes, alpha, beta, *_ = _rand_layer(rng, 64, 12, 32, 4, 4, 3)
    z = O.zero_point_from_beta(alpha, beta)
    ref = O.dequantize(codes, alpha, beta, 32)
    assert np.max(np.abs(O.dequantize_zero_point(codes, alpha, z, 32) - ref)) <= 1e-12 * np.max(np.abs(ref))
    np.testing.assert_allclose(O.beta_from_zero_point(alpha, z), beta, rtol=1e-14)
    assert np.max(np.abs(O.dequantize_zero_point(codes, alpha, -z, 32) - ref)) > 1e-3      # planted sign error
    with pytest.raises(ValueError):
        O.zero_point_from_beta(np.zeros((1, 1)), np.ones((1, 1)))
