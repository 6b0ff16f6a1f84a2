"""Parity of the format conversions with the oracle: whole-matrix dequantization (Eq. 1) and
Algorithm 1's zero-point form.  The packed codes and the factors are the ORACLE's, uploaded;
nothing the GPU produced is fed to the oracle."""
import numpy as np
import pytest
import torch

from oracle import qalora_oracle as O
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import LayerConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu

TOL = 5e-3


def _oracle_layer(cfg):
    t = make_inputs(cfg)
    codes, alpha, beta = O.quantize(t["W"].numpy(), cfg.group_size, cfg.bits)
    packed = torch.from_numpy(O.pack(codes, cfg.bits).view(np.int32)).cuda()
    qparams = torch.from_numpy(np.stack([alpha, beta], axis=-1).astype(np.float32)).cuda()
    return t, codes, alpha, beta, packed, qparams


@pytest.mark.parametrize("K,N,g,bits", [(64, 64, 32, 4), (320, 200, 32, 4), (192, 136, 64, 3), (256, 72, 128, 2),
                                        (1024, 1000, 32, 3), (2048, 264, 64, 2), (4096, 4096, 32, 4), (5120, 2048, 128, 3)])
def test_dequantize_is_the_rounded_oracle_value(K, N, g, bits):
    cfg = LayerConfig("deq", K, N, g, bits, 8, 1.0, 4, outlier_frac=0.01, seed=K + bits)
    _, codes, alpha, beta, packed, qparams = _oracle_layer(cfg)
    d = Q.desc(K, N, g, bits, 8, 1.0)
    ref = O.dequantize(codes, alpha, beta, g)            # exact in fp64: alpha * c has at most 28 bits
    W32 = torch.full((K, N), float("nan"), dtype=torch.float32, device="cuda")
    Q.qalora_dequantize(d, packed, qparams, W32)
    Wb = torch.zeros((K, N), dtype=torch.bfloat16, device="cuda")
    Q.qalora_dequantize(d, packed, qparams, Wb)
    torch.cuda.synchronize()
    ref32 = torch.from_numpy(ref.astype(np.float32))     # one rounding, as the kernel's fused multiply-add
    assert torch.equal(W32.cpu(), ref32)
    assert torch.equal(Wb.cpu(), ref32.to(torch.bfloat16))


def test_zero_point_import_export_and_forward():
    # an asymmetric INT4 layer given in Algorithm 1's form with INTEGER zero points
    K, N, g, bits, M = 256, 128, 32, 4, 9
    rng = np.random.default_rng(12)
    G = K // g
    codes = rng.integers(0, 16, size=(K, N)).astype(np.uint8)
    alpha = (rng.uniform(0.5, 2.0, size=(G, N)) * 1e-2).astype(np.float32)
    zero = rng.integers(0, 16, size=(G, N)).astype(np.float32)
    d = Q.desc(K, N, g, bits, 0, 1.0)
    qparams = torch.zeros((G, N, 2), dtype=torch.float32, device="cuda")
    Q.qalora_qparams_from_zero_point(d, torch.from_numpy(alpha).cuda(), torch.from_numpy(zero).cuda(), qparams)
    torch.cuda.synchronize()
    qp = qparams.cpu().numpy()
    assert np.array_equal(qp[..., 0], alpha)
    # -alpha * z is exact in fp64, so its float32 rounding is the kernel's single multiply
    assert np.array_equal(qp[..., 1], O.beta_from_zero_point(alpha, zero).astype(np.float32))
    # the imported layer computes x * alpha * (c - z)
    x = torch.randn(M, K, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = Q.alloc_workspace(d, M, Q.OP_FORWARD)
    packed = torch.from_numpy(O.pack(codes, bits).view(np.int32)).cuda()
    Q.qalora_forward(d, M, x.cuda(), packed, qparams, None, None, y, ws)
    torch.cuda.synchronize()
    y_ref = to_f64(x) @ O.dequantize_zero_point(codes, alpha, zero, g)
    assert np.max(np.abs(y.float().cpu().numpy() - y_ref)) <= TOL * np.max(np.abs(y_ref))
    # export gives the zero points back, up to the float32 rounding of beta (one ulp of z)
    a2, z2 = torch.zeros((G, N), device="cuda"), torch.zeros((G, N), device="cuda")
    Q.qalora_qparams_to_zero_point(d, qparams, a2, z2)
    torch.cuda.synchronize()
    assert np.array_equal(a2.cpu().numpy(), alpha)
    np.testing.assert_allclose(z2.cpu().numpy(), zero, rtol=1.2e-7, atol=0)
    np.testing.assert_allclose(z2.cpu().numpy(), O.zero_point_from_beta(alpha, qp[..., 1]), rtol=1.2e-7, atol=0)


def test_merge_in_zero_point_form_matches_algorithm_1():
    # z' = z - s * A B / alpha (Algorithm 1, merge_with_quantization) through import -> merge -> export
    cfg = LayerConfig("zpmerge", 256, 128, 64, 4, 16, 1.5, 4, seed=8)
    t, codes, alpha, beta, packed, qparams = _oracle_layer(cfg)
    d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, cfg.rank, cfg.scale)
    A, B = to_f64(t["A"]), to_f64(t["B"])
    z = O.zero_point_from_beta(alpha, beta)
    z_ref = O.merge_zero_point(z, alpha, A, B, cfg.scale)
    q2 = torch.empty_like(qparams)
    Q.qalora_merge(d, qparams, t["A"].cuda(), t["B"].cuda(), q2)
    a2, z2 = torch.zeros_like(q2[..., 0]).contiguous(), torch.zeros_like(q2[..., 0]).contiguous()
    Q.qalora_qparams_to_zero_point(d, q2, a2, z2)
    torch.cuda.synchronize()
    assert np.array_equal(a2.cpu().numpy(), alpha)
    assert np.max(np.abs(z2.cpu().numpy() - z_ref)) <= 1e-5 * np.max(np.abs(z_ref))


def test_format_calls_reject_bad_arguments():
    d = Q.desc(64, 64, 32, 4, 0, 1.0)
    codes, qparams = Q.alloc_packed(d)
    W = torch.zeros((64, 64), device="cuda")
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_dequantize(d, None, qparams, W)
    assert e.value.status == -2
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_dequantize(d, codes, qparams, W.view(-1)[1:])
    assert e.value.status == -4
    with pytest.raises(ValueError):
        Q.qalora_dequantize(d, codes, qparams, W.half())
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_qparams_to_zero_point(d, qparams, None, W)
    assert e.value.status == -2
