"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times.  Codes, packed words and (alpha, beta) are compared in full; y and dX on
a seeded sample of token rows (rows are independent, so the oracle evaluates
exactly those rows); dA, dB and the merged zeros in full (the oracle adds the
adapter gradients over row blocks)."""
import numpy as np
import pytest
import torch

from oracle import qalora_oracle as O
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import CONFIGS, make_inputs, to_f64

pytestmark = pytest.mark.gpu
TOL = 5e-3
SAMPLE_ROWS = 48


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


CASES = [
    # config, overrides
    ("cfg3_7b_up", {}),
    ("cfg3_7b_down", {}),
    ("cfg4_13b_up", {"bits": 3}),
    ("cfg4_13b_down", {"bits": 2}),
    ("cfg4_13b_attn", {"bits": 2}),
    ("cfg5_65b_attn", {"group_size": 64}),
    ("cfg5_65b_down", {"group_size": 128}),
    ("cfg5_65b_up", {}),
]


@pytest.mark.parametrize("name,over", CASES, ids=[c[0] + "".join(f"_{k[0]}{v}" for k, v in c[1].items()) for c in CASES])
def test_full_size_layer(name, over):
    cfg = CONFIGS[name].with_(**over)
    cpu = make_inputs(cfg)
    M, K, N, G, r, g, s = cfg.tokens, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank, cfg.group_size, cfg.scale
    d = Q.desc(K, N, g, cfg.bits, r, s)
    dev = {k: v.cuda() for k, v in cpu.items()}
    codes_d, qparams = Q.alloc_packed(d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Q.qalora_quantize(d, dev["W"], codes_d, qparams, status)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    wf = Q.alloc_workspace(d, M, Q.OP_FORWARD)
    Q.qalora_forward(d, M, dev["x"], codes_d, qparams, dev["A"], dev["B"], y, wf)
    assert Q.qalora_main_kernel_name() == "qalora_tc_kernel<fwd>"
    dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dA = torch.empty((G, r), dtype=torch.float32, device="cuda")
    dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
    wb = Q.alloc_workspace(d, M, Q.OP_BACKWARD)
    Q.qalora_backward(d, M, dev["x"], dev["dy"], codes_d, qparams, dev["A"], dev["B"], dx, dA, dB, wb)
    assert Q.qalora_main_kernel_name() == "qalora_tc_kernel<dx>"
    q2 = torch.empty_like(qparams)
    Q.qalora_merge(d, qparams, dev["A"], dev["B"], q2)
    torch.cuda.synchronize()
    assert Q.workspace_status(wf) == 0 and Q.workspace_status(wb) == 0 and int(status.item()) == 0

    # integer work: bit-exact, in full
    codes, alpha, beta = O.quantize(cpu["W"].numpy(), g, cfg.bits)
    assert np.array_equal(codes_d.cpu().numpy().view(np.uint32), O.pack(codes, cfg.bits))
    qp = qparams.cpu().numpy()
    assert np.array_equal(qp[..., 0], alpha) and np.array_equal(qp[..., 1], beta)
    del dev["W"]

    A, B = to_f64(cpu["A"]), to_f64(cpu["B"])
    rows = np.unique(np.concatenate([[0, M - 1, 255, 256], np.random.default_rng(cfg.seed).integers(0, M, SAMPLE_ROWS)]))
    rows_t = torch.from_numpy(rows)
    xs, dys = to_f64(cpu["x"][rows_t]), to_f64(cpu["dy"][rows_t])
    y_ref = O.forward(xs, codes, alpha, beta, g, A, B, s)
    assert rel_err(y[rows_t.cuda()].float().cpu().numpy(), y_ref) <= TOL
    dx_ref, _, _ = O.backward(xs, dys, codes, alpha, beta, g, A, B, s)
    assert rel_err(dx[rows_t.cuda()].float().cpu().numpy(), dx_ref) <= TOL

    dA_ref = np.zeros((G, r)); dB_ref = np.zeros((r, N))
    for m0 in range(0, M, 1024):                          # sums over token rows: add row blocks
        a, b = O.backward_adapter(to_f64(cpu["x"][m0:m0 + 1024]), to_f64(cpu["dy"][m0:m0 + 1024]), g, A, B, s)
        dA_ref += a; dB_ref += b
    assert rel_err(dA.cpu().numpy(), dA_ref) <= TOL
    assert rel_err(dB.cpu().numpy(), dB_ref) <= TOL
    q2n = q2.cpu().numpy()
    assert np.array_equal(q2n[..., 0], alpha)
    assert rel_err(q2n[..., 1], O.merge(beta, A, B, s)) <= TOL

    # the deployed layer at one token (the few-token kernel at full size) reproduces the adapted output
    d0 = Q.desc(K, N, g, cfg.bits, 0, s)
    x1 = dev["x"][rows_t[:1].cuda()].contiguous()
    y1 = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
    w1 = Q.alloc_workspace(d0, 1, Q.OP_FORWARD)
    Q.qalora_forward(d0, 1, x1, codes_d, q2, None, None, y1, w1)
    torch.cuda.synchronize()
    assert Q.qalora_main_kernel_name() == "qalora_gemv_kernel"
    assert rel_err(y1.float().cpu().numpy(), y_ref[:1]) <= TOL
