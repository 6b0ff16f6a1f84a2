"""Parity at the benchmark's full sizes, in the launch configuration bench.py
times: every shape x bit width of the 13B configuration, every shape x group size
of the 65B configuration, and both 7B MLP shapes.

Codes, packed words and (alpha, beta) are compared in full.  y and dX are compared
on ALL token rows for the 7B and 13B shapes; for the 65B shapes (where the fp64
oracle would need tens of seconds per case) on a seeded sample of token rows: rows
are independent, so the oracle evaluates exactly those rows.  dA, dB and the merged
zeros are compared in full everywhere (the oracle adds the adapter gradients over
row blocks).  The few-token forward is checked at full size too: the merged layer
at one token, and the adapted layer (rank 64) at 1 and 16 tokens.

Every comparison goes through `record_margin`, which keeps the worst
max|err| / max|ref| per case and output for the summary at the end of the run."""
import numpy as np
import pytest
import torch

from conftest import record_margin
from oracle import qalora_oracle as O
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import CONFIGS, LayerConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu
TOL = 5e-3
SAMPLE_ROWS = 48


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


CASES = [("cfg3_7b_up", {}), ("cfg3_7b_down", {})]
CASES += [(n, {"bits": b}) for n in ("cfg4_13b_up", "cfg4_13b_down", "cfg4_13b_attn") for b in (3, 2)]
CASES += [(n, {"group_size": g}) for n in ("cfg5_65b_up", "cfg5_65b_down", "cfg5_65b_attn") for g in (32, 64, 128)]


def case_id(c):
    return c[0] + "".join(f"_{k[0]}{v}" for k, v in c[1].items())


@pytest.mark.parametrize("name,over", CASES, ids=[case_id(c) for c in CASES])
def test_full_size_layer(name, over):
    case = case_id((name, over))
    cfg = CONFIGS[name].with_(**over)
    all_rows = not name.startswith("cfg5")            # the 65B shapes keep the row sample
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
    del dev["W"], cpu["W"]

    A, B = to_f64(cpu["A"]), to_f64(cpu["B"])
    if all_rows:
        rows = np.arange(M)
    else:
        rows = np.unique(np.concatenate([[0, M - 1, 255, 256], np.random.default_rng(cfg.seed).integers(0, M, SAMPLE_ROWS)]))
    rows_t = torch.from_numpy(rows)
    y_got = y[rows_t.cuda()].cpu()
    dx_got = dx[rows_t.cuda()].cpu()
    y_err = dx_err = y_max = dx_max = 0.0
    y_first = None
    for b0 in range(0, len(rows), 2048):               # row blocks keep the fp64 temporaries small
        rb = rows_t[b0:b0 + 2048]
        xs, dys = to_f64(cpu["x"][rb]), to_f64(cpu["dy"][rb])
        y_ref = O.forward(xs, codes, alpha, beta, g, A, B, s)
        dx_ref, _, _ = O.backward(xs, dys, codes, alpha, beta, g, A, B, s)
        if y_first is None:
            y_first = y_ref[:1].copy()
        y_err = max(y_err, float(np.max(np.abs(y_got[b0:b0 + 2048].double().numpy() - y_ref))))
        dx_err = max(dx_err, float(np.max(np.abs(dx_got[b0:b0 + 2048].double().numpy() - dx_ref))))
        y_max = max(y_max, float(np.max(np.abs(y_ref))))
        dx_max = max(dx_max, float(np.max(np.abs(dx_ref))))
    record_margin(case, "y", y_err / y_max, TOL)
    record_margin(case, "dX", dx_err / dx_max, TOL)

    dA_ref = np.zeros((G, r)); dB_ref = np.zeros((r, N))
    for m0 in range(0, M, 1024):                          # sums over token rows: add row blocks
        a, b = O.backward_adapter(to_f64(cpu["x"][m0:m0 + 1024]), to_f64(cpu["dy"][m0:m0 + 1024]), g, A, B, s)
        dA_ref += a; dB_ref += b
    record_margin(case, "dA", rel_err(dA.cpu().numpy(), dA_ref), TOL)
    record_margin(case, "dB", rel_err(dB.cpu().numpy(), dB_ref), TOL)
    q2n = q2.cpu().numpy()
    assert np.array_equal(q2n[..., 0], alpha)
    record_margin(case, "beta_merged", rel_err(q2n[..., 1], O.merge(beta, A, B, s)), TOL)

    # the deployed layer at one token (the few-token kernel at full size) reproduces the adapted output
    d0 = Q.desc(K, N, g, cfg.bits, 0, s)
    x1 = dev["x"][rows_t[:1].cuda()].contiguous()
    y1 = torch.empty((1, N), dtype=torch.bfloat16, device="cuda")
    w1 = Q.alloc_workspace(d0, 1, Q.OP_FORWARD)
    Q.qalora_forward(d0, 1, x1, codes_d, q2, None, None, y1, w1)
    torch.cuda.synchronize()
    assert Q.qalora_main_kernel_name() == "qalora_gemv_kernel"
    record_margin(case, "y_merged_m1", rel_err(y1.float().cpu().numpy(), y_first), TOL)

    # the adapted layer (rank r) on the few-token path at full size: 1 and 16 tokens
    rows16 = rows_t[:16] if len(rows_t) >= 16 else rows_t
    y16_ref = O.forward(to_f64(cpu["x"][rows16]), codes, alpha, beta, g, A, B, s)
    for m in (1, 16):
        xm = dev["x"][rows16[:m].cuda()].contiguous()
        ym = torch.empty((m, N), dtype=torch.bfloat16, device="cuda")
        wm = Q.alloc_workspace(d, m, Q.OP_FORWARD)
        Q.qalora_forward(d, m, xm, codes_d, qparams, dev["A"], dev["B"], ym, wm)
        torch.cuda.synchronize()
        assert Q.qalora_main_kernel_name() == "qalora_gemv_kernel" and Q.workspace_status(wm) == 0
        record_margin(case, f"y_adapted_m{m}", rel_err(ym.float().cpu().numpy(), y16_ref[:m]), TOL)


@pytest.mark.parametrize("name", ["cfg3_7b_up", "cfg3_7b_down"])
def test_two_hundred_thousand_rows_index_past_2_to_the_31(name):
    """200 000 token rows on the 7B MLP shapes: y (4096 -> 11008) resp. x and dX (11008 -> 4096)
    hold 2.2e9 elements, so every element offset of their last rows lies beyond 2^31 (and the
    byte offsets beyond 2^32).  The fp64 oracle cannot take this size, so the check is by
    properties that hold at any size: rows are independent in y and dX, hence the first and the
    last 256 rows must agree with a 256-row call on those rows alone (the paths checked against
    the oracle above); dA and dB are sums over the rows, hence equal to the sum of the results
    of eight 25 000-row calls.  x and dy are drawn on the device from a seeded generator."""
    cfg = CONFIGS[name]
    M, K, N, G, r, g, s = 200_000, cfg.d_in, cfg.d_out, cfg.groups, cfg.rank, cfg.group_size, cfg.scale
    assert M * max(K, N) > 2 ** 31
    cpu = make_inputs(cfg, need=("W", "A", "B"))
    d = Q.desc(K, N, g, cfg.bits, r, s)
    W, A, B = cpu["W"].cuda(), cpu["A"].cuda(), cpu["B"].cuda()
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, W, codes, qparams)
    del W
    gen = torch.Generator(device="cuda")
    gen.manual_seed(1234 + K)
    x = torch.empty((M, K), dtype=torch.bfloat16, device="cuda").normal_(0.0, 1.0, generator=gen)
    dy = torch.empty((M, N), dtype=torch.bfloat16, device="cuda").normal_(0.0, cfg.dy_std, generator=gen)

    def run(xs, dys):
        m = xs.shape[0]
        y = torch.empty((m, N), dtype=torch.bfloat16, device="cuda")
        dx = torch.empty((m, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.empty((G, r), dtype=torch.float32, device="cuda")
        dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
        ws = Q.alloc_workspace(d, m, Q.OP_TRAIN)
        Q.qalora_forward_train(d, m, xs, codes, qparams, A, B, y, ws)
        Q.qalora_backward_train(d, m, xs, dys, codes, qparams, A, B, dx, dA, dB, ws)
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0
        return y, dx, dA, dB

    y, dx, dA, dB = run(x, dy)
    case = f"{name}_m200000"
    for lo in (0, M - 256):
        ys, dxs, _, _ = run(x[lo:lo + 256].contiguous(), dy[lo:lo + 256].contiguous())
        # (the 256-row call cuts its reduction into parts: another summation order, within one bf16 step)
        record_margin(case, f"y_rows_{lo}", rel_err(y[lo:lo + 256].float().cpu().numpy(), ys.float().cpu().numpy()), 4e-3)
        record_margin(case, f"dX_rows_{lo}", rel_err(dx[lo:lo + 256].float().cpu().numpy(), dxs.float().cpu().numpy()), 4e-3)
    dA_sum = torch.zeros((G, r), dtype=torch.float64, device="cuda")
    dB_sum = torch.zeros((r, N), dtype=torch.float64, device="cuda")
    for lo in range(0, M, 25_000):
        _, _, dA_c, dB_c = run(x[lo:lo + 25_000], dy[lo:lo + 25_000])
        dA_sum += dA_c.double()
        dB_sum += dB_c.double()
    record_margin(case, "dA_additive", rel_err(dA.cpu().numpy(), dA_sum.cpu().numpy()), 1e-4)
    record_margin(case, "dB_additive", rel_err(dB.cpu().numpy(), dB_sum.cpu().numpy()), 1e-3)


VOCAB = 128256     # 1002 channel tiles of 128


@pytest.mark.parametrize("K,N", [(4096, VOCAB), (VOCAB, 4096)], ids=["to_vocabulary", "from_vocabulary"])
def test_vocabulary_sized_dimension(K, N):
    """A layer with 128256 output resp. input channels (an output head, an embedding-sized input):
    a thousand channel tiles, 525 M weights.  The oracle quantizes and contracts what it is
    asked for, so it is asked for samples that are exact by themselves: y on three ranges of
    output columns (a column of y needs that column of W alone), dX on three quantization groups
    of input channels (a channel of dX needs that row group of W alone), codes and (alpha, beta)
    on both samples, dA and dB in full (they do not involve W)."""
    g, bits, r, s, M = 32, 4, 64, 1.0, 300
    case = f"vocab_{K}x{N}"
    cfg = LayerConfig(case, K, N, g, bits, r, s, M, seed=91)
    cpu = make_inputs(cfg)
    d = Q.desc(K, N, g, bits, r, s)
    dev = {k: v.cuda() for k, v in cpu.items() if k != "W"}
    codes_d, qparams = Q.alloc_packed(d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    W_dev = cpu["W"].cuda()
    Q.qalora_quantize(d, W_dev, codes_d, qparams, status)
    del W_dev
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    words = codes_d.cpu().numpy().view(np.uint32).reshape(K // 32, N, -1)
    qp = qparams.cpu().numpy().reshape(K // g, N, 2)
    Wn = cpu["W"].numpy()
    x, A, B, dy = (to_f64(cpu[k]) for k in ("x", "A", "B", "dy"))

    # ---- output-column sample: quantization, forward (300, 16 and 1 rows), merge + merged forward
    cols = np.r_[0:256, N // 2 + 37:N // 2 + 237, N - 256:N]
    codes, alpha, beta = O.quantize(np.ascontiguousarray(Wn[:, cols]), g, bits)
    assert np.array_equal(words[:, cols, :], O.pack(codes, bits).reshape(K // 32, len(cols), -1))
    assert np.array_equal(qp[:, cols, 0], alpha) and np.array_equal(qp[:, cols, 1], beta)
    y_ref = O.forward(x, codes, alpha, beta, g, A, B[:, cols], s)
    q2 = torch.empty_like(qparams)
    Q.qalora_merge(d, qparams, dev["A"], dev["B"], q2)
    record_margin(case, "beta_merged", rel_err(q2.cpu().numpy().reshape(K // g, N, 2)[:, cols, 1], O.merge(beta, A, B[:, cols], s)), TOL)
    d0 = Q.desc(K, N, g, bits, 0, s)
    for m in (300, 16, 1):
        xm = dev["x"][:m].contiguous()
        y = torch.empty((m, N), dtype=torch.bfloat16, device="cuda")
        Q.qalora_forward(d, m, xm, codes_d, qparams, dev["A"], dev["B"], y, Q.alloc_workspace(d, m, Q.OP_FORWARD))
        record_margin(case, f"y_m{m}", rel_err(y.float().cpu().numpy()[:, cols], y_ref[:m]), TOL)
        Q.qalora_forward(d0, m, xm, codes_d, q2, None, None, y, Q.alloc_workspace(d0, m, Q.OP_FORWARD))
        record_margin(case, f"y_merged_m{m}", rel_err(y.float().cpu().numpy()[:, cols], y_ref[:m]), TOL)

    # ---- input-channel sample (whole quantization groups): quantization and dX; dA, dB in full
    groups = np.array([0, (K // g) // 2 + 3, K // g - 1])
    rows = (groups[:, None] * g + np.arange(g)[None, :]).reshape(-1)
    codes_k, alpha_k, beta_k = O.quantize(np.ascontiguousarray(Wn[rows, :]), g, bits)
    assert np.array_equal(words[groups * (g // 32)], O.pack(codes_k, bits).reshape(len(groups), N, -1))
    assert np.array_equal(qp[groups, :, 0], alpha_k) and np.array_equal(qp[groups, :, 1], beta_k)
    dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dA = torch.empty((K // g, r), dtype=torch.float32, device="cuda")
    dB = torch.empty((r, N), dtype=torch.float32, device="cuda")
    wb = Q.alloc_workspace(d, M, Q.OP_BACKWARD)
    Q.qalora_backward(d, M, dev["x"], dev["dy"], codes_d, qparams, dev["A"], dev["B"], dx, dA, dB, wb)
    torch.cuda.synchronize()
    assert Q.workspace_status(wb) == 0
    dx_ref, _, _ = O.backward(x[:, rows], dy, codes_k, alpha_k, beta_k, g, A[groups], B, s)
    record_margin(case, "dX", rel_err(dx.float().cpu().numpy()[:, rows], dx_ref), TOL)
    dA_ref, dB_ref = O.backward_adapter(x, dy, g, A, B, s)
    record_margin(case, "dA", rel_err(dA.cpu().numpy(), dA_ref), TOL)
    record_margin(case, "dB", rel_err(dB.cpu().numpy(), dB_ref), TOL)
