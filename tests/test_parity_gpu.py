"""Parity of the CUDA library (through its C ABI) against the CPU oracle on the
same seeded inputs.  Integer results (codes, packed words) and the quantization
parameters must be bit-exact; floating-point results must satisfy
max|gpu - ref| / max|ref| <= 5e-3 (bf16 inputs/outputs, fp32 accumulation)."""
import numpy as np
import pytest
import torch

from conftest import record_margin
from oracle import qalora_oracle as O
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import CONFIGS, LayerConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu
TOL = 5e-3


def rel_err(got, ref):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape
    if ref.size == 0:
        return 0.0
    denom = np.max(np.abs(ref))
    return float(np.max(np.abs(got - ref)) / (denom if denom > 0 else 1.0))


def margin(case, output, got, ref):
    """Compares one output with the oracle's and keeps the error for the end-of-run summary."""
    record_margin(case, output, rel_err(got, ref), TOL)


class GpuLayer:
    """Quantizes cfg's synthetic weights on the GPU and keeps everything on the device."""

    def __init__(self, cfg: LayerConfig, need=("W", "x", "A", "B", "dy")):
        self.cfg = cfg
        self.cpu = make_inputs(cfg, need=need)
        self.dev = {k: v.cuda() for k, v in self.cpu.items()}
        self.d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, cfg.rank, cfg.scale)
        self.codes, self.qparams = Q.alloc_packed(self.d)
        self.status = torch.zeros(1, dtype=torch.int32, device="cuda")
        Q.qalora_quantize(self.d, self.dev["W"], self.codes, self.qparams, self.status)
        torch.cuda.synchronize()

    def forward(self, x=None, qparams=None, rank=None):
        cfg = self.cfg
        x = self.dev["x"] if x is None else x
        d = self.d if rank is None else Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, rank, cfg.scale)
        m = x.shape[0]
        y = torch.empty((m, cfg.d_out), dtype=torch.bfloat16, device="cuda")
        ws = Q.alloc_workspace(d, m, Q.OP_FORWARD)
        Q.qalora_forward(d, m, x, self.codes, self.qparams if qparams is None else qparams,
                         self.dev.get("A") if d.rank else None, self.dev.get("B") if d.rank else None, y, ws)
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0
        return y

    def backward(self):
        cfg = self.cfg
        m = self.dev["x"].shape[0]
        dx = torch.empty((m, cfg.d_in), dtype=torch.bfloat16, device="cuda")
        dA = torch.full((cfg.groups, cfg.rank), float("nan"), dtype=torch.float32, device="cuda")
        dB = torch.full((cfg.rank, cfg.d_out), float("nan"), dtype=torch.float32, device="cuda")
        ws = Q.alloc_workspace(self.d, m, Q.OP_BACKWARD)
        Q.qalora_backward(self.d, m, self.dev["x"], self.dev["dy"], self.codes, self.qparams, self.dev["A"],
                          self.dev["B"], dx, dA, dB, ws)
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0
        return dx, dA, dB

    def oracle_quant(self):
        cfg = self.cfg
        return O.quantize(self.cpu["W"].numpy(), cfg.group_size, cfg.bits)


def check_quantize(layer: GpuLayer):
    cfg = layer.cfg
    codes, alpha, beta = layer.oracle_quant()
    packed = O.pack(codes, cfg.bits)
    got_words = layer.codes.cpu().numpy().view(np.uint32)
    assert np.array_equal(got_words, packed), "packed codes differ"
    qp = layer.qparams.cpu().numpy()
    assert np.array_equal(qp[..., 0], alpha) and np.array_equal(qp[..., 1], beta), "alpha/beta differ"
    assert int(layer.status.item()) == 0
    return codes, alpha, beta


SMALL = [
    # name, K, N, g, bits, r, s, M
    ("tiny4", 64, 64, 32, 4, 8, 1.0, 5),
    ("ragged4", 320, 200, 32, 4, 16, 0.5, 77),
    ("ragged3", 192, 136, 64, 3, 24, 1.5, 130),
    ("ragged2", 256, 72, 128, 2, 8, 2.0, 33),
    ("g64_4", 512, 384, 64, 4, 64, 1.0, 200),
    ("colwise", 128, 64, 128, 4, 8, 1.0, 16),
    # adapter coefficient zero and negative (few rows, the tokens-as-MMA-rows kernel, the large-tile kernels)
    ("s_zero_few", 512, 384, 32, 4, 16, 0.0, 6),
    ("s_zero_tc", 512, 512, 64, 3, 16, 0.0, 300),
    ("s_negative_mid", 512, 512, 32, 4, 24, -1.5, 50),
    ("s_negative_tc", 512, 384, 128, 2, 8, -0.5, 700),
    # group sizes other than 32, 64, 128 (multiples of 32): CUDA-core kernels whatever the other sizes are
    ("g96", 384, 136, 96, 4, 8, 1.0, 50),
    ("g256", 512, 256, 256, 3, 16, 1.0, 300),
    ("g1024", 1024, 128, 1024, 2, 8, 1.0, 20),
    # shapes the tensor-core kernels tile (N % 128 == 0, K % 128 == 0), ragged in M
    ("tc4", 256, 256, 32, 4, 16, 1.0, 300),
    ("tc3", 384, 256, 64, 3, 24, 0.75, 270),
    ("tc2", 256, 128, 128, 2, 8, 2.0, 515),
    ("tc4_r0pad", 1024, 640, 32, 4, 72, 1.0, 1000),
    # many-row pooling kernel (M >= 64, K % 256 == 0) with few, many and more-than-a-block's adapter columns
    ("pool_r8", 512, 256, 32, 4, 8, 1.0, 100),
    ("pool_r128", 768, 256, 64, 4, 128, 0.5, 70),
    ("pool_r256", 1024, 128, 128, 2, 256, 1.0, 65),
    # few tokens and a long reduction: the forward contraction is cut into parts that meet in scratch
    ("parts4", 2048, 256, 32, 4, 16, 1.0, 40),
    ("parts3", 1536, 384, 64, 3, 24, 0.75, 300),
    ("parts2", 4096, 128, 128, 2, 8, 1.5, 33),
    # 17 to 128 tokens on shapes with N % 256 == 0: the kernel with the tokens as the MMA rows (64- and
    # 128-row activation tiles, ragged counts, every bit width and group size, adapter ranks that are
    # not a multiple of the 64-wide adapter step)
    ("midm2", 512, 512, 128, 2, 8, 2.0, 100),
    ("midm3", 640, 256, 32, 3, 40, 1.0, 64),
    ("midm4_128", 256, 512, 64, 4, 16, 1.0, 128),
    ("midm4_33", 4096, 256, 32, 4, 72, 0.5, 33),
    ("midm4_r64_65", 1024, 768, 32, 4, 64, 1.0, 65),
    # the same kernel with the shortest reduction it takes (4 steps of 64 channels), odd step counts (5, 17, 19,
    # 65: the parts of a cut reduction are unequal) and reductions that are not a multiple of 128 channels
    ("midm_4st", 256, 2560, 128, 2, 8, 1.0, 50),
    ("midm_5st", 320, 256, 32, 4, 16, 1.0, 33),
    ("midm_17st", 1088, 256, 32, 4, 16, 1.0, 40),
    ("midm_19st", 1216, 768, 64, 3, 8, 1.0, 17),
    ("midm_65st", 4160, 512, 32, 4, 64, 1.0, 64),
    # more 128 x 256 tiles than SMs with a short last wave: that wave's tiles alone are cut into parts
    # (160 and 320 tiles: 12 and 24 in the strip; ragged last token tiles)
    ("tail4", 2048, 20480, 32, 4, 16, 1.0, 256),
    ("tail3", 1024, 20480, 64, 3, 8, 1.0, 300),
    ("tail2", 1024, 5120, 128, 2, 8, 1.0, 1000),      # 40 x 4 tiles: a strip of 3 channel tiles over all four token tiles
    ("tail_dx4", 5120, 1024, 32, 4, 16, 1.0, 1000),   # the same for the input gradient (40 x 4 tiles along the input channels)
    ("tail_dx3", 5120, 1152, 64, 3, 24, 1.0, 520),    # 40 x 3 tiles: none in a strip (120 < SMs); 1152 = 9 x 128 reduction
    # tile counts just above one and two full waves of SMs (149, 150, 185, 222, 295, 297 tiles with one token
    # tile; 150 and 297 with three): the last wave's strip holds 1 to 147 tiles and is cut into parts
    ("strip_f149", 256, 149 * 128, 32, 4, 16, 1.0, 200),
    ("strip_f150", 256, 150 * 128, 64, 3, 8, 1.0, 256),
    ("strip_f185", 512, 185 * 128, 32, 4, 16, 1.0, 130),
    ("strip_f222", 256, 222 * 128, 128, 2, 8, 1.0, 200),
    ("strip_f295", 256, 295 * 128, 32, 4, 8, 1.0, 255),
    ("strip_f297", 384, 297 * 128, 32, 4, 16, 1.0, 200),
    ("strip_f50x3", 512, 50 * 128, 32, 4, 16, 1.0, 520),
    ("strip_f99x3", 256, 99 * 128, 64, 4, 16, 1.0, 700),
    # the same for the input gradient (tiles along the input channels)
    ("strip_d149", 149 * 128, 256, 32, 4, 16, 1.0, 200),
    ("strip_d185", 185 * 128, 384, 64, 3, 8, 1.0, 130),
    ("strip_d297", 297 * 128, 256, 32, 4, 16, 1.0, 256),
    ("strip_d50x3", 50 * 128, 512, 128, 2, 8, 1.0, 520),
    # many tokens, several channel tiles, ragged token count
    ("pair4", 512, 256, 32, 4, 16, 1.0, 700),
    ("pair3", 384, 512, 64, 3, 24, 0.75, 530),
    ("pair2", 256, 768, 128, 2, 8, 2.0, 1100),
]


@pytest.mark.parametrize("case", SMALL, ids=[c[0] for c in SMALL])
def test_small_shapes_all_ops(case):
    name, K, N, g, bits, r, s, M = case
    cfg = LayerConfig(name, K, N, g, bits, r, s, M, dy_std=1.0, outlier_frac=0.01, seed=len(name) + K)
    layer = GpuLayer(cfg)
    codes, alpha, beta = check_quantize(layer)
    x, A, B, dy = (to_f64(layer.cpu[k]) for k in ("x", "A", "B", "dy"))
    y_ref = O.forward(x, codes, alpha, beta, g, A, B, s)
    margin(name, "y", layer.forward().float().cpu().numpy(), y_ref)
    dx, dA, dB = layer.backward()
    dx_ref, dA_ref, dB_ref = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    margin(name, "dX", dx.float().cpu().numpy(), dx_ref)
    margin(name, "dA", dA.cpu().numpy(), dA_ref)
    margin(name, "dB", dB.cpu().numpy(), dB_ref)
    # merge, then the plain quantized layer must reproduce the adapted one
    q2 = torch.empty_like(layer.qparams)
    Q.qalora_merge(layer.d, layer.qparams, layer.dev["A"], layer.dev["B"], q2)
    torch.cuda.synchronize()
    q2n = q2.cpu().numpy()
    assert np.array_equal(q2n[..., 0], alpha)
    margin(name, "beta_merged", q2n[..., 1], O.merge(beta, A, B, s))
    y_merged = layer.forward(qparams=q2, rank=0)
    margin(name, "y_merged", y_merged.float().cpu().numpy(), y_ref)
    # in-place merge gives the same bytes
    q3 = layer.qparams.clone()
    Q.qalora_merge(layer.d, q3, layer.dev["A"], layer.dev["B"], q3)
    torch.cuda.synchronize()
    assert torch.equal(q3, q2)


BOUNDARY_M = [1, 2, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 100, 127, 128, 129, 255, 256, 257, 384, 511, 512,
              513, 767, 1024, 1025]


@pytest.mark.parametrize("bits,g,r", [(4, 32, 24), (3, 64, 64)])
def test_token_counts_around_every_dispatch_boundary(bits, g, r):
    """One layer (1024 -> 6144: 48 channel tiles, so every kernel family is eligible somewhere),
    token counts on both sides of every row-count threshold of the dispatch (few-token kernel up
    to 16 or 32 rows, tokens-as-MMA-rows kernel up to 64 or 128, token-rows pooling from 512,
    256-token tiles with ragged tails).  y and dX of the first M rows do not depend on the rows
    behind them, so one oracle pass over all rows serves every M; dA and dB are sums over the rows
    and are taken from the oracle per M."""
    K, N, s = 1024, 6144, 0.75
    name = f"boundary_b{bits}"
    cfg = LayerConfig(name, K, N, g, bits, r, s, max(BOUNDARY_M), dy_std=1.0, outlier_frac=0.01, seed=31 + bits)
    layer = GpuLayer(cfg)
    codes, alpha, beta = check_quantize(layer)
    x, A, B, dy = (to_f64(layer.cpu[k]) for k in ("x", "A", "B", "dy"))
    y_ref = O.forward(x, codes, alpha, beta, g, A, B, s)
    dx_ref, _, _ = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    q2 = torch.empty_like(layer.qparams)
    Q.qalora_merge(layer.d, layer.qparams, layer.dev["A"], layer.dev["B"], q2)
    for M in BOUNDARY_M:
        xm, dym = layer.dev["x"][:M].contiguous(), layer.dev["dy"][:M].contiguous()
        # (scale of a slice's comparison: the slice's own largest reference value, as everywhere)
        margin(name, "y", layer.forward(x=xm).float().cpu().numpy(), y_ref[:M])
        margin(name, "y_merged", layer.forward(x=xm, qparams=q2, rank=0).float().cpu().numpy(), y_ref[:M])
        dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
        dA = torch.full((cfg.groups, r), float("nan"), dtype=torch.float32, device="cuda")
        dB = torch.full((r, N), float("nan"), dtype=torch.float32, device="cuda")
        ws = torch.full((max(Q.qalora_workspace_bytes(layer.d, M, Q.OP_BACKWARD), 16),), 0xFF, dtype=torch.uint8, device="cuda")
        Q.qalora_backward(layer.d, M, xm, dym, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], dx, dA, dB, ws)
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0, M
        _, dA_ref, dB_ref = O.backward(x[:M], dy[:M], codes, alpha, beta, g, A, B, s)
        margin(name, "dX", dx.float().cpu().numpy(), dx_ref[:M])
        margin(name, "dA", dA.cpu().numpy(), dA_ref)
        margin(name, "dB", dB.cpu().numpy(), dB_ref)
        # the fine-tuning pair (one workspace, the input pooled once) gives the bits of the separate calls
        wt = torch.full((max(Q.qalora_workspace_bytes(layer.d, M, Q.OP_TRAIN), 16),), 0xFF, dtype=torch.uint8, device="cuda")
        y_t = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        dx_t, dA_t, dB_t = torch.empty_like(dx), torch.empty_like(dA), torch.empty_like(dB)
        Q.qalora_forward_train(layer.d, M, xm, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], y_t, wt)
        Q.qalora_backward_train(layer.d, M, xm, dym, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], dx_t, dA_t, dB_t, wt)
        torch.cuda.synchronize()
        assert Q.workspace_status(wt) == 0, M
        assert torch.equal(y_t, layer.forward(x=xm)) and torch.equal(dx_t, dx), M
        assert torch.equal(dA_t, dA) and torch.equal(dB_t, dB), M


@pytest.mark.parametrize("M", [5, 100, 600])
def test_backward_outputs_can_be_skipped_one_by_one(M):
    """dx, dA or dB may be NULL: the other outputs are then the bits of the full call, and nothing
    else is written (few rows, the CUDA-core side kernels; 100 and 600 rows, the tensor-core ones
    with dB on the library's second stream)."""
    cfg = LayerConfig("skip_outputs", 512, 384, 32, 4, 16, 1.0, M, dy_std=1.0, seed=5 + M)
    layer = GpuLayer(cfg)
    dx, dA, dB = layer.backward()
    args = (layer.d, M, layer.dev["x"], layer.dev["dy"], layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"])
    for keep in ((1, 0, 0), (0, 1, 0), (0, 0, 1), (1, 1, 0), (0, 1, 1), (0, 0, 0)):
        outs = [torch.full_like(t, float("nan")) for t in (dx, dA, dB)]
        ws = torch.full((max(Q.qalora_workspace_bytes(layer.d, M, Q.OP_BACKWARD), 16),), 0xFF, dtype=torch.uint8, device="cuda")
        Q.qalora_backward(*args, *[o if k else None for o, k in zip(outs, keep)], ws)
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0
        for o, k, full in zip(outs, keep, (dx, dA, dB)):
            assert torch.equal(o, full) if k else bool(torch.isnan(o).all()), (M, keep)


def test_config1_full():
    cfg = CONFIGS["cfg1_512"]
    layer = GpuLayer(cfg)
    codes, alpha, beta = check_quantize(layer)
    x, A, B, dy = (to_f64(layer.cpu[k]) for k in ("x", "A", "B", "dy"))
    g, s = cfg.group_size, cfg.scale
    margin("cfg1_512", "y", layer.forward().float().cpu().numpy(), O.forward(x, codes, alpha, beta, g, A, B, s))
    dx, dA, dB = layer.backward()
    dx_ref, dA_ref, dB_ref = O.backward(x, dy, codes, alpha, beta, g, A, B, s)
    margin("cfg1_512", "dX", dx.float().cpu().numpy(), dx_ref)
    margin("cfg1_512", "dA", dA.cpu().numpy(), dA_ref)
    margin("cfg1_512", "dB", dB.cpu().numpy(), dB_ref)


@pytest.mark.parametrize("M", [1, 4, 16])
def test_config2_small_m_forward_and_merge(M):
    cfg = CONFIGS["cfg2_7b_attn"].with_(tokens=M)
    layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
    codes, alpha, beta = check_quantize(layer)
    x, A, B = (to_f64(layer.cpu[k]) for k in ("x", "A", "B"))
    g, s = cfg.group_size, cfg.scale
    y_ref = O.forward(x, codes, alpha, beta, g, A, B, s)
    margin(f"cfg2_7b_attn_m{M}", "y", layer.forward().float().cpu().numpy(), y_ref)
    q2 = torch.empty_like(layer.qparams)
    Q.qalora_merge(layer.d, layer.qparams, layer.dev["A"], layer.dev["B"], q2)
    margin(f"cfg2_7b_attn_m{M}", "beta_merged", q2.cpu().numpy()[..., 1], O.merge(beta, A, B, s))
    margin(f"cfg2_7b_attn_m{M}", "y_merged", layer.forward(qparams=q2, rank=0).float().cpu().numpy(), y_ref)


@pytest.mark.parametrize("K,N", [(128, 128), (384, 128), (640, 128), (896, 640), (1408, 256), (2176, 1152), (128, 19072)])
def test_few_token_forward_slice_counts(K, N):
    """Few-token kernel: reductions of 1, 3, 5, 7, 11 and 17 stages of 128 channels (so the slices of
    a column tile are unequal, and a layer of one stage cannot be cut at all) on 1 to 149 column
    tiles, i.e. every slice count the host can pick, with 1, 8, 16 and 32 rows, with and without
    the adapter, 4-bit g = 32 and 3-bit g = 128."""
    for bits, g, r in ((4, 32, 24), (3, 128, 0)):
        name = f"slices_{K}x{N}_b{bits}"
        cfg = LayerConfig(name, K, N, g, bits, max(r, 8), 1.25, 32, outlier_frac=0.01, seed=K + N + bits)
        layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
        codes, alpha, beta = check_quantize(layer)
        x, A, B = (to_f64(layer.cpu[k]) for k in ("x", "A", "B"))
        y_ref = O.forward(x, codes, alpha, beta, g, A if r else None, B if r else None, cfg.scale)
        for M in (1, 8, 16, 32):
            xm = layer.dev["x"][:M].contiguous()
            margin(name, "y", layer.forward(x=xm, rank=None if r else 0).float().cpu().numpy(), y_ref[:M])


@pytest.mark.parametrize("bits,g,M,r", [(4, 32, 1, 16), (4, 128, 8, 0), (3, 32, 16, 24), (3, 64, 3, 8),
                                       (2, 32, 9, 64), (2, 128, 1, 0), (4, 64, 16, 128),
                                       (4, 32, 17, 16), (4, 128, 32, 0), (3, 64, 25, 64), (2, 32, 32, 8), (4, 32, 5, 24), (2, 64, 12, 40)])
def test_few_token_forward_all_widths(bits, g, M, r):
    """The bandwidth-bound few-token kernel (N % 128 == 0, K % 128 == 0): every bit
    width, group sizes 32/64/128, with and without the adapter (ranks that are and are not
    multiples of the 16-row MMA step), M in every set of eight rows up to 32."""
    cfg = LayerConfig("gemv", 1280, 384, g, bits, max(r, 8), 1.25, M, outlier_frac=0.01, seed=bits * 100 + g + M)
    layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
    codes, alpha, beta = check_quantize(layer)
    x, A, B = (to_f64(layer.cpu[k]) for k in ("x", "A", "B"))
    if r == 0:
        y_ref = O.forward(x, codes, alpha, beta, g)
        got = layer.forward(rank=0)
    else:
        y_ref = O.forward(x, codes, alpha, beta, g, A, B, cfg.scale)
        got = layer.forward()
    assert Q.qalora_main_kernel_name() == "qalora_gemv_kernel"
    margin(f"few_token_b{bits}_g{g}_m{M}_r{r}", "y", got.float().cpu().numpy(), y_ref)


@pytest.mark.parametrize("M", [1, 8])
def test_few_token_forward_back_to_back_calls_share_a_workspace(M):
    """The few-token kernel starts while the pooling kernel that writes T = s pool(x) A is still
    running and may read T only once that kernel is complete.  Many calls in a row on one stream,
    with one workspace and inputs that change from call to call (a large layer, so that the main
    kernel is still streaming when the next call is queued): every output must be its own
    input's, never a mix with the neighbouring call's T."""
    cfg = LayerConfig("gemv_b2b", 4096, 1024, 32, 4, 64, 4.0, M, seed=77)
    layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
    codes, alpha, beta = check_quantize(layer)
    gen = torch.Generator(device="cpu").manual_seed(1234)
    calls = 6
    # large adapter weights make the adapter term as large as the base term, so that a stale T shows
    A = (torch.randn((cfg.groups, cfg.rank), generator=gen) * 0.5).to(torch.bfloat16)
    B = (torch.randn((cfg.rank, cfg.d_out), generator=gen) * 0.5).to(torch.bfloat16)
    xs = [(torch.randn((M, cfg.d_in), generator=gen) * (1.0 + i)).to(torch.bfloat16) for i in range(calls)]
    Ad, Bd = A.cuda(), B.cuda()
    xd = [x.cuda() for x in xs]
    ys = [torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda") for _ in range(calls)]
    ws = Q.alloc_workspace(layer.d, M, Q.OP_FORWARD)
    torch.cuda.synchronize()
    for i in range(calls):
        Q.qalora_forward(layer.d, M, xd[i], layer.codes, layer.qparams, Ad, Bd, ys[i], ws)
    torch.cuda.synchronize()
    assert Q.workspace_status(ws) == 0
    for i in range(calls):
        y_ref = O.forward(to_f64(xs[i]), codes, alpha, beta, cfg.group_size, to_f64(A), to_f64(B), cfg.scale)
        adapter = O.forward(to_f64(xs[i]), codes, alpha, beta, cfg.group_size, to_f64(A), to_f64(B), cfg.scale) - \
            O.forward(to_f64(xs[i]), codes, alpha, beta, cfg.group_size)
        assert np.max(np.abs(adapter)) > 0.2 * np.max(np.abs(y_ref))     # the case does exercise T
        assert rel_err(ys[i].float().cpu().numpy(), y_ref) <= TOL, i


def test_few_token_forward_replayed_from_a_cuda_graph():
    """The adapted few-token forward is two launches, the second one started beside the first
    (programmatic dependent launch).  Captured once into a CUDA graph and replayed with new
    input values in the same buffers, it must give each replay's own result."""
    cfg = LayerConfig("gemv_graph", 2048, 512, 64, 4, 32, 2.0, 4, seed=31)
    layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
    codes, alpha, beta = check_quantize(layer)
    A, B = to_f64(layer.cpu["A"]), to_f64(layer.cpu["B"])
    M = cfg.tokens
    x_static = torch.zeros((M, cfg.d_in), dtype=torch.bfloat16, device="cuda")
    y_static = torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    ws = Q.alloc_workspace(layer.d, M, Q.OP_FORWARD)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):                     # first call outside the capture: sets kernel attributes
        Q.qalora_forward(layer.d, M, x_static, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], y_static, ws)
    side.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for _ in range(3):                            # several calls in one graph, as a decoding loop would hold
            Q.qalora_forward(layer.d, M, x_static, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], y_static, ws)
    gen = torch.Generator(device="cpu").manual_seed(5)
    for rep in range(3):
        x = (torch.randn((M, cfg.d_in), generator=gen) * (rep + 1)).to(torch.bfloat16)
        x_static.copy_(x.cuda())
        torch.cuda.synchronize()
        graph.replay()
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 0
        y_ref = O.forward(to_f64(x), codes, alpha, beta, cfg.group_size, A, B, cfg.scale)
        assert rel_err(y_static.float().cpu().numpy(), y_ref) <= TOL, rep


def test_edge_cases():
    cfg = LayerConfig("edge", 64, 64, 32, 4, 8, 1.0, 3, seed=9)
    layer = GpuLayer(cfg)
    # constant groups and an all-zero matrix
    W = torch.zeros((64, 64), dtype=torch.float32)
    W[32:, 5] = 0.75
    W[:32, 7] = torch.linspace(-1, 1, 32)
    Wd = W.cuda()
    Q.qalora_quantize(layer.d, Wd, layer.codes, layer.qparams, layer.status)
    torch.cuda.synchronize()
    codes, alpha, beta = O.quantize(W.numpy(), 32, 4)
    assert np.array_equal(layer.codes.cpu().numpy().view(np.uint32), O.pack(codes, 4))
    qp = layer.qparams.cpu().numpy()
    assert np.array_equal(qp[..., 0], alpha) and np.array_equal(qp[..., 1], beta)
    # a non-finite weight raises the device status bit instead of trapping
    Wd[3, 3] = float("inf")
    Q.qalora_quantize(layer.d, Wd, layer.codes, layer.qparams, layer.status)
    torch.cuda.synchronize()
    assert int(layer.status.item()) & 1
    # m = 0 is a no-op that still succeeds
    empty = torch.empty((0, 64), dtype=torch.bfloat16, device="cuda")
    assert layer.forward(x=empty).shape == (0, 64)


def test_quantize_groups_with_extreme_scales():
    """Groups whose scale alpha is a subnormal (nearly equal tiny weights) or huge: 1 / alpha
    overflows or loses its precision there, so the kernel must take Eq. 1's division for them;
    the codes stay bit-exact."""
    K, N, g = 64, 128, 32
    d = Q.desc(K, N, g, 4, 8, 1.0)
    gen = torch.Generator(device="cpu").manual_seed(3)
    W = torch.randn((K, N), generator=gen, dtype=torch.float32) * 0.02
    W[:32, 0:8] = 1.2e-38 + torch.rand((32, 8), generator=gen) * 1.5e-38  # normal weights, alpha about 1e-39 (subnormal)
    W[:32, 8:16] = torch.rand((32, 8), generator=gen) * 3e-38             # alpha about 2e-39
    W[32:, 16:24] = 1e37 + torch.rand((32, 8), generator=gen) * 2e37      # alpha above 1e35
    W[32:, 24:32] = torch.rand((32, 8), generator=gen) * 1e-29            # alpha just below the fast range
    codes_d, qparams = Q.alloc_packed(d)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    Q.qalora_quantize(d, W.cuda(), codes_d, qparams, status)
    torch.cuda.synchronize()
    codes, alpha, beta = O.quantize(W.numpy(), g, 4)
    assert 0 < float(alpha[0, 0]) < 1.1e-38 and 0 < float(alpha[0, 8]) < 1.1e-38 and float(alpha[1, 16]) > 1e35   # the cases are what they claim to be
    assert np.array_equal(codes_d.cpu().numpy().view(np.uint32), O.pack(codes, 4))
    qp = qparams.cpu().numpy()
    assert np.array_equal(qp[..., 0], alpha) and np.array_equal(qp[..., 1], beta)
    assert int(status.item()) == 0


@pytest.mark.parametrize("case", [("simt", 320, 200, 77), ("tensor_core", 256, 256, 300), ("few_token", 1280, 384, 5),
                                  ("parts", 2048, 256, 40)],
                         ids=lambda c: c[0])
def test_status_word_is_cleared_whatever_the_workspace_held(case):
    """The workspace's content is undefined on entry; after a call that went well its first
    int32 must read 0 on every dispatch path, also when the workspace was full of 0xFF."""
    name, K, N, M = case
    cfg = LayerConfig("status_" + name, K, N, 32, 4, 16, 1.0, M, seed=K + M)
    layer = GpuLayer(cfg)
    y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.full((max(Q.qalora_workspace_bytes(layer.d, M, Q.OP_FORWARD), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    Q.qalora_forward(layer.d, M, layer.dev["x"], layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], y, ws)
    torch.cuda.synchronize()
    assert Q.workspace_status(ws) == 0
    assert torch.equal(y, layer.forward())
    wb = torch.full((Q.qalora_workspace_bytes(layer.d, M, Q.OP_BACKWARD),), 0xFF, dtype=torch.uint8, device="cuda")
    dx = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dA = torch.empty((cfg.groups, cfg.rank), dtype=torch.float32, device="cuda")
    dB = torch.empty((cfg.rank, N), dtype=torch.float32, device="cuda")
    Q.qalora_backward(layer.d, M, layer.dev["x"], layer.dev["dy"], layer.codes, layer.qparams, layer.dev["A"],
                      layer.dev["B"], dx, dA, dB, wb)
    torch.cuda.synchronize()
    assert Q.workspace_status(wb) == 0
    ref = layer.backward()
    assert torch.equal(dx, ref[0]) and torch.equal(dA, ref[1]) and torch.equal(dB, ref[2])


def test_an_expired_wait_raises_the_status_word_and_the_next_call_is_clean():
    """Failure detection without a fault: a test hook makes the producers of ONE few-token
    launch stop after two stages and shortens that launch's wait limit to a millisecond.  The
    consumers' bounded waits then run out; the kernel must come back by itself with the status
    word at 1 (outputs invalid), the context must stay usable, and the following ordinary
    call must give the very same bits as before."""
    import ctypes
    cfg = LayerConfig("expire", 8192, 512, 32, 4, 16, 1.0, 4, seed=11)    # 64 stages over at most 8 slices: 8 or more per block
    layer = GpuLayer(cfg, need=("W", "x", "A", "B"))
    lib = Q.load()
    hook = lib.qalora_debug_expire_next_few_token_wait
    hook.restype = ctypes.c_int
    hook.argtypes = [ctypes.c_int, ctypes.c_uint64]
    M = cfg.tokens
    d0 = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, 0, cfg.scale)
    ws = Q.alloc_workspace(d0, M, Q.OP_FORWARD)
    before = torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    Q.qalora_forward(d0, M, layer.dev["x"], layer.codes, layer.qparams, None, None, before, ws)
    torch.cuda.synchronize()
    assert Q.qalora_main_kernel_name() == "qalora_gemv_kernel" and Q.workspace_status(ws) == 0
    assert hook(2, 1_000_000) == 0
    broken = torch.empty_like(before)
    t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
    t0.record()
    Q.qalora_forward(d0, M, layer.dev["x"], layer.codes, layer.qparams, None, None, broken, ws)
    t1.record()
    torch.cuda.synchronize()                              # returns: the kernel gave up by itself
    assert Q.workspace_status(ws) == 1
    assert t0.elapsed_time(t1) < 1000.0                   # ms: far below the ordinary two-second limit
    after = torch.empty_like(before)
    Q.qalora_forward(d0, M, layer.dev["x"], layer.codes, layer.qparams, None, None, after, ws)
    torch.cuda.synchronize()
    assert Q.workspace_status(ws) == 0                    # the hook was one-shot and the word was cleared
    assert torch.equal(after, before)


def test_an_expired_wait_in_the_tensor_core_kernels_unwinds_and_the_next_call_is_clean():
    """The same for the tensor-core forward and dX kernels: the hook makes the activation producers
    of ONE launch stop after two reduction steps (every block is then in the middle of its first
    tile) and shortens that launch's wait limit to a millisecond.  Every role's bounded wait runs
    out, the blocks leave through their ordinary teardown (tensor memory released), the status word
    reads 1, and the following ordinary call gives the same bits as the one before."""
    import ctypes
    cfg = LayerConfig("expire_tc", 1024, 512, 32, 4, 16, 1.0, 512, seed=12)   # 8 tiles of 16 (+1) steps: one per block
    layer = GpuLayer(cfg)
    lib = Q.load()
    hook = lib.qalora_debug_expire_next_tc_wait
    hook.restype = ctypes.c_int
    hook.argtypes = [ctypes.c_int, ctypes.c_uint64]
    M, d = cfg.tokens, layer.d
    A, B = layer.dev["A"], layer.dev["B"]

    def fwd(ws):
        y = torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda")
        Q.qalora_forward(d, M, layer.dev["x"], layer.codes, layer.qparams, A, B, y, ws)
        torch.cuda.synchronize()                          # returns: the kernel gave up by itself
        return y

    def bwd(ws):
        dx = torch.empty((M, cfg.d_in), dtype=torch.bfloat16, device="cuda")
        dA = torch.empty((cfg.groups, cfg.rank), dtype=torch.float32, device="cuda")
        dB = torch.empty((cfg.rank, cfg.d_out), dtype=torch.float32, device="cuda")
        Q.qalora_backward(d, M, layer.dev["x"], layer.dev["dy"], layer.codes, layer.qparams, A, B, dx, dA, dB, ws)
        torch.cuda.synchronize()
        return dx

    for run, op, kernel in ((fwd, Q.OP_FORWARD, "qalora_tc_kernel<fwd>"), (bwd, Q.OP_BACKWARD, "qalora_tc_kernel<dx>")):
        ws = Q.alloc_workspace(d, M, op)
        before = run(ws)
        assert Q.qalora_main_kernel_name() == kernel and Q.workspace_status(ws) == 0
        assert hook(2, 1_000_000) == 0
        t0 = torch.cuda.Event(enable_timing=True); t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        run(ws)
        t1.record()
        torch.cuda.synchronize()
        assert Q.workspace_status(ws) == 1
        assert t0.elapsed_time(t1) < 1000.0               # ms: far below the ordinary two-second limit
        after = run(ws)
        assert Q.workspace_status(ws) == 0                # the hook was one-shot and the word was cleared
        assert torch.equal(after, before)


def test_backward_pass_in_a_cuda_graph_gives_the_same_bits():
    """The backward pass forks dB onto a stream of the library's own and joins it again inside
    the call.  Captured into a CUDA graph (after one ordinary call, which creates that stream) the
    fork and the join must become part of the graph: the replay gives the bits of the ordinary call."""
    cfg = LayerConfig("graph_bwd", 512, 384, 32, 4, 16, 1.0, 700, seed=31)
    layer = GpuLayer(cfg)
    M, d = cfg.tokens, layer.d
    ws = Q.alloc_workspace(d, M, Q.OP_BACKWARD)
    out = lambda: (torch.zeros((M, cfg.d_in), dtype=torch.bfloat16, device="cuda"),
                   torch.zeros((cfg.groups, cfg.rank), dtype=torch.float32, device="cuda"),
                   torch.zeros((cfg.rank, cfg.d_out), dtype=torch.float32, device="cuda"))
    run = lambda o: Q.qalora_backward(d, M, layer.dev["x"], layer.dev["dy"], layer.codes, layer.qparams,
                                      layer.dev["A"], layer.dev["B"], o[0], o[1], o[2], ws)
    ref = out()
    run(ref)
    torch.cuda.synchronize()
    got = out()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        run(got)
    for o in got:
        o.zero_()
    graph.replay()
    torch.cuda.synchronize()
    assert Q.workspace_status(ws) == 0
    for a, b in zip(got, ref):
        assert torch.equal(a, b)


def test_two_host_threads_run_forward_and_backward_side_by_side():
    """Two host threads, each with its own stream, workspace and outputs, run the forward and
    backward pass of the same layer at the same time (the library keeps its second stream and its
    probe per host thread, its set-up flags per device): both get the bits of a single-threaded run."""
    import threading
    cfg = LayerConfig("threads", 512, 384, 32, 4, 16, 1.0, 700, seed=41)
    layer = GpuLayer(cfg)
    M, d = cfg.tokens, layer.d
    ref_y = layer.forward()
    ref_b = layer.backward()
    results, errors = {}, []

    def worker(tag):
        try:
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                wf = Q.alloc_workspace(d, M, Q.OP_FORWARD)
                wb = Q.alloc_workspace(d, M, Q.OP_BACKWARD)
                for _ in range(5):
                    y = torch.empty((M, cfg.d_out), dtype=torch.bfloat16, device="cuda")
                    dx = torch.empty((M, cfg.d_in), dtype=torch.bfloat16, device="cuda")
                    dA = torch.empty((cfg.groups, cfg.rank), dtype=torch.float32, device="cuda")
                    dB = torch.empty((cfg.rank, cfg.d_out), dtype=torch.float32, device="cuda")
                    Q.qalora_forward(d, M, layer.dev["x"], layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"], y, wf)
                    Q.qalora_backward(d, M, layer.dev["x"], layer.dev["dy"], layer.codes, layer.qparams, layer.dev["A"],
                                      layer.dev["B"], dx, dA, dB, wb)
                stream.synchronize()
                results[tag] = (y, dx, dA, dB, Q.workspace_status(wf), Q.workspace_status(wb))
        except Exception as e:  # noqa: BLE001 - reported by the main thread
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for tag in range(2):
        y, dx, dA, dB, sf, sb = results[tag]
        assert sf == 0 and sb == 0
        assert torch.equal(y, ref_y) and torch.equal(dx, ref_b[0]) and torch.equal(dA, ref_b[1]) and torch.equal(dB, ref_b[2])


def test_results_do_not_depend_on_scheduling():
    cfg = LayerConfig("det", 256, 256, 32, 4, 16, 1.0, 300, seed=5)
    layer = GpuLayer(cfg)
    y1, b1 = layer.forward(), layer.backward()
    y2, b2 = layer.forward(), layer.backward()
    assert torch.equal(y1, y2)
    for a, b in zip(b1, b2):
        assert torch.equal(a, b)


def test_step_from_host_buffers_matches_device_calls():
    cfg = LayerConfig("hoststep", 512, 384, 64, 4, 64, 1.0, 300, seed=21)
    layer = GpuLayer(cfg)
    y = layer.forward()
    dx, dA, dB = layer.backward()
    pin = lambda t: t.pin_memory()
    hx, hdy = pin(layer.cpu["x"]), pin(layer.cpu["dy"])
    hy, hdx = pin(torch.empty_like(y, device="cpu")), pin(torch.empty_like(dx, device="cpu"))
    hdA, hdB = pin(torch.empty_like(dA, device="cpu")), pin(torch.empty_like(dB, device="cpu"))
    staging = torch.zeros(Q.qalora_step_host_bytes(layer.d, cfg.tokens), dtype=torch.uint8, device="cuda")
    Q.qalora_step_host(layer.d, cfg.tokens, hx, hdy, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"],
                       hy, hdx, hdA, hdB, staging)
    torch.cuda.synchronize()
    assert Q.workspace_status(staging) == 0
    assert torch.equal(hy, y.cpu()) and torch.equal(hdx, dx.cpu())
    assert torch.equal(hdA, dA.cpu()) and torch.equal(hdB, dB.cpu())


@pytest.mark.parametrize("pinned", [True, False], ids=["pinned", "pageable"])
def test_chunked_step_from_host_buffers(pinned):
    # 2348 rows: three pipelined chunks (1024, 1024 and a ragged 300).  Rows are independent in y
    # and dx, so dx and the full chunks of y match the whole-batch device calls bit for bit; the
    # 300-row chunk pools its input with the few-row kernel (another summation order of the rank-r
    # intermediate), so its y is held to the oracle's tolerance and to a few bf16 steps of the
    # whole-batch result.  dA and dB are sums over the chunks and are held to the oracle's tolerance.
    cfg = LayerConfig("hostchunks", 512, 384, 64, 4, 64, 1.0, 2348, seed=22)
    layer = GpuLayer(cfg)
    y = layer.forward()
    dx, dA, dB = layer.backward()
    pin = (lambda t: t.pin_memory()) if pinned else (lambda t: t.clone())   # pageable buffers: the copies are staged by the driver
    hx, hdy = pin(layer.cpu["x"]), pin(layer.cpu["dy"])
    hy, hdx = pin(torch.empty_like(y, device="cpu")), pin(torch.empty_like(dx, device="cpu"))
    hdA, hdB = pin(torch.empty_like(dA, device="cpu")), pin(torch.empty_like(dB, device="cpu"))
    staging = torch.zeros(Q.qalora_step_host_bytes(layer.d, cfg.tokens), dtype=torch.uint8, device="cuda")
    codes, alpha, beta = check_quantize(layer)
    xf, Af, Bf, dyf = (to_f64(layer.cpu[k]) for k in ("x", "A", "B", "dy"))
    _, dA_ref, dB_ref = O.backward(xf, dyf, codes, alpha, beta, cfg.group_size, Af, Bf, cfg.scale)
    y_ref = O.forward(xf, codes, alpha, beta, cfg.group_size, Af, Bf, cfg.scale)
    for _ in range(2):  # the second call reuses the library's streams and events
        hy.zero_(); hdx.zero_(); hdA.zero_(); hdB.zero_()
        Q.qalora_step_host(layer.d, cfg.tokens, hx, hdy, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"],
                           hy, hdx, hdA, hdB, staging)
        torch.cuda.synchronize()
        assert Q.workspace_status(staging) == 0
        assert torch.equal(hy[:2048], y[:2048].cpu()) and torch.equal(hdx, dx.cpu())
        assert rel_err(hy[2048:].float().numpy(), y_ref[2048:]) <= TOL
        assert rel_err(hy[2048:].float().numpy(), y[2048:].float().cpu().numpy()) <= 2e-3
        assert rel_err(hdA.numpy(), dA_ref) <= TOL and rel_err(hdB.numpy(), dB_ref) <= TOL
        # dB contracts the bf16 copy of the rank-r intermediate: a few of the tail chunk's entries round the other way
        assert rel_err(hdA.numpy(), dA.cpu().numpy()) <= 1e-5 and rel_err(hdB.numpy(), dB.cpu().numpy()) <= 5e-4


@pytest.mark.gpu
def test_host_step_whose_short_last_chunk_needs_more_scratch_than_a_full_one():
    # 2560 rows of a 1024 x 768 layer: two chunks of 1024 rows and one of 512, whose kernels cut
    # their reductions into more parts and keep larger fp32 partial results than a full chunk's.
    # The staging area must be sized for both; the results are those of the whole-batch device
    # calls (rows are independent in y and dx: bit for bit on the full chunks' rows).
    cfg = LayerConfig("hostchunks_tail", 1024, 768, 32, 4, 64, 1.0, 2560, seed=23)
    layer = GpuLayer(cfg)
    assert Q.qalora_workspace_bytes(layer.d, 512, Q.OP_TRAIN) > Q.qalora_workspace_bytes(layer.d, 1024, Q.OP_TRAIN)
    y = layer.forward()
    dx, dA, dB = layer.backward()
    pin = lambda t: t.pin_memory()
    hx, hdy = pin(layer.cpu["x"]), pin(layer.cpu["dy"])
    hy, hdx = pin(torch.zeros_like(y, device="cpu")), pin(torch.zeros_like(dx, device="cpu"))
    hdA, hdB = pin(torch.zeros_like(dA, device="cpu")), pin(torch.zeros_like(dB, device="cpu"))
    staging = torch.zeros(Q.qalora_step_host_bytes(layer.d, cfg.tokens), dtype=torch.uint8, device="cuda")
    Q.qalora_step_host(layer.d, cfg.tokens, hx, hdy, layer.codes, layer.qparams, layer.dev["A"], layer.dev["B"],
                       hy, hdx, hdA, hdB, staging)
    torch.cuda.synchronize()
    assert Q.workspace_status(staging) == 0
    assert torch.equal(hy[:2048], y[:2048].cpu()) and torch.equal(hdx[:2048], dx[:2048].cpu())
    # (the short chunk adds its partial results in another order: one bf16 step of the largest output at most)
    assert rel_err(hy[2048:].float().numpy(), y[2048:].float().cpu().numpy()) <= 4e-3
    assert rel_err(hdx[2048:].float().numpy(), dx[2048:].float().cpu().numpy()) <= 4e-3
    assert rel_err(hdA.numpy(), dA.cpu().numpy()) <= 1e-4 and rel_err(hdB.numpy(), dB.cpu().numpy()) <= 1e-3
