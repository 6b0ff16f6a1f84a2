"""qalora_forward_static is the forward pass for callers that have no way to
allocate device memory (for instance a plugin living inside an engine that owns
the whole device heap): its scratch is a fixed array built into the library.
It must give what qalora_forward gives, call after call, although every call
reuses the same scratch and finds the previous call's data in it.

This file is named so that pytest collects it last."""
import pytest
import torch

from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import LayerConfig, make_inputs

pytestmark = pytest.mark.gpu
TOL = 5e-3


def _rel(a, b):
    a, b = a.double(), b.double()
    return float((a - b).abs().max() / b.abs().max())


def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row():
    cfg = LayerConfig("noalloc", 512, 384, 64, 4, 64, 1.0, 200, seed=123)
    t = {k: v.cuda() for k, v in make_inputs(cfg, need=("W", "x", "A", "B")).items()}
    d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, cfg.rank, cfg.scale)
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, t["W"], codes, qparams)

    # two different batches (the second one small enough to take the few-token path),
    # so that the second call runs over scratch the first one has dirtied
    batches = [t["x"], (t["x"][:9] * 3).contiguous()]
    for x in batches:
        m = x.shape[0]
        want = torch.empty((m, cfg.d_out), dtype=torch.bfloat16, device="cuda")
        Q.qalora_forward(d, m, x, codes, qparams, t["A"], t["B"], want, Q.alloc_workspace(d, m, Q.OP_FORWARD))
        got = torch.full((m, cfg.d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
        Q.qalora_forward_static(d, m, x, codes, qparams, t["A"], t["B"], got)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        assert _rel(got, want) <= TOL
    # and once more with the first batch: still the same answer
    x = batches[0]
    again = torch.empty((x.shape[0], cfg.d_out), dtype=torch.bfloat16, device="cuda")
    Q.qalora_forward_static(d, x.shape[0], x, codes, qparams, t["A"], t["B"], again)
    want = torch.empty_like(again)
    Q.qalora_forward(d, x.shape[0], x, codes, qparams, t["A"], t["B"], want, Q.alloc_workspace(d, x.shape[0], Q.OP_FORWARD))
    torch.cuda.synchronize()
    assert _rel(again, want) <= TOL


def test_static_scratch_on_a_wide_layer_takes_what_fits_and_refuses_the_rest():
    """On a 4096-wide layer 17 rows still run on the few-token kernel, which needs no partial
    results: the built-in scratch is enough and the answer is qalora_forward's.  At 64 rows the
    forward pass cuts its reduction into parts that meet in scratch (several times rows x 4096
    floats), more than the array holds: the call is refused and nothing runs."""
    cfg = LayerConfig("noalloc_wide", 4096, 4096, 32, 4, 64, 1.0, 64, seed=124)
    t = {k: v.cuda() for k, v in make_inputs(cfg, need=("W", "x", "A", "B")).items()}
    d = Q.desc(cfg.d_in, cfg.d_out, cfg.group_size, cfg.bits, cfg.rank, cfg.scale)
    codes, qparams = Q.alloc_packed(d)
    Q.qalora_quantize(d, t["W"], codes, qparams)
    x17 = t["x"][:17].contiguous()
    assert Q.qalora_workspace_bytes(d, 17, Q.OP_FORWARD) <= Q.STATIC_SCRATCH_BYTES
    want = torch.empty((17, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    Q.qalora_forward(d, 17, x17, codes, qparams, t["A"], t["B"], want, Q.alloc_workspace(d, 17, Q.OP_FORWARD))
    for _ in range(2):
        got = torch.full((17, cfg.d_out), float("nan"), dtype=torch.bfloat16, device="cuda")
        Q.qalora_forward_static(d, 17, x17, codes, qparams, t["A"], t["B"], got)
        torch.cuda.synchronize()
        assert _rel(got, want) <= TOL
    assert Q.qalora_workspace_bytes(d, 64, Q.OP_FORWARD) > Q.STATIC_SCRATCH_BYTES
    y64 = torch.zeros((64, cfg.d_out), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_forward_static(d, 64, t["x"], codes, qparams, t["A"], t["B"], y64)
    assert e.value.status == -7
    torch.cuda.synchronize()
    assert float(y64.float().abs().max()) == 0.0          # nothing was launched


def test_static_scratch_refuses_requests_beyond_its_size():
    d = Q.desc(512, 384, 64, 4, 64, 1.0)
    too_many = Q.STATIC_SCRATCH_BYTES // (64 * 6) + 64
    assert Q.qalora_workspace_bytes(d, too_many, Q.OP_FORWARD) > Q.STATIC_SCRATCH_BYTES
    x = torch.zeros((too_many, 512), dtype=torch.bfloat16, device="cuda")
    y = torch.zeros((too_many, 384), dtype=torch.bfloat16, device="cuda")
    codes, qparams = Q.alloc_packed(d)
    A = torch.zeros((8, 64), dtype=torch.bfloat16, device="cuda")
    B = torch.zeros((64, 384), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_forward_static(d, too_many, x, codes, qparams, A, B, y)
    assert e.value.status == -7
    assert "scratch" in Q.status_string(-7)
