"""qalora_forward_group: several independent layers in one call.  Merged (rank 0) layers with a
few rows each take ONE kernel launch; the result must match the oracle layer by layer, and agree
with what one qalora_forward per layer gives.  Groups the one-launch path does not cover
(adapters, more rows) fall back to per-layer launches with the same results."""
import numpy as np
import pytest
import torch

from conftest import record_margin
from oracle import qalora_oracle as O
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200.synthetic import LayerConfig, make_inputs, to_f64

pytestmark = pytest.mark.gpu
TOL = 5e-3


def rel(got, ref):
    got, ref = np.asarray(got, dtype=np.float64), np.asarray(ref, dtype=np.float64)
    return float(np.max(np.abs(got - ref)) / np.max(np.abs(ref)))


def build_layers(shapes, bits, g, M, rank):
    out = []
    for i, (K, N) in enumerate(shapes):
        cfg = LayerConfig(f"group{i}", K, N, g, bits, max(rank, 8), 1.5, M, outlier_frac=0.01, seed=300 + 7 * i + bits)
        cpu = make_inputs(cfg, need=("W", "x", "A", "B"))
        d = Q.desc(K, N, g, bits, rank, cfg.scale)
        codes, qparams = Q.alloc_packed(d)
        Q.qalora_quantize(d, cpu["W"].cuda(), codes, qparams)
        out.append({"cfg": cfg, "cpu": cpu, "d": d, "codes": codes, "qparams": qparams, "x": cpu["x"].cuda(),
                    "A": cpu["A"].cuda() if rank else None, "B": cpu["B"].cuda() if rank else None,
                    "y": torch.full((M, N), float("nan"), dtype=torch.bfloat16, device="cuda")})
    return out


def run_group(layers, M):
    tuples = [(L["d"], L["x"], L["codes"], L["qparams"], L["A"], L["B"], L["y"]) for L in layers]
    ws = torch.full((max(Q.qalora_forward_group_workspace_bytes(tuples, M), 16),), 0xFF, dtype=torch.uint8, device="cuda")
    n0 = Q.qalora_kernel_launches()
    Q.qalora_forward_group(tuples, M, ws)
    torch.cuda.synchronize()
    assert Q.workspace_status(ws) == 0
    return Q.qalora_kernel_launches() - n0


def check_against_oracle(layers, M, case, rank):
    for i, L in enumerate(layers):
        cfg = L["cfg"]
        codes, alpha, beta = O.quantize(L["cpu"]["W"].numpy(), cfg.group_size, cfg.bits)
        x = to_f64(L["cpu"]["x"])
        if rank:
            y_ref = O.forward(x, codes, alpha, beta, cfg.group_size, to_f64(L["cpu"]["A"]), to_f64(L["cpu"]["B"]), cfg.scale)
        else:
            y_ref = O.forward(x, codes, alpha, beta, cfg.group_size)
        record_margin(case, f"y{i}", rel(L["y"].float().cpu().numpy(), y_ref), TOL)
        # and the same layer on its own
        alone = torch.empty_like(L["y"])
        Q.qalora_forward(L["d"], M, L["x"], L["codes"], L["qparams"], L["A"], L["B"], alone,
                         Q.alloc_workspace(L["d"], M, Q.OP_FORWARD))
        torch.cuda.synchronize()
        assert rel(L["y"].float().cpu().numpy(), alone.float().cpu().numpy()) <= 2 ** -7     # both are roundings of nearly equal sums


@pytest.mark.parametrize("bits,g,M", [(4, 32, 1), (4, 128, 8), (3, 64, 16), (2, 32, 5)])
def test_merged_layers_of_different_shapes_run_in_one_launch(bits, g, M):
    shapes = [(512, 384), (1280, 256), (512, 128), (2048, 640)]        # different d_in and d_out
    layers = build_layers(shapes, bits, g, M, rank=0)
    launches = run_group(layers, M)
    assert launches == 1 and Q.qalora_main_kernel_name() == "qalora_gemv_group_kernel"
    check_against_oracle(layers, M, f"group_b{bits}_g{g}_m{M}", 0)


def test_eight_layers_take_one_launch_and_nine_run_one_by_one():
    # the work list holds up to eight layers; one of them has a single 128-channel stage, so the
    # whole group runs with one slice per column tile
    shapes = [(512, 384), (1280, 256), (128, 128), (2048, 640), (384, 1152), (896, 128), (640, 512), (256, 256)]
    layers = build_layers(shapes, 4, 32, 3, rank=0)
    assert run_group(layers, 3) == 1 and Q.qalora_main_kernel_name() == "qalora_gemv_group_kernel"
    check_against_oracle(layers, 3, "group_of_8", 0)
    layers = build_layers(shapes + [(512, 128)], 4, 32, 3, rank=0)
    assert run_group(layers, 3) == 9
    check_against_oracle(layers, 3, "group_of_9", 0)


def test_groups_outside_the_one_launch_path_fall_back_layer_by_layer():
    # adapters: pooling kernel + few-token kernel per layer
    layers = build_layers([(512, 384), (1280, 256)], 4, 32, 4, rank=16)
    assert run_group(layers, 4) == 4
    check_against_oracle(layers, 4, "group_adapted_m4", 16)
    # many rows: the tensor-core path per layer (one of the shapes only tiles on the CUDA-core kernels)
    layers = build_layers([(512, 384), (320, 200)], 4, 32, 70, rank=0)
    assert run_group(layers, 70) >= 2
    check_against_oracle(layers, 70, "group_m70", 0)
    # an empty group and zero rows are no-ops
    Q.qalora_forward_group([], 4, torch.zeros(256, dtype=torch.uint8, device="cuda"))
    layers = build_layers([(512, 384)], 4, 32, 4, rank=0)
    with pytest.raises(Q.QaloraError) as e:                             # one bad layer rejects the whole call
        bad = [(L["d"], L["x"], L["codes"], L["qparams"], L["A"], L["B"], L["y"]) for L in layers] + \
              [(Q.desc(512, 384, 32, 4, 0, 1.0), None, layers[0]["codes"], layers[0]["qparams"], None, None, layers[0]["y"])]
        Q.qalora_forward_group(bad, 4, torch.zeros(4096, dtype=torch.uint8, device="cuda"))
    assert e.value.status == -2
