"""Seeded synthetic inputs for the QA-LoRA layer.

This module only draws random tensors.  It holds none of the method's
arithmetic and is the one piece shared by the CUDA path's tests and the CPU
oracle's tests, so that both sides see identical stored values.

Recipe (stands in for LLaMA projection weights and instruction-tuning batches,
which are not available offline): weights are Gaussian with standard deviation
0.02, optionally with a fraction of entries multiplied by 10 to mimic the
outlier channels of language-model weights; activations x are N(0, 1); the
adapter factors A, B are N(0, 0.02^2); the output gradient dy is N(0, dy_std^2).
All draws come from one `torch.Generator` on the CPU, in the fixed order
W, outlier mask, x, A, B, dy.  Tensors stored as bf16 are drawn in fp32 and
rounded once.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class LayerConfig:
    name: str
    d_in: int            # K
    d_out: int           # N
    group_size: int      # g (the paper's D_in / L)
    bits: int            # b
    rank: int            # r
    scale: float         # s
    tokens: int          # M
    dy_std: float = 1.0
    outlier_frac: float = 0.0
    outlier_gain: float = 10.0
    seed: int = 0

    @property
    def groups(self) -> int:
        return self.d_in // self.group_size

    def with_(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


# The benchmark configurations: LLaMA-shaped layers.
CONFIGS = {
    "cfg1_512": LayerConfig("cfg1_512", 512, 512, 32, 4, 16, 2.0, 64, 1.0, 0.0, 10.0, 0),
    "cfg2_7b_attn": LayerConfig("cfg2_7b_attn", 4096, 4096, 32, 4, 64, 1.0, 16, 1.0, 1e-3, 10.0, 1),
    "cfg3_7b_up": LayerConfig("cfg3_7b_up", 4096, 11008, 32, 4, 64, 1.0, 8192, 1e-2, 0.0, 10.0, 2),
    "cfg3_7b_down": LayerConfig("cfg3_7b_down", 11008, 4096, 32, 4, 64, 1.0, 8192, 1e-2, 0.0, 10.0, 2),
    "cfg4_13b_up": LayerConfig("cfg4_13b_up", 5120, 13824, 32, 3, 64, 1.0, 4096, 1e-2, 0.0, 10.0, 3),
    "cfg4_13b_down": LayerConfig("cfg4_13b_down", 13824, 5120, 32, 3, 64, 1.0, 4096, 1e-2, 0.0, 10.0, 3),
    "cfg4_13b_attn": LayerConfig("cfg4_13b_attn", 5120, 5120, 32, 3, 64, 1.0, 4096, 1e-2, 0.0, 10.0, 3),
    "cfg5_65b_up": LayerConfig("cfg5_65b_up", 8192, 22016, 32, 4, 64, 1.0, 8192, 1e-2, 0.0, 10.0, 4),
    "cfg5_65b_down": LayerConfig("cfg5_65b_down", 22016, 8192, 32, 4, 64, 1.0, 8192, 1e-2, 0.0, 10.0, 4),
    "cfg5_65b_attn": LayerConfig("cfg5_65b_attn", 8192, 8192, 32, 4, 64, 1.0, 8192, 1e-2, 0.0, 10.0, 4),
}


def make_inputs(cfg: LayerConfig, need=("W", "x", "A", "B", "dy")) -> dict:
    """Draw the tensors of one layer on the CPU.

    Returns a dict with W fp32 [K, N]; x bf16 [M, K]; A bf16 [G, r]; B bf16
    [r, N]; dy bf16 [M, N].  Every tensor is always drawn (so that the stream of
    random numbers does not depend on `need`); entries not in `need` are dropped
    before returning.
    """
    gen = torch.Generator(device="cpu")
    gen.manual_seed(cfg.seed)
    K, N, M, G, r = cfg.d_in, cfg.d_out, cfg.tokens, cfg.groups, cfg.rank
    out = {}
    W = torch.randn(K, N, generator=gen, dtype=torch.float32) * 0.02
    if cfg.outlier_frac > 0.0:
        mask = torch.rand(K, N, generator=gen) < cfg.outlier_frac
        W = torch.where(mask, W * cfg.outlier_gain, W)
    out["W"] = W if "W" in need else None
    del W
    x = torch.randn(M, K, generator=gen, dtype=torch.float32)
    out["x"] = x.to(torch.bfloat16) if "x" in need else None
    del x
    A = torch.randn(G, r, generator=gen, dtype=torch.float32) * 0.02
    out["A"] = A.to(torch.bfloat16) if "A" in need else None
    B = torch.randn(r, N, generator=gen, dtype=torch.float32) * 0.02
    out["B"] = B.to(torch.bfloat16) if "B" in need else None
    dy = torch.randn(M, N, generator=gen, dtype=torch.float32) * cfg.dy_std
    out["dy"] = dy.to(torch.bfloat16) if "dy" in need else None
    del dy
    return {k: v for k, v in out.items() if v is not None}


def to_f64(t: torch.Tensor):
    """Exact widening of a stored tensor to a numpy fp64 array."""
    return t.detach().cpu().to(torch.float64).numpy()


def make_optimizer_inputs(n: int, steps: int, seed: int = 0, grad_scales=(1e-4, 1.0)) -> dict:
    """Seeded inputs for the adapter update: float32 parameters N(0, 0.02^2) and one
    gradient array per step, N(0, scale^2) with the scales taken in turn (a small one
    keeps the joint norm below the clipping bound of 0.3 for short arrays, a large one
    exceeds it), so that both branches of the clipping rule are visited."""
    gen = torch.Generator(device="cpu").manual_seed(seed)
    param = torch.randn(n, generator=gen, dtype=torch.float32) * 0.02
    grads = [torch.randn(n, generator=gen, dtype=torch.float32) * grad_scales[t % len(grad_scales)]
             for t in range(steps)]
    return {"param": param, "grads": grads}
