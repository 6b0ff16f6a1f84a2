"""Data parallelism over token rows.

Rows of x are independent, so every rank runs the forward pass and dX on its own
rows with the (replicated) codes, qparams, A and B and exchanges nothing.  dA and
dB are sums over rows: one all-reduce (sum, fp32) of (G*r + r*N) values per layer
is the only exchange step.  torch.distributed carries it (NCCL between GPUs,
gloo on CPU in the tests)."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(m: int, rank: int, world: int):
    """Contiguous, balanced slice [start, stop) of m token rows owned by `rank`."""
    if not (0 <= rank < world):
        raise ValueError("rank outside the group")
    base, extra = divmod(m, world)
    start = rank * base + min(rank, extra)
    return start, start + base + (1 if rank < extra else 0)


def allreduce_adapter_grads(dA: torch.Tensor, dB: torch.Tensor, group=None):
    """Sums the per-rank adapter gradients in place over the process group."""
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(dA, op=dist.ReduceOp.SUM, group=group)
        dist.all_reduce(dB, op=dist.ReduceOp.SUM, group=group)
    return dA, dB


class AdapterBucket:
    """All trained values of a model (every layer's A [G][r] and B [r][N]) in flat arrays.

    One flat float32 gradient array means ONE all-reduce per step whatever the number of
    layers (bucket sized for launch latency, not per tensor), and one clipped-AdamW call
    (Section 4.1: AdamW, maximum gradient norm 0.3) whose norm is joint over all layers.
    `grads(i)` returns the (dA, dB) views that qalora_backward of layer i writes into;
    `factors(i)` the bf16 (A, B) views that qalora_forward reads.  Every view starts on a
    16-byte boundary because each size is a multiple of 8 (the rank is).
    """

    def __init__(self, layers, device="cpu"):
        # layers: iterable of (G, r, N)
        self.offsets = []
        n = 0
        for G, r, N in layers:
            if r <= 0 or r % 8 != 0:
                raise ValueError("rank must be a positive multiple of 8")
            self.offsets.append((n, n + G * r, (G, r), (r, N)))
            n += G * r + r * N
        self.n = n
        self.device = torch.device(device)
        z = lambda dt: torch.zeros(n, dtype=dt, device=self.device)
        self.grad, self.master, self.exp_avg, self.exp_avg_sq = z(torch.float32), z(torch.float32), z(torch.float32), z(torch.float32)
        self.bf16 = z(torch.bfloat16)
        self.norm = torch.zeros(2, dtype=torch.float32, device=self.device)
        self.step_count = 0
        self._workspace = None

    def _views(self, flat, i):
        a0, b0, sa, sb = self.offsets[i]
        return flat[a0:b0].view(sa), flat[b0:b0 + sb[0] * sb[1]].view(sb)

    def grads(self, i):
        return self._views(self.grad, i)

    def factors(self, i):
        return self._views(self.bf16, i)

    def load(self, i, A, B):
        """Sets layer i's master copy (float32) and its bf16 copy from given factors."""
        mA, mB = self._views(self.master, i)
        mA.copy_(A.to(torch.float32)); mB.copy_(B.to(torch.float32))
        bA, bB = self.factors(i)
        bA.copy_(mA.to(torch.bfloat16)); bB.copy_(mB.to(torch.bfloat16))

    def reduce(self, group=None):
        """Sums the gradient bucket over the data-parallel ranks: the step's only exchange."""
        if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
            dist.all_reduce(self.grad, op=dist.ReduceOp.SUM, group=group)
        return self.grad

    def update(self, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, max_grad_norm=0.3, stream=None):
        """Clipped AdamW on the device through the CUDA library (no CPU path)."""
        from . import binding as Q
        if self.device.type != "cuda":
            raise RuntimeError("AdapterBucket.update runs on a CUDA device only")
        if self._workspace is None:
            self._workspace = torch.zeros(Q.qalora_adamw_workspace_bytes(), dtype=torch.uint8, device=self.device)
        self.step_count += 1
        h = Q.adamw_hyper(self.step_count, lr, beta1, beta2, eps, weight_decay, max_grad_norm)
        Q.qalora_adamw_step(h, self.n, self.grad, self.master, self.exp_avg, self.exp_avg_sq, self.bf16, self.norm,
                            self._workspace, stream)


class AdaptedLayer:
    """One quantized layer of a data-parallel fine-tuning step: its descriptor, packed codes and
    (alpha, beta) (frozen, replicated on every rank) and the workspace its forward and backward
    pass share for `tokens` rows per rank (the pooled input is computed once per step).  The
    trained factors are not here: they live in the AdapterBucket."""

    def __init__(self, d, codes, qparams, tokens: int):
        from . import binding as Q
        self.d, self.codes, self.qparams, self.tokens = d, codes, qparams, tokens
        self.workspace = Q.alloc_workspace(d, tokens, Q.OP_TRAIN, device=codes.device)

    @property
    def shape(self):
        """(G, r, N): the entry AdapterBucket wants for this layer."""
        return self.d.d_in // self.d.group_size, self.d.rank, self.d.d_out


def finetune_step(layers, bucket: AdapterBucket, xs, dys, ys, dxs, lr, group=None, stream=None, **adamw):
    """One data-parallel fine-tuning step over `layers` (Section 4.1: only A and B are trained,
    AdamW with a maximum gradient norm), every piece of it a call into the CUDA library:

      forward of layer i from the bucket's bf16 factors  -> ys[i]  (keeps pool(x) and T for the backward pass)
      backward of layer i, dA and dB written STRAIGHT into the bucket's gradient views, dX -> dxs[i]
      ONE all-reduce of the whole gradient array over the ranks (the step's only exchange)
      ONE clipped AdamW update of every factor; it also refreshes the bf16 copies the next
      step's forward reads.

    xs[i] / dys[i] are this rank's rows of layer i's input and output gradient (each layer has its
    own here: the layers are independent linear layers, not a chain).  Everything is enqueued on
    `stream` (torch's current stream by default) without synchronizing."""
    from . import binding as Q
    for i, L in enumerate(layers):
        A, B = bucket.factors(i)
        Q.qalora_forward_train(L.d, L.tokens, xs[i], L.codes, L.qparams, A, B, ys[i], L.workspace, stream)
    for i, L in enumerate(layers):
        A, B = bucket.factors(i)
        dA, dB = bucket.grads(i)
        Q.qalora_backward_train(L.d, L.tokens, xs[i], dys[i], L.codes, L.qparams, A, B, dxs[i], dA, dB, L.workspace, stream)
    bucket.reduce(group)
    bucket.update(lr, stream=stream, **adamw)
