"""The multi-GPU path on CPU: two gloo ranks, each taking its slice of the token
rows; summing the per-rank adapter gradients with the package's all-reduce must
give the full-batch gradients, and the row slices must tile the batch."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import qalora_oracle as O
from paper_2309_14717_b200 import dp
from paper_2309_14717_b200.synthetic import LayerConfig, make_inputs, to_f64

CFG = LayerConfig("dp", 128, 48, 32, 4, 8, 1.5, 37, seed=3)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        t = make_inputs(CFG)
        lo, hi = dp.shard_rows(CFG.tokens, rank, world)
        dA, dB = O.backward_adapter(to_f64(t["x"][lo:hi]), to_f64(t["dy"][lo:hi]), CFG.group_size,
                                    to_f64(t["A"]), to_f64(t["B"]), CFG.scale)
        dA_t, dB_t = torch.from_numpy(dA).float(), torch.from_numpy(dB).float()
        dp.allreduce_adapter_grads(dA_t, dB_t)
        if rank == 0:
            out.put((dA_t.numpy(), dB_t.numpy()))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_ranks_sum_to_the_full_batch_gradients():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    dA, dB = out.get(timeout=90)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    t = make_inputs(CFG)
    dA_ref, dB_ref = O.backward_adapter(to_f64(t["x"]), to_f64(t["dy"]), CFG.group_size, to_f64(t["A"]),
                                        to_f64(t["B"]), CFG.scale)
    assert np.max(np.abs(dA - dA_ref)) <= 1e-5 * np.max(np.abs(dA_ref))
    assert np.max(np.abs(dB - dB_ref)) <= 1e-5 * np.max(np.abs(dB_ref))


@pytest.mark.parametrize("m,world", [(37, 2), (8192, 8), (5, 8), (0, 3)])
def test_row_slices_tile_the_batch(m, world):
    cuts = [dp.shard_rows(m, r, world) for r in range(world)]
    assert cuts[0][0] == 0 and cuts[-1][1] == m
    for (a, b), (c, d) in zip(cuts, cuts[1:]):
        assert b == c and a <= b
    sizes = [b - a for a, b in cuts]
    assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        dp.shard_rows(m, world, world)


LAYERS = [(4, 8, 48), (6, 16, 24), (4, 8, 40)]        # (G, r, N) of three layers


def _bucket_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        b = dp.AdapterBucket(LAYERS)
        for i in range(len(LAYERS)):
            dA, dB = b.grads(i)
            g = torch.Generator().manual_seed(100 * rank + i)
            dA.copy_(torch.randn(dA.shape, generator=g)); dB.copy_(torch.randn(dB.shape, generator=g))
        b.reduce()
        if rank == 0:
            out.put(b.grad.numpy().copy())
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_bucket_views_and_single_allreduce():
    b = dp.AdapterBucket(LAYERS)
    assert b.n == sum(G * r + r * N for G, r, N in LAYERS)
    spans = []
    for i, (G, r, N) in enumerate(LAYERS):
        dA, dB = b.grads(i)
        A, B = b.factors(i)
        assert dA.shape == (G, r) == A.shape and dB.shape == (r, N) == B.shape
        assert dA.data_ptr() % 16 == 0 and dB.data_ptr() % 16 == 0 and A.data_ptr() % 16 == 0 and B.data_ptr() % 16 == 0
        spans += [(dA.data_ptr(), dA.numel() * 4), (dB.data_ptr(), dB.numel() * 4)]
    spans.sort()
    assert spans[0][0] == b.grad.data_ptr() and sum(s for _, s in spans) == b.n * 4
    for (p, s), (q, _) in zip(spans, spans[1:]):
        assert p + s == q                                # the views tile the bucket without gaps
    with pytest.raises(ValueError):
        dp.AdapterBucket([(4, 12, 48)])
    with pytest.raises(RuntimeError):
        b.update(2e-5)                                   # no CPU path for the optimizer
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_bucket_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = out.get(timeout=90)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = np.zeros(b.n, dtype=np.float32)
    for rank in range(world):
        off = 0
        for i, (G, r, N) in enumerate(LAYERS):
            g = torch.Generator().manual_seed(100 * rank + i)
            for shape in ((G, r), (r, N)):
                t = torch.randn(shape, generator=g).numpy().ravel()
                want[off:off + t.size] += t
                off += t.size
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-6)
