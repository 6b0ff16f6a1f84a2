"""Parity of the CUDA adapter update (clipped AdamW, Section 4.1) with the fp64 oracle.

Both sides start from the same seeded float32 state and run the same gradients; the oracle
never sees a value the GPU produced.  Tolerances: the GPU keeps the state in float32, so a
parameter is compared against the accumulated movement t * lr (rounding a parameter of size
0.02-0.1 to float32 costs up to 4e-9 per step, 2e-4 of lr = 2e-5), the moments against
their largest magnitude."""
import numpy as np
import pytest
import torch

from oracle import optimizer_oracle as P
from paper_2309_14717_b200 import binding as Q
from paper_2309_14717_b200 import dp
from paper_2309_14717_b200.synthetic import make_optimizer_inputs

pytestmark = pytest.mark.gpu


def _run(n, steps, lr, wd, max_norm, seed, scales=(1e-4, 1.0)):
    t = make_optimizer_inputs(n, steps, seed, scales)
    dev = lambda a: a.cuda()
    p, m, v = dev(t["param"].clone()), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    pb = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
    norm = torch.zeros(2, device="cuda")
    ws = torch.zeros(Q.qalora_adamw_workspace_bytes(), dtype=torch.uint8, device="cuda")
    op, om, ov = [t["param"].double().numpy()], [np.zeros(n)], [np.zeros(n)]
    for s in range(1, steps + 1):
        g = t["grads"][s - 1]
        h = Q.adamw_hyper(s, lr, weight_decay=wd, max_grad_norm=max_norm)
        Q.qalora_adamw_step(h, n, dev(g), p, m, v, pb, norm, ws)
        torch.cuda.synchronize()
        # the oracle takes the hyperparameters as the C struct holds them (float32 values)
        op, om, ov, onorm, ocoef = P.adamw_step(op, [g.double().numpy()], om, ov, s, h.lr, h.beta1, h.beta2, h.eps,
                                                h.weight_decay, h.max_grad_norm)
        if n == 0:
            continue
        gn, gc = norm.cpu().tolist()
        assert gn == pytest.approx(onorm, rel=2e-6) and gc == pytest.approx(ocoef, rel=2e-6)
        move = s * lr * (1.0 + wd)
        assert np.max(np.abs(p.cpu().double().numpy() - op[0])) <= 1e-3 * move
        assert np.max(np.abs(m.cpu().double().numpy() - om[0])) <= 1e-5 * np.max(np.abs(om[0]))
        assert np.max(np.abs(v.cpu().double().numpy() - ov[0])) <= 1e-5 * np.max(np.abs(ov[0]))
        assert torch.equal(pb, p.to(torch.bfloat16))       # the bf16 copy is the master rounded once
    return p, m, v


@pytest.mark.parametrize("n", [0, 3, 8, 4099, 1_000_003, 5_000_000])
def test_adamw_matches_oracle_over_steps(n):
    _run(n, 4, 2e-5, 0.0, 0.3, seed=n % 97)


@pytest.mark.parametrize("wd,max_norm,lr", [(0.05, 0.3, 1e-3), (0.0, 0.0, 2e-5), (0.1, 1e-3, 1e-5)])
def test_adamw_variants(wd, max_norm, lr):
    _run(300_000, 3, lr, wd, max_norm, seed=5)


def test_both_sides_of_the_clipping_bound_are_visited():
    t = make_optimizer_inputs(4099, 2, 9)
    norms = [P.grad_norm([g.double().numpy()]) for g in t["grads"]]
    assert norms[0] < 0.3 < norms[1]


def test_update_is_reproducible_bit_for_bit():
    a = _run(1_000_003, 2, 2e-5, 0.0, 0.3, seed=1)
    b = _run(1_000_003, 2, 2e-5, 0.0, 0.3, seed=1)
    for x, y in zip(a, b):
        assert torch.equal(x, y)


def test_bucket_update_feeds_the_layers():
    layers = [(16, 8, 64), (8, 16, 32)]
    b = dp.AdapterBucket(layers, device="cuda")
    gen = torch.Generator().manual_seed(4)
    A0 = [torch.randn(G, r, generator=gen) * 0.02 for G, r, N in layers]
    B0 = [torch.randn(r, N, generator=gen) * 0.02 for G, r, N in layers]
    for i in range(len(layers)):
        b.load(i, A0[i].cuda(), B0[i].cuda())
    grads = []
    for i in range(len(layers)):
        dA, dB = b.grads(i)
        gA, gB = torch.randn(dA.shape, generator=gen), torch.randn(dB.shape, generator=gen)
        dA.copy_(gA.cuda()); dB.copy_(gB.cuda())
        grads += [gA.double().numpy(), gB.double().numpy()]
    b.reduce()                                             # one rank: nothing to exchange
    b.update(2e-5)
    torch.cuda.synchronize()
    params = []
    for i in range(len(layers)):
        params += [A0[i].double().numpy(), B0[i].double().numpy()]
    zeros = [np.zeros_like(q) for q in params]
    h = Q.adamw_hyper(1, 2e-5)
    new_p, _, _, onorm, ocoef = P.adamw_step(params, grads, zeros, [z.copy() for z in zeros], 1, h.lr, h.beta1, h.beta2,
                                             h.eps, h.weight_decay, h.max_grad_norm)
    assert b.norm[0].item() == pytest.approx(onorm, rel=2e-6) and ocoef < 1.0
    for i in range(len(layers)):
        A, B = b.factors(i)
        for got, want in ((A, new_p[2 * i]), (B, new_p[2 * i + 1])):
            want_bf16 = torch.from_numpy(want).to(torch.float32).to(torch.bfloat16)
            # bf16 of the fp32 master against bf16 of the oracle's value: equal except where the
            # float32 rounding of the master crosses a bf16 boundary (at most one bf16 ulp)
            diff = (got.cpu().float() - want_bf16.float()).abs()
            assert float(diff.max()) <= float(want_bf16.float().abs().max()) * 2.0 ** -7
            assert float((diff > 0).float().mean()) < 0.01


def test_bad_arguments_are_rejected_without_a_launch():
    z = torch.zeros(8, device="cuda")
    zb = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(Q.qalora_adamw_workspace_bytes(), dtype=torch.uint8, device="cuda")
    for h in (Q.adamw_hyper(0, 1e-3), Q.adamw_hyper(1, 1e-3, beta1=1.0), Q.adamw_hyper(1, -1.0),
              Q.adamw_hyper(1, 1e-3, eps=float("nan"))):
        with pytest.raises(Q.QaloraError) as e:
            Q.qalora_adamw_step(h, 8, z, z, z, z, zb, None, ws)
        assert e.value.status == -1
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_adamw_step(Q.adamw_hyper(1, 1e-3), 8, z, z, z, z, zb, None, ws[:16])
    assert e.value.status == -5
    with pytest.raises(Q.QaloraError) as e:
        Q.qalora_adamw_step(Q.adamw_hyper(1, 1e-3), 8, z[1:], z, z, z, zb, None, ws)
    assert e.value.status == -4
