"""Parity of the fused local-optimiser kernels and the replica averaging with the CPU oracle.

Tolerance: parameters within 1e-6 relative (normwise per replica, and max-abs against the largest
parameter) after each step; optimiser state within 1e-6 relative normwise.
"""
import numpy as np
import pytest
import torch

import oracle.abs_oracle as orc
import paper_2406_13936_b200 as pkg

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = pkg.Context(0)
    yield c
    c.close()


def f64(t):
    return t.detach().cpu().numpy().astype(np.float64)


def close(gpu, ref, tol=1e-6):
    g = f64(gpu)
    for m in range(ref.shape[0]):
        denom = np.linalg.norm(ref[m])
        assert np.linalg.norm(g[m] - ref[m]) <= tol * max(denom, 1e-30)
    assert np.abs(g - ref).max() <= tol * max(np.abs(ref).max(), 1e-30)


def replicas(seed, M, d, stride=None, offset=0, std=1.0):
    """[M, d] view (replica stride `stride`, start shifted by `offset` floats) of random values."""
    stride = stride or d
    gen = torch.Generator().manual_seed(seed)
    buf = torch.zeros(M * stride + offset + 8, device="cuda")
    view = buf[offset:offset + M * stride].view(M, stride)[:, :d]
    view.copy_((torch.randn((M, d), generator=gen) * std).cuda())
    return view


LAYOUTS = [(1, 1, None, 0), (1, 1000, None, 0), (3, 4099, 4100, 0), (8, 5000, None, 0), (2, 777, 780, 1),
           (5, 64, 67, 0), (8, 262147, None, 0)]


@pytest.mark.parametrize("average", [False, True])
@pytest.mark.parametrize("M,d,stride,offset", LAYOUTS)
def test_sgd_step(ctx, M, d, stride, offset, average):
    X = replicas(1, M, d, stride, offset)
    G = replicas(2, M, d, stride, offset)
    ref = orc.sgd_step(f64(X), f64(G), 0.1)
    if average:
        ref = orc.replica_average(ref)
    ctx.local_sgd_step(X, G, 0.1, average_after=average)
    close(X, ref)


@pytest.mark.parametrize("average", [False, True])
@pytest.mark.parametrize("M,d,stride,offset", LAYOUTS)
def test_adamw_steps(ctx, M, d, stride, offset, average):
    hp = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    X = replicas(3, M, d, stride, offset, std=0.02)
    m1 = replicas(4, M, d, stride, offset, std=0.0)
    m2 = replicas(5, M, d, stride, offset, std=0.0)
    for t in range(1, 5):
        G = replicas(10 + t, M, d, stride, offset, std=0.01)
        last = average and t == 4
        rx, rm, rv = orc.adamw_step(f64(X), f64(m1), f64(m2), f64(G), t=t, **hp)   # teacher-forced from GPU state
        if last:
            rx = orc.replica_average(rx)
        ctx.local_adamw_step(X, m1, m2, G, pkg.make_adamw_cfg(step=t, **hp), average_after=last)
        close(X, rx)
        close(m1, rm)
        close(m2, rv)


@pytest.mark.parametrize("average", [False, True])
@pytest.mark.parametrize("M,d,stride,offset", LAYOUTS[:5])
def test_shb_steps(ctx, M, d, stride, offset, average):
    X = replicas(6, M, d, stride, offset)
    U = replicas(7, M, d, stride, offset, std=0.0)
    for t in range(3):
        G = replicas(20 + t, M, d, stride, offset)
        rx, ru = orc.shb_step(f64(X), f64(U), f64(G), 0.05, 0.9, 1e-4)
        if average and t == 2:
            rx = orc.replica_average(rx)
        ctx.local_shb_step(X, U, G, 0.05, 0.9, 1e-4, average_after=(average and t == 2))
        close(X, rx)
        close(U, ru)


@pytest.mark.parametrize("M,d,stride,offset", LAYOUTS)
def test_replica_average(ctx, M, d, stride, offset):
    X = replicas(8, M, d, stride, offset)
    ref = orc.replica_average(f64(X))
    ctx.replica_average(X)
    close(X, ref)
    again = X.clone()
    ctx.replica_average(X)                      # idempotent up to rounding; identical replicas stay identical
    assert torch.equal(X[0], X[M - 1])
    close(X, f64(again))


def test_padding_between_replicas_is_untouched(ctx):
    M, d, stride = 3, 101, 128
    buf = torch.full((M * stride,), 7.0, device="cuda")
    X = buf.view(M, stride)[:, :d]
    G = torch.ones((M, stride), device="cuda")[:, :d]
    ctx.local_sgd_step(X, G, 0.5, average_after=True)
    assert torch.all(buf.view(M, stride)[:, d:] == 7.0)
    assert torch.all(X == 6.5)


def test_invalid_arguments(ctx):
    X = torch.zeros((2, 8), device="cuda")
    with pytest.raises(pkg.AbsError):
        ctx.local_adamw_step(X, X.clone(), X.clone(), X.clone(), pkg.make_adamw_cfg(1e-3, 0.9, 0.95, 1e-8, 0.0, 0))
    with pytest.raises(pkg.AbsError):
        ctx.local_adamw_step(X, X.clone(), X.clone(), X.clone(), pkg.make_adamw_cfg(1e-3, 1.0, 0.95, 1e-8, 0.0, 1))


def test_full_size_adamw_rounds_on_column_subsets(ctx):
    """The fused local AdamW configuration at full size: M=8 fp32 replicas of d=124,439,808 parameters,
    beta=(0.9, 0.95), wd=0.1, lr=3e-4, H=16 local steps per round with the averaging fused into the
    last, 20 rounds.  The update is coordinate-separable, so the oracle follows three column subsets
    (first, last and random 2^16 columns), restarted every round from the GPU's state."""
    from paper_2406_13936_b200 import inputs
    M, d, H, rounds, pool = 8, 124_439_808, 16, 20, 4
    hp = dict(lr=3e-4, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)
    X, m1, m2, grads = inputs.adamw_problem(4, M, d, pool=pool, device="cuda")
    gen = torch.Generator().manual_seed(1)
    cols = torch.cat([torch.arange(0, 1 << 16), torch.arange(d - (1 << 16), d),
                      torch.randint(0, d, (1 << 16,), generator=gen)]).cuda()
    g_sub = [f64(g[:, cols]) for g in grads]
    t = 0
    for k in range(rounds):
        xs, ms, vs = f64(X[:, cols]), f64(m1[:, cols]), f64(m2[:, cols])      # teacher forcing
        for h in range(H):
            t += 1
            last = h == H - 1
            ctx.local_adamw_step(X, m1, m2, grads[(t - 1) % pool], pkg.make_adamw_cfg(step=t, **hp),
                                 average_after=last)
            xs, ms, vs = orc.adamw_step(xs, ms, vs, g_sub[(t - 1) % pool], t=t, **hp)
            if last:
                xs = orc.replica_average(xs)
        close(X[:, cols], xs)
        close(m1[:, cols], ms)
        close(m2[:, cols], vs)
    assert torch.equal(X[0], X[M - 1])          # every replica holds the average after a round
