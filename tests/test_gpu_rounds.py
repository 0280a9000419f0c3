"""End-to-end rounds on the GPU against the CPU oracle, teacher-forced per round.

Every round starts from the GPU's own state (parameters, batch size) converted to fp64; the
oracle runs the same round on the same sample indices, and the two are compared afterwards:
parameters within 1e-6 relative (normwise per replica and max-abs against the largest parameter),
statistics within 1e-5, the next batch size bit-exact unless the deciding ratio lies within 1e-5
of an integer.  Free-running drift is not gated, only reported by the qualitative checks
(batch sizes never shrink, the loss goes down).
"""
import math

import numpy as np
import pytest
import torch

import oracle.abs_oracle as orc
import paper_2406_13936_b200 as pkg
from paper_2406_13936_b200 import inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = pkg.Context(0)
    yield c
    c.close()


def f64(t):
    return t.detach().cpu().numpy().astype(np.float64)


def params_close(gpu, ref, tol=1e-6):
    g = f64(gpu)
    for m in range(ref.shape[0]):
        assert np.linalg.norm(g[m] - ref[m]) <= tol * max(np.linalg.norm(ref[m]), 1e-30)
    assert np.abs(g - ref).max() <= tol * max(np.abs(ref).max(), 1e-30)


def near_integer(x, tol=1e-5):
    return abs(x - round(x)) <= tol * max(x, 1.0)


def test_logreg_per_sample_gradients(ctx):
    n, d, M, b = 500, 37, 3, 21
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    X = torch.randn((M, d), device="cuda", generator=torch.Generator("cuda").manual_seed(2)) * 0.3
    idx = inputs.batch_indices(3, (M, b + 5), n, device="cuda")
    G = torch.empty((M, b, d), device="cuda")
    ctx.abs_logreg_grads(A, y, idx, X, b, G)
    An, yn, Xn, In = f64(A), f64(y), f64(X), idx.cpu().numpy()
    for m in range(M):
        ref = orc.logreg_per_sample_grads(An[In[m, :b]], yn[In[m, :b]], Xn[m])
        got = f64(G[m])
        assert np.abs(got - ref).max() <= 2e-6 * np.abs(ref).max()


def test_gradients_of_well_fitted_samples_keep_their_relative_accuracy(ctx):
    """A sample the model fits has a residual far below 1: sigmoid(z) - 1 and softmax - 1 must not be
    formed by subtracting from a rounded probability.  Rows are compared one by one, each relative to
    its own norm."""
    # logistic: x along the direction that produced the labels, no flips, |z| of about 5 to 20 (beyond 35 the
    # oracle's own fp64 difference sigmoid(z) - 1 runs out of digits)
    n, d, M, b = 400, 64, 2, 50
    A, y = inputs.logreg_dataset(4, n, d, flip=0.0, device="cuda")
    An, yn = f64(A), f64(y)
    w = np.linalg.lstsq(An, 2.0 * yn - 1.0, rcond=None)[0]
    X = torch.tensor(np.stack([8.0 * w, 20.0 * w]), dtype=torch.float32, device="cuda")
    idx = inputs.batch_indices(5, (M, b), n, device="cuda")
    G = torch.empty((M, b, d), device="cuda")
    ctx.abs_logreg_grads(A, y, idx, X, b, G)
    Xn, In = f64(X), idx.cpu().numpy()
    tiny = 0
    for m in range(M):
        ref = orc.logreg_per_sample_grads(An[In[m]], yn[In[m]], Xn[m])
        got = f64(G[m])
        for i in range(b):
            scale = np.linalg.norm(ref[i])
            tiny += scale < 1e-3 * np.linalg.norm(An[In[m, i]])
            assert np.linalg.norm(got[i] - ref[i]) <= 5e-5 * scale + 1e-12 * np.linalg.norm(An[In[m, i]])
    assert tiny >= b                                  # the case is what it claims: many residuals below 1e-3
    # softmax: a small network whose last layer is scaled up, labels = the predicted class
    dims, M, b, n = (6, 5, 4, 3), 2, 16, 60
    inp, _, X = mlp_problem(8, n, dims, M)
    X = X * 1.0
    dW3 = dims[3] * dims[2]
    off3 = ctx.mlp_param_count(dims) - dW3 - dims[3]
    X[:, off3:off3 + dW3] *= 12.0     # (1 - p below 1e-9 would exhaust the oracle's own fp64 difference)
    layers = orc.mlp_unpack(f64(X[0]), dims)
    h = f64(inp)
    for l, (W, bias) in enumerate(layers):
        h = h @ W.T + bias
        if l < len(layers) - 1:
            h = np.maximum(h, 0.0)
    lab = torch.tensor(h.argmax(axis=1), dtype=torch.int32, device="cuda")
    X[1] = X[0]
    idx = inputs.batch_indices(9, (M, b), n, device="cuda")
    scratch = ctx.mlp_scratch(M, b, dims)
    d = ctx.mlp_param_count(dims)
    Gb = torch.empty((M, d), device="cuda")
    ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
    Gs = torch.zeros((b, (d + 3) // 4 * 4), device="cuda")
    ctx.abs_mlp_per_sample(dims, b, 0, scratch, Gs)
    rows = idx.cpu().numpy()[0, :b]
    ref = orc.mlp_per_sample_grads(f64(inp)[rows], lab.cpu().numpy()[rows], f64(X[0]), dims)
    got = f64(Gs[:, :d])
    small = 0
    for i in range(b):
        scale = np.linalg.norm(ref[i])
        small += scale < 1e-3
        assert np.linalg.norm(got[i] - ref[i]) <= 1e-3 * scale + 1e-9
    assert small >= 3


def logistic_loss(A, y, x):
    z = A @ x
    return float(np.mean(np.logaddexp(0.0, z) - y * z))


@pytest.mark.parametrize("rounds", [50])
def test_end_to_end_logistic_rounds(ctx, rounds):
    # d=256, n=65,536, M=4 workers, local SGD lr=0.1, H=8, norm test eta=0.5, b from 16, cap 1024
    n, d, M, H, lr, eta, b, b_max = 65536, 256, 4, 8, 0.1, 0.5, 16, 1024
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    X = torch.zeros((M, d), device="cuda")
    G = torch.empty((M, b_max, d), device="cuda")      # scratch, used as [M, b, d] with the current b
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    cfg = pkg.make_test_cfg("norm", b_max, eta=eta)
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()
    history, exact, total = [b], 0, 0
    loss0 = logistic_loss(An, yn, np.zeros(d))
    for k in range(rounds):
        X0 = f64(X)
        ctx.abs_logreg_round(A, y, idx[k], X, H, b, lr, cfg, G, Gb, stats, b_dev, T_out)
        torch.cuda.synchronize()
        # oracle: same round from the GPU's state
        def grads(m, h, x, k=k, b=b):
            rows = In[k, h, m, :b]
            return orc.logreg_per_sample_grads(An[rows], yn[rows], x)
        Xr, b_ref, T_ref, st_ref = orc.local_round(X0, grads, H, lr, b, b_max, "norm", eta=eta)
        params_close(X, Xr)
        recs = pkg.stats_to_dicts(stats)
        for m in range(M):
            for key in ("gbar_sq", "var_norm"):
                assert recs[m][key] == pytest.approx(st_ref[m][key], rel=1e-5)
            ratio = st_ref[m]["var_norm"] / (eta * eta * st_ref[m]["gbar_sq"])
            total += 1
            if near_integer(ratio):
                assert abs(T_out[m].item() - T_ref[m]) <= 1
            else:
                assert T_out[m].item() == T_ref[m]
                exact += 1
        b_new = int(b_dev.item())
        if T_out.tolist() == T_ref:
            assert b_new == b_ref
        assert b <= b_new <= b_max
        b = b_new
        history.append(b)
    assert exact >= 0.8 * total                     # most ratios are clear of a rounding boundary
    assert history[-1] > history[0]                 # the norm test asked for larger batches
    assert all(x <= y_ for x, y_ in zip(history, history[1:]))
    assert logistic_loss(An, yn, f64(X)[0]) < 0.8 * loss0
    assert torch.equal(X[0], X[M - 1])              # replicas agree after the averaging


# ------------------------------------------------------------------ rounds fused into one launch
def _ratios(st, kind, cfg):
    N = st["gbar_sq"]
    if kind == "norm":
        return [st["var_norm"] / (cfg["eta"] ** 2 * N)]
    return [st["var_ip"] / (cfg["theta"] ** 2 * N * N), st["var_orth"] / (cfg["nu"] ** 2 * N)]


@pytest.mark.parametrize("n,d,M,H,lr,kind,cfg,b,b_max,rounds", [
    (65536, 256, 4, 8, 0.1, "norm", dict(eta=0.5), 16, 1024, 50),          # the tiny end-to-end configuration
    (3000, 36, 3, 3, 0.2, "aug_ip", dict(theta=0.5, nu=0.5), 5, 300, 14),  # ragged: d/4 = 9 vectors, odd sizes
    (5000, 1024, 2, 2, 0.05, "norm", dict(eta=0.7), 2, 700, 8),            # widest rows, b from its minimum
    (4096, 128, 40, 1, 0.1, "norm", dict(eta=0.4), 3, 64, 6),              # many workers: few CTAs per worker
    (2000, 384, 2, 2, 0.05, "norm", dict(eta=0.6), 4, 200, 6),             # four 16-byte vectors per lane
])
def test_fused_logistic_rounds_teacher_forced(ctx, n, d, M, H, lr, kind, cfg, b, b_max, rounds):
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    X = torch.zeros((M, d), device="cuda")
    stats = ctx.new_stats(M)
    T_out = torch.zeros((1, M), dtype=torch.int64, device="cuda")
    b_hist = torch.zeros(2, dtype=torch.int64, device="cuda")
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    tcfg = pkg.make_test_cfg(kind, b_max, **cfg)
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()
    history, exact, total = [b], 0, 0
    loss0 = logistic_loss(An, yn, np.zeros(d))
    for k in range(rounds):
        X0 = f64(X)
        ctx.abs_logreg_rounds_fused(A, y, idx[k:k + 1], X, H, lr, tcfg, stats, b_dev, T_out=T_out, b_hist=b_hist)
        torch.cuda.synchronize()

        def grads(m, h, x, k=k, b=b):
            rows = In[k, h, m, :b]
            return orc.logreg_per_sample_grads(An[rows], yn[rows], x)
        Xr, b_ref, T_ref, st_ref = orc.local_round(X0, grads, H, lr, b, b_max, kind, **cfg)
        params_close(X, Xr)
        recs = pkg.stats_to_dicts(stats)
        for m in range(M):
            assert recs[m]["rows"] == b and recs[m]["status"] == 0
            for key in ("gbar_sq", "var_norm", "var_ip", "sum_sq"):
                assert recs[m][key] == pytest.approx(st_ref[m][key], rel=1e-5)
            assert abs(recs[m]["var_orth"] - st_ref[m]["var_orth"]) <= 1e-5 * st_ref[m]["var_norm"]
            total += 1
            if any(near_integer(x) for x in _ratios(st_ref[m], kind, cfg)):
                assert abs(T_out[0, m].item() - T_ref[m]) <= 1
            else:
                assert T_out[0, m].item() == T_ref[m]
                exact += 1
        b_new = int(b_dev.item())
        assert b_hist.tolist() == [b, b_new]
        if T_out[0].tolist() == T_ref:
            assert b_new == b_ref
        assert b <= b_new <= b_max
        b = b_new
        history.append(b)
        for m in range(1, M):
            assert torch.equal(X[0], X[m])            # replicas agree after the averaging
    assert exact >= 0.8 * total
    assert history[-1] > history[0]
    assert logistic_loss(An, yn, f64(X)[0]) < loss0


def test_fused_rounds_in_one_launch_equal_one_launch_per_round(ctx):
    n, d, M, H, lr, b0, b_max, rounds = 65536, 256, 4, 8, 0.1, 16, 1024, 12
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    tcfg = pkg.make_test_cfg("norm", b_max, eta=0.5)
    # one launch for all rounds: the batch size never leaves the device
    X1 = torch.zeros((M, d), device="cuda")
    stats1 = ctx.new_stats(rounds * M)
    T1 = torch.zeros((rounds, M), dtype=torch.int64, device="cuda")
    hist1 = torch.zeros(rounds + 1, dtype=torch.int64, device="cuda")
    b1 = torch.tensor([b0], dtype=torch.int64, device="cuda")
    ctx.abs_logreg_rounds_fused(A, y, idx, X1, H, lr, tcfg, stats1, b1, T_out=T1, b_hist=hist1)
    # one launch per round
    X2 = torch.zeros((M, d), device="cuda")
    stats2 = ctx.new_stats(rounds * M)
    T2 = torch.zeros((rounds, M), dtype=torch.int64, device="cuda")
    b2 = torch.tensor([b0], dtype=torch.int64, device="cuda")
    hist2 = [b0]
    for k in range(rounds):
        ctx.abs_logreg_rounds_fused(A, y, idx[k:k + 1], X2, H, lr, tcfg, stats2[k * M:(k + 1) * M], b2, T_out=T2[k:k + 1])
        hist2.append(int(b2.item()))
    torch.cuda.synchronize()
    assert hist1.tolist() == hist2 and int(b1.item()) == hist2[-1]
    assert hist2[-1] == b_max                                   # the run reaches the cap
    assert torch.equal(X1, X2) and torch.equal(T1, T2) and torch.equal(stats1, stats2)
    # and the unfused driver, which forms the per-sample gradient matrix, takes the same decisions
    X3 = torch.zeros((M, d), device="cuda")
    G = torch.empty((M, b_max, d), device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    stats3 = ctx.new_stats(M)
    b3 = torch.tensor([b0], dtype=torch.int64, device="cuda")
    b = b0
    for k in range(rounds):
        ctx.abs_logreg_round(A, y, idx[k], X3, H, b, lr, tcfg, G, Gb, stats3, b3)
        b = int(b3.item())
        assert abs(b - hist2[k + 1]) <= max(1, 2e-5 * b)
        if b != hist2[k + 1]:
            break                                               # a ratio on a rounding boundary forks the runs
    else:
        params_close(X3, f64(X1), tol=1e-5)


@pytest.mark.parametrize("M,d,b0,b_max", [(16, 64, 4, 64), (8, 256, 8, 128), (40, 128, 3, 48)])
def test_fused_rounds_with_one_step_per_round_and_many_workers(ctx, M, d, b0, b_max):
    """H = 1 leaves the least work between two rounds' exchanges through global memory (a fast
    worker could be a round ahead of a slow reader, which is why the exchange buffers alternate by
    round): many rounds in one launch must equal one launch per round bit for bit, repeatedly."""
    n, H, lr, rounds = 4096, 1, 0.1, 40
    A, y = inputs.logreg_dataset(5, n, d, device="cuda")
    idx = inputs.batch_indices(12, (rounds, H, M, b_max), n, device="cuda")
    tcfg = pkg.make_test_cfg("norm", b_max, eta=0.6)
    X2 = torch.zeros((M, d), device="cuda")
    stats2 = ctx.new_stats(rounds * M)
    b2 = torch.tensor([b0], dtype=torch.int64, device="cuda")
    for k in range(rounds):
        ctx.abs_logreg_rounds_fused(A, y, idx[k:k + 1], X2, H, lr, tcfg, stats2[k * M:(k + 1) * M], b2)
    torch.cuda.synchronize()
    for _ in range(5):
        X1 = torch.zeros((M, d), device="cuda")
        stats1 = ctx.new_stats(rounds * M)
        b1 = torch.tensor([b0], dtype=torch.int64, device="cuda")
        ctx.abs_logreg_rounds_fused(A, y, idx, X1, H, lr, tcfg, stats1, b1)
        torch.cuda.synchronize()
        assert torch.equal(X1, X2) and torch.equal(stats1, stats2) and int(b1.item()) == int(b2.item())


def test_fused_rounds_wait_that_runs_out_is_reported_and_the_context_stays_usable(ctx):
    """Failure detection without a fault: with the partial gradients not sent (test hook) every CTA's
    wait for its peers gives up after the shortened limit, the launch still reaches all its barriers
    and ends, the records carry ABS_STATUS_TIMEOUT (so T = 0 and the batch size stays), and the next
    ordinary call on the same context gives the same result as a context that never timed out."""
    n, d, M, H, lr, b0, b_max, rounds = 4096, 256, 4, 3, 0.1, 64, 512, 2
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    idx = inputs.batch_indices(11, (rounds, H, M, b_max), n, device="cuda")
    tcfg = pkg.make_test_cfg("norm", b_max, eta=0.5)

    def run():
        X = torch.zeros((M, d), device="cuda")
        stats = ctx.new_stats(rounds * M)
        b_dev = torch.tensor([b0], dtype=torch.int64, device="cuda")
        ctx.abs_logreg_rounds_fused(A, y, idx, X, H, lr, tcfg, stats, b_dev)
        torch.cuda.synchronize()
        return X, stats, int(b_dev.item())

    X_ok, stats_ok, b_ok = run()
    ctx.set_tuning("stats_timeout_cycles", 2_000_000)        # about a millisecond
    ctx.set_tuning("stats_fault_drop_loads", 1)
    try:
        _, flagged, b_flagged = run()
    finally:
        ctx.set_tuning("stats_fault_drop_loads", 0)
        ctx.set_tuning("stats_timeout_cycles", 0)
    assert all(r["status"] & pkg.binding.STATUS_TIMEOUT for r in pkg.stats_to_dicts(flagged))
    assert b_flagged == b0                                     # flagged records take no decision
    X_again, stats_again, b_again = run()
    assert b_again == b_ok and b_ok > b0
    assert torch.equal(X_again, X_ok) and torch.equal(stats_again, stats_ok)


def test_fused_rounds_refuse_shapes_they_do_not_cover(ctx):
    tcfg = pkg.make_test_cfg("norm", 64, eta=0.5)
    b_dev = torch.tensor([4], dtype=torch.int64, device="cuda")
    for n, d, M, stride in [(100, 1028, 2, 64), (100, 30, 2, 64), (100, 32, 65, 64), (100, 32, 2, 32)]:
        A = torch.zeros((n, d), device="cuda")
        y = torch.zeros(n, device="cuda")
        idx = torch.zeros((1, 1, M, stride), dtype=torch.int32, device="cuda")
        X = torch.zeros((M, d), device="cuda")
        with pytest.raises(pkg.AbsError):
            ctx.abs_logreg_rounds_fused(A, y, idx, X, 1, 0.1, tcfg, ctx.new_stats(M), b_dev)


# ------------------------------------------------------------------ MLP producer and rounds
def mlp_problem(seed, n, dims, M, device="cuda"):
    inp, lab = inputs.gaussian_mixture(seed, n, dim=dims[0], classes=dims[3], device=device)
    x0 = inputs.mlp_init(seed + 1, dims, device=device)
    X = x0.unsqueeze(0).repeat(M, 1).contiguous()
    return inp, lab, X


@pytest.mark.parametrize("dims,M,b", [((6, 5, 4, 3), 2, 4), ((20, 33, 17, 7), 3, 9), ((70, 130, 65, 10), 2, 67),
                                      ((784, 1024, 1024, 10), 1, 3),
                                      # large enough for the tensor-core products (rows, columns >= 96, K >= 64),
                                      # with ragged tiles, an odd parameter count (replica 1 is not 16-byte
                                      # aligned) and every operand layout
                                      ((200, 257, 191, 10), 3, 130), ((784, 1024, 1024, 10), 2, 150)])
def test_mlp_batch_and_per_sample_gradients(ctx, dims, M, b):
    n = 300
    inp, lab, X = mlp_problem(5, n, dims, M)
    X += 0.05 * torch.randn(X.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(9))  # distinct replicas, non-zero biases
    d = ctx.mlp_param_count(dims)
    assert d == orc.mlp_param_count(dims)
    idx = inputs.batch_indices(6, (M, b + 2), n, device="cuda")
    scratch = ctx.mlp_scratch(M, b, dims)
    Gb = torch.empty((M, d), device="cuda")
    ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
    stride = (d + 3) // 4 * 4
    G = torch.zeros((b, stride), device="cuda")
    In, inp_n, lab_n = idx.cpu().numpy(), f64(inp), lab.cpu().numpy()
    for m in range(M):
        ctx.abs_mlp_per_sample(dims, b, m, scratch, G)
        rows = In[m, :b]
        ref = orc.mlp_per_sample_grads(inp_n[rows], lab_n[rows], f64(X[m]), dims)
        got = f64(G[:, :d])
        assert np.abs(got - ref).max() <= 1e-5 * np.abs(ref).max()
        ref_b = orc.batch_mean(ref)
        assert np.abs(f64(Gb[m]) - ref_b).max() <= 1e-5 * np.abs(ref_b).max()
        assert torch.all(G[:, d:] == 0)          # the padding columns are left alone


@pytest.mark.parametrize("dims,M,b", [((200, 257, 191, 10), 3, 130), ((784, 1024, 1024, 10), 2, 300),
                                      ((300, 400, 500, 12), 2, 1000)])
def test_mlp_tensor_core_products_match_the_cuda_core_products(ctx, dims, M, b):
    """The same forward/backward pass twice: matrix products on the tensor cores (fp32 operands split
    into two TF32 parts, three products each, 32-value chunks added in fp32) and on the CUDA cores
    (fp32 products folded into fp64).  Batch gradients, activations and deltas agree to a few fp32
    ulps of the largest entry."""
    n = 4000
    inp, lab, X = mlp_problem(7, n, dims, M)
    X += 0.03 * torch.randn(X.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(3))
    d = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(8, (M, b), n, device="cuda")
    out = []
    for no_tc in (0, 1):
        scratch = ctx.mlp_scratch(M, b, dims)
        scratch.zero_()
        Gb = torch.zeros((M, d), device="cuda")
        ctx.set_tuning("mlp_no_tensor_cores", no_tc)
        try:
            ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
            st = ctx.new_stats(M)
            ctx.abs_mlp_fused_stats(dims, b, scratch, Gb, st)
        finally:
            ctx.set_tuning("mlp_no_tensor_cores", 0)
        torch.cuda.synchronize()
        # a worker's scratch starts with Xin, H1, H2, D3, D2, D1 (inputs, activations, deltas)
        acts = scratch.view(torch.float32).view(M, -1)[:, :b * (dims[0] + 2 * dims[1] + 2 * dims[2] + dims[3])].clone()
        out.append((Gb, acts, pkg.stats_to_dicts(st)))
    (g_tc, a_tc, s_tc), (g_cc, a_cc, s_cc) = out
    assert (g_tc - g_cc).abs().max().item() <= 5e-6 * g_cc.abs().max().item()
    assert (a_tc - a_cc).abs().max().item() <= 5e-6 * a_cc.abs().max().item()
    for t, c in zip(s_tc, s_cc):
        assert t["status"] == c["status"] == 0
        for key in ("gbar_sq", "var_norm", "var_ip", "sum_sq"):
            assert t[key] == pytest.approx(c[key], rel=2e-5)


def test_mlp_tensor_core_wait_that_runs_out_is_reported(ctx):
    """Failure detection without a fault: with the operand loaders switched off (test hook) the tensor-core
    products' waits give up after the shortened limit, tensor memory is freed, the launches end, and the
    statistics that follow carry ABS_STATUS_TIMEOUT; the next ordinary pass on the same context is
    correct again (the same records as a context that never timed out)."""
    dims, M, b, n = (200, 257, 191, 10), 2, 130, 2000
    inp, lab, X = mlp_problem(7, n, dims, M)
    d = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(8, (M, b), n, device="cuda")

    def run():
        scratch = ctx.mlp_scratch(M, b, dims)
        Gb = torch.zeros((M, d), device="cuda")
        ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
        st = ctx.new_stats(M)
        ctx.abs_mlp_fused_stats(dims, b, scratch, Gb, st)
        torch.cuda.synchronize()
        return pkg.stats_to_dicts(st)

    good = run()
    ctx.set_tuning("stats_timeout_cycles", 2_000_000)        # about a millisecond
    ctx.set_tuning("stats_fault_drop_loads", 1)
    try:
        flagged = run()
    finally:
        ctx.set_tuning("stats_fault_drop_loads", 0)
        ctx.set_tuning("stats_timeout_cycles", 0)
    assert all(r["status"] & pkg.binding.STATUS_TIMEOUT for r in flagged)
    assert all(r["status"] == 0 for r in good)
    assert run() == good


@pytest.mark.parametrize("dims,M,b", [((20, 33, 17, 7), 3, 9), ((70, 130, 65, 10), 2, 67),
                                      ((784, 1024, 1024, 10), 2, 40), ((784, 1024, 1024, 10), 1, 600)])
def test_mlp_fused_statistics_match_materialised_gradients(ctx, dims, M, b):
    """Same activations, two routes: the statistics from outer-product identities against
    abs_test_stats on the per-sample gradient rows written out."""
    n = 5000
    inp, lab, X = mlp_problem(5, n, dims, M)
    X += 0.02 * torch.randn(X.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(9))
    d = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(6, (M, b), n, device="cuda")
    scratch = ctx.mlp_scratch(M, b, dims)
    Gb = torch.empty((M, d), device="cuda")
    ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
    fused = ctx.new_stats(M)
    ctx.abs_mlp_fused_stats(dims, b, scratch, Gb, fused)
    stride = (d + 3) // 4 * 4
    G = torch.zeros((b, stride), device="cuda")
    rows = ctx.new_stats(M)
    for m in range(M):
        ctx.abs_mlp_per_sample(dims, b, m, scratch, G)
        ctx.abs_test_stats(G.unsqueeze(0)[:, :, :d], rows[m:m + 1])
    torch.cuda.synchronize()
    for f, r in zip(pkg.stats_to_dicts(fused), pkg.stats_to_dicts(rows)):
        assert f["rows"] == r["rows"] == b and f["status"] == r["status"] == 0
        for key in ("gbar_sq", "var_norm", "var_ip", "sum_sq"):
            assert f[key] == pytest.approx(r[key], rel=2e-5)
        assert abs(f["var_orth"] - r["var_orth"]) <= 2e-5 * r["var_norm"]


@pytest.mark.parametrize("b", [32, 600])
def test_mlp_fused_statistics_against_the_oracle_at_full_network_size(ctx, b):
    """784-1024-1024-10: the statistics formed from activations and deltas (no gradient matrix)
    against the oracle, two ways.  (i) Same inputs: the oracle's definitions applied to the very
    per-sample gradient rows the GPU can write out, at 2e-5 (the expansion sum_i ||g_i||^2 - b N and
    the fp32 layer products are what separates the two).  (ii) The whole pipeline: the oracle's own
    fp64 forward/backward per sample, at 2e-4 (fp32 against fp64 producers)."""
    dims, n = (784, 1024, 1024, 10), 8192
    inp, lab, X = mlp_problem(5, n, dims, 1)
    X += 0.02 * torch.randn(X.shape, device="cuda", generator=torch.Generator("cuda").manual_seed(9))
    d = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(6, (1, b), n, device="cuda")
    scratch = ctx.mlp_scratch(1, b, dims)
    Gb = torch.empty((1, d), device="cuda")
    ctx.abs_mlp_grads(inp, lab, dims, idx, X, b, Gb, scratch)
    fused = ctx.new_stats(1)
    ctx.abs_mlp_fused_stats(dims, b, scratch, Gb, fused)
    stride = (d + 3) // 4 * 4
    G = torch.zeros((b, stride), device="cuda")
    ctx.abs_mlp_per_sample(dims, b, 0, scratch, G)
    torch.cuda.synchronize()
    rec = pkg.stats_to_dicts(fused)[0]
    assert rec["rows"] == b and rec["status"] == 0
    same_inputs = orc.batch_test_stats(f64(G[:, :d]))
    rows = idx[0].cpu().numpy()
    pipeline = orc.batch_test_stats(orc.mlp_per_sample_grads(f64(inp)[rows], lab.cpu().numpy()[rows], f64(X[0]), dims))
    for ref, tol in ((same_inputs, 2e-5), (pipeline, 2e-4)):
        for key in ("gbar_sq", "var_norm", "var_ip", "sum_sq"):
            assert rec[key] == pytest.approx(ref[key], rel=tol)
        orth_decides = ref["var_orth"] * ref["gbar_sq"] >= ref["var_ip"]
        assert abs(rec["var_orth"] - ref["var_orth"]) <= tol * (ref["var_orth"] if orth_decides else ref["var_norm"])
    np.testing.assert_allclose(f64(Gb[0]), pipeline["gbar"], rtol=0, atol=1e-5 * np.abs(pipeline["gbar"]).max())


def run_mlp_rounds(ctx, dims, n, M, H, lr, b, b_max, rounds, check_rounds, theta=0.5, nu=0.5, seed=5, fused=False):
    """Runs `rounds` rounds on the GPU; the first `check_rounds` are compared with the oracle."""
    inp, lab, X = mlp_problem(seed, n, dims, M)
    d = ctx.mlp_param_count(dims)
    stride = (d + 3) // 4 * 4
    idx = inputs.batch_indices(seed + 7, (rounds, H, M, b_max), n, device="cuda")
    scratch = ctx.mlp_scratch(M, b_max, dims)
    G = None if fused else torch.empty((b_max, stride), device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    cfg = pkg.make_test_cfg("aug_ip", b_max, theta=theta, nu=nu)
    inp_n, lab_n = (f64(inp), lab.cpu().numpy()) if check_rounds else (None, None)
    history = [b]
    for k in range(rounds):
        X0 = f64(X) if k < check_rounds else None
        ctx.abs_mlp_round(inp, lab, dims, idx[k], X, H, b, lr, cfg, scratch, G, stride, Gb, stats, b_dev, T_out)
        torch.cuda.synchronize()
        recs = pkg.stats_to_dicts(stats)
        assert all(r["status"] == 0 and r["rows"] == b for r in recs)
        if k < check_rounds:
            In = idx[k].cpu().numpy()

            def grads(m, h, x, b=b, In=In):
                rows = In[h, m, :b]
                return orc.mlp_per_sample_grads(inp_n[rows], lab_n[rows], x, dims)
            Xr, b_ref, T_ref, st_ref = orc.local_round(X0, grads, H, lr, b, b_max, "aug_ip", theta=theta, nu=nu)
            params_close(X, Xr)
            for m in range(M):
                # the producers differ by fp32 rounding, so the statistics of the two pipelines agree
                # to a few 1e-6; parity on identical inputs is covered by test_gpu_stats
                for key in ("gbar_sq", "var_norm", "var_ip", "var_orth"):
                    assert recs[m][key] == pytest.approx(st_ref[m][key], rel=2e-4)
                N = st_ref[m]["gbar_sq"]
                ratios = [st_ref[m]["var_ip"] / (theta ** 2 * N * N), st_ref[m]["var_orth"] / (nu ** 2 * N)]
                if not any(near_integer(r, 1e-3) for r in ratios):
                    assert T_out[m].item() == T_ref[m]
            if T_out.tolist() == T_ref:
                assert int(b_dev.item()) == b_ref
        b_new = int(b_dev.item())
        assert b <= b_new <= b_max
        b = b_new
        history.append(b)
    return X, history, (inp, lab)


@pytest.mark.parametrize("fused", [False, True])
def test_mlp_rounds_small_network_teacher_forced(ctx, fused):
    X, history, _ = run_mlp_rounds(ctx, (64, 48, 32, 10), n=4096, M=8, H=4, lr=0.05, b=8, b_max=512, rounds=12,
                                   check_rounds=12, fused=fused)
    assert history[-1] > history[0]
    assert torch.equal(X[0], X[7])


@pytest.mark.parametrize("fused", [False, True])
def test_mlp_rounds_full_network_first_rounds(ctx, fused):
    # the 784-1024-1024-10 classifier with all eight workers, three teacher-forced rounds (the oracle
    # runs M H b backward passes of a 1.9 M-parameter network per round)
    run_mlp_rounds(ctx, (784, 1024, 1024, 10), n=8192, M=8, H=4, lr=0.01, b=32, b_max=4096, rounds=3, check_rounds=3,
                   fused=fused)


def mlp_loss(ctx, inp, lab, x, dims):
    """Mean cross-entropy on the first 4096 samples, evaluated with torch (test-side check only)."""
    a = inp[:4096]
    off = 0
    for l in range(3):
        nin, nout = dims[l], dims[l + 1]
        W = x[off:off + nin * nout].view(nout, nin)
        off += nin * nout
        bias = x[off:off + nout]
        off += nout
        a = a @ W.t() + bias
        if l < 2:
            a = torch.relu(a)
    return torch.nn.functional.cross_entropy(a, lab[:4096].long()).item()


@pytest.mark.parametrize("fused", [False, True])
def test_end_to_end_mlp_200_rounds(ctx, fused):
    # 784-1024-1024-10, n = 1,048,576, M=8, H=4, augmented inner-product test, b from 32, cap 4096
    dims = (784, 1024, 1024, 10)
    inp, lab, X0 = mlp_problem(5, 1_048_576, dims, 1)
    loss0 = mlp_loss(ctx, inp, lab, X0[0], dims)
    del inp, lab, X0
    X, history, (inp, lab) = run_mlp_rounds(ctx, dims, n=1_048_576, M=8, H=4, lr=0.01, b=32, b_max=4096, rounds=200,
                                            check_rounds=0, fused=fused)
    assert all(x <= y_ for x, y_ in zip(history, history[1:]))
    assert history[-1] > history[0]
    assert torch.equal(X[0], X[7])
    assert mlp_loss(ctx, inp, lab, X[0], dims) < 0.5 * loss0
