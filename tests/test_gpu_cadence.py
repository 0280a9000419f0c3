"""The cadence of the test and the outer loop's counters on the GPU against the CPU oracle.

Algorithm 1 runs the test after every local step and lets every worker keep its own batch size;
the practical rule takes the maximum over the workers; Algorithm 2 tests once per round.  Both count
the samples they process (B) and stop at B >= N.  Every round is teacher-forced: the oracle starts
from the GPU's parameters and sizes at the start of the round.  Inside a round the two sides are
compared step by step -- sizes and T bit-exactly (T may differ by one where the deciding ratio is
within 1e-5 of an integer; the rest of that round is then not compared), statistics at 1e-5,
parameters at 1e-6 after the averaging.
"""
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


def ratios_of(st, kind, cfg, eta=None):
    N = st["gbar_sq"]
    if kind == "norm":
        e = cfg["eta"] if eta is None else eta
        return [st["var_norm"] / (e ** 2 * N)]
    return [st["var_ip"] / (cfg["theta"] ** 2 * N * N), st["var_orth"] / (cfg["nu"] ** 2 * N)]


def compare_round(recs, T_gpu, used_gpu, ref, kind, cfg, etas, H, M, tol_stats=1e-5):
    """Step-by-step comparison of one round; returns True when every step of the round could be compared
    (no decision fell on a rounding boundary)."""
    _, _, b_used, T_ref, st_ref, _ = ref
    for h in range(H):
        assert used_gpu[h] == b_used[h]                      # the sizes this step ran with
        for m in range(M):
            rec, sr = recs[h * M + m], st_ref[h][m]
            assert rec["rows"] == b_used[h][m] and rec["status"] == 0
            for key in ("gbar_sq", "var_norm", "var_ip", "sum_sq"):
                assert rec[key] == pytest.approx(sr[key], rel=tol_stats)
            assert abs(rec["var_orth"] - sr["var_orth"]) <= tol_stats * sr["var_norm"]
        fork = False
        for m in range(M):
            eta = etas[m] if etas is not None else None
            if any(near_integer(x, max(tol_stats, 1e-5)) for x in ratios_of(st_ref[h][m], kind, cfg, eta)):
                assert abs(T_gpu[h][m] - T_ref[h][m]) <= 1
                fork = fork or T_gpu[h][m] != T_ref[h][m]
            else:
                assert T_gpu[h][m] == T_ref[h][m]
        if fork:
            return False
    return True


CADENCES = [
    # (per_worker, eta per worker)
    (True, None),
    (False, None),
    (True, [0.35, 0.5, 0.8, 0.6]),
]


LOGREG_TINY = (65536, 256, 4, 8, 0.1, "norm", dict(eta=0.5), 16, 1024, 12)          # the tiny end-to-end configuration
LOGREG_RAGGED = (3000, 36, 4, 3, 0.2, "aug_ip", dict(theta=0.5, nu=0.5), 5, 300, 8)  # ragged vectors, odd sizes
LOGREG_WIDE = (5000, 1024, 4, 2, 0.05, "norm", dict(eta=0.7), 2, 500, 6)             # widest rows, sizes from their minimum


@pytest.mark.parametrize("problem,per_worker,etas", [
    (LOGREG_TINY, True, None), (LOGREG_TINY, False, None), (LOGREG_TINY, True, [0.35, 0.5, 0.8, 0.6]),
    (LOGREG_RAGGED, True, None), (LOGREG_RAGGED, False, None),      # (per-worker constants belong to the norm test)
    (LOGREG_WIDE, True, None), (LOGREG_WIDE, False, None), (LOGREG_WIDE, True, [0.35, 0.5, 0.8, 0.6]),
])
def test_fused_rounds_with_the_test_after_every_step(ctx, problem, per_worker, etas):
    n, d, M, H, lr, kind, cfg, b0, b_max, rounds = problem
    A, y = inputs.logreg_dataset(1, n, d, device="cuda")
    idx = inputs.batch_indices(21, (rounds, H, M, b_max), n, device="cuda")
    X = torch.zeros((M, d), device="cuda")
    stats = ctx.new_stats(H * M)
    T_out = torch.zeros((1, H, M), dtype=torch.int64, device="cuda")
    b_hist = torch.zeros((1, H, M), dtype=torch.int64, device="cuda")
    sizes = [b0 + (m if per_worker else 0) for m in range(M)]        # unequal starts when the sizes are per worker
    b_dev = torch.tensor(sizes, dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    eta_dev = torch.tensor(etas, dtype=torch.float64, device="cuda") if etas is not None else None
    opts = pkg.make_round_opts(test_every_step=True, per_worker=per_worker, eta_m=eta_dev, ctl=ctl)
    tcfg = pkg.make_test_cfg(kind, b_max, **cfg)
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()
    whole, samples, grew_inside = 0, 0, False
    for k in range(rounds):
        X0 = f64(X)
        ctx.abs_logreg_rounds_fused_opts(A, y, idx[k:k + 1], X, H, lr, tcfg, opts, stats, b_dev, T_out=T_out,
                                         b_hist=b_hist)
        torch.cuda.synchronize()

        def grads(m, h, x, b, k=k):
            rows = In[k, h, m, :b]
            return orc.logreg_per_sample_grads(An[rows], yn[rows], x)
        ref = orc.local_round_per_step(X0, grads, H, lr, sizes, b_max, kind, shared=not per_worker,
                                       eta_per_worker=etas, **cfg)
        ok = compare_round(pkg.stats_to_dicts(stats), T_out[0].tolist(), b_hist[0].tolist(), ref, kind, cfg, etas, H, M)
        new_sizes = b_dev.tolist()
        used = b_hist[0].tolist()
        grew_inside = grew_inside or used[0] != used[-1]
        samples += sum(sum(row) for row in used)
        assert ctl.tolist()[:2] == [samples, k + 1]                   # B and k of Alg. 1
        if ok:
            whole += 1
            params_close(X, ref[0])
            assert new_sizes == ref[1] and sum(sum(row) for row in used) == ref[5]
        assert all(a <= c <= b_max for a, c in zip(sizes, new_sizes))
        if not per_worker:
            assert len(set(new_sizes)) == 1
        sizes = new_sizes
        for m in range(1, M):
            assert torch.equal(X[0], X[m])
    assert whole >= 0.75 * rounds
    assert grew_inside                                                # a size changed between two steps of one round


def test_fused_rounds_counters_and_stop_rule(ctx):
    """`while B < N` on the device: one launch is offered more rounds than the samples allow; it runs
    exactly the rounds a launch-per-round loop that reads B back would run, with the same results."""
    n, d, M, H, lr, b0, b_max, rounds = 8192, 128, 4, 4, 0.1, 8, 256, 30
    A, y = inputs.logreg_dataset(3, n, d, device="cuda")
    idx = inputs.batch_indices(23, (rounds, H, M, b_max), n, device="cuda")
    tcfg = pkg.make_test_cfg("norm", b_max, eta=0.5)
    for every, per_worker in ((False, False), (True, True), (True, False), (False, True)):
        per = H if every else 1
        # reference run: one launch per round, no stop, B accumulated on the host from the sizes used
        X2 = torch.zeros((M, d), device="cuda")
        st2 = ctx.new_stats(rounds * per * M)
        hist2 = torch.zeros((rounds, per, M), dtype=torch.int64, device="cuda")
        b2 = torch.full((M,), b0, dtype=torch.int64, device="cuda")
        opts2 = pkg.make_round_opts(test_every_step=every, per_worker=per_worker)
        B_after, X_after = [], []
        B = 0
        for k in range(rounds):
            ctx.abs_logreg_rounds_fused_opts(A, y, idx[k:k + 1], X2, H, lr, tcfg, opts2,
                                             st2[k * per * M:(k + 1) * per * M], b2, b_hist=hist2[k:k + 1])
            used = hist2[k].tolist()
            B += sum(sum(r) for r in used) * (1 if every else H)
            B_after.append(B)
            X_after.append(X2.clone())
        N = (B_after[9] + B_after[10]) // 2                            # stops after the 11th round
        K = next(i + 1 for i, v in enumerate(B_after) if v >= N)
        assert K == 11
        ctl = ctx.new_round_ctl(n_stop=N)
        opts1 = pkg.make_round_opts(test_every_step=every, per_worker=per_worker, ctl=ctl)
        X1 = torch.zeros((M, d), device="cuda")
        st1 = ctx.new_stats(rounds * per * M)
        hist1 = torch.full((rounds, per, M), -1, dtype=torch.int64, device="cuda")
        b1 = torch.full((M,), b0, dtype=torch.int64, device="cuda")
        ctx.abs_logreg_rounds_fused_opts(A, y, idx, X1, H, lr, tcfg, opts1, st1, b1, b_hist=hist1)
        torch.cuda.synchronize()
        assert ctl.tolist() == [B_after[K - 1], K, N, 0]
        assert torch.equal(hist1[:K], hist2[:K]) and bool((hist1[K:] == -1).all())   # later rounds never ran
        assert torch.equal(X1, X_after[K - 1])                         # x_{K,0}
        assert torch.equal(st1[:K * per * M], st2[:K * per * M])
        # a second launch on the same counters has nothing left to do
        ctx.abs_logreg_rounds_fused_opts(A, y, idx, X1, H, lr, tcfg, opts1, st1, b1, b_hist=hist1)
        torch.cuda.synchronize()
        assert ctl.tolist() == [B_after[K - 1], K, N, 0] and torch.equal(X1, X_after[K - 1])


def test_stop_rule_matches_the_oracle_loop(ctx):
    """Free-running comparison of the whole outer loop on a problem whose decisions are clear of
    rounding boundaries: the same K, B and size history as the oracle's `while B < N`."""
    n, d, M, H, lr, b0, b_max, rounds, N = 2048, 32, 2, 2, 0.2, 4, 64, 40, 1500
    A, y = inputs.logreg_dataset(4, n, d, device="cuda")
    idx = inputs.batch_indices(24, (rounds, H, M, b_max), n, device="cuda")
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()

    def grads(k, m, h, x, b):
        rows = In[k, h, m, :b]
        return orc.logreg_per_sample_grads(An[rows], yn[rows], x)
    for every in (False, True):
        x_hat, K, B, hist = orc.run_until_samples(np.zeros((M, d)), grads, H, lr, b0, b_max, "norm", N,
                                                  per_step=every, shared=True, eta=0.5)
        per = H if every else 1
        ctl = ctx.new_round_ctl(n_stop=N)
        opts = pkg.make_round_opts(test_every_step=every, per_worker=False, ctl=ctl)
        X = torch.zeros((M, d), device="cuda")
        hist_gpu = torch.full((rounds, per, M), -1, dtype=torch.int64, device="cuda")
        b_dev = torch.full((M,), b0, dtype=torch.int64, device="cuda")
        ctx.abs_logreg_rounds_fused_opts(A, y, idx, X, H, lr, pkg.make_test_cfg("norm", b_max, eta=0.5), opts,
                                         ctx.new_stats(rounds * per * M), b_dev, b_hist=hist_gpu)
        torch.cuda.synchronize()
        started = [row[0] for row in hist_gpu[:, 0].tolist() if row[0] >= 0]
        want = [h[0] if every else h for h in hist]
        if started != want:
            pytest.skip("a decision fell on a rounding boundary; the teacher-forced tests cover the rounds")
        assert ctl.tolist()[:2] == [B, K]
        assert np.abs(f64(X[0]) - x_hat).max() <= 1e-4 * np.abs(x_hat).max()      # K rounds of free-running fp32


@pytest.mark.parametrize("per_worker,etas", CADENCES)
def test_unfused_logistic_round_with_the_test_after_every_step(ctx, per_worker, etas):
    n, d, M, H, lr, b0, b_max, rounds = 4096, 64, 4, 3, 0.1, 6, 200, 6
    kind, cfg = "norm", dict(eta=0.5)
    A, y = inputs.logreg_dataset(2, n, d, device="cuda")
    idx = inputs.batch_indices(22, (rounds, H, M, b_max), n, device="cuda")
    X = torch.zeros((M, d), device="cuda")
    G = torch.empty((M * b_max, d), device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(H * M)
    T_out = torch.zeros((H, M), dtype=torch.int64, device="cuda")
    b_dev = torch.zeros(M, dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    eta_dev = torch.tensor(etas, dtype=torch.float64, device="cuda") if etas is not None else None
    opts = pkg.make_round_opts(test_every_step=True, per_worker=per_worker, eta_m=eta_dev, ctl=ctl)
    tcfg = pkg.make_test_cfg(kind, b_max, **cfg)
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()
    sizes = [b0 + (2 * m if per_worker else 0) for m in range(M)]
    samples, whole = 0, 0
    for k in range(rounds):
        X0 = f64(X)
        new_sizes = ctx.abs_logreg_round_per_step(A, y, idx[k], X, H, sizes, lr, tcfg, opts, G, Gb, stats, b_dev,
                                                  T_out=T_out)
        torch.cuda.synchronize()

        def grads(m, h, x, b, k=k):
            rows = In[k, h, m, :b]
            return orc.logreg_per_sample_grads(An[rows], yn[rows], x)
        ref = orc.local_round_per_step(X0, grads, H, lr, sizes, b_max, kind, shared=not per_worker,
                                       eta_per_worker=etas, **cfg)
        recs = pkg.stats_to_dicts(stats)
        used = [[recs[h * M + m]["rows"] for m in range(M)] for h in range(H)]
        ok = compare_round(recs, T_out.tolist(), used, ref, kind, cfg, etas, H, M)
        samples += sum(sum(r) for r in used)
        assert ctl.tolist()[:2] == [samples, k + 1]
        assert new_sizes == b_dev.tolist()
        if ok:
            whole += 1
            params_close(X, ref[0])
            assert new_sizes == ref[1]
        sizes = new_sizes
    assert whole >= rounds - 1


@pytest.mark.parametrize("per_worker", [True, False])
def test_mlp_round_with_the_test_after_every_step(ctx, per_worker):
    """The MLP problem: fp32 forward/backward on the GPU against the fp64 oracle, so the statistics of the
    two pipelines agree to a few 1e-6 only (2e-4 here, decisions exempt within 1e-3 of an integer)."""
    dims, n, M, H, lr, b0, b_max, rounds = (64, 48, 32, 10), 4096, 4, 3, 0.05, 8, 256, 5
    kind, cfg = "aug_ip", dict(theta=0.5, nu=0.5)
    inp, lab = inputs.gaussian_mixture(5, n, dim=dims[0], classes=dims[3], device="cuda")
    X = inputs.mlp_init(6, dims, device="cuda").unsqueeze(0).repeat(M, 1).contiguous()
    d = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(25, (rounds, H, M, b_max), n, device="cuda")
    scratch = ctx.mlp_scratch(M, b_max, dims)
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(H * M)
    T_out = torch.zeros((H, M), dtype=torch.int64, device="cuda")
    b_dev = torch.zeros(M, dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    opts = pkg.make_round_opts(test_every_step=True, per_worker=per_worker, ctl=ctl)
    tcfg = pkg.make_test_cfg(kind, b_max, **cfg)
    inp_n, lab_n, In = f64(inp), lab.cpu().numpy(), idx.cpu().numpy()
    sizes = [b0 + (3 * m if per_worker else 0) for m in range(M)]
    samples = 0
    for k in range(rounds):
        X0 = f64(X)
        new_sizes = ctx.abs_mlp_round_per_step(inp, lab, dims, idx[k], X, H, sizes, lr, tcfg, opts, scratch, Gb, stats,
                                               b_dev, T_out=T_out)
        torch.cuda.synchronize()

        def grads(m, h, x, b, k=k):
            rows = In[k, h, m, :b]
            return orc.mlp_per_sample_grads(inp_n[rows], lab_n[rows], x, dims)
        ref = orc.local_round_per_step(X0, grads, H, lr, sizes, b_max, kind, shared=not per_worker, **cfg)
        recs = pkg.stats_to_dicts(stats)
        used = [[recs[h * M + m]["rows"] for m in range(M)] for h in range(H)]
        _, b_ref, b_used, T_ref, st_ref, _ = ref
        same = True
        for h in range(H):
            if not same:
                break
            assert used[h] == b_used[h]
            for m in range(M):
                for key in ("gbar_sq", "var_norm", "var_ip", "var_orth"):
                    assert recs[h * M + m][key] == pytest.approx(st_ref[h][m][key], rel=2e-4)
                if any(near_integer(x, 1e-3) for x in ratios_of(st_ref[h][m], kind, cfg)):
                    same = same and T_out[h, m].item() == T_ref[h][m]
                else:
                    assert T_out[h, m].item() == T_ref[h][m]
        samples += sum(sum(r) for r in used)
        assert ctl.tolist()[:2] == [samples, k + 1]
        if same:
            params_close(X, ref[0])
            assert new_sizes == b_ref
        sizes = new_sizes


def test_per_round_drivers_count_samples(ctx):
    """Algorithm 2's counter in the enqueue-only drivers: B += H M b_k and k += 1 per round."""
    n, d, M, H, lr, b, b_max, rounds = 4096, 64, 3, 2, 0.1, 8, 128, 5
    A, y = inputs.logreg_dataset(2, n, d, device="cuda")
    idx = inputs.batch_indices(26, (rounds, H, M, b_max), n, device="cuda")
    X = torch.zeros((M, d), device="cuda")
    G = torch.empty((M, b_max, d), device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    tcfg = pkg.make_test_cfg("norm", b_max, eta=0.5)
    B = 0
    for k in range(rounds):
        ctx.abs_logreg_round(A, y, idx[k], X, H, b, lr, tcfg, G, Gb, stats, b_dev, ctl=ctl)
        B += orc.samples_of_round(H, M, b)
        b = int(b_dev.item())
        assert ctl.tolist()[:2] == [B, k + 1]
    dims = (20, 16, 12, 5)
    inp, lab = inputs.gaussian_mixture(5, 1000, dim=dims[0], classes=dims[3], device="cuda")
    Xm = inputs.mlp_init(6, dims, device="cuda").unsqueeze(0).repeat(M, 1).contiguous()
    dm = ctx.mlp_param_count(dims)
    idx = inputs.batch_indices(27, (2, H, M, 64), 1000, device="cuda")
    scratch = ctx.mlp_scratch(M, 64, dims)
    Gbm = torch.empty((M, dm), device="cuda")
    b_dev = torch.tensor([8], dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    b, B = 8, 0
    for k in range(2):
        ctx.abs_mlp_round(inp, lab, dims, idx[k], Xm, H, b, 0.05, pkg.make_test_cfg("aug_ip", 64, theta=0.5, nu=0.5),
                          scratch, None, 0, Gbm, stats, b_dev, ctl=ctl)
        B += H * M * b
        b = int(b_dev.item())
        assert ctl.tolist()[:2] == [B, k + 1]


# ------------------------------------------------------------------ Algorithm 2 as printed
@pytest.mark.parametrize("problem", ["logreg", "mlp"])
def test_rounds_with_the_test_on_the_workers_batch_gradients(ctx, problem):
    """Algorithm 2 ("actual implementation"): no per-sample statistics; after the averaging the M batch
    gradients of the round's last local step give Var = b/(M-1) sum ||g^m - gbar||^2 and
    T = ceil(Var / (M eta^2 ||gbar||^2)).  Teacher-forced rounds against the oracle; B counts H M b."""
    M, H, eta, rounds = 4, 3, 0.5, 6
    if problem == "logreg":
        n, d, lr, b, b_max = 8192, 64, 0.1, 8, 4096
        A, y = inputs.logreg_dataset(9, n, d, device="cuda")
        X = torch.zeros((M, d), device="cuda")
        G = torch.empty((M, b_max, d), device="cuda")
        An, yn = f64(A), f64(y)
        tol_stats = 1e-5
    else:
        dims, n, lr, b, b_max = (64, 48, 32, 10), 4096, 0.05, 8, 2048
        inp, lab = inputs.gaussian_mixture(5, n, dim=dims[0], classes=dims[3], device="cuda")
        X = inputs.mlp_init(6, dims, device="cuda").unsqueeze(0).repeat(M, 1).contiguous()
        d = ctx.mlp_param_count(dims)
        scratch = ctx.mlp_scratch(M, b_max, dims)
        inp_n, lab_n = f64(inp), lab.cpu().numpy()
        tol_stats = 2e-4                        # fp32 forward/backward against the fp64 oracle
    idx = inputs.batch_indices(28, (rounds, H, M, b_max), n, device="cuda")
    In = idx.cpu().numpy()
    Gb = torch.empty((M, d), device="cuda")
    stats = ctx.new_stats(M)
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    b_dev = torch.tensor([b], dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    cfg = pkg.make_test_cfg("norm_workers", b_max, eta=eta)
    B, grew = 0, False
    for k in range(rounds):
        X0 = f64(X)
        if problem == "logreg":
            ctx.abs_logreg_round(A, y, idx[k], X, H, b, lr, cfg, G, Gb, stats, b_dev, T_out=T_out, ctl=ctl)

            def batch_grads(m, h, x, k=k, b=b):
                rows = In[k, h, m, :b]
                return orc.batch_mean(orc.logreg_per_sample_grads(An[rows], yn[rows], x))
        else:
            ctx.abs_mlp_round(inp, lab, dims, idx[k], X, H, b, lr, cfg, scratch, None, 0, Gb, stats, b_dev,
                              T_out=T_out, ctl=ctl)

            def batch_grads(m, h, x, k=k, b=b):
                rows = In[k, h, m, :b]
                return orc.batch_mean(orc.mlp_per_sample_grads(inp_n[rows], lab_n[rows], x, dims))
        torch.cuda.synchronize()
        Xr, b_ref, T_ref, st_ref, samples = orc.local_round_worker_test(X0, batch_grads, H, lr, b, b_max, eta)
        params_close(X, Xr)
        rec = pkg.stats_to_dicts(stats)[0]
        assert rec["rows"] == M and rec["status"] == 0
        for key in ("gbar_sq", "var_norm"):
            assert rec[key] == pytest.approx(st_ref[key], rel=tol_stats)
        ratio = b / M * st_ref["var_norm"] / (eta * eta * st_ref["gbar_sq"])
        if near_integer(ratio, max(tol_stats, 1e-5)):
            assert abs(T_out[0].item() - T_ref) <= 1
        else:
            assert T_out[0].item() == T_ref
        B += samples
        assert ctl.tolist()[:2] == [B, k + 1]
        b_new = int(b_dev.item())
        if T_out[0].item() == T_ref:
            assert b_new == b_ref
        grew = grew or b_new > b
        assert b <= b_new <= b_max
        b = b_new
    assert grew


def test_fused_rounds_with_the_test_on_the_workers_batch_gradients(ctx):
    """Algorithm 2 inside the one-launch rounds: teacher-forced against the oracle round by round, and
    many rounds in one launch equal to a launch per round, with the counter on the device."""
    n, d, M, H, lr, eta, b0, b_max, rounds = 8192, 64, 4, 3, 0.1, 0.5, 8, 4096, 10
    A, y = inputs.logreg_dataset(9, n, d, device="cuda")
    idx = inputs.batch_indices(28, (rounds, H, M, b_max), n, device="cuda")
    An, yn, In = f64(A), f64(y), idx.cpu().numpy()
    cfg = pkg.make_test_cfg("norm_workers", b_max, eta=eta)
    X = torch.zeros((M, d), device="cuda")
    stats = ctx.new_stats(rounds * M)
    T_out = torch.zeros((rounds, M), dtype=torch.int64, device="cuda")
    b_dev = torch.tensor([b0], dtype=torch.int64, device="cuda")
    b, sizes = b0, [b0]
    for k in range(rounds):
        X0 = f64(X)
        ctx.abs_logreg_rounds_fused(A, y, idx[k:k + 1], X, H, lr, cfg, stats[k * M:(k + 1) * M], b_dev, T_out=T_out[k:k + 1])
        torch.cuda.synchronize()

        def batch_grads(m, h, x, k=k, b=b):
            rows = In[k, h, m, :b]
            return orc.batch_mean(orc.logreg_per_sample_grads(An[rows], yn[rows], x))
        Xr, b_ref, T_ref, st_ref, _ = orc.local_round_worker_test(X0, batch_grads, H, lr, b, b_max, eta)
        params_close(X, Xr)
        rec = pkg.stats_to_dicts(stats[k * M:k * M + 1])[0]
        assert rec["rows"] == M and rec["status"] == pkg.binding.STATUS_NORM_ONLY
        for key in ("gbar_sq", "var_norm"):
            assert rec[key] == pytest.approx(st_ref[key], rel=1e-5)
        ratio = b / M * st_ref["var_norm"] / (eta * eta * st_ref["gbar_sq"])
        if near_integer(ratio):
            assert abs(T_out[k, 0].item() - T_ref) <= 1
        else:
            assert T_out[k, 0].item() == T_ref
        b_new = int(b_dev.item())
        if T_out[k, 0].item() == T_ref:
            assert b_new == b_ref
        b = b_new
        sizes.append(b)
    assert sizes[-1] > sizes[0]
    # all rounds in one launch, with the counters: the same parameters and decisions, B = H M sum_k b_k
    X1 = torch.zeros((M, d), device="cuda")
    stats1 = ctx.new_stats(rounds * M)
    T1 = torch.zeros((rounds, M), dtype=torch.int64, device="cuda")
    b1 = torch.full((M,), b0, dtype=torch.int64, device="cuda")
    ctl = ctx.new_round_ctl()
    ctx.abs_logreg_rounds_fused_opts(A, y, idx, X1, H, lr, cfg, pkg.make_round_opts(ctl=ctl), stats1, b1, T_out=T1)
    torch.cuda.synchronize()
    assert torch.equal(X1, X) and torch.equal(T1[:, 0], T_out[:, 0]) and b1.tolist() == [sizes[-1]] * M
    assert ctl.tolist()[:2] == [H * M * sum(sizes[:-1]), rounds]
    # the unfused driver forms the same statistics with the library's statistics kernels
    X3 = torch.zeros((M, d), device="cuda")
    G = torch.empty((M, b_max, d), device="cuda")
    Gb = torch.empty((M, d), device="cuda")
    st3 = ctx.new_stats(M)
    b3 = torch.tensor([b0], dtype=torch.int64, device="cuda")
    b = b0
    for k in range(rounds):
        ctx.abs_logreg_round(A, y, idx[k], X3, H, b, lr, cfg, G, Gb, st3, b3)
        b = int(b3.item())
        if b != sizes[k + 1]:
            assert abs(b - sizes[k + 1]) <= 1          # a ratio on a rounding boundary forks the runs
            break
    else:
        params_close(X3, f64(X), tol=1e-5)


def test_workers_test_is_refused_where_it_does_not_apply(ctx):
    cfg = pkg.make_test_cfg("norm_workers", 64, eta=0.5)
    A, y = inputs.logreg_dataset(9, 256, 32, device="cuda")
    idx = inputs.batch_indices(28, (1, 1, 2, 64), 256, device="cuda")
    X = torch.zeros((2, 32), device="cuda")
    b_dev = torch.tensor([4, 4], dtype=torch.int64, device="cuda")
    for opts in (pkg.make_round_opts(test_every_step=True), pkg.make_round_opts(per_worker=True)):
        with pytest.raises(pkg.AbsError):                  # Algorithm 2 tests once per round, one size for all
            ctx.abs_logreg_rounds_fused_opts(A, y, idx, X, 1, 0.1, cfg, opts, ctx.new_stats(2), b_dev)
    X1 = torch.zeros((1, 32), device="cuda")              # one worker has no variance over workers
    with pytest.raises(pkg.AbsError):
        ctx.abs_logreg_round(A, y, idx[0, :, :1], X1, 1, 4, 0.1, cfg, torch.empty((1, 64, 32), device="cuda"),
                             torch.empty((1, 32), device="cuda"), ctx.new_stats(1), torch.tensor([4], dtype=torch.int64, device="cuda"))
    idx1 = inputs.batch_indices(28, (1, 1, 1, 64), 256, device="cuda")
    with pytest.raises(pkg.AbsError):
        ctx.abs_logreg_rounds_fused(A, y, idx1, X1, 1, 0.1, cfg, ctx.new_stats(1), b_dev[:1])
