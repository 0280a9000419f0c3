"""Pins for the CPU oracle: every check here compares the oracle with something
other than itself -- a hand-worked example, a library routine on a special
case, an exact-rational evaluation of a different (pairwise) formula on tiny
inputs, closed-form expectations, or an algebraic invariant."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle.abs_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- worked example
def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, rest = line.split(None, 1)
            out[key] = rest
    return out


def test_worked_example_matches_hand_computation():
    g = _read_golden("worked_example_b3_d2.txt")
    G = np.array([[float(v) for v in row.split()] for row in g["G"].split(";")])
    s = orc.batch_test_stats(G)
    np.testing.assert_allclose(s["gbar"], [float(v) for v in g["gbar"].split()], rtol=0, atol=1e-15)
    assert s["gbar_sq"] == pytest.approx(float(Fraction(g["gbar_sq"])), rel=1e-14)
    assert s["var_norm"] == pytest.approx(float(Fraction(g["var_norm"])), rel=1e-14)
    np.testing.assert_allclose(s["c"], [float(v) for v in g["c"].split()], rtol=1e-14)
    assert s["var_ip"] == pytest.approx(float(Fraction(g["var_ip"])), rel=1e-14)
    assert s["var_orth"] == pytest.approx(float(Fraction(g["var_orth"])), rel=1e-13)
    assert s["sum_sq"] == pytest.approx(float(Fraction(g["sum_sq"])), rel=1e-14)
    assert orc.batch_test_statistic(s, "norm", eta=0.5) == int(g["T_norm_eta_half"])
    assert orc.batch_test_statistic(s, "aug_ip", theta=0.5, nu=0.5) == int(g["T_augip_half_half"])


# ---------------------------------------------------------------- library special case
@pytest.mark.parametrize("b,d", [(2, 1), (3, 7), (16, 33), (64, 257)])
def test_var_norm_is_sum_of_unbiased_column_variances(b, d):
    rng = np.random.default_rng(10 + b)
    G = rng.standard_normal((b, d)) * 3.0 + rng.standard_normal(d)
    s = orc.batch_test_stats(G)
    assert s["var_norm"] == pytest.approx(np.var(G, axis=0, ddof=1).sum(), rel=1e-12)
    np.testing.assert_allclose(s["gbar"], G.mean(axis=0), rtol=1e-13, atol=1e-15)
    assert s["var_ip"] == pytest.approx(np.var(G @ G.mean(axis=0), ddof=1), rel=1e-10)


def test_b2_special_case():
    rng = np.random.default_rng(3)
    G = rng.standard_normal((2, 19))
    s = orc.batch_test_stats(G)
    assert s["var_norm"] == pytest.approx(0.5 * np.sum((G[0] - G[1]) ** 2), rel=1e-13)


# ---------------------------------------------------------------- exact rationals, pairwise forms
def _exact_pairwise(G):
    """U-statistic (pairwise-difference) forms in exact rational arithmetic:
    Var(h) = 1/(b(b-1)) sum_{i<k} ||h_i - h_k||^2, for h = g, <g, gbar>, o."""
    b, d = len(G), len(G[0])
    F = [[Fraction(v) for v in row] for row in G]
    pairs = list(itertools.combinations(range(b), 2))
    denom = Fraction(b * (b - 1))
    gram = [[sum(F[i][j] * F[k][j] for j in range(d)) for k in range(b)] for i in range(b)]
    var_norm = sum(sum((F[i][j] - F[k][j]) ** 2 for j in range(d)) for i, k in pairs) / denom
    c = [sum(gram[i]) / b for i in range(b)]               # <g_i, gbar> from the Gram matrix
    N = sum(sum(row) for row in gram) / (b * b)             # ||gbar||^2 = 1^T K 1 / b^2
    var_ip = sum((c[i] - c[k]) ** 2 for i, k in pairs) / denom
    if N == 0:
        var_orth = var_norm
    else:
        gbar = [sum(F[i][j] for i in range(b)) / b for j in range(d)]
        o = [[F[i][j] - c[i] / N * gbar[j] for j in range(d)] for i in range(b)]
        var_orth = sum(sum((o[i][j] - o[k][j]) ** 2 for j in range(d)) for i, k in pairs) / denom
    return var_norm, var_ip, var_orth, N, c


def _check_against_exact(G):
    s = orc.batch_test_stats(np.array(G, dtype=np.float64))
    var_norm, var_ip, var_orth, N, c = _exact_pairwise(G)
    scale = max(1.0, float(var_norm))
    assert abs(s["var_norm"] - float(var_norm)) <= 1e-12 * scale
    assert abs(s["gbar_sq"] - float(N)) <= 1e-12 * max(1.0, float(N))
    assert abs(s["var_ip"] - float(var_ip)) <= 1e-11 * max(1.0, float(var_ip))
    assert abs(s["var_orth"] - float(var_orth)) <= 1e-11 * scale
    np.testing.assert_allclose(s["c"], [float(v) for v in c], rtol=0, atol=1e-12 * max(1.0, float(N)))


@pytest.mark.parametrize("b,d", [(2, 1), (2, 2), (2, 3), (2, 4), (3, 1), (3, 2), (4, 1), (4, 2)])
def test_exhaustive_ternary_inputs(b, d):
    # every G in {-1, 0, 1}^(b x d) with b*d <= 8
    for flat in itertools.product((-1, 0, 1), repeat=b * d):
        G = [list(flat[i * d:(i + 1) * d]) for i in range(b)]
        _check_against_exact(G)


@pytest.mark.parametrize("seed", range(40))
def test_random_integer_inputs_exact(seed):
    rng = np.random.default_rng(seed)
    b = int(rng.integers(2, 5))
    d = int(rng.integers(1, 9))
    G = rng.integers(-9, 10, size=(b, d)).tolist()
    _check_against_exact(G)


# ---------------------------------------------------------------- invariants and special cases
def test_identical_rows_give_exact_zero():
    row = np.random.default_rng(0).standard_normal(100)
    s = orc.batch_test_stats(np.tile(row, (8, 1)))
    # the mean of 8 equal rows carries at most a few ulps of rounding
    assert s["var_norm"] <= 1e-28 * s["gbar_sq"] and s["var_ip"] <= 1e-28 * s["gbar_sq"] ** 2
    assert s["var_orth"] <= 1e-28 * s["gbar_sq"]
    two = orc.batch_test_stats(np.tile(row, (2, 1)))          # b = 2: the mean is exact
    assert two["var_norm"] == 0.0 and two["var_ip"] == 0.0
    assert orc.batch_test_statistic(s, "norm", eta=0.5) <= 1


@pytest.mark.parametrize("seed", range(6))
def test_norm_variance_splits_into_ip_and_orthogonal_parts(seed):
    rng = np.random.default_rng(100 + seed)
    b, d = int(rng.integers(2, 40)), int(rng.integers(2, 300))
    G = rng.standard_normal((b, d)) * rng.uniform(0.1, 10) + rng.standard_normal(d)
    s = orc.batch_test_stats(G)
    assert s["var_norm"] == pytest.approx(s["var_ip"] / s["gbar_sq"] + s["var_orth"], rel=1e-11)
    # exact means: mean_i c_i = N; sum_sq = (b-1) Var_norm + b N
    assert np.mean(s["c"]) == pytest.approx(s["gbar_sq"], rel=1e-12)
    assert s["sum_sq"] == pytest.approx((b - 1) * s["var_norm"] + b * s["gbar_sq"], rel=1e-12)


def test_parallel_rows_have_no_orthogonal_variance():
    rng = np.random.default_rng(5)
    u = rng.standard_normal(50)
    a = rng.uniform(0.5, 2.0, size=9)
    s = orc.batch_test_stats(np.outer(a, u))
    assert s["var_orth"] <= 1e-24 * s["var_norm"]
    # Var_ip / N = Var_norm, and Var_norm = Var(a) ||u||^2
    assert s["var_ip"] / s["gbar_sq"] == pytest.approx(s["var_norm"], rel=1e-12)
    assert s["var_norm"] == pytest.approx(np.var(a, ddof=1) * (u @ u), rel=1e-12)


def test_orthogonal_perturbations_have_no_inner_product_variance():
    rng = np.random.default_rng(6)
    d, b = 40, 7
    mean = rng.standard_normal(d)
    P = rng.standard_normal((b, d))
    P -= P.mean(axis=0)                       # perturbations sum to zero
    P -= np.outer(P @ mean, mean) / (mean @ mean)   # and are orthogonal to the mean
    s = orc.batch_test_stats(mean + P)
    assert s["var_ip"] <= 1e-24 * s["gbar_sq"] ** 2
    assert s["var_orth"] == pytest.approx(s["var_norm"], rel=1e-12)
    assert s["var_norm"] == pytest.approx(np.sum(P * P) / (b - 1), rel=1e-12)


def test_scale_permutation_and_duplication():
    rng = np.random.default_rng(8)
    b, d, k = 6, 31, 3
    G = rng.standard_normal((b, d)) + 0.3
    s = orc.batch_test_stats(G)
    s7 = orc.batch_test_stats(7.0 * G)
    for kind, cfg in (("norm", dict(eta=0.5)), ("aug_ip", dict(theta=0.5, nu=0.5))):
        assert orc.batch_test_statistic(s, kind, **cfg) == orc.batch_test_statistic(s7, kind, **cfg)
    assert s7["var_norm"] == pytest.approx(49.0 * s["var_norm"], rel=1e-13)
    assert s7["var_ip"] == pytest.approx(7.0 ** 4 * s["var_ip"], rel=1e-13)
    sp = orc.batch_test_stats(G[rng.permutation(b)])
    for key in ("gbar_sq", "var_norm", "var_ip", "var_orth"):
        assert sp[key] == pytest.approx(s[key], rel=1e-12)
    sd = orc.batch_test_stats(np.repeat(G, k, axis=0))
    f = k * (b - 1) / (k * b - 1)
    assert sd["gbar_sq"] == pytest.approx(s["gbar_sq"], rel=1e-12)
    for key in ("var_norm", "var_ip", "var_orth"):
        assert sd[key] == pytest.approx(f * s[key], rel=1e-11)


def test_zero_mean_and_all_zero_inputs():
    G = np.array([[1.0, -2.0], [-1.0, 2.0]])
    s = orc.batch_test_stats(G)
    assert s["status"] & orc.STATUS_ZERO_MEAN
    assert s["var_orth"] == s["var_norm"] == 10.0
    b_next, T = orc.next_batch([s], b_cur=2, b_max=64, kind="norm", eta=0.5)
    assert b_next == 64 and T == [orc.T_SATURATE]
    z = orc.batch_test_stats(np.zeros((3, 4)))
    b_next, T = orc.next_batch([z], b_cur=3, b_max=64, kind="aug_ip", theta=0.5, nu=0.5)
    assert b_next == 3 and T == [0]


def test_non_finite_input_is_flagged_and_gives_no_decision():
    G = np.ones((3, 4))
    G[1, 2] = np.inf
    with np.errstate(invalid="ignore"):
        s = orc.batch_test_stats(G)
    assert s["status"] & orc.STATUS_NONFINITE
    assert orc.next_batch([s], 3, 100, "norm", eta=0.5) == (3, [0])


# ---------------------------------------------------------------- isotropic Gaussian closed forms
def test_isotropic_gaussian_expectations():
    # g_i = mu + sigma z_i: (b-1) Var_norm / sigma^2 ~ chi2_{(b-1)d}; E N = |mu|^2 + sigma^2 d / b;
    # given gbar, (b-1) Var_ip / (sigma^2 N) ~ chi2_{b-1}; E Var_orth = sigma^2 (d - 1).
    rng = np.random.default_rng(2024)
    b, d, sigma, reps = 8, 64, 1.7, 400
    mu = rng.standard_normal(d) / math.sqrt(d)
    acc = np.zeros(4)
    for _ in range(reps):
        s = orc.batch_test_stats(mu + sigma * rng.standard_normal((b, d)))
        acc += [s["var_norm"], s["gbar_sq"], s["var_ip"] / s["gbar_sq"], s["var_orth"]]
    acc /= reps
    sd_mean = lambda rel_sd: 5.0 * rel_sd / math.sqrt(reps)
    assert acc[0] == pytest.approx(sigma ** 2 * d, rel=sd_mean(math.sqrt(2.0 / ((b - 1) * d))))
    assert acc[1] == pytest.approx(mu @ mu + sigma ** 2 * d / b, rel=sd_mean(0.3))
    assert acc[2] == pytest.approx(sigma ** 2, rel=sd_mean(math.sqrt(2.0 / (b - 1))))
    assert acc[3] == pytest.approx(sigma ** 2 * (d - 1), rel=sd_mean(math.sqrt(2.0 / ((b - 1) * (d - 1)))))


def test_noise_dominated_norm_test_asks_for_about_b_over_eta_sq():
    rng = np.random.default_rng(77)
    b, d, eta = 64, 20000, 0.5
    G = rng.standard_normal(d) / math.sqrt(d) + 10.0 * rng.standard_normal((b, d))
    T = orc.batch_test_statistic(orc.batch_test_stats(G), "norm", eta=eta)
    assert T == pytest.approx(b / eta ** 2, rel=0.05)


# ---------------------------------------------------------------- next-batch integer logic
def _fake(var_norm=0.0, var_ip=0.0, var_orth=0.0, N=1.0, status=0):
    return dict(var_norm=var_norm, var_ip=var_ip, var_orth=var_orth, gbar_sq=N, status=status)


@pytest.mark.parametrize("ratio,T", [(0.0, 0), (0.2, 1), (1.0, 1), (1.0000001, 2), (16.0, 16), (16.5, 17)])
def test_ceiling_and_growth_rule(ratio, T):
    s = _fake(var_norm=ratio * 0.25, N=1.0)        # eta = 1/2 -> ratio = var / 0.25
    assert orc.batch_test_statistic(s, "norm", eta=0.5) == T
    for b in (1, 2, 16, 17, 40):
        b_next, _ = orc.next_batch([s], b, 10 ** 6, "norm", eta=0.5)
        # "increase only if the test is violated" == max{T, b}: (1/b) Var <= eta^2 N  <=>  T <= b
        violated = ratio / b > 1.0
        assert b_next == (T if violated else b)
        assert b_next >= b


def test_max_over_workers_cap_and_scaling_factors():
    stats = [_fake(var_norm=0.25 * r) for r in (3.2, 90.5, 17.0)]
    assert orc.next_batch(stats, 8, 1024, "norm", eta=0.5) == (91, [4, 91, 17])
    assert orc.next_batch(stats, 8, 64, "norm", eta=0.5) == (64, [4, 91, 17])
    assert orc.next_batch(stats, 200, 1024, "norm", eta=0.5)[0] == 200
    # rows that are means of s samples, extra divisor M (Eq. test_stat_actual / Alg. 2)
    assert orc.batch_test_statistic(stats[1], "norm", eta=0.5, row_weight=32, divisor=4) == math.ceil(90.5 * 8)
    s = _fake(var_ip=0.25 * 4 * 7.3, var_orth=0.25 * 2 * 3.1, N=2.0)
    assert orc.batch_test_statistic(s, "aug_ip", theta=0.5, nu=0.5) == 8
    s = _fake(var_ip=0.25 * 4 * 1.3, var_orth=0.25 * 2 * 3.1, N=2.0)
    assert orc.batch_test_statistic(s, "aug_ip", theta=0.5, nu=0.5) == 4
    assert orc.batch_test_statistic(_fake(var_norm=1e300, N=1e-300), "norm", eta=0.5) == orc.T_SATURATE


def test_worker_gradient_estimator_matches_per_sample_variance_in_expectation():
    # Section 4.3: Var over workers of batch gradients, times b_local, estimates the per-sample variance.
    rng = np.random.default_rng(31)
    M, b_local, d, sigma, reps = 4, 16, 32, 2.0, 300
    est = 0.0
    for _ in range(reps):
        samples = 0.5 + sigma * rng.standard_normal((M, b_local, d))
        est += b_local * orc.batch_test_stats(samples.mean(axis=1))["var_norm"]
    assert est / reps == pytest.approx(sigma ** 2 * d, rel=0.05)


# ---------------------------------------------------------------- local updates
def test_sgd_and_average_closed_forms():
    X = np.array([[1.0, 2.0], [3.0, -4.0]])
    g = np.array([[0.5, 0.25], [-1.0, 2.0]])
    Y = X
    for _ in range(4):
        Y = orc.sgd_step(Y, g, 0.125)
    np.testing.assert_array_equal(Y, X - 0.5 * g)          # exactly representable
    A = orc.replica_average(Y)
    np.testing.assert_array_equal(A[0], A[1])
    np.testing.assert_allclose(A.sum(axis=0), Y.sum(axis=0), rtol=1e-15)
    np.testing.assert_array_equal(orc.replica_average(A), A)


def test_sgd_matches_torch_optimiser():
    rng = np.random.default_rng(1)
    x0 = rng.standard_normal((3, 17))
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=0.1)
    X = x0
    for t in range(5):
        g = rng.standard_normal(x0.shape)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        X = orc.sgd_step(X, g, 0.1)
    np.testing.assert_allclose(X, p.detach().numpy(), rtol=1e-14, atol=1e-15)


def test_shb_matches_torch_momentum_sgd():
    rng = np.random.default_rng(2)
    x0 = rng.standard_normal((2, 23))
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=0.05, momentum=0.9, weight_decay=1e-4)
    X, U = x0, np.zeros_like(x0)
    for t in range(6):
        g = rng.standard_normal(x0.shape)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        X, U = orc.shb_step(X, U, g, 0.05, 0.9, 1e-4)
    np.testing.assert_allclose(X, p.detach().numpy(), rtol=1e-13, atol=1e-15)


def test_adamw_matches_torch_optimiser():
    rng = np.random.default_rng(3)
    x0 = rng.standard_normal((2, 29)) * 0.02
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    hp = dict(lr=3e-4, betas=(0.9, 0.95), eps=1e-8, weight_decay=0.1)
    opt = torch.optim.AdamW([p], **hp)
    X, m, v = x0, np.zeros_like(x0), np.zeros_like(x0)
    for t in range(1, 21):
        g = rng.standard_normal(x0.shape) * 0.01
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        X, m, v = orc.adamw_step(X, m, v, g, 3e-4, 0.9, 0.95, 1e-8, 0.1, t)
    np.testing.assert_allclose(X, p.detach().numpy(), rtol=1e-12, atol=1e-16)


def test_adamw_closed_forms():
    x0 = np.array([[0.5, -0.25, 2.0]])
    g = np.array([[0.01, -0.03, 0.002]])
    lr, wd, eps = 1e-2, 0.1, 1e-8
    X, m, v = orc.adamw_step(x0, 0 * x0, 0 * x0, g, lr, 0.9, 0.95, eps, wd, 1)
    np.testing.assert_allclose(X, x0 * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-13)
    # constant gradient: bias-corrected moments stay at g and g^2
    X, m, v = x0, 0 * x0, 0 * x0
    for t in range(1, 8):
        Xp = X
        X, m, v = orc.adamw_step(X, m, v, g, lr, 0.9, 0.95, eps, wd, t)
        np.testing.assert_allclose(m / (1 - 0.9 ** t), g, rtol=1e-12)
        np.testing.assert_allclose(v / (1 - 0.95 ** t), g * g, rtol=1e-12)
        np.testing.assert_allclose(X, Xp * (1 - lr * wd) - lr * g / (np.abs(g) + eps), rtol=1e-11)


# ---------------------------------------------------------------- producers vs autograd
def test_logreg_per_sample_gradients_match_autograd():
    rng = np.random.default_rng(4)
    b, d = 5, 12
    A = rng.standard_normal((b, d))
    y = (rng.uniform(size=b) < 0.5).astype(np.float64)
    x = rng.standard_normal(d)
    G = orc.logreg_per_sample_grads(A, y, x)
    xt = torch.tensor(x, requires_grad=True)
    for i in range(b):
        loss = torch.nn.functional.binary_cross_entropy_with_logits(
            torch.tensor(A[i]) @ xt, torch.tensor(y[i]))
        (gi,) = torch.autograd.grad(loss, xt)
        np.testing.assert_allclose(G[i], gi.numpy(), rtol=1e-11, atol=1e-14)


def test_mlp_per_sample_gradients_match_autograd():
    rng = np.random.default_rng(5)
    dims = (6, 5, 4, 3)
    b = 4
    x = rng.standard_normal(orc.mlp_param_count(dims)) * 0.5
    inp = rng.standard_normal((b, dims[0]))
    lab = rng.integers(0, dims[-1], size=b)
    G = orc.mlp_per_sample_grads(inp, lab, x, dims)
    xt = torch.tensor(x, requires_grad=True)
    for i in range(b):
        off, a = 0, torch.tensor(inp[i])
        for l in range(3):
            nin, nout = dims[l], dims[l + 1]
            W = xt[off:off + nin * nout].reshape(nout, nin)
            off += nin * nout
            bias = xt[off:off + nout]
            off += nout
            a = W @ a + bias
            if l < 2:
                a = torch.relu(a)
        loss = torch.nn.functional.cross_entropy(a.unsqueeze(0), torch.tensor([int(lab[i])]))
        (gi,) = torch.autograd.grad(loss, xt)
        np.testing.assert_allclose(G[i], gi.numpy(), rtol=1e-10, atol=1e-13)


def test_bf16_widening_is_exact():
    t = torch.randn(1000, generator=torch.Generator().manual_seed(0)).to(torch.bfloat16)
    bits = t.view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(orc.bf16_bits_to_f64(bits), t.to(torch.float64).numpy())


def test_round_structure_on_a_quadratic():
    # f(x; xi) = 0.5 ||x - xi||^2: per-sample gradient x - xi; check one round by hand.
    rng = np.random.default_rng(9)
    M, H, b, d, lr = 2, 3, 4, 5, 0.1
    xi = rng.standard_normal((M, H, b, d))
    X0 = np.tile(rng.standard_normal(d), (M, 1))
    X, b_next, T, stats = orc.local_round(
        X0, lambda m, h, x: x - xi[m, h], H, lr, b, 1000, "norm", eta=0.5)
    Y = X0.copy()
    for h in range(H):
        for m in range(M):
            if h == H - 1:
                last = Y[m] - xi[m, h]
                assert stats[m]["var_norm"] == pytest.approx(np.var(last, axis=0, ddof=1).sum(), rel=1e-12)
            Y[m] = Y[m] - lr * (Y[m] - xi[m, h].mean(axis=0))
    np.testing.assert_allclose(X, np.tile(Y.mean(axis=0), (M, 1)), rtol=1e-13)
    assert b_next == max([b] + T)


# ---------------------------------------------------------------- per-worker sizes, merged sub-batches
def test_per_worker_batch_sizes():
    stats = [_fake(var_norm=0.25 * r) for r in (3.2, 90.5, 17.0)]
    b, T = orc.next_batch_local(stats, [8, 8, 40], 64, "norm", eta=0.5)
    assert T == [4, 91, 17] and b == [8, 64, 40]
    # a worker with a looser constant asks for less: eta_m = 1 quarters the ratio of eta = 1/2
    b, T = orc.next_batch_local(stats, [2, 2, 2], 1000, "norm", eta_per_worker=[0.5, 1.0, 0.25])
    assert T == [4, math.ceil(90.5 / 4), 68] and b == T


@pytest.mark.parametrize("n_a,n_b", [(2, 2), (5, 3), (16, 1), (1, 7)])
def test_merged_sub_batches_equal_the_whole_batch(n_a, n_b):
    rng = np.random.default_rng(n_a * 10 + n_b)
    G = rng.standard_normal((n_a + n_b, 33)) * 2.0 + 0.7
    whole = orc.batch_test_stats(G) if n_a + n_b >= 2 else None
    def part(rows):
        if rows.shape[0] >= 2:
            s = orc.batch_test_stats(rows)
            return s["gbar"], s["var_norm"]
        return rows[0], 0.0                       # a single row: no spread
    ma, va = part(G[:n_a])
    mb, vb = part(G[n_a:])
    mean, n, var, N = orc.merge_norm_stats(ma, n_a, va, mb, n_b, vb)
    assert n == n_a + n_b
    np.testing.assert_allclose(mean, whole["gbar"], rtol=1e-13, atol=1e-15)
    assert var == pytest.approx(whole["var_norm"], rel=1e-12)
    assert N == pytest.approx(whole["gbar_sq"], rel=1e-12)


# ---------------------------------------------------------------- Algorithm 1: the test after every local step
# f(x; xi) = 0.5 (x - xi)^2 in one dimension: per-sample gradient x - xi, so the batch variance is the
# sample variance of the xi's and the batch gradient is x - mean(xi).  All numbers below are worked by hand.
_XI = {(0, 0): [0, 4, 9], (0, 1): [1, 5, 3], (1, 0): [4, 4, 7], (1, 1): [2, 3, 8]}


def _toy_grads(m, h, x, b):
    return x[None, :] - np.array(_XI[(m, h)][:b], dtype=np.float64)[:, None]


def test_per_step_round_by_hand_per_worker():
    # worker 1: step 0, b=2, xi={0,4}: Var=8, gbar=3-2=1, T=ceil(8/(1/4))=32 -> b=min(3,32)=3, x=2.5
    #           step 1, b=3, xi={1,5,3}: Var=4, gbar=-1/2, T=ceil(4/(1/16))=64, x=2.75
    # worker 2: step 0, b=2, xi={4,4}: Var=0, gbar=-1, T=0 -> b=2, x=3.5
    #           step 1, b=2, xi={2,3}: Var=1/2, gbar=1, T=ceil((1/2)/(1/4))=2, x=3
    X, b, used, T, stats, samples = orc.local_round_per_step(
        np.array([[3.0], [3.0]]), _toy_grads, 2, 0.5, [2, 2], 3, "norm", eta=0.5)
    assert used == [[2, 2], [3, 2]] and T == [[32, 0], [64, 2]] and b == [3, 2]
    assert samples == 2 + 3 + 2 + 2
    np.testing.assert_allclose(X, [[2.875], [2.875]], rtol=1e-15)
    assert stats[1][0]["var_norm"] == pytest.approx(4.0, rel=1e-15)
    assert stats[1][0]["gbar_sq"] == pytest.approx(0.25, rel=1e-15)


def test_per_step_round_by_hand_shared_size():
    # as above, but after step 0 both workers continue with max(3, 2) = 3:
    # worker 2, step 1, b=3, xi={2,3,8}: mean 13/3, Var=31/3, gbar=3.5-13/3=-5/6, N=25/36,
    #           T=ceil((31/3)/((1/4)(25/36)))=ceil(59.52)=60, x=3.5+5/12
    X, b, used, T, _, samples = orc.local_round_per_step(
        np.array([[3.0], [3.0]]), _toy_grads, 2, 0.5, [2, 2], 3, "norm", shared=True, eta=0.5)
    assert used == [[2, 2], [3, 3]] and T == [[32, 0], [64, 60]] and b == [3, 3]
    assert samples == 10
    np.testing.assert_allclose(X, [[(2.75 + 3.5 + 5.0 / 12.0) / 2.0]] * 2, rtol=1e-15)


def test_per_step_round_with_per_worker_constants():
    # eta_1 = 1 quarters worker 1's ratios (8/1 = 8 -> b=3; 4/(1/4) = 16), eta_2 = 1/4 quadruples worker 2's
    # (step 1: (1/2)/((1/16) 1) = 8 -> b=min(3,8)=3)
    _, b, used, T, _, _ = orc.local_round_per_step(
        np.array([[3.0], [3.0]]), _toy_grads, 2, 0.5, [2, 2], 3, "norm", eta_per_worker=[1.0, 0.25])
    assert T == [[8, 0], [16, 8]] and used == [[2, 2], [3, 2]] and b == [3, 3]


def test_sample_counter_and_stop_rule():
    # identical samples xi = c: zero variance, T = 0, the batch size never moves; each step contracts
    # x - c by (1 - lr); Alg. 2 counts H M b samples per round and stops at the first K with B >= N
    c, x0, lr, H, M, b = 2.0, 10.0, 0.25, 2, 2, 3
    grads = lambda k, m, h, x, bb: np.tile(x - c, (bb, 1))
    x_hat, K, B, hist = orc.run_until_samples(np.full((M, 1), x0), grads, H, lr, b, 64, "norm", 50, eta=0.5)
    assert (K, B) == (5, 60) and hist == [3] * 5          # 12 samples per round: 48 < 50 <= 60
    assert x_hat[0] == pytest.approx(c + (x0 - c) * (1 - lr) ** (H * K), rel=1e-14)
    assert orc.samples_of_round(H, M, b) == 12
    # Alg. 1 counts the sizes actually used: the hand-worked round above uses 9 samples
    grads1 = lambda k, m, h, x, bb: _toy_grads(m, h, x, bb)
    for N, K_exp in ((9, 1), (10, 2)):
        _, K, B, hist = orc.run_until_samples(np.array([[3.0], [3.0]]), grads1, 2, 0.5, 2, 3, "norm", N,
                                              per_step=True, shared=False, eta=0.5)
        assert K == K_exp and hist[0] == [2, 2] and (B == 9 if K == 1 else B > 9)
    assert hist[1] == [3, 2]                               # the second round starts from the sizes the first ended with


def test_worker_gradient_round_by_hand():
    # Alg. 2 on f(x; xi) = 0.5 (x - xi)^2 with two workers, one dimension, H = 2, lr = 1/2, b = 4, eta = 1/2.
    # Batch gradients are x - (mean of the worker's batch), here given directly as x - c[m][h]:
    #   worker 1: c = 1 then 2:  x: 3 -> 3 - (3-1)/2 = 2 -> g = 2 - 2 = 0,  x stays 2
    #   worker 2: c = 5 then 6:  x: 3 -> 3 - (3-5)/2 = 4 -> g = 4 - 6 = -2, x = 4 + 1 = 5
    # average (2 + 5) / 2 = 3.5; gbar = -1, ||gbar||^2 = 1; 1/(M-1) sum (g - gbar)^2 = 1 + 1 = 2;
    # Var = b * 2 = 8; T = ceil(8 / (2 * (1/4) * 1)) = 16; B += H M b = 16.
    c = [[1.0, 2.0], [5.0, 6.0]]
    X, b_next, T, stats, samples = orc.local_round_worker_test(
        np.array([[3.0], [3.0]]), lambda m, h, x: x - c[m][h], 2, 0.5, 4, 1000, 0.5)
    np.testing.assert_allclose(X, [[3.5], [3.5]], rtol=1e-15)
    assert stats["gbar_sq"] == pytest.approx(1.0, rel=1e-15) and stats["var_norm"] == pytest.approx(2.0, rel=1e-15)
    assert (T, b_next, samples) == (16, 16, 16)
    # capped, and never smaller than the current size
    assert orc.local_round_worker_test(np.array([[3.0], [3.0]]), lambda m, h, x: x - c[m][h], 2, 0.5, 4, 10, 0.5)[1] == 10
    # gradients that nearly agree (g^1 = 1, g^2 = 1.2): ratio b (g1-g2)^2 / (eta^2 (g1+g2)^2) = 40 * 0.04 / 1.21, T = 2 < b
    c2 = [[1.0, 1.0], [5.0, 2.8]]
    _, b_next, T, _, _ = orc.local_round_worker_test(np.array([[3.0], [3.0]]), lambda m, h, x: x - c2[m][h], 2, 0.5, 40, 100, 0.5)
    assert (T, b_next) == (2, 40)
    # the estimator: for batch gradients that are means of b i.i.d. samples, b * Var_m(g^m) estimates the
    # per-sample variance (Section 4.3); checked in expectation elsewhere (test_worker_gradient_estimator_...)
