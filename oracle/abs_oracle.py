"""Plain fp64 CPU oracle for the adaptive-batch-size test and the local updates.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only the test-suite, the smoke
check and the benchmark's CPU-baseline leg may import it.  It shares no code
with the CUDA library and imports nothing but numpy.  Every function is the
paper's definition written out the slow way, in double precision, in the
paper's notation, so that a reader can check it against the paper by eye:

    b        local batch size |B|                     (Section 3.1)
    g_i      per-sample gradient, row i of G[b, d]    (Eq. batch_grad)
    gbar     batch gradient (1/b) sum_i g_i           (Eq. batch_grad)
    Var      batch variance with the 1/(b-1) factor   (Eq. def_var)
    eta      norm-test constant                       (Eq. approx_norm)
    T        test statistic, a ceiling                (Eq. norm_test, Alg. 1)
    M, H     workers, local steps per round           (Eq. local_sgd_alt)

Pins (see tests/test_oracle_pins.py): numpy's ddof=1 column variance, the
pairwise-difference U-statistic forms evaluated in exact rational arithmetic on
tiny inputs, the b=2 special case, the split Var_norm = Var_ip/N + Var_orth,
parallel / orthogonal special cases, the chi-square expectations for isotropic
Gaussian rows, a hand-worked example, torch.optim.SGD / torch.optim.AdamW in
fp64, and torch.autograd per-sample gradients for the two producer models;
the round functions (local_round, local_round_per_step, run_until_samples) on
a one-dimensional quadratic whose batch sizes, test statistics, iterates and
sample counts are worked by hand.

Parity unpinned (no printed value or independent definition exists in the
paper): the choice of AdamW variant itself (the paper only cites the optimiser;
the rule below is the decoupled-weight-decay rule of the cited work and is
pinned to torch.optim.AdamW), and the inner-product / orthogonality test
formulas (the paper only cites them; the formulas are those of the cited
adaptive-sampling work).
"""
import math

import numpy as np

STATUS_NONFINITE = 1  # some input or intermediate was not finite
STATUS_ZERO_MEAN = 2  # ||gbar||^2 == 0, the ratios are undefined
T_SATURATE = 1 << 62  # ceilings at or above this are reported as this value


# ----------------------------------------------------------------------------
# input widening
# ----------------------------------------------------------------------------
def bf16_bits_to_f64(bits):
    """Widen bfloat16 bit patterns (uint16) exactly to float64.

    A bfloat16 is the upper half of an IEEE binary32, so the widening is a
    16-bit shift followed by the exact float32 -> float64 conversion.
    """
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    as_f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


# ----------------------------------------------------------------------------
# the batch-size test statistics
# ----------------------------------------------------------------------------
def batch_mean(h):
    """E_{i in B}[h_i] = (1/b) sum_i h_i  (text below Eq. def_var; Eq. batch_grad)."""
    h = np.asarray(h, dtype=np.float64)
    b = h.shape[0]
    total = np.zeros(h.shape[1:], dtype=np.float64)
    for i in range(b):
        total = total + h[i]
    return total / b


def batch_variance(h):
    """Var_{i in B}(h_i) = 1/(b-1) sum_i ||h_i - E[h]||^2  (Eq. def_var).

    h is [b] (scalars) or [b, k] (vectors); the squared Euclidean norm of each
    centred row is formed explicitly and the rows are summed one by one.
    """
    h = np.asarray(h, dtype=np.float64)
    b = h.shape[0]
    if b < 2:
        raise ValueError("the batch variance needs b >= 2 (Eq. def_var divides by b-1)")
    mean = batch_mean(h)
    acc = 0.0
    for i in range(b):
        diff = np.atleast_1d(h[i] - mean)
        acc += float(np.dot(diff, diff))
    return acc / (b - 1)


def batch_test_stats(G):
    """All statistics of one worker's batch G[b, d] (rows = per-sample gradients).

    Returns a dict with
      gbar      batch gradient                                   (Eq. batch_grad)
      gbar_sq   N = ||gbar||^2                                    (rhs of Eq. approx_norm)
      var_norm  Var_i(g_i)                                        (Eq. def_var)
      c         c_i = <g_i, gbar>
      var_ip    Var_i(<g_i, gbar>)            (inner-product test of the cited work)
      var_orth  Var_i(g_i - (c_i / N) gbar)   (orthogonality test of the cited work)
      sum_sq    sum_i ||g_i||^2
      status    STATUS_* bits
    When N == 0 the projection onto gbar is the zero vector, so the orthogonal
    component of g_i is g_i itself and var_orth equals var_norm.
    """
    G = np.asarray(G, dtype=np.float64)
    if G.ndim != 2:
        raise ValueError("G must be [b, d]")
    b, d = G.shape
    if b < 2:
        raise ValueError("b >= 2 required (Eq. def_var)")
    gbar = batch_mean(G)
    N = float(np.dot(gbar, gbar))
    var_norm = batch_variance(G)

    c = np.empty(b, dtype=np.float64)
    for i in range(b):
        c[i] = float(np.dot(G[i], gbar))
    var_ip = batch_variance(c)

    # orthogonal components o_i = g_i - (c_i / N) gbar, their mean, their variance
    coef = c / N if N > 0.0 else np.zeros(b)
    obar = np.zeros(d, dtype=np.float64)
    for i in range(b):
        obar = obar + (G[i] - coef[i] * gbar)
    obar = obar / b
    acc = 0.0
    for i in range(b):
        diff = (G[i] - coef[i] * gbar) - obar
        acc += float(np.dot(diff, diff))
    var_orth = acc / (b - 1)

    sum_sq = 0.0
    for i in range(b):
        sum_sq += float(np.dot(G[i], G[i]))

    status = 0
    if not (math.isfinite(N) and math.isfinite(var_norm) and math.isfinite(var_ip)
            and math.isfinite(var_orth) and math.isfinite(sum_sq)):
        status |= STATUS_NONFINITE
    if N == 0.0:
        status |= STATUS_ZERO_MEAN
    return dict(gbar=gbar, gbar_sq=N, var_norm=var_norm, c=c, var_ip=var_ip,
                var_orth=var_orth, sum_sq=sum_sq, rows=b, status=status)


# ----------------------------------------------------------------------------
# next batch size
# ----------------------------------------------------------------------------
def _ratio(num, den):
    """num/den with the degenerate cases fixed: 0/x = 0 (also 0/0), x/0 = +inf."""
    if num == 0.0:
        return 0.0
    if den == 0.0:
        return math.inf
    return num / den


def _ceil_saturating(x):
    """Ceiling of a non-negative double as a Python int, saturating at 2^62."""
    if x >= float(T_SATURATE):
        return T_SATURATE
    return int(math.ceil(x))


def batch_test_statistic(stats, kind, eta=0.0, theta=0.0, nu=0.0, row_weight=1.0, divisor=1.0):
    """Per-worker T (Alg. 1: T = ceil(Var / (eta^2 ||gbar||^2)); Eq. norm_test, Eq. test_stat).

    kind "norm":  T = ceil( s/D * Var_norm / (eta^2 N) )
    kind "aug_ip": T = max( ceil( s/D * Var_ip / (theta^2 N^2) ),
                            ceil( s/D * Var_orth / (nu^2 N) ) )
    s = row_weight is the number of samples one row stands for (the variance of
    a mean of s samples is 1/s of the per-sample variance, Section 4.3), and
    D = divisor is the extra M of Eq. test_stat_actual.  A record flagged
    non-finite yields T = 0 (no decision).
    """
    if stats["status"] & STATUS_NONFINITE:
        return 0
    N = stats["gbar_sq"]
    scale = row_weight / divisor
    if kind == "norm":
        return _ceil_saturating(scale * _ratio(stats["var_norm"], eta * eta * N))
    if kind == "aug_ip":
        t_ip = _ceil_saturating(scale * _ratio(stats["var_ip"], theta * theta * N * N))
        t_orth = _ceil_saturating(scale * _ratio(stats["var_orth"], nu * nu * N))
        return max(t_ip, t_orth)
    raise ValueError("unknown test kind %r" % (kind,))


def next_batch(stats_per_worker, b_cur, b_max, kind, **cfg):
    """Shared next local batch size.

    b^m_{k+1} = max{T^m, b^m_k} (Alg. 1), all workers then take the maximum
    over m (display below Eq. test_stat), capped at the maximum local batch
    size.  Returns (b_next, [T^1..T^M]).
    """
    T = [batch_test_statistic(s, kind, **cfg) for s in stats_per_worker]
    b_next = b_cur
    for t in T:
        b_next = max(b_next, t)
    return min(b_max, b_next), T


def next_batch_local(stats_per_worker, b_cur_per_worker, b_max, kind, eta_per_worker=None, **cfg):
    """Per-worker next local batch sizes, b^m_{k+1} = max{T^m, b^m_k} capped at b_max, with one
    norm-test constant eta_m per worker (Eq. approx_norm_local, Eq. test_stat, Alg. 1) and no
    maximum over the workers.  Returns ([b^1..b^M], [T^1..T^M])."""
    out, T = [], []
    for m, s in enumerate(stats_per_worker):
        c = dict(cfg)
        if eta_per_worker is not None:
            c["eta"] = eta_per_worker[m]
        t = batch_test_statistic(s, kind, **c)
        T.append(t)
        out.append(min(b_max, max(b_cur_per_worker[m], t)))
    return out, T


def merge_norm_stats(mean_a, n_a, var_a, mean_b, n_b, var_b):
    """Batch gradient and norm-test variance of the union of two disjoint sub-batches from their
    own means and variances (gradient accumulation over micro-batches, Section 6):
      mean = (n_a mean_a + n_b mean_b) / n
      sum_i ||g_i - mean||^2 = S_a + S_b + ||mean_a - mean_b||^2 n_a n_b / n,  S = (n-1) Var (Eq. def_var)
    Returns (mean, n, var, ||mean||^2)."""
    mean_a = np.asarray(mean_a, dtype=np.float64)
    mean_b = np.asarray(mean_b, dtype=np.float64)
    n = n_a + n_b
    mean = (n_a * mean_a + n_b * mean_b) / n
    diff = mean_a - mean_b
    S = (n_a - 1) * var_a + (n_b - 1) * var_b + float(np.dot(diff, diff)) * n_a * n_b / n
    return mean, n, S / (n - 1), float(np.dot(mean, mean))


# ----------------------------------------------------------------------------
# local updates
# ----------------------------------------------------------------------------
def sgd_step(X, Gb, lr):
    """x^m <- x^m - alpha * g^m for every replica m (Eq. local_sgd_alt, first line)."""
    X = np.asarray(X, dtype=np.float64)
    Gb = np.asarray(Gb, dtype=np.float64)
    return X - lr * Gb


def replica_average(X):
    """x^m <- (1/M) sum_m x^m for every m (Eq. local_sgd_alt, second line)."""
    X = np.asarray(X, dtype=np.float64)
    M = X.shape[0]
    mean = np.zeros(X.shape[1:], dtype=np.float64)
    for m in range(M):
        mean = mean + X[m]
    mean = mean / M
    return np.broadcast_to(mean, X.shape).copy()


def adamw_step(X, Mom1, Mom2, Gb, lr, beta1, beta2, eps, weight_decay, t):
    """One AdamW step with decoupled weight decay, step counter t (1-based).

    m <- beta1 m + (1-beta1) g ;  v <- beta2 v + (1-beta2) g^2
    x <- x (1 - lr wd)
    x <- x - lr * (m / (1-beta1^t)) / ( sqrt(v / (1-beta2^t)) + eps )
    The paper names AdamW as an inner optimiser (Section 4.2) and gives its
    hyper-parameters (Appendix C.2); the rule is the cited optimiser's.
    Returns (X, Mom1, Mom2).
    """
    X = np.asarray(X, dtype=np.float64)
    Mom1 = np.asarray(Mom1, dtype=np.float64)
    Mom2 = np.asarray(Mom2, dtype=np.float64)
    Gb = np.asarray(Gb, dtype=np.float64)
    m = beta1 * Mom1 + (1.0 - beta1) * Gb
    v = beta2 * Mom2 + (1.0 - beta2) * Gb * Gb
    mhat = m / (1.0 - beta1 ** t)
    vhat = v / (1.0 - beta2 ** t)
    x = X * (1.0 - lr * weight_decay)
    x = x - lr * mhat / (np.sqrt(vhat) + eps)
    return x, m, v


def shb_step(X, Buf, Gb, lr, momentum, weight_decay):
    """Local stochastic heavy ball (momentum SGD) step, the inner optimiser of
    the paper's image experiments (Section 6.1; momentum 0.9, weight decay 1e-4).

    g <- g + wd x ;  u <- momentum u + g ;  x <- x - lr u
    Returns (X, Buf).
    """
    X = np.asarray(X, dtype=np.float64)
    Buf = np.asarray(Buf, dtype=np.float64)
    g = np.asarray(Gb, dtype=np.float64) + weight_decay * X
    u = momentum * Buf + g
    return X - lr * u, u


# ----------------------------------------------------------------------------
# producers: per-sample gradients of the two synthetic models
# ----------------------------------------------------------------------------
def logreg_per_sample_grads(A, y, x):
    """Per-sample gradients of the logistic loss, rows (sigmoid(a_i^T x) - y_i) a_i.

    A [b, d] features, y [b] labels in {0, 1}, x [d] parameters; no bias, no
    regulariser (Alg. 1, per-sample gradient step).
    """
    A = np.asarray(A, dtype=np.float64)
    y = np.asarray(y, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    b = A.shape[0]
    G = np.empty_like(A)
    for i in range(b):
        z = float(np.dot(A[i], x))
        p = 1.0 / (1.0 + math.exp(-z)) if z >= 0 else math.exp(z) / (1.0 + math.exp(z))
        G[i] = (p - y[i]) * A[i]
    return G


MLP_DIMS = (784, 1024, 1024, 10)


def mlp_param_count(dims=MLP_DIMS):
    return sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))


def mlp_unpack(x, dims=MLP_DIMS):
    """Split the flat parameter vector into [(W_l [out, in], bias_l [out])]; layout
    W1, b1, W2, b2, W3, b3 with each W row-major [out][in]."""
    x = np.asarray(x, dtype=np.float64)
    out, off = [], 0
    for l in range(len(dims) - 1):
        nin, nout = dims[l], dims[l + 1]
        W = x[off:off + nout * nin].reshape(nout, nin)
        off += nout * nin
        bias = x[off:off + nout]
        off += nout
        out.append((W, bias))
    return out


def mlp_per_sample_grads(inputs, labels, x, dims=MLP_DIMS):
    """Per-sample gradients of softmax cross-entropy through a ReLU MLP.

    inputs [b, dims[0]], labels [b] ints, x flat parameters.  Row i of the
    result is the gradient of the loss of sample i alone, in the flat layout of
    mlp_unpack.  Back-propagation is done sample by sample.
    """
    inputs = np.asarray(inputs, dtype=np.float64)
    layers = mlp_unpack(x, dims)
    L = len(layers)
    b = inputs.shape[0]
    G = np.empty((b, mlp_param_count(dims)), dtype=np.float64)
    for i in range(b):
        acts = [inputs[i]]
        pre = []
        for l, (W, bias) in enumerate(layers):
            z = W @ acts[-1] + bias
            pre.append(z)
            acts.append(np.maximum(z, 0.0) if l < L - 1 else z)
        logits = acts[-1]
        shifted = logits - logits.max()
        prob = np.exp(shifted)
        prob = prob / prob.sum()
        delta = prob.copy()
        delta[int(labels[i])] -= 1.0
        grads = [None] * L
        for l in range(L - 1, -1, -1):
            W, _ = layers[l]
            grads[l] = (np.outer(delta, acts[l]), delta.copy())
            if l > 0:
                delta = (W.T @ delta) * (pre[l - 1] > 0.0)
        off = 0
        for (dW, db) in grads:
            G[i, off:off + dW.size] = dW.reshape(-1)
            off += dW.size
            G[i, off:off + db.size] = db
            off += db.size
    return G


# ----------------------------------------------------------------------------
# one communication round (Alg. 2 structure, per-sample statistic of Alg. 1)
# ----------------------------------------------------------------------------
def local_round(X, per_sample_grads, batches, lr, b_cur, b_max, kind, **cfg):
    """One round: H local SGD steps per worker, the test on the last step's
    per-sample gradients, model averaging, batch-size update.

    X [M, d] replicas at the start of the round; per_sample_grads(m, h, x)
    returns G[b, d] of worker m's batch at local step h evaluated at x;
    batches is only its length H.  The test is evaluated once per round
    (Section 4.3, last paragraph) on the gradients of local step H-1.
    Returns (X_next, b_next, T list, stats list).
    """
    X = np.array(X, dtype=np.float64)
    M = X.shape[0]
    H = batches
    stats = [None] * M
    for h in range(H):
        Gb = np.empty_like(X)
        for m in range(M):
            G = per_sample_grads(m, h, X[m])
            Gb[m] = batch_mean(G)
            if h == H - 1:
                stats[m] = batch_test_stats(G)
        X = sgd_step(X, Gb, lr)
    X = replica_average(X)
    b_next, T = next_batch(stats, b_cur, b_max, kind, **cfg)
    return X, b_next, T, stats


# ----------------------------------------------------------------------------
# Algorithm 1 as printed: the test after every local step, per worker
# ----------------------------------------------------------------------------
def local_round_per_step(X, per_sample_grads, H, lr, b_cur, b_max, kind, shared=False,
                         eta_per_worker=None, **cfg):
    """One round of Alg. 1: for every worker m and local step h = 0..H-1
        sample a batch of the worker's current size b^m_{k,h},
        per-sample gradients at x^m_{k,h}, their mean (Eq. batch_grad) and variance (Eq. def_var),
        T^m_{k,h} (the ceiling of Alg. 1; Eq. test_stat),
        b^m_{k,h+1} = max{T^m_{k,h}, b^m_{k,h}}  (capped at the maximum local batch size),
        x^m_{k,h+1} = x^m_{k,h} - lr * batch gradient,
    then the model averaging (Eq. local_sgd_alt, second line).

    X [M, d]; per_sample_grads(m, h, x, b) returns G[b, d] of worker m's batch of size b at step h;
    b_cur is the list [b^1_{k,0} .. b^M_{k,0}].  With shared=True every worker continues with the
    maximum over the workers (the practical rule below Eq. test_stat), applied after every step.
    eta_per_worker gives the constants eta_m of Eq. approx_norm_local.
    Returns (X_next, b_next [M], b_used [H][M], T [H][M], stats [H][M], samples) where
    samples = sum_m sum_h b^m_{k,h} is the round's term of the counter B of Alg. 1.
    """
    X = np.array(X, dtype=np.float64)
    M = X.shape[0]
    b = [int(v) for v in b_cur]
    if len(b) != M:
        raise ValueError("one current batch size per worker")
    b_used, T_hist, stats_hist = [], [], []
    samples = 0
    for h in range(H):
        Gb = np.empty_like(X)
        stats = [None] * M
        for m in range(M):
            G = per_sample_grads(m, h, X[m], b[m])
            if G.shape[0] != b[m]:
                raise ValueError("the batch of worker %d at step %d must have %d rows" % (m, h, b[m]))
            Gb[m] = batch_mean(G)
            stats[m] = batch_test_stats(G)
            samples += b[m]
        b_used.append(list(b))
        b, T = next_batch_local(stats, b, b_max, kind, eta_per_worker=eta_per_worker, **cfg)
        if shared:
            b = [max(b)] * M
        T_hist.append(T)
        stats_hist.append(stats)
        X = sgd_step(X, Gb, lr)
    X = replica_average(X)
    return X, b, b_used, T_hist, stats_hist, samples


def samples_of_round(H, M, b):
    """The round's term of the sample counter in Alg. 2: B <- B + H M b_k."""
    return H * M * b


def run_until_samples(X0, per_sample_grads, H, lr, b0, b_max, kind, n_samples, per_step=False,
                      shared=True, max_rounds=10 ** 6, **cfg):
    """The outer loop of Alg. 1 / Alg. 2: rounds k = 0, 1, ... while B < N, the counter B growing
    by the samples each round processed; the output is x_hat = x^1_{K,0}, K the first round count
    with B >= N.

    per_sample_grads(k, m, h, x, b) returns G[b, d].  per_step=False runs local_round (the test once
    per round on the last step, B += H M b); per_step=True runs local_round_per_step (B += sum_m
    sum_h b^m_{k,h}).  Returns (x_hat, K, B, history) with history[k] = the batch sizes round k
    started with (an int, or a list per worker for per_step).
    """
    X = np.array(X0, dtype=np.float64)
    M = X.shape[0]
    B, k = 0, 0
    b = [int(b0)] * M if per_step else int(b0)
    history = []
    while B < n_samples and k < max_rounds:
        history.append(list(b) if per_step else b)
        if per_step:
            X, b, _, _, _, used = local_round_per_step(
                X, lambda m, h, x, bb, k=k: per_sample_grads(k, m, h, x, bb), H, lr, b, b_max, kind,
                shared=shared, **cfg)
            B += used
        else:
            X, b_next, _, _ = local_round(
                X, lambda m, h, x, k=k, b=b: per_sample_grads(k, m, h, x, b), H, lr, b, b_max, kind, **cfg)
            B += samples_of_round(H, M, b)
            b = b_next
        k += 1
    return X[0].copy(), k, B, history


# ----------------------------------------------------------------------------
# Algorithm 2 as printed: the test on the workers' batch gradients
# ----------------------------------------------------------------------------
def local_round_worker_test(X, batch_grads, H, lr, b_cur, b_max, eta):
    """One round of Alg. 2 ("actual implementation"): H local SGD steps per worker on batch
    gradients only, model averaging, then the norm test from the WORKERS' batch gradients:
        gbar = (1/M) sum_m g^m,
        Var  = b * 1/(M-1) sum_m ||g^m - gbar||^2          (the estimator of Section 4.3),
        T    = ceil( Var / (M eta^2 ||gbar||^2) )          (Eq. test_stat_actual),
        b_next = max{T, b}  (capped at the maximum local batch size),
    where g^m is worker m's batch gradient of the round's last local step (the gradients that
    exist when the models are synchronised).  The sample counter grows by H M b.

    X [M, d]; batch_grads(m, h, x) returns the batch gradient [d] of worker m at local step h.
    Returns (X_next, b_next, T, stats of the M gradients as rows, samples).
    """
    X = np.array(X, dtype=np.float64)
    M = X.shape[0]
    if M < 2:
        raise ValueError("the variance over workers needs M >= 2")
    Gb = np.empty_like(X)
    for h in range(H):
        for m in range(M):
            Gb[m] = np.asarray(batch_grads(m, h, X[m]), dtype=np.float64)
        X = sgd_step(X, Gb, lr)
    X = replica_average(X)
    stats = batch_test_stats(Gb)                      # rows = workers: var_norm = 1/(M-1) sum ||g^m - gbar||^2
    T = batch_test_statistic(stats, "norm", eta=eta, row_weight=float(b_cur), divisor=float(M))
    b_next = min(b_max, max(b_cur, T))
    return X, b_next, T, stats, samples_of_round(H, M, b_cur)
