"""Seeded synthetic inputs shaped like the paper's workloads.

This module only draws random numbers and lays them out; it contains none of
the method's arithmetic (no means, variances, tests or optimiser updates), so
both the CUDA path and the CPU checker can be fed from it.  Everything is a
torch tensor on the requested device; the same seed gives the same values on
the same device type.

Recipes
  gaussian_rows       rows g_i = mu + sigma z_i with mu_j ~ N(0, 1/d), z ~ N(0, 1):
                      per-sample gradients of a noise-dominated model
                      (stands in for the ResNet-scale gradients of Section 6.1)
  student_t_rows      bf16 rows = shared mean direction + Student-t(3) noise of
                      scale 1e-3: heavy-tailed per-micro-batch gradients of a
                      language model (stands in for Section 6.2)
  adamw_problem       M identical replicas x_0 ~ N(0, 0.02^2), zero moments and a
                      small pool of gradient tensors ~ N(0, 1e-4)
  logreg_dataset      a_i ~ N(0, I), labels from a seeded w* with label flips
  gaussian_mixture    10-class Gaussian mixture for the MLP producer
  batch_indices       i.i.d. uniform sample indices (with replacement), drawn once
"""
import math

import torch


def _gen(seed, device):
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def gaussian_rows(seed, M, b, d, sigma, device="cpu", dtype=torch.float32):
    """G[M, b, d]: g_i = mu + sigma * z_i, mu_j ~ N(0, 1/d) shared by all rows."""
    gen = _gen(seed, device)
    mu = torch.empty(d, device=device, dtype=torch.float32).normal_(0.0, 1.0 / math.sqrt(d), generator=gen)
    G = torch.empty((M, b, d), device=device, dtype=torch.float32)
    for m in range(M):
        # row by row keeps the temporaries small for the 100 GB cases
        for i in range(b):
            row = G[m, i]
            row.normal_(0.0, 1.0, generator=gen)
            row.mul_(sigma).add_(mu)
    return G if dtype == torch.float32 else G.to(dtype)


def student_t_rows(seed, M, b, d, scale=1e-3, dof=3, mean_frac=0.1, device="cpu",
                   dtype=torch.bfloat16):
    """G[M, b, d] in `dtype`: shared mean vector (norm mean_frac * E||noise row||,
    random direction) + scale * Student-t(dof) noise, rounded to `dtype` once."""
    gen = _gen(seed, device)
    direction = torch.empty(d, device=device, dtype=torch.float32).normal_(generator=gen)
    direction /= direction.norm()
    noise_row_norm = scale * math.sqrt(dof / (dof - 2.0) * d)
    mean_vec = direction * (mean_frac * noise_row_norm)
    G = torch.empty((M, b, d), device=device, dtype=dtype)
    z = torch.empty(d, device=device, dtype=torch.float32)
    chi = torch.empty(d, device=device, dtype=torch.float32)
    tmp = torch.empty(d, device=device, dtype=torch.float32)
    for m in range(M):
        for i in range(b):
            z.normal_(generator=gen)
            chi.zero_()
            for _ in range(dof):
                tmp.normal_(generator=gen)
                chi.addcmul_(tmp, tmp)
            chi.div_(dof).sqrt_()
            z.div_(chi).mul_(scale).add_(mean_vec)
            G[m, i].copy_(z)
    return G


def tile_columns(small, d):
    """Repeat the columns of small[..., d0] periodically up to width d.  The result is allocated
    once and filled period by period, so a 100 GB tensor needs no second copy of itself."""
    d0 = small.shape[-1]
    out = torch.empty(tuple(small.shape[:-1]) + (d,), device=small.device, dtype=small.dtype)
    for lo in range(0, d, d0):
        w = min(d0, d - lo)
        out[..., lo:lo + w].copy_(small[..., :w])
    return out


def adamw_problem(seed, M, d, pool=4, x_std=0.02, grad_std=0.01, device="cpu"):
    """(X[M,d], Mom1[M,d], Mom2[M,d], grads[pool][M,d]); all replicas start at the same x_0."""
    gen = _gen(seed, device)
    x0 = torch.empty(d, device=device, dtype=torch.float32).normal_(0.0, x_std, generator=gen)
    X = x0.unsqueeze(0).repeat(M, 1).contiguous()
    Mom1 = torch.zeros((M, d), device=device, dtype=torch.float32)
    Mom2 = torch.zeros((M, d), device=device, dtype=torch.float32)
    grads = [torch.empty((M, d), device=device, dtype=torch.float32).normal_(0.0, grad_std, generator=gen)
             for _ in range(pool)]
    return X, Mom1, Mom2, grads


def logreg_dataset(seed, n, d, flip=0.1, device="cpu"):
    """(A[n,d] fp32, y[n] fp32 in {0,1}): y = 1[<a, w*> > 0], flipped with probability `flip`."""
    gen = _gen(seed, device)
    A = torch.empty((n, d), device=device, dtype=torch.float32).normal_(generator=gen)
    w_star = torch.empty(d, device=device, dtype=torch.float32).normal_(generator=gen)
    y = (A @ w_star > 0).to(torch.float32)
    flips = torch.rand(n, device=device, generator=gen) < flip
    y = torch.where(flips, 1.0 - y, y)
    return A, y


def gaussian_mixture(seed, n, dim=784, classes=10, device="cpu"):
    """(inputs[n,dim] fp32, labels[n] int32): class means ~ N(0, I), unit noise, uniform labels."""
    gen = _gen(seed, device)
    means = torch.empty((classes, dim), device=device, dtype=torch.float32).normal_(generator=gen)
    labels = torch.randint(0, classes, (n,), device=device, generator=gen, dtype=torch.int64)
    inputs = torch.empty((n, dim), device=device, dtype=torch.float32).normal_(generator=gen)
    inputs += means[labels]
    return inputs, labels.to(torch.int32)


def mlp_init(seed, dims=(784, 1024, 1024, 10), device="cpu"):
    """Flat parameter vector [W1, b1, W2, b2, ...], W_l row-major [out][in] ~ N(0, 2/in), zero biases."""
    gen = _gen(seed, device)
    parts = []
    for l in range(len(dims) - 1):
        nin, nout = dims[l], dims[l + 1]
        W = torch.empty((nout, nin), device=device, dtype=torch.float32).normal_(
            0.0, math.sqrt(2.0 / nin), generator=gen)
        parts += [W.reshape(-1), torch.zeros(nout, device=device, dtype=torch.float32)]
    return torch.cat(parts)


def batch_indices(seed, shape, n, device="cpu"):
    """int32 tensor of `shape` with i.i.d. uniform indices in [0, n) (sampling with replacement)."""
    gen = _gen(seed, device)
    return torch.randint(0, n, tuple(shape), device=device, generator=gen, dtype=torch.int64).to(torch.int32)


def bf16_bits(t):
    """The raw 16-bit patterns of a bfloat16 tensor as a numpy uint16 array (on the host)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")
