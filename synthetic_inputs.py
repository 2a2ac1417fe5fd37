"""Seeded synthetic inputs shaped like the workloads AdaCGD is measured on.

This module only draws numbers.  It holds none of the method's arithmetic (no
gradient, no compressor, no trigger) and is the one module that both the CPU
oracle's tests and the CUDA path's tests / benchmark import, so that both sides
consume bit-identical binary32 arrays.

Workloads (n workers, dimension d, m samples per worker):

  c1  n=4    d=1 000      m=100    dense logistic + non-convex reg, Top-K {10,50,100,500}
  c2  n=20   d=8 000      m=2 000  same generator, Top-K {d/1000,d/100,d/10,d}, bidirectional
  c3  n=100  d=100 000    m=500    CSR 1 % density, logistic + l2, Top-K and quantiser mix
  c4  n=16   d=1 000 000  m=256    dense least squares, Top-K {1e3,1e4,1e5}
  c5  n=8    d=25 000 000          compression-only stress: heavy-tailed gradient-like rows

The paper's own experiments use LIBSVM data sets split over n=20 clients; they are
not available here and these generators stand in for them.
"""
from __future__ import annotations

import numpy as np

F32 = np.float32

TOPK = 0
QUANT = 1

WORKLOADS = {
    "c1": dict(n=4, d=1000, m=100, loss=0, lam=0.1, layout="dense", iters=100,
               worker=[(TOPK, 10), (TOPK, 50), (TOPK, 100), (TOPK, 500)], master=[]),
    "c2": dict(n=20, d=8000, m=2000, loss=0, lam=0.1, layout="dense", iters=1000,
               worker=[(TOPK, 8), (TOPK, 80), (TOPK, 800), (TOPK, 8000)],
               master=[(TOPK, 8), (TOPK, 80), (TOPK, 800), (TOPK, 8000)]),
    "c3": dict(n=100, d=100000, m=500, loss=1, lam=1e-3, layout="csr", density=0.01, iters=500,
               worker=[(TOPK, 100), (TOPK, 1000), (QUANT, 2), (QUANT, 4), (TOPK, 10000), (QUANT, 8)],
               master=[]),
    "c4": dict(n=16, d=1000000, m=256, loss=2, lam=0.0, layout="dense", iters=200,
               worker=[(TOPK, 1000), (TOPK, 10000), (TOPK, 100000)], master=[]),
    "c5": dict(n=8, d=25000000, blocks=100, period=4, iters=50,
               worker=[(TOPK, 25000), (TOPK, 250000), (TOPK, 2500000)],
               master=[(TOPK, 25000), (TOPK, 250000), (TOPK, 2500000)]),
}


def logistic_problem(n, d, m, seed=0, shift_var=0.5, flip=0.05):
    """Dense classification data: a ~ N(0, I) + mu_i with a per-worker shift
    mu_i ~ N(0, shift_var I); labels sign(a . x*) with x* ~ N(0, I), a fraction
    `flip` of them negated.  Returns (A [n,m,d] f32, y [n,m] f32 in {-1,+1})."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x_star = rng.standard_normal(d)
    A = np.empty((n, m, d), dtype=F32)
    y = np.empty((n, m), dtype=F32)
    for i in range(n):
        mu = np.sqrt(shift_var) * rng.standard_normal(d)
        a = (rng.standard_normal((m, d)) + mu).astype(F32)
        lab = np.where(a.astype(np.float64) @ x_star >= 0, 1.0, -1.0)
        lab = np.where(rng.random(m) < flip, -lab, lab)
        A[i] = a
        y[i] = lab.astype(F32)
    return A, y


def least_squares_problem(n, d, m, seed=0, noise_var=0.01):
    """A_i ~ N(0, 1/d) entrywise, b_i = A_i x* + N(0, noise_var), x* ~ N(0, I).
    Returns (A [n,m,d] f32, b [n,m] f32, x_star [d] f64)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    x_star = rng.standard_normal(d)
    A = np.empty((n, m, d), dtype=F32)
    b = np.empty((n, m), dtype=F32)
    for i in range(n):
        a = (rng.standard_normal((m, d)) / np.sqrt(d)).astype(F32)
        A[i] = a
        b[i] = (a.astype(np.float64) @ x_star + np.sqrt(noise_var) * rng.standard_normal(m)).astype(F32)
    return A, b, x_star


def sparse_logistic_problem(n, d, m, density=0.01, seed=0, flip=0.05):
    """CSR classification data: every row has round(density*d) distinct columns
    drawn uniformly, values ~ U(0,1), rows scaled to unit l2 norm in binary32.
    Labels as in `logistic_problem`.  Returns per-worker CSR triplets
    (rowptr int64 [n, m+1], col int32 [n, m*k], val f32 [n, m*k]) and y [n,m]."""
    rng = np.random.Generator(np.random.PCG64(seed))
    k = max(1, int(round(density * d)))
    x_star = rng.standard_normal(d)
    rowptr = np.tile(np.arange(0, (m + 1) * k, k, dtype=np.int64), (n, 1))
    col = np.empty((n, m * k), dtype=np.int32)
    val = np.empty((n, m * k), dtype=F32)
    y = np.empty((n, m), dtype=F32)
    for i in range(n):
        for r in range(m):
            c = np.sort(rng.choice(d, size=k, replace=False)).astype(np.int32)
            v = rng.random(k).astype(F32)
            v = (v / F32(np.sqrt(np.sum(v.astype(np.float64) ** 2)))).astype(F32)
            col[i, r * k:(r + 1) * k] = c
            val[i, r * k:(r + 1) * k] = v
            z = float(v.astype(np.float64) @ x_star[c])
            y[i, r] = 1.0 if z >= 0 else -1.0
        flips = rng.random(m) < flip
        y[i] = np.where(flips, -y[i], y[i])
    return rowptr, col, val, y


def sparse_problem_with_dense_columns(n, d, m, dense_cols=64, extra=16, seed=0):
    """CSR classification data whose first `dense_cols` columns are stored in every sample row while
    every row has only `extra` more columns, drawn uniformly from the rest: a few very long columns
    next to many short ones.  Values ~ U(0,1), labels +-1 uniformly.  Same return layout as
    `sparse_logistic_problem`."""
    rng = np.random.Generator(np.random.PCG64(seed))
    k = dense_cols + extra
    rowptr = np.tile(np.arange(0, (m + 1) * k, k, dtype=np.int64), (n, 1))
    col = np.empty((n, m * k), dtype=np.int32)
    val = rng.random((n, m * k)).astype(F32)
    y = np.where(rng.random((n, m)) < 0.5, -1.0, 1.0).astype(F32)
    head = np.arange(dense_cols, dtype=np.int32)
    for i in range(n):
        for r in range(m):
            tail = np.sort(rng.choice(d - dense_cols, size=extra, replace=False)).astype(np.int32) + dense_cols
            col[i, r * k:(r + 1) * k] = np.concatenate([head, tail])
    return rowptr, col, val, y


def stress_vectors(n, d, blocks=100, period=4, seed=0, device="cpu"):
    """Gradient-like rows for the compression-only workload.

    u_i: Student-t (nu=3) entries times a per-block scale s_b = 1e-2*exp(N(0,1)),
    constant on `blocks` contiguous blocks (the same scales on every worker).
    The "gradient" at step t moves on a cycle of `period` buffers
        X^t = u_i + 0.1*(cos(2 pi t/period) e1_i + sin(2 pi t/period) e2_i),
    e1_i, e2_i drawn like u_i.  The estimator starts at a perturbed copy
        G^0 = X^0 + 0.3 * s_b * N(0,1).
    Returns (Xs: list of `period` torch tensors [n,d] f32, G0 [n,d] f32) on `device`."""
    import math
    import torch

    gen = torch.Generator(device=device)
    gen.manual_seed(seed)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, device=device, dtype=torch.float32)

    scale_b = 1e-2 * torch.exp(randn(blocks))
    edges = [(b * d) // blocks for b in range(blocks + 1)]
    scale = torch.empty(d, device=device, dtype=torch.float32)
    for b in range(blocks):
        scale[edges[b]:edges[b + 1]] = scale_b[b]

    def student_rows():
        out = torch.empty(n, d, device=device, dtype=torch.float32)
        for i in range(n):  # row by row keeps temporaries small at d = 25e6
            chi = randn(d) ** 2 + randn(d) ** 2 + randn(d) ** 2
            out[i] = randn(d) / torch.sqrt(chi / 3.0) * scale
        return out

    u, e1, e2 = student_rows(), student_rows(), student_rows()
    Xs = []
    for t in range(period):
        ang = 2.0 * math.pi * t / period
        Xs.append(u + 0.1 * (math.cos(ang) * e1 + math.sin(ang) * e2))
    G0 = torch.empty(n, d, device=device, dtype=torch.float32)
    for i in range(n):
        G0[i] = Xs[0][i] + 0.3 * scale * randn(d)
    return Xs, G0


def tie_vectors(rows, d, seed=0, levels=5):
    """Small-integer rows with many exact ties, zeros and signed zeros: the
    adversarial input for the (|v| descending, index ascending) tie rule and
    for trigger comparisons that hold with equality."""
    rng = np.random.Generator(np.random.PCG64(seed))
    X = rng.integers(-levels, levels + 1, size=(rows, d)).astype(F32)
    G = rng.integers(-levels, levels + 1, size=(rows, d)).astype(F32)
    Y = rng.integers(-levels, levels + 1, size=(rows, d)).astype(F32)
    neg = rng.random((rows, d)) < 0.1
    X = np.where(neg & (X == 0), F32(-0.0), X).astype(F32)
    return X, G, Y


def gaussian_rows(rows, d, seed=0, drift=0.3, move=0.1):
    """Continuous test rows: X ~ N(0,1), G = X + drift*N(0,1), Y = X + move*N(0,1)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    X = rng.standard_normal((rows, d)).astype(F32)
    G = (X + drift * rng.standard_normal((rows, d))).astype(F32)
    Y = (X + move * rng.standard_normal((rows, d))).astype(F32)
    return X, G, Y


def smoothness_estimate(A, loss: int, lam: float, iters: int = 30, seed: int = 0) -> float:
    """Upper estimate of the smoothness constant of f = (1/n) sum f_i by power iteration
    (binary64, host): lambda_max of (1/(n m)) sum_i A_i^T A_i, times 1/4 for the logistic
    losses, plus the regulariser's curvature bound (2 lam for x^2/(1+x^2), lam for l2).
    Used only to pick a step size gamma for the workloads."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n, m, d = A.shape
    v = rng.standard_normal(d)
    v /= np.linalg.norm(v)
    lam_max = 0.0
    for _ in range(iters):
        w = np.zeros(d)
        for i in range(n):
            Ai = A[i].astype(np.float64)
            w += Ai.T @ (Ai @ v)
        w /= n * m
        lam_max = float(np.linalg.norm(w))
        v = w / max(lam_max, 1e-300)
    if loss == 2:
        return lam_max
    return 0.25 * lam_max + (2.0 * lam if loss == 0 else lam)


def csr_global(rowptr, col, val):
    """Concatenates per-worker CSR triplets (as returned by `sparse_logistic_problem`) into one CSR
    over all n*m sample rows: (rowptr int64 [n*m+1], col int32 [nnz], val float32 [nnz])."""
    n, m1 = rowptr.shape
    out = [np.zeros(1, dtype=np.int64)]
    base = 0
    for i in range(n):
        out.append(rowptr[i, 1:] + base)
        base += int(rowptr[i, -1])
    return np.concatenate(out), np.ascontiguousarray(col.reshape(-1)), np.ascontiguousarray(val.reshape(-1))
