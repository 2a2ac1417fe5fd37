"""Parity at the benchmark's full sizes, in the launch configurations bench.py times.  Workload c5
(8 rows of 25e6 entries): every worker row and the master row are checked against the oracle bit for bit
(the oracle rows run in a pool of spawned processes), and through properties that hold at any size.  Workloads c2, c3, c4: gradients
of sampled workers against the oracle (rel 1e-5) and the selections of an iteration on sampled rows."""
import multiprocessing as mp
import os

import numpy as np
import pytest

import synthetic_inputs as S
from oracle import adacgd_oracle as O

pytestmark = pytest.mark.gpu
F32 = np.float32


def test_c5_full_size_step():
    import torch
    import paper_2211_00188_b200 as pkg

    W = S.WORKLOADS["c5"]
    n, d = W["n"], W["d"]
    dev = torch.device("cuda:0")
    Xs, G = S.stress_vectors(n, d, W["blocks"], W["period"], seed=0, device=dev)
    eng = pkg.AdaCGD(n, d, W["worker"], 1.0, W["master"], 1.0)
    X, Y = Xs[1], Xs[0]
    G_before = G.clone()
    gt_old = G.mean(0)
    gm = gt_old.clone().view(1, d)
    gm_before = gm.clone()
    gt_new = torch.empty(d, device=dev)
    level = torch.zeros(n, dtype=torch.int32, device=dev)
    bits = torch.zeros(n, dtype=torch.int64, device=dev)
    mlevel = torch.zeros(1, dtype=torch.int32, device=dev)
    eng.compress(X, G, Y, mean_out=gt_new, level=level, bits=bits)
    eng.compress(gt_new.view(1, d), gm, gt_old.view(1, d), W["master"], 1.0, level=mlevel)
    torch.cuda.synchronize()
    assert eng.get_state("flags") == 0
    levels = level.cpu().tolist()

    # properties for every row: a level j changes at most K_j entries, skips change none, and the
    # changed entries become exactly fl(g + fl(x - g))
    for i in range(n):
        changed = (G[i] != G_before[i])
        nchanged = int(changed.sum())
        if levels[i] == 0:
            assert nchanged == 0
            continue
        K = W["worker"][levels[i] - 1][1]
        assert 0 < nchanged <= K
        want = G_before[i] + (X[i] - G_before[i])
        assert torch.equal(G[i][changed], want[changed])
        # every changed entry is at least as large in magnitude as every unchanged one
        v = (X[i] - G_before[i]).abs()
        assert float(v[changed].min()) >= float(v[~changed].max())
        assert int(bits[i]) == K * (32 + 25)          # ceil(log2 25e6) = 25

    # the mean in worker order, bit for bit (numpy float32, left to right)
    Gh = G.cpu().numpy()
    assert np.array_equal(gt_new.cpu().numpy().view(np.uint32), O.server_mean(Gh).view(np.uint32))

    # every worker row and the master row against the oracle: level, bits, number of entries written, and the
    # estimator bit for bit.  The nine oracle calls run side by side in spawned processes (a process forked
    # after the first CUDA call would not be safe).
    jobs = [(G_before[i].cpu().numpy(), Y[i].cpu().numpy(), X[i].cpu().numpy(), W["worker"], 1.0) for i in range(n)]
    jobs.append((gm_before[0].cpu().numpy(), gt_old.cpu().numpy(), gt_new.cpu().numpy(), W["master"], 1.0))
    with mp.get_context("spawn").Pool(min(len(jobs), max(1, (os.cpu_count() or 2) // 2))) as pool:
        refs = pool.starmap(O.adacgd, jobs)
    for i in range(n):
        ref = refs[i]
        assert levels[i] == ref["level"] and int(bits[i]) == ref["bits"], (i, levels[i], ref["level"])
        assert np.array_equal(Gh[i].view(np.uint32), ref["out"].view(np.uint32)), i
        if ref["kept"] is not None:
            assert len(ref["kept"]) == W["worker"][ref["level"] - 1][1]
    mref = refs[n]
    assert int(mlevel.item()) == mref["level"]
    assert np.array_equal(gm[0].cpu().numpy().view(np.uint32), mref["out"].view(np.uint32))


def relerr(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def check_rows_after_one_step(eng, rows, G_before, Y_before, cands, zeta, recs, levels):
    """The rows `rows` of a step the engine has just run, against the oracle's compressor fed with the
    engine's own gradients: level, bits and the updated estimator row, bit for bit."""
    X = eng.get_state("grad").cpu().numpy()
    G_after = eng.get_state("G").cpu().numpy()
    for i in rows:
        ref = O.adacgd(G_before[i], Y_before[i], X[i], cands, zeta)
        assert levels[0][i] == ref["level"], (i, levels[0][i], ref["level"])
        assert np.array_equal(G_after[i].view(np.uint32), ref["out"].view(np.uint32)), i
    return X, G_after


def test_c2_full_size_lockstep():
    # workload c2 as benchmarked (20 x 8 000, 2 000 samples per worker, bidirectional): two lock-step iterations
    from test_step_gpu import lockstep
    import torch
    W = S.WORKLOADS["c2"]
    A, t = S.logistic_problem(W["n"], W["d"], W["m"], seed=0)
    gamma = 0.5 / S.smoothness_estimate(A, W["loss"], W["lam"], iters=8)
    lockstep(torch, A, t, W["loss"], W["lam"], gamma, W["worker"], 1.0, W["master"], 1.0, T=2)


def test_c3_full_size_gradient_and_step():
    # workload c3 as benchmarked (100 x 100 000, CSR 1 %, 500 samples per worker, Top-K and quantisers mixed)
    import scipy.sparse as sp
    import torch
    import paper_2211_00188_b200 as pkg
    W = S.WORKLOADS["c3"]
    n, d, m = W["n"], W["d"], W["m"]
    rowptr, col, val, y = S.sparse_logistic_problem(n, d, m, density=W["density"], seed=0)
    dev = torch.device("cuda:0")
    csr = tuple(torch.from_numpy(a).to(dev) for a in S.csr_global(rowptr, col, val))
    eng = pkg.AdaCGD(n, d, W["worker"], 1.0, W["master"], 1.0, loss=W["loss"], lam=W["lam"], csr=csr,
                     target=torch.from_numpy(y).to(dev), x0=torch.zeros(d, device=dev), gamma=0.5 / (0.25 + W["lam"]))
    sample = [0, 57, 99]
    prob = dict(A=[sp.csr_matrix((val[i], col[i], rowptr[i]), shape=(m, d)) for i in sample],
                target=[y[i] for i in sample], loss=W["loss"], lam=W["lam"])
    x = (0.3 * np.random.Generator(np.random.PCG64(3)).standard_normal(d)).astype(F32)
    out = torch.zeros(n, d, device=dev)
    eng.gradient(torch.from_numpy(x).to(dev), out)
    want = O.all_gradients(prob, x)
    got = out.cpu().numpy()
    for k, i in enumerate(sample):
        assert relerr(got[i], want[k]) <= 1e-5, (i, relerr(got[i], want[k]))
    # one iteration from the initial state: sampled rows against the oracle's compressor
    eng.step(3)
    G_before = eng.get_state("G").cpu().numpy()
    Y_before = eng.get_state("grad").cpu().numpy()
    recs, levels = eng.step(1, report=True)
    check_rows_after_one_step(eng, sample, G_before, Y_before, W["worker"], 1.0, recs, levels)
    assert eng.get_state("flags") == 0


def test_c4_full_size_gradient_and_step():
    # workload c4 as benchmarked (16 x 1 000 000, 256 samples per worker, 16.4 GB of features drawn on the device)
    import torch
    import paper_2211_00188_b200 as pkg
    W = S.WORKLOADS["c4"]
    n, d, m = W["n"], W["d"], W["m"]
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(0)
    A = torch.empty(n, m, d, device=dev)
    for i in range(n):
        A[i] = torch.randn(m, d, generator=gen, device=dev) / d ** 0.5
    xs = torch.randn(d, generator=gen, device=dev)
    tgt = torch.einsum("nmd,d->nm", A, xs) + 0.1 * torch.randn(n, m, generator=gen, device=dev)
    gamma = 0.5 / ((1.0 + (n * m / d) ** 0.5) ** 2 / (n * m))
    eng = pkg.AdaCGD(n, d, W["worker"], 1.0, W["master"], 1.0, loss=W["loss"], lam=W["lam"], A=A, target=tgt,
                     x0=torch.zeros(d, device=dev), gamma=gamma)
    sample = [0, 11]
    x = (0.5 * np.random.Generator(np.random.PCG64(4)).standard_normal(d)).astype(F32)
    out = torch.zeros(n, d, device=dev)
    eng.gradient(torch.from_numpy(x).to(dev), out)
    for i in sample:
        want = O.local_gradient(A[i].cpu().numpy(), tgt[i].cpu().numpy(), x, W["loss"], W["lam"])
        got = out[i].cpu().numpy()
        assert relerr(got, want) <= 1e-5, (i, relerr(got, want))
        assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max()
    del out
    eng.step(2)
    G_before = eng.get_state("G").cpu().numpy()
    Y_before = eng.get_state("grad").cpu().numpy()
    recs, levels = eng.step(1, report=True)
    _, G_after = check_rows_after_one_step(eng, sample, G_before, Y_before, W["worker"], 1.0, recs, levels)
    # the server mean of the full 16 x 1e6 state, bit for bit
    assert np.array_equal(eng.get_state("gt").cpu().numpy().view(np.uint32), O.server_mean(G_after).view(np.uint32))
    assert eng.get_state("flags") == 0
