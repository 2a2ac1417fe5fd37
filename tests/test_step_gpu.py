"""Parity of the full iteration (stages a0-a5, Algorithm 1 / Algorithm 2) between the
CUDA path and the CPU oracle: gradients and iterates to rel 1e-5 in lock-step,
selections bit-exact on identical inputs, loss to rel 1e-3 free-running."""
import numpy as np
import pytest

import synthetic_inputs as S
from oracle import adacgd_oracle as O

pytestmark = pytest.mark.gpu
F32 = np.float32
TOPK, QUANT = 0, 1


@pytest.fixture(scope="module")
def torch():
    import torch as t
    return t


def relerr(a, b):
    a, b = np.asarray(a, np.float64), np.asarray(b, np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def make_engine(torch, A, target, loss, lam, x0, gamma, wc, wz, mc=(), mz=0.0, g0_mode=1):
    import paper_2211_00188_b200 as pkg
    dev = torch.device("cuda:0")
    n, m, d = A.shape
    Ad = torch.from_numpy(A).to(dev)
    td = torch.from_numpy(target).to(dev)
    xd = torch.from_numpy(x0).to(dev)
    return pkg.AdaCGD(n, d, wc, wz, mc, mz, loss=loss, lam=lam, A=Ad, target=td, x0=xd, gamma=gamma, g0_mode=g0_mode)


def oracle_problem(A, target, loss, lam):
    return dict(A=[A[i] for i in range(A.shape[0])], target=[target[i] for i in range(A.shape[0])], loss=loss, lam=lam)


@pytest.mark.parametrize("loss,n,m,d", [(0, 3, 50, 1000), (0, 2, 37, 1001), (1, 2, 64, 4096), (2, 3, 40, 777),
                                        (2, 2, 16, 40000), (0, 2, 9, 33001), (0, 20, 300, 800)])
def test_gradient_and_loss(torch, loss, n, m, d):
    if loss == 2:
        A, t, _ = S.least_squares_problem(n, d, m, seed=d)
    else:
        A, t = S.logistic_problem(n, d, m, seed=d)
    lam = 0.1 if loss != 2 else 0.0
    x = (0.3 * np.random.Generator(np.random.PCG64(1)).standard_normal(d)).astype(F32)
    eng = make_engine(torch, A, t, loss, lam, x, 1.0, [(TOPK, 1)], 0.0)
    xd = torch.from_numpy(x).cuda()
    out = torch.zeros(n, d, device="cuda:0")
    f = eng.gradient(xd, out, want_loss=True)
    prob = oracle_problem(A, t, loss, lam)
    want = O.all_gradients(prob, x)
    got = out.cpu().numpy()
    for i in range(n):
        assert relerr(got[i], want[i]) <= 1e-5, (i, relerr(got[i], want[i]))
    assert abs(f - O.global_loss(prob, x)) <= 1e-6 * abs(O.global_loss(prob, x))
    # the state after init holds the same gradients (g0_mode 1: G = grad)
    assert relerr(eng.get_state("grad").cpu().numpy(), want) <= 1e-5
    assert np.array_equal(eng.get_state("G").cpu().numpy(), eng.get_state("grad").cpu().numpy())


def push_state(eng, torch, st):
    for k_gpu, k_or in (("x", "x"), ("G", "G"), ("grad", "X"), ("gt", "gt"), ("gm", "gm")):
        eng.set_state(k_gpu, torch.from_numpy(np.ascontiguousarray(st[k_or])))


def lockstep(torch, A, t, loss, lam, gamma, wc, wz, mc, mz, T, g0_mode=1):
    n, m, d = A.shape
    x0 = np.zeros(d, F32)
    prob = oracle_problem(A, t, loss, lam)
    st = O.init_state(prob, x0, wc, g0_mode)
    eng = make_engine(torch, A, t, loss, lam, x0, gamma, wc, wz, mc, mz, g0_mode)
    # init parity: same estimators up to the gradient tolerance
    assert relerr(eng.get_state("G").cpu().numpy(), st["G"]) <= 1e-5 or g0_mode != 1
    levels_seen = set()
    for it in range(T):
        push_state(eng, torch, st)
        before = {k: np.copy(v) for k, v in st.items() if isinstance(v, np.ndarray)}
        recs, levels = eng.step(1, report=True)
        O.step(st, prob, gamma, wc, wz, mc, mz)
        gx = eng.get_state("x").cpu().numpy()
        ggrad = eng.get_state("grad").cpu().numpy()
        assert np.array_equal(gx.view(np.uint32), st["x"].view(np.uint32)), it       # same two roundings
        assert relerr(ggrad, st["X"]) <= 1e-5, (it, relerr(ggrad, st["X"]))
        assert np.abs(ggrad - st["X"]).max() <= 1e-5 * np.abs(st["X"]).max()
        f_ref = O.global_loss(prob, st["x"])
        assert abs(recs[0]["loss"] - f_ref) <= 1e-5 * abs(f_ref)
        # selections: run the oracle's compressor on the GPU's own gradients
        G_ref, res = O.compress_rows(ggrad, before["G"], before["X"], wc, wz)
        assert levels[0] == [r["level"] for r in res], it
        assert recs[0]["bits_up"] == sum(r["bits"] for r in res)
        gG = eng.get_state("G").cpu().numpy()
        assert np.array_equal(gG.view(np.uint32), G_ref.view(np.uint32)), it
        gt_ref = O.server_mean(G_ref)
        assert np.array_equal(eng.get_state("gt").cpu().numpy().view(np.uint32), gt_ref.view(np.uint32))
        mres = O.adacgd(before["gm"], before["gt"], gt_ref, list(mc), mz)
        assert np.array_equal(eng.get_state("gm").cpu().numpy().view(np.uint32), mres["out"].view(np.uint32)), it
        assert recs[0]["master_level"] == mres["level"] and recs[0]["bits_down"] == mres["bits"]
        levels_seen.update(levels[0])
    return levels_seen


def test_lockstep_c1_shape(torch):
    # workload c1: n=4, d=1000, m=100, logistic + non-convex regulariser, Top-K {10,50,100,500}
    W = S.WORKLOADS["c1"]
    A, t = S.logistic_problem(W["n"], W["d"], W["m"], seed=0)
    gamma = 0.5 / S.smoothness_estimate(A, W["loss"], W["lam"])
    seen = lockstep(torch, A, t, W["loss"], W["lam"], gamma, W["worker"], 1.0, [], 0.0, T=40)
    assert len(seen) >= 2


def test_lockstep_bidirectional_small_c2_shape(torch):
    A, t = S.logistic_problem(5, 800, 200, seed=1)
    gamma = 0.5 / S.smoothness_estimate(A, 0, 0.1)
    cands = [(TOPK, 1), (TOPK, 8), (TOPK, 80), (TOPK, 800)]
    lockstep(torch, A, t, 0, 0.1, gamma, cands, 1.0, cands, 1.0, T=25)


def test_lockstep_least_squares_and_quantisers(torch):
    A, t, _ = S.least_squares_problem(4, 3000, 64, seed=2)
    gamma = 0.5 / S.smoothness_estimate(A, 2, 0.0)
    lockstep(torch, A, t, 2, 0.0, gamma, [(TOPK, 3), (QUANT, 2), (TOPK, 300), (QUANT, 8)], 0.5,
             [(QUANT, 4), (TOPK, 1500)], 0.25, T=15, g0_mode=0)
    lockstep(torch, A, t, 2, 0.0, gamma, [(TOPK, 30), (TOPK, 300)], 2.0, [], 0.0, T=10, g0_mode=2)


def free_run(torch, A, t, loss, lam, gamma, wc, wz, mc, mz, T, wide=False):
    n, m, d = A.shape
    x0 = np.zeros(d, F32)
    prob = oracle_problem(A, t, loss, lam)
    if wide:   # long runs: the oracle's binary64 copy of the features is made once instead of at every product
        prob["A"] = [a.astype(np.float64) for a in prob["A"]]
    st = O.init_state(prob, x0, wc)
    eng = make_engine(torch, A, t, loss, lam, x0, gamma, wc, wz, mc, mz)
    recs, levels = eng.step(T, report=True)
    for it in range(T):
        O.step(st, prob, gamma, wc, wz, mc, mz)
    return recs, levels, O.global_loss(prob, st["x"]), O.global_loss(prob, x0), st, eng


def test_free_running_c1_loss_trajectory(torch):
    W = S.WORKLOADS["c1"]
    A, t = S.logistic_problem(W["n"], W["d"], W["m"], seed=0)
    gamma = 0.5 / S.smoothness_estimate(A, W["loss"], W["lam"])
    recs, levels, f_ref, f0, st, eng = free_run(torch, A, t, W["loss"], W["lam"], gamma, W["worker"], 1.0, [], 0.0,
                                                W["iters"])
    assert abs(recs[-1]["loss"] - f_ref) <= 1e-3 * abs(f_ref)
    assert f_ref < 0.9 * f0                                      # the run makes progress
    assert eng.get_state("step") == W["iters"]
    assert eng.get_state("bits_up") == sum(r["bits_up"] for r in recs)
    assert eng.get_state("bits_down") == sum(r["bits_down"] for r in recs)
    assert relerr(eng.get_state("x").cpu().numpy(), st["x"]) <= 1e-2


def test_step_records_do_not_depend_on_how_steps_are_batched(torch):
    # The record of an iteration is written by the next iteration's first kernel, or by a closing kernel at the end of a
    # batch: one call of 300 steps (more than the 256 records the device holds, replayed as graphs of two), 300 calls of
    # one step, and calls of 1, 2, 3, ... steps must give the same records, levels, counters and state, bit for bit.
    W = S.WORKLOADS["c1"]
    A, t = S.logistic_problem(W["n"], W["d"], W["m"], seed=5)
    gamma = 0.5 / S.smoothness_estimate(A, W["loss"], W["lam"])
    x0 = np.zeros(W["d"], F32)
    T = 300
    runs = []
    for plan in ([T], [1] * T, list(range(1, 24)) + [T - sum(range(1, 24))]):
        assert sum(plan) == T
        eng = make_engine(torch, A, t, W["loss"], W["lam"], x0, gamma, W["worker"], 1.0)
        recs, levels = [], []
        for k in plan:
            r, l = eng.step(k, report=True)
            recs += r
            levels += l
        runs.append((recs, levels, eng.get_state("step"), eng.get_state("bits_up"), eng.get_state("x").cpu().numpy()))
        eng.close()
    ref = runs[0]
    assert ref[2] == T and len(ref[0]) == T
    assert len({r["loss"] for r in ref[0]}) > T // 2             # the records are those of different iterations
    for other in runs[1:]:
        assert other[0] == ref[0] and other[1] == ref[1]
        assert other[2] == ref[2] and other[3] == ref[3]
        assert np.array_equal(other[4].view(np.uint32), ref[4].view(np.uint32))


def test_free_running_c2_bidirectional(torch):
    # workload c2 as benchmarked (20 x 8 000, 2 000 samples per worker, worker and master Top-K {8, 80, 800, 8000}),
    # both sides left to run on their own for as many of its 1 000 iterations as the oracle does in about two minutes
    W = S.WORKLOADS["c2"]
    A, t = S.logistic_problem(W["n"], W["d"], W["m"], seed=0)
    gamma = 0.5 / S.smoothness_estimate(A, W["loss"], W["lam"], iters=8)
    T = 400
    recs, levels, f_ref, f0, st, eng = free_run(torch, A, t, W["loss"], W["lam"], gamma, W["worker"], 1.0, W["master"], 1.0,
                                                T, wide=True)
    assert abs(recs[-1]["loss"] - f_ref) <= 1e-3 * abs(f_ref)
    assert f_ref < 0.9 * f0
    assert eng.get_state("step") == T
    assert len({l for lv in levels for l in lv}) >= 2 and len({r["master_level"] for r in recs}) >= 2


def test_free_running_c4_shape_scaled(torch):
    # the shape of workload c4 (least squares, A ~ N(0, 1/d), Top-K {0.1 %, 1 %, 10 %}) at 8 x 100 000 with 64 samples
    # per worker: large enough for the sampled single-pass pipeline
    n, d, m = 8, 100_000, 64
    A, t, _ = S.least_squares_problem(n, d, m, seed=5)
    gamma = 0.5 / S.smoothness_estimate(A, 2, 0.0, iters=8)
    wc = [(TOPK, 100), (TOPK, 1000), (TOPK, 10_000)]
    # n m < d: the minimum of the objective is zero and the loss falls by a factor of about 0.7 per iteration, so
    # the run is compared where the loss is still far above the resolution of binary32 gradients
    T = 12
    recs, levels, f_ref, f0, st, eng = free_run(torch, A, t, 2, 0.0, gamma, wc, 1.0, [], 0.0, T, wide=True)
    assert abs(recs[-1]["loss"] - f_ref) <= 1e-3 * abs(f_ref)
    assert f_ref < 0.1 * f0
    assert eng.get_state("fallbacks") == 0


def test_free_running_gd_special_case_matches_closed_form(torch):
    # Top-d, zeta = 0, identity master: plain gradient descent (Eq. 2)
    A, t, _ = S.least_squares_problem(3, 64, 40, seed=3)
    n, m, d = A.shape
    H = sum(A[i].astype(np.float64).T @ A[i].astype(np.float64) for i in range(n)) / (n * m)
    c = sum(A[i].astype(np.float64).T @ t[i].astype(np.float64) for i in range(n)) / (n * m)
    x_star = np.linalg.solve(H, c)
    gamma = 1.0 / np.linalg.eigvalsh(H).max()
    T = 50
    eng = make_engine(torch, A, t, 2, 0.0, np.ones(d, F32), gamma, [(TOPK, d)], 0.0)
    recs, levels = eng.step(T, report=True)
    want = x_star + np.linalg.matrix_power(np.eye(d) - np.float64(F32(gamma)) * H, T) @ (np.ones(d) - x_star)
    assert np.allclose(eng.get_state("x").cpu().numpy(), want, rtol=0, atol=5e-5 * np.abs(want).max())
    losses = [r["loss"] for r in recs]
    assert all(b <= a * (1 + 1e-6) for a, b in zip(losses, losses[1:]))
    assert all(lv == [1] * n for lv in levels)


def test_state_roundtrip_and_errors(torch):
    import paper_2211_00188_b200 as pkg
    A, t = S.logistic_problem(2, 100, 10, seed=4)
    eng = make_engine(torch, A, t, 0, 0.1, np.zeros(100, F32), 0.1, [(TOPK, 5)], 1.0)
    x = torch.arange(100, dtype=torch.float32)
    eng.set_state("x", x)
    assert torch.equal(eng.get_state("x").cpu(), x)
    G = torch.randn(2, 100)
    eng.set_state("G", G)
    assert torch.equal(eng.get_state("G").cpu(), G)
    eng.set_state("step", 41)
    eng.step(1)
    assert eng.get_state("step") == 42
    with pytest.raises(pkg.AdacgdError):
        eng.set_state("x", torch.zeros(99))
    with pytest.raises(pkg.AdacgdError):
        pkg.AdaCGD(2, 100, [(TOPK, 5)], 1.0, loss=0, lam=0.1, A=torch.zeros(2, 10, 100, device="cuda"),
                   target=torch.zeros(2, 10, device="cuda"), x0=torch.zeros(100, device="cuda"), gamma=-1.0)


# ---------------------------------------------------------------- sparse features (workload c3 shape)
def make_sparse(torch, n, d, m, density, seed, wc, wz, mc=(), mz=0.0, lam=1e-3, gamma=1.0, g0_mode=1):
    import scipy.sparse as sp
    import paper_2211_00188_b200 as pkg
    rowptr, col, val, y = S.sparse_logistic_problem(n, d, m, density=density, seed=seed)
    grp, gcol, gval = S.csr_global(rowptr, col, val)
    dev = torch.device("cuda:0")
    csr = tuple(torch.from_numpy(a).to(dev) for a in (grp, gcol, gval))
    x0 = np.zeros(d, F32)
    eng = pkg.AdaCGD(n, d, wc, wz, mc, mz, loss=1, lam=lam, csr=csr, target=torch.from_numpy(y).to(dev),
                     x0=torch.from_numpy(x0).to(dev), gamma=gamma, g0_mode=g0_mode)
    A = [sp.csr_matrix((val[i], col[i], rowptr[i]), shape=(m, d)) for i in range(n)]
    prob = dict(A=A, target=[y[i] for i in range(n)], loss=1, lam=lam)
    return eng, prob, x0


def test_sparse_gradient_and_loss(torch):
    n, d, m = 5, 3000, 40
    eng, prob, x0 = make_sparse(torch, n, d, m, 0.01, 7, [(TOPK, 1)], 0.0)
    x = (0.5 * np.random.Generator(np.random.PCG64(2)).standard_normal(d)).astype(F32)
    out = torch.zeros(n, d, device="cuda:0")
    f = eng.gradient(torch.from_numpy(x).cuda(), out, want_loss=True)
    want = O.all_gradients(prob, x)
    got = out.cpu().numpy()
    for i in range(n):
        assert relerr(got[i], want[i]) <= 1e-5
    assert abs(f - O.global_loss(prob, x)) <= 1e-6 * abs(O.global_loss(prob, x))


def sparse_engine_and_oracle(torch, rowptr, col, val, y, d, lam=1e-3):
    import scipy.sparse as sp
    import paper_2211_00188_b200 as pkg
    n, m = y.shape
    dev = torch.device("cuda:0")
    csr = tuple(torch.from_numpy(a).to(dev) for a in S.csr_global(rowptr, col, val))
    eng = pkg.AdaCGD(n, d, [(TOPK, 1)], 0.0, loss=1, lam=lam, csr=csr, target=torch.from_numpy(y).to(dev),
                     x0=torch.zeros(d, device=dev), gamma=1.0)
    A = [sp.csr_matrix((val[i], col[i], rowptr[i]), shape=(m, d)) for i in range(n)]
    return eng, dict(A=A, target=[y[i] for i in range(n)], loss=1, lam=lam)


@pytest.mark.parametrize("shape", ["two_column_blocks", "three_column_blocks_ragged", "long_columns", "many_samples", "dense", "very_wide"])
def test_sparse_gradient_kernel_routes(torch, shape):
    # the routes of the sparse gradient pair: forward with x cut into several shared-memory blocks (d above 49 152),
    # backward spans that do not fit a CTA's buffer (a few columns stored in every row), more samples per worker than
    # the backward kernel keeps residuals for (plain kernels), and columns too long on average for spans at all
    if shape == "two_column_blocks":
        n, d, m = 2, 60_000, 24
        data = S.sparse_logistic_problem(n, d, m, density=0.01, seed=61)
    elif shape == "three_column_blocks_ragged":
        n, d, m = 3, 100_003, 9
        data = S.sparse_logistic_problem(n, d, m, density=0.002, seed=62)
    elif shape == "long_columns":
        n, d, m = 2, 50_000, 300
        data = S.sparse_problem_with_dense_columns(n, d, m, dense_cols=64, extra=16, seed=63)
    elif shape == "many_samples":
        n, d, m = 2, 2_000, 9_000
        data = S.sparse_logistic_problem(n, d, m, density=0.005, seed=64)
    elif shape == "very_wide":
        n, d, m = 2, 400_000, 6      # more column blocks than the blocked forward kernel takes: one warp per row
        data = S.sparse_logistic_problem(n, d, m, density=1e-4, seed=67)
    else:
        n, d, m = 2, 300, 400
        data = S.sparse_logistic_problem(n, d, m, density=0.3, seed=65)
    rowptr, col, val, y = data
    eng, prob = sparse_engine_and_oracle(torch, rowptr, col, val, y, d)
    x = (0.5 * np.random.Generator(np.random.PCG64(66)).standard_normal(d)).astype(F32)
    out = torch.zeros(n, d, device="cuda:0")
    f = eng.gradient(torch.from_numpy(x).cuda(), out, want_loss=True)
    want = O.all_gradients(prob, x)
    got = out.cpu().numpy()
    for i in range(n):
        assert relerr(got[i], want[i]) <= 1e-5, (i, relerr(got[i], want[i]))
        assert np.abs(got[i] - want[i]).max() <= 1e-5 * np.abs(want[i]).max()
    assert abs(f - O.global_loss(prob, x)) <= 1e-6 * abs(O.global_loss(prob, x))


def test_sparse_lockstep_mixed_candidates(torch):
    # the candidate mix of workload c3 (Top-K and 2/4/8-bit quantisers in the user's order), scaled down
    n, d, m = 6, 4000, 50
    wc = [(TOPK, 4), (TOPK, 40), (QUANT, 2), (QUANT, 4), (TOPK, 400), (QUANT, 8)]
    eng, prob, x0 = make_sparse(torch, n, d, m, 0.01, 8, wc, 1.0, gamma=2.0)
    st = O.init_state(prob, x0, wc)
    seen = set()
    for it in range(12):
        push_state(eng, torch, st)
        before = {k: np.copy(v) for k, v in st.items() if isinstance(v, np.ndarray)}
        recs, levels = eng.step(1, report=True)
        O.step(st, prob, 2.0, wc, 1.0)
        ggrad = eng.get_state("grad").cpu().numpy()
        assert relerr(ggrad, st["X"]) <= 1e-5
        G_ref, res = O.compress_rows(ggrad, before["G"], before["X"], wc, 1.0)
        assert levels[0] == [r["level"] for r in res], it
        assert np.array_equal(eng.get_state("G").cpu().numpy().view(np.uint32), G_ref.view(np.uint32)), it
        assert np.array_equal(eng.get_state("gt").cpu().numpy().view(np.uint32), O.server_mean(G_ref).view(np.uint32))
        seen.update(levels[0])
    assert len(seen) >= 2


def test_free_running_c3_shape_scaled(torch):
    # the shape of workload c3 (CSR 1 %, logistic + l2, Top-K and 2/4/8-bit quantisers mixed) at 10 x 20 000 with 100
    # samples per worker, both sides left to run on their own
    n, d, m = 10, 20_000, 100
    wc = [(TOPK, 20), (TOPK, 200), (QUANT, 2), (QUANT, 4), (TOPK, 2000), (QUANT, 8)]
    gamma = 0.5 / (0.25 + 1e-3)
    eng, prob, x0 = make_sparse(torch, n, d, m, 0.01, 11, wc, 1.0, gamma=gamma)
    st = O.init_state(prob, x0, wc)
    T = 100
    recs, levels = eng.step(T, report=True)
    for it in range(T):
        O.step(st, prob, gamma, wc, 1.0)
    f_ref, f0 = O.global_loss(prob, st["x"]), O.global_loss(prob, x0)
    assert abs(recs[-1]["loss"] - f_ref) <= 1e-3 * abs(f_ref)
    assert f_ref < 0.96 * f0
    assert len({l for lv in levels for l in lv}) >= 2


def test_lockstep_random_sweep(torch):
    # seeded sweep over whole iterations: the three objectives, worker and master lists with Top-K and quantisers,
    # the three initialisations, several triggers and shapes (short rows and the mid-size route)
    rng = np.random.Generator(np.random.PCG64(123))
    for case in range(6):
        n = int(rng.integers(2, 6))
        d = int(rng.choice([257, 1000, 4096, 40_000]))
        m = int(rng.choice([16, 40]))
        loss = case % 3
        if loss == 2:
            A, t, _ = S.least_squares_problem(n, d, m, seed=200 + case)
        else:
            A, t = S.logistic_problem(n, d, m, seed=200 + case)
        lam = 0.0 if loss == 2 else (0.1 if loss == 0 else 1e-3)
        gamma = 0.5 / S.smoothness_estimate(A, loss, lam)

        def cands():
            ks = sorted(set(int(k) for k in (d * np.array([1e-3, 1e-2, 0.1, 1.0]) * rng.uniform(0.5, 1.2, 4))))
            ks = [k for i, k in enumerate(ks) if k > 0 and (i == 0 or ks[i - 1] < d)][:int(rng.integers(1, 5))]
            c = [(TOPK, k) for k in ks]
            if rng.random() < 0.5:
                c.insert(int(rng.integers(0, len(c) + 1)), (QUANT, int(rng.integers(2, 9))))
            return c

        wc = cands()
        mc = cands() if case % 2 == 0 else []
        lockstep(torch, A, t, loss, lam, gamma, wc, float(rng.choice([0.0, 0.5, 1.0, 2.0])), mc,
                 float(rng.choice([0.25, 1.0])), T=int(rng.integers(4, 9)), g0_mode=case % 3)


def test_sparse_lockstep_random_sweep(torch):
    # seeded sweep over CSR problems: densities, row lengths on both sides of the short-row limit, empty columns,
    # master compression on and off
    rng = np.random.Generator(np.random.PCG64(321))
    for case in range(5):
        n = int(rng.integers(2, 6))
        d = int(rng.choice([999, 5000, 40_000]))
        m = int(rng.choice([7, 33]))
        density = float(rng.choice([0.002, 0.01, 0.05]))
        ks = sorted(set(int(k) for k in (d * np.array([1e-3, 1e-2, 0.2]) * rng.uniform(0.5, 1.5, 3))))
        wc = [(TOPK, k) for k in ks if 0 < k < d]
        if case % 2 == 0:
            wc.insert(int(rng.integers(0, len(wc) + 1)), (QUANT, int(rng.integers(2, 9))))
        mc = [(TOPK, max(1, d // 50)), (TOPK, d)] if case % 2 == 1 else []
        wz, mz = float(rng.choice([0.0, 1.0, 3.0])), 0.5
        gamma = float(rng.choice([0.5, 2.0]))
        eng, prob, x0 = make_sparse(torch, n, d, m, density, 300 + case, wc, wz, mc, mz, gamma=gamma)
        st = O.init_state(prob, x0, wc)
        for it in range(5):
            push_state(eng, torch, st)
            before = {k: np.copy(v) for k, v in st.items() if isinstance(v, np.ndarray)}
            recs, levels = eng.step(1, report=True)
            O.step(st, prob, gamma, wc, wz, mc, mz)
            ggrad = eng.get_state("grad").cpu().numpy()
            assert relerr(ggrad, st["X"]) <= 1e-5, (case, it)
            G_ref, res = O.compress_rows(ggrad, before["G"], before["X"], wc, wz)
            assert levels[0] == [r["level"] for r in res], (case, it)
            assert np.array_equal(eng.get_state("G").cpu().numpy().view(np.uint32), G_ref.view(np.uint32)), (case, it)
            gt_ref = O.server_mean(G_ref)
            assert np.array_equal(eng.get_state("gt").cpu().numpy().view(np.uint32), gt_ref.view(np.uint32))
            mres = O.adacgd(before["gm"], before["gt"], gt_ref, list(mc), mz)
            assert np.array_equal(eng.get_state("gm").cpu().numpy().view(np.uint32), mres["out"].view(np.uint32)), (case, it)
