"""Pins for the CPU oracle: it is checked against what the paper and the
mathematics fix, never against itself or against the CUDA path."""
import itertools
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import adacgd_oracle as O

F32 = np.float32
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


# ---------------------------------------------------------------- exact sums
def test_sumsq_matches_fsum_of_exact_squares():
    # squares of binary32 values are exact in binary64 and math.fsum returns the
    # correctly rounded sum of its binary64 arguments
    r = rng(1)
    for scale in (1.0, 1e-20, 1e18, 1e-38):
        w = (r.standard_normal(4097) * scale).astype(F32)
        want = math.fsum(float(t) * float(t) for t in w)
        assert O.sumsq(w) == want
    mixed = np.array([1e19, 1.0, 1e-19, 3e-39, -1e19, 2.5], dtype=F32)  # incl. a subnormal
    assert O.sumsq(mixed) == math.fsum(float(t) * float(t) for t in mixed)
    assert O.sumsq(np.zeros(0, dtype=F32)) == 0.0


def test_sumsq_is_exact_rational():
    w = np.array([1.5, -2.25, 2.0 ** -149, 2.0 ** -126, 3.0], dtype=F32)
    want = sum(Fraction(float(t)) ** 2 for t in w)
    assert Fraction(O.sumsq_units(w), 2 ** 298) == want


def test_sumsq_rejects_nonfinite():
    with pytest.raises(FloatingPointError):
        O.sumsq(np.array([1.0, np.inf], dtype=F32))


# ------------------------------------------------------------------- Top-K
def brute_force_topk(v, K):
    """Best K-term approximation by enumeration: minimise the exact residual
    energy; among minimisers take the lexicographically smallest index set,
    which is what 'lowest index wins among equal magnitudes' selects."""
    d = len(v)
    sq = [Fraction(float(t)) ** 2 for t in v]
    best = None
    for S in itertools.combinations(range(d), K):
        resid = sum(sq) - sum(sq[i] for i in S)
        cand = (resid, S)
        if best is None or cand < best:
            best = cand
    return list(best[1]), best[0]


def test_topk_exhaustive_small_integers():
    vals = [-2.0, -1.0, -0.0, 0.0, 1.0, 2.0]
    for d in (1, 2, 3, 4):
        for v in itertools.product(vals, repeat=d):
            v = np.array(v, dtype=F32)
            for K in range(1, d + 1):
                kept, resid = brute_force_topk(v, K)
                assert sorted(O.topk_kept(v, K).tolist()) == kept
                assert Fraction(O.candidate_error(v, (O.TOPK, K))) == resid


def test_topk_random_vs_enumeration():
    r = rng(2)
    for trial in range(40):
        d = int(r.integers(5, 10))
        v = r.integers(-3, 4, size=d).astype(F32) if trial % 2 else r.standard_normal(d).astype(F32)
        for K in (1, 2, d // 2, d - 1):
            kept, resid = brute_force_topk(v, K)
            assert sorted(O.topk_kept(v, K).tolist()) == kept
            out = O.topk(v, K)
            assert np.array_equal(out[kept], v[kept]) and np.count_nonzero(out) <= K


def test_topk_vs_python_sort_d64():
    r = rng(3)
    for trial in range(50):
        d = 64
        v = (r.integers(-4, 5, size=d) * (0.5 if trial % 3 else 1.0)).astype(F32)
        order = sorted(range(d), key=lambda i: (-abs(float(v[i])), i))
        for K in (1, 7, 32, 63, 64, 100):
            assert O.topk_kept(v, K).tolist() == order[:K]


def test_topk_contraction_bound_and_monotonicity():
    # Eq. 4 with alpha = K/d: the d-K smallest squares average at most the overall mean
    r = rng(4)
    for d in (10, 257, 4096):
        for law in ("normal", "cauchy", "ties"):
            v = {"normal": r.standard_normal(d), "cauchy": r.standard_cauchy(d),
                 "ties": r.integers(-2, 3, size=d)}[law].astype(F32)
            total = Fraction(O.sumsq(v))
            prev_err, prev_kept = None, set()
            for K in sorted({1, 2, d // 10 + 1, d // 2, d - 1, d}):
                err = Fraction(O.candidate_error(v, (O.TOPK, K)))
                assert err <= (1 - Fraction(K, d)) * total * (1 + Fraction(1, 2 ** 50))
                kept = set(O.topk_kept(v, K).tolist())
                assert prev_kept <= kept and len(kept) == K          # nested
                if prev_err is not None:
                    assert err <= prev_err                            # non-increasing in K
                prev_err, prev_kept = err, kept
            assert O.candidate_error(v, (O.TOPK, d)) == 0.0


def test_golden_topk_ties():
    for case in json.load(open(GOLDEN))["topk_ties"]:
        v = np.array(case["v"], dtype=F32)
        assert sorted(O.topk_kept(v, case["K"]).tolist()) == case["kept"], case


# --------------------------------------------------------------- quantiser
def test_golden_quantize():
    for case in json.load(open(GOLDEN))["quantize"]:
        q = O.quantize(np.array(case["v"], dtype=F32), case["bits"])
        want = np.array(case["q"], dtype=F32)
        assert np.array_equal(q, want) and np.array_equal(np.signbit(q), np.signbit(want)), case


def test_quantize_contraction_idempotence_and_limit():
    r = rng(5)
    for d in (3, 100, 5000):
        v = (r.standard_normal(d) * 10 ** r.uniform(-3, 3)).astype(F32)
        total = O.sumsq(v)
        prev = None
        for b in (2, 3, 4, 8, 12, 16):
            q = O.quantize(v, b)
            err = O.candidate_error(v, (O.QUANT, b))
            assert err <= (1 - 1 / d) * total * (1 + 1e-6)             # Eq. 4 with alpha = 1/d
            assert np.all(np.abs(q) <= np.abs(v).max() * (1 + 1e-6))
            assert np.all((np.sign(q) == np.sign(v)) | (q == 0))
            # re-quantising a grid vector reproduces it (up to one rounding of code*step)
            q2 = O.quantize(q, b)
            assert np.allclose(q2, q, rtol=1e-6, atol=0)
            # at most 2^(b-1)-1 positive levels
            assert len(np.unique(np.abs(q))) <= (1 << (b - 1))
            if prev is not None:
                assert err <= prev * (1 + 1e-6)
            prev = err
        assert prev <= total * 2.0 ** -28        # 16 bits: relative error ~ (2^-16)^2
    assert not O.quantize(np.zeros(7, dtype=F32), 4).any()


# ------------------------------------------------------- 3PC special cases
def random_triplet(r, d, integer=False):
    if integer:
        return tuple(r.integers(-3, 4, size=d).astype(F32) for _ in range(3))
    x = r.standard_normal(d).astype(F32)
    h = (x + 0.5 * r.standard_normal(d)).astype(F32)
    y = (x + 0.3 * r.standard_normal(d)).astype(F32)
    return h, y, x


def test_golden_adacgd_hand_examples():
    for case in json.load(open(GOLDEN))["adacgd"]:
        h, y, x = (np.array(case[k], dtype=F32) for k in ("h", "y", "x"))
        cands = [tuple(c) for c in case["cands"]]
        for z in case["by_zeta"]:
            res = O.adacgd(h, y, x, cands, z["zeta"])
            assert res["D"] == case["D"] and res["err"] == case["err"], case["cite"]
            assert res["level"] == z["level"], (case["cite"], z)
            assert res["out"].tolist() == [float(t) for t in z["out"]]
            assert res["bits"] == z["bits"]
            assert (res["kept"].tolist() if res["kept"] is not None else None) == z["kept"]


def test_golden_message_bit_patterns():
    # Eq. 7 bit for bit, signs of zero included: a Top-K message touches the kept entries only, a quantised one
    # every entry.  Compared as uint32 patterns (== and array_equal do not see the sign of a zero).
    for case in json.load(open(GOLDEN))["message_bit_patterns"]:
        h = np.array([int(b, 16) for b in case["h_bits"]], dtype=np.uint32).view(F32)
        x = np.array([int(b, 16) for b in case["x_bits"]], dtype=np.uint32).view(F32)
        want = np.array([int(b, 16) for b in case["out_bits"]], dtype=np.uint32)
        cand = tuple(case["cand"])
        y = np.zeros_like(x)
        assert O.ef21(h, y, x, cand).view(np.uint32).tolist() == want.tolist(), case["cite"]
        # zeta = 0 with one candidate applies that candidate (x != h): the same update through Eq. 11
        res = O.adacgd(h, y, x, [cand], 0.0)
        assert res["level"] == 1 and res["out"].view(np.uint32).tolist() == want.tolist(), case["cite"]
        # the inputs are untouched
        assert h.view(np.uint32).tolist() == [int(b, 16) for b in case["h_bits"]]


def test_zeta_zero_is_ef21():
    # Section 4.3: zeta = 0 reduces AdaCGD to EF21 (with the last candidate)
    r = rng(6)
    cands = [(O.TOPK, 3), (O.TOPK, 10), (O.TOPK, 40)]
    for _ in range(20):
        h, y, x = random_triplet(r, 100)
        res = O.adacgd(h, y, x, cands, 0.0)
        assert res["level"] == 3
        assert np.array_equal(res["out"], O.ef21(h, y, x, cands[-1]))


def test_single_candidate_is_clag_and_lag():
    # Section 4.3: m = 1 gives CLAG (Eq. 8); CLAG with the identity is LAG
    r = rng(7)
    hits = set()
    for trial in range(60):
        h, y, x = random_triplet(r, 50, integer=(trial % 3 == 0))
        zeta = float(r.choice([0.0, 0.5, 1.0, 3.0, 50.0]))
        res = O.adacgd(h, y, x, [(O.TOPK, 5)], zeta)
        assert np.array_equal(res["out"], O.clag(h, y, x, (O.TOPK, 5), zeta))
        hits.add(res["level"])
        res_id = O.adacgd(h, y, x, [(O.TOPK, 50)], zeta)
        want = O.lag(h, y, x, zeta)
        # h + (x - h) equals x only up to one rounding (the server receives x - h)
        assert np.allclose(res_id["out"], want, rtol=0, atol=2e-6 * np.abs(x).max())
    assert hits == {0, 1}


def test_lemma_adacgd_is_ada3pc():
    # Lemma 1: one LAG compressor followed by the m EF21 compressors, with the
    # skip test and the triggers P_1..P_{m-1} as predicates, reproduces AdaCGD
    r = rng(8)
    cands = [(O.TOPK, 2), (O.QUANT, 3), (O.TOPK, 20), (O.TOPK, 64)]
    levels = set()
    for trial in range(80):
        h, y, x = random_triplet(r, 64, integer=(trial % 4 == 0))
        zeta = float(r.choice([0.0, 0.1, 0.5, 1.0, 2.0, 10.0]))

        def rhs(h, y, x):
            return float(F32(zeta)) * O.sumsq((x - y).astype(F32))

        comps = [lambda h, y, x: O.lag(h, y, x, zeta)] + \
                [lambda h, y, x, c=c: O.ef21(h, y, x, c) for c in cands]
        preds = [lambda h, y, x: O.sumsq((x - h).astype(F32)) <= rhs(h, y, x)] + \
                [lambda h, y, x, c=c: O.candidate_error((x - h).astype(F32), c) <= rhs(h, y, x)
                 for c in cands[:-1]]
        res = O.adacgd(h, y, x, cands, zeta)
        assert np.array_equal(res["out"], O.ada3pc(h, y, x, comps, preds))
        levels.add(res["level"])
    assert len(levels) >= 4


def test_golden_adaptive_3pc_menu():
    for case in json.load(open(GOLDEN))["adaptive_3pc"]:
        h, y, x = (np.array(case[k], dtype=F32) for k in ("h", "y", "x"))
        cands = [tuple(c) for c in case["cands"]]
        for z in case["cases"]:
            res = O.adaptive_3pc(h, y, x, cands, [tuple(q) for q in z["preds"]])
            assert res["level"] == z["level"], z
            assert res["out"].tolist() == [float(t) for t in z["out"]], z


def test_adaptive_3pc_menu_is_definition_3_and_contains_adacgd():
    # (a) the menu version against Definition 3 written with callables (`ada3pc`), the compressors being "keep h" and
    # separately composed EF21 steps; (b) Eq. 10 at every level is AdaCGD (Eq. 11); (c) no skipping and one candidate
    # is EF21 (Eq. 7); (d) a trigger that always holds at level j stops there
    r = rng(21)
    for trial in range(30):
        d = int(r.integers(3, 40))
        h, y, x = random_triplet(r, d, integer=(trial % 3 == 0))
        ks = sorted(set(int(k) for k in r.integers(1, d + 1, size=3)))
        cands = [(O.TOPK, k) for k in ks]
        if trial % 2:
            cands.insert(int(r.integers(0, len(cands) + 1)), (O.QUANT, int(r.integers(2, 6))))
        m = len(cands)
        scale = O.sumsq((x - h).astype(F32))
        preds = []
        for j in range(m):
            kind = int(r.integers(0, 5))
            param = float(r.choice([0.0, 0.1, 0.5, 1.0, 2.0])) * (scale if kind == O.PRED_ABSOLUTE else 1.0)
            preds.append((kind, param))
        res = O.adaptive_3pc(h, y, x, cands, preds)
        # (a)
        comps = [lambda h_, y_, x_: h_.copy()] + [(lambda c: (lambda h_, y_, x_: O.ef21(h_, y_, x_, c)))(c) for c in cands]

        def make_pred(j):
            def P(h_, y_, x_):   # the level's error on the difference vector: x - (h + C(x - h)) = v - C(v)
                v_ = (x_ - h_).astype(F32)
                return O.trigger_holds(preds[j], O.sumsq(v_) if j == 0 else O.candidate_error(v_, cands[j - 1]), h_, y_, x_)
            return P
        want = O.ada3pc(h, y, x, comps, [make_pred(j) for j in range(m)])
        assert np.array_equal(res["out"].view(np.uint32), want.view(np.uint32)), (trial, preds)
        # (b)
        for zeta in (0.0, 0.5, 2.0):
            a = O.adacgd(h, y, x, cands, zeta)
            b = O.adaptive_3pc(h, y, x, cands, [(O.PRED_LAZY, zeta)] * m)
            assert a["level"] == b["level"] and np.array_equal(a["out"].view(np.uint32), b["out"].view(np.uint32))
        # (c)
        e = O.adaptive_3pc(h, y, x, cands[:1], [(O.PRED_NEVER, 0.0)])
        assert e["level"] == 1 and np.array_equal(e["out"].view(np.uint32), O.ef21(h, y, x, cands[0]).view(np.uint32))
        # (d)
        j = int(r.integers(0, m))
        stop = O.adaptive_3pc(h, y, x, cands, [(O.PRED_NEVER, 0.0)] * j + [(O.PRED_ALWAYS, 0.0)] * (m - j))
        assert stop["level"] == j


def test_trigger_postcondition_and_monotone_in_zeta():
    r = rng(9)
    cands = [(O.TOPK, 1), (O.TOPK, 8), (O.QUANT, 4), (O.TOPK, 100)]
    for _ in range(30):
        h, y, x = random_triplet(r, 200)
        last = None
        for zeta in (0.0, 0.05, 0.3, 1.0, 3.0, 1e6):
            res = O.adacgd(h, y, x, cands, zeta)
            j, bound = res["level"], float(F32(zeta)) * res["D"]
            assert all(res["err"][i] > bound for i in range(j))          # smallest index (Eq. 9)
            if j < len(cands):
                assert res["err"][j] <= bound
                # the error actually committed, measured on the stored estimator
                assert O.sumsq((x - res["out"]).astype(F32)) <= bound * (1 + 1e-5)
            if last is not None:
                assert j <= last                                          # larger zeta, stronger compression
            last = j
        assert last == 0


def test_message_bits_formula():
    assert O.message_bits((O.TOPK, 10), 1000) == 10 * (32 + 10)
    assert O.message_bits((O.TOPK, 1000), 1000) == 32000
    assert O.message_bits((O.TOPK, 5), 1024) == 5 * 42 and O.message_bits((O.TOPK, 5), 1025) == 5 * 43
    assert O.message_bits((O.QUANT, 4), 1000) == 32 + 4000


# ----------------------------------------------------------------- objectives
@pytest.mark.parametrize("loss,lam", [(O.LOGISTIC_NCVX, 0.1), (O.LOGISTIC_L2, 0.05), (O.LEAST_SQUARES, 0.0)])
def test_gradient_matches_central_differences(loss, lam):
    r = rng(10 + loss)
    m, d = 30, 12
    A = r.standard_normal((m, d)).astype(F32)
    t = (np.sign(r.standard_normal(m)) if loss != O.LEAST_SQUARES else r.standard_normal(m)).astype(F32)
    x = r.standard_normal(d).astype(F32)
    g = O.local_gradient(A, t, x, loss, lam).astype(np.float64)
    eps = 1e-6
    for j in range(d):
        e = np.zeros(d)
        e[j] = eps
        fd = (O.local_loss(A, t, x.astype(np.float64) + e, loss, lam)
              - O.local_loss(A, t, x.astype(np.float64) - e, loss, lam)) / (2 * eps)
        assert abs(fd - g[j]) <= 1e-6 * max(1.0, abs(fd)) + 2e-7


def test_logistic_loss_closed_form_values():
    # at x = 0 every sample contributes log 2 and the regulariser vanishes
    A = rng(11).standard_normal((7, 5)).astype(F32)
    y = np.array([1, -1, 1, 1, -1, -1, 1], dtype=F32)
    assert abs(O.local_loss(A, y, np.zeros(5, F32), O.LOGISTIC_NCVX, 0.1) - math.log(2)) < 1e-15
    # gradient at 0: -(1/m) sum y_l a_l / 2
    g0 = O.local_gradient(A, y, np.zeros(5, F32), O.LOGISTIC_NCVX, 0.1)
    want = -(A.astype(np.float64) * y[:, None]).sum(0) / (2 * 7)
    assert np.allclose(g0, want, rtol=1e-6, atol=1e-7)
    # one sample, one feature: f = log(1+exp(-y a x)) + lam x^2/(1+x^2)
    a, yy, xx, lam = 0.75, -1.0, 1.5, 0.1
    f = O.local_loss(np.array([[a]], F32), np.array([yy], F32), np.array([xx], F32), O.LOGISTIC_NCVX, lam)
    assert abs(f - (math.log1p(math.exp(-yy * a * xx)) + lam * xx * xx / (1 + xx * xx))) < 1e-12


def test_sparse_and_dense_gradients_agree():
    import scipy.sparse as sp
    r = rng(12)
    dense = (r.random((20, 40)) * (r.random((20, 40)) < 0.2)).astype(F32)
    y = np.sign(r.standard_normal(20)).astype(F32)
    x = r.standard_normal(40).astype(F32)
    gd = O.local_gradient(dense, y, x, O.LOGISTIC_L2, 1e-3)
    gs = O.local_gradient(sp.csr_matrix(dense), y, x, O.LOGISTIC_L2, 1e-3)
    assert np.array_equal(gd, gs) or np.allclose(gd, gs, rtol=1e-6, atol=1e-9)


def small_lsq(seed=13, n=3, m=12, d=6):
    r = rng(seed)
    A = [r.standard_normal((m, d)).astype(F32) for _ in range(n)]
    xs = r.standard_normal(d)
    b = [(a.astype(np.float64) @ xs + 0.1 * r.standard_normal(m)).astype(F32) for a in A]
    prob = dict(A=A, target=b, loss=O.LEAST_SQUARES, lam=0.0)
    H = sum(a.astype(np.float64).T @ a.astype(np.float64) for a in A) / (n * m)
    c = sum(a.astype(np.float64).T @ bb.astype(np.float64) for a, bb in zip(A, b)) / (n * m)
    return prob, H, c


def test_server_mean_definition():
    G = rng(14).standard_normal((7, 33)).astype(F32)
    assert np.allclose(O.server_mean(G), G.astype(np.float64).mean(0), rtol=1e-6, atol=1e-7)
    assert np.array_equal(O.server_mean(G[:1]), G[0])
    two = np.array([[1.0, 3.0], [2.0, 5.0]], dtype=F32)
    assert O.server_mean(two).tolist() == [1.5, 4.0]


def test_identity_everything_is_gradient_descent_closed_form():
    # Top-d workers, zeta = 0, identity master: Algorithm 1 is plain GD (Eq. 2), whose
    # iterates on a quadratic are x^T - x* = (I - gamma H)^T (x^0 - x*)
    prob, H, c = small_lsq()
    d = H.shape[0]
    x_star = np.linalg.solve(H, c)
    L = np.linalg.eigvalsh(H).max()
    gamma = 1.0 / L
    x0 = np.ones(d, dtype=F32)
    st = O.init_state(prob, x0)
    cands = [(O.TOPK, d)]
    T = 25
    losses = [O.global_loss(prob, st["x"])]
    for _ in range(T):
        rep = O.step(st, prob, gamma, cands, 0.0)
        assert rep["levels"] == [1] * 3
        losses.append(O.global_loss(prob, st["x"]))
    want = x_star + np.linalg.matrix_power(np.eye(d) - gamma * H, T) @ (x0.astype(np.float64) - x_star)
    assert np.allclose(st["x"], want, rtol=0, atol=2e-5 * np.abs(want).max())
    assert all(b <= a + 1e-12 for a, b in zip(losses, losses[1:]))       # monotone descent, gamma <= 1/L
    assert st["step"] == T and st["bits_up"] == T * 3 * 32 * d


def test_compressed_run_converges_to_closed_form_optimum():
    # EF21-type estimators converge to the exact gradients on a strongly convex
    # quadratic, so the iterates reach the closed-form minimiser
    prob, H, c = small_lsq(seed=15, n=4, m=20, d=8)
    x_star = np.linalg.solve(H, c)
    L = np.linalg.eigvalsh(H).max()
    st = O.init_state(prob, np.zeros(8, dtype=F32))
    cands = [(O.TOPK, 1), (O.TOPK, 2), (O.TOPK, 4)]
    f0 = O.global_loss(prob, st["x"])
    seen = set()
    for _ in range(600):
        rep = O.step(st, prob, 0.25 / L, cands, 1.0, master_cands=[(O.TOPK, 2), (O.TOPK, 8)], master_zeta=0.5)
        seen.update(rep["levels"])
    f_star = O.global_loss(prob, x_star)
    assert O.global_loss(prob, st["x"]) - f_star <= 1e-6 * (f0 - f_star)
    assert np.allclose(st["x"], x_star, atol=1e-3)
    assert len(seen) >= 2
    # the server mean invariant of Algorithm 1: g~ is the mean of the g~_i
    assert np.array_equal(st["gt"], O.server_mean(st["G"]))


def test_alg2_three_point_arguments():
    # worker: h = g~_i^t, y = grad f_i(x^t), x = grad f_i(x^{t+1}); master: h = g^t, y = g~^t
    prob, H, c = small_lsq(seed=16)
    st = O.init_state(prob, np.full(6, 0.5, dtype=F32), g0_mode=0)
    wc, mc = [(O.TOPK, 1), (O.TOPK, 3)], [(O.TOPK, 2), (O.TOPK, 6)]
    for _ in range(5):
        before = {k: np.copy(v) for k, v in st.items() if isinstance(v, np.ndarray)}
        rep = O.step(st, prob, 0.1, wc, 0.7, mc, 0.3)
        x_new = (before["x"] - (F32(0.1) * before["gm"]).astype(F32)).astype(F32)
        assert np.array_equal(st["x"], x_new)
        grads = O.all_gradients(prob, x_new)
        for i in range(3):
            want = O.adacgd(before["G"][i], before["X"][i], grads[i], wc, 0.7)
            assert np.array_equal(st["G"][i], want["out"]) and rep["levels"][i] == want["level"]
        gt = O.server_mean(st["G"])
        want_m = O.adacgd(before["gm"], before["gt"], gt, mc, 0.3)
        assert np.array_equal(st["gm"], want_m["out"]) and np.array_equal(st["gt"], gt)
