"""The comparison protocol (Section 6, Appendix C): candidate lists of the five methods, the
communication-budget stopping rule and the step-size sweep.  Host logic runs on a scripted
stand-in for the engine; the GPU cases run the real engine against the oracle's separately
coded EF21 / LAG / CLAG compressors."""
import numpy as np
import pytest

import synthetic_inputs as S
from oracle import adacgd_oracle as O
from paper_2211_00188_b200 import protocol as P
from paper_2211_00188_b200.binding import TOPK

F32 = np.float32


class ScriptedEngine:
    """Returns scripted per-round bits and losses; records the batch sizes it was asked for."""

    def __init__(self, n, d, worker, bits, losses):
        self.n, self.d, self.worker = n, d, list(worker)
        self.bits, self.losses, self.pos, self.calls = list(bits), list(losses), 0, []

    def step(self, k, report=False):
        assert report
        self.calls.append(k)
        recs = [dict(loss=self.losses[self.pos + i], bits_up=self.bits[self.pos + i]) for i in range(k)]
        levels = [[0] * self.n for _ in range(k)]
        self.pos += k
        return recs, levels


def test_method_sets():
    d = 1000
    assert P.method_set("gd", d) == ([(TOPK, d)], 0.0)
    assert P.method_set("ef21", d) == ([(TOPK, 1)], 0.0)
    assert P.method_set("lag", d, zeta=4.0) == ([(TOPK, d)], 4.0)
    assert P.method_set("clag", d, K=7, zeta=2.0) == ([(TOPK, 7)], 2.0)
    cands, z = P.method_set("adacgd", d, zeta=1.0)
    assert cands == [(TOPK, 1), (TOPK, 10), (TOPK, 100), (TOPK, 500)] and z == 1.0
    assert P.topk_ladder(8, (0.001, 0.01, 0.5)) == [(TOPK, 1), (TOPK, 4)]      # duplicates dropped
    with pytest.raises(ValueError):
        P.method_set("sgd", d)


def test_max_bits_matches_the_oracle_formula():
    for d in (1, 2, 1000, 1024, 1025):
        for cands in ([(TOPK, 1)], [(TOPK, 3), (TOPK, d)], [(TOPK, 5), (1, 4)]):
            want = 3 * max(O.message_bits(c, d) for c in cands)
            assert P.max_bits_per_round(3, d, cands) == want


def test_budget_stops_at_the_round_that_spends_it():
    n, d = 2, 100
    worker = [(TOPK, 10)]
    worst = P.max_bits_per_round(n, d, worker)          # 2 * 10 * (32 + 7) = 780
    assert worst == 780
    bits = [780, 0, 390, 780, 780, 0, 0, 780, 780, 780] + [780] * 50
    eng = ScriptedEngine(n, d, worker, bits, np.linspace(1.0, 0.5, len(bits)))
    rec = P.run_to_budget(eng, 4000, batch=4)
    cum = np.cumsum(bits)
    stop = int(np.argmax(cum >= 4000))                  # first round at or above the budget
    assert len(rec["loss"]) == stop + 1 and rec["bits_up"][-1] == cum[stop] and rec["bits_up"][-2] < 4000
    assert eng.pos == stop + 1                          # the engine did not run past it
    assert max(eng.calls) <= 4 and eng.calls[-1] == 1   # batches far from the budget, single rounds near it
    # a method that never sends anything ends at max_rounds
    eng = ScriptedEngine(n, d, worker, [0] * 40, [1.0] * 40)
    rec = P.run_to_budget(eng, 1000, max_rounds=25, batch=8)
    assert len(rec["loss"]) == 25 and rec["bits_up"][-1] == 0


def test_gamma_sweep_picks_the_lowest_finite_loss():
    finals = {0: 0.9, 1: 0.7, 2: 0.4, 3: float("nan"), 4: float("inf")}

    def make(gamma):
        e = int(round(np.log2(gamma / 0.125)))
        return ScriptedEngine(1, 10, [(TOPK, 1)], [36] * 10, [1.0] * 4 + [finals[e]] * 6)

    res = P.gamma_sweep(make, 0.125, 5 * 36, exponents=range(5))
    assert res["best"] == 2 and set(res["runs"]) == set(range(5))
    assert all(len(r["loss"]) == 5 for r in res["runs"].values())


# ----------------------------------------------------------------------------- GPU
def oracle_round(st, prob, gamma, method, K, zeta):
    """One round with the oracle's separately coded compressor of `method` (not through adacgd())."""
    x = (st["x"] - (F32(gamma) * st["gm"]).astype(F32)).astype(F32)
    X = O.all_gradients(prob, x)
    d = x.size
    new = []
    for i in range(X.shape[0]):
        h, y = st["G"][i], st["X"][i]
        if method == "gd":
            new.append(O.ef21(h, y, X[i], (TOPK, d)))
        elif method == "ef21":
            new.append(O.ef21(h, y, X[i], (TOPK, K)))
        elif method == "lag":
            new.append(O.lag(h, y, X[i], zeta))
        else:
            new.append(O.clag(h, y, X[i], (TOPK, K), zeta))
    G = np.stack(new)
    gt = O.server_mean(G)
    st.update(x=x, Y=st["X"], X=X, G=G, gt=gt, gm=gt.copy())


@pytest.mark.gpu
@pytest.mark.parametrize("method", ["gd", "ef21", "lag", "clag"])
def test_baselines_are_the_engine_with_the_right_list(method):
    """Lock-step over a few rounds: the engine configured by method_set reproduces the oracle's own
    GD / EF21 / LAG / CLAG update (estimators bitwise when fed the same gradients)."""
    import torch
    import paper_2211_00188_b200 as pkg

    n, d, m = 4, 600, 60
    A, t = S.logistic_problem(n, d, m, seed=5)
    lam, loss = 0.1, 0
    gamma = 0.5 / S.smoothness_estimate(A, loss, lam)
    K, zeta = 3, 2.0
    cands, z = P.method_set(method, d, K=K, zeta=zeta)
    prob = dict(A=[A[i] for i in range(n)], target=[t[i] for i in range(n)], loss=loss, lam=lam)
    x0 = np.zeros(d, F32)
    st = O.init_state(prob, x0, cands)
    dev = torch.device("cuda:0")
    eng = pkg.AdaCGD(n, d, cands, z, loss=loss, lam=lam, A=torch.from_numpy(A).to(dev),
                     target=torch.from_numpy(t).to(dev), x0=torch.from_numpy(x0).to(dev), gamma=gamma)
    skipped = 0
    for it in range(12):
        for k_gpu, k_or in (("x", "x"), ("G", "G"), ("grad", "X"), ("gt", "gt"), ("gm", "gm")):
            eng.set_state(k_gpu, torch.from_numpy(np.ascontiguousarray(st[k_or])))
        before_G, before_X = st["G"].copy(), st["X"].copy()
        recs, levels = eng.step(1, report=True)
        # the oracle's round on the GPU's own gradients, so that selections can be compared exactly
        ggrad = eng.get_state("grad").cpu().numpy()
        oracle_round(st, prob, gamma, method, K, zeta)
        assert np.abs(ggrad - st["X"]).max() <= 1e-5 * np.abs(st["X"]).max()
        want = []
        for i in range(n):
            if method in ("gd", "ef21"):
                want.append(O.ef21(before_G[i], before_X[i], ggrad[i], cands[0]))
            elif method == "lag":
                want.append(O.lag(before_G[i], before_X[i], ggrad[i], zeta))
            else:
                want.append(O.clag(before_G[i], before_X[i], ggrad[i], cands[0], zeta))
        got = eng.get_state("G").cpu().numpy()
        if method == "lag":
            # LAG's own definition copies x; the engine adds the full difference, h + (x - h), which
            # may differ from x in the last bit (Eq. 7 taken literally).  The skip decision is exact.
            for i in range(n):
                sent = not np.array_equal(want[i].view(np.uint32), before_G[i].view(np.uint32))
                assert (levels[0][i] != 0) == sent
                if sent:
                    assert np.abs(got[i] - want[i]).max() <= 1e-6 * np.abs(want[i]).max()
                else:
                    assert np.array_equal(got[i].view(np.uint32), before_G[i].view(np.uint32))
        else:
            assert np.array_equal(got.view(np.uint32), np.stack(want).view(np.uint32)), (method, it)
        skipped += sum(1 for lv in levels[0] if lv == 0)
        if method in ("gd", "ef21"):
            assert levels[0] == [1] * n and recs[0]["bits_up"] == n * O.message_bits(cands[0], d)
    if method in ("lag", "clag"):
        assert skipped > 0          # the trigger does skip rounds at this zeta


@pytest.mark.gpu
def test_run_to_budget_on_the_engine():
    import torch
    import paper_2211_00188_b200 as pkg

    n, d, m = 4, 500, 50
    A, t = S.logistic_problem(n, d, m, seed=6)
    gamma = 0.5 / S.smoothness_estimate(A, 0, 0.1)
    cands, z = P.method_set("adacgd", d, zeta=1.0)
    dev = torch.device("cuda:0")
    eng = pkg.AdaCGD(n, d, cands, z, loss=0, lam=0.1, A=torch.from_numpy(A).to(dev), target=torch.from_numpy(t).to(dev),
                     x0=torch.zeros(d, device=dev), gamma=gamma)
    budget = 40 * P.max_bits_per_round(n, d, cands) // 10
    rec = P.run_to_budget(eng, budget, batch=16)
    assert rec["bits_up"][-1] >= budget and (len(rec["bits_up"]) == 1 or rec["bits_up"][-2] < budget)
    assert eng.get_state("bits_up") == rec["bits_up"][-1] and eng.get_state("step") == len(rec["loss"])
    assert rec["loss"][-1] < rec["loss"][0]


@pytest.mark.gpu
def test_gamma_sweep_on_the_engine():
    import torch
    import paper_2211_00188_b200 as pkg

    n, d, m = 3, 300, 30
    A, t, _ = S.least_squares_problem(n, d, m, seed=9)
    base = 0.125 / S.smoothness_estimate(A, 2, 0.0)
    cands, z = P.method_set("clag", d, K=5, zeta=1.0)
    dev = torch.device("cuda:0")
    Ad, td = torch.from_numpy(A).to(dev), torch.from_numpy(t).to(dev)

    def make(gamma):
        return pkg.AdaCGD(n, d, cands, z, loss=2, lam=0.0, A=Ad, target=td, x0=torch.zeros(d, device=dev), gamma=gamma)

    budget = 60 * P.max_bits_per_round(n, d, cands)
    res = P.gamma_sweep(make, base, budget, exponents=range(0, 7), max_rounds=400)
    finals = {e: r["loss"][-1] for e, r in res["runs"].items()}
    finite = {e: v for e, v in finals.items() if np.isfinite(v)}
    assert res["best"] == min(finite, key=finite.get)
    assert finite and finals[res["best"]] <= min(finite.values())
    assert all(r["bits_up"][-1] >= budget or len(r["loss"]) == 400 for r in res["runs"].values())
