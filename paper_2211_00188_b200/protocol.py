"""The paper's comparison protocol on top of the AdaCGD engine (Section 6 and Appendix C).

Every method of the comparison is AdaCGD with a particular candidate list and trigger, so one
engine runs them all; this module only chooses the lists, drives `adacgd_step` until a
communication budget is spent and sweeps the step size.  All arithmetic stays in the kernels.

  gd      Top-d, zeta = 0          every worker sends its full gradient each round (Eq. 2 with the identity)
  ef21    one Top-K, zeta = 0      EF21 (Eq. 7): the trigger never skips
  lag     Top-d, zeta > 0          LAG (Section 2.3): send everything or nothing
  clag    one Top-K, zeta > 0      CLAG (Eq. 8)
  adacgd  a ladder of Top-K        AdaCGD (Section 4.3, Eq. 11): skip, then K_1 < K_2 < ...
"""
from __future__ import annotations

from typing import Callable, Dict, Iterable, List, Optional, Sequence, Tuple

from .binding import TOPK, message_bits

Cand = Tuple[int, int]
METHODS = ("gd", "ef21", "lag", "clag", "adacgd")


def topk_ladder(d: int, fractions: Sequence[float] = (0.001, 0.01, 0.1, 0.5)) -> List[Cand]:
    """Top-K candidates at the given fractions of d, strongest compression first, duplicates
    dropped (the experiments' ladder ends at 50 % of d, Appendix C)."""
    ks: List[int] = []
    for f in sorted(fractions):
        k = min(d, max(1, int(round(f * d))))
        if not ks or k > ks[-1]:
            ks.append(k)
    return [(TOPK, k) for k in ks]


def method_set(method: str, d: int, *, K: int = 1, zeta: float = 1.0,
               ladder: Optional[Sequence[Cand]] = None) -> Tuple[List[Cand], float]:
    """Candidate list and trigger that make the engine run `method` (see the module text).  K is the
    Top-K of EF21 and CLAG; the experiments use Top-1 for both (Section 6)."""
    if method == "gd":
        return [(TOPK, d)], 0.0
    if method == "ef21":
        return [(TOPK, int(K))], 0.0
    if method == "lag":
        return [(TOPK, d)], float(zeta)
    if method == "clag":
        return [(TOPK, int(K))], float(zeta)
    if method == "adacgd":
        return list(ladder) if ladder is not None else topk_ladder(d), float(zeta)
    raise ValueError(f"unknown method {method!r}; one of {METHODS}")


def max_bits_per_round(n: int, d: int, cands: Sequence[Cand]) -> int:
    """Upper bound of the bits n workers send in one round: the largest message of the list, as the
    library counts it (adacgd_message_bits)."""
    return n * max((message_bits(c, d) for c in cands), default=0)


def run_to_budget(engine, bit_budget: int, *, max_rounds: int = 1_000_000, batch: int = 64) -> Dict[str, list]:
    """Iterates until the workers have sent at least `bit_budget` bits (the paper's stopping rule:
    methods are compared at equal communication, Appendix C) or `max_rounds` rounds have run.
    Rounds are enqueued in batches that cannot cross the budget, and one at a time near it, so the
    engine stops exactly at the round that spends it.  Returns the per-round records:
    {"loss": [...], "bits_up": cumulative [...], "levels": [[...], ...]}."""
    worst = max_bits_per_round(engine.n, engine.d, engine.worker)
    out: Dict[str, list] = {"loss": [], "bits_up": [], "levels": []}
    sent, rounds = 0, 0
    while sent < bit_budget and rounds < max_rounds:
        safe = (bit_budget - sent) // worst if worst > 0 else batch
        k = int(max(1, min(batch, safe, max_rounds - rounds)))
        recs, levels = engine.step(k, report=True)
        for r, lv in zip(recs, levels):
            sent += int(r["bits_up"])
            rounds += 1
            out["loss"].append(float(r["loss"]))
            out["bits_up"].append(sent)
            out["levels"].append(list(lv))
        if worst == 0:
            break
    return out


def gamma_sweep(make_engine: Callable[[float], object], base_gamma: float, bit_budget: int, *,
                exponents: Iterable[int] = range(0, 9), max_rounds: int = 1_000_000) -> Dict[str, object]:
    """The step-size search of the experiments: gamma = 2^e * base_gamma for e = 0..8, each run to
    the same bit budget; the best run is the one with the lowest final loss that stayed finite.
    `make_engine(gamma)` returns a fresh engine.  Returns {"best": e, "runs": {e: record}}."""
    runs: Dict[int, Dict[str, list]] = {}
    best, best_loss = None, float("inf")
    for e in exponents:
        eng = make_engine(base_gamma * (2.0 ** e))
        rec = run_to_budget(eng, bit_budget, max_rounds=max_rounds)
        close = getattr(eng, "close", None)
        if close:
            close()
        runs[e] = rec
        final = rec["loss"][-1] if rec["loss"] else float("inf")
        if final == final and final < best_loss:   # NaN-safe
            best, best_loss = e, final
    return {"best": best, "runs": runs}
