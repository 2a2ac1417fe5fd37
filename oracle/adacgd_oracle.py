"""Plain CPU oracle for one AdaCGD iteration (arXiv 2211.00188).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It shares no code with the CUDA path.

What is restated here, and from which passage of the paper:

* contractive compressors (Definition 1 "Biased or contractive compression
  operator", Eq. 4): Top-K (Section 2.1) and a deterministic uniform quantiser
  (the abstract names quantisation; the paper never writes one out, so the
  quantiser below is this project's reading -- *parity unpinned against the paper*);
* the EF21 compressor  C^EF_{h,y}(x) = h + C(x - h)            (Eq. 7);
* the CLAG / LAG compressors                                   (Eq. 8, Eq. 5);
* the Ada3PC compressor (Definition 3, Eq. 9 "first predicate that holds"), with callables
  (`ada3pc`) and with the small menu of triggers the library evaluates (`adaptive_3pc`);
* the AdaCGD compressor and its trigger  ||x - C^{EF,j}(x)||^2 <= zeta ||x - y||^2
  (Eq. 10 and the Definition of Section 4.3, Eq. 11);
* the bidirectional loop (Algorithm 1, with the three-point arguments of Algorithm 2);
* the experiment's objective, logistic loss + non-convex regulariser (Section 6),
  plus the l2-regularised logistic and the least-squares objectives of the
  synthetic workloads.

Arithmetic conventions (they are this project's reading where the paper is silent):

* vectors are IEEE binary32; every elementwise operation below is ONE binary32
  operation with round-to-nearest-even, written as a numpy float32 expression;
* a squared norm is the EXACT real sum of the exact squares of its binary32
  terms, rounded once to binary64.  Squares of binary32 numbers are integer
  multiples of 2**-298, so the sum is carried as a Python integer;
* the trigger compares  err_j <= fl64(double(zeta) * D)  on those binary64 values;
* Top-K keeps the first K entries under the total order
  (|v| descending, index ascending); |v| is compared on the bit pattern with the
  sign bit cleared, so -0 == +0 and subnormals are ordinary values;
* local gradients are accumulated in binary64 and rounded once to binary32.

Parity unpinned (the paper gives nothing to check these against): the bit-count
formula `message_bits`, the quantiser `quantize`, the default lambda of the
l2-regularised workload.
"""
from __future__ import annotations

from fractions import Fraction

import numpy as np

F32 = np.float32
TOPK = 0
QUANT = 1

# Squares of binary32 values are integer multiples of 2**-_SQ_SCALE.
_SQ_SCALE = 298


# --------------------------------------------------------------------------
# exact squared norms
# --------------------------------------------------------------------------
def _as_f32(v) -> np.ndarray:
    return np.ascontiguousarray(v, dtype=F32)


def magnitude_key(v) -> np.ndarray:
    """Bit pattern of |v| (uint32): the sort key of Top-K."""
    return _as_f32(v).view(np.uint32) & np.uint32(0x7FFFFFFF)


def sumsq_units(w) -> int:
    """Exact sum of w_k**2 over a binary32 array, as an integer count of 2**-298."""
    w = _as_f32(w).ravel()
    if w.size == 0:
        return 0
    bits = w.view(np.uint32)
    expo = ((bits >> np.uint32(23)) & np.uint32(0xFF)).astype(np.int64)
    if np.any(expo == 0xFF):
        raise FloatingPointError("non-finite entry")
    frac = (bits & np.uint32(0x7FFFFF)).astype(np.uint64)
    # value = mant * 2**(eff - 150); subnormals have eff = 1 and no hidden bit
    mant = np.where(expo > 0, frac | np.uint64(0x800000), frac)
    eff = np.where(expo > 0, expo, 1)
    sq = mant * mant  # < 2**48, exact in uint64
    total = 0
    for e in np.unique(eff):
        s = sq[eff == e]
        lo = int(np.sum(s & np.uint64(0xFFFFFF), dtype=np.uint64))
        hi = int(np.sum(s >> np.uint64(24), dtype=np.uint64))
        total += ((hi << 24) + lo) << (2 * int(e) - 2)
    return total


def units_to_double(units: int) -> float:
    """Round an integer count of 2**-298 to the nearest binary64 (ties to even)."""
    return float(Fraction(units, 1 << _SQ_SCALE))


def sumsq(w) -> float:
    """||w||^2 under the exact-sum convention."""
    return units_to_double(sumsq_units(w))


# --------------------------------------------------------------------------
# contractive compressors  (Eq. 4)
# --------------------------------------------------------------------------
def topk_order(v) -> np.ndarray:
    """Indices of v sorted by (|v| descending, index ascending)."""
    key = magnitude_key(v).astype(np.int64)
    return np.argsort(-key, kind="stable")


def topk_kept(v, K: int) -> np.ndarray:
    """Indices kept by Top-K (Section 2.1); K >= d keeps everything."""
    v = _as_f32(v)
    return topk_order(v)[: min(int(K), v.size)]


def topk(v, K: int) -> np.ndarray:
    """Top-K sparsifier: the K largest-magnitude entries, zero elsewhere."""
    v = _as_f32(v)
    out = np.zeros_like(v)
    kept = topk_kept(v, K)
    out[kept] = v[kept]
    return out


def quantize(v, bits: int) -> np.ndarray:
    """Deterministic uniform quantiser with 2**(bits-1)-1 positive levels.

    s = max|v|, L = 2**(bits-1) - 1, inv = fl(L / s), step = fl(s / L),
    code = min(L, rint(fl(|v| * inv)))  (ties to even),
    Q(v) = copysign(fl(code * step), v); Q = 0 when s = 0.
    """
    v = _as_f32(v)
    if not 2 <= bits <= 16:
        raise ValueError("bits must be in [2,16]")
    a = np.abs(v)
    s = F32(a.max()) if v.size else F32(0)
    if s == 0:
        return np.zeros_like(v)
    L = F32((1 << (bits - 1)) - 1)
    inv = F32(L / s)
    step = F32(s / L)
    code = np.minimum(L, np.rint((a * inv).astype(F32))).astype(F32)
    return np.copysign((code * step).astype(F32), v).astype(F32)


def apply_candidate(v, cand) -> np.ndarray:
    kind, param = cand
    if kind == TOPK:
        return topk(v, param)
    if kind == QUANT:
        return quantize(v, param)
    raise ValueError("unknown candidate kind")


def message_bits(cand, d: int) -> int:
    """Bits a worker sends for one candidate (the paper counts communication
    cost but prints no formula; this is the project's reading).
    Top-K, K < d: K * (32 + ceil(log2 d)); K >= d: 32 d; b-bit quantiser: 32 + b d."""
    kind, param = cand
    if kind == TOPK:
        if param >= d:
            return 32 * d
        idx_bits = max(1, int(d - 1).bit_length())
        return int(param) * (32 + idx_bits)
    return 32 + int(param) * d


# --------------------------------------------------------------------------
# three point compressors
# --------------------------------------------------------------------------
def apply_shifted(h, v, cand) -> np.ndarray:
    """h + C(v) in binary32.  A Top-K message is sparse: the receiver adds it at the kept
    indices and leaves every other entry of h as it is (so a -0.0 outside the kept set stays
    -0.0); a quantised message is dense and is added everywhere."""
    kind, param = cand
    if kind == TOPK:
        out = h.copy()
        kept = topk_kept(v, param)
        out[kept] = (h[kept] + v[kept]).astype(F32)
        return out
    return (h + apply_candidate(v, cand)).astype(F32)


def ef21(h, y, x, cand) -> np.ndarray:
    """EF21 compressor (Eq. 7): h + C(x - h), every operation in binary32."""
    h = _as_f32(h)
    x = _as_f32(x)
    v = (x - h).astype(F32)
    return apply_shifted(h, v, cand)


def lag(h, y, x, zeta) -> np.ndarray:
    """LAG compressor (Section 2.3 / Eq. 8 with the identity): h if
    ||x-h||^2 <= zeta ||x-y||^2, else x."""
    h, y, x = _as_f32(h), _as_f32(y), _as_f32(x)
    if sumsq((x - h).astype(F32)) <= float(F32(zeta)) * sumsq((x - y).astype(F32)):
        return h.copy()
    return x.copy()


def clag(h, y, x, cand, zeta) -> np.ndarray:
    """CLAG compressor (Eq. 8): h + C(x-h) if ||x-h||^2 > zeta ||x-y||^2, else h."""
    h, y, x = _as_f32(h), _as_f32(y), _as_f32(x)
    if sumsq((x - h).astype(F32)) > float(F32(zeta)) * sumsq((x - y).astype(F32)):
        return ef21(h, y, x, cand)
    return h.copy()


def ada3pc(h, y, x, compressors, predicates) -> np.ndarray:
    """Ada3PC (Definition 3, Eq. 9): apply the first compressor whose predicate
    holds; the last one if none does.  `compressors` has m entries and
    `predicates` m-1, each a callable of (h, y, x)."""
    assert len(predicates) == len(compressors) - 1
    for C, P in zip(compressors, predicates):
        if P(h, y, x):
            return C(h, y, x)
    return compressors[-1](h, y, x)


def candidate_error(v, cand) -> float:
    """||v - C(v)||^2, the left side of the trigger (Eq. 10) written on the
    difference vector v = x - h:  x - (h + C(x-h)) = v - C(v)."""
    v = _as_f32(v)
    return sumsq((v - apply_candidate(v, cand)).astype(F32))


def adacgd(h, y, x, cands, zeta):
    """AdaCGD compressor (Section 4.3, Eq. 11).

    Level 0 ("skip") returns h when ||x-h||^2 <= zeta ||x-y||^2.  Otherwise the
    candidates are tried in the given order (strongest compression first) and
    the first whose EF21 output satisfies the trigger is applied; the last
    candidate is applied when none does.  With an empty candidate list the
    compressor is the identity (used for an uncompressed master).

    Returns a dict: out (new estimator), level (0..m), bits, err (m+1 values:
    ||v||^2 then one per candidate), D (= ||x-y||^2), kept (sorted indices
    written by a Top-K level, None otherwise).
    """
    h, y, x = _as_f32(h), _as_f32(y), _as_f32(x)
    d = x.size
    m = len(cands)
    if m == 0:
        return dict(out=x.copy(), level=0, bits=32 * d, err=[0.0], D=0.0, kept=None)
    v = (x - h).astype(F32)
    D = sumsq((x - y).astype(F32))
    rhs = float(F32(zeta)) * D
    err = [sumsq(v)] + [candidate_error(v, c) for c in cands]
    level = m
    for j in range(m + 1):
        if err[j] <= rhs:
            level = j
            break
    if level == 0:
        return dict(out=h.copy(), level=0, bits=0, err=err, D=D, kept=None)
    cand = cands[level - 1]
    out = apply_shifted(h, v, cand)
    kept = np.sort(topk_kept(v, cand[1])) if cand[0] == TOPK else None
    return dict(out=out, level=level, bits=message_bits(cand, d), err=err, D=D, kept=kept)


# Triggers the library evaluates for the adaptive compressor of Definition 3 (Eq. 9); each is a
# condition P(h, y, x) -> {0, 1} on the level's error E = ||x - C_{h,y}(x)||^2 (E = ||x - h||^2 for
# keeping h), under the exact-sum convention above.
PRED_LAZY = 0      # E <= param * ||x - y||^2      (Eq. 10)
PRED_ABSOLUTE = 1  # E <= param
PRED_RELATIVE = 2  # E <= param * ||x - h||^2
PRED_NEVER = 3
PRED_ALWAYS = 4


def trigger_holds(pred, E: float, h, y, x) -> bool:
    """One condition P_j(h, y, x) of Definition 3, from the menu above."""
    kind, param = pred
    if kind == PRED_NEVER:
        return False
    if kind == PRED_ALWAYS:
        return True
    par = float(F32(param))
    if kind == PRED_LAZY:
        return E <= par * sumsq((_as_f32(x) - _as_f32(y)).astype(F32))
    if kind == PRED_RELATIVE:
        return E <= par * sumsq((_as_f32(x) - _as_f32(h)).astype(F32))
    if kind == PRED_ABSOLUTE:
        return E <= par
    raise ValueError("unknown trigger kind")


def adaptive_3pc(h, y, x, cands, preds):
    """Adaptive three-point compressor (Definition 3, Eq. 9) over the compressors
    C^0 = "keep h" and C^j = EF21 with candidate j (Eq. 7), j = 1..m, with the triggers
    preds[0..m-1] from the menu above: the first compressor whose trigger holds is applied, the
    last one if none does.  AdaCGD (Eq. 11) is the case preds = [(PRED_LAZY, zeta)] * m.
    Returns the same dict as `adacgd`."""
    h, y, x = _as_f32(h), _as_f32(y), _as_f32(x)
    d, m = x.size, len(cands)
    assert len(preds) == m and m >= 1
    v = (x - h).astype(F32)
    D = sumsq((x - y).astype(F32))
    err = [sumsq(v)] + [candidate_error(v, c) for c in cands]
    level = m
    for j in range(m):
        if trigger_holds(preds[j], err[j], h, y, x):
            level = j
            break
    if level == 0:
        return dict(out=h.copy(), level=0, bits=0, err=err, D=D, kept=None)
    cand = cands[level - 1]
    out = apply_shifted(h, v, cand)
    kept = np.sort(topk_kept(v, cand[1])) if cand[0] == TOPK else None
    return dict(out=out, level=level, bits=message_bits(cand, d), err=err, D=D, kept=kept)


# --------------------------------------------------------------------------
# objectives  (Section 6 and the synthetic workloads)
# --------------------------------------------------------------------------
LOGISTIC_NCVX = 0   # (1/m) sum log(1+exp(-y a.x)) + lam * sum x_j^2/(1+x_j^2)
LOGISTIC_L2 = 1     # (1/m) sum log(1+exp(-y a.x)) + (lam/2) ||x||^2
LEAST_SQUARES = 2   # ||A x - b||^2 / (2 m)


def _matvec64(A, x64):
    if hasattr(A, "tocsr"):
        return np.asarray(A.astype(np.float64) @ x64).ravel()
    return np.asarray(A, dtype=np.float64) @ x64   # features already held in binary64 are used as they are


def _rmatvec64(A, r64):
    if hasattr(A, "tocsr"):
        return np.asarray(A.astype(np.float64).T @ r64).ravel()
    return np.asarray(A, dtype=np.float64).T @ r64


def local_loss(A, target, x, loss: int, lam: float) -> float:
    """f_i(x) in binary64."""
    x64 = np.asarray(x, dtype=np.float64)
    z = _matvec64(A, x64)
    t = np.asarray(target, dtype=np.float64)
    m = z.size
    if loss == LEAST_SQUARES:
        return float(np.sum((z - t) ** 2) / (2.0 * m))
    data = float(np.sum(np.logaddexp(0.0, -t * z)) / m)
    if loss == LOGISTIC_NCVX:
        return data + float(lam) * float(np.sum(x64 ** 2 / (1.0 + x64 ** 2)))
    if loss == LOGISTIC_L2:
        return data + 0.5 * float(lam) * float(np.sum(x64 ** 2))
    raise ValueError("unknown loss")


def local_gradient(A, target, x, loss: int, lam: float) -> np.ndarray:
    """grad f_i(x): binary64 accumulation, one rounding to binary32."""
    x64 = np.asarray(x, dtype=np.float64)
    z = _matvec64(A, x64)
    t = np.asarray(target, dtype=np.float64)
    m = z.size
    if loss == LEAST_SQUARES:
        g = _rmatvec64(A, (z - t) / m)
    else:
        # d/dz log(1+exp(-t z)) = -t * sigma(-t z),  sigma(u) = exp(-log(1+exp(-u)))
        sig = np.exp(-np.logaddexp(0.0, t * z))
        g = _rmatvec64(A, (-t * sig) / m)
        if loss == LOGISTIC_NCVX:
            g = g + float(lam) * 2.0 * x64 / (1.0 + x64 ** 2) ** 2
        elif loss == LOGISTIC_L2:
            g = g + float(lam) * x64
        else:
            raise ValueError("unknown loss")
    return g.astype(F32)


# --------------------------------------------------------------------------
# the loop  (Algorithm 1 with the three-point arguments of Algorithm 2)
# --------------------------------------------------------------------------
def server_mean(G) -> np.ndarray:
    """(1/n) sum_i g_i in binary32: left-to-right over workers, one division."""
    G = _as_f32(G)
    acc = G[0].copy()
    for i in range(1, G.shape[0]):
        acc = (acc + G[i]).astype(F32)
    return (acc / F32(G.shape[0])).astype(F32)


def all_gradients(problem, x) -> np.ndarray:
    return np.stack([local_gradient(A, t, x, problem["loss"], problem["lam"])
                     for A, t in zip(problem["A"], problem["target"])])


def global_loss(problem, x) -> float:
    vals = [local_loss(A, t, x, problem["loss"], problem["lam"])
            for A, t in zip(problem["A"], problem["target"])]
    return float(np.mean(vals))


def init_state(problem, x0, worker_cands=(), g0_mode: int = 1) -> dict:
    """Inputs of Algorithm 1: x^0, g_i^0, g~^0 = mean, g^0 = g~^0.
    g0_mode 0: g_i^0 = 0; 1: g_i^0 = grad f_i(x^0); 2: g_i^0 = C^1(grad f_i(x^0))
    with the strongest candidate (the CLAG initialisation of Section 2.3)."""
    x = _as_f32(x0).copy()
    X = all_gradients(problem, x)
    if g0_mode == 0:
        G = np.zeros_like(X)
    elif g0_mode == 1:
        G = X.copy()
    else:
        G = np.stack([apply_candidate(row, worker_cands[0]) for row in X])
    gt = server_mean(G)
    return dict(x=x, X=X, Y=X.copy(), G=G, gt=gt, gm=gt.copy(), step=0,
                bits_up=0, bits_down=0)


def compress_rows(X, G, Y, cands, zeta):
    """Worker side of one iteration on given arrays: every row i gets
    g_i <- AdaCGD_{h=g_i, y=Y_i}(X_i).  Returns (G_new, list of per-row dicts)."""
    X, G, Y = _as_f32(X), _as_f32(G), _as_f32(Y)
    res = [adacgd(G[i], Y[i], X[i], cands, zeta) for i in range(X.shape[0])]
    return np.stack([r["out"] for r in res]), res


def step(state, problem, gamma, worker_cands, worker_zeta,
         master_cands=(), master_zeta=0.0) -> dict:
    """One iteration of Algorithm 2; returns the per-step report."""
    x = (state["x"] - (F32(gamma) * state["gm"]).astype(F32)).astype(F32)
    X = all_gradients(problem, x)
    G, res = compress_rows(X, state["G"], state["X"], worker_cands, worker_zeta)
    gt_new = server_mean(G)
    mres = adacgd(state["gm"], state["gt"], gt_new, list(master_cands), master_zeta)
    bits = sum(r["bits"] for r in res)
    state.update(x=x, Y=state["X"], X=X, G=G, gt=gt_new, gm=mres["out"],
                 step=state["step"] + 1,
                 bits_up=state["bits_up"] + bits,            # workers -> server
                 bits_down=state["bits_down"] + mres["bits"])  # server broadcast
    return dict(levels=[r["level"] for r in res], bits=[r["bits"] for r in res],
                master_level=mres["level"], master_bits=mres["bits"],
                worker=res, master=mres)
