"""Parity of stages a2-a4 (+ the server mean) between the CUDA path, called through
the C ABI, and the CPU oracle on identical binary32 inputs.  Integer results (levels,
bits, kept index sets) and the estimators must agree bit for bit."""
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


def gpu_compress(torch, X, G, Y, cands, zeta, want_mean=True, engine=None, want_kept=True):
    import paper_2211_00188_b200 as pkg
    rows, d = X.shape
    dev = torch.device("cuda:0")
    eng = engine or pkg.AdaCGD(rows, d, cands, zeta)
    Xd, Gd, Yd = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (X, G, Y))
    m = len(cands)
    level = torch.full((rows,), -7, dtype=torch.int32, device=dev)
    bits = torch.zeros(rows, dtype=torch.int64, device=dev)
    err = torch.zeros(rows, m + 1, dtype=torch.float64, device=dev)
    D = torch.zeros(rows, dtype=torch.float64, device=dev)
    stride = d
    # without the kept-index outputs the update kernel takes its streaming path
    kept_idx = torch.full((rows, stride), -1, dtype=torch.int32, device=dev) if want_kept else None
    kept_cnt = torch.zeros(rows, dtype=torch.int64, device=dev) if want_kept else None
    mean = torch.zeros(d, dtype=torch.float32, device=dev) if want_mean else None
    eng.compress(Xd, Gd, Yd, cands, zeta, mean_out=mean, level=level, bits=bits, err=err, D=D,
                 kept_idx=kept_idx, kept_cnt=kept_cnt)
    torch.cuda.synchronize()
    kept = None
    if want_kept:
        cnt = kept_cnt.cpu().numpy()
        idx = kept_idx.cpu().numpy()
        kept = [np.sort(idx[i, :cnt[i]]) for i in range(rows)]
    return dict(G=Gd.cpu().numpy(), level=level.cpu().numpy(), bits=bits.cpu().numpy(), err=err.cpu().numpy(),
                D=D.cpu().numpy(), kept=kept, list_levels=eng.get_state("list_levels"),
                mean=mean.cpu().numpy() if want_mean else None, rechecks=eng.get_state("rechecks"), fallbacks=eng.get_state("fallbacks"),
                flags=eng.get_state("flags"), engine=eng)


def assert_bitwise(a, b, what):
    a, b = np.ascontiguousarray(a, F32), np.ascontiguousarray(b, F32)
    bad = np.nonzero(a.view(np.uint32) != b.view(np.uint32))
    assert bad[0].size == 0, f"{what}: {bad[0].size} mismatches, first at {tuple(x[0] for x in bad)}"


def check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=False):
    got = gpu_compress(torch, X, G, Y, cands, zeta)
    G_ref, res = O.compress_rows(X, G, Y, cands, zeta)
    if both_update_paths:
        again = gpu_compress(torch, X, G, Y, cands, zeta, want_kept=False)
        assert_bitwise(again["G"], G_ref, "G (streaming update)")
        assert_bitwise(again["mean"], O.server_mean(G_ref), "mean (streaming update)")
        assert again["level"].tolist() == [r["level"] for r in res] and again["bits"].tolist() == [r["bits"] for r in res]
    rows, d = X.shape
    for i, r in enumerate(res):
        assert got["level"][i] == r["level"], (i, got["level"][i], r["level"], r["err"], r["D"])
        assert got["bits"][i] == r["bits"], i
        # err and D are diagnostics: binary32 chains of 64 terms, relative error <= 66 * 2^-24 (the bound the
        # library certifies its comparisons against); the decisions taken from them are exact
        assert np.allclose(got["err"][i], r["err"], rtol=ERR_RTOL, atol=0), (i, got["err"][i], r["err"])
        assert np.isclose(got["D"][i], r["D"], rtol=ERR_RTOL, atol=0)
        if r["kept"] is not None:
            assert np.array_equal(got["kept"][i], r["kept"]), (i, r["level"])
        else:
            assert got["kept"][i].size == 0
    assert_bitwise(got["G"], G_ref, "G")
    assert_bitwise(got["mean"], O.server_mean(G_ref), "mean")
    assert got["flags"] == 0
    return got, res


CANDS3 = [(TOPK, 3), (TOPK, 30), (TOPK, 300)]
ERR_RTOL = 66 * 2.0 ** -24


@pytest.mark.parametrize("d", [1, 2, 3, 5, 17, 1000, 1023, 1024, 1025, 4096, 5000, 70001])
@pytest.mark.parametrize("rows", [1, 3])
def test_topk_gaussian_shapes(torch, rows, d):
    X, G, Y = S.gaussian_rows(rows, d, seed=d + rows)
    cands = [(TOPK, k) for k in sorted({1, max(1, d // 100), max(1, d // 10), max(1, d // 2)})]
    for zeta in (0.0, 1.0, 4.0):
        check_against_oracle(torch, X, G, Y, cands, zeta)


@pytest.mark.parametrize("zeta", [0.0, 0.25, 1.0, 4.0, 1e30])
def test_zeta_sweep_reaches_every_level(torch, zeta):
    X, G, Y = S.gaussian_rows(8, 20000, seed=1, drift=0.4, move=0.5)
    got, res = check_against_oracle(torch, X, G, Y, [(TOPK, 20), (TOPK, 2000), (TOPK, 10000), (TOPK, 20000)], zeta)
    if zeta == 0.0:
        assert set(got["level"].tolist()) == {4}      # EF21 with the last candidate (Section 4.3)
    if zeta == 1e30:
        assert set(got["level"].tolist()) == {0}      # every worker skips


def test_levels_differ_across_rows(torch):
    # rows with different staleness pick different levels in one call
    rows, d = 6, 30000
    X, G, Y = S.gaussian_rows(rows, d, seed=2)
    rng = np.random.Generator(np.random.PCG64(5))
    for i, drift in enumerate([0.05, 0.1004, 0.11, 0.12, 0.2, 0.5]):
        G[i] = (X[i] + drift * rng.standard_normal(d)).astype(F32)
    got, _ = check_against_oracle(torch, X, G, Y, [(TOPK, 30), (TOPK, 3000), (TOPK, 15000)], 1.0)
    assert len(set(got["level"].tolist())) >= 3


@pytest.mark.parametrize("d", [7, 1000, 4099, 20000, 50000])   # 20000: a short row whose first-digit lists overflow
def test_ties_and_equalities_use_the_exact_path(torch, d):
    # small integers: many equal magnitudes (lowest index wins), signed zeros, and
    # trigger comparisons that hold with equality, which only exact sums decide
    X, G, Y = S.tie_vectors(4, d, seed=d)
    total = 0
    for zeta in (0.0, 0.5, 1.0, 2.0):
        cands = [(TOPK, k) for k in sorted({1, max(2, d // 7), max(3, d // 2), d - 1 if d > 4 else d})]
        got, _ = check_against_oracle(torch, X, G, Y, cands, zeta)
        total += got["rechecks"]
    # and a row built so that ||v - C(v)||^2 == zeta * D exactly
    x = np.zeros(d, F32); x[: min(d, 6)] = [3, -1, 2, 0.5, 0, 0][: min(d, 6)]
    y = x.copy(); y[0] -= 1.0
    h = np.zeros(d, F32)
    # (Top-4 is last and has no trigger of its own: the equality is at a level that is tested)
    got, res = check_against_oracle(torch, x[None], h[None], y[None], [(TOPK, 1), (TOPK, 2), (TOPK, 3), (TOPK, 4)], 0.25)
    if d >= 6:
        assert res[0]["level"] == 3 and got["rechecks"] >= 1


def test_degenerate_rows(torch):
    d = 3000
    z = np.zeros((1, d), F32)
    one = np.ones((1, d), F32)
    cands = [(TOPK, 5), (TOPK, 500)]
    check_against_oracle(torch, z, z, z, cands, 1.0)                 # v = 0, D = 0: skip
    check_against_oracle(torch, one, z, one, cands, 1.0)             # D = 0, all |v| equal: last candidate, ties by index
    check_against_oracle(torch, one, z, z, cands, 0.5)               # all equal magnitudes
    check_against_oracle(torch, one, z, z, cands, 1.0)               # ||v||^2 == D: skip by equality
    neg = -one
    check_against_oracle(torch, neg, z, one, [(TOPK, 1), (TOPK, d)], 0.1)   # identity last
    check_against_oracle(torch, neg, z, one, [(TOPK, d + 5)], 0.0)          # K > d
    tiny = np.full((2, d), 1e-42, F32)                                # subnormal differences
    tiny[1, ::3] = 3e-45
    check_against_oracle(torch, tiny, z[[0, 0]], z[[0, 0]], cands, 0.3)
    big = np.full((1, d), 1e18, F32); big[0, 5] = 3e19                # squares near the top of binary32 range
    check_against_oracle(torch, big, z, (big * F32(0.5)).astype(F32), cands, 0.2)


def test_heavy_tailed_block_scaled_rows(torch):
    Xs, G0 = S.stress_vectors(3, 120000, blocks=10, period=4, seed=3, device="cpu")
    X, Y, G = Xs[1].numpy(), Xs[0].numpy(), G0.numpy()
    for zeta in (0.0, 1.0):
        check_against_oracle(torch, X, G, Y, [(TOPK, 120), (TOPK, 1200), (TOPK, 12000)], zeta)


@pytest.mark.parametrize("d", [9, 1000, 12345, 40000])   # the last one is past the short-row kernel: three-pass path
def test_quantiser_and_mixed_candidates(torch, d):
    X, G, Y = S.gaussian_rows(3, d, seed=d)
    for zeta in (0.0, 0.05, 0.5, 2.0):
        check_against_oracle(torch, X, G, Y, [(QUANT, 2), (QUANT, 4), (QUANT, 8)], zeta)
        check_against_oracle(torch, X, G, Y, [(TOPK, 1), (TOPK, max(2, d // 100)), (QUANT, 2), (QUANT, 4),
                                              (TOPK, max(3, d // 10)), (QUANT, 8)], zeta)


def test_identity_set_copies(torch):
    X, G, Y = S.gaussian_rows(3, 2049, seed=4)
    got = gpu_compress(torch, X, G, Y, [], 0.0)
    assert_bitwise(got["G"], X, "G")
    assert_bitwise(got["mean"], O.server_mean(X), "mean")
    assert got["level"].tolist() == [0, 0, 0] and got["bits"].tolist() == [32 * 2049] * 3


def test_master_step_is_the_same_call_with_one_row(torch):
    # Algorithm 2: g^{t+1} = C^M_{g^t, g~^t}(g~^{t+1})
    n, d = 5, 40000
    X, G, Y = S.gaussian_rows(n, d, seed=6)
    wc, mc = [(TOPK, 40), (TOPK, 4000)], [(TOPK, 400), (TOPK, 20000)]
    got = gpu_compress(torch, X, G, Y, wc, 1.0)
    G_ref, _ = O.compress_rows(X, G, Y, wc, 1.0)
    gt_new = O.server_mean(G_ref)
    rng = np.random.Generator(np.random.PCG64(9))
    gt_old = (gt_new + 0.2 * rng.standard_normal(d)).astype(F32)
    gm = (gt_old + 0.1 * rng.standard_normal(d)).astype(F32)
    got_m = gpu_compress(torch, got["mean"][None], gm[None], gt_old[None], mc, 0.5, engine=got["engine"])
    ref_m = O.adacgd(gm, gt_old, gt_new, mc, 0.5)
    assert got_m["level"][0] == ref_m["level"] and got_m["bits"][0] == ref_m["bits"]
    assert_bitwise(got_m["G"][0], ref_m["out"], "gm")


def test_repeated_calls_are_deterministic_and_reuse_the_context(torch):
    X, G, Y = S.gaussian_rows(4, 33333, seed=7)
    a = gpu_compress(torch, X, G, Y, CANDS3, 1.0)
    b = gpu_compress(torch, X, G, Y, CANDS3, 1.0, engine=a["engine"])
    c = gpu_compress(torch, X[:2, :1000].copy(), G[:2, :1000].copy(), Y[:2, :1000].copy(), CANDS3, 1.0, engine=a["engine"])
    assert_bitwise(a["G"], b["G"], "G")
    assert np.array_equal(a["err"], b["err"]) and np.array_equal(a["level"], b["level"])
    G_ref, res = O.compress_rows(X[:2, :1000], G[:2, :1000], Y[:2, :1000], CANDS3, 1.0)
    assert_bitwise(c["G"], G_ref, "G small")


def test_nonfinite_rows_are_flagged_and_left_unchanged(torch):
    X, G, Y = S.gaussian_rows(3, 5000, seed=8)
    X[1, 77] = np.inf
    got = gpu_compress(torch, X, G, Y, CANDS3, 0.0)
    assert got["flags"] & 1
    assert got["level"][1] == 0
    assert_bitwise(got["G"][1], G[1], "flagged row")
    G_ref, res = O.compress_rows(X[[0, 2]], G[[0, 2]], Y[[0, 2]], CANDS3, 0.0)
    assert_bitwise(got["G"][[0, 2]], G_ref, "other rows")


def test_argument_errors(torch):
    import paper_2211_00188_b200 as pkg
    eng = pkg.AdaCGD(2, 100, CANDS3[:1], 1.0)
    X = torch.zeros(3, 100, device="cuda:0")
    with pytest.raises(pkg.AdacgdError) as e:
        eng.compress(X, X.clone(), X)
    assert e.value.status == 1
    X = torch.zeros(2, 100, device="cuda:0")
    with pytest.raises(pkg.AdacgdError) as e:
        eng.compress(X, X.clone(), X, [(TOPK, 9), (TOPK, 3)], 1.0)
    assert e.value.status == 2
    with pytest.raises(pkg.AdacgdError):
        eng.step(1)
    # the context reports the device it is bound to (the one that was current at adacgd_init)
    assert eng.get_state("device") == torch.cuda.current_device() == 0


@pytest.mark.parametrize("n", [1, 3, 6])
def test_host_entry_point(torch, n):
    # the rows travel in up to four groups, results going back while the next group comes in
    import paper_2211_00188_b200 as pkg
    d = 10000
    X, G, Y = S.gaussian_rows(n, d, seed=10)
    eng = pkg.AdaCGD(n, d, CANDS3, 1.0, host_staging=True)
    Xh, Gh, Yh = (torch.from_numpy(a.copy()).pin_memory() for a in (X, G, Y))
    mean = torch.zeros(d).pin_memory()
    level = torch.zeros(n, dtype=torch.int32).pin_memory()
    bits = torch.zeros(n, dtype=torch.int64).pin_memory()
    eng.compress_host(Xh, Gh, Yh, mean_out=mean, level=level, bits=bits)
    G_ref, res = O.compress_rows(X, G, Y, CANDS3, 1.0)
    assert_bitwise(Gh.numpy(), G_ref, "G")
    assert_bitwise(mean.numpy(), O.server_mean(G_ref), "mean")
    assert level.tolist() == [r["level"] for r in res] and bits.tolist() == [r["bits"] for r in res]


def sampled_granules(d):
    """The granules (16 consecutive entries) of a row of d entries that the sampling kernel reads:
    one per window of `win` granules, at an offset hashed from the window index."""
    ngran = (d + 15) // 16
    win = min(max(ngran // 8192, 1), 64)
    w = np.arange((ngran + win - 1) // win, dtype=np.uint64)
    h = (w * np.uint64(2654435761)) & np.uint64(0xFFFFFFFF)
    h ^= h >> np.uint64(15)
    h = (h * np.uint64(2246822519)) & np.uint64(0xFFFFFFFF)
    h ^= h >> np.uint64(13)
    span = np.minimum(np.uint64(ngran) - w * np.uint64(win), np.uint64(win))
    return (w * np.uint64(win) + h % span).astype(np.int64)


def test_single_pass_falls_back_when_the_sample_misleads(torch):
    # d = 1e6: one granule of 16 entries out of every 7 is sampled.  Large entries are placed
    # only in granules the sample never sees, so every bracket misses the true threshold and
    # the row must take the full radix select; the result may not change.
    d = 1_000_000
    X, G, Y = S.gaussian_rows(2, d, seed=31, drift=0.01, move=0.02)
    hidden = np.ones(d, dtype=bool)
    seen = sampled_granules(d)
    assert len(seen) == 8929 and len(np.unique(seen)) == len(seen) and seen.max() < 62500
    for k in range(16):
        hidden[np.minimum(seen * 16 + k, d - 1)] = False
    rng = np.random.Generator(np.random.PCG64(32))
    X[0, hidden] += (5.0 * rng.standard_normal(int(hidden.sum()))).astype(F32)
    got, _ = check_against_oracle(torch, X, G, Y, [(TOPK, 1000), (TOPK, 10000), (TOPK, 100000)], 0.5)
    assert got["fallbacks"] == 1          # row 0 only; row 1 is homogeneous


def side_path_rows():
    """Five rows of 1e6 entries that need, in ONE call, every side path of the single-pass route: a row whose sample
    misleads (full select), a row with a crowded threshold bin (list levels), a row of a few distinct magnitudes (list
    overflow, tie groups far larger than the ranking buffers), a row whose skip trigger holds with equality at
    zeta = 14.25 (exact sums), and an ordinary row."""
    d = 1_000_000
    X, G, Y = S.gaussian_rows(5, d, seed=61, drift=0.3, move=0.01)
    # row 0: large entries only where the sampling kernel never looks
    hidden = np.ones(d, dtype=bool)
    seen = sampled_granules(d)
    for k in range(16):
        hidden[np.minimum(seen * 16 + k, d - 1)] = False
    rng = np.random.Generator(np.random.PCG64(62))
    bump = (5.0 * rng.standard_normal(int(hidden.sum()))).astype(F32)
    X[0, hidden] += bump
    Y[0, hidden] += bump                                  # D stays small: the row does not skip
    # row 1: 30 000 magnitudes within a few units in the last place around the 1 % threshold
    v = (X[1] - G[1]).astype(F32)
    t = np.sort(np.abs(v))[-10_000]
    where = rng.choice(d, 30_000, replace=False)
    near = (F32(t) * (1.0 + 1e-7 * rng.integers(-3, 4, 30_000))).astype(F32) * rng.choice([-1.0, 1.0], 30_000).astype(F32)
    G[1, where] = 0.0
    X[1, where] = near
    Y[1, where] = near
    # row 2: small integers (seven magnitudes), Y equal to X but for 1000 entries
    Xt, Gt, _ = S.tie_vectors(1, d, seed=63, levels=3)
    X[2], G[2] = Xt[0], Gt[0]
    Y[2] = X[2]
    Y[2, :1000] += 1.0
    # row 3: ||v||^2 = 14.25 and D = 1 exactly
    X[3] = 0.0
    X[3, :4] = [3, -1, 2, 0.5]
    G[3] = 0.0
    Y[3] = X[3]
    Y[3, 0] -= 1.0
    return X, G, Y, [(TOPK, 1000), (TOPK, 10_000), (TOPK, 100_000)], 14.25


def test_all_side_paths_in_one_call(torch):
    # the cooperative side-path kernel with every phase needed at once, each by another row
    X, G, Y, cands, zeta = side_path_rows()
    got, res = check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)
    assert [r["level"] for r in res] == [3, 3, 3, 0, 3]
    assert got["fallbacks"] >= 2 and got["list_levels"] >= 1 and got["rechecks"] >= 1


def test_block_scaled_rows_keep_the_single_pass(torch):
    # contiguous blocks of very different scale (the structure of the c5 workload) at a size where
    # each block is only a few dozen tiles long: the sample must still bracket every threshold
    Xs, G0 = S.stress_vectors(2, 4_000_000, blocks=100, period=4, seed=36, device="cpu")
    got, _ = check_against_oracle(torch, Xs[1].numpy(), G0.numpy(), Xs[0].numpy(),
                                  [(TOPK, 4000), (TOPK, 40000), (TOPK, 400000)], 1.0)
    assert got["fallbacks"] == 0


def test_single_pass_list_overflow_falls_back(torch):
    # a few distinct magnitudes over 400k entries: any bracket holds far more keys than a list
    # segment can take, which must route the row through the full select
    X, G, Y = S.tie_vectors(2, 400_000, seed=33, levels=3)
    got, _ = check_against_oracle(torch, X, G, Y, [(TOPK, 400), (TOPK, 40000), (TOPK, 200000)], 1.0)
    assert got["fallbacks"] == 2


def test_single_pass_fallback_rows_with_quantisers(torch):
    # Top-K and quantiser candidates mixed, on rows that all fall back to the full select (their lists overflow) in a
    # shape where the fallback kernels run on fewer CTAs per row than the streaming pass: every error sum of a row
    # must be taken over the CTAs of the pass that wrote it.  zeta sits between one half and the whole of the 2-bit
    # quantiser's error, so that an error summed over too few CTAs would pass the trigger.
    X, G, Y = S.tie_vectors(40, 200_000, seed=37, levels=1)
    cands = [(TOPK, 100), (QUANT, 2), (TOPK, 50_000), (QUANT, 8)]
    got, res = check_against_oracle(torch, X, G, Y, cands, 0.25, both_update_paths=True)
    assert got["fallbacks"] == 40
    assert {r["level"] for r in res} == {4}
    # one long row: 367 CTAs in the streaming pass, 296 in the fallback kernels
    X, G, Y = S.tie_vectors(1, 3_000_000, seed=38, levels=1)
    cands = [(TOPK, 1000), (QUANT, 2), (TOPK, 750_000), (QUANT, 8)]
    got, res = check_against_oracle(torch, X, G, Y, cands, 0.25)
    assert got["fallbacks"] == 1 and res[0]["level"] == 4


def test_large_row_many_tiles(torch):
    X, G, Y = S.gaussian_rows(2, 3_000_001, seed=34)
    got, _ = check_against_oracle(torch, X, G, Y, [(TOPK, 3000), (TOPK, 30000), (TOPK, 300000)], 1.0)
    assert got["fallbacks"] == 0
    Xs, G0 = S.stress_vectors(2, 2_000_000, blocks=20, period=4, seed=35, device="cpu")
    check_against_oracle(torch, Xs[2].numpy(), G0.numpy(), Xs[1].numpy(),
                         [(TOPK, 2000), (TOPK, 20000), (TOPK, 200000)], 1.0)


@pytest.mark.parametrize("d", [5000, 70001, 600000])
def test_small_tie_groups_at_the_threshold(torch, d):
    # values on a grid of 1/256: a handful of equal magnitudes at every threshold, of which only the
    # lowest indices may be kept
    X, G, Y = S.gaussian_rows(3, d, seed=40 + d % 7)
    X, G, Y = (np.round(a * 256) / 256 for a in (X, G, Y))
    X, G, Y = X.astype(F32), G.astype(F32), Y.astype(F32)
    cands = [(TOPK, max(1, d // 1000)), (TOPK, d // 100), (TOPK, d // 10), (TOPK, d // 2)]
    for zeta in (0.0, 1.0):
        check_against_oracle(torch, X, G, Y, cands, zeta)


def test_nonfinite_rows_on_the_single_pass_path(torch):
    # large enough for the sampled single-pass pipeline: Inf in X - G (row 0), NaN only in X - Y (row 2)
    X, G, Y = S.gaussian_rows(3, 300_000, seed=41)
    X[0, 1234] = -np.inf
    Y[2, 99] = np.nan
    got = gpu_compress(torch, X, G, Y, [(TOPK, 300), (TOPK, 30000)], 1.0)
    assert got["flags"] & 1
    assert got["level"][0] == 0 and got["level"][2] == 0
    assert_bitwise(got["G"][[0, 2]], G[[0, 2]], "flagged rows")
    G_ref, res = O.compress_rows(X[[1]], G[[1]], Y[[1]], [(TOPK, 300), (TOPK, 30000)], 1.0)
    assert_bitwise(got["G"][[1]], G_ref, "clean row")
    assert got["level"][1] == res[0]["level"]


@pytest.mark.parametrize("d", [700_000, 700_001])
def test_single_pass_eight_candidates(torch, d):
    # the most brackets a set can have, on rows with and without 16-byte alignment; both update paths
    X, G, Y = S.gaussian_rows(2, d, seed=50)
    cands = [(TOPK, k) for k in (70, 700, 2000, 7000, 20000, 70000, 200000, 350000)]
    got, _ = check_against_oracle(torch, X, G, Y, cands, 1.0, both_update_paths=True)
    assert got["fallbacks"] == 0


def test_single_pass_many_short_rows(torch):
    # more rows than one tile of decisions holds, each only twenty tiles long (every element is sampled)
    X, G, Y = S.gaussian_rows(40, 20_000, seed=51)
    got, res = check_against_oracle(torch, X, G, Y, [(TOPK, 20), (TOPK, 200), (TOPK, 2000)], 0.5, both_update_paths=True)
    assert got["fallbacks"] == 0 and len({r["level"] for r in res}) >= 1


def test_single_pass_with_quantisers(torch):
    # quantisers need the row maximum first, so the level is picked by its own kernel after the list pass
    X, G, Y = S.gaussian_rows(2, 600_000, seed=52)
    cands = [(TOPK, 600), (QUANT, 2), (TOPK, 60000), (QUANT, 8)]
    for zeta in (0.05, 1.0):
        check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)


@pytest.mark.parametrize("d", [60_000, 60_001])
def test_single_pass_quantiser_errors_inside_the_streaming_pass(torch, d):
    # rows short enough that the sampling kernel reads every element: it then also yields the row maximum, and the
    # streaming pass evaluates up to three quantisers itself (no separate pass, level picked with the collection)
    X, G, Y = S.gaussian_rows(12, d, seed=55)
    X[3] *= 1e-3; G[3] *= 1e-3; Y[3] *= 1e-3                     # rows of different scale
    X[7, 11] = 40.0                                                # one dominant entry: coarse quantisers lose the rest
    cands = [(TOPK, 60), (QUANT, 2), (TOPK, 600), (QUANT, 4), (TOPK, 6000), (QUANT, 8)]
    seen = set()
    for zeta in (0.02, 0.3, 5.0, 8.5):
        got, res = check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)
        seen.update(r["level"] for r in res)
        assert got["fallbacks"] == 0
    assert seen >= {0, 2, 4, 6}                                    # skip, a Top-K level, two quantiser levels


def test_single_pass_crowded_threshold_bin(torch):
    # 30 000 magnitudes within a few units in the last place around the 1 % threshold: the first-digit bin of
    # that bracket holds far more keys than the collection buffer, so the row takes the three-level list passes
    d = 1_000_000
    X, G, Y = S.gaussian_rows(2, d, seed=53, drift=0.3, move=0.3)
    v = (X[0] - G[0]).astype(F32)
    t = np.sort(np.abs(v))[-10_000]                     # the 1 % threshold of row 0
    rng = np.random.Generator(np.random.PCG64(54))
    where = rng.choice(d, 30_000, replace=False)
    near = (F32(t) * (1.0 + 1e-7 * rng.integers(-3, 4, 30_000))).astype(F32) * rng.choice([-1.0, 1.0], 30_000).astype(F32)
    G[0, where] = 0.0
    X[0, where] = near                                   # v = X - 0 exactly
    got, _ = check_against_oracle(torch, X, G, Y, [(TOPK, 1000), (TOPK, 10_000), (TOPK, 100_000)], 1.0,
                                  both_update_paths=True)
    assert got["fallbacks"] == 0 and got["list_levels"] >= 1


def test_short_rows_random_sweep(torch):
    # seeded sweep over the short-row kernel: random shapes, candidate lists (Top-K up to and beyond d, quantisers,
    # in any admissible order), triggers, and a mix of continuous and tie-heavy rows
    rng = np.random.Generator(np.random.PCG64(77))
    for case in range(48):
        rows = int(rng.integers(1, 6))
        d = int(rng.choice([1, 2, 3, 4, 5, 31, 32, 33, 255, 256, 257, 1000, 1023, 1025, 2999]))
        if case % 3 == 0:
            X, G, Y = S.tie_vectors(rows, d, seed=1000 + case, levels=int(rng.integers(1, 6)))
        else:
            X, G, Y = S.gaussian_rows(rows, d, seed=1000 + case, drift=float(rng.choice([0.0, 0.01, 0.3])),
                                      move=float(rng.choice([0.0, 0.1])))
        if case % 5 == 0:
            Y = G.copy()                      # |X - G| == |X - Y| everywhere: the equality shortcut of the skip test
        ks = sorted(set(int(k) for k in rng.integers(1, max(2, 2 * d), size=int(rng.integers(0, 5)))))
        ks = [k for i, k in enumerate(ks) if i == 0 or ks[i - 1] < d]          # only the last Top-K may reach d
        qs = sorted(set(int(b) for b in rng.integers(2, 17, size=int(rng.integers(0, 3)))))
        cands, ki, qi = [], 0, 0
        while ki < len(ks) or qi < len(qs):    # interleave, each kind in increasing order
            take_k = ki < len(ks) and (qi >= len(qs) or rng.random() < 0.5)
            if take_k:
                cands.append((TOPK, ks[ki])); ki += 1
            else:
                cands.append((QUANT, qs[qi])); qi += 1
        cands = cands[:8]
        if not cands:
            cands = [(TOPK, 1)]
        zeta = float(rng.choice([0.0, 0.1, 1.0, 3.0, 1e30]))
        check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)


def test_single_pass_random_sweep(torch):
    # seeded sweep over the sampled single-pass pipeline: odd and even row lengths, heavy ties, rows equal to their
    # previous gradient, blocks of very different scale, quantisers mixed in, several triggers
    rng = np.random.Generator(np.random.PCG64(88))
    for case in range(8):
        rows = int(rng.integers(1, 4))
        d = int(rng.choice([524_288, 600_001, 750_000, 1_000_003])) // (1 if rows == 1 else 1)
        kind = case % 4
        if kind == 0:
            X, G, Y = S.gaussian_rows(rows, d, seed=2000 + case)
        elif kind == 1:   # values on a coarse grid: tie groups at every threshold
            X, G, Y = S.gaussian_rows(rows, d, seed=2000 + case)
            X, G, Y = ((np.round(a * 64) / 64).astype(F32) for a in (X, G, Y))
        elif kind == 2:   # contiguous blocks of very different scale
            X, G, Y = S.gaussian_rows(rows, d, seed=2000 + case)
            scale = np.repeat(np.exp(2.0 * rng.standard_normal(50)), -(-d // 50))[:d].astype(F32)
            X, G, Y = (a * scale for a in (X, G, Y))
        else:             # most of the row unchanged since the last round
            X, G, Y = S.gaussian_rows(rows, d, seed=2000 + case)
            same = rng.random(d) < 0.9
            G[:, same] = X[:, same]
        ks = sorted(set(int(k) for k in (d * np.array([1e-4, 1e-3, 1e-2, 0.1, 0.5]) * rng.uniform(0.5, 1.5, 5))))
        ks = [k for k in ks if 0 < k < d][:int(rng.integers(1, 6))]
        cands = [(TOPK, k) for k in ks]
        if case % 2 == 1:
            cands.insert(int(rng.integers(0, len(cands) + 1)), (QUANT, int(rng.integers(2, 9))))
        zeta = float(rng.choice([0.0, 0.3, 1.0, 4.0]))
        check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)


def test_three_pass_random_sweep(torch):
    # seeded sweep over the mid-size route (rows too long for the short-row kernel, problem too small for the
    # sampled pipeline): aligned and unaligned rows, ties, quantisers, identity as the last candidate
    rng = np.random.Generator(np.random.PCG64(99))
    for case in range(8):
        d = int(rng.choice([32_769, 40_000, 65_537, 100_000, 131_071]))
        rows = int(rng.integers(1, max(2, min(5, (1 << 19) // d))))
        if case % 3 == 1:
            X, G, Y = S.tie_vectors(rows, d, seed=3000 + case, levels=3)
        else:
            X, G, Y = S.gaussian_rows(rows, d, seed=3000 + case, drift=float(rng.choice([0.01, 0.3])))
        ks = sorted(set(int(k) for k in (d * np.array([1e-4, 1e-2, 0.2, 1.0]) * rng.uniform(0.6, 1.4, 4))))
        ks = [k for i, k in enumerate(ks) if k > 0 and (i == 0 or ks[i - 1] < d)]
        cands = [(TOPK, k) for k in ks]
        if case % 2 == 0:
            cands.insert(int(rng.integers(0, len(cands) + 1)), (QUANT, int(rng.integers(2, 17))))
        zeta = float(rng.choice([0.0, 0.5, 1.0, 1e30]))
        check_against_oracle(torch, X, G, Y, cands, zeta, both_update_paths=True)


@pytest.mark.parametrize("cands", [[], [(TOPK, 7), (QUANT, 4), (TOPK, 9999)]])
def test_host_entry_point_unaligned_and_identity(torch, cands):
    import paper_2211_00188_b200 as pkg
    n, d = 5, 9999
    X, G, Y = S.gaussian_rows(n, d, seed=12)
    eng = pkg.AdaCGD(n, d, cands, 0.7, host_staging=True)
    Xh, Gh, Yh = (torch.from_numpy(a.copy()).pin_memory() for a in (X, G, Y))
    mean = torch.zeros(d).pin_memory()
    level = torch.full((n,), -3, dtype=torch.int32).pin_memory()
    eng.compress_host(Xh, Gh, Yh, mean_out=mean, level=level)
    if cands:
        G_ref, res = O.compress_rows(X, G, Y, cands, 0.7)
        assert level.tolist() == [r["level"] for r in res]
    else:
        G_ref = X.copy()                      # the identity compressor sends the gradient itself
    assert_bitwise(Gh.numpy(), G_ref, "G")
    assert_bitwise(mean.numpy(), O.server_mean(G_ref), "mean")


# ---------------------------------------------------------------- triggers other than Eq. 10 (Definition 3)
PRED_LAZY, PRED_ABSOLUTE, PRED_RELATIVE, PRED_NEVER, PRED_ALWAYS = 0, 1, 2, 3, 4


def check_menu_against_oracle(torch, X, G, Y, cands, preds):
    import paper_2211_00188_b200 as pkg
    rows, d = X.shape
    dev = torch.device("cuda:0")
    eng = pkg.AdaCGD(rows, d, cands, 1.0)
    Xd, Gd, Yd = (torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in (X, G, Y))
    level = torch.full((rows,), -7, dtype=torch.int32, device=dev)
    bits = torch.zeros(rows, dtype=torch.int64, device=dev)
    mean = torch.zeros(d, dtype=torch.float32, device=dev)
    eng.compress(Xd, Gd, Yd, cands, 1.0, mean_out=mean, level=level, bits=bits, preds=preds)
    torch.cuda.synchronize()
    refs = [O.adaptive_3pc(G[i], Y[i], X[i], cands, preds) for i in range(rows)]
    assert level.cpu().tolist() == [r["level"] for r in refs], (preds, level.cpu().tolist(), [r["level"] for r in refs])
    assert bits.cpu().tolist() == [r["bits"] for r in refs]
    G_ref = np.stack([r["out"] for r in refs])
    assert_bitwise(Gd.cpu().numpy(), G_ref, "G")
    assert_bitwise(mean.cpu().numpy(), O.server_mean(G_ref), "mean")
    return [r["level"] for r in refs], eng


@pytest.mark.parametrize("rows,d", [(3, 900), (2, 70_001), (3, 600_000)])
def test_trigger_menu_on_every_route(torch, rows, d):
    # the conditions of Definition 3 the library evaluates, on the short-row kernel, the three-pass route and the
    # sampled single-pass pipeline: absolute budgets, fractions of ||x - h||^2, per-level zeta, never / always
    X, G, Y = S.gaussian_rows(rows, d, seed=70 + rows)
    cands = [(TOPK, max(1, d // 1000)), (TOPK, d // 100), (QUANT, 4), (TOPK, d // 10)]
    e0 = O.sumsq((X[0] - G[0]).astype(F32))
    seen = set()
    for preds in ([(PRED_NEVER, 0.0)] + [(PRED_ABSOLUTE, 0.995 * e0)] * 3,
                  [(PRED_ABSOLUTE, 0.5 * e0)] * 4,
                  [(PRED_RELATIVE, 0.97), (PRED_RELATIVE, 0.97), (PRED_RELATIVE, 0.8), (PRED_RELATIVE, 0.05)],
                  [(PRED_RELATIVE, 1.0)] * 4,
                  [(PRED_NEVER, 0.0), (PRED_LAZY, 5.0), (PRED_LAZY, 2.0), (PRED_LAZY, 0.1)],
                  [(PRED_LAZY, 0.5), (PRED_NEVER, 0.0), (PRED_ALWAYS, 0.0), (PRED_NEVER, 0.0)],
                  [(PRED_NEVER, 0.0)] * 4,
                  [(PRED_LAZY, 0.0), (PRED_ABSOLUTE, 0.0), (PRED_RELATIVE, 0.0), (PRED_RELATIVE, 0.3)]):
        lv, _ = check_menu_against_oracle(torch, X, G, Y, cands, preds)
        seen.update(lv)
    assert seen == {0, 1, 2, 3, 4}


def test_trigger_menu_equalities_take_the_exact_path(torch):
    # small integers: the budgets are met with equality or missed by one unit in the last place of the sum
    X, G, Y = S.tie_vectors(4, 5000, seed=75)
    cands = [(TOPK, 50), (TOPK, 500), (TOPK, 2500)]
    errs = [O.adaptive_3pc(G[0], Y[0], X[0], cands, [(PRED_NEVER, 0.0)] * 3)["err"]][0]
    rechecks = 0
    for target in (1, 2):
        for tweak in (0.0, -1.0, 1.0):
            budget = float(np.float32(errs[target] + tweak))      # integers below 2^24: exact in binary32
            preds = [(PRED_NEVER, 0.0)] + [(PRED_ABSOLUTE, budget)] * 2
            lv, eng = check_menu_against_oracle(torch, X, G, Y, cands, preds)
            rechecks += eng.get_state("rechecks")
    preds = [(PRED_RELATIVE, 1.0), (PRED_RELATIVE, 0.5), (PRED_RELATIVE, 0.5)]
    check_menu_against_oracle(torch, X, G, Y, cands, preds)
    assert rechecks > 0


def test_trigger_menu_argument_errors(torch):
    import paper_2211_00188_b200 as pkg
    eng = pkg.AdaCGD(2, 100, CANDS3[:2], 1.0)
    X = torch.zeros(2, 100, device="cuda:0")
    with pytest.raises(pkg.AdacgdError) as e:
        eng.compress(X, X.clone(), X, CANDS3[:2], 1.0, preds=[(9, 1.0), (PRED_LAZY, 1.0)])
    assert e.value.status == 1
    with pytest.raises(pkg.AdacgdError) as e:
        eng.compress(X, X.clone(), X, CANDS3[:2], 1.0, preds=[(PRED_ABSOLUTE, -1.0), (PRED_LAZY, 1.0)])
    assert e.value.status == 1
    with pytest.raises(ValueError):
        eng.compress(X, X.clone(), X, CANDS3[:2], 1.0, preds=[(PRED_LAZY, 1.0)])
