"""adacgd_compress_noalloc: the compression step for callers that are not allowed to
allocate device memory (they are only handed buffers, e.g. a plug-in inside an
application whose allocator already owns the whole GPU).  It must give exactly what
adacgd_compress gives, call after call, although all its calls share one built-in
scratch array that still holds the previous call's contents."""
import numpy as np
import pytest

import synthetic_inputs as S
from oracle import adacgd_oracle as O

pytestmark = pytest.mark.gpu
TOPK, QUANT = 0, 1


def run_both(torch, pkg, X, G, Y, cands, zeta):
    dev = torch.device("cuda:0")
    rows, d = X.shape
    out = []
    for which in ("workspace", "noalloc"):
        Xd, Gd, Yd = (torch.from_numpy(a.copy()).to(dev) for a in (X, G, Y))
        mean = torch.zeros(d, device=dev)
        level = torch.full((rows,), -1, dtype=torch.int32, device=dev)
        bits = torch.zeros(rows, dtype=torch.int64, device=dev)
        if which == "workspace":
            eng = pkg.AdaCGD(rows, d, cands, zeta)
            eng.compress(Xd, Gd, Yd, mean_out=mean, level=level, bits=bits)
        else:
            pkg.compress_noalloc(Xd, Gd, Yd, cands, zeta, mean_out=mean, level=level, bits=bits)
        torch.cuda.synchronize()
        out.append((Gd.cpu().numpy(), mean.cpu().numpy(), level.cpu().tolist(), bits.cpu().tolist()))
    return out


def test_noalloc_matches_workspace_entry_point_on_consecutive_calls():
    import torch
    import paper_2211_00188_b200 as pkg

    # two calls in a row with different shapes, data and candidate sets: the second one
    # starts from a scratch array full of the first one's histograms and records
    calls = [
        (S.gaussian_rows(4, 50000, seed=21), [(TOPK, 50), (TOPK, 500), (TOPK, 5000)], 1.0),
        (S.tie_vectors(3, 7001, seed=22), [(TOPK, 7), (QUANT, 3), (TOPK, 700), (QUANT, 8)], 0.5),
        (S.gaussian_rows(1, 300, seed=23), [(TOPK, 3), (TOPK, 300)], 0.0),
    ]
    levels_seen = set()
    for (X, G, Y), cands, zeta in calls:
        (G0, m0, l0, b0), (G1, m1, l1, b1) = run_both(torch, pkg, X, G, Y, cands, zeta)
        assert l0 == l1 and b0 == b1
        assert np.array_equal(G0.view(np.uint32), G1.view(np.uint32))
        assert np.array_equal(m0.view(np.uint32), m1.view(np.uint32))
        assert not np.array_equal(G1, G) or set(l1) == {0}
        levels_seen.update(l1)
    assert len(levels_seen) >= 2


def noalloc_against_oracle(torch, pkg, X, G, Y, cands, zeta):
    dev = torch.device("cuda:0")
    rows, d = X.shape
    Xd, Gd, Yd = (torch.from_numpy(a.copy()).to(dev) for a in (X, G, Y))
    mean = torch.zeros(d, device=dev)
    level = torch.full((rows,), -1, dtype=torch.int32, device=dev)
    bits = torch.zeros(rows, dtype=torch.int64, device=dev)
    pkg.compress_noalloc(Xd, Gd, Yd, cands, zeta, mean_out=mean, level=level, bits=bits)
    torch.cuda.synchronize()
    G_ref, res = O.compress_rows(X, G, Y, cands, zeta)
    assert level.cpu().tolist() == [r["level"] for r in res]
    assert bits.cpu().tolist() == [r["bits"] for r in res]
    assert np.array_equal(Gd.cpu().numpy().view(np.uint32), G_ref.view(np.uint32))
    assert np.array_equal(mean.cpu().numpy().view(np.uint32), O.server_mean(G_ref).view(np.uint32))
    return [r["level"] for r in res]


def test_noalloc_matches_the_oracle_at_the_maximum_shape_and_unaligned():
    # the largest shape the built-in scratch takes, on heavy-tailed block-scaled rows, then (the scratch now
    # full of that call's tables) rows whose length is not a multiple of four, with ties and quantisers
    import torch
    import paper_2211_00188_b200 as pkg

    n, d = pkg.NOALLOC_MAX_ROWS, pkg.NOALLOC_MAX_D
    Xs, G0 = S.stress_vectors(n, d, blocks=64, period=4, seed=24, device="cpu")
    lv = noalloc_against_oracle(torch, pkg, Xs[1].numpy(), G0.numpy(), Xs[0].numpy(),
                                [(TOPK, d // 1000), (TOPK, d // 100), (TOPK, d // 10)], 1.0)
    assert any(l > 0 for l in lv)
    X, G, Y = S.gaussian_rows(3, 100_003, seed=25)
    X, G, Y = (np.round(a * 64) / 64 for a in (X, G, Y))          # a few equal magnitudes at every threshold
    lv = noalloc_against_oracle(torch, pkg, X.astype(np.float32), G.astype(np.float32), Y.astype(np.float32),
                                [(TOPK, 100), (QUANT, 3), (TOPK, 10_000), (QUANT, 8)], 0.3)
    assert any(l > 0 for l in lv)


def test_noalloc_leaves_a_nonfinite_row_unchanged_at_level_zero():
    # there is no context to hold a status word: a row with Inf or NaN is reported through its level (0)
    # and an untouched estimator, the other rows are compressed as usual
    import torch
    import paper_2211_00188_b200 as pkg

    X, G, Y = S.gaussian_rows(3, 40_000, seed=26)
    X[1, 77] = np.inf
    cands = [(TOPK, 40), (TOPK, 4000)]
    dev = torch.device("cuda:0")
    Xd, Gd, Yd = (torch.from_numpy(a.copy()).to(dev) for a in (X, G, Y))
    level = torch.full((3,), -1, dtype=torch.int32, device=dev)
    pkg.compress_noalloc(Xd, Gd, Yd, cands, 0.0, level=level)
    torch.cuda.synchronize()
    got = Gd.cpu().numpy()
    assert level.cpu().tolist()[1] == 0 and np.array_equal(got[1].view(np.uint32), G[1].view(np.uint32))
    G_ref, res = O.compress_rows(X[[0, 2]], G[[0, 2]], Y[[0, 2]], cands, 0.0)
    assert [level.cpu().tolist()[i] for i in (0, 2)] == [r["level"] for r in res] == [2, 2]
    assert np.array_equal(got[[0, 2]].view(np.uint32), G_ref.view(np.uint32))


def test_noalloc_rejects_shapes_beyond_the_builtin_scratch():
    import torch
    import paper_2211_00188_b200 as pkg

    dev = torch.device("cuda:0")
    too_many_rows = torch.zeros(pkg.NOALLOC_MAX_ROWS + 1, 64, device=dev)
    with pytest.raises(pkg.AdacgdError) as e:
        pkg.compress_noalloc(too_many_rows, too_many_rows.clone(), too_many_rows, [(TOPK, 4)], 1.0)
    assert e.value.status == 1 and "ADACGD_NOALLOC_MAX_ROWS" in str(e.value)
    too_wide = torch.zeros(1, pkg.NOALLOC_MAX_D + 4, device=dev)
    with pytest.raises(pkg.AdacgdError) as e:
        pkg.compress_noalloc(too_wide, too_wide.clone(), too_wide, [(TOPK, 4)], 1.0)
    assert e.value.status == 1
    widest = torch.zeros(pkg.NOALLOC_MAX_ROWS, pkg.NOALLOC_MAX_D, device=dev)
    pkg.compress_noalloc(widest, widest.clone(), widest, [(TOPK, 4)], 1.0)   # the stated maximum fits
    torch.cuda.synchronize()
