"""Parity at the benchmark's full size (workload c5: 8 rows of 25e6 entries, the launch
configuration bench.py times): one sampled worker row and the master row are checked against
the oracle bit for bit; every other row through properties that hold at any size."""
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

    # one worker row and the master row against the oracle
    i = 3
    ref = O.adacgd(G_before[i].cpu().numpy(), Y[i].cpu().numpy(), X[i].cpu().numpy(), W["worker"], 1.0)
    assert levels[i] == ref["level"] and int(bits[i]) == ref["bits"]
    assert np.array_equal(Gh[i].view(np.uint32), ref["out"].view(np.uint32))
    mref = O.adacgd(gm_before[0].cpu().numpy(), gt_old.cpu().numpy(), gt_new.cpu().numpy(), W["master"], 1.0)
    assert int(mlevel.item()) == mref["level"]
    assert np.array_equal(gm[0].cpu().numpy().view(np.uint32), mref["out"].view(np.uint32))
