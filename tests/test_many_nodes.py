"""GPU parity of the path for very many nodes with short vectors (Section 5.3, "Mean estimation on synthetic
data": p = 220,000 nodes, r = 11, q = floor(e^r / 3), d in 20 .. 100): vote -> mean inside runs of consecutive groups
-> geometric median / coordinate median over the set means, against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_12205_b200 as dx
import workloads as wl
from helpers import rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5


def bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


def run(w, r):
    X = w.X.to(DEV)
    members = torch.as_tensor(w.members, device=DEV)
    M, win = dx.detox_vote_hier_mean_many(X, r, members, w.set_offsets)
    Xh = w.X.cpu().numpy()
    Zo, wo = oracle.vote(Xh, w.members, r)
    G = len(wo)
    Mo = oracle.hier_mean(Zo, w.set_offsets, np.arange(G, dtype=np.int32))
    assert win.cpu().numpy().tolist() == wo.tolist()
    assert rel_l2(M.cpu().numpy(), Mo) <= TOL
    return X, members, M, Zo, wo, Mo


@pytest.mark.parametrize("d", [20, 100])
def test_the_papers_synthetic_experiment_at_full_size(d):
    w = wl.make_mean_estimation(d=d, seed=d)
    assert w.p == 220_000 and w.q == 19_958
    X, members, M, Zo, wo, Mo = run(w, 11)
    # the filter leaves a handful of Byzantine votes at most (Theorem 1): the estimate stays near the true mean, zero
    gm = dx.agg_geometric_median(M, iters=32)
    assert rel_l2(gm.cpu().numpy(), oracle.geometric_median(Mo, iters=32)) <= TOL
    med = dx.agg_coord_median(M)
    assert np.array_equal(bits(med), oracle.coord_median(M.cpu().numpy()).view(np.uint32))
    assert float(torch.linalg.vector_norm(gm)) < 1.0 and float(torch.linalg.vector_norm(med)) < 1.0
    # votes only
    _, win2 = dx.detox_vote_hier_mean_many(X, 11, members)
    assert win2.cpu().numpy().tolist() == wo.tolist()


@pytest.mark.parametrize("r,G,d,q", [(1, 40, 7, 0), (3, 1000, 33, 300), (5, 64, 1, 60), (15, 10, 1024, 40), (11, 300, 100, 1500)])
def test_small_shapes_with_groups_that_have_no_majority(r, G, d, q):
    w = wl.make_mean_estimation(d=d, p=r * G, r=r, q=q, n_sets=min(G, 7), seed=r + G)
    if r >= 5:                                   # three different values inside group 0: no majority
        grp = w.members[:r]
        for t, i in enumerate(grp[: r // 2 + 1]):
            w.X[int(i), d - 1] = float(t + 1) * 3.0
    _, _, _, _, wo, _ = run(w, r)
    if r >= 5:
        assert wo[0] == -1
