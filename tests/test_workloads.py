"""The input generators: partitions, placements, attacks, and the E[q_hat] closed forms of the paper."""
import os

import numpy as np
import pytest
import torch

import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "qhat_r3_closed_form.txt")


def test_groups_and_sets_are_partitions():
    rng = np.random.default_rng(0)
    m = wl.make_groups(45, 3, rng)
    assert sorted(m.tolist()) == list(range(45))
    offs, sm = wl.make_sets(15, 5, rng)
    assert offs.tolist() == [0, 5, 10, 15] and sorted(sm.tolist()) == list(range(15))
    offs, sm = wl.make_sets(15, 7, rng)                      # 7 and 8 (Appendix B.1)
    assert offs.tolist() == [0, 7, 15]
    offs, sm = wl.make_sets(15, None, rng)
    assert offs.tolist() == [0, 15]


def test_r3_closed_form_matches_golden_and_general_formula():
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        p, q, val = line.split()
        p, q = int(p), int(q)
        closed = (p / 3) * q * (q - 1) * (3 * p - 2 * q - 2) / (p * (p - 1) * (p - 2))
        assert abs(closed - float(val)) < 5e-5
        assert abs(wl.expected_byzantine_votes(p, q, 3) - closed) < 1e-12


@pytest.mark.parametrize("p,q,r", [(45, 5, 3), (45, 9, 3), (105, 15, 3), (45, 9, 5)])
def test_random_placement_matches_expected_byzantine_votes(p, q, r):
    rng = np.random.default_rng(123)
    members = wl.make_groups(p, r, rng)
    trials = 20000
    tot = 0
    groups = members.reshape(p // r, r)
    for _ in range(trials):
        byz = wl.place_byzantine(p, r, q, members, "random", rng)
        tot += int((byz[groups].sum(axis=1) > r // 2).sum())
    mean = tot / trials
    exp = wl.expected_byzantine_votes(p, q, r)
    assert abs(mean - exp) < 5 * np.sqrt(max(exp, 0.05) / trials) + 0.01


def test_placements():
    rng = np.random.default_rng(1)
    members = wl.make_groups(45, 3, rng)
    groups = members.reshape(15, 3)
    byz = wl.place_byzantine(45, 3, 5, members, "worst", rng)
    per = np.sort(byz[groups].sum(axis=1))[::-1]
    assert byz.sum() == 5 and per[:4].tolist() == [2, 1, 1, 1] and per[4:].sum() == 0
    byz = wl.place_byzantine(45, 3, 5, members, "distinct", rng)
    assert byz.sum() == 5 and byz[groups].sum(axis=1).max() == 1


def test_workload_rows_copies_and_attacks():
    spec = wl.WorkloadSpec("t", n=15, r=3, d=1001, sigma=0.01, q=2, attack="reverse", placement="distinct", seed=3)
    w = wl.make_workload(spec)
    assert w.ld % 32 == 0 and w.X.shape == (15, w.ld) and not w.X[:, spec.d:].any()
    X = w.data().numpy()
    for j in range(w.G):
        grp = w.members[j * 3:(j + 1) * 3]
        h = w.honest_member[j]
        for i in grp:
            if w.byzantine[i]:
                assert np.array_equal(X[i], np.float32(-100.0) * X[h])
            else:
                assert X[i].tobytes() == X[h].tobytes()
    assert w.q_hat == 0
    assert abs(float(X[w.honest_member[0]].std()) - 0.01) < 1e-3

    spec = wl.WorkloadSpec("t", n=45, r=3, d=500, sigma=1e-3, q=5, attack="alie", placement="worst", set_size=5, seed=4)
    w = wl.make_workload(spec)
    X = w.data().numpy().astype(np.float64)
    hon = X[~w.byzantine]
    v = (hon.mean(0) - hon.std(0)).astype(np.float32)
    for i in np.nonzero(w.byzantine)[0]:
        np.testing.assert_allclose(w.data().numpy()[i], v, rtol=1e-6, atol=1e-12)
    assert w.q_hat == 1 and w.S == 3

    # same seed, same bits
    w2 = wl.make_workload(spec)
    assert torch.equal(w.X, w2.X) and np.array_equal(w.members, w2.members)


def test_named_configs_shapes():
    c = wl.CONFIGS
    assert (c["cfg1"].n, c["cfg1"].d, c["cfg1"].q) == (15, 100_000, 2)
    assert (c["cfg2"].n, c["cfg2"].d, c["cfg2"].q, c["cfg2"].attack) == (45, 11_173_962, 5, "alie")
    assert (c["cfg3"].q, c["cfg3"].attack) == (9, "reverse")
    assert (c["cfg4"].n, c["cfg4"].d, c["cfg4"].q, c["cfg4"].coord_scales) == (105, 28_000_000, 15, True)
    assert len(wl.sweep_specs()) == 4 * 3 * 2


def test_mean_estimation_inputs_follow_the_papers_recipe():
    # Section 5.3, "Mean estimation on synthetic data": p = 220000, r = 11, q = floor(e^11 / 3) = 19958
    import math
    w = wl.make_mean_estimation(d=20, p=22_000, r=11, seed=1)
    assert w.q == math.floor(math.exp(11) / 3) == 19958                   # q does not depend on p
    w = wl.make_mean_estimation(d=30, p=2200, r=11, q=200, n_sets=7, seed=1)
    X = w.X.numpy()
    assert X.shape == (2200, 30) and sorted(w.members.tolist()) == list(range(2200))
    assert int(w.byzantine.sum()) == 200
    np.testing.assert_allclose(np.linalg.norm(X[w.byzantine], axis=1), 100.0, rtol=1e-6)
    groups = w.members.reshape(-1, 11)
    for grp in groups[:20]:
        hon = [i for i in grp if not w.byzantine[i]]
        assert all(np.array_equal(X[hon[0]], X[i]) for i in hon)          # bitwise copies inside a group
    # honest vectors are means of 20 draws of N(0, I): variance 1/20 per coordinate
    hon_rows = X[~w.byzantine]
    assert abs(hon_rows.var() - 1 / 20) < 0.005
    assert w.set_offsets[0] == 0 and w.set_offsets[-1] == 200 and len(w.set_offsets) == 8
    assert set(np.diff(w.set_offsets).tolist()) <= {28, 29}
