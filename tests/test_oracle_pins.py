"""Pins for the CPU oracle: each part is checked against something other than itself.

vote        : honest-majority invariant (Section 3.1), no-majority => 0 (Section 3), brute force over
              member subsets, whole-vector / bitwise semantics.
hier mean   : exact integer closed forms, reduction to the plain mean of Section 2.
median      : counting definition by brute force, library median, ordering of special values.
distances   : library fp64 distances, symmetry, exact power-of-two scaling.
Krum family : brute-force subset definitions on tiny inputs, hand-worked examples, reductions.
"""
import itertools

import numpy as np
import pytest

import oracle


def rng(seed=0):
    return np.random.default_rng(seed)


# ----------------------------------------------------------------------------------------- vote

@pytest.mark.parametrize("r", [1, 3, 5, 7])
def test_vote_honest_majority_returns_honest_gradient_exactly(r):
    g = rng(1)
    G, d = 6, 37
    n = G * r
    members = g.permutation(n).astype(np.int32)
    honest = g.standard_normal((G, d)).astype(np.float32)
    X = np.empty((n, d), np.float32)
    exp_w = []
    for j in range(G):
        grp = members[j * r:(j + 1) * r]
        nbyz = g.integers(0, (r - 1) // 2 + 1)          # at most floor((r-1)/2) Byzantine members
        byz = set(g.choice(grp, size=nbyz, replace=False).tolist())
        for i in grp:
            X[i] = honest[j]
            if int(i) in byz:
                X[i] = -100.0 * honest[j] if g.random() < 0.5 else 7.0  # colluding or not: still a minority
        exp_w.append(min(int(i) for i in grp if int(i) not in byz))
    Z, w = oracle.vote(X, members, r)
    assert Z.tobytes() == honest.tobytes()
    assert w.tolist() == exp_w


def test_vote_no_majority_gives_zero():
    d = 5
    X = np.arange(3 * d, dtype=np.float32).reshape(3, d)          # three different rows
    Z, w = oracle.vote(X, [0, 1, 2], 3)
    assert w.tolist() == [-1] and not Z.any()
    # r = 5 split 2-2-1: a plurality is not a majority
    a, b, c = np.ones(d, np.float32), 2 * np.ones(d, np.float32), 3 * np.ones(d, np.float32)
    X5 = np.stack([a, b, a, b, c])
    Z, w = oracle.vote(X5, [0, 1, 2, 3, 4], 5)
    assert w.tolist() == [-1] and not Z.any()
    # 3-1-1 is a majority
    X5 = np.stack([c, a, b, a, a])
    Z, w = oracle.vote(X5, [0, 1, 2, 3, 4], 5)
    assert w.tolist() == [1] and np.array_equal(Z[0], a)


def test_vote_byzantine_majority_wins_when_colluding():
    d = 9
    g = rng(2).standard_normal(d).astype(np.float32)
    bad = (-100 * g).astype(np.float32)
    X = np.stack([bad, g, bad])
    Z, w = oracle.vote(X, [0, 1, 2], 3)
    assert w.tolist() == [0] and Z[0].tobytes() == bad.tobytes()


def test_vote_is_whole_vector_and_bitwise():
    d = 11
    g = rng(3).standard_normal(d).astype(np.float32)
    h = g.copy(); h[-1] = np.nextafter(h[-1], np.float32(np.inf))       # differs in the last coordinate only
    k = g.copy(); k[0] = np.nextafter(k[0], np.float32(np.inf))         # differs in the first one only
    Z, w = oracle.vote(np.stack([g, h, k]), [0, 1, 2], 3)
    assert w.tolist() == [-1]
    z = np.zeros(d, np.float32); nz = z.copy(); nz[4] = -0.0             # -0.0 and +0.0 are different words
    Z, w = oracle.vote(np.stack([z, nz, nz]), [0, 1, 2], 3)
    assert w.tolist() == [1] and np.signbit(Z[0, 4])
    q = g.copy(); q[2] = np.nan                                          # same NaN payload: equal as bits
    Z, w = oracle.vote(np.stack([q, g, q.copy()]), [0, 1, 2], 3)
    assert w.tolist() == [0] and np.isnan(Z[0, 2])


def test_vote_brute_force_tiny():
    g = rng(4)
    for trial in range(200):
        r = int(g.choice([3, 5]))
        G = int(g.integers(1, 4)) if r == 3 else 1
        n, d = G * r, int(g.integers(1, 9))
        members = g.permutation(n).astype(np.int32)
        X = g.integers(0, 2, size=(n, d)).astype(np.float32)              # small alphabet => coincidences
        Z, w = oracle.vote(X, members, r)
        for j in range(G):
            grp = sorted(int(i) for i in members[j * r:(j + 1) * r])
            found = None
            for size in range(r // 2 + 1, r + 1):
                for sub in itertools.combinations(grp, size):
                    if all(np.array_equal(X[sub[0]], X[s]) for s in sub):
                        cand = min(i for i in grp if np.array_equal(X[i], X[sub[0]]))
                        found = cand if found is None else found
                        assert found == cand                              # a strict majority is unique
            if found is None:
                assert w[j] == -1 and not Z[j].any()
            else:
                assert w[j] == found and np.array_equal(Z[j], X[found])


# ----------------------------------------------------------------------------------- hier mean

def test_hier_mean_exact_integers_uneven_sets():
    G, d = 15, 6
    Z = rng(5).integers(-1000, 1000, size=(G, d)).astype(np.float32)
    perm = rng(6).permutation(G).astype(np.int32)
    offs = np.array([0, 7, 15], np.int32)                                 # 7 and 8 out of 15 (Appendix B.1)
    M = oracle.hier_mean(Z, offs, perm)
    for s in range(2):
        idx = perm[offs[s]:offs[s + 1]]
        exp = (Z[idx].astype(np.int64).sum(0) / len(idx)).astype(np.float32)
        assert np.array_equal(M[s], exp)


def test_hier_mean_single_set_is_plain_mean_and_zero_rows_count():
    G, d = 5, 1000
    Z = rng(7).standard_normal((G, d)).astype(np.float32)
    Z[3] = 0.0                                                            # a no-majority vote is an ordinary member
    M = oracle.hier_mean(Z, [0, G], np.arange(G))
    exp = (Z.astype(np.float64).sum(0) / G).astype(np.float32)
    assert np.array_equal(M[0], exp)
    assert np.array_equal(oracle.mean_rows(Z), exp)


# -------------------------------------------------------------------------------------- median

@pytest.mark.parametrize("m", [1, 2, 3, 4, 5, 7, 8, 15, 16, 45, 105])
def test_median_matches_library_median(m):
    X = rng(m).standard_normal((m, 257)).astype(np.float32)
    got = oracle.coord_median(X)
    if m % 2:
        assert np.array_equal(got, np.median(X, axis=0))
    else:
        s = np.sort(X, axis=0)
        assert np.array_equal(got, (s[m // 2 - 1] + s[m // 2]) * np.float32(0.5))


def test_median_counting_definition_brute_force():
    g = rng(11)
    for m in (3, 5, 7, 9):
        X = g.integers(-3, 4, size=(m, 64)).astype(np.float32)            # many ties
        got = oracle.coord_median(X)
        for c in range(X.shape[1]):
            col = X[:, c]
            assert got[c] in col
            assert (col < got[c]).sum() <= (m - 1) // 2 and (col > got[c]).sum() <= (m - 1) // 2


def test_median_total_order_on_special_values():
    nan, inf = np.float32(np.nan), np.float32(np.inf)
    nnan = np.float32(-np.nan) if np.signbit(np.float32(-np.nan)) else -nan
    # ascending under the convention: -NaN < -Inf < -1 < -0 < +0 < 1 < +Inf < +NaN
    ladder = np.array([np.copysign(nan, -1), -inf, -1.0, -0.0, 0.0, 1.0, inf, nan], np.float32)
    for lo in range(len(ladder) - 2):
        col = ladder[[lo + 2, lo, lo + 1]].reshape(3, 1)                   # shuffled triple
        got = oracle.coord_median(col)[0]
        assert got.tobytes() == ladder[lo + 1].tobytes()
    assert nnan is not None


def test_median_row_subset():
    X = rng(12).standard_normal((9, 33)).astype(np.float32)
    rows = [7, 2, 5]
    assert np.array_equal(oracle.coord_median(X, rows), np.median(X[rows], axis=0))


# ----------------------------------------------------------------------------------- distances

def test_sqdist_matches_library_and_invariants():
    m, d = 7, 501
    X = rng(13).standard_normal((m, d)).astype(np.float32)
    D = oracle.sqdist(X)
    X64 = X.astype(np.float64)
    exp = ((X64[:, None, :] - X64[None, :, :]) ** 2).sum(-1)
    np.testing.assert_allclose(D, exp, rtol=1e-13, atol=0)
    assert np.array_equal(D, D.T) and not np.diag(D).any()
    X2 = X.copy(); X2[4] = X2[1]
    assert oracle.sqdist(X2)[1, 4] == 0.0
    assert np.array_equal(oracle.sqdist(X * np.float32(8.0)), 64.0 * D)   # exact under power-of-two scaling
    # not a Gram matrix in disguise: one-hot rows at distance sqrt(2)
    E = np.eye(3, dtype=np.float32)
    assert np.array_equal(oracle.sqdist(E), 2.0 * (1 - np.eye(3)))


# ---------------------------------------------------------------------------------- Krum family

def brute_krum_scores(D, alive, f):
    idx = [i for i in range(len(D)) if alive[i]]
    nb = min(max(len(idx) - f - 2, 1), len(idx) - 1)
    out = np.full(len(D), np.inf)
    for i in idx:
        others = [j for j in idx if j != i]
        out[i] = min((sum(sorted(D[i, list(sub)])) for sub in itertools.combinations(others, nb)), default=0.0)
    return out


def test_krum_scores_brute_force_subsets():
    g = rng(14)
    for trial in range(40):
        m = int(g.integers(3, 10))
        f = int(g.integers(0, max((m - 3) // 2, 0) + 1))
        X = g.integers(-8, 9, size=(m, int(g.integers(1, 9)))).astype(np.float32)   # integer data: exact sums
        D = oracle.sqdist(X)
        alive = np.ones(m, np.uint8)
        if trial % 2:
            alive[g.choice(m, size=int(g.integers(0, m - 1)), replace=False)] = 0
        got = oracle.krum_scores(D, f, alive)
        assert np.array_equal(got, brute_krum_scores(D, alive, f))


def test_krum_hand_worked_line_example():
    # Points on a line: 0, 1, 3, 10.  Squared distances: (0,1)=1 (0,3)=9 (0,10)=100 (1,3)=4 (1,10)=81 (3,10)=49.
    # m = 4, f = 0 -> m - f - 2 = 2 neighbours: scores 1+9, 1+4, 4+9, 49+81.
    X = np.array([[0.0], [1.0], [3.0], [10.0]], np.float32)
    out, sel, sc, D = oracle.multikrum(X, f=0, m_sel=2)
    assert sc.tolist() == [10.0, 5.0, 13.0, 130.0]
    assert sel.tolist() == [0, 1] and out.tolist() == [0.5]
    # f = 1 -> one neighbour: scores 1, 1, 4, 49; the tie between rows 0 and 1 goes to the lower index.
    out, sel, sc, _ = oracle.multikrum(X, f=1, m_sel=1)
    assert sc.tolist() == [1.0, 1.0, 4.0, 49.0] and sel.tolist() == [0] and out.tolist() == [0.0]
    # three rows with f = 1 would leave 0 neighbours; the count is clamped to one neighbour.
    out, sel, sc, _ = oracle.multikrum(X[:3], f=1, m_sel=1)
    assert sc.tolist() == [1.0, 1.0, 4.0] and sel.tolist() == [0]


def test_multikrum_f0_all_selected_is_plain_mean_and_equivariance():
    m, d = 9, 300
    X = rng(15).standard_normal((m, d)).astype(np.float32)
    out, sel, _, _ = oracle.multikrum(X, f=0, m_sel=m)
    assert sel.tolist() == list(range(m))
    assert np.array_equal(out, (X.astype(np.float64).sum(0) / m).astype(np.float32))
    X[6] *= 50.0                                                           # an outlier must not be selected
    out, sel, sc, _ = oracle.multikrum(X, f=1, m_sel=m - 1)
    assert 6 not in sel.tolist()
    perm = rng(16).permutation(m)
    _, selp, scp, _ = oracle.multikrum(X[perm], f=1, m_sel=m - 1)
    np.testing.assert_allclose(scp, sc[perm], rtol=1e-12)
    assert sorted(perm[selp].tolist()) == sel.tolist()
    _, sel2, sc2, _ = oracle.multikrum(X * np.float32(4.0), f=1, m_sel=m - 1)
    assert sel2.tolist() == sel.tolist() and np.array_equal(sc2, 16.0 * sc)


def brute_bulyan_select(D, f):
    m = len(D)
    alive = np.ones(m, np.uint8)
    sel = []
    for _ in range(m - 2 * f):
        sc = brute_krum_scores(D, alive, f)
        best = min((i for i in range(m) if alive[i]), key=lambda i: (sc[i], i))
        sel.append(best)
        alive[best] = 0
    return sel


def test_bulyan_select_brute_force():
    g = rng(17)
    for trial in range(25):
        f = int(g.integers(0, 2))
        m = int(g.integers(4 * f + 3, 10))
        X = g.integers(-8, 9, size=(m, int(g.integers(1, 9)))).astype(np.float32)
        D = oracle.sqdist(X)
        assert oracle.bulyan_select(D, f).tolist() == brute_bulyan_select(D, f)


def test_bulyan_hand_worked_scalar_example():
    # d = 1, values 0 1 2 3 4 5 100, f = 1: theta = 5, beta = 3.  Round 1: 4 neighbours each among 7 rows;
    # the centre-most rows win first.  Whatever the order, 100 is never among the 5 selected (its
    # distances dominate), so the selected values are five of 0..5, and the result is the mean of the
    # three values around their median.
    X = np.array([[0.0], [1.0], [2.0], [3.0], [4.0], [5.0], [100.0]], np.float32)
    out, sel, D = oracle.bulyan(X, f=1)
    assert 6 not in sel.tolist() and len(set(sel.tolist())) == 5
    vals = sorted(X[sel, 0].tolist())
    assert out[0] == np.float32(sum(vals[1:4]) / 3.0)
    assert sel.tolist() == brute_bulyan_select(D, 1)


def test_bulyan_selection_order_worked_by_hand():
    # The same column, every round written out (squared distances; ties go to the lower index):
    #   round 1, 7 rows, 4 neighbours: scores 30 15 10 10 15 30 37254      -> row 2 (ties with row 3)
    #   round 2, 6 rows, 3 neighbours: rows 0 1 3 4 5 6: 26 14 9 11 21 27650 -> row 3
    #   round 3, 5 rows, 2 neighbours: rows 0 1 4 5 6: 17 10 10 17 18241    -> row 1 (ties with row 4)
    #   round 4, 4 rows, 1 neighbour : rows 0 4 5 6: 16 1 1 9025            -> row 4 (ties with row 5)
    #   round 5, 3 rows, 3 - 1 - 2 = 0 neighbours, clamped to 1: rows 0 5 6: 25 25 9025 -> row 0 (ties with row 5)
    # Selected values 2 3 1 4 0: median 2, the three closest are 1 2 3, mean 2.
    X = np.array([[0.0], [1.0], [2.0], [3.0], [4.0], [5.0], [100.0]], np.float32)
    out, sel, D = oracle.bulyan(X, f=1)
    assert sel.tolist() == [2, 3, 1, 4, 0]
    assert out.tolist() == [2.0]
    alive = np.ones(7, np.uint8)
    assert oracle.krum_scores(D, 1, alive).tolist() == [30.0, 15.0, 10.0, 10.0, 15.0, 30.0, 37254.0]
    alive[[2, 3]] = 0
    assert oracle.krum_scores(D, 1, alive)[[0, 1, 4, 5, 6]].tolist() == [17.0, 10.0, 10.0, 17.0, 18241.0]


def test_trimmed_around_median_reductions_and_brute_force():
    g = rng(18)
    theta, d = 9, 200
    X = g.standard_normal((12, d)).astype(np.float32)
    rows = g.choice(12, size=theta, replace=False)
    # beta = 1: the coordinate median of the selected rows; beta = theta: their mean
    assert np.array_equal(oracle.trimmed_around_median(X, rows, 1), np.median(X[rows], axis=0))
    assert np.array_equal(oracle.trimmed_around_median(X, rows, theta),
                          (X[rows].astype(np.float64).sum(0) / theta).astype(np.float32))
    # brute force: among all beta-subsets, the one with the smallest total |v - med|
    for beta in (3, 5):
        got = oracle.trimmed_around_median(X, rows, beta)
        V = X[rows]
        assert (got >= V.min(0)).all() and (got <= V.max(0)).all()
        for c in range(0, d, 7):
            v = V[:, c].astype(np.float64)
            med = np.median(v)
            best = min(itertools.combinations(range(theta), beta), key=lambda s: sum(abs(v[list(s)] - med)))
            assert got[c] == np.float32(sum(v[list(best)]) / beta)


def test_trimmed_around_median_tie_takes_smaller_value():
    # values -2 -1 0 1 2: median 0; beta = 2 -> {0, -1} (equal distance: the smaller value), mean -0.5
    X = np.array([[2.0], [-1.0], [0.0], [1.0], [-2.0]], np.float32)
    assert oracle.trimmed_around_median(X, [0, 1, 2, 3, 4], 2).tolist() == [-0.5]
    assert oracle.trimmed_around_median(X, [0, 1, 2, 3, 4], 3).tolist() == [0.0]
    assert oracle.trimmed_around_median(X, [0, 1, 2, 3, 4], 4).tolist() == [-0.5]


def test_bulyan_f0_is_plain_mean():
    m, d = 7, 123
    X = rng(19).standard_normal((m, d)).astype(np.float32)
    out, sel, _ = oracle.bulyan(X, f=0)
    assert sorted(sel.tolist()) == list(range(m))
    assert np.array_equal(out, (X.astype(np.float64).sum(0) / m).astype(np.float32))


# ------------------------------------------------------------------------------------- pipeline

def test_pipeline_q0_is_plain_mean():
    # With no Byzantine node and mean/mean the DETOX output is the plain mean of Section 2.
    G, r, d = 6, 3, 400
    honest = rng(20).standard_normal((G, d)).astype(np.float32)
    members = rng(21).permutation(G * r).astype(np.int32)
    X = np.empty((G * r, d), np.float32)
    for j in range(G):
        X[members[j * r:(j + 1) * r]] = honest[j]
    exp = (honest.astype(np.float64).sum(0) / G).astype(np.float32)
    res = oracle.detox_aggregate(X, members, r, "none", None, None, "mean")
    assert np.array_equal(res["out"], exp)
    res = oracle.detox_aggregate(X, members, r, "none", None, None, "multikrum", f=0, m_sel=G)
    assert np.array_equal(res["out"], exp)
    res = oracle.detox_aggregate(X, members, r, "none", None, None, "bulyan", f=0)
    assert np.array_equal(res["out"], exp)
    # equal-size sets: mean of set means = plain mean up to the intermediate fp32 rounding
    res = oracle.detox_aggregate(X, members, r, "mean", [0, 3, 6], np.arange(6), "mean")
    np.testing.assert_allclose(res["out"], exp, rtol=0, atol=1e-6)


def test_pipeline_honest_majority_equals_aggregator_on_true_gradients():
    G, r, d = 5, 3, 256
    honest = rng(22).standard_normal((G, d)).astype(np.float32)
    members = rng(23).permutation(G * r).astype(np.int32)
    X = np.empty((G * r, d), np.float32)
    for j in range(G):
        grp = members[j * r:(j + 1) * r]
        X[grp] = honest[j]
        X[grp[j % r]] = -100.0 * honest[j]                                 # one Byzantine member per group
    res = oracle.detox_aggregate(X, members, r, "none", None, None, "coord_median")
    assert np.array_equal(res["out"], np.median(honest, axis=0))
    assert np.array_equal(res["Z"], honest)


def test_pipeline_krum_family_inside_vote_sets():
    # Section 5.2, setups 2 and 3: the aggregator inside every vote group, then the mean.
    G, r, d = 15, 3, 128
    honest = rng(30).standard_normal((G, d)).astype(np.float32)
    members = rng(31).permutation(G * r).astype(np.int32)
    X = np.empty((G * r, d), np.float32)
    for j in range(G):
        X[members[j * r:(j + 1) * r]] = honest[j]
    sm = rng(32).permutation(G).astype(np.int32)
    # no Byzantine node, f = 0: Multi-Krum keeps everything -> mean of the two set means (7 and 8 votes)
    res = oracle.detox_aggregate(X, members, r, "multikrum", [0, 7, 15], sm, "mean", f=0, m_sel=0)
    exp = (honest[sm[:7]].astype(np.float64).mean(0).astype(np.float32).astype(np.float64) +
           honest[sm[7:]].astype(np.float64).mean(0).astype(np.float32)) / 2
    np.testing.assert_allclose(res["out"], exp, rtol=0, atol=1e-6)
    assert sorted(res["sel"].tolist()) == list(range(G))
    # one Byzantine vote (a colluding pair wins group sm[3]): Multi-Krum(f=1) drops it from its set
    bad = int(sm[3])
    X[members[bad * r:bad * r + 2]] = 50.0 * honest[bad]
    res = oracle.detox_aggregate(X, members, r, "multikrum", [0, 7, 15], sm, "mean", f=1, m_sel=0)
    assert bad not in res["sel"].tolist() and len(res["sel"]) == 6 + 7
    assert res["sel_workers"].tolist() == res["winner"][res["sel"]].tolist()
    # Bulyan over one set of 15 with f = 2, then the mean of a single result = Bulyan on the votes
    res = oracle.detox_aggregate(X, members, r, "bulyan", [0, 15], sm, "mean", f=2)
    direct, sel, _ = oracle.bulyan(res["Z"][sm], 2)
    assert np.array_equal(res["out"], direct) and res["sel"].tolist() == sm[sel].tolist()
    assert bad not in res["sel"].tolist()


def test_trimmed_mean_against_library_and_reductions():
    from scipy import stats
    X = rng(40).standard_normal((12, 300)).astype(np.float32)
    np.testing.assert_allclose(oracle.trimmed_mean(X, 3), stats.trim_mean(X.astype(np.float64), 0.25, axis=0),
                               rtol=1e-6)
    assert np.array_equal(oracle.trimmed_mean(X, 0), (X.astype(np.float64).sum(0) / 12).astype(np.float32))
    Y = rng(41).standard_normal((9, 50)).astype(np.float32)
    assert np.array_equal(oracle.trimmed_mean(Y, 4), np.median(Y, axis=0))      # one value left: the median
    Z = np.array([[5.0], [1.0], [100.0], [3.0], [-7.0]], np.float32)            # sorted -7 1 3 5 100
    assert oracle.trimmed_mean(Z, 1).tolist() == [3.0]


# ----------------------------------------------------------------------------- geometric median

def _objective(X, y):
    return float(np.sqrt(((X.astype(np.float64) - y.astype(np.float64)) ** 2).sum(1)).sum())


def test_geometric_median_zero_iterations_is_the_mean_and_symmetric_points_stay():
    X = rng(50).standard_normal((7, 40)).astype(np.float32)
    assert np.array_equal(oracle.geometric_median(X, iters=0), (X.astype(np.float64).sum(0) / 7).astype(np.float32))
    ang = np.arange(6) * np.pi / 3
    P = np.stack([np.cos(ang), np.sin(ang)], 1).astype(np.float32) * 4 + np.float32(2.5)   # regular hexagon
    np.testing.assert_allclose(oracle.geometric_median(P, iters=50), [2.5, 2.5], atol=1e-6)


def test_geometric_median_is_a_stationary_point_and_the_objective_never_rises():
    # 3-4-5 triangle (all angles < 120 degrees): at the Fermat point the three unit vectors cancel
    T = np.array([[0.0, 0.0], [3.0, 0.0], [0.0, 4.0]], np.float32)
    y = oracle.geometric_median(T, iters=300).astype(np.float64)
    u = (T - y) / np.linalg.norm(T - y, axis=1, keepdims=True)
    assert np.abs(u.sum(0)).max() < 1e-5
    X = rng(51).standard_normal((9, 25)).astype(np.float32)
    obj = [_objective(X, oracle.geometric_median(X, iters=t)) for t in range(12)]
    assert all(b <= a + 1e-9 for a, b in zip(obj, obj[1:])) and obj[-1] < obj[0]
    g = oracle.geometric_median(X, iters=400).astype(np.float64)
    u = (X - g) / np.linalg.norm(X - g, axis=1, keepdims=True)
    assert np.abs(u.sum(0)).max() < 1e-4


def test_geometric_median_resists_an_outlier_and_is_equivariant():
    X = (rng(52).standard_normal((8, 30)) * 0.1).astype(np.float32)
    X[3] = 1000.0
    g = oracle.geometric_median(X, iters=100)
    assert np.linalg.norm(g) < 1.0 < np.linalg.norm(X.mean(0))        # the mean is dragged away, the median is not
    assert np.array_equal(oracle.geometric_median(X * np.float32(4), iters=20), oracle.geometric_median(X, iters=20) * 4)
    shift = np.float32(3.0)
    np.testing.assert_allclose(oracle.geometric_median(X + shift, iters=20), oracle.geometric_median(X, iters=20) + shift,
                               atol=1e-4)


def test_sign_majority_against_numpy_and_hand_worked_column():
    X = rng(60).standard_normal((9, 500)).astype(np.float32)
    X[:, 3] = 0.0
    X[0, 4] = np.nan
    exp = np.sign(np.where(np.isnan(X), 0.0, np.sign(X)).sum(0)).astype(np.float32)
    assert np.array_equal(oracle.sign_majority(X), exp)
    col = np.array([[2.0], [-1.0], [-3.0], [0.0], [5.0], [-0.0]], np.float32)   # two up, two down, two zeros: a tie
    assert oracle.sign_majority(col).tolist() == [0.0]
    assert oracle.sign_majority(col[:3]).tolist() == [-1.0]
    assert np.array_equal(oracle.sign_majority(X, [2, 5, 7]), np.sign(np.sign(X[[2, 5, 7]]).sum(0)).astype(np.float32))


def test_selection_checker_accepts_the_oracles_own_sequence_and_rejects_a_wrong_one():
    from helpers import check_bulyan_selection
    X = np.array([[0.0], [1.0], [2.0], [3.0], [4.0], [5.0], [100.0]], np.float32)
    D = oracle.sqdist(X)
    assert check_bulyan_selection(D, 1, [2, 3, 1, 4, 0], 1e-9) is True
    assert check_bulyan_selection(D, 1, [3, 2, 1, 4, 0], 1e-9) is False     # rows 2 and 3 tie exactly in round 1
    with pytest.raises(AssertionError):
        check_bulyan_selection(D, 1, [6, 3, 1, 4, 0], 1e-9)
