"""GPU parity: the CUDA library against the CPU oracle, element by element, on seeded inputs small enough
for the oracle to finish in seconds but spanning several tiles and ragged tails.

Bars: bit-exact votes, winners, medians and index sets; relative L2 <= 1e-5 on means and averaged
outputs (fp32 sums on the device against fp64 sums in the oracle)."""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_12205_b200 as dx
import workloads as wl
from helpers import bulyan_min_gap, multikrum_min_gap, rel_l2

pytestmark = pytest.mark.gpu
TOL = 1e-5
DEV = "cuda:0"


def dev(a):
    return torch.as_tensor(np.ascontiguousarray(a)).to(DEV)


def padded(a, ld=None, offset=0):
    """Copy a [rows, d] host array into a device buffer with row stride ld (and an element offset)."""
    rows, d = a.shape
    ld = ld or wl.padded_ld(d)
    buf = torch.full((rows * ld + offset + 8,), float("nan"), dtype=torch.float32, device=DEV)
    view = buf[offset: offset + rows * ld].view(rows, ld)[:, :d]
    view.copy_(torch.as_tensor(a))
    return view


def bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


# ------------------------------------------------------------------------------------------ vote

@pytest.mark.parametrize("r,G,d", [(3, 5, 100_000), (3, 4, 4099), (1, 3, 1000), (5, 3, 8193), (7, 2, 2050),
                                   (9, 2, 1027), (11, 1, 5000), (15, 1, 3001), (3, 2, 1), (3, 2, 3), (5, 1, 6)])
@pytest.mark.parametrize("layout", ["aligned", "odd_ld"])
def test_vote_matches_oracle(r, G, d, layout):
    rng = np.random.default_rng(r * 1000 + G + d)
    n = r * G
    members = rng.permutation(n).astype(np.int32)
    X = np.empty((n, d), np.float32)
    for j in range(G):
        grp = members[j * r:(j + 1) * r]
        g = rng.standard_normal(d).astype(np.float32)
        X[grp] = g
        kind = j % 4
        if kind == 1:                               # a Byzantine minority
            for i in grp[: (r - 1) // 2]:
                X[i] = -100 * g
        elif kind == 2 and r >= 3:                  # a colluding Byzantine majority
            for i in grp[: (r + 1) // 2]:
                X[i] = 7.0
        elif kind == 3 and r >= 3:                  # nobody agrees, differing only in the last coordinate
            for t, i in enumerate(grp):
                X[i, -1] = np.float32(t + 1)
    Xd = padded(X) if layout == "aligned" else padded(X, ld=d + (1 if d % 2 == 0 else 2), offset=1)
    Z, w = dx.detox_vote(Xd, r, members)
    Zo, wo = oracle.vote(X, members, r)
    assert w.cpu().numpy().tolist() == wo.tolist()
    assert np.array_equal(bits(Z), Zo.view(np.uint32))
    _, w2 = dx.detox_vote(Xd, r, members, want_Z=False)
    assert w2.cpu().numpy().tolist() == wo.tolist()


def test_vote_is_bitwise_on_special_values():
    d = 2000
    g = np.random.default_rng(5).standard_normal(d).astype(np.float32)
    a = g.copy(); a[1234] = -0.0
    b = g.copy(); b[1234] = 0.0
    c = g.copy(); c[77] = np.nan
    X = np.stack([a, b, a, c, c.copy(), g, a, b, g])
    members = np.arange(9, dtype=np.int32)
    Z, w = dx.detox_vote(padded(X), 3, members)
    Zo, wo = oracle.vote(X, members, 3)
    assert w.cpu().numpy().tolist() == wo.tolist() == [0, 3, -1]
    assert np.array_equal(bits(Z), Zo.view(np.uint32))


# ------------------------------------------------------------------------------------- hier mean

@pytest.mark.parametrize("G,d,offs", [(15, 10_001, [0, 7, 15]), (15, 4096, [0, 5, 10, 15]), (5, 3, [0, 5]),
                                      (35, 2500, [0, 5, 10, 15, 20, 25, 30, 35]), (6, 1, [0, 1, 6])])
def test_hier_mean_matches_oracle(G, d, offs):
    rng = np.random.default_rng(G + d)
    Z = (rng.standard_normal((G, d)) * 1e-3).astype(np.float32)
    Z[G // 2] = 0.0
    Z[0] *= -100
    sm = rng.permutation(G).astype(np.int32)
    M = dx.detox_hier_mean(padded(Z), offs, sm)
    Mo = oracle.hier_mean(Z, offs, sm)
    for s in range(len(offs) - 1):
        assert rel_l2(M[s].cpu().numpy(), Mo[s]) <= TOL
    M2 = dx.detox_hier_mean(padded(Z, ld=d + 3, offset=1), offs, sm)
    assert rel_l2(M2.cpu().numpy(), Mo) <= TOL


# ---------------------------------------------------------------------------------------- median

@pytest.mark.parametrize("m", list(range(1, 42)) + [45, 47, 48, 64, 65, 75, 100, 105, 127, 128, 129, 130, 200, 225, 255, 256, 257, 300])
def test_coord_median_bit_exact(m):
    rng = np.random.default_rng(m)
    d = 3000 + m if m <= 33 else 1000 + m
    X = (rng.standard_normal((m, d)) * 1e-3).astype(np.float32)
    X[:, 5] = 0.25                                   # all equal
    X[:, 6] = np.round(X[:, 6] * 2e3)                # many ties
    got = dx.agg_coord_median(padded(X))
    assert np.array_equal(bits(got), oracle.coord_median(X).view(np.uint32))
    got = dx.agg_coord_median(padded(X, ld=d + 1, offset=3))
    assert np.array_equal(bits(got), oracle.coord_median(X).view(np.uint32))


@pytest.mark.parametrize("m", [3, 5, 8, 15, 47])
def test_coord_median_special_values(m):
    rng = np.random.default_rng(100 + m)
    d = 1024
    pool = np.array([np.nan, -np.nan, np.inf, -np.inf, 0.0, -0.0, 1.0, -1.0, 1e-45, -1e-45, 3e38], np.float32)
    X = rng.choice(pool, size=(m, d)).astype(np.float32)
    if m % 2 == 0:
        X = np.where(np.isfinite(X), X, np.float32(2.0))  # the even-count average is only defined on finite values
    got = dx.agg_coord_median(padded(X))
    assert np.array_equal(bits(got), oracle.coord_median(X).view(np.uint32))


@pytest.mark.parametrize("m,trim", [(5, 1), (7, 0), (12, 3), (15, 7), (27, 6), (35, 8), (64, 16), (105, 26), (225, 56),
                                    (300, 75),
                                    # two lanes per coordinate: every network half size from 72 to 128, both parities
                                    (129, 1), (130, 40), (144, 0), (145, 72), (159, 20), (160, 79), (176, 3), (181, 22),
                                    (192, 50), (200, 99), (209, 10), (224, 100), (240, 1), (241, 120), (255, 60),
                                    (256, 127)])
def test_trimmed_mean_matches_oracle(m, trim):
    X = (np.random.default_rng(m).standard_normal((m, 2000 + m)) * 1e-3).astype(np.float32)
    X[0] *= -100
    got = dx.agg_trimmed_mean(padded(X), trim)
    assert rel_l2(got.cpu().numpy(), oracle.trimmed_mean(X, trim)) <= TOL


@pytest.mark.parametrize("m,d,iters", [(3, 20_001, 10), (7, 4099, 25), (15, 10_000, 8), (32, 3000, 5), (1, 500, 3),
                                       (5, 1, 4), (9, 1003, 0)])
def test_geometric_median_matches_oracle(m, d, iters):
    X = (np.random.default_rng(m + d).standard_normal((m, d)) * 1e-3).astype(np.float32)
    if m > 2:
        X[m - 1] *= -100                                   # a Byzantine row
    ref = oracle.geometric_median(X, iters=iters)
    assert rel_l2(dx.agg_geometric_median(padded(X), iters=iters).cpu().numpy(), ref) <= TOL
    assert rel_l2(dx.agg_geometric_median(padded(X, ld=d + 3, offset=1), iters=iters).cpu().numpy(), ref) <= TOL


@pytest.mark.parametrize("m,d", [(1, 100), (3, 4099), (4, 1001), (15, 20_000), (45, 3000), (200, 513)])
def test_sign_majority_bit_exact(m, d):
    X = np.random.default_rng(m * d).standard_normal((m, d)).astype(np.float32)
    X[:, 1] = 0.0
    X[0, 2] = np.nan
    X[:, 5] = -1.0                                          # the constant attack of Section 5.2
    assert np.array_equal(bits(dx.agg_sign_majority(padded(X))), oracle.sign_majority(X).view(np.uint32))
    assert np.array_equal(bits(dx.agg_sign_majority(padded(X, ld=d + 1, offset=1))),
                          oracle.sign_majority(X).view(np.uint32))


def test_pipeline_signsgd_pairing():
    # Section 5.2, setup 4: sign majority inside the vote sets and over their results; constant attack (-1)
    spec = wl.WorkloadSpec("p", n=45, r=3, d=30_001, sigma=1.0, q=5, attack="constant", placement="worst", set_size=5,
                           seed=8)
    w = wl.make_workload(spec)
    w.X[:, :spec.d] = torch.sign(w.X[:, :spec.d])           # workers send signs
    pipe = dx.Pipeline(45, 3, spec.d, w.members, dx.AGG_SIGN_MAJORITY, w.set_offsets, w.set_members,
                       dx.AGG_SIGN_MAJORITY)
    res = dx.detox_aggregate(pipe, w.X.to(DEV)[:, :spec.d])
    ref = oracle.detox_aggregate(w.data().numpy(), w.members, 3, "sign_majority", w.set_offsets, w.set_members,
                                 "sign_majority")
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert np.array_equal(bits(res["out"]), ref["out"].view(np.uint32))


# ------------------------------------------------------------------------------------ Multi-Krum

def krum_inputs(m, d, seed, copies=1, outliers=0):
    rng = np.random.default_rng(seed)
    base = (rng.standard_normal((m, d)) * 1e-3).astype(np.float32)
    base *= (1.0 + 0.2 * rng.uniform(-1, 1, size=(m, 1))).astype(np.float32)   # well separated scores
    if copies > 1:
        for i in range(0, m - copies + 1, copies):
            base[i + 1:i + copies] = base[i]
    for i in range(outliers):
        base[m - 1 - i] = -100 * base[m - 1 - i]
    return base


@pytest.mark.parametrize("m,d,f,m_sel,copies", [
    (3, 20_001, 1, 1, 1), (5, 4097, 1, 3, 1), (9, 10_000, 2, 7, 3), (15, 33_333, 3, 12, 1), (16, 2048, 0, 16, 1),
    (17, 5000, 3, 14, 1), (45, 20_011, 5, 40, 3), (64, 3000, 10, 54, 1), (105, 4100, 15, 90, 3), (130, 1000, 20, 100, 1),
    (1, 100, 0, 1, 1), (2, 100, 0, 1, 1)])
def test_multikrum_matches_oracle(m, d, f, m_sel, copies):
    for attempt in range(16):                        # seeds with a near-tie at the selection boundary are skipped
        X = krum_inputs(m, d, seed=m * 7 + d + 1000 * attempt, copies=copies, outliers=min(f, m // 4))
        out_o, sel_o, sc_o, _ = oracle.multikrum(X, f, m_sel)
        if multikrum_min_gap(sc_o, m_sel) > 1e-4:
            break
    else:
        pytest.fail("no seed without a near-tie")
    out, sel, sc = dx.agg_multikrum(padded(X), f, m_sel)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6, atol=1e-30)
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL
    if copies > 1:                                   # bitwise-equal rows must get bitwise-equal scores
        s = sc.cpu().numpy()
        for i in range(0, m - copies + 1 - min(f, m // 4), copies):
            assert len(set(s[i:i + copies].tolist())) == 1


def test_multikrum_unaligned_rows():
    X = krum_inputs(9, 1001, seed=3)
    out_o, sel_o, sc_o, _ = oracle.multikrum(X, 2, 5)
    out, sel, sc = dx.agg_multikrum(padded(X, ld=1003, offset=1), 2, 5)
    assert sel.cpu().numpy().tolist() == sel_o.tolist() and rel_l2(out.cpu().numpy(), out_o) <= TOL


# ---------------------------------------------------------------------------------------- Bulyan

@pytest.mark.parametrize("m,d,f,copies", [(7, 10_001, 1, 1), (15, 20_000, 3, 1), (15, 4099, 1, 3), (11, 2048, 2, 1),
                                          (27, 3000, 6, 1), (45, 8000, 9, 3), (45, 5000, 4, 1), (64, 2000, 5, 1),
                                          (105, 1500, 10, 3), (5, 1000, 0, 1), (36, 1200, 1, 1), (150, 1100, 10, 1), (225, 1000, 22, 3),
                                          (256, 700, 30, 1)])
def test_bulyan_matches_oracle(m, d, f, copies):
    for attempt in range(16):                        # seeds with a near-tie in some selection round are skipped
        X = krum_inputs(m, d, seed=m * 11 + d + 1000 * attempt, copies=copies, outliers=f)
        out_o, sel_o, D_o = oracle.bulyan(X, f)
        # many rows mean many successive decisions among closely spaced scores: the screen is relaxed to a
        # few times the tested score accuracy (2e-6) there
        if bulyan_min_gap(D_o, f) > (1e-4 if m <= 64 else 5e-6):
            break
    else:
        pytest.fail("no seed without a near-tie")
    out, sel = dx.agg_bulyan(padded(X), f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL


# -------------------------------------------------------------------------------------- pipeline

def run_pipeline(w, a0, a1, f=0, m_sel=1):
    spec = w.spec
    pipe = dx.Pipeline(spec.n, spec.r, spec.d, w.members, a0, w.set_offsets if a0 == dx.AGG_MEAN else None,
                       w.set_members if a0 == dx.AGG_MEAN else None, a1, f, m_sel)
    Xd = w.X.to(DEV)[:, :spec.d]
    res = dx.detox_aggregate(pipe, Xd)
    names = {dx.AGG_MEAN: "mean", dx.AGG_COORD_MEDIAN: "coord_median", dx.AGG_MULTIKRUM: "multikrum",
             dx.AGG_BULYAN: "bulyan", dx.AGG_TRIMMED_MEAN: "trimmed_mean",
             dx.AGG_GEOMETRIC_MEDIAN: "geometric_median"}
    ref = oracle.detox_aggregate(w.data().numpy(), w.members, spec.r, "mean" if a0 == dx.AGG_MEAN else "none",
                                 w.set_offsets, w.set_members, names[a1], f, m_sel)
    return res, ref


def test_pipeline_cfg1_vote_then_median_is_bit_exact():
    w = wl.make_workload(wl.CONFIGS["cfg1"])
    res, ref = run_pipeline(w, dx.AGG_NONE, dx.AGG_COORD_MEDIAN)
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert np.array_equal(bits(res["out"]), ref["out"].view(np.uint32))
    direct = dx.agg_coord_median(w.X.to(DEV)[:, :w.spec.d])
    assert np.array_equal(bits(direct), oracle.coord_median(w.data().numpy()).view(np.uint32))


@pytest.mark.parametrize("a1,f,m_sel", [(dx.AGG_MULTIKRUM, 1, 1), (dx.AGG_COORD_MEDIAN, 0, 1), (dx.AGG_MEAN, 0, 1),
                                        (dx.AGG_TRIMMED_MEAN, 1, 1), (dx.AGG_GEOMETRIC_MEDIAN, 0, 1)])
def test_pipeline_vote_mean_then_a1(a1, f, m_sel):
    spec = wl.WorkloadSpec("p", n=45, r=3, d=50_003, sigma=1e-3, q=5, attack="alie", placement="worst", set_size=5,
                           group_jitter=0.05, seed=11)
    w = wl.make_workload(spec)
    res, ref = run_pipeline(w, dx.AGG_MEAN, a1, f, m_sel)
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    if a1 == dx.AGG_MULTIKRUM:
        assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("a1,f,m_sel", [(dx.AGG_BULYAN, 3, 1), (dx.AGG_MULTIKRUM, 3, 10)])
def test_pipeline_vote_then_krum_family_maps_worker_ids(a1, f, m_sel):
    spec = wl.WorkloadSpec("p", n=45, r=3, d=30_001, sigma=1e-3, q=9, attack="reverse", placement="random",
                           group_jitter=0.05, seed=5)
    w = wl.make_workload(spec)
    res, ref = run_pipeline(w, dx.AGG_NONE, a1, f, m_sel)
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert res["sel_workers"].cpu().numpy().tolist() == ref["sel_workers"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


def test_pipeline_no_majority_group_becomes_zero_vote():
    spec = wl.WorkloadSpec("p", n=15, r=3, d=9001, sigma=1e-2, q=0, seed=2)
    w = wl.make_workload(spec)
    grp = w.members[:3]
    w.X[int(grp[0]), 17] += 1.0
    w.X[int(grp[1]), 9000] += 1.0                      # three different rows in group 0
    res, ref = run_pipeline(w, dx.AGG_NONE, dx.AGG_MEAN)
    assert ref["winner"][0] == -1 and res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("a1,f", [(dx.AGG_COORD_MEDIAN, 0), (dx.AGG_TRIMMED_MEAN, 1), (dx.AGG_TRIMMED_MEAN, 3)])
@pytest.mark.parametrize("n", [15, 27, 105])
def test_pipeline_order_statistics_over_votes_with_a_zero_vote(a1, f, n):
    """The order-statistic kernels read the votes through winner[]; a group without a majority is a zero row there
    (the row list holds -1), which takes the masked loads instead of the plain ones."""
    if 2 * f >= n // 3:
        pytest.skip("nothing would be left of the votes")
    spec = wl.WorkloadSpec("p", n=n, r=3, d=5003, sigma=1e-2, q=0, seed=n)
    w = wl.make_workload(spec)
    grp = w.members[3:6]
    w.X[int(grp[0]), 0] += 1.0
    w.X[int(grp[2]), 5002] -= 1.0                      # three different rows in group 1
    res, ref = run_pipeline(w, dx.AGG_NONE, a1, f)
    assert ref["winner"][1] == -1 and res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    if a1 == dx.AGG_COORD_MEDIAN:
        assert np.array_equal(bits(res["out"]), ref["out"].view(np.uint32))
    else:
        assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("r,G,set_size,d", [(3, 15, 5, 20_003), (3, 15, 7, 4097), (5, 6, 2, 3001), (1, 8, 3, 1000),
                                            (7, 4, None, 2500)])
def test_pipeline_fused_vote_mean_handles_no_majority_and_uneven_sets(r, G, set_size, d):
    spec = wl.WorkloadSpec("p", n=r * G, r=r, d=d, sigma=1e-2, q=0, set_size=set_size, seed=r + G)
    w = wl.make_workload(spec)
    if r >= 3:                                          # group 1: nobody agrees -> zero vote inside its set
        for t, i in enumerate(w.members[r:2 * r]):
            w.X[int(i), (t * 37) % d] += 1.0 + t
        i = int(w.members[0])                           # group 0: one dissenter, still a majority
        w.X[i, d - 1] = -w.X[i, d - 1] - 1.0
    for a1 in (dx.AGG_MEAN, dx.AGG_COORD_MEDIAN):
        res, ref = run_pipeline(w, dx.AGG_MEAN, a1)
        assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
        if r >= 3:
            assert ref["winner"][1] == -1 and ref["winner"][0] >= 0
        assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL
    # the fused pass gives the same set means, bit for bit, as vote followed by detox_hier_mean
    Xd = w.X.to(DEV)[:, :d]
    Z, _ = dx.detox_vote(Xd, r, w.members)
    M = dx.detox_hier_mean(Z, w.set_offsets, w.set_members)
    pipe = dx.Pipeline(spec.n, r, d, w.members, dx.AGG_MEAN, w.set_offsets, w.set_members, dx.AGG_MEAN)
    M2, w2 = dx.detox_vote_hier_mean(Xd, r, w.members, w.set_offsets, w.set_members)
    assert np.array_equal(bits(M2.contiguous()), bits(M.contiguous()))
    fused = dx.detox_aggregate(pipe, Xd)["out"]
    two_step = dx.detox_aggregate(dx.Pipeline(w.S, 1, d, np.arange(w.S), dx.AGG_NONE, None, None, dx.AGG_MEAN),
                                  M)["out"]
    assert np.array_equal(bits(fused), bits(two_step))


@pytest.mark.parametrize("r,set_size,S", [(3, 5, 1), (3, 3, 2), (3, 5, 3), (3, 2, 4), (3, 5, 5), (5, 1, 6), (3, 5, 7), (3, 4, 8),
                                          (3, 3, 9), (1, 2, 12), (3, 5, 15), (3, 2, 16), (3, 1, 17)])
@pytest.mark.parametrize("broken", [False, True])
def test_pipeline_vote_set_means_and_coordinatewise_a1_in_one_pass(r, set_size, S, broken):
    """With A_0 = mean and a coordinate-wise A_1 over at most 16 set means the whole step is one pass over X (set
    means and A_1 in registers).  It must give, bit for bit, what the separate entry points give (fused vote + set
    means, then the order-statistic or mean kernel over them), with and without a group that has no majority, and
    match the oracle; 17 sets take the separate kernels."""
    G = set_size * S
    d = 4099 + 64 * S                                   # a ragged tail
    spec = wl.WorkloadSpec("p", n=r * G, r=r, d=d, sigma=1e-2, q=0, set_size=set_size, seed=31 * S + r)
    w = wl.make_workload(spec)
    assert w.S == S
    if broken and r >= 3:                               # the last group: nobody agrees -> zero vote inside its set
        for t, i in enumerate(w.members[r * (G - 1):r * G]):
            w.X[int(i), (t * 53) % d] += 1.0 + t
    Xd = w.X.to(DEV)[:, :d]
    M, _ = dx.detox_vote_hier_mean(Xd, r, w.members, w.set_offsets, w.set_members)
    cases = [(dx.AGG_COORD_MEDIAN, 0), (dx.AGG_MEAN, 0)]
    if S >= 3:
        cases.append((dx.AGG_TRIMMED_MEAN, 1))
    if S >= 7:
        cases.append((dx.AGG_TRIMMED_MEAN, 3))
    for a1, f in cases:
        res, ref = run_pipeline(w, dx.AGG_MEAN, a1, f)
        assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
        if broken and r >= 3:
            assert ref["winner"][G - 1] == -1
        out = res["out"]
        if a1 == dx.AGG_COORD_MEDIAN:
            two_step = dx.agg_coord_median(M)
            assert np.array_equal(bits(out), bits(two_step))
            assert np.array_equal(bits(out), ref["out"].view(np.uint32)) or rel_l2(out.cpu().numpy(), ref["out"]) <= TOL
        elif a1 == dx.AGG_MEAN:
            two_step = dx.detox_aggregate(dx.Pipeline(S, 1, d, np.arange(S), dx.AGG_NONE, None, None, dx.AGG_MEAN), M)["out"]
            assert np.array_equal(bits(out), bits(two_step))
        assert rel_l2(out.cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("a0,f,m_sel,offs,a1", [("multikrum", 1, 0, [0, 7, 15], "mean"), ("bulyan", 2, 0, [0, 15], "mean"),
                                                 ("multikrum", 1, 3, [0, 5, 10, 15], "coord_median")])
def test_pipeline_krum_family_inside_vote_sets(a0, f, m_sel, offs, a1):
    # the paper's preferred pairings (Section 5.2, setups 2 and 3; set shapes of Appendix B.1)
    code = {"multikrum": dx.AGG_MULTIKRUM, "bulyan": dx.AGG_BULYAN, "mean": dx.AGG_MEAN,
            "coord_median": dx.AGG_COORD_MEDIAN}
    for attempt in range(16):
        spec = wl.WorkloadSpec("p", n=45, r=3, d=20_011, sigma=1e-3, q=5, attack="alie", placement="worst",
                               group_jitter=0.1, seed=40 + attempt)
        w = wl.make_workload(spec)
        sm = np.random.default_rng(spec.seed).permutation(15).astype(np.int32)
        ref = oracle.detox_aggregate(w.data().numpy(), w.members, 3, a0, offs, sm, a1, f, m_sel)
        gaps = []
        for s in range(len(offs) - 1):
            Zs = ref["Z"][sm[offs[s]:offs[s + 1]]]
            if a0 == "multikrum":
                keep = m_sel if m_sel > 0 else len(Zs) - f
                gaps.append(multikrum_min_gap(oracle.multikrum(Zs, f, keep, want_out=False)[2], keep))
            else:
                gaps.append(bulyan_min_gap(oracle.sqdist(Zs), f))
        if min(gaps) > 1e-4:
            break
    else:
        pytest.fail("no seed without a near-tie")
    pipe = dx.Pipeline(45, 3, spec.d, w.members, code[a0], offs, sm, code[a1], f, m_sel)
    res = dx.detox_aggregate(pipe, w.X.to(DEV)[:, :spec.d])
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert res["sel_workers"].cpu().numpy().tolist() == ref["sel_workers"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


def test_q0_pipeline_is_plain_mean():
    spec = wl.WorkloadSpec("p", n=21, r=3, d=12_345, sigma=1e-3, q=0, seed=9)
    w = wl.make_workload(spec)
    honest = w.data().numpy()[w.honest_member]
    exp = (honest.astype(np.float64).sum(0) / w.G).astype(np.float32)
    for a1, f, m_sel in [(dx.AGG_MEAN, 0, 1), (dx.AGG_MULTIKRUM, 0, w.G), (dx.AGG_BULYAN, 0, 1)]:
        res, _ = run_pipeline(w, dx.AGG_NONE, a1, f, m_sel)
        assert rel_l2(res["out"].cpu().numpy(), exp) <= TOL
