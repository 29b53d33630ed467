"""GPU parity at the edges of the supported ranges: the largest row counts and group sizes, the
fallback paths (rows that are not 16-byte aligned, row counts beyond the tensor-core and register
kernels), one-column inputs, and the device status word."""
import numpy as np
import pytest
import torch

import oracle
import paper_1907_12205_b200 as dx
from helpers import bulyan_min_gap, multikrum_min_gap, rel_l2
from test_parity_small import bits, krum_inputs, padded

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(params=["auto", "tf32"])
def split(request):
    """Runs a test once with the default operand split of the tensor-core distance pass (fp16 pairs first) and once
    with the split-TF32 kernels from the start."""
    prev = dx.tc_split_mode(dx.SPLIT_TF32 if request.param == "tf32" else dx.SPLIT_AUTO)
    yield request.param
    dx.tc_split_mode(prev)


@pytest.mark.parametrize("r,G,d", [(3, 341, 257), (15, 68, 130), (1, 1024, 33), (5, 204, 64)])
def test_vote_largest_group_counts(r, G, d):
    rng = np.random.default_rng(G)
    n = r * G
    members = rng.permutation(n).astype(np.int32)
    X = np.empty((n, d), np.float32)
    for j in range(G):
        grp = members[j * r:(j + 1) * r]
        X[grp] = rng.standard_normal(d).astype(np.float32)
        if r >= 3 and j % 3 == 0:
            X[grp[0]] *= -100
        if r >= 3 and j % 7 == 0:
            for t, i in enumerate(grp):
                X[i, t % d] += t + 1
    Z, w = dx.detox_vote(padded(X), r, members)
    Zo, wo = oracle.vote(X, members, r)
    assert w.cpu().numpy().tolist() == wo.tolist()
    assert np.array_equal(bits(Z), Zo.view(np.uint32))


def test_hier_mean_largest_set_counts():
    rng = np.random.default_rng(1)
    G, d = 1024, 40
    Z = rng.standard_normal((G, d)).astype(np.float32)
    perm = rng.permutation(G).astype(np.int32)
    for offs in (np.arange(G + 1), np.array([0, G]), np.array([0, 1, 1000, G])):
        M = dx.detox_hier_mean(padded(Z), offs.astype(np.int32), perm)
        assert rel_l2(M.cpu().numpy(), oracle.hier_mean(Z, offs, perm)) <= TOL


@pytest.mark.parametrize("m,d", [(300, 200), (513, 70), (1024, 40), (1024, 1), (1, 1), (2, 1), (105, 1), (225, 1)])
def test_coord_median_beyond_the_register_kernels_and_single_column(m, d):
    X = np.random.default_rng(m + d).standard_normal((m, d)).astype(np.float32)
    assert np.array_equal(bits(dx.agg_coord_median(padded(X))), oracle.coord_median(X).view(np.uint32))


@pytest.mark.parametrize("m,d,f,m_sel,odd", [(300, 700, 30, 270, False), (1024, 48, 100, 900, False),
                                              (45, 3001, 5, 40, True), (105, 1001, 10, 95, True), (3, 1, 0, 2, False)])
def test_multikrum_fallback_paths(m, d, f, m_sel, odd):
    for attempt in range(16):
        X = krum_inputs(m, d, seed=m + d + 1000 * attempt, copies=1, outliers=min(f, 4))
        out_o, sel_o, sc_o, _ = oracle.multikrum(X, f, m_sel)
        if multikrum_min_gap(sc_o, m_sel) > 1e-5:
            break
    Xd = padded(X, ld=d + (1 if d % 2 == 0 else 2), offset=1) if odd else padded(X)
    out, sel, sc = dx.agg_multikrum(Xd, f, m_sel)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6, atol=1e-30)
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL


@pytest.mark.parametrize("m,d", [
    (17, 63), (18, 64), (32, 65), (33, 4097), (63, 9473), (64, 129), (65, 4100), (80, 9472 + 31), (96, 2000),
    (127, 3001), (128, 1000), (129, 1000), (144, 2049), (240, 777), (256, 640),
    (20, 2_500_001), (100, 2_450_003), (140, 2_430_000)])   # last three: more than one output slot (4 x 4096 columns) per CTA
def test_tensor_core_distance_kernels_at_their_size_boundaries(m, d, split):
    """Row counts on both sides of every switch of the tensor-core kernels (64 and 128 rows, tile sizes that are
    multiples of 16) and column counts around the 32- and 64-column copies, with a ragged tail."""
    f = max((m - 3) // 4, 0)
    X = krum_inputs(m, d, seed=3 * m + d, copies=2 if m % 2 == 0 else 1, outliers=min(f, 3))
    _, _, sc_o, _ = oracle.multikrum(X, f, 1)
    _, _, sc = dx.agg_multikrum(padded(X), f, 1)
    s = sc.cpu().numpy()
    np.testing.assert_allclose(s, sc_o, rtol=2e-6, atol=1e-30)
    if m % 2 == 0:                                   # bitwise-equal rows must get bitwise-equal scores
        for i in range(0, m - 2 - min(f, 3), 2):
            assert s[i] == s[i + 1]


def test_bulyan_many_rows_through_the_shared_memory_stage_two():
    m, d, f = 400, 96, 20                      # theta = 360 rows enter stage 2: beyond the register kernels
    for attempt in range(8):
        X = krum_inputs(m, d, seed=77 + 1000 * attempt, copies=1, outliers=f)
        out_o, sel_o, D_o = oracle.bulyan(X, f)
        if bulyan_min_gap(D_o, f) > 5e-6:
            break
    out, sel = dx.agg_bulyan(padded(X), f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL


def test_status_word_is_clear_after_the_tensor_core_path():
    m, d = 64, 5000
    X = padded(krum_inputs(m, d, seed=5))
    ws = torch.full((dx.agg_multikrum_workspace_bytes(m, d),), 0xFF, dtype=torch.uint8, device="cuda:0")
    dx.agg_multikrum(X, 5, 50, ws=ws)
    torch.cuda.synchronize()
    assert int(ws[:4].view(torch.int32).item()) == 0       # first word of the workspace: device-side status


def test_pipeline_with_the_largest_worker_count():
    import workloads as wl
    spec = wl.WorkloadSpec("p", n=1023, r=3, d=300, sigma=1e-3, q=100, attack="reverse", placement="random",
                           set_size=11, group_jitter=0.05, seed=3)
    w = wl.make_workload(spec)
    pipe = dx.Pipeline(spec.n, 3, spec.d, w.members, dx.AGG_MEAN, w.set_offsets, w.set_members, dx.AGG_COORD_MEDIAN)
    res = dx.detox_aggregate(pipe, w.X.to("cuda:0")[:, :spec.d])
    ref = oracle.detox_aggregate(w.data().numpy(), w.members, 3, "mean", w.set_offsets, w.set_members, "coord_median")
    assert res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("a1,f,m_sel", [("median", 0, 1), ("multikrum", 4, 30)])
def test_pipeline_replays_from_a_cuda_graph(a1, f, m_sel):
    # Everything is enqueued on the caller's stream with host tables passed as kernel parameters, so a step
    # can be captured once and replayed on new data in the same buffers.
    import workloads as wl
    code = {"median": dx.AGG_COORD_MEDIAN, "multikrum": dx.AGG_MULTIKRUM}[a1]
    oname = {"median": "coord_median", "multikrum": "multikrum"}[a1]
    specs = [wl.WorkloadSpec("g", n=105, r=3, d=6001, sigma=1e-3, q=10, attack="reverse", placement="random",
                             set_size=5, group_jitter=0.2, seed=s) for s in (1, 2)]
    w0 = wl.make_workload(specs[0])
    a0 = dx.AGG_MEAN if a1 == "median" else dx.AGG_NONE
    pipe = dx.Pipeline(105, 3, 6001, w0.members, a0, w0.set_offsets, w0.set_members, code, f, m_sel)
    X = w0.X.to("cuda:0")
    out = torch.empty(6001, dtype=torch.float32, device="cuda:0")
    winner = torch.empty(35, dtype=torch.int32, device="cuda:0")
    sel = torch.empty(max(pipe.n_selected, 1), dtype=torch.int32, device="cuda:0")
    selw = torch.empty(max(pipe.n_selected, 1), dtype=torch.int32, device="cuda:0")
    ws = torch.empty(pipe.workspace_bytes(), dtype=torch.uint8, device="cuda:0")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        dx.detox_aggregate(pipe, X[:, :6001], out=out, winner=winner, sel=sel, sel_workers=selw, ws=ws)   # warm-up
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            dx.detox_aggregate(pipe, X[:, :6001], out=out, winner=winner, sel=sel, sel_workers=selw, ws=ws)
    for spec in specs:
        w = wl.make_workload(spec)            # new gradients, moved onto the captured partition (the tables are
        Xn = torch.empty_like(w.X)            # kernel parameters baked into the graph)
        Xn[torch.as_tensor(w0.members, dtype=torch.long)] = w.X[torch.as_tensor(w.members, dtype=torch.long)]
        X.copy_(Xn)
        out.zero_()
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.detox_aggregate(Xn.numpy()[:, :6001], w0.members, 3, "mean" if a1 == "median" else "none",
                                     w0.set_offsets, w0.set_members, oname, f, m_sel)
        assert winner.cpu().numpy().tolist() == ref["winner"].tolist()
        assert rel_l2(out.cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("a1,f,m_sel", [("multikrum", 2, 9), ("bulyan", 2, 1)])
def test_pipeline_long_rows_with_a_zero_vote_through_the_staged_distance_kernel(a1, f, m_sel):
    """Twelve votes read through winner[] at a length that takes the bulk-copy distance kernel (9 to 16 rows, at
    least 606,208 columns), with one group that has no majority (its vote is the zero row) and d % 4 = 1."""
    import workloads as wl
    spec = wl.WorkloadSpec("p", n=36, r=3, d=640_001, sigma=1e-3, q=0, group_jitter=0.05, seed=11)
    w = wl.make_workload(spec)
    grp = w.members[3:6]
    w.X[int(grp[0]), 5] += 1.0
    w.X[int(grp[1]), 640_000] += 1.0                   # three different rows in group 1
    code = dx.AGG_MULTIKRUM if a1 == "multikrum" else dx.AGG_BULYAN
    pipe = dx.Pipeline(36, 3, spec.d, w.members, dx.AGG_NONE, None, None, code, f, m_sel)
    res = dx.detox_aggregate(pipe, w.X.to("cuda:0")[:, :spec.d])
    ref = oracle.detox_aggregate(w.data().numpy(), w.members, 3, "none", None, None, a1, f, m_sel)
    assert ref["winner"][1] == -1 and res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("M", list(range(9, 17)))
def test_bulk_copy_distance_kernel_for_every_row_count(M):
    """9 to 16 rows of just over 606,208 columns take the bulk-copy ring (one template instance per row count):
    a ragged last tile, a length that is not a multiple of four, and, through the pipeline, a zero vote."""
    d = 606_208 + 4 * 37 + 1
    for attempt in range(8):
        X = krum_inputs(M, d, seed=50 * M + 1000 * attempt, copies=1, outliers=2)
        out_o, sel_o, sc_o, _ = oracle.multikrum(X, 2, M - 3)
        if multikrum_min_gap(sc_o, M - 3) > 1e-5:
            break
    out, sel, sc = dx.agg_multikrum(padded(X), 2, M - 3)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6, atol=1e-30)
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL
    # the same rows as the votes of M groups of three, the second group without a majority (its vote is zero)
    import workloads as wl
    spec = wl.WorkloadSpec("p", n=3 * M, r=3, d=d, sigma=1e-3, q=0, group_jitter=0.2, seed=M)
    w = wl.make_workload(spec)
    grp = w.members[3:6]
    w.X[int(grp[0]), 7] += 1.0
    w.X[int(grp[1]), d - 1] += 1.0
    pipe = dx.Pipeline(3 * M, 3, d, w.members, dx.AGG_NONE, None, None, dx.AGG_MULTIKRUM, 1, M - 2)
    res = dx.detox_aggregate(pipe, w.X.to("cuda:0")[:, :d])
    ref = oracle.detox_aggregate(w.data().numpy(), w.members, 3, "none", None, None, "multikrum", 1, M - 2)
    assert ref["winner"][1] == -1 and res["winner"].cpu().numpy().tolist() == ref["winner"].tolist()
    assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL


@pytest.mark.parametrize("m,d", [(9, 5001), (20, 5001), (140, 3000), (9, 700_001)])
def test_a_row_with_an_infinite_entry_is_never_selected(m, d, split):
    """A Byzantine row may hold anything.  One +Inf makes the row infinitely far from every other row on both
    sides (direct differences give Inf; the Gram path's NaN counts as Inf), so Multi-Krum and Bulyan leave it out
    and the selections match the oracle."""
    f = 2 if m >= 11 else 1
    for attempt in range(8):
        X = krum_inputs(m, d, seed=9 * m + 1000 * attempt, copies=1, outliers=1)
        X[3, d // 2] = np.inf
        _, sel_o, sc_o, D_o = oracle.multikrum(X, f, m - f, want_out=False)
        if multikrum_min_gap(sc_o[np.isfinite(sc_o)], m - f) > 1e-5 and bulyan_min_gap(D_o, f) > 5e-6:
            break
    assert 3 not in sel_o.tolist()
    out, sel, sc = dx.agg_multikrum(padded(X), f, m - f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    assert torch.isfinite(out).all()
    _, bsel = dx.agg_bulyan(padded(X), f)
    bsel_o = oracle.bulyan_select(D_o, f)
    assert 3 not in bsel_o.tolist() and bsel.cpu().numpy().tolist() == bsel_o.tolist()


def correlated_rows(m, d, ratio, seed, copies=1, outliers=0):
    """x_i = mu + eps_i: a common vector of `ratio` times the length of the individual parts (honest gradients of one
    loss at one model share a direction)."""
    rng = np.random.default_rng(seed)
    eps = krum_inputs(m, d, seed=seed + 1, copies=copies, outliers=0)
    mu = (rng.standard_normal(d) * 1e-3 * ratio).astype(np.float32)
    X = eps + mu
    for i in range(outliers):
        X[m - 1 - i] = -100 * X[m - 1 - i]
    return X


@pytest.mark.parametrize("ratio", [1, 10, 100])
@pytest.mark.parametrize("m", [45, 105, 225])
def test_tensor_core_distances_on_rows_that_share_a_large_common_vector(m, ratio, split):
    d = 150_003
    f = m // 10
    for attempt in range(8):
        X = correlated_rows(m, d, ratio, seed=31 * m + ratio + 1000 * attempt, copies=3 if m == 105 else 1, outliers=f)
        out_o, sel_o, sc_o, D_o = oracle.multikrum(X, f, m - f)
        if multikrum_min_gap(sc_o, m - f) > 1e-5:
            break
    out, sel, sc = dx.agg_multikrum(padded(X), f, m - f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6, atol=1e-30)
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL
    D = dx.agg_pairwise_sqdist(padded(X)).cpu().numpy()
    honest = m - f
    np.testing.assert_allclose(D[:honest, :honest], D_o[:honest, :honest], rtol=2e-6, atol=0)
    if m == 105:                                     # bitwise-equal rows: distance exactly zero, equal scores
        s = sc.cpu().numpy()
        for i in range(0, honest - 3, 3):
            assert D[i, i + 1] == 0.0 and D[i, i + 2] == 0.0 and s[i] == s[i + 1] == s[i + 2]


@pytest.mark.parametrize("m", [45, 140])
def test_a_centring_row_that_is_only_central_where_it_is_sampled_is_withdrawn(m, split):
    """The row subtracted from all rows is chosen on 32 evenly spaced blocks of 64 columns.  A Byzantine row that sits
    in the middle of the others there and holds huge values everywhere else would, once subtracted, wipe out the
    differences between the honest rows.  The library checks the exact norms after the pass and repeats it without
    that row; distances and selection must come out right."""
    d, ratio, f = 100_000, 3, 4
    X = correlated_rows(m, d, ratio, seed=5 * m, outliers=0)
    nb_all = (d + 63) // 64
    sampled = np.zeros(d, bool)
    for b in range(32):
        c0 = (nb_all * b // 32) * 64
        sampled[c0:c0 + 64] = True
    bad = X[: m - 1].astype(np.float64).mean(axis=0).astype(np.float32)   # the centre of the others where sampled ...
    bad[~sampled] = 1e30                                                   # ... and far away everywhere else
    X[m - 1] = bad
    _, sel_o, sc_o, D_o = oracle.multikrum(X, f, m - f, want_out=False)
    assert m - 1 not in sel_o.tolist()
    _, sel, sc = dx.agg_multikrum(padded(X), f, m - f)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy()[: m - 1], sc_o[: m - 1], rtol=2e-5)
