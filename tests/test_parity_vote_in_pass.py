"""GPU parity of the pipeline when the filtering step (Section 3) runs inside the tensor-core distance pass: more than
16 votes of groups of three under a Krum-type A_1.  No vote is stored; winner[] comes out of the pass and everything
after the distances reads the winners' rows.  Winners and index sets bit for bit, outputs by relative L2 <= 1e-5,
against the CPU oracle, over every launch shape of the pass (one or two boxes of member rows per stage; four, two or
one group of transform warps), with Byzantine members, with a group that has no majority (the pass is then repeated on
stored votes) and with an entry outside the fp16 range (likewise)."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
import paper_1907_12205_b200 as dx
import workloads as wl
from helpers import check_bulyan_selection, multikrum_min_gap, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
TOL = 1e-5
GAP, NEAR_TIE = 1e-5, 5e-6


def screened(spec, f, m_sel, spoil=None):
    """The first seed whose oracle scores over the votes have no near-tie at the Multi-Krum cut."""
    for bump in range(8):
        sp = dataclasses.replace(spec, seed=spec.seed + 1000 * bump)
        w = wl.make_workload(sp)
        if spoil is not None:
            spoil(w)
        Xh = w.data().numpy()
        Zo, wo = oracle.vote(Xh, w.members, sp.r)
        Dz = oracle.sqdist(Zo)
        if multikrum_min_gap(oracle.krum_scores(Dz, f), m_sel) > GAP:
            return w, Xh, Zo, wo, Dz
    pytest.fail("no seed without a near-tie")


def run_both(w, Xh, Zo, wo, Dz, f, m_sel):
    sp = w.spec
    Xd = w.X.to(DEV)[:, : sp.d]
    pipe = dx.Pipeline(sp.n, sp.r, sp.d, w.members, dx.AGG_NONE, None, None, dx.AGG_MULTIKRUM, f, m_sel)
    ws = torch.empty(pipe.workspace_bytes(), dtype=torch.uint8, device=DEV)
    res = dx.detox_aggregate(pipe, Xd, ws=ws)
    assert dx.read_status(ws) == 0
    ref = oracle.detox_aggregate(Xh, w.members, sp.r, "none", None, None, "multikrum", f, m_sel)
    assert res["winner"].cpu().numpy().tolist() == wo.tolist()
    assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist()
    assert res["sel_workers"].cpu().numpy().tolist() == ref["sel_workers"].tolist()
    assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL
    pipe = dx.Pipeline(sp.n, sp.r, sp.d, w.members, dx.AGG_NONE, None, None, dx.AGG_BULYAN, f, 1)
    ws = torch.empty(pipe.workspace_bytes(), dtype=torch.uint8, device=DEV)
    res = dx.detox_aggregate(pipe, Xd, ws=ws)
    assert dx.read_status(ws) == 0
    assert res["winner"].cpu().numpy().tolist() == wo.tolist()
    sel = res["sel"].cpu().numpy()
    check_bulyan_selection(Dz, f, sel, NEAR_TIE)
    assert rel_l2(res["out"].cpu().numpy(), oracle.trimmed_around_median(Zo, sel, len(sel) - 2 * f)) <= TOL
    assert res["sel_workers"].cpu().numpy().tolist() == wo[sel].tolist()


# n = 3 G: 17 and 32 votes (four transform groups), 33, 35, 42 (two groups, one box), 43 and 64 (two groups, two boxes),
# 65, 75 and 85 (one group, two boxes)
@pytest.mark.parametrize("n", [51, 96, 99, 105, 126, 129, 192, 195, 225, 255])
@pytest.mark.parametrize("attack", ["reverse", "alie"])
def test_vote_inside_the_distance_pass_every_launch_shape(n, attack):
    G = n // 3
    f = min(2, (G - 3) // 4)
    spec = wl.WorkloadSpec("p", n=n, r=3, d=70_001 if n % 2 else 300_004, sigma=1e-3, q=n // 10, attack=attack,
                           placement="random", group_jitter=0.02, seed=n)
    before = dx.tc_repeated_passes()
    run_both(*screened(spec, f, G - f), f, G - f)
    assert dx.tc_repeated_passes() == before      # the pass that votes while it reads was not repeated


@pytest.mark.parametrize("n", [105, 225])
def test_a_group_without_a_majority_sends_the_pass_to_stored_votes(n):
    """Three different rows in one group: its vote is the zero row (Section 3), which the pass that votes piece by
    piece cannot know in advance; the distances then come from stored votes."""
    G = n // 3
    f = 2

    def spoil(w):
        grp = w.members[6:9]
        w.X[int(grp[0]), 5] += 1.0
        w.X[int(grp[1]), w.spec.d - 1] += 1.0

    spec = wl.WorkloadSpec("p", n=n, r=3, d=150_001, sigma=1e-3, q=n // 10, attack="reverse", placement="random",
                           group_jitter=0.02, seed=3 * n)
    w, Xh, Zo, wo, Dz = screened(spec, f, G - f, spoil)
    assert wo[2] == -1
    run_both(w, Xh, Zo, wo, Dz, f, G - f)


def test_an_entry_outside_the_fp16_range_repeats_the_pass_on_stored_votes():
    n, G, f = 105, 35, 2

    def spoil(w):
        for i in w.members[12:15]:
            w.X[int(i), 33_331] = 40.0            # 40,000 x the row's typical entry, in a column the sample does not see

    spec = wl.WorkloadSpec("p", n=n, r=3, d=150_001, sigma=1e-3, q=0, group_jitter=0.02, seed=77)
    w, Xh, Zo, wo, Dz = screened(spec, f, G - f, spoil)
    before = dx.tc_repeated_passes()
    run_both(w, Xh, Zo, wo, Dz, f, G - f)
    assert dx.tc_repeated_passes() > before


def test_votes_that_share_a_large_common_vector():
    """Honest gradients of one loss at one model share a direction: the rows subtracted inside the pass are member
    rows of X picked on the column sample."""
    n, G, f = 105, 35, 2
    spec = wl.WorkloadSpec("p", n=n, r=3, d=200_003, sigma=1e-3, q=10, attack="reverse", placement="random",
                           group_jitter=0.02, seed=5)
    rng = np.random.default_rng(1)
    mu = torch.from_numpy((rng.standard_normal(spec.d) * 1e-2).astype(np.float32))

    def spoil(w):
        for i in range(n):
            if not w.byzantine[i]:
                w.X[i, : spec.d] += mu

    w, Xh, Zo, wo, Dz = screened(spec, f, G - f, spoil)
    run_both(w, Xh, Zo, wo, Dz, f, G - f)
