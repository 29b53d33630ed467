"""GPU parity over the sweep (n x attack at d = 1,000,000, plus one point at 225 rows of ResNet-18 size): every leg
that `bench.py --sweep` times is checked against the CPU oracle with the same parameters.

Votes, winners, medians and index sets bit for bit; averaged outputs by relative L2 <= 1e-5.  Seeds whose fp64
oracle scores have a near-tie at the Multi-Krum cut are skipped (next seed).  Bulyan takes up to 181 successive
decisions among scores that the replicated rows and the sweep's +-2 % group scales keep within 1e-6 of each other
at some round for practically every seed, so its selection is checked round by round instead: each pick must be the
oracle's, or, at such a near-tie, a remaining row whose oracle score is within 5e-6 of the minimum; the stage-two
result is then compared with the oracle's on the rows that were picked."""
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
CODE = {"none": dx.AGG_NONE, "mean": dx.AGG_MEAN, "coord_median": dx.AGG_COORD_MEDIAN, "multikrum": dx.AGG_MULTIKRUM,
        "bulyan": dx.AGG_BULYAN}


def bits(t):
    return t.detach().cpu().numpy().view(np.uint32)


def screened(spec):
    """The first seed (spec.seed, +1000, ...) without a near-tie at the Multi-Krum cuts of the sweep's legs."""
    for bump in range(8):
        sp = dataclasses.replace(spec, seed=spec.seed + 1000 * bump)
        w = wl.make_workload(sp, device=DEV)
        Xh = w.X.cpu().numpy()[:, : sp.d]
        legs = wl.sweep_legs(sp, w.G, w.S)
        Zo, wo = oracle.vote(Xh, w.members, sp.r)
        Dz, Dx = oracle.sqdist(Zo), oracle.sqdist(Xh)
        fv = legs["detox_multikrum"]["f"]
        if (multikrum_min_gap(oracle.krum_scores(Dz, fv), w.G - fv) > GAP and
                multikrum_min_gap(oracle.krum_scores(Dx, sp.q), sp.n - sp.q) > GAP):
            return w, Xh, legs, Zo, wo, Dz, Dx
    pytest.fail("no seed without a near-tie")


def check_bulyan(X_rows, D_o, f, out, sel):
    """sel: the GPU's selection among the rows of X_rows (host); out: its stage-two result."""
    sel = sel.cpu().numpy()
    check_bulyan_selection(D_o, f, sel, NEAR_TIE)
    ref = oracle.trimmed_around_median(X_rows, sel, len(sel) - 2 * f)
    assert rel_l2(out.cpu().numpy(), ref) <= TOL


@pytest.mark.parametrize("n", [15, 45, 105, 225])
@pytest.mark.parametrize("attack", ["reverse", "alie"])
def test_sweep_point_every_leg(n, attack):
    spec = [s for s in wl.sweep_specs(ns=(n,), ds=(1_000_000,), attacks=(attack,))][0]
    w, Xh, legs, Zo, wo, Dz, Dx = screened(spec)
    sp = w.spec
    Xd = w.X[:, : sp.d]
    for name, leg in legs.items():
        if name.startswith("detox_"):
            mean0 = leg["a0"] == "mean"
            pipe = dx.Pipeline(sp.n, sp.r, sp.d, w.members, CODE[leg["a0"]], w.set_offsets if mean0 else None,
                               w.set_members if mean0 else None, CODE[leg["a1"]], leg["f"], leg["m_sel"])
            res = dx.detox_aggregate(pipe, Xd)
            assert res["winner"].cpu().numpy().tolist() == wo.tolist(), name
            if leg["a1"] == "bulyan":
                check_bulyan(Zo, Dz, leg["f"], res["out"], res["sel"])
                assert res["sel_workers"].cpu().numpy().tolist() == wo[res["sel"].cpu().numpy()].tolist(), name
                continue
            ref = oracle.detox_aggregate(Xh, w.members, sp.r, leg["a0"], w.set_offsets, w.set_members, leg["a1"],
                                         leg["f"], leg["m_sel"])
            if ref["sel"] is not None:
                assert res["sel"].cpu().numpy().tolist() == ref["sel"].tolist(), name
                assert res["sel_workers"].cpu().numpy().tolist() == ref["sel_workers"].tolist(), name
            if leg["a1"] == "coord_median" and not mean0:
                assert np.array_equal(bits(res["out"]), ref["out"].view(np.uint32)), name
            else:
                assert rel_l2(res["out"].cpu().numpy(), ref["out"]) <= TOL, name
        elif leg["a1"] == "coord_median":
            assert np.array_equal(bits(dx.agg_coord_median(Xd)), oracle.coord_median(Xh).view(np.uint32)), name
        elif leg["a1"] == "multikrum":
            out, sel, sc = dx.agg_multikrum(Xd, leg["f"], leg["m_sel"])
            out_o, sel_o, sc_o, _ = oracle.multikrum(Xh, leg["f"], leg["m_sel"])
            assert sel.cpu().numpy().tolist() == sel_o.tolist(), name
            np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6, atol=1e-30)
            assert rel_l2(out.cpu().numpy(), out_o) <= TOL, name
        else:
            out, sel = dx.agg_bulyan(Xd, leg["f"])
            check_bulyan(Xh, Dx, leg["f"], out, sel)


def test_225_rows_of_resnet18_size_direct_legs():
    """The two-lane order-statistic kernel and the wide tensor-core distance kernel over many slabs and CTAs.
    The fp64 distance pass of the oracle takes tens of seconds here, so it runs once per seed and its matrix is
    reused for the near-tie screen and for the check of Bulyan's selection."""
    base = wl.sweep_specs(ns=(225,), ds=(wl.RESNET18_D,), attacks=("reverse",))[0]
    for bump in range(4):
        spec = dataclasses.replace(base, seed=base.seed + 1000 * bump)
        w = wl.make_workload(spec, device=DEV)
        Xh = w.X.cpu().numpy()[:, : spec.d]
        legs = wl.sweep_legs(spec, w.G, w.S)
        f, m_sel = legs["direct_multikrum"]["f"], legs["direct_multikrum"]["m_sel"]
        out_o, sel_o, sc_o, D_o = oracle.multikrum(Xh, f, m_sel)
        if multikrum_min_gap(sc_o, m_sel) > GAP:
            break
        del w, Xh
    else:
        pytest.fail("no seed without a near-tie")
    Xd = w.X[:, : spec.d]
    assert np.array_equal(bits(dx.agg_coord_median(Xd)), oracle.coord_median(Xh).view(np.uint32))
    out, sel, sc = dx.agg_multikrum(Xd, f, m_sel)
    assert sel.cpu().numpy().tolist() == sel_o.tolist()
    np.testing.assert_allclose(sc.cpu().numpy(), sc_o, rtol=2e-6)
    assert rel_l2(out.cpu().numpy(), out_o) <= TOL
    out, sel = dx.agg_bulyan(Xd, f, out=out)
    check_bulyan(Xh, D_o, f, out, sel)
