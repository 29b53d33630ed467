"""GPU checks that stand in for a memory checker and a race detector: run-to-run bitwise determinism of every
entry point, guard bands around every buffer the library writes, the bounded device-side wait giving up by
itself, and the device status word of the pipeline."""
import numpy as np
import pytest
import torch

import paper_1907_12205_b200 as dx
import workloads as wl

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
GUARD = 64            # guard elements (4 bytes each) on either side of a buffer
PATTERN = 0x5A5AA5A5


class Guarded:
    """A device buffer of `numel` 4-byte elements (or bytes) with a fixed pattern before and after it."""

    def __init__(self, numel, dtype=torch.float32, align_bytes=256):
        item = torch.empty(0, dtype=dtype).element_size()
        words = (numel * item + 3) // 4
        lead = max(GUARD, align_bytes // 4)
        self.raw = torch.full((lead + words + GUARD,), PATTERN, dtype=torch.int32, device=DEV)
        assert (self.raw.data_ptr() + lead * 4) % align_bytes == 0   # the payload is aligned like a fresh allocation
        self.lead, self.words = lead, words
        self.view = self.raw[lead: lead + words].view(torch.uint8)[: numel * item].view(dtype)

    def intact(self):
        a = self.raw[: self.lead]
        b = self.raw[self.lead + self.words:]
        return bool((a == PATTERN).all().item()) and bool((b == PATTERN).all().item())


def workload(n, d, seed=4, q=None, attack="reverse", set_size=5):
    spec = wl.WorkloadSpec("t", n=n, r=3, d=d, sigma=1e-3, q=n // 10 if q is None else q, attack=attack,
                           placement="random", set_size=set_size, group_jitter=0.1, seed=seed)
    return wl.make_workload(spec, device=DEV)


def matrix_in_guards(X, ld):
    rows, d = X.shape
    g = Guarded(rows * ld)
    v = g.view.view(rows, ld)
    v[:, :d].copy_(X)
    return g, v[:, :d]


# ------------------------------------------------------------------------------------- determinism

@pytest.mark.parametrize("n,d", [(45, 300_007), (105, 150_001), (225, 70_003)])
def test_every_entry_point_is_bitwise_reproducible(n, d):
    w = workload(n, d)
    X = w.X[:, :d]
    G, S = w.G, w.S

    def run_all():
        res = []
        Z, win = dx.detox_vote(X, 3, w.members)
        res += [Z, win]
        res.append(dx.detox_hier_mean(Z, w.set_offsets, w.set_members))
        res += list(dx.detox_vote_hier_mean(X, 3, w.members, w.set_offsets, w.set_members))
        res.append(dx.agg_coord_median(X))
        res.append(dx.agg_trimmed_mean(X, n // 4))
        res.append(dx.agg_sign_majority(X))
        res.append(dx.agg_geometric_median(Z[: min(G, 32)], iters=4))
        res += list(dx.agg_multikrum(X, n // 10, n - n // 10))
        res += list(dx.agg_bulyan(X, n // 10))
        for a0, a1, f, m_sel in [(dx.AGG_MEAN, dx.AGG_COORD_MEDIAN, 0, 1), (dx.AGG_NONE, dx.AGG_MULTIKRUM, 2, G - 2),
                                 (dx.AGG_NONE, dx.AGG_BULYAN, 2, 1), (dx.AGG_MULTIKRUM, dx.AGG_MEAN, 1, 0)]:
            sets = a0 != dx.AGG_NONE
            p = dx.Pipeline(n, 3, d, w.members, a0, w.set_offsets if sets else None, w.set_members if sets else None,
                            a1, f, m_sel)
            r = dx.detox_aggregate(p, X)
            res += [r["out"], r["winner"]] + ([r["sel"]] if r["sel"] is not None else [])
        torch.cuda.synchronize()
        return [t.clone() for t in res]

    first, second = run_all(), run_all()
    assert len(first) == len(second)
    for k, (a, b) in enumerate(zip(first, second)):
        assert torch.equal(a.view(torch.uint8), b.view(torch.uint8)), f"output {k} differs between two runs"


# ------------------------------------------------------------------------------------- guard bands

@pytest.mark.parametrize("n,d", [(15, 4097), (45, 10_001), (45, 640_003), (105, 5003), (225, 2050), (300, 777)])
def test_nothing_is_written_outside_the_callers_buffers(n, d):
    """Every output and workspace buffer sits between two guard bands holding a fixed pattern; after each call the
    bands must be untouched.  Row strides are the padded ones of the workloads, so a row's padding columns (also
    pattern-filled here) must stay untouched as well."""
    w = workload(n, d)
    X = w.X[:, :d]
    G, S, ld = w.G, w.S, w.ld
    bufs = []

    def guarded(numel, dtype=torch.float32):
        g = Guarded(numel, dtype)
        bufs.append(g)
        return g.view

    def rows_buf(rows):
        g = Guarded(rows * ld)
        bufs.append(g)
        return g.view.view(rows, ld)[:, :d], g.view.view(rows, ld)[:, d:]

    def ws(nbytes):
        return guarded(max(nbytes, 256), torch.uint8)

    pads = []
    Z, zpad = rows_buf(G); pads.append(zpad)
    M, mpad = rows_buf(S); pads.append(mpad)
    win = guarded(G, torch.int32)
    out = guarded(d)
    dx.detox_vote(X, 3, w.members, Z=Z, winner=win, ws=ws(dx.detox_vote_workspace_bytes(n, 3)))
    dx.detox_vote(X, 3, w.members, want_Z=False, winner=win, ws=ws(dx.detox_vote_workspace_bytes(n, 3)))
    dx.detox_hier_mean(Z, w.set_offsets, w.set_members, M=M)
    dx.detox_vote_hier_mean(X, 3, w.members, w.set_offsets, w.set_members, M=M, winner=win,
                            ws=ws(dx.detox_vote_workspace_bytes(n, 3)))
    dx.agg_coord_median(X, out=out)
    dx.agg_trimmed_mean(X, n // 4, out=out)
    dx.agg_sign_majority(X, out=out)
    dx.agg_geometric_median(Z[: min(G, 32)], iters=3, out=out,
                            ws=ws(dx.load().agg_geometric_median_workspace_bytes(min(G, 32), d)))
    f = n // 10
    dx.agg_multikrum(X, f, n - f, out=out, sel=guarded(n - f, torch.int32), scores=guarded(n, torch.float64),
                     ws=ws(dx.agg_multikrum_workspace_bytes(n, d)))
    dx.agg_bulyan(X, f, out=out, sel=guarded(n - 2 * f, torch.int32), ws=ws(dx.agg_bulyan_workspace_bytes(n, d)))
    fv = 1 if G >= 7 else 0
    for a0, a1, ff, m_sel in [(dx.AGG_MEAN, dx.AGG_COORD_MEDIAN, 0, 1), (dx.AGG_NONE, dx.AGG_COORD_MEDIAN, 0, 1),
                              (dx.AGG_NONE, dx.AGG_MULTIKRUM, fv, G - fv), (dx.AGG_NONE, dx.AGG_BULYAN, fv, 1),
                              (dx.AGG_MEAN, dx.AGG_MULTIKRUM, 0, 1), (dx.AGG_MULTIKRUM, dx.AGG_MEAN, 0, 0)]:
        sets = a0 != dx.AGG_NONE
        p = dx.Pipeline(n, 3, d, w.members, a0, w.set_offsets if sets else None, w.set_members if sets else None,
                        a1, ff, m_sel)
        k = max(p.n_selected, 1)
        dx.detox_aggregate(p, X, out=out, winner=win, sel=guarded(k, torch.int32), sel_workers=guarded(k, torch.int32),
                           ws=ws(p.workspace_bytes()))
    torch.cuda.synchronize()
    for k, g in enumerate(bufs):
        assert g.intact(), f"guard band of buffer {k} was overwritten"
    for p_ in pads:
        if p_.numel():
            assert bool((p_.contiguous().view(torch.int32) == PATTERN).all().item()), "row padding was overwritten"


# ------------------------------------------------------------------------------------- bounded waits, status word

def test_a_wait_that_nothing_completes_gives_up_and_reports_it():
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    dx.detox_selftest_bounded_wait(100_000, status=status)
    torch.cuda.synchronize()                       # returns: the kernel ended by itself
    assert int(status.item()) == 5                 # DETOX_ERR_TIMEOUT
    assert dx.status_string(5) == "device-side wait timed out"
    # the context is intact: ordinary work still runs
    X = torch.randn(9, 1000, device=DEV)
    assert torch.isfinite(dx.agg_coord_median(X)).all()


@pytest.mark.parametrize("a0,a1,G", [("none", "multikrum", 35), ("none", "bulyan", 12), ("mean", "multikrum", 35),
                                    ("multikrum", "mean", 35)])
def test_pipeline_status_word_is_the_first_word_of_its_workspace_and_clear(a0, a1, G):
    n, d = 3 * G, 650_000 if G <= 16 else 9000
    w = workload(n, d, q=0, attack="none")
    code = {"none": dx.AGG_NONE, "mean": dx.AGG_MEAN, "multikrum": dx.AGG_MULTIKRUM, "bulyan": dx.AGG_BULYAN}
    sets = a0 != "none"
    p = dx.Pipeline(n, 3, d, w.members, code[a0], w.set_offsets if sets else None, w.set_members if sets else None,
                    code[a1], 1, 0 if a0 == "multikrum" else 2)
    ws = torch.full((p.workspace_bytes(),), 0xFF, dtype=torch.uint8, device=DEV)
    dx.detox_aggregate(p, w.X[:, :d], ws=ws)
    assert dx.read_status(ws) == 0
    dx.check_status(ws)
