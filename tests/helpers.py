"""Shared test helpers (host side only): error norms and the near-tie screen for Krum-type decisions."""
import numpy as np

import oracle


def rel_l2(y, ref) -> float:
    y = np.asarray(y, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    num = np.linalg.norm(y - ref)
    return float(num) if den == 0.0 else float(num / den)


def _gap_after(sorted_scores: np.ndarray, k: int) -> float:
    """Relative gap between the k-th and (k+1)-th smallest *distinct-valued* neighbours at the cut."""
    a, b = sorted_scores[k - 1], sorted_scores[k]
    if a == b:
        return np.inf  # an exact tie is decided by index on both sides
    return abs(b - a) / max(abs(a), abs(b), 1e-300)


def multikrum_min_gap(scores: np.ndarray, m_sel: int) -> float:
    s = np.sort(scores)
    return np.inf if m_sel >= len(s) else _gap_after(s, m_sel)


def bulyan_min_gap(D: np.ndarray, f: int) -> float:
    """Smallest relative gap between the best and the next distinct score over all selection rounds."""
    m = D.shape[0]
    alive = np.ones(m, np.uint8)
    worst = np.inf
    for _ in range(m - 2 * f):
        sc = oracle.krum_scores(D, f, alive)
        live = np.sort(sc[alive.astype(bool)])
        best = live[0]
        others = live[(live != best) & np.isfinite(live)]   # (rows at infinite distance never compete)
        if len(others) and np.isfinite(best):
            worst = min(worst, abs(others[0] - best) / max(abs(others[0]), abs(best), 1e-300))
        pick = min((i for i in range(m) if alive[i]), key=lambda i: (sc[i], i))
        alive[pick] = 0
    return worst


def check_bulyan_selection(D: np.ndarray, f: int, sel, tol: float) -> bool:
    """Checks a Bulyan selection sequence against the oracle's scores, round by round, following the sequence
    itself: every pick must be a remaining row whose fp64 score is the minimum (ties: the lowest index) or, at a
    near-tie, within `tol` (relative) of the minimum.  Returns True when every pick was the oracle's own."""
    m = D.shape[0]
    alive = np.ones(m, np.uint8)
    exact = True
    assert len(sel) == m - 2 * f
    for rnd, pick in enumerate(int(x) for x in sel):
        sc = oracle.krum_scores(D, f, alive)
        best = min((i for i in range(m) if alive[i]), key=lambda i: (sc[i], i))
        assert 0 <= pick < m and alive[pick], f"round {rnd}: row {pick} is not a remaining row"
        if pick != best:
            exact = False
            gap = abs(sc[pick] - sc[best]) / max(abs(sc[best]), 1e-300)
            assert gap <= tol, f"round {rnd}: picked row {pick} (score {sc[pick]}) over row {best} ({sc[best]})"
        alive[pick] = 0
    return exact
