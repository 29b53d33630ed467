"""CPU oracle for the DETOX aggregation path: thin ctypes wrapper over oracle/detox_oracle.c.

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by the smoke check and by the benchmark's CPU-baseline
leg; never by the CUDA library or its Python binding.  Every array is a host numpy array; fp32 in,
fp64 accumulation inside, fp32 (values) / int32 (indices) out.

Pin status: vote, hier_mean, coord_median, trimmed_mean, sqdist are pinned by tests/test_oracle_pins.py.
Krum scores, Multi-Krum and Bulyan are pinned to brute-force subset definitions on tiny inputs and
to their reductions; beyond those cases: parity unpinned (the paper cites them without a definition).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "detox_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile detox_oracle.c with gcc (OpenMP over coordinates / row pairs)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_F = ctypes.POINTER(ctypes.c_float)
_D = ctypes.POINTER(ctypes.c_double)
_I = ctypes.POINTER(ctypes.c_int32)
_U8 = ctypes.POINTER(ctypes.c_uint8)
_i64 = ctypes.c_int64
_int = ctypes.c_int


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        lib.oracle_num_threads.restype = _int
        lib.oracle_vote.argtypes = [_F, _i64, _int, _int, _i64, _I, _F, _i64, _I]
        lib.oracle_hier_mean.argtypes = [_F, _i64, _int, _i64, _I, _I, _int, _F, _i64]
        lib.oracle_mean_rows.argtypes = [_F, _i64, _i64, _I, _int, _F]
        lib.oracle_coord_median.argtypes = [_F, _i64, _int, _i64, _I, _F]
        lib.oracle_sqdist.argtypes = [_F, _i64, _int, _i64, _D]
        lib.oracle_krum_scores.argtypes = [_D, _int, _U8, _int, _D]
        lib.oracle_multikrum.argtypes = [_F, _i64, _int, _i64, _int, _int, _F, _I, _D, _D]
        lib.oracle_bulyan_select.argtypes = [_D, _int, _int, _I]
        lib.oracle_trimmed_around_median.argtypes = [_F, _i64, _i64, _I, _int, _int, _F]
        lib.oracle_trimmed_mean.argtypes = [_F, _i64, _int, _i64, _int, _F]
        lib.oracle_geometric_median.argtypes = [_F, _i64, _int, _i64, _int, ctypes.c_double, _F]
        lib.oracle_sign_majority.argtypes = [_F, _i64, _int, _i64, _I, _F]
        lib.oracle_bulyan.argtypes = [_F, _i64, _int, _i64, _int, _F, _I, _D]
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _mat(X) -> Tuple[np.ndarray, int]:
    """Accept a torch CPU tensor or a numpy array [rows, cols] whose rows are contiguous; return (array, ld)."""
    if hasattr(X, "detach"):
        X = X.detach().cpu().numpy()
    X = np.asarray(X)
    if X.dtype != np.float32 or X.ndim != 2:
        raise TypeError("expected a 2-D float32 matrix")
    if X.shape[1] > 1 and X.strides[1] != 4:
        X = np.ascontiguousarray(X)
    if X.strides[0] % 4 != 0:
        X = np.ascontiguousarray(X)
    return X, (X.strides[0] // 4 if X.shape[0] > 1 else max(X.shape[1], 1))


def _fp(a: np.ndarray):
    return a.ctypes.data_as(_F)


def _ip(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(_I)


def _idx(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle: bad arguments to {what}")


def vote(X, members: Sequence[int], r: int):
    """Majority vote per node group.  Returns (Z [G, d] float32, winner [G] int32)."""
    X, ld = _mat(X)
    n, d = X.shape
    members = _idx(members)
    G = n // r
    Z = np.empty((G, d), dtype=np.float32)
    winner = np.empty(G, dtype=np.int32)
    _check(_load().oracle_vote(_fp(X), ld, n, r, d, _ip(members), _fp(Z), d, _ip(winner)), "vote")
    return Z, winner


def hier_mean(Z, set_offsets, set_members):
    Z, ldz = _mat(Z)
    G, d = Z.shape
    so, sm = _idx(set_offsets), _idx(set_members)
    S = len(so) - 1
    M = np.empty((S, d), dtype=np.float32)
    _check(_load().oracle_hier_mean(_fp(Z), ldz, G, d, _ip(so), _ip(sm), S, _fp(M), d), "hier_mean")
    return M


def mean_rows(X, rows=None):
    X, ld = _mat(X)
    m, d = X.shape
    rows = _idx(np.arange(m) if rows is None else rows)
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_mean_rows(_fp(X), ld, d, _ip(rows), len(rows), _fp(out)), "mean_rows")
    return out


def coord_median(X, rows=None):
    X, ld = _mat(X)
    m, d = X.shape
    r = None if rows is None else _idx(rows)
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_coord_median(_fp(X), ld, m if r is None else len(r), d, _ip(r), _fp(out)), "coord_median")
    return out


def trimmed_mean(X, trim: int):
    X, ld = _mat(X)
    m, d = X.shape
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_trimmed_mean(_fp(X), ld, m, d, trim, _fp(out)), "trimmed_mean")
    return out


def sign_majority(X, rows=None):
    X, ld = _mat(X)
    m, d = X.shape
    r = None if rows is None else _idx(rows)
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_sign_majority(_fp(X), ld, m if r is None else len(r), d, _ip(r), _fp(out)), "sign_majority")
    return out


def geometric_median(X, iters: int = 32, eps: float = 1e-12):
    X, ld = _mat(X)
    m, d = X.shape
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_geometric_median(_fp(X), ld, m, d, iters, float(eps), _fp(out)), "geometric_median")
    return out


def sqdist(X):
    X, ld = _mat(X)
    m, d = X.shape
    D = np.empty((m, m), dtype=np.float64)
    _check(_load().oracle_sqdist(_fp(X), ld, m, d, D.ctypes.data_as(_D)), "sqdist")
    return D


def krum_scores(D: np.ndarray, f: int, alive=None):
    D = np.ascontiguousarray(D, dtype=np.float64)
    m = D.shape[0]
    a = None if alive is None else np.ascontiguousarray(np.asarray(alive, dtype=np.uint8))
    sc = np.empty(m, dtype=np.float64)
    _check(_load().oracle_krum_scores(D.ctypes.data_as(_D), m, None if a is None else a.ctypes.data_as(_U8), f,
                                      sc.ctypes.data_as(_D)), "krum_scores")
    return sc


def multikrum(X, f: int, m_sel: int, want_out: bool = True):
    """Returns (out [d] float32 or None, sel [m_sel] int32 ascending, scores [m] float64, D [m, m] float64)."""
    X, ld = _mat(X)
    m, d = X.shape
    out = np.empty(d, dtype=np.float32) if want_out else None
    sel = np.empty(max(m_sel, 0), dtype=np.int32)
    sc = np.empty(m, dtype=np.float64)
    D = np.empty((m, m), dtype=np.float64)
    _check(_load().oracle_multikrum(_fp(X), ld, m, d, f, m_sel, None if out is None else _fp(out), _ip(sel),
                                    sc.ctypes.data_as(_D), D.ctypes.data_as(_D)), "multikrum")
    return out, sel, sc, D


def bulyan_select(D: np.ndarray, f: int):
    D = np.ascontiguousarray(D, dtype=np.float64)
    m = D.shape[0]
    sel = np.empty(max(m - 2 * f, 0), dtype=np.int32)
    _check(_load().oracle_bulyan_select(D.ctypes.data_as(_D), m, f, _ip(sel)), "bulyan_select")
    return sel


def trimmed_around_median(X, rows, beta: int):
    X, ld = _mat(X)
    _, d = X.shape
    rows = _idx(rows)
    out = np.empty(d, dtype=np.float32)
    _check(_load().oracle_trimmed_around_median(_fp(X), ld, d, _ip(rows), len(rows), beta, _fp(out)),
           "trimmed_around_median")
    return out


def bulyan(X, f: int, want_out: bool = True):
    """Returns (out [d] float32 or None, sel [m - 2f] int32 in selection order, D [m, m] float64)."""
    X, ld = _mat(X)
    m, d = X.shape
    out = np.empty(d, dtype=np.float32) if want_out else None
    sel = np.empty(max(m - 2 * f, 0), dtype=np.int32)
    D = np.empty((m, m), dtype=np.float64)
    _check(_load().oracle_bulyan(_fp(X), ld, m, d, f, None if out is None else _fp(out), _ip(sel),
                                 D.ctypes.data_as(_D)), "bulyan")
    return out, sel, D


A0_NONE, A0_MEAN = "none", "mean"


def detox_aggregate(X, members, r: int, a0: str, set_offsets, set_members, a1: str, f: int = 0,
                    m_sel: int = 1, gm_iters: int = 32, gm_eps: float = 1e-12):
    """Algorithm 1 (filtering step + hierarchical aggregation) with A_0 in {none, mean, multikrum, bulyan}
    and A_1 in {mean, coord_median, multikrum, bulyan}.

    Returns dict(out, winner, sel) where sel indexes the rows that entered A_1 (votes when a0 is
    "none", sets when a0 is "mean"), and sel_workers maps them through winner[] when a0 is "none".
    """
    Z, winner = vote(X, members, r)
    sel = None
    sel_votes = None
    if a0 in ("multikrum", "bulyan"):
        # Section 5.2, setups 2 and 3: the robust aggregator inside every vote group, then A_1 over the results.
        # f and m_sel belong to A_0; m_sel = 0 means "all but f" of each group.
        so, sm = np.asarray(set_offsets), np.asarray(set_members)
        outs, sel_votes = [], []
        for s in range(len(so) - 1):
            idx = sm[so[s]:so[s + 1]]
            if a0 == "multikrum":
                keep = m_sel if m_sel > 0 else max(len(idx) - f, 1)
                o, loc, _, _ = multikrum(Z[idx], f, keep)
            else:
                o, loc, _ = bulyan(Z[idx], f)
            outs.append(o)
            sel_votes.extend(int(v) for v in idx[loc])
        rows = np.stack(outs)
        sel_votes = np.asarray(sel_votes, dtype=np.int32)
    elif a0 == "sign_majority":
        so, sm = np.asarray(set_offsets), np.asarray(set_members)
        rows = np.stack([sign_majority(Z, sm[so[s]:so[s + 1]]) for s in range(len(so) - 1)])
    else:
        rows = Z if a0 == A0_NONE else hier_mean(Z, set_offsets, set_members)
    if a1 == "mean":
        out = mean_rows(rows)
    elif a1 == "sign_majority":
        out = sign_majority(rows)
    elif a1 == "coord_median":
        out = coord_median(rows)
    elif a1 == "trimmed_mean":
        out = trimmed_mean(rows, f)
    elif a1 == "geometric_median":
        out = geometric_median(rows, gm_iters, gm_eps)
    elif a1 == "multikrum":
        out, sel, _, _ = multikrum(rows, f, m_sel)
    elif a1 == "bulyan":
        out, sel, _ = bulyan(rows, f)
    else:
        raise ValueError(a1)
    sel_workers = None
    if sel_votes is not None:
        sel, sel_workers = sel_votes, winner[sel_votes]
    elif sel is not None and a0 == A0_NONE:
        sel_workers = winner[sel]
    return dict(out=out, winner=winner, sel=sel, sel_workers=sel_workers, rows=rows, Z=Z)
