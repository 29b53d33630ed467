"""ctypes binding of libdetox.so: argument marshalling only.

Every function has the name and the meaning of the C entry point in include/detox.h.  Tensors are
torch CUDA tensors used as device memory; matrices may be column-sliced views (the row stride is
passed as `ld`).  Output and workspace buffers are created here when the caller passes none.  There
is no CPU path: if the library is not built, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libdetox.so")

AGG_NONE, AGG_MEAN, AGG_COORD_MEDIAN, AGG_MULTIKRUM, AGG_BULYAN, AGG_TRIMMED_MEAN, AGG_GEOMETRIC_MEDIAN, AGG_SIGN_MAJORITY = range(8)
MAX_ROWS, MAX_R = 1024, 15

EXPORTS = (
    "detox_status_string", "detox_vote_workspace_bytes", "detox_vote", "detox_vote_noalloc", "detox_hier_mean",
    "detox_vote_hier_mean",
    "agg_coord_median_workspace_bytes", "agg_coord_median", "agg_trimmed_mean", "agg_sign_majority", "agg_geometric_median_workspace_bytes", "agg_geometric_median", "agg_multikrum_workspace_bytes", "agg_multikrum",
    "agg_bulyan_workspace_bytes", "agg_bulyan", "detox_aggregate_workspace_bytes", "detox_aggregate",
    "detox_selftest_bounded_wait", "agg_pairwise_sqdist_workspace_bytes", "agg_pairwise_sqdist",
    "detox_kernel_launch_count", "detox_vote_hier_mean_many", "detox_tc_split_mode", "detox_tc_repeated_passes",
)


class DetoxError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {status_string(code)} (status {code})")


class PipelineDesc(ctypes.Structure):
    _fields_ = [
        ("n", ctypes.c_int32), ("r", ctypes.c_int32), ("d", ctypes.c_int64),
        ("members", ctypes.POINTER(ctypes.c_int32)),
        ("a0", ctypes.c_int32), ("n_sets", ctypes.c_int32),
        ("set_offsets", ctypes.POINTER(ctypes.c_int32)), ("set_members", ctypes.POINTER(ctypes.c_int32)),
        ("a1", ctypes.c_int32), ("f", ctypes.c_int32), ("m_sel", ctypes.c_int32),
        ("gm_iters", ctypes.c_int32), ("gm_eps", ctypes.c_float),
    ]


_lib = None
_vp, _i64, _int, _sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
_ip = ctypes.POINTER(ctypes.c_int32)


def load() -> ctypes.CDLL:
    """Load libdetox.so (built in-tree by paper_1907_12205_b200.build).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is not built; run `python -m paper_1907_12205_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    lib.detox_status_string.restype = ctypes.c_char_p
    lib.detox_status_string.argtypes = [_int]
    lib.detox_vote_workspace_bytes.restype = _sz
    lib.detox_vote_workspace_bytes.argtypes = [_int, _int]
    lib.detox_vote.argtypes = [_vp, _i64, _int, _int, _i64, _ip, _vp, _i64, _vp, _vp, _sz, _vp]
    lib.detox_vote_noalloc.argtypes = [_vp, _i64, _int, _int, _i64, _ip, _vp, _i64, _vp, _vp]
    lib.detox_vote_hier_mean.argtypes = [_vp, _i64, _int, _int, _i64, _ip, _ip, _ip, _int, _vp, _i64, _vp, _vp, _sz, _vp]
    lib.detox_hier_mean.argtypes = [_vp, _i64, _int, _i64, _ip, _ip, _int, _vp, _i64, _vp]
    for name in ("agg_coord_median", "agg_multikrum", "agg_bulyan"):
        fn = getattr(lib, name + "_workspace_bytes")
        fn.restype = _sz
        fn.argtypes = [_int, _i64]
    lib.agg_coord_median.argtypes = [_vp, _i64, _int, _i64, _vp, _vp, _sz, _vp]
    lib.agg_trimmed_mean.argtypes = [_vp, _i64, _int, _i64, _int, _vp, _vp]
    lib.agg_geometric_median_workspace_bytes.restype = _sz
    lib.agg_geometric_median_workspace_bytes.argtypes = [_int, _i64]
    lib.agg_geometric_median.argtypes = [_vp, _i64, _int, _i64, _int, ctypes.c_float, _vp, _vp, _sz, _vp]
    lib.agg_sign_majority.argtypes = [_vp, _i64, _int, _i64, _vp, _vp]
    lib.agg_multikrum.argtypes = [_vp, _i64, _int, _i64, _int, _int, _vp, _vp, _vp, _vp, _sz, _vp]
    lib.agg_bulyan.argtypes = [_vp, _i64, _int, _i64, _int, _vp, _vp, _vp, _sz, _vp]
    lib.detox_aggregate_workspace_bytes.restype = _sz
    lib.detox_aggregate_workspace_bytes.argtypes = [ctypes.POINTER(PipelineDesc)]
    lib.detox_aggregate.argtypes = [ctypes.POINTER(PipelineDesc), _vp, _i64, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
    lib.detox_selftest_bounded_wait.argtypes = [_vp, _i64, _vp]
    lib.agg_pairwise_sqdist_workspace_bytes.restype = _sz
    lib.agg_pairwise_sqdist_workspace_bytes.argtypes = [_int, _i64]
    lib.agg_pairwise_sqdist.argtypes = [_vp, _i64, _int, _i64, _vp, _vp, _sz, _vp]
    lib.detox_vote_hier_mean_many.argtypes = [_vp, _i64, _i64, _int, _int, _vp, _ip, _int, _vp, _i64, _vp, _vp]
    lib.detox_tc_split_mode.argtypes = [_int]
    lib.detox_tc_split_mode.restype = _int
    lib.detox_tc_repeated_passes.restype = ctypes.c_ulonglong
    lib.detox_tc_repeated_passes.argtypes = []
    lib.detox_kernel_launch_count.restype = ctypes.c_ulonglong
    lib.detox_kernel_launch_count.argtypes = []
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().detox_status_string(int(code)).decode()


def _check(code: int, what: str):
    if code != 0:
        raise DetoxError(code, what)


def _mat(X: torch.Tensor):
    if not (isinstance(X, torch.Tensor) and X.is_cuda and X.dtype == torch.float32 and X.dim() == 2):
        raise TypeError("expected a 2-D float32 CUDA tensor")
    if X.shape[1] > 1 and X.stride(1) != 1:
        raise ValueError("rows must be contiguous")
    ld = X.stride(0) if X.shape[0] > 1 else max(X.stride(0), X.shape[1])
    return X.data_ptr(), int(ld), int(X.shape[0]), int(X.shape[1])


def _host_i32(a: Sequence[int]) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ws(nbytes: int, ws: Optional[torch.Tensor], device):
    if ws is None:
        ws = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)
    return ws, ws.data_ptr(), ws.numel() * ws.element_size()


def read_status(ws: torch.Tensor, stream=None) -> int:
    """The device status word of a finished call: the first int32 of the workspace that was passed to agg_multikrum,
    agg_bulyan or detox_aggregate.  Synchronises the stream.  0, or 5 (DETOX_ERR_TIMEOUT) when a bounded device-side
    wait ran out and the call's outputs are not valid."""
    (torch.cuda.current_stream() if stream is None else stream).synchronize()
    return int(ws[:4].view(torch.int32).item())


def check_status(ws: torch.Tensor, what: str = "device status", stream=None):
    """Raises DetoxError if the device status word of a finished call is not 0 (synchronises the stream)."""
    _check(read_status(ws, stream), what)


def detox_selftest_bounded_wait(limit_cycles: int = 100_000, status: Optional[torch.Tensor] = None, stream=None):
    """Runs the library's bounded wait on a barrier that nothing completes; returns the int32 status tensor, which
    reads 5 (DETOX_ERR_TIMEOUT) once the stream has been synchronised."""
    if status is None:
        status = torch.empty(1, dtype=torch.int32, device="cuda")
    _check(load().detox_selftest_bounded_wait(status.data_ptr(), int(limit_cycles), _stream(stream)),
           "detox_selftest_bounded_wait")
    return status


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def detox_vote_workspace_bytes(n: int, r: int) -> int:
    return int(load().detox_vote_workspace_bytes(n, r))


def detox_vote(X, r: int, members, Z: Optional[torch.Tensor] = None, winner: Optional[torch.Tensor] = None,
               want_Z: bool = True, ws: Optional[torch.Tensor] = None, stream=None):
    """Majority vote per node group.  Returns (Z or None, winner)."""
    lib = load()
    xp, ld, n, d = _mat(X)
    mem = _host_i32(members)
    if Z is None and want_Z:
        ldz = (d + 31) // 32 * 32
        Z = torch.empty((n // max(r, 1), ldz), dtype=torch.float32, device=X.device)[:, :d]
    if winner is None:
        winner = torch.empty(max(n // max(r, 1), 1), dtype=torch.int32, device=X.device)[: n // max(r, 1)]
    zp, ldz = (None, 0) if Z is None else (Z.data_ptr(), Z.stride(0) if Z.shape[0] > 1 else max(Z.stride(0), d))
    ws, wp, wb = _ws(lib.detox_vote_workspace_bytes(n, r), ws, X.device)
    _check(lib.detox_vote(xp, ld, n, r, d, mem.ctypes.data_as(_ip), zp, ldz, winner.data_ptr(), wp, wb,
                          _stream(stream)), "detox_vote")
    return Z, winner


NOALLOC_MAX_GROUPS = 256


def detox_vote_noalloc(X, r: int, members, Z: torch.Tensor, winner: torch.Tensor, stream=None):
    """detox_vote for callers that cannot allocate: the scratch is a fixed array inside the library,
    and Z (or None) and winner must be passed in, so neither the library nor this wrapper allocates
    device memory.  At most NOALLOC_MAX_GROUPS node groups.  Calls that overlap on the GPU race on
    the shared scratch; the first call on a device should come before any stream capture."""
    lib = load()
    xp, ld, n, d = _mat(X)
    mem = _host_i32(members)
    zp, ldz = (None, 0) if Z is None else (Z.data_ptr(), Z.stride(0) if Z.shape[0] > 1 else max(Z.stride(0), d))
    _check(lib.detox_vote_noalloc(xp, ld, n, r, d, mem.ctypes.data_as(_ip), zp, ldz, winner.data_ptr(),
                                  _stream(stream)), "detox_vote_noalloc")
    return Z, winner


def detox_hier_mean(Z, set_offsets, set_members, M: Optional[torch.Tensor] = None, stream=None):
    lib = load()
    zp, ldz, G, d = _mat(Z)
    so, sm = _host_i32(set_offsets), _host_i32(set_members)
    S = len(so) - 1
    if M is None:
        ldm = (d + 31) // 32 * 32
        M = torch.empty((max(S, 1), ldm), dtype=torch.float32, device=Z.device)[:S, :d]
    ldm = M.stride(0) if M.shape[0] > 1 else max(M.stride(0), d)
    _check(lib.detox_hier_mean(zp, ldz, G, d, so.ctypes.data_as(_ip), sm.ctypes.data_as(_ip), S, M.data_ptr(), ldm,
                               _stream(stream)), "detox_hier_mean")
    return M


def detox_vote_hier_mean(X, r: int, members, set_offsets, set_members, M: Optional[torch.Tensor] = None,
                         winner: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """Vote and mean over each vote set in one pass.  Returns (M [S, d], winner [G])."""
    lib = load()
    xp, ld, n, d = _mat(X)
    mem, so, sm = _host_i32(members), _host_i32(set_offsets), _host_i32(set_members)
    S = len(so) - 1
    if M is None:
        ldm = (d + 31) // 32 * 32
        M = torch.empty((max(S, 1), ldm), dtype=torch.float32, device=X.device)[:S, :d]
    ldm = M.stride(0) if M.shape[0] > 1 else max(M.stride(0), d)
    if winner is None:
        winner = torch.empty(max(n // max(r, 1), 1), dtype=torch.int32, device=X.device)[: n // max(r, 1)]
    ws, wp, wb = _ws(lib.detox_vote_workspace_bytes(n, r), ws, X.device)
    _check(lib.detox_vote_hier_mean(xp, ld, n, r, d, mem.ctypes.data_as(_ip), so.ctypes.data_as(_ip),
                                    sm.ctypes.data_as(_ip), S, M.data_ptr(), ldm, winner.data_ptr(), wp, wb,
                                    _stream(stream)), "detox_vote_hier_mean")
    return M, winner


def detox_vote_hier_mean_many(X, r: int, members_dev: torch.Tensor, set_offsets=None, M: Optional[torch.Tensor] = None,
                              winner: Optional[torch.Tensor] = None, stream=None):
    """Vote and set means for very many nodes with short vectors.  members_dev: int32 CUDA tensor [n];
    set_offsets: host, in groups (None: votes only).  Returns (M [S, d] or None, winner [n / r])."""
    lib = load()
    xp, ld, n, d = _mat(X)
    if not (members_dev.is_cuda and members_dev.dtype == torch.int32 and members_dev.numel() == n):
        raise TypeError("members_dev: int32 CUDA tensor with one entry per node")
    G = n // max(r, 1)
    if winner is None:
        winner = torch.empty(max(G, 1), dtype=torch.int32, device=X.device)[:G]
    so, S, mp, ldm = None, 0, None, 0
    if set_offsets is not None:
        so = _host_i32(set_offsets)
        S = len(so) - 1
        if M is None:
            M = torch.empty((max(S, 1), (d + 31) // 32 * 32), dtype=torch.float32, device=X.device)[:S, :d]
        mp, ldm = M.data_ptr(), (M.stride(0) if M.shape[0] > 1 else max(M.stride(0), d))
    _check(lib.detox_vote_hier_mean_many(xp, ld, n, r, d, members_dev.data_ptr(),
                                         None if so is None else so.ctypes.data_as(_ip), S, mp, ldm, winner.data_ptr(),
                                         _stream(stream)), "detox_vote_hier_mean_many")
    return M, winner


def agg_coord_median_workspace_bytes(m: int, d: int) -> int:
    return int(load().agg_coord_median_workspace_bytes(m, d))


def agg_coord_median(X, out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    _check(lib.agg_coord_median(xp, ld, m, d, out.data_ptr(), _ptr(ws), 0 if ws is None else ws.numel(),
                                _stream(stream)), "agg_coord_median")
    return out


def agg_trimmed_mean(X, trim: int, out: Optional[torch.Tensor] = None, stream=None):
    """Coordinate-wise mean after dropping the `trim` smallest and `trim` largest values."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    _check(lib.agg_trimmed_mean(xp, ld, m, d, trim, out.data_ptr(), _stream(stream)), "agg_trimmed_mean")
    return out


def agg_sign_majority(X, out: Optional[torch.Tensor] = None, stream=None):
    """Coordinate-wise sign(sum of signs): -1, 0 or +1 per coordinate."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    _check(lib.agg_sign_majority(xp, ld, m, d, out.data_ptr(), _stream(stream)), "agg_sign_majority")
    return out


def agg_geometric_median(X, iters: int = 32, eps: float = 1e-12, out: Optional[torch.Tensor] = None,
                         ws: Optional[torch.Tensor] = None, stream=None):
    """Geometric median of at most 32 rows by `iters` Weiszfeld iterations started at the mean."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    ws, wp, wb = _ws(lib.agg_geometric_median_workspace_bytes(m, d), ws, X.device)
    _check(lib.agg_geometric_median(xp, ld, m, d, iters, eps, out.data_ptr(), wp, wb, _stream(stream)),
           "agg_geometric_median")
    return out


SPLIT_AUTO, SPLIT_TF32 = 0, 1


def tc_split_mode(mode: int = -1) -> int:
    """Sets which operand split the tensor-core distance pass tries first (SPLIT_AUTO: fp16 pairs, SPLIT_TF32);
    returns the previous mode; without an argument only queries."""
    return int(load().detox_tc_split_mode(int(mode)))


def tc_repeated_passes() -> int:
    """Calls on the current device whose tensor-core distance pass had to be repeated so far (synchronises)."""
    return int(load().detox_tc_repeated_passes())


def kernel_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load().detox_kernel_launch_count())


def agg_pairwise_sqdist_workspace_bytes(m: int, d: int) -> int:
    return int(load().agg_pairwise_sqdist_workspace_bytes(m, d))


def agg_pairwise_sqdist(X, D: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """Squared distances between the rows: D [m, m] float64, symmetric, zero diagonal."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if D is None:
        D = torch.empty((m, m), dtype=torch.float64, device=X.device)
    ws, wp, wb = _ws(lib.agg_pairwise_sqdist_workspace_bytes(m, d), ws, X.device)
    _check(lib.agg_pairwise_sqdist(xp, ld, m, d, D.data_ptr(), wp, wb, _stream(stream)), "agg_pairwise_sqdist")
    return D


def agg_multikrum_workspace_bytes(m: int, d: int) -> int:
    return int(load().agg_multikrum_workspace_bytes(m, d))


def agg_multikrum(X, f: int, m_sel: int, out: Optional[torch.Tensor] = None, sel: Optional[torch.Tensor] = None,
                  scores: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None, stream=None):
    """Returns (out [d] float32, sel [m_sel] int32 ascending, scores [m] float64)."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    if sel is None:
        sel = torch.empty(max(m_sel, 1), dtype=torch.int32, device=X.device)[: max(m_sel, 0)]
    if scores is None:
        scores = torch.empty(m, dtype=torch.float64, device=X.device)
    ws, wp, wb = _ws(lib.agg_multikrum_workspace_bytes(m, d), ws, X.device)
    _check(lib.agg_multikrum(xp, ld, m, d, f, m_sel, out.data_ptr(), sel.data_ptr(), scores.data_ptr(), wp, wb,
                             _stream(stream)), "agg_multikrum")
    return out, sel, scores


def agg_bulyan_workspace_bytes(m: int, d: int) -> int:
    return int(load().agg_bulyan_workspace_bytes(m, d))


def agg_bulyan(X, f: int, out: Optional[torch.Tensor] = None, sel: Optional[torch.Tensor] = None,
               ws: Optional[torch.Tensor] = None, stream=None):
    """Returns (out [d] float32, sel [m - 2f] int32 in selection order)."""
    lib = load()
    xp, ld, m, d = _mat(X)
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=X.device)
    if sel is None:
        sel = torch.empty(max(m - 2 * f, 1), dtype=torch.int32, device=X.device)[: max(m - 2 * f, 0)]
    ws, wp, wb = _ws(lib.agg_bulyan_workspace_bytes(m, d), ws, X.device)
    _check(lib.agg_bulyan(xp, ld, m, d, f, out.data_ptr(), sel.data_ptr(), wp, wb, _stream(stream)), "agg_bulyan")
    return out, sel


class Pipeline:
    """Holds the host-side description of one DETOX configuration (Algorithm 1 + Algorithm 2)."""

    def __init__(self, n: int, r: int, d: int, members, a0: int = AGG_NONE, set_offsets=None, set_members=None,
                 a1: int = AGG_COORD_MEDIAN, f: int = 0, m_sel: int = 1, gm_iters: int = 32, gm_eps: float = 1e-12):
        self.members = _host_i32(members)
        self.set_offsets = None if set_offsets is None else _host_i32(set_offsets)
        self.set_members = None if set_members is None else _host_i32(set_members)
        self.desc = PipelineDesc()
        self.desc.n, self.desc.r, self.desc.d = n, r, d
        self.desc.members = self.members.ctypes.data_as(_ip)
        self.desc.a0 = a0
        self.desc.n_sets = 0 if self.set_offsets is None else len(self.set_offsets) - 1
        self.desc.set_offsets = None if self.set_offsets is None else self.set_offsets.ctypes.data_as(_ip)
        self.desc.set_members = None if self.set_members is None else self.set_members.ctypes.data_as(_ip)
        self.desc.a1, self.desc.f, self.desc.m_sel = a1, f, m_sel
        self.desc.gm_iters, self.desc.gm_eps = gm_iters, gm_eps
        self.n, self.r, self.d, self.a0, self.a1, self.f, self.m_sel = n, r, d, a0, a1, f, m_sel

    @property
    def G(self) -> int:
        return self.n // self.r

    @property
    def rows_into_a1(self) -> int:
        return self.desc.n_sets if self.a0 != AGG_NONE else self.G

    @property
    def n_selected(self) -> int:
        if self.a0 in (AGG_MULTIKRUM, AGG_BULYAN):      # chosen inside every vote set, concatenated in set order
            sizes = np.diff(self.set_offsets)
            if self.a0 == AGG_BULYAN:
                return int(sum(k - 2 * self.f for k in sizes))
            return int(sum(self.m_sel if self.m_sel > 0 else max(k - self.f, 1) for k in sizes))
        if self.a1 == AGG_MULTIKRUM:
            return self.m_sel
        if self.a1 == AGG_BULYAN:
            return self.rows_into_a1 - 2 * self.f
        return 0

    def workspace_bytes(self) -> int:
        return int(load().detox_aggregate_workspace_bytes(ctypes.byref(self.desc)))


def detox_aggregate_workspace_bytes(pipe: Pipeline) -> int:
    return pipe.workspace_bytes()


def detox_aggregate(pipe: Pipeline, X, out: Optional[torch.Tensor] = None, winner: Optional[torch.Tensor] = None,
                    sel: Optional[torch.Tensor] = None, sel_workers: Optional[torch.Tensor] = None,
                    ws: Optional[torch.Tensor] = None, stream=None):
    """Vote -> A_0 -> A_1.  Returns dict(out, winner, sel, sel_workers).

    sel lists the rows chosen by the Krum-type stage: rows that entered A_1 when A_1 is Multi-Krum / Bulyan;
    vote (group) indices, set after set, when A_0 is Multi-Krum / Bulyan.  sel_workers gives the same rows
    as worker ids whenever sel indexes votes."""
    lib = load()
    xp, ld, n, d = _mat(X)
    if n != pipe.n or d != pipe.d:
        raise ValueError("X does not match the pipeline description")
    dev = X.device
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=dev)
    if winner is None:
        winner = torch.empty(pipe.G, dtype=torch.int32, device=dev)
    k = pipe.n_selected
    if k > 0 and sel is None:
        sel = torch.empty(k, dtype=torch.int32, device=dev)
    if k > 0 and sel_workers is None and pipe.a0 != AGG_MEAN:
        sel_workers = torch.empty(k, dtype=torch.int32, device=dev)
    need = pipe.workspace_bytes()
    if need == 0:
        raise DetoxError(1, "detox_aggregate_workspace_bytes")
    ws, wp, wb = _ws(need, ws, dev)
    _check(lib.detox_aggregate(ctypes.byref(pipe.desc), xp, ld, out.data_ptr(), winner.data_ptr(), _ptr(sel),
                               _ptr(sel_workers), wp, wb, _stream(stream)), "detox_aggregate")
    return dict(out=out, winner=winner, sel=sel, sel_workers=sel_workers)
