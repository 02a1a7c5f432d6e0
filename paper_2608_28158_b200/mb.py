"""ctypes binding of the harts_mb_* entry points (same names as the C ABI).  Argument marshalling only."""
from __future__ import annotations

import ctypes as C

import numpy as np

from .binding import lib, _check, _I32P

_I64P = C.POINTER(C.c_int64)
_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64
SOURCES = {0: "natural", 1: "exact", 2: "evolved", 3: "greedy"}


class _MbView(C.Structure):
    _fields_ = [(n, _i32) for n in ("n_traj", "n_mb", "D", "source", "refined", "natural_mb", "n_candidates",
                                    "reserved")] + \
               [("T", _i64), ("J", _i64 * 3), ("total_work_all", _i64), ("natural_work", _i64)] + \
               [(n, _I32P) for n in ("traj_leaf", "traj_len", "traj_lcp", "traj_mb")] + \
               [("mb_work", _I64P), ("mb_replica", _I32P), ("mb_slot", _I32P)]


lib.harts_mb_plan.argtypes = [_i32, _I32P, _I32P, _I32P, _I32P, _i32, _i64, C.POINTER(_vp)]
lib.harts_mb_plan_free.argtypes = [_vp]
lib.harts_mb_plan_free.restype = None
lib.harts_mb_plan_view.argtypes = [_vp, C.POINTER(_MbView)]
lib.harts_mb_extract.argtypes = [_vp, _i32, _i32, _i32, _I32P, _I32P, _I32P, _I32P, _I32P, _I32P, _I32P]
lib.harts_mb_greedy_trace.argtypes = [_vp, _i32, _i32, _i32, _I32P, _I32P, _I32P, _I64P, _I32P]
for _n in ("harts_mb_plan", "harts_mb_plan_view", "harts_mb_extract", "harts_mb_greedy_trace"):
    getattr(lib, _n).restype = _i32


class MbPlan:
    """Host plan (owned by the library) with its arrays copied into numpy."""

    def __init__(self, handle):
        self._h = handle
        v = _MbView()
        _check(lib.harts_mb_plan_view(handle, C.byref(v)), "harts_mb_plan_view")
        for n in ("n_traj", "n_mb", "D", "refined", "natural_mb", "n_candidates", "T", "total_work_all", "natural_work"):
            setattr(self, n, int(getattr(v, n)))
        self.source = SOURCES[int(v.source)]
        self.J = tuple(int(x) for x in v.J)
        arr = lambda p, n: np.ctypeslib.as_array(p, shape=(n,)).copy() if n else np.zeros(0, np.int32)  # noqa: E731
        for n in ("traj_leaf", "traj_len", "traj_lcp", "traj_mb"):
            setattr(self, n, arr(getattr(v, n), self.n_traj))
        for n in ("mb_work", "mb_replica", "mb_slot"):
            setattr(self, n, arr(getattr(v, n), self.n_mb))

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h:
            lib.harts_mb_plan_free(h)

    def greedy_trace(self, order, policy):
        """(trajectory, microbatch, created, delta) of every step of the greedy's placement pass."""
        n = self.n_traj
        x, mb, created = (np.empty(n, np.int32) for _ in range(3))
        delta = np.empty(n, np.int64)
        cnt = _i32(0)
        ip = lambda a: a.ctypes.data_as(_I32P)  # noqa: E731
        _check(lib.harts_mb_greedy_trace(self._h, order, policy, n, ip(x), ip(mb), ip(created),
                                         delta.ctypes.data_as(_I64P), C.byref(cnt)), "harts_mb_greedy_trace")
        return x, mb, created, delta

    def extract(self, mb):
        """(tree_node_ptr, node_parent, node_fork_off, node_len, node_src) of one microbatch's compact forest."""
        nt, nn = _i32(0), _i32(0)
        _check(lib.harts_mb_extract(self._h, mb, 0, 0, None, None, None, None, None, C.byref(nt), C.byref(nn)),
               "harts_mb_extract")
        ptr = np.empty(nt.value + 1, np.int32)
        par, off, ln, src = (np.empty(max(nn.value, 1), np.int32) for _ in range(4))
        ip = lambda a: a.ctypes.data_as(_I32P)  # noqa: E731
        _check(lib.harts_mb_extract(self._h, mb, nt.value, nn.value, ip(ptr), ip(par), ip(off), ip(ln), ip(src),
                                    C.byref(nt), C.byref(nn)), "harts_mb_extract")
        return ptr, par[:nn.value], off[:nn.value], ln[:nn.value], src[:nn.value]


def harts_mb_plan(tree_node_ptr, node_parent, node_fork_off, node_len, D, T) -> MbPlan:
    arrs = [np.ascontiguousarray(np.asarray(a), dtype=np.int32) for a in
            (tree_node_ptr, node_parent, node_fork_off, node_len)]
    h = _vp()
    _check(lib.harts_mb_plan(len(arrs[0]) - 1, *(a.ctypes.data_as(_I32P) for a in arrs), D, T, C.byref(h)),
           "harts_mb_plan")
    return MbPlan(h)
