"""Python face of the per-channel-decay oracle (gk_oracle.c).  TEST INFRASTRUCTURE ONLY.

``forest_eval`` evaluates every root-to-leaf trajectory of a forest on its own (token recurrence with the diagonal
decay of Eq. 1, Section 2.2) and brings the results to compact rows through the semantic map m of Eq. 3: outputs of
all copies of a compact row must agree, gradients of L = sum_c <dO_c, o_c> are accumulated over the copies, each copy
carrying dO_c / multiplicity (Eq. 20)."""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

from .la_oracle import trajectories

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libgkoracle.so")
_lib = None


def build(force: bool = False) -> str:
    src = os.path.join(_HERE, "gk_oracle.c")
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", _SO, src, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        _lib.harts_gk_oracle_traj_fwd.argtypes = [ctypes.c_int] * 3 + [dp] * 5
        _lib.harts_gk_oracle_traj_fwd.restype = None
        _lib.harts_gk_oracle_traj_bwd.argtypes = [ctypes.c_int] * 3 + [dp] * 9
        _lib.harts_gk_oracle_traj_bwd.restype = None
    return _lib


def _f64(x):
    if x is None:
        return None
    if hasattr(x, "detach"):
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def traj_fwd(q, k, v, g):
    """One trajectory, one head: q,k,g [T,dk], v [T,dv] -> o [T,dv]."""
    q, k, v, g = map(_f64, (q, k, v, g))
    T, dk = q.shape
    o = np.zeros((T, v.shape[1]))
    _load().harts_gk_oracle_traj_fwd(T, dk, v.shape[1], _p(q), _p(k), _p(v), _p(g), _p(o))
    return o


def traj_bwd(q, k, v, g, dO):
    q, k, v, g, dO = map(_f64, (q, k, v, g, dO))
    T, dk = q.shape
    dv = v.shape[1]
    dq, dk_, dv_, dg = np.zeros((T, dk)), np.zeros((T, dk)), np.zeros((T, dv)), np.zeros((T, dk))
    _load().harts_gk_oracle_traj_bwd(T, dk, dv, _p(q), _p(k), _p(v), _p(g), _p(dO), _p(dq), _p(dk_), _p(dv_), _p(dg))
    return dq, dk_, dv_, dg


def forest_eval(forest, q, k, v, g, dO=None):
    """q,k,g [C,H,dk], v,dO [C,H,dv] on compact tokens in canonical order -> dict(o, copy_gap[, dq, dk, dv, dg])."""
    q, k, v, g, dO = map(_f64, (q, k, v, g, dO))
    C, H, dk = q.shape
    dv = v.shape[2]
    assert C == forest.n_tokens and g.shape == q.shape
    ptr, rows = trajectories(forest)
    mult = np.bincount(rows, minlength=C).astype(np.float64)
    o = np.full((C, H, dv), np.nan)
    grads = None if dO is None else [np.zeros((C, H, dk)), np.zeros((C, H, dk)), np.zeros((C, H, dv)), np.zeros((C, H, dk))]
    jobs = [(x, h) for x in range(len(ptr) - 1) for h in range(H)]

    def run(job):
        x, h = job
        r = rows[ptr[x]:ptr[x + 1]]
        tq, tk, tv, tg = (np.ascontiguousarray(a[r, h]) for a in (q, k, v, g))
        out = traj_fwd(tq, tk, tv, tg)
        grad = None
        if dO is not None:
            grad = traj_bwd(tq, tk, tv, tg, np.ascontiguousarray(dO[r, h] / mult[r, None]))
        return x, h, r, out, grad

    gap = 0.0
    with ThreadPoolExecutor(max_workers=os.cpu_count() or 4) as pool:
        for x, h, r, out, grad in pool.map(run, jobs):          # results are merged here, one at a time
            seen = ~np.isnan(o[r, h, 0])
            if seen.any():
                gap = max(gap, float(np.abs(o[r[seen], h] - out[seen]).max()))
            o[r[~seen], h] = out[~seen]
            if grad is not None:
                for acc, part in zip(grads, grad):
                    np.add.at(acc[:, h], r, part)
    res = {"o": o, "copy_gap": gap, "S": int(ptr[-1])}
    if grads is not None:
        res.update(dq=grads[0], dk=grads[1], dv=grads[2], dg=grads[3])
    return res
