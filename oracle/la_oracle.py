"""Python face of the fp64 oracle (test infrastructure only; see oracle/__init__.py).

* ``trajectories``    -- the semantic map m of Eq. 3: every root-to-leaf trajectory as the
                         list of compact (canonical) token indices it visits.
* ``forest_eval``     -- runs la_oracle.c (token recurrence per trajectory, Section 2.2 /
                         Eq. 1 specialised to a scalar gate) over a forest.
* ``compact_dfs_fwd`` -- a second, independent formulation used only as a pin: one
                         depth-first walk of the tree that carries the state across forks
                         (what prefix sharing means, Section 2.1), no trajectories expanded.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force: bool = False) -> str:
    src = os.path.join(_HERE, "la_oracle.c")
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(src):
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _SO, src, "-lm"])
    return _SO


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        dp = ctypes.POINTER(ctypes.c_double)
        lp = ctypes.POINTER(ctypes.c_longlong)
        _lib.harts_oracle_traj_fwd.argtypes = [ctypes.c_int] * 3 + [dp] * 5
        _lib.harts_oracle_traj_fwd.restype = None
        _lib.harts_oracle_traj_bwd.argtypes = [ctypes.c_int] * 3 + [dp] * 10
        _lib.harts_oracle_traj_bwd.restype = None
        _lib.harts_oracle_forest.argtypes = ([ctypes.c_int, lp, lp, ctypes.c_longlong] + [ctypes.c_int] * 3
                                             + [dp] * 11)
        _lib.harts_oracle_forest.restype = ctypes.c_int
    return _lib


def _f64(x):
    if x is None:
        return None
    if hasattr(x, "detach"):                      # torch tensor (any dtype, bf16 included)
        x = x.detach().cpu().double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _ptr(a, ct=ctypes.c_double):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def traj_fwd(q, k, v, g):
    """One trajectory, one head: q,k [T,dk], v [T,dv], g [T] -> o [T,dv]."""
    q, k, v, g = map(_f64, (q, k, v, g))
    T, dk = q.shape
    dv = v.shape[1]
    o = np.zeros((T, dv))
    _load().harts_oracle_traj_fwd(T, dk, dv, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(o))
    return o


def traj_bwd(q, k, v, g, dO):
    q, k, v, g, dO = map(_f64, (q, k, v, g, dO))
    T, dk = q.shape
    dv = v.shape[1]
    dq, dk_, dv_, dg = np.zeros((T, dk)), np.zeros((T, dk)), np.zeros((T, dv)), np.zeros(T)
    _load().harts_oracle_traj_bwd(T, dk, dv, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(dO),
                                  _ptr(dq), _ptr(dk_), _ptr(dv_), _ptr(dg), None)
    return dq, dk_, dv_, dg


def trajectories(forest):
    """(traj_ptr int64 [n_traj+1], traj_rows int64 [S]): canonical token index of every semantic
    position, trajectory by trajectory.  A node's end is a trajectory end unless a child forks
    exactly there."""
    base = forest.token_base()
    ptr, rows = [0], []
    for t in range(forest.n_trees):
        lo = int(forest.tree_node_ptr[t])
        par, off, ln = (a.tolist() for a in forest.tree(t))
        n = len(par)
        continued = [False] * n
        for i in range(1, n):
            if off[i] == ln[par[i]]:
                continued[par[i]] = True
        for leaf in range(n):
            if continued[leaf]:
                continue
            pieces = []
            node, upto = leaf, ln[leaf]
            while node >= 0:                      # walk up: the parent contributes its first fork_off tokens
                pieces.append(np.arange(base[lo + node], base[lo + node] + upto, dtype=np.int64))
                node, upto = par[node], off[node]
            pieces.reverse()
            rows.extend(pieces)
            ptr.append(ptr[-1] + sum(len(p) for p in pieces))
    traj_rows = np.concatenate(rows) if rows else np.zeros(0, dtype=np.int64)
    return np.asarray(ptr, dtype=np.int64), traj_rows


def forest_eval(forest, q, k, v, g, dO=None):
    """Trajectory-wise fp64 evaluation of a whole forest on compact tensors in canonical order.

    q,k [C,H,dk], v,dO [C,H,dv], g [C,H] (numpy or torch, any float dtype).  Returns a dict with
    o and, when dO is given, dq, dk, dv, dg (all fp64 numpy), the largest disagreement between
    copies of one compact row (``copy_gap``), the trajectory-wise token count and the thread count.
    """
    q, k, v, g, dO = map(_f64, (q, k, v, g, dO))
    C, H, dk = q.shape
    dv = v.shape[2]
    assert C == forest.n_tokens
    traj_ptr, traj_rows = trajectories(forest)
    o = np.zeros((C, H, dv))
    grads = [None] * 4
    if dO is not None:
        grads = [np.zeros((C, H, dk)), np.zeros((C, H, dk)), np.zeros((C, H, dv)), np.zeros((C, H))]
    gap = ctypes.c_double(0.0)
    nthreads = _load().harts_oracle_forest(
        len(traj_ptr) - 1, _ptr(traj_ptr, ctypes.c_longlong), _ptr(traj_rows, ctypes.c_longlong), C, H, dk, dv,
        _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(dO), _ptr(o), *(_ptr(a) for a in grads), ctypes.byref(gap))
    out = {"o": o, "copy_gap": gap.value, "threads": nthreads, "S": int(traj_ptr[-1]),
           "traj_ptr": traj_ptr, "traj_rows": traj_rows}
    if dO is not None:
        out.update(dq=grads[0], dk=grads[1], dv=grads[2], dg=grads[3])
    return out


def compact_dfs_fwd(forest, q, k, v, g):
    """Forward outputs from one walk of the tree, state carried across forks (numpy loops; small
    inputs only).  Independent of ``trajectories`` and of la_oracle.c."""
    q, k, v, g = map(_f64, (q, k, v, g))
    C, H, dk = q.shape
    dv = v.shape[2]
    base = forest.token_base()
    o = np.zeros((C, H, dv))
    for t in range(forest.n_trees):
        lo = int(forest.tree_node_ptr[t])
        par, off, ln = (a.tolist() for a in forest.tree(t))
        n = len(par)
        kids = [[] for _ in range(n)]
        for i in range(1, n):
            kids[par[i]].append(i)
        entry = {0: np.zeros((H, dk, dv))}
        for node in range(n):                      # parents precede children
            S = entry.pop(node).copy()
            want = {}
            for c in kids[node]:
                want.setdefault(off[c], []).append(c)
            for i in range(ln[node]):
                r = base[lo + node] + i
                S = np.exp(g[r])[:, None, None] * S + k[r][:, :, None] * v[r][:, None, :]
                o[r] = np.einsum("hi,hij->hj", q[r], S)
                for c in want.get(i + 1, []):
                    entry[c] = S.copy()
    return o
