"""ctypes binding of the harts_logp_* entry points (same names as the C ABI).  Argument marshalling only."""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from .binding import lib, _check, _ptr, _stream, _DTYPE_CODE, _I32P

_I64P = C.POINTER(C.c_int64)
_vp, _i32, _i64 = C.c_void_p, C.c_int32, C.c_int64

lib.harts_logp_positions.argtypes = [_i32, _I32P, _I32P, _I32P, _I32P, _I32P, _I32P, _i64, _I32P, _I32P, _I64P, _I64P,
                                     _I64P]
lib.harts_logp_csr.argtypes = [_i32, _i64, _I32P, _I32P, _I32P]
lib.harts_logp_multiplicity.argtypes = [_i32, _I32P, _I32P, _I32P, _I32P, _I32P, _i64, _I32P]
lib.harts_logp_fwd.argtypes = [_vp, _i32, _i32, _i32, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp]
lib.harts_logp_bwd.argtypes = [_vp, _i32, _i32, _i32, _i64, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _i64, _i32, _i32, _vp,
                               _vp]
lib.harts_logp_fwd_shard.argtypes = [_vp, _i32, _i32, _i32, _i64, _i32, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.harts_logp_combine.argtypes = [_i32, _i32, _i64, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
for _n in ("harts_logp_positions", "harts_logp_csr", "harts_logp_multiplicity", "harts_logp_fwd", "harts_logp_bwd", "harts_logp_fwd_shard",
           "harts_logp_combine"):
    getattr(lib, _n).restype = _i32


def _i32arr(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def _ip(a):
    return None if a is None else a.ctypes.data_as(_I32P)


def harts_logp_positions(tree_node_ptr, node_parent, node_fork_off, node_len, token_id, row_of_token=None):
    """(m int32 [P], y int32 [P], traj_pos_ptr int64 [n_traj+1]) on the host."""
    ptr, par, off, ln = map(_i32arr, (tree_node_ptr, node_parent, node_fork_off, node_len))
    tok = _i32arr(token_id)
    rot = None if row_of_token is None else _i32arr(row_of_token)
    n_pos, n_traj = C.c_int64(0), C.c_int64(0)
    _check(lib.harts_logp_positions(len(ptr) - 1, _ip(ptr), _ip(par), _ip(off), _ip(ln), _ip(rot), _ip(tok), 0, None,
                                    None, None, C.byref(n_pos), C.byref(n_traj)), "harts_logp_positions")
    m = np.empty(max(n_pos.value, 1), np.int32)
    y = np.empty(max(n_pos.value, 1), np.int32)
    tp = np.empty(n_traj.value + 1, np.int64)
    _check(lib.harts_logp_positions(len(ptr) - 1, _ip(ptr), _ip(par), _ip(off), _ip(ln), _ip(rot), _ip(tok),
                                    n_pos.value, _ip(m), _ip(y), tp.ctypes.data_as(_I64P), C.byref(n_pos),
                                    C.byref(n_traj)), "harts_logp_positions")
    return m[:n_pos.value], y[:n_pos.value], tp


def harts_logp_multiplicity(tree_node_ptr, node_parent, node_fork_off, node_len, row_of_token=None, n_rows=None):
    """int32 [n_rows] on the host: the number of trajectories that contain each compact token (Eq. 20)."""
    ptr, par, off, ln = map(_i32arr, (tree_node_ptr, node_parent, node_fork_off, node_len))
    rot = None if row_of_token is None else _i32arr(row_of_token)
    n_rows = int(ln.sum()) if n_rows is None else int(n_rows)
    mult = np.empty(max(n_rows, 1), np.int32)
    _check(lib.harts_logp_multiplicity(len(ptr) - 1, _ip(ptr), _ip(par), _ip(off), _ip(ln), _ip(rot), n_rows, _ip(mult)),
           "harts_logp_multiplicity")
    return mult[:n_rows]


def harts_logp_csr(n_rows, m):
    """(row_pos_ptr int32 [n_rows+1], row_pos int32 [P]) on the host."""
    m = _i32arr(m)
    ptr = np.empty(n_rows + 1, np.int32)
    pos = np.empty(max(len(m), 1), np.int32)
    _check(lib.harts_logp_csr(n_rows, len(m), _ip(m), _ip(ptr), _ip(pos)), "harts_logp_csr")
    return ptr, pos[:len(m)]


def harts_logp_fwd(z, m, y, lse, lam, V=None, dev_status=None, stream=None):
    n_rows = z.shape[0]
    V = z.shape[1] if V is None else V
    _check(lib.harts_logp_fwd(_ptr(z), _DTYPE_CODE[z.dtype], n_rows, V, z.stride(0) if n_rows else V, m.numel(),
                              _ptr(m), _ptr(y), _ptr(lse), _ptr(lam), _ptr(dev_status), _stream(stream)),
           "harts_logp_fwd")


def harts_logp_bwd(z, y, row_pos_ptr, row_pos, lse, g, dz, V=None, v_begin=0, V_total=None, dev_status=None,
                   stream=None):
    n_rows = z.shape[0]
    V = z.shape[1] if V is None else V
    V_total = V if V_total is None else V_total
    _check(lib.harts_logp_bwd(_ptr(z), _DTYPE_CODE[z.dtype], n_rows, V, z.stride(0) if n_rows else V, y.numel(),
                              _ptr(y), _ptr(row_pos_ptr), _ptr(row_pos), _ptr(lse), _ptr(g), _ptr(dz),
                              dz.stride(0) if n_rows else V, v_begin, V_total, _ptr(dev_status), _stream(stream)),
           "harts_logp_bwd")


def harts_logp_fwd_shard(z, v_begin, m, y, row_max, row_sum, target, V=None, dev_status=None, stream=None):
    n_rows = z.shape[0]
    V = z.shape[1] if V is None else V
    _check(lib.harts_logp_fwd_shard(_ptr(z), _DTYPE_CODE[z.dtype], n_rows, V, z.stride(0) if n_rows else V, v_begin,
                                    m.numel(), _ptr(m), _ptr(y), _ptr(row_max), _ptr(row_sum), _ptr(target),
                                    _ptr(dev_status), _stream(stream)), "harts_logp_fwd_shard")


def harts_logp_combine(n_shards, n_rows, m, row_max, row_sum, target, lse, lam, stream=None):
    _check(lib.harts_logp_combine(n_shards, n_rows, m.numel(), _ptr(m), _ptr(row_max), _ptr(row_sum), _ptr(target),
                                  _ptr(lse), _ptr(lam), _stream(stream)), "harts_logp_combine")
