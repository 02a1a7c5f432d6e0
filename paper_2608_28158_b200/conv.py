"""ctypes binding of the harts_conv_* entry points (same names as the C ABI).  Argument marshalling only."""
from __future__ import annotations

import ctypes as C

import numpy as np

from .binding import lib, _check, _ptr, _stream, _DTYPE_CODE, _I32P

_vp, _i32 = C.c_void_p, C.c_int32
lib.harts_conv_index.argtypes = [_i32] + [_I32P] * 9
lib.harts_conv_fwd.argtypes = [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _vp]
lib.harts_conv_scratch_bytes.argtypes = [_i32, _i32, C.POINTER(C.c_size_t)]
lib.harts_conv_bwd.argtypes = [_vp] * 9 + [_i32] * 4 + [_vp]
for _n in ("harts_conv_index", "harts_conv_fwd", "harts_conv_scratch_bytes", "harts_conv_bwd"):
    getattr(lib, _n).restype = _i32


def _i32arr(a):
    return np.ascontiguousarray(np.asarray(a), dtype=np.int32)


def harts_conv_index(tree_node_ptr, node_parent, node_fork_off, node_len, row_of_token=None):
    """(prev_row [C], next_row [C], child_ptr [C+1], child_row [C - n_trees]) int32 on the host."""
    ptr, par, off, ln = map(_i32arr, (tree_node_ptr, node_parent, node_fork_off, node_len))
    rot = None if row_of_token is None else _i32arr(row_of_token)
    n = int(ln.sum())
    prev = np.empty(max(n, 1), np.int32)
    nxt = np.empty(max(n, 1), np.int32)
    cptr = np.empty(n + 1, np.int32)
    crow = np.empty(max(n - (len(ptr) - 1), 1), np.int32)
    ip = lambda a: None if a is None else a.ctypes.data_as(_I32P)  # noqa: E731
    _check(lib.harts_conv_index(len(ptr) - 1, ip(ptr), ip(par), ip(off), ip(ln), ip(rot), ip(prev), ip(nxt), ip(cptr),
                                ip(crow)), "harts_conv_index")
    return prev[:n], nxt[:n], cptr, crow[:max(n - (len(ptr) - 1), 0)]


def harts_conv_fwd(x, W, prev_row, y, stream=None):
    n, D = x.shape
    _check(lib.harts_conv_fwd(_ptr(x), _ptr(W), _ptr(prev_row), _ptr(y), n, D, W.shape[1], _DTYPE_CODE[x.dtype],
                              _stream(stream)), "harts_conv_fwd")


def harts_conv_scratch_bytes(D, w):
    n = C.c_size_t(0)
    _check(lib.harts_conv_scratch_bytes(D, w, C.byref(n)), "harts_conv_scratch_bytes")
    return int(n.value)


def harts_conv_bwd(x, W, dy, next_row, child_ptr, child_row, dx, dW, scratch, stream=None):
    n, D = x.shape
    _check(lib.harts_conv_bwd(_ptr(x), _ptr(W), _ptr(dy), _ptr(next_row), _ptr(child_ptr), _ptr(child_row), _ptr(dx),
                              _ptr(dW), _ptr(scratch), n, D, W.shape[1], _DTYPE_CODE[x.dtype], _stream(stream)),
           "harts_conv_bwd")
