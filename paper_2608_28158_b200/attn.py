"""ctypes binding of the harts_attn_* entry points (same names as the C ABI).  Argument marshalling only."""
from __future__ import annotations

import ctypes as C

import numpy as np
import torch

from .binding import lib, _check, _ptr, _stream, _DTYPE_CODE, _I32P

_vp, _i32, _i64, _f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
lib.harts_attn_index.argtypes = [_i32] + [_I32P] * 5 + [_i64, _I32P, C.POINTER(_i64)]
lib.harts_attn_fwd.argtypes = [_I32P, _vp, _vp, _vp, _vp, _vp, _vp, _i32, _i32, _i32, _f32, _i32, _vp, _vp]
lib.harts_attn_bwd.argtypes = [_I32P, _vp] + [_vp] * 10 + [_i32, _i32, _i32, _f32, _i32, _vp, _vp]
for _n in ("harts_attn_index", "harts_attn_fwd", "harts_attn_bwd"):
    getattr(lib, _n).restype = _i32

HEADER_WORDS = 24
_ARRAYS = ("piece_row0", "piece_len", "piece_parent", "anc_ptr", "anc_row0", "anc_len", "desc_ptr", "desc_piece",
           "q_item", "kv_item")


class AttnIndex:
    """The index blob on the host (numpy int32) and, after ``upload``, on the device."""

    def __init__(self, blob):
        self.host = blob
        self.n_rows, self.n_pieces, self.n_anc_runs, self.n_desc, self.n_q_items, self.n_kv_items = map(int, blob[:6])
        sizes = (self.n_pieces, self.n_pieces, self.n_pieces, self.n_pieces + 1, self.n_anc_runs, self.n_anc_runs,
                 self.n_pieces + 1, self.n_desc, 2 * self.n_q_items, 2 * self.n_kv_items)
        for name, off, n in zip(_ARRAYS, blob[8:18], sizes):
            setattr(self, name, blob[off:off + n])
        self.dev = None

    def upload(self, device="cuda"):
        self.dev = torch.as_tensor(self.host).to(device)
        return self


def harts_attn_index(tree_node_ptr, node_parent, node_fork_off, node_len, row_of_token=None) -> AttnIndex:
    arrs = [np.ascontiguousarray(np.asarray(a), dtype=np.int32) for a in
            (tree_node_ptr, node_parent, node_fork_off, node_len)]
    rot = None if row_of_token is None else np.ascontiguousarray(np.asarray(row_of_token), dtype=np.int32)
    ip = lambda a: None if a is None else a.ctypes.data_as(_I32P)  # noqa: E731
    n = _i64(0)
    _check(lib.harts_attn_index(len(arrs[0]) - 1, *map(ip, arrs), ip(rot), 0, None, C.byref(n)), "harts_attn_index")
    blob = np.zeros(n.value, np.int32)
    _check(lib.harts_attn_index(len(arrs[0]) - 1, *map(ip, arrs), ip(rot), n.value, ip(blob), C.byref(n)),
           "harts_attn_index")
    return AttnIndex(blob)


def harts_attn_fwd(index: AttnIndex, q, k, v, o, lse, scale, dev_status=None, stream=None):
    _check(lib.harts_attn_fwd(index.host.ctypes.data_as(_I32P), _ptr(index.dev), _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                              _ptr(lse), q.shape[1], k.shape[1], q.shape[2], scale, _DTYPE_CODE[q.dtype],
                              _ptr(dev_status), _stream(stream)), "harts_attn_fwd")


def harts_attn_bwd(index: AttnIndex, q, k, v, o, lse, dO, dq, dk_, dv_, delta, scale, dev_status=None, stream=None):
    _check(lib.harts_attn_bwd(index.host.ctypes.data_as(_I32P), _ptr(index.dev), _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                              _ptr(lse), _ptr(dO), _ptr(dq), _ptr(dk_), _ptr(dv_), _ptr(delta), q.shape[1], k.shape[1],
                              q.shape[2], scale, _DTYPE_CODE[q.dtype], _ptr(dev_status), _stream(stream)),
           "harts_attn_bwd")
