"""ctypes binding with the C ABI's names.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import build as _build

HARTS_OK = 0
HARTS_FP32, HARTS_BF16 = 0, 1
HARTS_FLAG_FMA_KERNELS = 1
HARTS_FLAG_CHECK_TABLES = 2
HARTS_FLAG_ROUND_LAUNCHES = 16
_DTYPE_CODE = {torch.float32: HARTS_FP32, torch.bfloat16: HARTS_BF16}

_I32P = C.POINTER(C.c_int32)


class HartsError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {harts_la_strerror(code)} ({code})")
        self.code = code


class _View(C.Structure):
    _counts = ("chunk", "n_rounds", "n_rows", "n_replay", "n_seq", "n_slots", "n_chunks", "n_rg_rows")
    _arrays = ("row_of_token", "round_seq_ptr", "seq_tree", "seq_own_begin", "seq_own_len", "seq_start_pos",
               "seq_init_slot", "seq_replay_ptr", "replay_row", "seq_req_ptr", "slot_chunk", "seq_chunk_ptr",
               "slot_cons_ptr", "slot_cons_seq", "rg_row", "rg_ptr", "rg_entry", "seq_order")
    _fields_ = [(n, C.c_int32) for n in _counts] + [(n, _I32P) for n in _arrays]


class Tables(C.Structure):
    _counts = ("chunk", "n_rows", "n_replay", "n_seq", "n_slots", "n_chunks", "n_rg_rows")
    _arrays = ("seq_own_begin", "seq_init_slot", "seq_replay_ptr", "replay_row", "seq_req_ptr", "slot_chunk",
               "seq_chunk_ptr", "slot_cons_ptr", "slot_cons_seq", "rg_row", "rg_ptr", "rg_entry", "seq_order")
    _fields_ = [(n, C.c_int32) for n in _counts] + [(n, C.c_void_p) for n in _arrays]


def _load():
    path = _build.build()      # recompiles only what is older than its sources
    lib = C.CDLL(path)
    vp, i32, u32, sz = C.c_void_p, C.c_int32, C.c_uint32, C.c_size_t
    lib.harts_la_strerror.argtypes = [i32]
    lib.harts_la_strerror.restype = C.c_char_p
    lib.harts_la_plan.argtypes = [i32, _I32P, _I32P, _I32P, _I32P, i32, C.POINTER(vp)]
    lib.harts_la_plan_free.argtypes = [vp]
    lib.harts_la_plan_free.restype = None
    lib.harts_la_plan_view.argtypes = [vp, C.POINTER(_View)]
    lib.harts_la_plan_device_bytes.argtypes = [vp, C.POINTER(sz)]
    lib.harts_la_plan_upload.argtypes = [vp, vp, vp]
    lib.harts_la_plan_tables.argtypes = [vp, vp, C.POINTER(Tables)]
    lib.harts_la_workspace_bytes.argtypes = [C.POINTER(Tables), i32, i32, i32, i32, u32, C.POINTER(sz), C.POINTER(sz)]
    lib.harts_la_fwd_seqs.argtypes = [C.POINTER(Tables), i32, i32] + [vp] * 7 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_bwd_seqs.argtypes = [C.POINTER(Tables), i32, i32] + [vp] * 11 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_bwd_finish.argtypes = [C.POINTER(Tables)] + [vp] * 4 + [i32] * 4 + [vp]
    lib.harts_la_fwd.argtypes = [vp, vp, i32] + [vp] * 7 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_bwd.argtypes = [vp, vp, i32] + [vp] * 11 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_check.argtypes = [vp, vp]
    lib.harts_la_bwd_static.argtypes = [vp, vp] + [vp] * 10 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_bwd_static.restype = i32
    lib.harts_la_selftest_timeout.argtypes = [vp, vp, vp]
    lib.harts_la_selftest_timeout.restype = i32
    lib.harts_la_expand.argtypes = [i32, _I32P, _I32P, _I32P, _I32P, C.c_int64, C.c_int64, _I32P, C.POINTER(C.c_int64),
                                    C.POINTER(C.c_int64), C.POINTER(C.c_int64)]
    lib.harts_la_expand.restype = i32
    lib.harts_la_step_host.argtypes = [vp, vp] + [vp] * 23 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_step_host.restype = i32
    lib.harts_la_gk_workspace_bytes.argtypes = [C.POINTER(Tables), i32, i32, i32, i32, C.POINTER(sz), C.POINTER(sz)]
    lib.harts_la_gk_fwd.argtypes = [vp, vp, i32] + [vp] * 7 + [i32] * 4 + [u32, vp, vp]
    lib.harts_la_gk_bwd.argtypes = [vp, vp, i32] + [vp] * 11 + [i32] * 4 + [u32, vp, vp]
    for name in ("harts_la_gk_workspace_bytes", "harts_la_gk_fwd", "harts_la_gk_bwd"):
        getattr(lib, name).restype = i32
    for name in ("harts_la_plan", "harts_la_plan_view", "harts_la_plan_device_bytes", "harts_la_plan_upload",
                 "harts_la_plan_tables", "harts_la_workspace_bytes", "harts_la_fwd_seqs", "harts_la_bwd_seqs",
                 "harts_la_bwd_finish", "harts_la_fwd", "harts_la_bwd", "harts_la_check"):
        getattr(lib, name).restype = i32
    return lib


lib = _load()


def harts_la_strerror(code: int) -> str:
    return lib.harts_la_strerror(code).decode()


def _check(code, where):
    if code != HARTS_OK:
        raise HartsError(code, where)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class _PlanHandle:
    """Owns the library's plan object; freed when the last user (the Plan or one of its array views) is gone."""

    def __init__(self, handle):
        self.h = handle

    def __del__(self):
        h, self.h = getattr(self, "h", None), None
        if h:
            lib.harts_la_plan_free(h)


class _PlanArray(np.ndarray):
    """Read-only view of a plan table in the library's memory; keeps the plan alive."""
    _owner = None

    def __array_finalize__(self, obj):
        self._owner = getattr(obj, "_owner", None)


class Plan:
    """Host plan (owned by the library) plus, after ``upload``, its device index blob.  The index arrays are
    read-only views of the library's memory (no copies); each keeps the plan alive."""

    def __init__(self, handle):
        self._handle = _PlanHandle(handle)
        self._h = handle
        v = _View()
        _check(lib.harts_la_plan_view(handle, C.byref(v)), "harts_la_plan_view")
        for n in _View._counts:
            setattr(self, n, int(getattr(v, n)))
        sizes = dict(row_of_token=self.n_rows, round_seq_ptr=self.n_rounds + 1, seq_tree=self.n_seq,
                     seq_own_begin=self.n_seq + 1, seq_own_len=self.n_seq, seq_start_pos=self.n_seq,
                     seq_init_slot=self.n_seq, seq_replay_ptr=self.n_seq + 1, replay_row=self.n_replay,
                     seq_req_ptr=self.n_seq + 1, slot_chunk=self.n_slots, seq_chunk_ptr=self.n_seq + 1,
                     slot_cons_ptr=self.n_slots + 1, slot_cons_seq=None, rg_row=self.n_rg_rows,
                     rg_ptr=self.n_rg_rows + 1 if self.n_rg_rows else 1, rg_entry=self.n_replay,
                     seq_order=self.n_seq)
        for n in _View._arrays:
            size = sizes[n]
            if n == "slot_cons_seq":
                size = int(self.slot_cons_ptr[-1])
            if size:
                arr = np.ctypeslib.as_array(getattr(v, n), shape=(size,)).view(_PlanArray)
                arr._owner = self._handle
                arr.flags.writeable = False
            else:
                arr = np.zeros(0, np.int32)
            setattr(self, n, arr)
        self.C, self.R = self.n_rows, self.n_replay
        self.blob = None
        self.tables = None

    def upload(self, device="cuda", stream=None):
        n = C.c_size_t(0)
        _check(lib.harts_la_plan_device_bytes(self._h, C.byref(n)), "harts_la_plan_device_bytes")
        self.blob = torch.empty(max(int(n.value), 16), dtype=torch.uint8, device=device)
        _check(lib.harts_la_plan_upload(self._h, _ptr(self.blob), _stream(stream)), "harts_la_plan_upload")
        self.tables = Tables()
        _check(lib.harts_la_plan_tables(self._h, _ptr(self.blob), C.byref(self.tables)), "harts_la_plan_tables")
        return self


def harts_la_plan(tree_node_ptr, node_parent, node_fork_off, node_len, chunk=64) -> Plan:
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in (tree_node_ptr, node_parent, node_fork_off, node_len)]
    handle = C.c_void_p()
    code = lib.harts_la_plan(len(arrs[0]) - 1, *(a.ctypes.data_as(_I32P) for a in arrs), int(chunk), C.byref(handle))
    _check(code, "harts_la_plan")
    return Plan(handle)


def harts_la_workspace_bytes(tables, H, dk, dv, dtype, flags=0):
    a, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib.harts_la_workspace_bytes(C.byref(tables), H, dk, dv, dtype, flags, C.byref(a), C.byref(b)),
           "harts_la_workspace_bytes")
    return int(a.value), int(b.value)


def _dims(q, v):
    return q.shape[1], q.shape[2], v.shape[2], _DTYPE_CODE[q.dtype]


def harts_la_fwd_seqs(tables, seq_lo, seq_hi, q, k, v, g, o, slots, chunk_states, flags=0, dev_status=None,
                      stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_fwd_seqs(C.byref(tables), seq_lo, seq_hi, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(o),
                                 _ptr(slots), _ptr(chunk_states), H, dk, dv, dt, flags, _ptr(dev_status),
                                 _stream(stream)), "harts_la_fwd_seqs")


def harts_la_bwd_seqs(tables, seq_lo, seq_hi, q, k, v, g, dO, dq, dk_, dv_, dg, chunk_states, scratch, flags=0,
                      dev_status=None, stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_bwd_seqs(C.byref(tables), seq_lo, seq_hi, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(dO),
                                 _ptr(dq), _ptr(dk_), _ptr(dv_), _ptr(dg), _ptr(chunk_states), _ptr(scratch), H, dk,
                                 dv, dt, flags, _ptr(dev_status), _stream(stream)), "harts_la_bwd_seqs")


def harts_la_bwd_finish(tables, dk_, dv_, dg, scratch, stream=None):
    H, dk, dv = dk_.shape[1], dk_.shape[2], dv_.shape[2]
    _check(lib.harts_la_bwd_finish(C.byref(tables), _ptr(dk_), _ptr(dv_), _ptr(dg), _ptr(scratch), H, dk, dv,
                                   _DTYPE_CODE[dk_.dtype], _stream(stream)), "harts_la_bwd_finish")


def harts_la_fwd(plan, round, q, k, v, g, o, slots, chunk_states, flags=0, dev_status=None, stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_fwd(plan._h, _ptr(plan.blob), round, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(o),
                            _ptr(slots), _ptr(chunk_states), H, dk, dv, dt, flags, _ptr(dev_status),
                            _stream(stream)), "harts_la_fwd")


def harts_la_bwd(plan, round, q, k, v, g, dO, dq, dk_, dv_, dg, chunk_states, scratch, flags=0, dev_status=None,
                 stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_bwd(plan._h, _ptr(plan.blob), round, _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(dO), _ptr(dq),
                            _ptr(dk_), _ptr(dv_), _ptr(dg), _ptr(chunk_states), _ptr(scratch), H, dk, dv, dt, flags,
                            _ptr(dev_status), _stream(stream)), "harts_la_bwd")


def harts_la_bwd_static(plan, q, k, v, g, dO, dq, dk_, dv_, dg, chunk_states, flags=0, dev_status=None, stream=None):
    """All backward rounds and the replay fold with the scratch area inside the library (a fixed device array):
    for callers that cannot provide or allocate a scratch buffer.  Raises HartsError(-7) when the problem needs
    more scratch than that array holds.  Calls that overlap on the GPU race on the shared array."""
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_bwd_static(plan._h, _ptr(plan.blob), _ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(dO), _ptr(dq),
                                   _ptr(dk_), _ptr(dv_), _ptr(dg), _ptr(chunk_states), H, dk, dv, dt, flags,
                                   _ptr(dev_status), _stream(stream)), "harts_la_bwd_static")


def harts_la_gk_workspace_bytes(tables, H, dk, dv, dtype):
    a, b = C.c_size_t(0), C.c_size_t(0)
    _check(lib.harts_la_gk_workspace_bytes(C.byref(tables), H, dk, dv, dtype, C.byref(a), C.byref(b)),
           "harts_la_gk_workspace_bytes")
    return int(a.value), int(b.value)


def harts_la_gk_fwd(plan, round, q, k, v, gk, o, slots, chunk_states, flags=0, dev_status=None, stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_gk_fwd(plan._h, _ptr(plan.blob), round, _ptr(q), _ptr(k), _ptr(v), _ptr(gk), _ptr(o),
                               _ptr(slots), _ptr(chunk_states), H, dk, dv, dt, flags, _ptr(dev_status),
                               _stream(stream)), "harts_la_gk_fwd")


def harts_la_gk_bwd(plan, round, q, k, v, gk, dO, dq, dk_, dv_, dgk, chunk_states, scratch, flags=0, dev_status=None,
                    stream=None):
    H, dk, dv, dt = _dims(q, v)
    _check(lib.harts_la_gk_bwd(plan._h, _ptr(plan.blob), round, _ptr(q), _ptr(k), _ptr(v), _ptr(gk), _ptr(dO),
                               _ptr(dq), _ptr(dk_), _ptr(dv_), _ptr(dgk), _ptr(chunk_states), _ptr(scratch), H, dk, dv,
                               dt, flags, _ptr(dev_status), _stream(stream)), "harts_la_gk_bwd")


def harts_la_selftest_timeout(dev_status, dev_report=None, stream=None):
    _check(lib.harts_la_selftest_timeout(_ptr(dev_status), _ptr(dev_report), _stream(stream)), "harts_la_selftest_timeout")


def harts_la_check(dev_status, stream=None):
    _check(lib.harts_la_check(_ptr(dev_status), _stream(stream)), "harts_la_check")


class Workspace:
    """Caller-owned device buffers for one plan: slots, chunk states, backward scratch, status word."""

    def __init__(self, plan: Plan, H, dk, dv, dtype, flags=0, device="cuda"):
        if plan.tables is None:
            plan.upload(device)
        cs_bytes, sc_bytes = harts_la_workspace_bytes(plan.tables, H, dk, dv, _DTYPE_CODE[dtype], flags)
        self.slots = torch.empty(max(plan.n_slots, 1) * H * dk * dv, dtype=torch.float32, device=device)
        self.chunk_states = torch.empty(cs_bytes, dtype=torch.uint8, device=device)
        self.scratch = torch.empty(sc_bytes, dtype=torch.uint8, device=device)
        self.dev_status = torch.zeros(4, dtype=torch.int32, device=device)
        self.flags = flags


def run_fwd_bwd(plan: Plan, ws: Workspace, q, k, v, g, dO, out=None, backward=True, stream=None):
    """All rounds forward (and backward) on device tensors in physical row order."""
    if out is None:
        out = {"o": torch.empty_like(v)}
        if backward:
            out.update(dq=torch.empty_like(q), dk=torch.empty_like(k), dv=torch.empty_like(v),
                       dg=torch.empty_like(g))
    harts_la_fwd(plan, 0, q, k, v, g, out["o"], ws.slots, ws.chunk_states, ws.flags, ws.dev_status, stream)
    if backward:
        harts_la_bwd(plan, 0, q, k, v, g, dO, out["dq"], out["dk"], out["dv"], out["dg"], ws.chunk_states,
                     ws.scratch, ws.flags, ws.dev_status, stream)
    return out


def harts_la_step_host(plan, ws, host_in: dict, dev_in: dict, dev_out: dict, host_out: dict, stream=None):
    """One step on HOST buffers through the library: inputs copied in, all rounds forward and backward, results copied
    out, everything enqueued on one stream (no synchronisation here)."""
    H, dk, dv, dt = _dims(dev_in["q"], dev_in["v"])
    args = [_ptr(host_in[n]) for n in ("q", "k", "v", "g", "dO")] + [_ptr(host_out[n]) for n in ("o", "dq", "dk", "dv", "dg")]
    args += [_ptr(dev_in[n]) for n in ("q", "k", "v", "g", "dO")] + [_ptr(dev_out[n]) for n in ("o", "dq", "dk", "dv", "dg")]
    _check(lib.harts_la_step_host(plan._h, _ptr(plan.blob), *args, _ptr(ws.slots), _ptr(ws.chunk_states),
                                  _ptr(ws.scratch), H, dk, dv, dt, ws.flags, _ptr(ws.dev_status), _stream(stream)),
           "harts_la_step_host")


def run_fwd_bwd_host(plan: Plan, ws: Workspace, host_in: dict, dev_in: dict, dev_out: dict, host_out: dict):
    """End-to-end step on HOST buffers (harts_la_step_host), then a synchronisation.  Buffers are preallocated by the
    caller."""
    harts_la_step_host(plan, ws, host_in, dev_in, dev_out, host_out)
    torch.cuda.current_stream().synchronize()
    return host_out


class HostPipeline:
    """End-to-end steps on HOST buffers with the copies of neighbouring steps overlapped: three streams (inputs
    in, kernels, results out) and two sets of device tensors, so that while step i computes, the inputs of step
    i+1 arrive and the results of step i-1 leave.  Every step still copies all of its inputs from the (pinned)
    host buffers and all of its results back; the kernels of successive steps share one workspace and run in order."""

    def __init__(self, plan: Plan, ws: Workspace, like_in: dict, like_out: dict):
        self.plan, self.ws = plan, ws
        self.sets = [({n: torch.empty_like(x) for n, x in like_in.items()},
                      {n: torch.empty_like(x) for n, x in like_out.items()}) for _ in range(2)]
        self.s_in, self.s_run, self.s_out = (torch.cuda.Stream() for _ in range(3))
        self.ev_in = [torch.cuda.Event() for _ in range(2)]
        self.ev_run = [torch.cuda.Event() for _ in range(2)]
        self.ev_out = [torch.cuda.Event() for _ in range(2)]
        self.n = 0

    def step(self, host_in: dict, host_out: dict):
        i = self.n % 2
        dev_in, dev_out = self.sets[i]
        with torch.cuda.stream(self.s_in):
            if self.n >= 2:
                self.s_in.wait_event(self.ev_run[i])          # the kernels of step n-2 have read this input set
            for n in ("q", "k", "v", "g", "dO"):
                dev_in[n].copy_(host_in[n], non_blocking=True)
            self.ev_in[i].record(self.s_in)
        with torch.cuda.stream(self.s_run):
            self.s_run.wait_event(self.ev_in[i])
            if self.n >= 2:
                self.s_run.wait_event(self.ev_out[i])         # the results of step n-2 have left this output set
            run_fwd_bwd(self.plan, self.ws, dev_in["q"], dev_in["k"], dev_in["v"], dev_in["g"], dev_in["dO"], out=dev_out,
                        stream=self.s_run)
            self.ev_run[i].record(self.s_run)
        with torch.cuda.stream(self.s_out):
            self.s_out.wait_event(self.ev_run[i])
            for n in ("o", "dq", "dk", "dv", "dg"):
                host_out[n].copy_(dev_out[n], non_blocking=True)
            self.ev_out[i].record(self.s_out)
        self.n += 1

    def finish(self):
        for s in (self.s_in, self.s_run, self.s_out):
            s.synchronize()


def harts_la_expand(tree_node_ptr, node_parent, node_fork_off, node_len):
    """Trajectory-wise view of a forest (the conventional baseline of Section 5): returns (length of every
    root-to-leaf trajectory, canonical compact token index of every expanded position)."""
    arrs = [np.ascontiguousarray(a, dtype=np.int32) for a in (tree_node_ptr, node_parent, node_fork_off, node_len)]
    ptrs = [a.ctypes.data_as(_I32P) for a in arrs]
    n_traj, n_tok = C.c_int64(0), C.c_int64(0)
    _check(lib.harts_la_expand(len(arrs[0]) - 1, *ptrs, 0, 0, None, None, C.byref(n_traj), C.byref(n_tok)),
           "harts_la_expand")
    lens = np.empty(n_traj.value, np.int32)
    src = np.empty(n_tok.value, np.int64)
    _check(lib.harts_la_expand(len(arrs[0]) - 1, *ptrs, n_traj.value, n_tok.value, lens.ctypes.data_as(_I32P),
                               src.ctypes.data_as(C.POINTER(C.c_int64)), C.byref(n_traj), C.byref(n_tok)),
           "harts_la_expand")
    return lens, src


def expand_trajectories(tree_node_ptr, node_parent, node_fork_off, node_len):
    """The expanded problem as forest arrays (every trajectory a single-node tree) plus the source-token map."""
    lens, src = harts_la_expand(tree_node_ptr, node_parent, node_fork_off, node_len)
    n = len(lens)
    forest = (np.arange(n + 1, dtype=np.int32), np.full(n, -1, np.int32), np.zeros(n, np.int32), lens)
    return forest, src
