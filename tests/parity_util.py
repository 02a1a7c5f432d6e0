"""Shared helpers for the GPU parity tests: run a forest through the C ABI and through the oracle."""
import numpy as np
import torch

import paper_2608_28158_b200 as H
from oracle import la_oracle as lo
from workloads import CONFIGS, config_forest, make_inputs

TORCH_DTYPE = {"fp32": torch.float32, "bf16": torch.bfloat16}


def rel_err(x, ref):
    """Relative Frobenius error.  Where the reference is (numerically) zero -- e.g. dg of a one-token
    trajectory, which is exactly 0 -- the denominator falls back to 1e-3 per element, i.e. the
    difference is held to an absolute bound instead."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    return float(np.linalg.norm(x - ref) / max(np.linalg.norm(ref), 1e-3 * np.sqrt(ref.size)))


def row_err(x, ref):
    """Largest per-row error: a row is the feature vector of one (token, head) -- for dg, its one number -- and its
    error is measured against max(norm of the reference row, RMS norm of a row of the tensor), so that a row that is
    nearly zero is held to the tensor's typical size.  One wrong row among half a million moves the Frobenius error
    of the tensor by nothing; it moves this."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    width = x.shape[-1] if x.ndim == 3 else 1
    x, ref = x.reshape(-1, width), ref.reshape(-1, width)
    floor = max(np.sqrt((ref ** 2).mean() * width), 1e-3 * np.sqrt(width))
    return float((np.linalg.norm(x - ref, axis=1) / np.maximum(np.linalg.norm(ref, axis=1), floor)).max())


def plan_of(fo, chunk=64):
    return H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, chunk)


def to_physical(plan, canon: dict, device="cuda"):
    """canonical-order tensors -> physical-row-order device tensors"""
    rows = torch.as_tensor(plan.row_of_token.astype(np.int64), device=canon["q"].device)
    out = {}
    for n, x in canon.items():
        y = torch.empty_like(x)
        y[rows] = x
        out[n] = y.to(device)
    return out


GUARD = 4096      # elements of guard band on either side of every output tensor


def guarded_like(x):
    """A tensor like x that sits between two guard bands filled with a bit pattern no kernel produces; check() fails if
    anything was written outside the tensor (canary rows around every output)."""
    n = x.numel()
    flat = torch.empty(n + 2 * GUARD, dtype=x.dtype, device=x.device)
    pattern = torch.full((1,), -12345.0, dtype=x.dtype, device=x.device)
    flat[:GUARD] = pattern
    flat[GUARD + n:] = pattern
    view = flat[GUARD:GUARD + n].view(x.shape)
    view.fill_(float("nan"))

    def check():
        assert bool((flat[:GUARD] == pattern).all()) and bool((flat[GUARD + n:] == pattern).all()), "write outside an output"
    return view, check


def run_gpu(fo, inp_canon, flags=0, backward=True, chunk=64):
    """Returns (plan, outputs in CANONICAL order as device tensors).  Every output sits between guard bands that must
    come back untouched, and starts as NaN so that a row nobody wrote shows up."""
    plan = plan_of(fo, chunk).upload()
    phys = to_physical(plan, inp_canon)
    H_, dk, dv = phys["q"].shape[1], phys["q"].shape[2], phys["v"].shape[2]
    ws = H.Workspace(plan, H_, dk, dv, phys["q"].dtype, flags)
    like = {"o": phys["v"], "dq": phys["q"], "dk": phys["k"], "dv": phys["v"], "dg": phys["g"]}
    out, checks = {}, []
    for n in (("o", "dq", "dk", "dv", "dg") if backward else ("o",)):
        out[n], chk = guarded_like(like[n])
        checks.append(chk)
    H.run_fwd_bwd(plan, ws, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"], out=out, backward=backward)
    H.harts_la_check(ws.dev_status)
    for chk in checks:
        chk()
    rows = torch.as_tensor(plan.row_of_token.astype(np.int64), device="cuda")
    return plan, {n: x[rows] for n, x in out.items()}


def oracle_subset(fo, inp_canon, tree_ids, heads, backward=True):
    """Oracle on the given trees and heads.  Returns (canonical token indices of the subset, results)."""
    base = fo.token_base()
    tok = np.concatenate([np.arange(base[fo.tree_node_ptr[t]], base[fo.tree_node_ptr[t + 1]]) for t in tree_ids])
    sub = fo.subset(tree_ids)
    ti = torch.as_tensor(tok, device=inp_canon["q"].device)
    hi = torch.as_tensor(heads, device=inp_canon["q"].device)
    pick = {n: x[ti][:, hi].cpu() for n, x in inp_canon.items()}
    res = lo.forest_eval(sub, pick["q"], pick["k"], pick["v"], pick["g"], pick["dO"] if backward else None)
    return tok, res


def compare(out_canon, tok, heads, ref, names=("o", "dq", "dk", "dv", "dg"), rows=False):
    """Relative Frobenius error per tensor; with rows=True also the largest per-row error (keys "<name>.row")."""
    ti = torch.as_tensor(tok, device="cuda")
    hi = torch.as_tensor(heads, device="cuda")
    errs = {}
    for n in names:
        got = out_canon[n][ti][:, hi].float().cpu().numpy()
        errs[n] = rel_err(got, ref[n])
        if rows:
            errs[n + ".row"] = row_err(got, ref[n])
    return errs


def config_case(name, device="cpu"):
    cfg = CONFIGS[name]
    fo = config_forest(name)
    inp = make_inputs(fo.n_tokens, cfg["H"], cfg["dk"], cfg["dv"], cfg["dtype"], cfg["seed"], device=device)
    return cfg, fo, inp
