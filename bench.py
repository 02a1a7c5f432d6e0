#!/usr/bin/env python
"""Benchmark of the tree-packed linear-attention hot path (forward + backward over all rounds).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg3] [--impl ours|reference]

One step = one pass of the whole path over one batch: every forward round, every backward round and
the replay-gradient fold, on synthetic trees and tensors of the named configuration.  Prints ONE
JSON line.  ``value`` is compact tokens per second with inputs resident in HBM; ``e2e`` is the same
metric through the host-buffer call (pinned host inputs copied in, results copied out, inside the
timed region).  With N > 1 (torchrun) every rank runs its own copy of the workload (weak scaling,
no collective on the data path); time is the maximum over ranks.

``--workload logp`` runs the second path instead, the compact-to-semantic log-probability (one step = its
forward + backward over one microbatch of compact logit rows), ``--workload conv`` the tree-aware causal
convolution that precedes the linear-attention core, ``--workload attn`` full attention on compact tokens; all
print the same JSON keys.

``--impl reference`` times the fp64 CPU oracle (oracle/), as it stands, on the host cores, on a
bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tree-packed linear-attn fwd+bwd compact tokens/s"
UNIT = "compact tokens/s"
L2_BYTES = 126 * 1024 * 1024


# --------------------------------------------------------------------------------------------------
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [x.strip() for x in line.split(",")]))

    def mark(self):
        """Host time now; summary(t0, t1) keeps the samples taken between two marks."""
        return time.time()

    def __exit__(self, *exc):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for stamp, r in self.rows:
            if len(r) < 6 or (t0 is not None and not (t0 <= stamp <= t1 + 0.05)):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for n, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------------
def oracle_sample(name, seconds_hint=15.0):
    """The fp64 oracle on a bounded sample of the workload: whole trees, a few heads."""
    import torch
    from oracle import la_oracle
    from workloads import CONFIGS, config_forest, make_inputs

    cfg = CONFIGS[name]
    fo = config_forest(name)
    heads = sorted({0, cfg["H"] // 2, cfg["H"] - 1})
    # about 40k semantic token-heads per second on 8 cores: take trees until the budget is used
    budget = 40000.0 * seconds_hint * max(1, (os.cpu_count() or 8)) / 8
    base = fo.token_base()
    trees, sem = [], 0
    from workloads.trees import tree_counts
    for t in range(fo.n_trees):
        c, s, _ = tree_counts(*(a.tolist() for a in fo.tree(t)))
        if trees and (sem + s) * len(heads) > budget:
            break
        trees.append(t)
        sem += s
    sub = fo.subset(trees)
    inp = make_inputs(sub.n_tokens, len(heads), cfg["dk"], cfg["dv"], cfg["dtype"], cfg["seed"])
    t0 = time.perf_counter()
    res = la_oracle.forest_eval(sub, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
    dt = time.perf_counter() - t0
    # compact tokens/s at the configuration's head count: the sample covered len(heads) of H heads
    value = sub.n_tokens * len(heads) / cfg["H"] / dt
    return {"value": value, "unit": UNIT, "cores": res["threads"], "kind": "oracle",
            "sample": f"{name}: trees {trees[0]}..{trees[-1]} ({sub.n_tokens} compact / {res['S']} trajectory-wise "
                      f"tokens), {len(heads)} of {cfg['H']} heads, fwd+bwd, {dt:.1f} s",
            "semantic_token_heads_per_s": res["S"] * len(heads) / dt, "seconds": dt}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times, secs, last = [], [], None
    # every step is a bounded sample; its size shrinks with the step count so that the whole run stays within minutes
    hint = min(8.0, 150.0 / max(1, args.warmup + args.steps))
    for i in range(args.warmup + args.steps):
        last = oracle_sample(args.workload, seconds_hint=hint)
        if i >= args.warmup:
            times.append(last["value"])
            secs.append(last["seconds"])
    value = statistics.mean(times)
    from workloads import CONFIGS
    cfg = CONFIGS[args.workload]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(secs) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "H": cfg["H"], "dk": cfg["dk"], "dv": cfg["dv"], "chunk": 64},
            "cpu_baseline": {"kind": last["kind"], "cores": last["cores"], "sample": last["sample"], "value": value,
                             "unit": UNIT},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------------------------------
# Second workload: compact-to-semantic log-probability (Eqs. 17, 19), `--workload logp`
# --------------------------------------------------------------------------------------------------
LOGP_METRIC = "mapped log-prob fwd+bwd compact rows/s"
LOGP_UNIT = "compact rows/s"
LOGP_V = 157184            # vocabulary of the evaluated model
LOGP_ROWS = 65536          # compact-row capacity of one microbatch


def logp_forest(rank=0, capacity=LOGP_ROWS):
    """Whole trees of cfg3, starting at a rank-dependent tree, while they fit the microbatch capacity.  A capacity
    below the first tree's size (a small case for a profiler capture) gives copies of the cfg0b tree instead."""
    from workloads import CONFIGS, make_forest
    fo = config_forest_cached("cfg3")
    base = fo.token_base()
    first = (3 * rank) % fo.n_trees
    trees, rows = [], 0
    for t in list(range(first, fo.n_trees)) + list(range(first)):
        c = int(base[fo.tree_node_ptr[t + 1]] - base[fo.tree_node_ptr[t]])
        if rows + c > capacity:
            break
        trees.append(t)
        rows += c
    if not trees:
        tree = CONFIGS["cfg0b"]["build"]()[0]
        n = max(1, capacity // sum(tree[2]))
        return make_forest([tree] * n), f"{n} x cfg0b"
    return fo.subset(trees), f"cfg3 trees {trees}"


def config_forest_cached(name):
    from workloads import config_forest
    return config_forest(name)


def logp_oracle_sample(small=False, copies=1):
    """The fp64 oracle of Eqs. 17/19 on small trees at the full vocabulary.  The full leg first times one cfg0b
    tree, then sizes a forest of such trees to about 12 s of work and reports that run."""
    from oracle import logp_oracle
    from workloads import CONFIGS, make_forest, make_logits, make_logp_grad
    # small: a 256-row tree (root 128, one child at its end, one forking at offset 100) for the many-step arm
    tree = ([-1, 0, 0], [0, 128, 100], [128, 64, 64]) if small else CONFIGS["cfg0b"]["build"]()[0]
    fo = make_forest([tree] * copies)
    name = "three-node tree" if small else f"{copies} x cfg0b tree"
    data = make_logits(fo.n_tokens, LOGP_V, "bf16", 0)
    m, y, _ = logp_oracle.positions(fo, data["token_id"].numpy())
    g = make_logp_grad(len(m), 0, keep=1.0).double().numpy()
    z = data["z"].double().numpy()
    t0 = time.perf_counter()
    logp_oracle.mapped_logp(z, m, y)
    logp_oracle.mapped_logp_grad(z, m, y, g)
    dt = time.perf_counter() - t0
    if not small and copies == 1 and dt < 8.0:
        return logp_oracle_sample(False, copies=int(min(8, max(2, round(12.0 / dt)))))
    return {"value": fo.n_tokens / dt, "unit": LOGP_UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{name}: {fo.n_tokens} compact rows, {len(m)} positions, V={LOGP_V}, fwd+bwd, {dt:.1f} s",
            "seconds": dt}


def run_logp_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    vals, secs, last = [], [], None
    for i in range(args.warmup + args.steps):
        last = logp_oracle_sample(small=True)
        if i >= args.warmup:
            vals.append(last["value"])
            secs.append(last["seconds"])
    value = statistics.mean(vals)
    print(json.dumps({
        "impl": "reference", "metric": LOGP_METRIC, "value": value, "unit": LOGP_UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(secs) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "logp", "V": LOGP_V},
        "cpu_baseline": {"kind": last["kind"], "cores": last["cores"], "sample": last["sample"], "value": value,
                         "unit": LOGP_UNIT},
        "e2e": {"value": value, "unit": LOGP_UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# --------------------------------------------------------------------------------------------------
def max_over_ranks(values, device):
    """Element-wise maximum of a few per-rank timings over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def trajectory_wise_ms(H, fo, cfg, inp, flags, trees_per_batch=4):
    """Forward + backward of the SAME kernels on the expanded problem (every root-to-leaf trajectory its own
    zero-state sequence, the conventional baseline), in batches of trees that fit in memory.  Returns
    (milliseconds summed over the batches, trajectory-wise token count)."""
    import torch
    from workloads import make_forest

    base = fo.token_base()
    total_ms, total_rows = 0.0, 0
    for lo in range(0, fo.n_trees, trees_per_batch):
        ids = list(range(lo, min(fo.n_trees, lo + trees_per_batch)))
        sub = fo.subset(ids)
        tok0 = int(base[fo.tree_node_ptr[ids[0]]])
        (ptr, par, off, ln), src = H.expand_trajectories(sub.tree_node_ptr, sub.node_parent, sub.node_fork_off,
                                                         sub.node_len)
        plan = H.harts_la_plan(ptr, par, off, ln, cfg["chunk"]).upload()
        # expanded rows in plan order: physical row r holds canonical expanded token inv[r]
        inv = np.empty(plan.C, dtype=np.int64)
        inv[plan.row_of_token] = np.arange(plan.C)
        gather = torch.as_tensor(src[inv] + tok0, device="cuda")
        ex = {n: x.index_select(0, gather) for n, x in inp.items()}
        ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], ex["q"].dtype, flags)
        out = None
        for it in range(2):                      # one warm-up, one timed
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            out = H.run_fwd_bwd(plan, ws, ex["q"], ex["k"], ex["v"], ex["g"], ex["dO"], out=out)
            b.record()
            torch.cuda.synchronize()
        H.harts_la_check(ws.dev_status)
        total_ms += a.elapsed_time(b)
        total_rows += plan.C
        del ex, ws, out, plan
        torch.cuda.empty_cache()
    return total_ms, total_rows


def per_config_table(args):
    """Compact tokens/s, strict roofline fraction and trajectory-wise speedup of every bf16 configuration (cfg0 is
    fp32 and runs the FMA kernels).  Opt-in (--per-config): printed to stderr, the JSON line is unchanged."""
    import torch
    import paper_2608_28158_b200 as H
    from workloads import CONFIGS, config_forest, make_inputs

    peaks = measured_peaks()
    rows = []
    for name in ("cfg0", "cfg1", "cfg2", "cfg3", "cfg4"):
        cfg = CONFIGS[name]
        fo = config_forest(name)
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, cfg["chunk"]).upload()
        canon = make_inputs(plan.C, cfg["H"], cfg["dk"], cfg["dv"], cfg["dtype"], cfg["seed"], device="cuda")
        rows_t = torch.as_tensor(plan.row_of_token.astype(np.int64), device="cuda")
        inp = {}
        for n, x in canon.items():
            y = torch.empty_like(x)
            y[rows_t] = x
            inp[n] = y
        ws = H.Workspace(plan, cfg["H"], cfg["dk"], cfg["dv"], inp["q"].dtype)
        out = None
        for _ in range(3):
            out = H.run_fwd_bwd(plan, ws, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"], out=out)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(5):
            H.run_fwd_bwd(plan, ws, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"], out=out)
        b.record()
        torch.cuda.synchronize()
        H.harts_la_check(ws.dev_status)
        ms = a.elapsed_time(b) / 5
        del inp, ws, out
        t_ms, t_rows = trajectory_wise_ms(H, fo, cfg, canon, 0, trees_per_batch=4)
        elem = canon["q"].element_size()
        th = plan.C * cfg["H"]
        bytes_ = th * ((6 * cfg["dk"] + 5 * cfg["dv"]) * elem + 12)
        rows.append((name, plan.C, t_rows, plan.R, plan.n_rounds, plan.n_seq, ms, plan.C / ms * 1e3,
                     bytes_ / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms, t_ms / ms))
        del canon
        torch.cuda.empty_cache()
    print("config  compact  traj-wise  replay  rounds  seqs   ms/step  compact tok/s  strict-roof  speedup vs traj-wise",
          file=sys.stderr)
    for r in rows:
        print(f"{r[0]:6s} {r[1]:8d} {r[2]:10d} {r[3]:7d} {r[4]:7d} {r[5]:6d} {r[6]:8.3f} {r[7]:14.0f} {r[8]:11.3f} {r[9]:10.2f}",
              file=sys.stderr)


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2608_28158_b200 as H
    from workloads import CONFIGS, config_forest, make_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    cfg = CONFIGS[args.workload]
    fo = config_forest(args.workload)
    t_plans = []
    for _ in range(3):                                 # host planning time: median of three calls
        t0 = time.perf_counter()
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, cfg["chunk"])
        t_plans.append(time.perf_counter() - t0)
    t_plan = statistics.median(t_plans)
    plan.upload()
    Hh, dk, dv = cfg["H"], cfg["dk"], cfg["dv"]
    # every rank draws its own tensors (independent batches of the same shape)
    inp = make_inputs(plan.C, Hh, dk, dv, cfg["dtype"], cfg["seed"] + 100 * rank, device="cuda")
    flags = H.HARTS_FLAG_FMA_KERNELS if args.fma else 0
    ws = H.Workspace(plan, Hh, dk, dv, inp["q"].dtype, flags)
    out = {"o": torch.empty_like(inp["v"]), "dq": torch.empty_like(inp["q"]), "dk": torch.empty_like(inp["k"]),
           "dv": torch.empty_like(inp["v"]), "dg": torch.empty_like(inp["g"])}
    elem = inp["q"].element_size()
    in_bytes = sum(x.numel() * x.element_size() for x in inp.values())
    out_bytes = sum(x.numel() * x.element_size() for x in out.values())
    stream = torch.cuda.current_stream()
    K = plan.n_rounds

    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    launch_times = {"fwd": [], "bwd": [], "fold": []}

    def step(record):
        marks = []
        for r in range(1, K + 1):
            a, b = ev(), ev()
            a.record(stream)
            H.harts_la_fwd(plan, r, inp["q"], inp["k"], inp["v"], inp["g"], out["o"], ws.slots, ws.chunk_states,
                           flags, ws.dev_status)
            b.record(stream)
            marks.append(("fwd", a, b))
        for r in range(K, 0, -1):
            a, b = ev(), ev()
            a.record(stream)
            H.harts_la_bwd_seqs(plan.tables, int(plan.round_seq_ptr[r - 1]), int(plan.round_seq_ptr[r]), inp["q"],
                                inp["k"], inp["v"], inp["g"], inp["dO"], out["dq"], out["dk"], out["dv"], out["dg"],
                                ws.chunk_states, ws.scratch, flags, ws.dev_status)
            b.record(stream)
            marks.append(("bwd", a, b))
        a, b = ev(), ev()
        a.record(stream)
        H.harts_la_bwd_finish(plan.tables, out["dk"], out["dv"], out["dg"], ws.scratch)
        b.record(stream)
        marks.append(("fold", a, b))
        if record:
            return marks
        return None

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    all_marks = []
    t_begin, t_end = ev(), ev()
    with ClockSampler(local) as clocks:            # started before the warm-up so that it is sampling by then
        for _ in range(args.warmup):
            step(False)
        H.harts_la_check(ws.dev_status)
        # a short region gives the 50 ms sampler nothing to see: keep the GPU under the same load a little longer
        # before the timed steps when the whole region is under a second
        barrier()
        t_host0 = clocks.mark()
        t_begin.record(stream)
        for _ in range(args.steps):
            all_marks.append(step(True))
        t_end.record(stream)
        barrier()
        t_host1 = clocks.mark()
    ms_total = t_begin.elapsed_time(t_end)
    H.harts_la_check(ws.dev_status)
    for marks in all_marks:
        for kind, a, b in marks:
            launch_times[kind].append(a.elapsed_time(b))

    # ---- end to end through host buffers -----------------------------------------------------------
    e2e = None
    if not args.no_e2e:
        pinned = True
        try:
            host_in = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in inp.items()}
            host_out = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in out.items()}
        except RuntimeError:
            pinned = False
            host_in = {n: torch.empty(x.shape, dtype=x.dtype) for n, x in inp.items()}
            host_out = {n: torch.empty(x.shape, dtype=x.dtype) for n, x in out.items()}
        for n in inp:
            host_in[n].copy_(inp[n])
        torch.cuda.synchronize()
        e2e_steps = max(1, min(args.steps, args.e2e_steps))
        H.run_fwd_bwd_host(plan, ws, host_in, inp, out, host_out)       # warm-up; also the unpipelined reference
        barrier()
        a, b = ev(), ev()
        a.record(stream)
        H.run_fwd_bwd_host(plan, ws, host_in, inp, out, host_out)
        b.record(stream)
        barrier()
        serial_ms = a.elapsed_time(b)
        # pipelined: the copies of neighbouring steps overlap (three streams, two device buffer sets); every step
        # still moves all of its inputs in and all of its results out
        pipe = H.HostPipeline(plan, ws, inp, out)
        pipe.step(host_in, host_out)                                    # warm-up of the streams
        pipe.finish()
        barrier()
        t0 = time.perf_counter()
        a, b = ev(), ev()
        a.record(pipe.s_in)
        for _ in range(e2e_steps):
            pipe.step(host_in, host_out)
        b.record(pipe.s_out)
        pipe.finish()
        barrier()
        e2e_ms = a.elapsed_time(b) / e2e_steps
        e2e = {"ms_per_step": e2e_ms, "steps": e2e_steps, "pinned": pinned, "serial_ms_per_step": serial_ms,
               "wall_ms_per_step": (time.perf_counter() - t0) * 1e3 / e2e_steps}
        del pipe
        del host_in, host_out

    # ---- the same kernels, trajectory-wise (Section 5 baseline) ---------------------------------------------
    traj = None
    if world == 1 and not args.no_trajwise:
        # inputs are in physical order here; the expansion wants canonical order
        rows = torch.as_tensor(plan.row_of_token.astype(np.int64), device="cuda")
        canon = {n: x[rows] for n, x in inp.items()}
        t_ms, t_rows = trajectory_wise_ms(H, fo, cfg, canon, flags)
        traj = {"ms": t_ms, "rows": t_rows}
        del canon

    # ---- reduce over ranks ------------------------------------------------------------------------
    ms_step = ms_total / args.steps
    if world > 1:
        ms_step, e2e_ms_max = max_over_ranks([ms_step, e2e["ms_per_step"] if e2e else 0.0], "cuda")
        if e2e:
            e2e["ms_per_step"] = e2e_ms_max
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    tokens = plan.C * world
    value = tokens / (ms_step * 1e-3)
    th = plan.C * Hh                                  # token-heads per rank and step
    # algorithmic (compulsory) bytes per token-head: fwd reads q,k,v,g and writes o; bwd reads q,k,v,dO,g
    # and writes dq,dk,dv,dg
    fwd_bytes = th * ((2 * dk + 2 * dv) * elem + 4)
    bwd_bytes = th * ((4 * dk + 3 * dv) * elem + 8)
    flops_fwd = th * (2 * 64 * dk + 2 * 64 * dv + 4 * dk * dv)
    flops_bwd = th * (5 * 2 * 64 * (dk + dv) // 2 + 4 * 2 * dk * dv)
    bwd_ms = sum(launch_times["bwd"]) / args.steps
    fwd_ms = sum(launch_times["fwd"]) / args.steps
    fold_ms = sum(launch_times["fold"]) / args.steps
    hbm_peak = peaks["hbm_gbs"]
    achieved = bwd_bytes / (bwd_ms * 1e-3) / 1e9
    # DRAM bytes per token-head of the backward kernel from the ncu capture on cfg2 (profiles/
    # tc_bwd_kernel_cfg2_ncu_full.md), scaled to this workload's token-heads; traffic grows in proportion to them
    BWD_DRAM_BYTES_PER_TOKEN_HEAD = 2356.0
    bwd_traffic_per_launch = (BWD_DRAM_BYTES_PER_TOKEN_HEAD * th / K) if (dk == 128 and not args.fma and elem == 2) \
        else None
    t_roof_bytes = (fwd_bytes + bwd_bytes) / (hbm_peak * 1e9)
    t_roof_flops = (flops_fwd + flops_bwd) / (peaks["bf16_tflops_sustained"] * 1e12)
    clock = clocks.summary(t_host0, t_host1)
    if not clock["samples"]:
        clock = clocks.summary()
        clock["note"] = "timed region shorter than the sampling period: samples cover warm-up + timed region"
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": cfg["dtype"] if cfg["dtype"] != "fp32" else "f32", "data": "synthetic",
        "config": {"workload": args.workload, "H": Hh, "dk": dk, "dv": dv, "chunk": cfg["chunk"],
                   "compact_tokens": plan.C, "replay_rows": plan.R, "rounds": plan.n_rounds,
                   "sequences": plan.n_seq, "slots": plan.n_slots, "chunks": plan.n_chunks,
                   "l2": f"inputs larger than L2 ({in_bytes / 2**30:.2f} GiB read per step)"
                         if in_bytes > 2 * L2_BYTES else "inputs smaller than L2: no flush (small workload)",
                   "kernels": "fma" if args.fma or cfg["dtype"] == "fp32" else "default",
                   "plan_ms": t_plan * 1e3},
        "roofline": {"bound": "hbm", "kernel": "backward packed call (all rounds)", "achieved": achieved,
                     "peak": hbm_peak, "unit": "GB/s", "frac": achieved / hbm_peak, "traffic": bwd_traffic_per_launch,
                     "traffic_note": "bytes per launch (mean over the rounds), scaled from the ncu capture on cfg2",
                     "algorithmic_bytes_per_launch": bwd_bytes / K,
                     "peak_source": peaks["source"],
                     "whole_path": {"roof_ms": max(t_roof_bytes, t_roof_flops) * 1e3,
                                    "frac_strict": max(t_roof_bytes, t_roof_flops) * 1e3 / ms_step,
                                    "frac_strict_nominal": max((fwd_bytes + bwd_bytes) / 8e12,
                                                               (flops_fwd + flops_bwd) / 2.25e15) * 1e3 / ms_step}},
        "kernel_ms": {"fwd": fwd_ms, "bwd": bwd_ms, "fold": fold_ms},
        # per step: K forward calls, K backward calls each preceded by the hand-off reduction when the plan has
        # exported boundaries, and the replay-gradient fold
        "gpu_launches": (2 * K + (K if plan.n_slots else 0) + (1 if plan.n_rg_rows else 0)) * args.steps,
        "clocks": clock,
    }
    if e2e:
        line["e2e"] = {"value": tokens / (e2e["ms_per_step"] * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": in_bytes, "d2h_bytes_per_step": out_bytes, "steps": e2e["steps"],
                       "pinned_host_memory": e2e["pinned"],
                       "overlap": "copies of neighbouring steps overlap the kernels (3 streams, 2 device buffer sets)",
                       "unpipelined_value": tokens / (e2e["serial_ms_per_step"] * 1e-3)}
    # method traffic on top of the compulsory bytes: replayed rows (k, v, g read in both passes, gradient
    # contributions written and folded), state hand-offs (initial state read + its gradient written, slot written +
    # consumers' gradients read), chunk states (written by the forward, read by the backward, 2 B per element)
    n_side = int((plan.seq_init_slot >= 0).sum())
    method_bytes = (fwd_bytes + bwd_bytes + plan.R * Hh * (6 * dk * elem + 12)
                    + (n_side + plan.n_slots) * Hh * dk * dv * 4 * 2 + plan.n_chunks * Hh * dk * dv * 2 * 2)
    line["roofline"]["whole_path"]["frac_method"] = max(method_bytes / (hbm_peak * 1e9), t_roof_flops) * 1e3 / ms_step
    if traj:
        line["trajectory_wise"] = {"ms": traj["ms"], "rows": traj["rows"], "rows_ratio": traj["rows"] / plan.C,
                                   "speedup": traj["ms"] / ms_step,
                                   "speedup_with_plan": traj["ms"] / (ms_step + t_plan * 1e3),
                                   "paper_context": "4.81-4.87x F/B/Grad on a whole hybrid MoE model, 8x H20-3e (Table 4)"}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = oracle_sample(args.workload)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    elif args.per_config:
        del inp, out, ws
        torch.cuda.empty_cache()
        per_config_table(args)


def run_logp(args):
    """One step = forward (row max / sum-exp over V, lambda for every position) + backward (dz for every compact row)."""
    import torch
    import torch.distributed as dist

    import paper_2608_28158_b200 as H
    from workloads import make_logits, make_logp_grad

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fo, trees = logp_forest(rank, args.logp_rows)
    C, V = fo.n_tokens, LOGP_V
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    data = make_logits(C, V, "bf16", 50 + rank, device="cuda")
    t0 = time.perf_counter()
    m, y, _ = H.harts_logp_positions(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                     data["token_id"].cpu().numpy(), plan.row_of_token)
    ptr, pos = H.harts_logp_csr(C, m)
    t_host = time.perf_counter() - t0
    P = len(m)
    z = data["z"]
    dev = {"m": torch.as_tensor(m).cuda(), "y": torch.as_tensor(y).cuda(), "ptr": torch.as_tensor(ptr).cuda(),
           "pos": torch.as_tensor(pos).cuda(), "g": make_logp_grad(P, 50 + rank, device="cuda", keep=1.0)}
    lse = torch.empty(C, device="cuda")
    lam = torch.empty(P, device="cuda")
    dz = torch.empty_like(z)
    status = torch.zeros(2, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def step(marks=None):
        a, b, c = ev(), ev(), ev()
        a.record(stream)
        H.harts_logp_fwd(z, dev["m"], dev["y"], lse, lam, dev_status=status)
        b.record(stream)
        H.harts_logp_bwd(z, dev["y"], dev["ptr"], dev["pos"], lse, dev["g"], dz, dev_status=status)
        c.record(stream)
        if marks is not None:
            marks.append((a, b, c))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    marks = []
    t_begin, t_end = ev(), ev()
    with ClockSampler(local) as clocks:
        for _ in range(args.warmup):
            step()
        H.harts_la_check(status)
        barrier()
        h0 = clocks.mark()
        t_begin.record(stream)
        for _ in range(args.steps):
            step(marks)
        t_end.record(stream)
        barrier()
        h1 = clocks.mark()
    H.harts_la_check(status)
    ms_step = t_begin.elapsed_time(t_end) / args.steps
    fwd_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in marks)
    bwd_ms = statistics.mean(b.elapsed_time(c) for _, b, c in marks)

    e2e = None
    if not args.no_e2e:
        small = {n: x for n, x in dev.items()}
        host_in = {"z": torch.empty(z.shape, dtype=z.dtype, pin_memory=True)}
        host_in.update({n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in small.items()})
        host_out = {"lam": torch.empty(P, pin_memory=True), "dz": torch.empty(z.shape, dtype=z.dtype, pin_memory=True)}
        host_in["z"].copy_(z)
        for n, x in small.items():
            host_in[n].copy_(x)
        torch.cuda.synchronize()

        def e2e_step():
            z.copy_(host_in["z"], non_blocking=True)
            for n, x in small.items():
                x.copy_(host_in[n], non_blocking=True)
            step()
            host_out["lam"].copy_(lam, non_blocking=True)
            host_out["dz"].copy_(dz, non_blocking=True)

        e2e_step()
        barrier()
        a, b = ev(), ev()
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        e2e = {"ms": a.elapsed_time(b) / n_e2e, "steps": n_e2e,
               "h2d": sum(x.numel() * x.element_size() for x in host_in.values()),
               "d2h": sum(x.numel() * x.element_size() for x in host_out.values())}
        del host_in, host_out

    if world > 1:
        ms_step, e2e_ms = max_over_ranks([ms_step, e2e["ms"] if e2e else 0.0], "cuda")
        if e2e:
            e2e["ms"] = e2e_ms
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    row_bytes = V * z.element_size()
    fwd_bytes = C * row_bytes + P * 12 + C * 4              # z once; m, y read and lambda written; lse written
    bwd_bytes = 2 * C * row_bytes + P * 12 + C * 12         # z read, dz written; y, g, row_pos; lse, row_pos_ptr
    achieved = bwd_bytes / (bwd_ms * 1e-3) / 1e9
    clock = clocks.summary(h0, h1)
    if not clock["samples"]:
        clock = clocks.summary()
    line = {
        "metric": LOGP_METRIC, "value": C * world / (ms_step * 1e-3), "unit": LOGP_UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "logp", "V": V, "compact_rows": C, "positions": P, "trees": trees,
                   "action_mask": "every position selected (no idle rows)",
                   "l2": f"inputs larger than L2 ({C * row_bytes / 2**30:.2f} GiB of logits)",
                   "host_index_ms": t_host * 1e3},
        "roofline": {"bound": "hbm", "kernel": "dz_kernel (backward)", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                     "algorithmic_bytes_per_launch": bwd_bytes, "peak_source": peaks["source"],
                     "forward": {"achieved": fwd_bytes / (fwd_ms * 1e-3) / 1e9,
                                 "frac": fwd_bytes / (fwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                     "whole_path": {"roof_ms": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3,
                                    "frac_strict": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms_step}},
        "kernel_ms": {"fwd": fwd_ms, "bwd": bwd_ms},
        "gpu_launches": 3 * args.steps,
        "clocks": clock,
    }
    if e2e:
        line["e2e"] = {"value": C * world / (e2e["ms"] * 1e-3), "unit": LOGP_UNIT, "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"], "pinned_host_memory": True}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = logp_oracle_sample()
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# Third workload: tree-aware causal convolution before the linear-attention core (Section 4.2), `--workload conv`
# --------------------------------------------------------------------------------------------------
CONV_METRIC = "tree-aware causal conv fwd+bwd compact tokens/s"
CONV_W = 4


def conv_oracle_sample(small=False):
    from oracle import conv_oracle
    from workloads import CONFIGS, config_forest, make_conv_inputs, make_forest
    D = 256 if small else 4096
    fo = config_forest("cfg0b") if small else make_forest(CONFIGS["cfg1"]["build"]() * 2)
    inp = make_conv_inputs(fo.n_tokens, D, CONV_W, "bf16", 0)
    x, dy, W = (inp[n].double().numpy() for n in ("x", "dy", "W"))
    t0 = time.perf_counter()
    conv_oracle.conv_fwd(fo, x, W)
    conv_oracle.conv_bwd(fo, x, W, dy)
    dt = time.perf_counter() - t0
    # compact tokens/s at the benchmark's channel count (the sample has D channels of 4096)
    return {"value": fo.n_tokens * D / 4096 / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{fo.n_tokens} compact tokens ({'cfg0b tree' if small else '2 x cfg1 tree'}), {D} of 4096 channels, w={CONV_W}, fwd+bwd, {dt:.1f} s",
            "seconds": dt}


def run_conv_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    vals, secs, last = [], [], None
    for i in range(args.warmup + args.steps):
        last = conv_oracle_sample(small=True)
        if i >= args.warmup:
            vals.append(last["value"])
            secs.append(last["seconds"])
    value = statistics.mean(vals)
    print(json.dumps({
        "impl": "reference", "metric": CONV_METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(secs) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "conv", "D": 4096, "w": CONV_W},
        "cpu_baseline": {"kind": last["kind"], "cores": last["cores"], "sample": last["sample"], "value": value,
                         "unit": UNIT},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_conv(args):
    """One step = forward + backward (dx, dW) of the width-4 depthwise convolution over cfg3's compact tokens,
    D = 32 heads x 128 = 4096 channels (the q/k/v projections each see one such call)."""
    import torch
    import torch.distributed as dist

    import paper_2608_28158_b200 as H
    from workloads import config_forest, make_conv_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fo = config_forest(args.conv_trees)
    C, D, w = fo.n_tokens, 4096, CONV_W
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    t0 = time.perf_counter()
    prev, nxt, cptr, crow = H.harts_conv_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                               plan.row_of_token)
    t_host = time.perf_counter() - t0
    inp = make_conv_inputs(C, D, w, "bf16", 70 + rank, device="cuda")
    idx = {n: torch.as_tensor(np.ascontiguousarray(a)).cuda() for n, a in
           (("prev", prev), ("next", nxt), ("cptr", cptr), ("crow", crow))}
    y, dx, dW = torch.empty_like(inp["x"]), torch.empty_like(inp["x"]), torch.empty_like(inp["W"])
    scratch = torch.empty(H.harts_conv_scratch_bytes(D, w), dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def step(marks=None):
        a, b, c = ev(), ev(), ev()
        a.record(stream)
        H.harts_conv_fwd(inp["x"], inp["W"], idx["prev"], y)
        b.record(stream)
        H.harts_conv_bwd(inp["x"], inp["W"], inp["dy"], idx["next"], idx["cptr"], idx["crow"], dx, dW, scratch)
        c.record(stream)
        if marks is not None:
            marks.append((a, b, c))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    marks = []
    t_begin, t_end = ev(), ev()
    with ClockSampler(local) as clocks:
        for _ in range(args.warmup):
            step()
        barrier()
        h0 = clocks.mark()
        t_begin.record(stream)
        for _ in range(args.steps):
            step(marks)
        t_end.record(stream)
        barrier()
        h1 = clocks.mark()
    ms_step = t_begin.elapsed_time(t_end) / args.steps
    fwd_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in marks)
    bwd_ms = statistics.mean(b.elapsed_time(c) for _, b, c in marks)
    e2e = None
    if not args.no_e2e:
        host = {n: torch.empty(inp[n].shape, dtype=inp[n].dtype, pin_memory=True) for n in ("x", "dy", "W")}
        for n in host:
            host[n].copy_(inp[n])
        out_h = {"y": torch.empty(y.shape, dtype=y.dtype, pin_memory=True),
                 "dx": torch.empty(y.shape, dtype=y.dtype, pin_memory=True), "dW": torch.empty(dW.shape, pin_memory=True)}
        torch.cuda.synchronize()

        def e2e_step():
            for n in host:
                inp[n].copy_(host[n], non_blocking=True)
            step()
            out_h["y"].copy_(y, non_blocking=True)
            out_h["dx"].copy_(dx, non_blocking=True)
            out_h["dW"].copy_(dW, non_blocking=True)

        e2e_step()
        barrier()
        a, b = ev(), ev()
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        e2e = {"ms": a.elapsed_time(b) / n_e2e, "steps": n_e2e,
               "h2d": sum(t.numel() * t.element_size() for t in host.values()),
               "d2h": sum(t.numel() * t.element_size() for t in out_h.values())}
        del host, out_h
    if world > 1:
        ms_step, e2e_ms = max_over_ranks([ms_step, e2e["ms"] if e2e else 0.0], "cuda")
        if e2e:
            e2e["ms"] = e2e_ms
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    unit = C * D * 2
    fwd_bytes, bwd_bytes = 2 * unit + C * 4, 3 * unit + C * 4
    achieved = bwd_bytes / (bwd_ms * 1e-3) / 1e9
    clock = clocks.summary(h0, h1)
    if not clock["samples"]:
        clock = clocks.summary()
    line = {
        "metric": CONV_METRIC, "value": C * world / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "conv", "trees": args.conv_trees, "compact_tokens": C, "D": D, "w": w,
                   "l2": f"inputs larger than L2 ({unit / 2**30:.2f} GiB per tensor)", "host_index_ms": t_host * 1e3},
        "roofline": {"bound": "hbm", "kernel": "conv_bwd_kernel", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": None,
                     "algorithmic_bytes_per_launch": bwd_bytes, "peak_source": peaks["source"],
                     "forward": {"achieved": fwd_bytes / (fwd_ms * 1e-3) / 1e9,
                                 "frac": fwd_bytes / (fwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                     "whole_path": {"roof_ms": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3,
                                    "frac_strict": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms_step}},
        "kernel_ms": {"fwd": fwd_ms, "bwd": bwd_ms},
        "gpu_launches": 3 * args.steps,
        "clocks": clock,
    }
    if e2e:
        line["e2e"] = {"value": C * world / (e2e["ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"], "pinned_host_memory": True}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = conv_oracle_sample()
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------------
# Fourth workload: full attention on compact tokens (Section 3.4, Eqs. 21-22), `--workload attn`
# --------------------------------------------------------------------------------------------------
ATTN_METRIC = "compact-token attention fwd+bwd compact tokens/s"
ATTN_H, ATTN_D = 16, 128


def attn_oracle_sample(small=False, copies=1):
    """The fp64 attention oracle on copies of the cfg0b tree, 2 of the 16 heads."""
    from oracle import attn_oracle
    from workloads import CONFIGS, make_attn_inputs, make_forest
    heads = 1 if small else 2
    fo = make_forest([CONFIGS["cfg0b"]["build"]()[0]] * copies)
    inp = make_attn_inputs(fo.n_tokens, heads, heads, ATTN_D, "bf16", 0)
    q, k, v, dO = (inp[n].double().numpy() for n in ("q", "k", "v", "dO"))
    t0 = time.perf_counter()
    attn_oracle.attn_fwd(fo, q, k, v, ATTN_D ** -0.5)
    attn_oracle.attn_bwd(fo, q, k, v, dO, ATTN_D ** -0.5)
    dt = time.perf_counter() - t0
    if not small and copies == 1 and dt < 8.0:
        return attn_oracle_sample(False, copies=int(min(32, max(2, round(12.0 / dt)))))
    return {"value": fo.n_tokens * heads / ATTN_H / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{copies} x cfg0b tree ({fo.n_tokens} compact tokens), {heads} of {ATTN_H} heads, fwd+bwd, {dt:.1f} s",
            "seconds": dt}


def run_attn_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    vals, secs, last = [], [], None
    for i in range(args.warmup + args.steps):
        last = attn_oracle_sample(small=True)
        if i >= args.warmup:
            vals.append(last["value"])
            secs.append(last["seconds"])
    value = statistics.mean(vals)
    print(json.dumps({
        "impl": "reference", "metric": ATTN_METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(secs) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "attn", "Hq": ATTN_H, "Hkv": ATTN_H, "d": ATTN_D},
        "cpu_baseline": {"kind": last["kind"], "cores": last["cores"], "sample": last["sample"], "value": value,
                         "unit": UNIT},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def run_attn(args):
    """One step = forward + backward of multi-head attention (16 heads, d = 128, bf16) over the compact tokens of
    a forest (default cfg2): every token attends to its ancestors in the tree and to itself."""
    import torch
    import torch.distributed as dist

    import paper_2608_28158_b200 as H
    from workloads import config_forest, make_attn_inputs

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    fo = config_forest(args.attn_trees)
    C, Hq, Hkv, d = fo.n_tokens, ATTN_H, args.attn_kv_heads, ATTN_D
    scale = d ** -0.5
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    t0 = time.perf_counter()
    index = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, plan.row_of_token)
    t_host = time.perf_counter() - t0
    index.upload()
    anc = np.array([int(index.anc_len[index.anc_ptr[p]:index.anc_ptr[p + 1]].sum()) for p in range(index.n_pieces)],
                   dtype=np.int64)
    L = index.piece_len.astype(np.int64)
    pairs = int((L * anc + L * (L + 1) // 2).sum())             # visible (query, key) pairs per head
    inp = make_attn_inputs(C, Hq, Hkv, d, "bf16", 90 + rank, device="cuda")
    o, lse = torch.empty_like(inp["q"]), torch.empty(C, Hq, device="cuda")
    grads = {"dq": torch.empty_like(inp["q"]), "dk": torch.empty_like(inp["k"]), "dv": torch.empty_like(inp["v"])}
    delta = torch.empty(C, Hq, device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731

    def step(marks=None):
        a, b, c = ev(), ev(), ev()
        a.record(stream)
        H.harts_attn_fwd(index, inp["q"], inp["k"], inp["v"], o, lse, scale, dev_status=status)
        b.record(stream)
        H.harts_attn_bwd(index, inp["q"], inp["k"], inp["v"], o, lse, inp["dO"], grads["dq"], grads["dk"], grads["dv"],
                         delta, scale, dev_status=status)
        c.record(stream)
        if marks is not None:
            marks.append((a, b, c))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    marks = []
    t_begin, t_end = ev(), ev()
    with ClockSampler(local) as clocks:
        for _ in range(args.warmup):
            step()
        H.harts_la_check(status)
        barrier()
        h0 = clocks.mark()
        t_begin.record(stream)
        for _ in range(args.steps):
            step(marks)
        t_end.record(stream)
        barrier()
        h1 = clocks.mark()
    H.harts_la_check(status)
    ms_step = t_begin.elapsed_time(t_end) / args.steps
    fwd_ms = statistics.mean(a.elapsed_time(b) for a, b, _ in marks)
    bwd_ms = statistics.mean(b.elapsed_time(c) for _, b, c in marks)
    e2e = None
    if not args.no_e2e:
        host = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in inp.items()}
        for n in host:
            host[n].copy_(inp[n])
        out_h = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in
                 list(grads.items()) + [("o", o)]}
        torch.cuda.synchronize()

        def e2e_step():
            for n in host:
                inp[n].copy_(host[n], non_blocking=True)
            step()
            out_h["o"].copy_(o, non_blocking=True)
            for n in grads:
                out_h[n].copy_(grads[n], non_blocking=True)

        e2e_step()
        barrier()
        a, b = ev(), ev()
        n_e2e = max(1, min(args.steps, args.e2e_steps))
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        e2e = {"ms": a.elapsed_time(b) / n_e2e, "steps": n_e2e,
               "h2d": sum(t.numel() * t.element_size() for t in host.values()),
               "d2h": sum(t.numel() * t.element_size() for t in out_h.values())}
        del host, out_h
    if world > 1:
        ms_step, e2e_ms = max_over_ranks([ms_step, e2e["ms"] if e2e else 0.0], "cuda")
        if e2e:
            e2e["ms"] = e2e_ms
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    peak = peaks["bf16_tflops_sustained"]
    fwd_flops = 4.0 * d * pairs * Hq                     # Q K^T and P V on the visible pairs only
    bwd_flops = 2.5 * fwd_flops                          # five GEMMs (the kernels execute seven: S and dP twice)
    achieved = bwd_flops / (bwd_ms * 1e-3) / 1e12
    clock = clocks.summary(h0, h1)
    if not clock["samples"]:
        clock = clocks.summary()
    line = {
        "metric": ATTN_METRIC, "value": C * world / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "attn", "trees": args.attn_trees, "compact_tokens": C, "Hq": Hq, "Hkv": Hkv, "d": d,
                   "pieces": index.n_pieces, "visible_pairs_per_head": pairs,
                   "mean_context": pairs / C, "l2": "flushed by the step itself: q, k, v, dO, o and the gradients "
                   f"({9 * C * Hq * d * 2 / 2**30:.2f} GiB) exceed L2", "host_index_ms": t_host * 1e3},
        "roofline": {"bound": "tensor", "kernel": "backward call (attn_dq_kernel + attn_dkv_kernel)",
                     "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak, "traffic": None,
                     "algorithmic_flops_per_launch": bwd_flops, "executed_flops_per_launch": bwd_flops * 7 / 5,
                     "peak_source": peaks["source"] + " (sustained bf16 GEMM)",
                     "forward": {"achieved": fwd_flops / (fwd_ms * 1e-3) / 1e12,
                                 "frac": fwd_flops / (fwd_ms * 1e-3) / 1e12 / peak},
                     "whole_path": {"roof_ms": (fwd_flops + bwd_flops) / (peak * 1e12) * 1e3,
                                    "frac_strict": (fwd_flops + bwd_flops) / (peak * 1e12) * 1e3 / ms_step}},
        "kernel_ms": {"fwd": fwd_ms, "bwd": bwd_ms},
        "gpu_launches": 4 * args.steps,
        "clocks": clock,
    }
    if e2e:
        line["e2e"] = {"value": C * world / (e2e["ms"] * 1e-3), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"],
                       "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"], "pinned_host_memory": True}
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = attn_oracle_sample()
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--fma", action="store_true", help="force the fp32-FMA kernels")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-trajwise", action="store_true")
    ap.add_argument("--logp-rows", type=int, default=LOGP_ROWS, help="compact-row capacity of the logp workload")
    ap.add_argument("--conv-trees", default="cfg3", help="forest of the conv workload (cfg2: a small case for captures)")
    ap.add_argument("--attn-trees", default="cfg2", help="forest of the attn workload (cfg1: a small case for captures)")
    ap.add_argument("--attn-kv-heads", type=int, default=ATTN_H, help="kv heads of the attn workload (16 = MHA)")
    ap.add_argument("--per-config", action="store_true", help="also print a table over all configurations to stderr")
    args = ap.parse_args()
    if args.workload == "logp":
        (run_logp_reference if args.impl == "reference" else run_logp)(args)
    elif args.workload == "conv":
        (run_conv_reference if args.impl == "reference" else run_conv)(args)
    elif args.workload == "attn":
        (run_attn_reference if args.impl == "reference" else run_attn)(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
