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

Timing: W warm-up steps, then blocks of exactly K steps each, every block bracketed by a barrier and a device
synchronisation and timed with CUDA events on the launching stream; when K steps take less than about two seconds,
several blocks are run back to back and the MEDIAN block gives ``ms_per_step`` (the per-block times and clock medians
are kept under ``timing``).  With ``--gpus N`` and no torchrun environment the script starts its N ranks itself.
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
# Scaffold shared by every workload: ranks, timed blocks, end-to-end steps, JSON line
# --------------------------------------------------------------------------------------------------
class Ranks:
    """This process' place in the job (torchrun's environment, or a single rank) and the job-wide barrier."""

    def __init__(self):
        import torch
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        torch.cuda.set_device(self.local)
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))

    def barrier(self):
        import torch
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    def close(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


def max_over_ranks(values, device):
    """Element-wise maximum of a few per-rank timings over all ranks (identity when not distributed)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def plan_blocks(steps, est_ms_per_step, target_ms=2000.0, most=9):
    """How many blocks of `steps` steps to time: one when a block already lasts `target_ms`, else enough blocks to
    fill it (an odd number, so that the median is a measured block), at most `most`."""
    block = max(steps * est_ms_per_step, 1e-3)
    if block >= target_ms:
        return 1
    n = min(most, int(-(-target_ms // block)))
    return n if n % 2 == 1 else min(most, n + 1)


def time_blocks(work, args, ranks):
    """Warm-up, then the timed blocks.  Returns ms_per_step (median block, each block the max over ranks), the
    per-launch event pairs of every timed step, and the clocks sampled during the blocks."""
    import torch
    stream = torch.cuda.current_stream()
    ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
    marks, block_ms, block_host = [], [], []
    with ClockSampler(ranks.local) as clocks:      # started before the warm-up so that it is sampling by then
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(args.warmup):
            work.step(None)
        b.record(stream)
        ranks.barrier()
        work.check()
        est = max_over_ranks([a.elapsed_time(b) / max(1, args.warmup)], "cuda")[0]
        n_blocks = args.blocks if args.blocks > 0 else plan_blocks(args.steps, est)
        for _ in range(n_blocks):
            ranks.barrier()
            h0 = clocks.mark()
            a, b = ev(), ev()
            a.record(stream)
            for _ in range(args.steps):
                work.step(marks)
            b.record(stream)
            ranks.barrier()
            block_host.append((h0, clocks.mark()))
            block_ms.append(a.elapsed_time(b))
    work.check()
    block_ms = max_over_ranks(block_ms, "cuda")
    clock = clocks.summary(block_host[0][0], block_host[-1][1])
    if not clock["samples"]:
        clock = clocks.summary()
        clock["note"] = "timed region shorter than the sampling period: samples cover warm-up + timed region"
    per_block = [clocks.summary(h0, h1)["sm_mhz"] for h0, h1 in block_host]
    kernel_ms = {}
    for name, a, b in marks:
        kernel_ms.setdefault(name, []).append(a.elapsed_time(b))
    n_steps = n_blocks * args.steps
    return {"ms_per_step": statistics.median(block_ms) / args.steps,
            "kernel_ms": {n: sum(v) / n_steps for n, v in kernel_ms.items()},
            "clocks": clock,
            "timing": {"blocks": n_blocks, "steps_per_block": args.steps,
                       "block_ms_per_step": [x / args.steps for x in block_ms], "block_sm_mhz": per_block,
                       "ms_per_step": "median block"}}


def host_copies(tensors):
    """Pinned host twins of a dict of device tensors, filled with their contents."""
    import torch
    host = {n: torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for n, x in tensors.items()}
    for n, x in tensors.items():
        host[n].copy_(x)
    torch.cuda.synchronize()
    return host


def time_e2e(work, dev_in, dev_out, n_steps, ranks):
    """End-to-end steps on one stream: every step copies all inputs from pinned host memory, runs the path and copies
    all results back, inside the timed region."""
    import torch
    stream = torch.cuda.current_stream()
    host_in, host_out = host_copies(dev_in), host_copies(dev_out)

    def e2e_step():
        for n, x in dev_in.items():
            x.copy_(host_in[n], non_blocking=True)
        work.step(None)
        for n, x in dev_out.items():
            host_out[n].copy_(x, non_blocking=True)

    e2e_step()
    ranks.barrier()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(n_steps):
        e2e_step()
    b.record(stream)
    ranks.barrier()
    nbytes = lambda d: sum(t.numel() * t.element_size() for t in d.values())  # noqa: E731
    return {"ms": a.elapsed_time(b) / n_steps, "steps": n_steps, "h2d": nbytes(host_in), "d2h": nbytes(host_out)}


# ---- measured DRAM traffic of the dominant kernels -----------------------------------------------------------------
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "traffic.json")


def measured_traffic(kernel):
    """DRAM bytes per unit of `kernel` from the last profiler capture, or None when there is none or when a source
    file of the kernel has changed since (the record carries the sources' hash; see paper_2608_28158_b200/traffic.py)."""
    from paper_2608_28158_b200 import traffic
    rec = traffic.load(TRAFFIC_FILE).get(kernel)
    if not rec or rec.get("source_sha256") != traffic.source_hash(rec.get("sources", [])):
        return None
    return rec


def hbm_roofline(kernel, bytes_per_launch, ms, peaks, traffic_per_launch, **extra):
    achieved = bytes_per_launch / (ms * 1e-3) / 1e9
    out = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
           "frac": achieved / peaks["hbm_gbs"], "traffic": traffic_per_launch,
           "algorithmic_bytes_per_launch": bytes_per_launch, "peak_source": peaks["source"]}
    out.update(extra)
    return out
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


class LaWorkload:
    """The hot path: one step = every forward round, every backward round and the replay-gradient fold of a
    configuration (default cfg3)."""
    metric, unit = METRIC, UNIT

    def __init__(self, args, ranks):
        import torch
        import paper_2608_28158_b200 as H
        from workloads import CONFIGS, config_forest, make_inputs
        self.H, self.args, self.ranks = H, args, ranks
        self.cfg = cfg = CONFIGS[args.workload]
        self.fo = fo = config_forest(args.workload)
        t_plans = []
        for _ in range(3):                                 # host planning time: median of three calls
            t0 = time.perf_counter()
            plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, cfg["chunk"])
            t_plans.append(time.perf_counter() - t0)
        self.t_plan = statistics.median(t_plans)
        self.plan = plan.upload()
        Hh, dk, dv = cfg["H"], cfg["dk"], cfg["dv"]
        # every rank draws its own tensors (independent batches of the same shape)
        self.inp = inp = make_inputs(plan.C, Hh, dk, dv, cfg["dtype"], cfg["seed"] + 100 * ranks.rank, device="cuda")
        self.flags = (H.HARTS_FLAG_FMA_KERNELS if args.fma else 0) | (H.HARTS_FLAG_ROUND_LAUNCHES if args.round_launches else 0)
        self.ws = H.Workspace(plan, Hh, dk, dv, inp["q"].dtype, self.flags)
        self.out = {"o": torch.empty_like(inp["v"]), "dq": torch.empty_like(inp["q"]), "dk": torch.empty_like(inp["k"]),
                    "dv": torch.empty_like(inp["v"]), "dg": torch.empty_like(inp["g"])}
        self.units = plan.C
        self.stream = torch.cuda.current_stream()

    def step(self, marks):
        import torch
        H, plan, inp, out, ws, stream = self.H, self.plan, self.inp, self.out, self.ws, self.stream
        ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
        K = plan.n_rounds

        def timed(name, call):
            if marks is None:
                call()
                return
            a, b = ev(), ev()
            a.record(stream)
            call()
            b.record(stream)
            marks.append((name, a, b))

        if self.one_launch()[0]:
            # round 0 = all rounds; on a problem this small the library runs them in one launch per pass, and
            # the backward call includes the replay-gradient fold
            timed("fwd", lambda: H.harts_la_fwd(plan, 0, inp["q"], inp["k"], inp["v"], inp["g"], out["o"], ws.slots,
                                               ws.chunk_states, self.flags, ws.dev_status))
            timed("bwd", lambda: H.harts_la_bwd(plan, 0, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"], out["dq"],
                                               out["dk"], out["dv"], out["dg"], ws.chunk_states, ws.scratch, self.flags,
                                               ws.dev_status))
            return
        # one call per round (what round 0 does on a problem of this size), so that every round's launch is timed alone
        for r in range(1, K + 1):
            timed("fwd", lambda: H.harts_la_fwd(plan, r, inp["q"], inp["k"], inp["v"], inp["g"], out["o"], ws.slots,
                                               ws.chunk_states, self.flags, ws.dev_status))
        for r in range(K, 0, -1):
            timed("bwd", lambda: H.harts_la_bwd_seqs(plan.tables, int(plan.round_seq_ptr[r - 1]),
                                                    int(plan.round_seq_ptr[r]), inp["q"], inp["k"], inp["v"], inp["g"],
                                                    inp["dO"], out["dq"], out["dk"], out["dv"], out["dg"],
                                                    ws.chunk_states, ws.scratch, self.flags, ws.dev_status))
        timed("fold", lambda: H.harts_la_bwd_finish(plan.tables, out["dk"], out["dv"], out["dg"], ws.scratch))

    def one_launch(self):
        """(forward, backward): True where the library's all-rounds call runs as one launch per pass -- bf16 d = 128
        kernels, more than one round, and at most 8 (sequence, head) items per resident CTA (two CTAs per SM in the
        forward, one in the backward)."""
        import torch
        sms = torch.cuda.get_device_properties(0).multi_processor_count
        tc = self.cfg["dk"] == 128 and not self.args.fma and self.inp["q"].element_size() == 2
        ok = tc and 1 < self.plan.n_rounds <= 32 and not self.args.round_launches
        items = self.plan.n_seq * self.cfg["H"]
        return ok and items <= 16 * sms, ok and items <= 8 * sms

    def check(self):
        self.H.harts_la_check(self.ws.dev_status)

    def e2e(self, n_steps):
        """Through host buffers, pipelined: the copies of neighbouring steps overlap the kernels (three streams, two
        device buffer sets); every step still moves all of its inputs in and all of its results out."""
        import torch
        H, plan, ws, inp, out, ranks = self.H, self.plan, self.ws, self.inp, self.out, self.ranks
        host_in, host_out = host_copies(inp), host_copies(out)
        stream = torch.cuda.current_stream()
        ev = lambda: torch.cuda.Event(enable_timing=True)  # noqa: E731
        H.run_fwd_bwd_host(plan, ws, host_in, inp, out, host_out)       # warm-up; then the unpipelined reference
        ranks.barrier()
        a, b = ev(), ev()
        a.record(stream)
        H.run_fwd_bwd_host(plan, ws, host_in, inp, out, host_out)
        b.record(stream)
        ranks.barrier()
        serial_ms = a.elapsed_time(b)
        pipe = H.HostPipeline(plan, ws, inp, out)
        pipe.step(host_in, host_out)                                    # warm-up of the streams
        pipe.finish()
        ranks.barrier()
        a, b = ev(), ev()
        a.record(pipe.s_in)
        for _ in range(n_steps):
            pipe.step(host_in, host_out)
        b.record(pipe.s_out)
        pipe.finish()
        ranks.barrier()
        nbytes = lambda d: sum(t.numel() * t.element_size() for t in d.values())  # noqa: E731
        return {"ms": a.elapsed_time(b) / n_steps, "steps": n_steps, "h2d": nbytes(host_in), "d2h": nbytes(host_out),
                "extra": {"overlap": "copies of neighbouring steps overlap the kernels (3 streams, 2 device buffer sets)",
                          "unpipelined_value": plan.C * ranks.world / (serial_ms * 1e-3)}}

    def describe(self, ms_step, kernel_ms, peaks):
        plan, cfg, args = self.plan, self.cfg, self.args
        Hh, dk, dv = cfg["H"], cfg["dk"], cfg["dv"]
        elem = self.inp["q"].element_size()
        K = plan.n_rounds
        th = plan.C * Hh                                  # token-heads per rank and step
        # algorithmic (compulsory) bytes per token-head: fwd reads q,k,v,g and writes o; bwd reads q,k,v,dO,g and
        # writes dq,dk,dv,dg
        fwd_bytes = th * ((2 * dk + 2 * dv) * elem + 4)
        bwd_bytes = th * ((4 * dk + 3 * dv) * elem + 8)
        flops_fwd = th * (2 * 64 * dk + 2 * 64 * dv + 4 * dk * dv)
        flops_bwd = th * (5 * 2 * 64 * (dk + dv) // 2 + 4 * 2 * dk * dv)
        in_bytes = sum(x.numel() * x.element_size() for x in self.inp.values())
        tc = dk == 128 and not args.fma and elem == 2
        rec = measured_traffic("tc_bwd_kernel") if tc else None
        traffic = rec["dram_bytes_per_unit"] * th / K if rec else None
        t_bytes = (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9)
        t_flops = (flops_fwd + flops_bwd) / (peaks["bf16_tflops_sustained"] * 1e12)
        # method traffic on top of the compulsory bytes: replayed rows (k, v, g read in both passes, gradient
        # contributions written and folded), state hand-offs (initial state read + its gradient written, slot written
        # + consumers' gradients read), chunk states (written by the forward, read by the backward, 2 B per element)
        n_side = int((plan.seq_init_slot >= 0).sum())
        method_bytes = (fwd_bytes + bwd_bytes + plan.R * Hh * (6 * dk * elem + 12)
                        + (n_side + plan.n_slots) * Hh * dk * dv * 4 * 2 + plan.n_chunks * Hh * dk * dv * 2 * 2)
        roof = hbm_roofline(
            "backward packed call (all rounds)", bwd_bytes / K, kernel_ms["bwd"] / K, peaks, traffic,
            traffic_note=(f"bytes per launch (mean over the rounds): {rec['dram_bytes_per_unit']:.0f} B per token-head "
                          f"from the ncu capture on {rec['workload']} at commit {rec['commit']}, scaled by token-heads"
                          if rec else "no capture of the current kernel sources on record"),
            forward={"achieved": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9,
                     "frac": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
            whole_path={"roof_ms": max(t_bytes, t_flops) * 1e3, "frac_strict": max(t_bytes, t_flops) * 1e3 / ms_step,
                        "frac_strict_nominal": max((fwd_bytes + bwd_bytes) / 8e12,
                                                   (flops_fwd + flops_bwd) / 2.25e15) * 1e3 / ms_step,
                        "frac_method": max(method_bytes / (peaks["hbm_gbs"] * 1e9), t_flops) * 1e3 / ms_step})
        return {
            "dtype": cfg["dtype"] if cfg["dtype"] != "fp32" else "f32",
            "config": {"workload": args.workload, "H": Hh, "dk": dk, "dv": dv, "chunk": cfg["chunk"],
                       "compact_tokens": plan.C, "replay_rows": plan.R, "rounds": plan.n_rounds,
                       "sequences": plan.n_seq, "slots": plan.n_slots, "chunks": plan.n_chunks,
                       "l2": f"inputs larger than L2 ({in_bytes / 2**30:.2f} GiB read per step)"
                             if in_bytes > 2 * L2_BYTES else "inputs smaller than L2: no flush (small workload)",
                       "kernels": "fma" if args.fma or cfg["dtype"] == "fp32" else "default",
                       "plan_ms": self.t_plan * 1e3},
            "roofline": roof,
            "gpu_launches_per_step": self.launches_per_step()}

    def launches_per_step(self):
        """Kernels per step: one launch per round and pass (each backward round preceded by the hand-off reduction when
        the plan exports boundaries) plus the replay-gradient fold -- or, on problems with few items per CTA, one
        launch for all forward rounds and one for all backward rounds."""
        plan, K = self.plan, self.plan.n_rounds
        one_fwd, one_bwd = self.one_launch()
        fwd = 1 if one_fwd else K
        bwd = 1 if one_bwd else K + (K if plan.n_slots else 0)
        return fwd + bwd + (1 if plan.n_rg_rows else 0)

    def extras(self, ms_step):
        """The same kernels, trajectory-wise (the conventional baseline of Section 5); one GPU only."""
        import torch
        if self.ranks.world > 1 or self.args.no_trajwise:
            return {}
        rows = torch.as_tensor(self.plan.row_of_token.astype(np.int64), device="cuda")
        canon = {n: x[rows] for n, x in self.inp.items()}      # the expansion wants canonical order
        t_ms, t_rows = trajectory_wise_ms(self.H, self.fo, self.cfg, canon, self.flags)
        return {"trajectory_wise": {
            "ms": t_ms, "rows": t_rows, "rows_ratio": t_rows / self.plan.C, "speedup": t_ms / ms_step,
            "speedup_with_plan": t_ms / (ms_step + self.t_plan * 1e3),
            "paper_context": "4.81-4.87x F/B/Grad on a whole hybrid MoE model, 8x H20-3e (Table 4)"}}

    def cpu_baseline(self):
        return oracle_sample(self.args.workload)

    def reference_sample(self, hint):
        return oracle_sample(self.args.workload, seconds_hint=hint)
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


class LogpWorkload:
    """One step = forward (row max / sum-exp over V, lambda for every position) + backward (dz for every compact row)."""
    metric, unit = LOGP_METRIC, LOGP_UNIT

    def __init__(self, args, ranks):
        import torch
        import paper_2608_28158_b200 as H
        from workloads import make_logits, make_logp_grad
        self.H, self.args, self.ranks = H, args, ranks
        fo, self.trees = logp_forest(ranks.rank, args.logp_rows)
        self.C, self.V = C, V = fo.n_tokens, LOGP_V
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
        data = make_logits(C, V, "bf16", 50 + ranks.rank, device="cuda")
        t0 = time.perf_counter()
        m, y, _ = H.harts_logp_positions(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                         data["token_id"].cpu().numpy(), plan.row_of_token)
        ptr, pos = H.harts_logp_csr(C, m)
        self.t_host = time.perf_counter() - t0
        self.P = P = len(m)
        self.z = data["z"]
        self.dev = {"m": torch.as_tensor(m).cuda(), "y": torch.as_tensor(y).cuda(), "ptr": torch.as_tensor(ptr).cuda(),
                    "pos": torch.as_tensor(pos).cuda(), "g": make_logp_grad(P, 50 + ranks.rank, device="cuda", keep=1.0)}
        self.lse, self.lam, self.dz = torch.empty(C, device="cuda"), torch.empty(P, device="cuda"), torch.empty_like(self.z)
        self.status = torch.zeros(2, dtype=torch.int32, device="cuda")
        self.units = C
        self.stream = torch.cuda.current_stream()

    def step(self, marks):
        import torch
        H, dev = self.H, self.dev
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record(self.stream)
        H.harts_logp_fwd(self.z, dev["m"], dev["y"], self.lse, self.lam, dev_status=self.status)
        b.record(self.stream)
        H.harts_logp_bwd(self.z, dev["y"], dev["ptr"], dev["pos"], self.lse, dev["g"], self.dz, dev_status=self.status)
        c.record(self.stream)
        if marks is not None:
            marks += [("fwd", a, b), ("bwd", b, c)]

    def check(self):
        self.H.harts_la_check(self.status)

    def e2e(self, n_steps):
        dev_in = dict(self.dev, z=self.z)
        return time_e2e(self, dev_in, {"lam": self.lam, "dz": self.dz}, n_steps, self.ranks)

    def describe(self, ms_step, kernel_ms, peaks):
        C, V, P = self.C, self.V, self.P
        row_bytes = V * self.z.element_size()
        fwd_bytes = C * row_bytes + P * 12 + C * 4              # z once; m, y read and lambda written; lse written
        bwd_bytes = 2 * C * row_bytes + P * 12 + C * 12         # z read, dz written; y, g, row_pos; lse, row_pos_ptr
        roof_ms = (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3
        return {"dtype": "bf16",
                "config": {"workload": "logp", "V": V, "compact_rows": C, "positions": P, "trees": self.trees,
                           "action_mask": "every position selected (no idle rows)",
                           "l2": f"inputs larger than L2 ({C * row_bytes / 2**30:.2f} GiB of logits)",
                           "host_index_ms": self.t_host * 1e3},
                "roofline": hbm_roofline("dz_kernel (backward)", bwd_bytes, kernel_ms["bwd"], peaks, None,
                                         forward={"achieved": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9,
                                                  "frac": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                                         whole_path={"roof_ms": roof_ms, "frac_strict": roof_ms / ms_step}),
                "gpu_launches_per_step": 3}

    def extras(self, ms_step):
        return {}

    def cpu_baseline(self):
        return logp_oracle_sample()
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


class ConvWorkload:
    """One step = forward + backward (dx, dW) of the width-4 depthwise convolution over cfg3's compact tokens,
    D = 32 heads x 128 = 4096 channels (the q/k/v projections each see one such call)."""
    metric, unit = CONV_METRIC, UNIT

    def __init__(self, args, ranks):
        import torch
        import paper_2608_28158_b200 as H
        from workloads import config_forest, make_conv_inputs
        self.H, self.args, self.ranks = H, args, ranks
        fo = config_forest(args.conv_trees)
        self.C, self.D, self.w = C, D, w = fo.n_tokens, 4096, CONV_W
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
        t0 = time.perf_counter()
        prev, nxt, cptr, crow = H.harts_conv_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                                   plan.row_of_token)
        self.t_host = time.perf_counter() - t0
        self.inp = make_conv_inputs(C, D, w, "bf16", 70 + ranks.rank, device="cuda")
        self.idx = {n: torch.as_tensor(np.ascontiguousarray(a)).cuda() for n, a in
                    (("prev", prev), ("next", nxt), ("cptr", cptr), ("crow", crow))}
        self.y, self.dx = torch.empty_like(self.inp["x"]), torch.empty_like(self.inp["x"])
        self.dW = torch.empty_like(self.inp["W"])
        self.scratch = torch.empty(H.harts_conv_scratch_bytes(D, w), dtype=torch.uint8, device="cuda")
        self.units = C
        self.stream = torch.cuda.current_stream()

    def step(self, marks):
        import torch
        H, inp, idx = self.H, self.inp, self.idx
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record(self.stream)
        H.harts_conv_fwd(inp["x"], inp["W"], idx["prev"], self.y)
        b.record(self.stream)
        H.harts_conv_bwd(inp["x"], inp["W"], inp["dy"], idx["next"], idx["cptr"], idx["crow"], self.dx, self.dW,
                         self.scratch)
        c.record(self.stream)
        if marks is not None:
            marks += [("fwd", a, b), ("bwd", b, c)]

    def check(self):
        pass

    def e2e(self, n_steps):
        dev_in = {n: self.inp[n] for n in ("x", "dy", "W")}
        return time_e2e(self, dev_in, {"y": self.y, "dx": self.dx, "dW": self.dW}, n_steps, self.ranks)

    def describe(self, ms_step, kernel_ms, peaks):
        C, D = self.C, self.D
        unit = C * D * 2
        fwd_bytes, bwd_bytes = 2 * unit + C * 4, 3 * unit + C * 4
        roof_ms = (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3
        return {"dtype": "bf16",
                "config": {"workload": "conv", "trees": self.args.conv_trees, "compact_tokens": C, "D": D, "w": self.w,
                           "l2": f"inputs larger than L2 ({unit / 2**30:.2f} GiB per tensor)",
                           "host_index_ms": self.t_host * 1e3},
                "roofline": hbm_roofline("conv_bwd_kernel", bwd_bytes, kernel_ms["bwd"], peaks, None,
                                         forward={"achieved": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9,
                                                  "frac": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                                         whole_path={"roof_ms": roof_ms, "frac_strict": roof_ms / ms_step}),
                "gpu_launches_per_step": 3}

    def extras(self, ms_step):
        return {}

    def cpu_baseline(self):
        return conv_oracle_sample()
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


class AttnWorkload:
    """One step = forward + backward of multi-head attention (16 heads, d = 128, bf16) over the compact tokens of
    a forest (default cfg2): every token attends to its ancestors in the tree and to itself."""
    metric, unit = ATTN_METRIC, UNIT

    def __init__(self, args, ranks):
        import torch
        import paper_2608_28158_b200 as H
        from workloads import config_forest, make_attn_inputs
        self.H, self.args, self.ranks = H, args, ranks
        fo = config_forest(args.attn_trees)
        self.C, self.Hq, self.Hkv, self.d = C, Hq, Hkv, d = fo.n_tokens, ATTN_H, args.attn_kv_heads, ATTN_D
        self.scale = d ** -0.5
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
        t0 = time.perf_counter()
        self.index = index = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len,
                                                plan.row_of_token)
        self.t_host = time.perf_counter() - t0
        index.upload()
        anc = np.array([int(index.anc_len[index.anc_ptr[p]:index.anc_ptr[p + 1]].sum()) for p in range(index.n_pieces)],
                       dtype=np.int64)
        L = index.piece_len.astype(np.int64)
        self.pairs = int((L * anc + L * (L + 1) // 2).sum())             # visible (query, key) pairs per head
        self.inp = inp = make_attn_inputs(C, Hq, Hkv, d, "bf16", 90 + ranks.rank, device="cuda")
        self.o, self.lse = torch.empty_like(inp["q"]), torch.empty(C, Hq, device="cuda")
        self.grads = {"dq": torch.empty_like(inp["q"]), "dk": torch.empty_like(inp["k"]), "dv": torch.empty_like(inp["v"])}
        self.delta = torch.empty(C, Hq, device="cuda")
        self.status = torch.zeros(4, dtype=torch.int32, device="cuda")
        self.units = C
        self.stream = torch.cuda.current_stream()

    def step(self, marks):
        import torch
        H, inp, g = self.H, self.inp, self.grads
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record(self.stream)
        H.harts_attn_fwd(self.index, inp["q"], inp["k"], inp["v"], self.o, self.lse, self.scale, dev_status=self.status)
        b.record(self.stream)
        H.harts_attn_bwd(self.index, inp["q"], inp["k"], inp["v"], self.o, self.lse, inp["dO"], g["dq"], g["dk"], g["dv"],
                         self.delta, self.scale, dev_status=self.status)
        c.record(self.stream)
        if marks is not None:
            marks += [("fwd", a, b), ("bwd", b, c)]

    def check(self):
        self.H.harts_la_check(self.status)

    def e2e(self, n_steps):
        return time_e2e(self, dict(self.inp), dict(self.grads, o=self.o), n_steps, self.ranks)

    def describe(self, ms_step, kernel_ms, peaks):
        C, Hq, d, pairs = self.C, self.Hq, self.d, self.pairs
        peak = peaks["bf16_tflops_sustained"]
        fwd_flops = 4.0 * d * pairs * Hq                     # Q K^T and P V on the visible pairs only
        bwd_flops = 2.5 * fwd_flops                          # five GEMMs (the kernels execute seven: S and dP twice)
        achieved = bwd_flops / (kernel_ms["bwd"] * 1e-3) / 1e12
        roof_ms = (fwd_flops + bwd_flops) / (peak * 1e12) * 1e3
        return {"dtype": "bf16",
                "config": {"workload": "attn", "trees": self.args.attn_trees, "compact_tokens": C, "Hq": Hq,
                           "Hkv": self.Hkv, "d": d, "pieces": self.index.n_pieces, "visible_pairs_per_head": pairs,
                           "mean_context": pairs / C,
                           "l2": "flushed by the step itself: q, k, v, dO, o and the gradients "
                                 f"({9 * C * Hq * d * 2 / 2**30:.2f} GiB) exceed L2",
                           "host_index_ms": self.t_host * 1e3},
                "roofline": {"bound": "tensor", "kernel": "backward call (attn_dq_kernel + attn_dkv_kernel)",
                             "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                             "traffic": None, "algorithmic_flops_per_launch": bwd_flops,
                             "executed_flops_per_launch": bwd_flops * 7 / 5,
                             "peak_source": peaks["source"] + " (sustained bf16 GEMM)",
                             "forward": {"achieved": fwd_flops / (kernel_ms["fwd"] * 1e-3) / 1e12,
                                         "frac": fwd_flops / (kernel_ms["fwd"] * 1e-3) / 1e12 / peak},
                             "whole_path": {"roof_ms": roof_ms, "frac_strict": roof_ms / ms_step}},
                "gpu_launches_per_step": 4}

    def extras(self, ms_step):
        return {}

    def cpu_baseline(self):
        return attn_oracle_sample()
# --------------------------------------------------------------------------------------------------
# Fifth workload: the per-channel-decay recurrence (Diag(gamma) term of Eq. 1), `--workload gk`
# --------------------------------------------------------------------------------------------------
GK_METRIC = "tree-packed per-channel-decay linear-attn fwd+bwd compact tokens/s"
GK_CONFIG = "cfg2"


def gk_oracle_sample(small=False):
    """The fp64 per-channel oracle on whole trees of the workload's forest, one head."""
    from oracle import gk_oracle
    from workloads import CONFIGS, config_forest, make_gk, make_inputs
    cfg = CONFIGS[GK_CONFIG]
    fo = config_forest("cfg0b") if small else config_forest(GK_CONFIG).subset([0])
    d = cfg["dk"]
    inp = make_inputs(fo.n_tokens, 1, d, d, "bf16", 0)
    gk = make_gk(fo.n_tokens, 1, d, 0)
    t0 = time.perf_counter()
    res = gk_oracle.forest_eval(fo, inp["q"], inp["k"], inp["v"], gk, inp["dO"])
    dt = time.perf_counter() - t0
    return {"value": fo.n_tokens / cfg["H"] / dt, "unit": UNIT, "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{'cfg0b tree' if small else GK_CONFIG + ' tree 0'}: {fo.n_tokens} compact / {res['S']} "
                      f"trajectory-wise tokens, 1 of {cfg['H']} heads, fwd+bwd, {dt:.1f} s", "seconds": dt}


class GkWorkload:
    """One step = every forward round and every backward round (with the replay-gradient fold) of the per-channel-
    decay calls on cfg2's forest (16 heads, d = 128, bf16)."""
    metric, unit = GK_METRIC, UNIT

    def __init__(self, args, ranks):
        import torch
        import paper_2608_28158_b200 as H
        from workloads import CONFIGS, config_forest, make_gk, make_inputs
        self.H, self.args, self.ranks = H, args, ranks
        self.trees = trees = getattr(args, "gk_trees", GK_CONFIG)
        self.cfg = cfg = CONFIGS[trees]
        fo = config_forest(trees)
        self.plan = plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).upload()
        Hh, d = cfg["H"], cfg["dk"]
        self.inp = inp = make_inputs(plan.C, Hh, d, d, "bf16", 60 + ranks.rank, device="cuda")
        inp["g"] = make_gk(plan.C, Hh, d, 60 + ranks.rank, device="cuda")
        cs, sc = H.harts_la_gk_workspace_bytes(plan.tables, Hh, d, d, H.HARTS_BF16)
        self.slots = torch.empty(max(plan.n_slots, 1) * Hh * d * d, device="cuda")
        self.cs = torch.empty(cs, dtype=torch.uint8, device="cuda")
        self.scratch = torch.empty(sc, dtype=torch.uint8, device="cuda")
        self.status = torch.zeros(4, dtype=torch.int32, device="cuda")
        self.out = {"o": torch.empty_like(inp["v"]), "dq": torch.empty_like(inp["q"]), "dk": torch.empty_like(inp["k"]),
                    "dv": torch.empty_like(inp["v"]), "dg": torch.empty_like(inp["g"])}
        self.units = plan.C
        self.stream = torch.cuda.current_stream()
        self.flags = H.HARTS_FLAG_ROUND_LAUNCHES if getattr(args, "round_launches", False) else 0

    def step(self, marks):
        import torch
        H, plan, inp, out = self.H, self.plan, self.inp, self.out
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        a.record(self.stream)
        H.harts_la_gk_fwd(plan, 0, inp["q"], inp["k"], inp["v"], inp["g"], out["o"], self.slots, self.cs,
                          flags=self.flags, dev_status=self.status)
        b.record(self.stream)
        H.harts_la_gk_bwd(plan, 0, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"], out["dq"], out["dk"], out["dv"],
                          out["dg"], self.cs, self.scratch, flags=self.flags, dev_status=self.status)
        c.record(self.stream)
        if marks is not None:
            marks += [("fwd", a, b), ("bwd", b, c)]

    def check(self):
        self.H.harts_la_check(self.status)

    def e2e(self, n_steps):
        return time_e2e(self, dict(self.inp), dict(self.out), n_steps, self.ranks)

    def describe(self, ms_step, kernel_ms, peaks):
        plan, cfg = self.plan, self.cfg
        Hh, d = cfg["H"], cfg["dk"]
        th = plan.C * Hh
        # compulsory bytes per token-head (bf16 tensors, fp32 per-channel gate and its gradient): forward reads q, k, v, g
        # and writes o; backward reads q, k, v, dO, g and writes dq, dk, dv, dg.  The chunk states (bf16, written by the
        # forward and read by the backward) come on top and are not counted.
        fwd_bytes = th * (3 * d * 2 + 4 * d + 2 * d)
        bwd_bytes = th * (4 * d * 2 + 4 * d + 3 * d * 2 + 4 * d)
        K = plan.n_rounds
        # beside the HBM figure: the time the special-function unit needs for the exponentials of the decayed operands
        # (anchored q / k tiles, q~ / k~, the factors applied to the block products: about 135 k per chunk-head in both
        # passes together when every chunk is mild, 16 per clock and SM)
        import torch
        one_launch = (not self.flags and 1 < K <= 32 and
                      plan.n_seq * Hh <= 8 * torch.cuda.get_device_properties(0).multi_processor_count)
        chunk_heads = plan.n_chunks * Hh
        sfu_ms = chunk_heads * 135e3 / (148 * 16 * 1.965e9) * 1e3
        roof = hbm_roofline("gk_mma_bwd_kernel (all rounds)", bwd_bytes / K, kernel_ms["bwd"] / K, peaks, None,
                            forward={"achieved": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9,
                                     "frac": fwd_bytes / (kernel_ms["fwd"] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                            whole_path={"roof_ms": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3,
                                        "frac_strict": (fwd_bytes + bwd_bytes) / (peaks["hbm_gbs"] * 1e9) * 1e3 / ms_step,
                                        "exponential_unit_ms": sfu_ms, "frac_exponential_unit": sfu_ms / ms_step})
        return {"dtype": "bf16",
                "config": {"workload": "gk", "trees": self.trees, "H": Hh, "dk": d, "dv": d, "chunk": 64,
                           "compact_tokens": plan.C, "rounds": K, "sequences": plan.n_seq, "chunks": plan.n_chunks,
                           "inputs": "bf16 q, k, v, dO; fp32 per-channel log-decay; dense products on the tensor cores "
                                     "(mma.sync, bf16 operands, fp32 accumulation), in-block pair sums in fp32 on the CUDA cores",
                           "l2": "inputs larger than L2"},
                "roofline": roof,
                # all rounds in one launch per pass on a problem with at most 8 items per SM (the library's rule), else one
                # launch per round and pass with the hand-off reduction before every backward round; plus the fold
                "gpu_launches_per_step": (2 if one_launch else 2 * K + (K if plan.n_slots else 0)) + (1 if plan.n_rg_rows else 0)}

    def extras(self, ms_step):
        return {}

    def cpu_baseline(self):
        return gk_oracle_sample()


# --------------------------------------------------------------------------------------------------
# Driver: one workload -> one JSON line
# --------------------------------------------------------------------------------------------------
WORKLOADS = {"logp": LogpWorkload, "conv": ConvWorkload, "attn": AttnWorkload, "gk": GkWorkload}    # anything else: a cfg name


def workload_class(name):
    return WORKLOADS.get(name, LaWorkload)


def measure(args, ranks, short=False):
    """Builds the workload, times it and returns its JSON line as a dict (None on ranks other than 0)."""
    import torch
    work = workload_class(args.workload)(args, ranks)
    t = time_blocks(work, args, ranks)
    e2e = None
    if not args.no_e2e and not short:
        e2e = work.e2e(max(1, min(args.steps, args.e2e_steps)))
        if ranks.world > 1:
            e2e["ms"] = max_over_ranks([e2e["ms"]], "cuda")[0]
    ms_step = t["ms_per_step"]
    line = None
    if ranks.rank == 0:
        peaks = measured_peaks()
        d = work.describe(ms_step, t["kernel_ms"], peaks)
        units = work.units * ranks.world
        line = {"metric": work.metric, "value": units / (ms_step * 1e-3), "unit": work.unit, "n_gpus": ranks.world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": d["dtype"], "data": "synthetic",
                "config": d["config"], "roofline": d["roofline"], "kernel_ms": t["kernel_ms"],
                "gpu_launches": d["gpu_launches_per_step"] * args.steps * t["timing"]["blocks"],
                "clocks": t["clocks"], "timing": t["timing"]}
        if e2e:
            line["e2e"] = {"value": units / (e2e["ms"] * 1e-3), "unit": work.unit, "h2d_bytes_per_step": e2e["h2d"],
                           "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"], "pinned_host_memory": True}
            line["e2e"].update(e2e.get("extra", {}))
        if not short:
            line.update(work.extras(ms_step))
    del work
    torch.cuda.empty_cache()
    return line


def other_paths(args, ranks):
    """Short runs of the three other built paths (log-probability, convolution, attention) for the record: value,
    kernel times, roofline fraction and clocks of each, without their end-to-end and CPU legs."""
    import copy
    out = {}
    for name in ("logp", "conv", "attn", "gk"):
        a = copy.copy(args)
        a.workload, a.steps, a.warmup, a.blocks = name, min(args.steps, 5), 3, 1
        try:
            line = measure(a, ranks, short=True)
        except Exception as e:                       # a failure here must not lose the main line
            out[name] = {"error": f"{type(e).__name__}: {e}"}
            continue
        out[name] = {"metric": line["metric"], "value": line["value"], "unit": line["unit"], "steps": a.steps,
                     "ms_per_step": line["ms_per_step"], "kernel_ms": line["kernel_ms"],
                     "roofline": {k: line["roofline"][k] for k in ("bound", "kernel", "achieved", "peak", "unit", "frac")},
                     "roofline_forward_frac": line["roofline"]["forward"]["frac"],
                     "roofline_whole_path_frac": line["roofline"]["whole_path"]["frac_strict"],
                     "clocks": line["clocks"], "workload": line["config"]}
    return out


def run_ours(args):
    ranks = Ranks()
    line = measure(args, ranks)
    if ranks.rank == 0:
        la = workload_class(args.workload) is LaWorkload
        if la and ranks.world == 1 and not args.no_other_paths:
            line["other_paths"] = other_paths(args, ranks)
        if ranks.world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = REFERENCE_SAMPLES[args.workload if not la else "la"](args, False)
        print(json.dumps(line))
    ranks.close()
    if ranks.world == 1 and args.per_config:
        per_config_table(args)


# ---- reference arm: the oracle, as it stands, on the host cores ------------------------------------------------------
def _la_sample(args, many_steps):
    # every step is a bounded sample; its size shrinks with the step count so that the whole run stays within minutes
    hint = min(8.0, 150.0 / max(1, args.warmup + args.steps)) if many_steps else 15.0
    return oracle_sample(args.workload, seconds_hint=hint)


REFERENCE_SAMPLES = {"la": _la_sample,
                     "logp": lambda args, many: logp_oracle_sample(small=many),
                     "conv": lambda args, many: conv_oracle_sample(small=many),
                     "attn": lambda args, many: attn_oracle_sample(small=many),
                     "gk": lambda args, many: gk_oracle_sample(small=many)}


def reference_config(args):
    if args.workload == "logp":
        return LOGP_METRIC, LOGP_UNIT, {"workload": "logp", "V": LOGP_V}
    if args.workload == "conv":
        return CONV_METRIC, UNIT, {"workload": "conv", "D": 4096, "w": CONV_W}
    if args.workload == "attn":
        return ATTN_METRIC, UNIT, {"workload": "attn", "Hq": ATTN_H, "Hkv": ATTN_H, "d": ATTN_D}
    if args.workload == "gk":
        return GK_METRIC, UNIT, {"workload": "gk", "trees": GK_CONFIG, "H": 16, "dk": 128, "dv": 128, "chunk": 64}
    from workloads import CONFIGS
    cfg = CONFIGS[args.workload]
    return METRIC, UNIT, {"workload": args.workload, "H": cfg["H"], "dk": cfg["dk"], "dv": cfg["dv"], "chunk": 64}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample = REFERENCE_SAMPLES[args.workload if args.workload in WORKLOADS else "la"]
    vals, secs, last = [], [], None
    for i in range(args.warmup + args.steps):
        last = sample(args, True)
        if i >= args.warmup:
            vals.append(last["value"])
            secs.append(last["seconds"])
    value = statistics.mean(vals)
    metric, unit, config = reference_config(args)
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": statistics.mean(secs) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config,
        "cpu_baseline": {"kind": last["kind"], "cores": last["cores"], "sample": last["sample"], "value": value,
                         "unit": unit},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


# ---- N ranks on one node ----------------------------------------------------------------------------------------------
def spawn_command(argv, gpus, port):
    """The torchrun command that starts `gpus` ranks of this script with the same arguments."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py")] + list(argv)


def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--blocks", type=int, default=0, help="timed blocks of --steps steps (0: enough for ~2 s)")
    ap.add_argument("--fma", action="store_true", help="force the fp32-FMA kernels")
    ap.add_argument("--round-launches", action="store_true",
                    help="one launch per round also on small problems (HARTS_FLAG_ROUND_LAUNCHES)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-trajwise", action="store_true")
    ap.add_argument("--no-other-paths", action="store_true", help="skip the short runs of the logp / conv / attn paths")
    ap.add_argument("--logp-rows", type=int, default=LOGP_ROWS, help="compact-row capacity of the logp workload")
    ap.add_argument("--conv-trees", default="cfg3", help="forest of the conv workload (cfg2: a small case for captures)")
    ap.add_argument("--attn-trees", default="cfg2", help="forest of the attn workload (cfg1: a small case for captures)")
    ap.add_argument("--gk-trees", default=GK_CONFIG, help="forest (and head count) of the gk workload: cfg1, cfg2 or cfg3")
    ap.add_argument("--attn-kv-heads", type=int, default=ATTN_H, help="kv heads of the attn workload (16 = MHA)")
    ap.add_argument("--per-config", action="store_true", help="also print a table over all configurations to stderr")
    args = ap.parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: become the launcher of one process per GPU (replicas, no collective on the data path)
        sys.exit(subprocess.call(spawn_command(argv, args.gpus, free_port())))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
