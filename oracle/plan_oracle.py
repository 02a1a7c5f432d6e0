"""Independent pure-Python minimum-call planner (test infrastructure only).

Follows Section 3.3 in the paper's notation: segments [s_v, e_v) (maximal fork-free token
paths), resume anchors a(p) = B*floor(p/B) (Eq. 2), a_v = a(s_v), b_v = a(e_v), the two call
counts T_pre / T_in (Eqs. 11-14), the recovery pass of Algorithm 1, the replay total of
Eq. 15, and the compact physical ordering of Section 4.2 (tokens of a sequence contiguous,
sequences of a round adjacent).

Readings the paper leaves open, fixed here (and identically in the product, so that plans
can be compared bit for bit):
  * child order at a fork: the continuation piece of a split node first, then the forked
    nodes in input order; "first child that fits" refers to this order;
  * sequences are ordered by (round, canonical index of their first own token); physical
    rows follow that order with no padding rows;
  * slots (requested boundary states) are numbered by (producing sequence, chunk index);
  * a side branch launched in the same round as its parent sequence (ready anchor, Eq. 11)
    inherits that sequence's initial state and start anchor; its replay rows may come from
    several ancestor segments.

Also here: a brute-force minimum call count under the execution model of Section 3.3 (last
paragraph before "Replay cost"), and two executions of a plan -- numpy fp64 forward, torch
fp64 autograd -- that check the plan's bookkeeping (state sources, replay rows, requests)
without any chunk arithmetic.
"""
from __future__ import annotations

import itertools
import sys
from dataclasses import dataclass, field

import numpy as np


def anchor(p: int, B: int) -> int:
    """Eq. 2."""
    return B * (p // B)


# ----------------------------------------------------------------------------------------------
# Segment tree (Section 3.3, "Execution model")
# ----------------------------------------------------------------------------------------------
@dataclass
class Segment:
    s: int                       # absolute position of the first token
    e: int                       # exclusive end
    pieces: list                 # [(node, lo, hi)] node-local token ranges, in order
    children: list = field(default_factory=list)
    parent: int = -1


def segment_tree(par, off, ln):
    """Node tree of one rollout tree -> list of Segment (index 0 is the root)."""
    n = len(par)
    forks = [dict() for _ in range(n)]            # node -> {offset: [forked children in input order]}
    for i in range(1, n):
        assert 0 <= par[i] < i and 1 <= off[i] <= ln[par[i]] and ln[i] >= 1
        forks[par[i]].setdefault(off[i], []).append(i)
    segs = []

    def grow(node, lo, abs_lo, parent):
        """Start a segment at offset lo of node; extend it until a real fork or a leaf end."""
        seg = Segment(abs_lo, abs_lo, [], [], parent)
        idx = len(segs)
        segs.append(seg)
        while True:
            cuts = sorted(o for o in forks[node] if o > lo)
            hi = cuts[0] if cuts else ln[node]
            seg.pieces.append((node, lo, hi))
            seg.e += hi - lo
            forked = forks[node].get(hi, [])
            if hi < ln[node]:
                # a fork inside the node: the node's own continuation first, then the forked nodes
                seg.children = [(node, hi)] + [(c, 0) for c in forked]
                break
            if len(forked) == 1:                  # a single child at the node's end: no fork, same segment
                node, lo = forked[0], 0
                continue
            seg.children = [(c, 0) for c in forked]   # >= 2 children, or none (leaf)
            break
        kids = seg.children
        seg.children = []
        for c, o in kids:
            seg.children.append(grow(c, o, seg.e, idx))
        return idx

    sys.setrecursionlimit(max(sys.getrecursionlimit(), 4 * n + 1000))
    grow(0, 0, 0, -1)
    return segs


# ----------------------------------------------------------------------------------------------
# Algorithm 1, first pass: T_pre, T_in
# ----------------------------------------------------------------------------------------------
def call_counts(segs, B):
    n = len(segs)
    Tpre, Tin = [0] * n, [0] * n
    order = []
    stack = [0]
    while stack:
        v = stack.pop()
        order.append(v)
        stack += segs[v].children
    for v in reversed(order):                     # children before parents
        ch = segs[v].children
        if not ch:
            Tpre[v] = Tin[v] = 1                  # Eq. 12
            continue
        best = None
        for o in ch:                              # Eq. 13
            h = max([Tpre[u] for u in ch if u != o], default=0)
            c = max(Tin[o], 1 + h)
            best = c if best is None else min(best, c)
        Tin[v] = best
        a_v = anchor(segs[v].s, B)
        if segs[v].e < a_v + B:                   # Eq. 11 / Eq. 14, first case
            Tpre[v] = max(Tpre[u] for u in ch)
        else:
            Tpre[v] = Tin[v]
    return Tpre, Tin


# ----------------------------------------------------------------------------------------------
# Algorithm 1, recovery
# ----------------------------------------------------------------------------------------------
@dataclass
class Seq:
    round: int                   # 1-based, as in Algorithm 1
    start: int                   # absolute start anchor (multiple of B)
    init: object                 # None (zero state) or (producer Seq, chunk index)
    segs: list = field(default_factory=list)
    replay_from: int = -1        # segment whose end is the fork this sequence hangs off (-1: root)
    tree: int = 0


def recover(segs, B, Tpre, Tin, tree=0):
    seqs = []

    def rec(v, ready, K_round, r, q):
        q.segs.append(v)
        ch = segs[v].children
        if not ch:
            return
        a_v = anchor(segs[v].s, B)
        b_v = anchor(segs[v].e, B)
        same = ready and segs[v].e < a_v + B
        delta = 0 if same else 1
        K_side = K_round - delta
        Hb = {o: (Tpre[o] if same else Tin[o]) for o in ch}
        f = sum(1 for u in ch if Tpre[u] > K_side)
        direct = None
        for o in ch:
            if Hb[o] <= K_round and f - (1 if Tpre[o] > K_side else 0) == 0:
                direct = o
                break
        assert direct is not None
        rec(direct, same, K_round, r, q)
        for u in ch:
            if u == direct:
                continue
            if same:
                qu = Seq(r, q.start, q.init, [], v, tree)          # from S_{a_v}: q's own initial state
                assert q.start == a_v == b_v
            else:
                c = (b_v - q.start) // B                           # request S_{b_v} from q
                assert c >= 1 and q.start + c * B == b_v
                qu = Seq(r + 1, b_v, (q, c), [], v, tree)
            seqs.append(qu)
            rec(u, True, K_side, r + delta, qu)

    q0 = Seq(1, 0, None, [], -1, tree)
    seqs.append(q0)
    rec(0, True, Tpre[0], 1, q0)
    return seqs


def replay_total(segs, B):
    """Eq. 15."""
    return sum((len(s.children) - 1) * (s.e % B) for s in segs if s.children)


# ----------------------------------------------------------------------------------------------
# Brute force: minimum number of sequential calls over every choice of direct continuations
# ----------------------------------------------------------------------------------------------
def brute_force_calls(segs, B):
    internal = [v for v in range(len(segs)) if segs[v].children]
    best = None
    for choice in itertools.product(*[segs[v].children for v in internal]):
        direct = dict(zip(internal, choice))
        head_start = {0: 0}       # sequence (named by its head segment) -> start anchor
        head_round = {0: 1}
        head_of = {0: 0}
        worst = 1
        for v in range(len(segs)):                # parents precede children
            h = head_of[v]
            for u in segs[v].children:
                if direct[v] == u:
                    head_of[u] = h
                    continue
                b_v = anchor(segs[v].e, B)
                head_of[u] = u
                head_start[u] = b_v
                # S_{b_v} is h's own initial state (ready when h starts) or is produced inside h's call
                head_round[u] = head_round[h] if b_v == head_start[h] else head_round[h] + 1
                worst = max(worst, head_round[u])
        best = worst if best is None else min(best, worst)
    return best


# ----------------------------------------------------------------------------------------------
# Full plan with the compact physical ordering and the index tables
# ----------------------------------------------------------------------------------------------
@dataclass
class Plan:
    chunk: int
    n_rounds: int
    C: int
    R: int
    n_seq: int
    n_slots: int
    row_of_token: np.ndarray
    round_seq_ptr: np.ndarray
    seq_tree: np.ndarray
    seq_own_begin: np.ndarray
    seq_own_len: np.ndarray
    seq_start_pos: np.ndarray
    seq_init_slot: np.ndarray
    seq_replay_ptr: np.ndarray
    replay_row: np.ndarray
    seq_req_ptr: np.ndarray
    slot_chunk: np.ndarray
    seq_chunk_ptr: np.ndarray
    slot_cons_ptr: np.ndarray
    slot_cons_seq: np.ndarray
    rg_row: np.ndarray
    rg_ptr: np.ndarray
    rg_entry: np.ndarray

    FIELDS = ("row_of_token", "round_seq_ptr", "seq_tree", "seq_own_begin", "seq_own_len", "seq_start_pos",
              "seq_init_slot", "seq_replay_ptr", "replay_row", "seq_req_ptr", "slot_chunk", "seq_chunk_ptr",
              "slot_cons_ptr", "slot_cons_seq", "rg_row", "rg_ptr", "rg_entry")


def plan_forest(forest, B: int) -> Plan:
    base = forest.token_base()
    all_seqs = []
    tree_segs = []
    R = 0
    for t in range(forest.n_trees):
        par, off, ln = (a.tolist() for a in forest.tree(t))
        segs = segment_tree(par, off, ln)
        Tpre, Tin = call_counts(segs, B)
        seqs = recover(segs, B, Tpre, Tin, tree=t)
        assert max(q.round for q in seqs) == Tpre[0]
        R += replay_total(segs, B)
        tree_segs.append(segs)
        all_seqs += seqs

    lo_of_tree = [int(x) for x in forest.tree_node_ptr]

    def seg_tokens(t, v):
        """canonical token indices of segment v of tree t"""
        out = []
        for node, lo, hi in tree_segs[t][v].pieces:
            b = int(base[lo_of_tree[t] + node])
            out.append(np.arange(b + lo, b + hi, dtype=np.int64))
        return np.concatenate(out)

    def first_token(q):
        node, lo, _ = tree_segs[q.tree][q.segs[0]].pieces[0]
        return int(base[lo_of_tree[q.tree] + node]) + lo

    all_seqs.sort(key=lambda q: (q.round, first_token(q)))
    n_seq = len(all_seqs)
    index_of = {id(q): i for i, q in enumerate(all_seqs)}
    n_rounds = max(q.round for q in all_seqs)
    C = forest.n_tokens

    row_of_token = np.full(C, -1, dtype=np.int64)
    own_begin, own_len = [], []
    row = 0
    for q in all_seqs:
        toks = np.concatenate([seg_tokens(q.tree, v) for v in q.segs])
        row_of_token[toks] = np.arange(row, row + len(toks))
        own_begin.append(row)
        own_len.append(len(toks))
        row += len(toks)
    assert row == C and (row_of_token >= 0).all()

    # replay rows: absolute positions [start, s_first) along the ancestor path, path order
    replay_ptr, replay_row = [0], []
    for q in all_seqs:
        segs = tree_segs[q.tree]
        first = segs[q.segs[0]]
        need = first.s - q.start
        assert 0 <= need < B and q.start % B == 0
        rows_rev = []
        v = q.replay_from
        while need > 0:
            toks = seg_tokens(q.tree, v)
            take = min(need, len(toks))
            rows_rev.append(row_of_token[toks[len(toks) - take:]])
            need -= take
            v = segs[v].parent
        for piece in reversed(rows_rev):
            replay_row += piece.tolist()
        replay_ptr.append(len(replay_row))
    assert len(replay_row) == R

    # slots: unique (producer sequence, chunk index), numbered in that order
    wanted = sorted({(index_of[id(q.init[0])], q.init[1]) for q in all_seqs if q.init is not None})
    slot_id = {key: i for i, key in enumerate(wanted)}
    init_slot = [(-1 if q.init is None else slot_id[(index_of[id(q.init[0])], q.init[1])]) for q in all_seqs]
    req_ptr = [0]
    for i in range(n_seq):
        req_ptr.append(req_ptr[-1] + sum(1 for (s, _) in wanted if s == i))
    slot_chunk = [c for (_, c) in wanted]

    cons = [[] for _ in wanted]
    for i, s in enumerate(init_slot):
        if s >= 0:
            cons[s].append(i)
    cons_ptr = [0]
    for c in cons:
        cons_ptr.append(cons_ptr[-1] + len(c))

    targets = {}
    for e, r in enumerate(replay_row):
        targets.setdefault(r, []).append(e)
    rg_row = sorted(targets)
    rg_ptr = [0]
    rg_entry = []
    for r in rg_row:
        rg_entry += targets[r]
        rg_ptr.append(len(rg_entry))

    chunk_ptr = [0]
    for i in range(n_seq):
        virt = (replay_ptr[i + 1] - replay_ptr[i]) + own_len[i]
        chunk_ptr.append(chunk_ptr[-1] + (virt + B - 1) // B)

    round_ptr = [0] * (n_rounds + 1)
    for q in all_seqs:
        round_ptr[q.round] += 1
    round_ptr = np.cumsum(round_ptr)

    i32 = lambda x: np.asarray(x, dtype=np.int32)  # noqa: E731
    return Plan(B, n_rounds, C, R, n_seq, len(wanted), i32(row_of_token), i32(round_ptr),
                i32([q.tree for q in all_seqs]), i32(own_begin), i32(own_len), i32([q.start for q in all_seqs]),
                i32(init_slot), i32(replay_ptr), i32(replay_row), i32(req_ptr), i32(slot_chunk), i32(chunk_ptr),
                i32(cons_ptr), i32([s for c in cons for s in c]), i32(rg_row), i32(rg_ptr), i32(rg_entry))


# ----------------------------------------------------------------------------------------------
# Executing a plan with the token recurrence (no chunk arithmetic): bookkeeping check
# ----------------------------------------------------------------------------------------------
def simulate_plan_fwd(plan, q, k, v, g):
    """q,k,v,g on PHYSICAL rows ([C,H,d] fp64 numpy).  Runs the rounds as planned (Section 3.4,
    "Round-wise execution"): initial state from a slot or zero, replay rows update the state
    only, own rows also produce outputs, requested chunk-boundary states go to their slots."""
    C, H, dk = q.shape
    dv = v.shape[2]
    B = plan.chunk
    o = np.full((C, H, dv), np.nan)
    slots = [None] * plan.n_slots
    for r in range(plan.n_rounds):
        produced = {}
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            s0 = plan.seq_init_slot[i]
            S = np.zeros((H, dk, dv)) if s0 < 0 else slots[s0].copy()   # must come from an earlier round
            rep = plan.replay_row[plan.seq_replay_ptr[i]:plan.seq_replay_ptr[i + 1]]
            rows = list(rep) + list(range(plan.seq_own_begin[i], plan.seq_own_begin[i] + plan.seq_own_len[i]))
            req = {int(plan.slot_chunk[s]): s for s in range(plan.seq_req_ptr[i], plan.seq_req_ptr[i + 1])}
            for j, row in enumerate(rows):
                if j % B == 0 and (j // B) in req:
                    produced[req[j // B]] = S.copy()
                S = np.exp(g[row])[:, None, None] * S + k[row][:, :, None] * v[row][:, None, :]
                if j >= len(rep):
                    assert np.isnan(o[row]).all()                       # written exactly once
                    o[row] = np.einsum("hi,hij->hj", q[row], S)
            assert all(c * B < len(rows) for c in req)
        for s, val in produced.items():            # visible only after the call returns
            slots[s] = val
    return o


def simulate_plan_autograd(plan, q, k, v, g, dO):
    """Same execution in torch fp64 with autograd: returns o and dq, dk, dv, dg on physical rows.
    Gradients reach ancestors through the slot tensors and through the gathered replay rows."""
    import torch
    q, k, v, g = (torch.tensor(np.asarray(x), dtype=torch.float64, requires_grad=True) for x in (q, k, v, g))
    dO = torch.tensor(np.asarray(dO), dtype=torch.float64)
    C, H, dk = q.shape
    dv = v.shape[2]
    B = plan.chunk
    outs = [None] * C
    slots = [None] * plan.n_slots
    for r in range(plan.n_rounds):
        produced = {}
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            s0 = plan.seq_init_slot[i]
            S = torch.zeros(H, dk, dv, dtype=torch.float64) if s0 < 0 else slots[s0]
            rep = plan.replay_row[plan.seq_replay_ptr[i]:plan.seq_replay_ptr[i + 1]]
            rows = list(rep) + list(range(plan.seq_own_begin[i], plan.seq_own_begin[i] + plan.seq_own_len[i]))
            req = {int(plan.slot_chunk[s]): s for s in range(plan.seq_req_ptr[i], plan.seq_req_ptr[i + 1])}
            for j, row in enumerate(rows):
                if j % B == 0 and (j // B) in req:
                    produced[req[j // B]] = S
                S = torch.exp(g[row])[:, None, None] * S + k[row][:, :, None] * v[row][:, None, :]
                if j >= len(rep):
                    outs[row] = torch.einsum("hi,hij->hj", q[row], S)
        for s, val in produced.items():
            slots[s] = val
    o = torch.stack(outs)
    (o * dO).sum().backward()
    return tuple(x.detach().numpy() for x in (o, q.grad, k.grad, v.grad, g.grad))


def simulate_plan_bwd_tables(plan, q, k, v, g, dO):
    """Reverse pass over a plan that routes every gradient through the plan's OWN backward tables (no autograd):
    the chunk-start states a backward would re-read are stored and addressed with `seq_chunk_ptr`; at a requested
    boundary the initial-state gradients of the consuming sequences are collected through `slot_cons_ptr` /
    `slot_cons_seq` (Section 3.4, "Differentiable boundary states": several consumers of one boundary are summed);
    gradients of replayed rows are kept per replay entry and folded into their producer rows through `rg_row` /
    `rg_ptr` / `rg_entry` (Section 4.2: the gather's backward accumulates into the unique producer row).  Inside a
    chunk it is the plain reverse token recurrence, so a wrong table shows up against the trajectory-wise oracle.
    Inputs on PHYSICAL rows, fp64 numpy.  Returns dq, dk, dv, dg on physical rows."""
    C, H, dk_ = q.shape
    dv_ = v.shape[2]
    B = plan.chunk
    n_chunks = int(plan.seq_chunk_ptr[-1])
    chunk_state = [None] * n_chunks
    slots = [None] * plan.n_slots
    seq_rows = []
    for r in range(plan.n_rounds):
        produced = {}
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            s0 = plan.seq_init_slot[i]
            S = np.zeros((H, dk_, dv_)) if s0 < 0 else slots[s0].copy()
            rep = list(plan.replay_row[plan.seq_replay_ptr[i]:plan.seq_replay_ptr[i + 1]])
            rows = rep + list(range(plan.seq_own_begin[i], plan.seq_own_begin[i] + plan.seq_own_len[i]))
            req = {int(plan.slot_chunk[s]): s for s in range(plan.seq_req_ptr[i], plan.seq_req_ptr[i + 1])}
            assert plan.seq_chunk_ptr[i + 1] - plan.seq_chunk_ptr[i] == (len(rows) + B - 1) // B
            for j, row in enumerate(rows):
                if j % B == 0:
                    chunk_state[plan.seq_chunk_ptr[i] + j // B] = S.copy()
                    if (j // B) in req:
                        produced[req[j // B]] = S.copy()
                S = np.exp(g[row])[:, None, None] * S + k[row][:, :, None] * v[row][:, None, :]
        for s, val in produced.items():
            slots[s] = val
    assert all(x is not None for x in chunk_state)

    dq, dk, dv, dg = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v), np.zeros_like(g)
    ds0 = [None] * plan.n_seq                           # gradient w.r.t. each sequence's initial state
    rk = np.zeros((len(plan.replay_row), H, dk_))       # gradients of replayed rows, per replay entry
    rv = np.zeros((len(plan.replay_row), H, dv_))
    rgr = np.zeros((len(plan.replay_row), H))
    for r in reversed(range(plan.n_rounds)):
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            n_rep = int(plan.seq_replay_ptr[i + 1] - plan.seq_replay_ptr[i])
            rows = list(plan.replay_row[plan.seq_replay_ptr[i]:plan.seq_replay_ptr[i + 1]]) + \
                list(range(plan.seq_own_begin[i], plan.seq_own_begin[i] + plan.seq_own_len[i]))
            req = {int(plan.slot_chunk[s]): s for s in range(plan.seq_req_ptr[i], plan.seq_req_ptr[i + 1])}
            carry = np.zeros((H, dk_, dv_))             # dL/dS after the current token, already decayed to it
            for c in reversed(range((len(rows) + B - 1) // B)):
                lo_, hi_ = c * B, min((c + 1) * B, len(rows))
                # recompute the states inside the chunk from its stored start state
                S_prev = [chunk_state[plan.seq_chunk_ptr[i] + c]]
                for j in range(lo_, hi_):
                    row = rows[j]
                    S_prev.append(np.exp(g[row])[:, None, None] * S_prev[-1] + k[row][:, :, None] * v[row][:, None, :])
                for j in reversed(range(lo_, hi_)):
                    row = rows[j]
                    S_t, S_tm1 = S_prev[j - lo_ + 1], S_prev[j - lo_]
                    dS = carry
                    if j >= n_rep:
                        dS = dS + q[row][:, :, None] * dO[row][:, None, :]
                        dq[row] = np.einsum("hij,hj->hi", S_t, dO[row])
                    gk = np.einsum("hij,hj->hi", dS, v[row])
                    gv = np.einsum("hij,hi->hj", dS, k[row])
                    gg = np.exp(g[row]) * np.einsum("hij,hij->h", S_tm1, dS)
                    if j >= n_rep:
                        dk[row], dv[row], dg[row] = gk, gv, gg
                    else:
                        e = plan.seq_replay_ptr[i] + j
                        rk[e], rv[e], rgr[e] = gk, gv, gg
                    carry = np.exp(g[row])[:, None, None] * dS
                if c in req:                            # boundary c was exported: add every consumer's gradient
                    s = req[c]
                    for u in plan.slot_cons_seq[plan.slot_cons_ptr[s]:plan.slot_cons_ptr[s + 1]]:
                        assert ds0[u] is not None       # consumers run in a later round: already done
                        carry = carry + ds0[u]
            ds0[i] = carry
    for n, row in enumerate(plan.rg_row):
        for e in plan.rg_entry[plan.rg_ptr[n]:plan.rg_ptr[n + 1]]:
            dk[row] += rk[e]
            dv[row] += rv[e]
            dg[row] += rgr[e]
    return dq, dk, dv, dg
