"""Pins for the pure-Python planner (oracle/plan_oracle.py): the paper's worked examples, the
strict boundary cases, brute-force minimum call counts, Eq. 15, and fp64 execution of the plan
against the trajectory-wise oracle (forward with numpy, backward with autograd)."""
import os
import random

import numpy as np
import pytest

from oracle import la_oracle as lo
from oracle import plan_oracle as po
from workloads import make_forest, config_forest, make_inputs, CONFIGS

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def one_tree(par, off, ln):
    return make_forest([(par, off, ln)])


def seq_table(plan):
    out = []
    for r in range(plan.n_rounds):
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            out.append((r + 1, int(plan.seq_own_len[i]), int(plan.seq_replay_ptr[i + 1] - plan.seq_replay_ptr[i]),
                        int(plan.seq_start_pos[i]), int(plan.seq_init_slot[i])))
    return out


def test_fig2_worked_example():
    B = 64
    # v0=[0,B-1) -> v1 (2 tokens) and v2; v1=[B-1,B+1) -> v3, v4
    fo = one_tree([-1, 0, 0, 1, 1], [0, B - 1, B - 1, 2, 2], [B - 1, 2, 40, 30, 20])
    p = po.plan_forest(fo, B)
    facts = dict(line.split() for line in open(os.path.join(GOLDEN, "fig2_example.txt")) if not line.startswith("#"))
    assert p.n_rounds == int(facts["rounds"])
    tab = seq_table(p)
    assert sum(1 for t in tab if t[0] == 1) == int(facts["round1_sequences"])
    assert sum(1 for t in tab if t[0] == 2) == int(facts["round2_sequences"])
    # round 1: v0->v1->v3 (63+2+30 own tokens, zero state) and v2 with replay B-1 from the zero state
    assert (1, B - 1 + 2 + 30, 0, 0, -1) in tab
    assert (1, 40, B - 1, 0, -1) in tab
    # round 2: v4 from S_B (chunk index 1 of the root sequence), replay [B, B+1)
    assert (2, 20, 1, B, 0) in tab
    assert p.slot_chunk.tolist() == [int(facts["v4_state_chunk"])] and p.R == B - 1 + 1


@pytest.mark.parametrize("fork,rounds,replay", [(63, 1, 63), (64, 2, 0), (65, 2, 1)])
def test_strict_boundary_cases(fork, rounds, replay):
    # a root of `fork` tokens with two leaves: B-1 -> same round; B -> replay 0 but next round; B+1 -> next round
    fo = one_tree([-1, 0, 0], [0, fork, fork], [fork, 10, 10])
    p = po.plan_forest(fo, 64)
    assert p.n_rounds == rounds and p.R == replay


def test_fig1_example():
    # T1 = A.B.D, T2 = A.B.E, T3 = A.C ; with |A| >= chunk: call 1 = [A,B,D], call 2 = {[C],[E]}
    fo = one_tree([-1, 0, 0, 1, 1], [0, 100, 100, 80, 80], [100, 80, 50, 30, 30])
    p = po.plan_forest(fo, 64)
    assert p.n_rounds == 2
    assert [t[:2] for t in seq_table(p)] == [(1, 210), (2, 50), (2, 30)]
    # short shared pieces: everything starts in one call from the zero state
    fo = one_tree([-1, 0, 0, 1, 1], [0, 30, 30, 10, 10], [30, 10, 50, 30, 30])
    assert po.plan_forest(fo, 64).n_rounds == 1


def test_fig3_example_two_consumers_share_a_state():
    # P0 (one chunk) then P1 (inside the next chunk), three-way fork A,B,C inside that chunk
    fo = one_tree([-1, 0, 0, 0], [0, 84, 84, 84], [84, 40, 30, 20])
    p = po.plan_forest(fo, 64)
    tab = seq_table(p)
    assert tab == [(1, 124, 0, 0, -1), (2, 30, 20, 64, 0), (2, 20, 20, 64, 0)]
    assert p.n_slots == 1 and p.slot_cons_seq.tolist() == [1, 2]
    # both replays read P1's rows 64..83 of the round-1 sequence
    assert p.replay_row.tolist() == list(range(64, 84)) * 2


def test_cfg0_plan():
    p = po.plan_forest(config_forest("cfg0"), 64)
    assert (p.C, p.R, p.n_rounds, p.n_seq, p.n_slots) == (718, 36, 2, 3, 2)
    # round 1 = root pieces + A (384 rows, requests boundaries 1 and 4); round 2 = [replay 36 | C] and X+B
    assert seq_table(p) == [(1, 384, 0, 0, -1), (2, 134, 0, 256, 1), (2, 200, 36, 64, 0)]
    assert p.slot_chunk.tolist() == [1, 4]
    assert p.replay_row.tolist() == list(range(64, 100))


def test_cfg0b_plan_shared_slot_and_same_round_replay():
    p = po.plan_forest(config_forest("cfg0b"), 64)
    assert (p.n_rounds, p.R) == (2, 80)
    tab = seq_table(p)
    # [X,B] and [replay 44 = X's rows | B2] both start from S_256; C from S_64
    assert tab[0] == (1, 384, 0, 0, -1)
    assert sorted(tab[1:]) == sorted([(2, 134, 0, 256, 1), (2, 200, 36, 64, 0), (2, 50, 44, 256, 1)])


def random_tree(rng, max_nodes, max_len):
    n = rng.randint(1, max_nodes)
    par, off, ln = [-1], [0], [rng.randint(1, max_len)]
    for i in range(1, n):
        p = rng.randint(0, i - 1)
        par.append(p)
        off.append(rng.randint(1, ln[p]))
        ln.append(rng.randint(1, max_len))
    return par, off, ln


def test_minimum_calls_against_brute_force():
    rng = random.Random(0)
    B = 4
    for _ in range(1500):
        par, off, ln = random_tree(rng, 9, 2 * B + 1)
        segs = po.segment_tree(par, off, ln)
        Tpre, Tin = po.call_counts(segs, B)
        seqs = po.recover(segs, B, Tpre, Tin)
        assert Tpre[0] == po.brute_force_calls(segs, B) == max(q.round for q in seqs), (par, off, ln)
        # every segment executed exactly once
        assert sorted(v for q in seqs for v in q.segs) == list(range(len(segs)))
        # segments are maximal: no segment has exactly one child
        assert all(len(s.children) != 1 for s in segs)


def check_plan_invariants(plan, forest):
    B = plan.chunk
    assert sorted(plan.row_of_token.tolist()) == list(range(plan.C))
    assert (plan.seq_start_pos % B == 0).all()
    rep_len = np.diff(plan.seq_replay_ptr)
    assert (rep_len < B).all() and rep_len.sum() == plan.R
    assert plan.seq_own_len.sum() == plan.C
    for r in range(plan.n_rounds):
        for i in range(plan.round_seq_ptr[r], plan.round_seq_ptr[r + 1]):
            s = plan.seq_init_slot[i]
            if s >= 0:      # the producer ran exactly one round earlier
                producer = int(np.searchsorted(plan.seq_req_ptr, s, side="right") - 1)
                pr = int(np.searchsorted(plan.round_seq_ptr, producer, side="right") - 1)
                assert pr == r - 1
            else:
                assert plan.seq_start_pos[i] == 0


def test_random_forests_plan_executes_to_oracle():
    rng = random.Random(1)
    for trial in range(12):
        B = rng.choice([2, 4, 8])
        trees = [random_tree(rng, 8, 3 * B) for _ in range(rng.randint(1, 3))]
        fo = make_forest(trees)
        plan = po.plan_forest(fo, B)
        check_plan_invariants(plan, fo)
        inp = {n: x.double().numpy() for n, x in make_inputs(fo.n_tokens, 2, 3, 2, "fp32", trial).items()}
        ref = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
        phys = {n: np.empty_like(x) for n, x in inp.items()}
        for n in inp:
            phys[n][plan.row_of_token] = inp[n]
        o = po.simulate_plan_fwd(plan, phys["q"], phys["k"], phys["v"], phys["g"])
        np.testing.assert_allclose(o[plan.row_of_token], ref["o"], rtol=1e-11, atol=1e-12)
        if trial < 6:
            _, dq, dk, dv, dg = po.simulate_plan_autograd(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
            for mine, name in ((dq, "dq"), (dk, "dk"), (dv, "dv"), (dg, "dg")):
                np.testing.assert_allclose(mine[plan.row_of_token], ref[name], rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("name", ["cfg0", "cfg0b"])
def test_cfg0_plan_executes_to_oracle(name):
    fo = config_forest(name)
    cfg = CONFIGS[name]
    plan = po.plan_forest(fo, cfg["chunk"])
    check_plan_invariants(plan, fo)
    inp = {n: x.double().numpy() for n, x in make_inputs(fo.n_tokens, 1, 4, 3, "fp32", 3).items()}
    ref = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
    phys = {n: np.empty_like(x) for n, x in inp.items()}
    for n in inp:
        phys[n][plan.row_of_token] = inp[n]
    o, dq, dk, dv, dg = po.simulate_plan_autograd(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    np.testing.assert_allclose(o[plan.row_of_token], ref["o"], rtol=1e-11, atol=1e-12)
    for mine, n in ((dq, "dq"), (dk, "dk"), (dv, "dv"), (dg, "dg")):
        np.testing.assert_allclose(mine[plan.row_of_token], ref[n], rtol=1e-9, atol=1e-11)


@pytest.mark.parametrize("name", ["cfg1", "cfg2", "cfg4"])
def test_config_plans_are_valid(name):
    fo = config_forest(name)
    plan = po.plan_forest(fo, 64)
    check_plan_invariants(plan, fo)
    if name == "cfg2":
        ptr, _ = lo.trajectories(fo)
        assert plan.C == 149270 and 5.4 <= ptr[-1] / plan.C <= 5.9


def test_appendix_totals_are_self_consistent():
    for line in open(os.path.join(GOLDEN, "appendix_cases.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, calls, segs, R, per_call, members = [x.strip() for x in line.split(";")]
        per_call = [int(x) for x in per_call.split()]
        members = [[int(x) for x in part.split()] for part in members.split("|")]
        assert len(per_call) == int(calls) == len(members)
        assert sum(per_call) == int(R)
        assert [sum(m) for m in members] == per_call
        assert all(0 <= x < 64 for m in members for x in m)


def _phys_inputs(fo, plan, H, dk, dv, seed):
    inp = {n: x.double().numpy() for n, x in make_inputs(fo.n_tokens, H, dk, dv, "fp32", seed).items()}
    phys = {n: np.empty_like(x) for n, x in inp.items()}
    for n in inp:
        phys[n][plan.row_of_token] = inp[n]
    return inp, phys


def test_backward_tables_route_gradients_to_the_oracle():
    """Pins the plan's backward tables (slot consumers, replayed-row gradient CSR, chunk-state addressing): a plain
    reverse token recurrence that takes every hand-off and replay gradient THROUGH those tables must reproduce the
    trajectory-wise oracle."""
    rng = random.Random(11)
    cases = [config_forest("cfg0"), config_forest("cfg0b")]
    cases += [make_forest([random_tree(rng, rng.randint(2, 9), 40) for _ in range(rng.randint(1, 3))]) for _ in range(14)]
    seen_shared_slot = seen_multi_replay = 0
    for n, fo in enumerate(cases):
        B = 64 if n < 2 else rng.choice([4, 8])
        plan = po.plan_forest(fo, B)
        inp, phys = _phys_inputs(fo, plan, 2, 3, 2, 100 + n)
        ref = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
        got = po.simulate_plan_bwd_tables(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
        for mine, name in zip(got, ("dq", "dk", "dv", "dg")):
            np.testing.assert_allclose(mine[plan.row_of_token], ref[name], rtol=1e-9, atol=1e-11, err_msg=f"{n} {name}")
        seen_shared_slot += int((np.diff(plan.slot_cons_ptr) > 1).any())
        seen_multi_replay += int((np.diff(plan.rg_ptr) > 1).any())
    assert seen_shared_slot >= 3 and seen_multi_replay >= 3     # the cases do exercise summed consumers


@pytest.mark.parametrize("table", ["slot_cons_seq", "slot_cons_ptr", "rg_entry", "rg_row", "seq_chunk_ptr"])
def test_a_wrong_backward_table_is_caught(table):
    """The pin above has teeth: corrupting any one backward table changes the gradients (or trips a check)."""
    fo = config_forest("cfg0b")
    plan = po.plan_forest(fo, 64)
    inp, phys = _phys_inputs(fo, plan, 1, 3, 2, 5)
    ref = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
    bad = getattr(plan, table).copy()
    if table == "slot_cons_seq":
        assert len(bad) >= 2
        bad[0] = bad[1]                       # one consumer counted twice, another dropped
    elif table == "slot_cons_ptr":
        bad[-1] -= 1                          # last consumer dropped
    elif table == "rg_entry":
        bad[0] = bad[-1]                      # a replay entry folded into the wrong row
    elif table == "rg_row":
        bad[0] += 1
    else:
        bad[1:] += 1                          # chunk states read from the neighbouring chunk
    setattr(plan, table, bad)
    try:
        got = po.simulate_plan_bwd_tables(plan, phys["q"], phys["k"], phys["v"], phys["g"], phys["dO"])
    except (AssertionError, IndexError, TypeError):
        return
    worst = max(np.abs(m[plan.row_of_token] - ref[n]).max() for m, n in zip(got, ("dq", "dk", "dv", "dg")))
    assert worst > 1e-6
