"""harts_mb_plan (C ABI, host) against the oracle pieces: costs, guarantees, brute force over contiguous cuts."""
import random

import numpy as np
import pytest

import paper_2608_28158_b200 as H
from oracle import mb_oracle as mo
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _plan(fo, D, T):
    return H.harts_mb_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, D, T)


def _lex_trajs(fo, plan):
    """The oracle's trajectories re-ordered like the plan (matched by the node they end in and their length)."""
    trajs = mo.trajectory_tokens(fo)
    base = fo.token_base()
    by_last = {t[-1]: t for t in trajs}                         # last canonical token identifies a trajectory
    out = []
    for leaf, ln in zip(plan.traj_leaf, plan.traj_len):
        t = by_last[int(base[leaf + 1]) - 1]
        assert len(t) == ln
        out.append(t)
    return out


def test_order_lengths_and_adjacent_lcp():
    rnd = random.Random(3)
    for _ in range(60):
        fo = make_forest([random_tree(rnd, 9, 9) for _ in range(rnd.randint(1, 3))])
        plan = _plan(fo, 1, 10 ** 6)
        trajs = _lex_trajs(fo, plan)
        assert len(trajs) == plan.n_traj == len(mo.trajectory_tokens(fo))
        assert plan.traj_lcp[0] == 0
        for i in range(1, len(trajs)):
            assert plan.traj_lcp[i] == mo.lcp(trajs[i - 1], trajs[i])
        # a depth-first order: Eq. 5 over the whole batch equals the trie count
        assert plan.total_work_all == mo.trie_cost(trajs) == fo.n_tokens
        assert plan.n_mb == 1 and plan.J[0] == fo.n_tokens       # everything fits one microbatch


def test_guarantees_and_objective_on_random_forests():
    rnd = random.Random(4)
    for _ in range(80):
        fo = make_forest([random_tree(rnd, 9, 12) for _ in range(rnd.randint(1, 4))])
        n = len(mo.trajectory_tokens(fo))
        D = rnd.choice([1, 2, 3])
        longest = max(len(t) for t in mo.trajectory_tokens(fo))
        T = rnd.randint(longest, max(longest, fo.n_tokens))
        if n < D:
            with pytest.raises(H.HartsError):
                _plan(fo, D, T)
            continue
        try:
            plan = _plan(fo, D, T)
        except H.HartsError:
            continue                                             # no grouping with K mod D = 0 exists (rare, tiny N)
        trajs = _lex_trajs(fo, plan)
        J, works = mo.check_plan(trajs, plan.traj_mb, plan.mb_replica, plan.mb_slot, D, T)
        assert J == plan.J and works == plan.mb_work.tolist()
        # the schedule follows the stated rule
        replica, slot, tail = mo.slot_schedule(works, D)
        assert tail == plan.J[1:] and slot == plan.mb_slot.tolist()


def test_exact_mode_matches_brute_force_over_contiguous_cuts():
    rnd = random.Random(5)
    checked = 0
    for _ in range(200):
        fo = make_forest([random_tree(rnd, 7, 10) for _ in range(2)])
        raw = mo.trajectory_tokens(fo)
        if not 3 <= len(raw) <= 8:
            continue
        longest = max(len(t) for t in raw)
        T = rnd.randint(longest, longest + fo.n_tokens // 2)
        D = rnd.choice([1, 2])
        try:
            plan = _plan(fo, D, T)
        except H.HartsError:
            continue
        trajs = _lex_trajs(fo, plan)
        # no contiguous partition with a K of the search range beats the selected plan's total work
        G = mo.trie_cost(trajs)
        kmin = D * max(1, -(-G // (T * D)))
        kmax = max(kmin, min(D * -(-plan.natural_mb // D), D * (len(trajs) // D)))
        best = None
        for K in range(kmin, kmax + 1, D):
            if K > len(trajs):
                break
            b = mo.best_contiguous(trajs, K, T)
            if b is not None and (best is None or b[0] < best):
                best = b[0]
        if best is not None:
            assert plan.J[0] <= best
            checked += 1
    assert checked >= 30


def test_prefix_aware_beats_prefix_blind_on_cfg2():
    """cfg2's eight trees at the paper's capacity: trajectories that share long prefixes stay together."""
    fo = config_forest("cfg2")
    plan = _plan(fo, 2, 65536)
    assert plan.n_mb % 2 == 0 and plan.mb_work.max() <= 65536
    assert plan.J[0] <= plan.natural_work
    assert plan.J[0] < 1.15 * plan.total_work_all              # close to the single-trie bound
    assert plan.J[0] < 0.5 * int(plan.traj_len.sum())           # far below one-trajectory-per-row cost


def test_large_batch_takes_the_heuristic_path_and_keeps_the_guarantees():
    """cfg4 (16,996 trajectories, above the exact-search threshold) at a capacity that forces cuts inside trees."""
    fo = config_forest("cfg4")
    D, T = 4, 5000
    plan = _plan(fo, D, T)
    assert plan.n_traj > 512 and plan.n_mb % D == 0
    assert np.bincount(plan.traj_mb, minlength=plan.n_mb).min() >= 1              # non-empty, exact coverage
    assert np.bincount(plan.mb_replica, minlength=D).tolist() == [plan.n_mb // D] * D
    total = 0
    for mb in range(plan.n_mb):                                                     # work recounted from the sub-forest
        ptr, par, off, ln, src = plan.extract(mb)
        assert int(ln.sum()) == plan.mb_work[mb] <= T
        total += int(ln.sum())
    assert total == plan.J[0] <= plan.natural_work
    replica, slot, tail = mo.slot_schedule(plan.mb_work.tolist(), D)
    assert tail == plan.J[1:]


def test_extract_gives_the_microbatch_forest():
    rnd = random.Random(6)
    for _ in range(30):
        fo = make_forest([random_tree(rnd, 8, 10) for _ in range(3)])
        raw = mo.trajectory_tokens(fo)
        longest = max(len(t) for t in raw)
        try:
            plan = _plan(fo, 1, longest + 5)
        except H.HartsError:
            continue
        for mb in range(plan.n_mb):
            ptr, par, off, ln, src = plan.extract(mb)
            sub = make_forest([(par[ptr[t]:ptr[t + 1]].tolist(), off[ptr[t]:ptr[t + 1]].tolist(), ln[ptr[t]:ptr[t + 1]].tolist())
                               for t in range(len(ptr) - 1)])
            assert sub.n_tokens == plan.mb_work[mb]              # compact tokens of the microbatch
            want = sorted(int(l) for l, m in zip(plan.traj_len, plan.traj_mb) if m == mb)
            assert sorted(len(t) for t in mo.trajectory_tokens(sub)) == want
            H.harts_la_plan(sub.tree_node_ptr, sub.node_parent, sub.node_fork_off, sub.node_len, 64)   # plannable


def test_errors():
    fo = config_forest("cfg0")
    with pytest.raises(H.HartsError):
        _plan(fo, 1, 100)                                        # a trajectory longer than T
    with pytest.raises(H.HartsError):
        _plan(fo, 4, 10 ** 6)                                    # fewer trajectories than replicas
    with pytest.raises(H.HartsError):
        H.harts_mb_plan([0, 2], [-1, 0], [0, 9], [4, 4], 1, 100)


def test_greedy_increments_and_destinations_follow_eq10():
    """Every step of the planner's greedy placement pass -- the processing order, the work increase it claims
    (Eq. 10 through the LCP index), the destination under best-fit / max-shared, the moment a new microbatch is
    opened -- against the oracle's pass, which takes the increase from the trie count with and without the
    candidate.  A greedy that ignored sharing, used the wrong neighbours or broke ties differently fails here."""
    rnd = random.Random(12)
    shared_steps = 0
    for trial in range(40):
        fo = make_forest([random_tree(rnd, 9, 12) for _ in range(rnd.randint(1, 4))])
        all_t = mo.trajectory_tokens(fo)
        longest = max(len(t) for t in all_t)
        T = rnd.randint(longest, max(longest, fo.n_tokens // 2 + longest))
        try:
            plan = _plan(fo, 1, T)
        except H.HartsError:
            continue
        trajs = _lex_trajs(fo, plan)
        orders = mo.greedy_orders(trajs)
        for order in range(4):
            for policy in range(2):
                x, mb, created, delta = plan.greedy_trace(order, policy)
                want = mo.greedy_place(trajs, orders[order], T, best_fit=(policy == 0))
                got = list(zip(x.tolist(), mb.tolist(), created.tolist(), delta.tolist()))
                assert got == want, (trial, order, policy)
                shared_steps += sum(1 for (i, _, c, d) in want if not c and d < len(trajs[i]))
    assert shared_steps > 200                                    # sharing did decide many placements
