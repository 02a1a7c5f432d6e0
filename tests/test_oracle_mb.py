"""Pins of the microbatch-planning oracle pieces (Section 3.2, Eqs. 5-6) against the trie they summarise."""
import random

import numpy as np

from oracle import mb_oracle as mo
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def test_eq5_equals_the_trie_count_in_any_depth_first_order():
    rnd = random.Random(1)
    for _ in range(60):
        fo = make_forest([random_tree(rnd, 8, 9) for _ in range(rnd.randint(1, 3))])
        trajs = mo.trajectory_tokens(fo)
        order = sorted(range(len(trajs)), key=lambda i: trajs[i])          # lexicographic = a depth-first order
        srt = [trajs[i] for i in order]
        assert mo.interval_cost_eq5(srt) == mo.trie_cost(trajs)
        a, b = sorted(rnd.sample(range(len(srt) + 1), 2)) if len(srt) > 1 else (0, 1)
        assert mo.interval_cost_eq5(srt[a:b]) == mo.trie_cost(srt[a:b])


def test_eq6_cut_loss_and_range_minimum_rule():
    rnd = random.Random(2)
    for _ in range(40):
        fo = make_forest([random_tree(rnd, 9, 7) for _ in range(2)])
        srt = sorted(mo.trajectory_tokens(fo))
        n = len(srt)
        L = [0] + [mo.lcp(srt[i - 1], srt[i]) for i in range(1, n)]
        for t in range(1, n):
            a, b = rnd.randint(0, t - 1), rnd.randint(t, n - 1)
            W = lambda x, y: mo.trie_cost(srt[x:y + 1])                    # noqa: E731
            assert W(a, t - 1) + W(t, b) - W(a, b) == L[t]                 # Eq. 6
            assert mo.lcp(srt[a], srt[b]) == min(L[a + 1:b + 1])          # pairwise LCP = minimum adjacent LCP


def test_five_node_tree_costs_by_hand():
    # trajectories: root+A (384), root+X+B (390), root[:100]+C (300); all together 718 compact tokens
    fo = config_forest("cfg0")
    trajs = mo.trajectory_tokens(fo)
    assert sorted(map(len, trajs)) == [300, 384, 390]
    assert mo.trie_cost(trajs) == 718
    by_len = {len(t): t for t in trajs}
    assert mo.lcp(by_len[384], by_len[390]) == 256 and mo.lcp(by_len[384], by_len[300]) == 100
    assert mo.trie_cost([by_len[384], by_len[390]]) == 384 + 390 - 256
    assert mo.best_contiguous(sorted(trajs), 1, 718) == (718, 718)
    assert mo.best_contiguous(sorted(trajs), 1, 717) is None


def test_slot_schedule_rule():
    replica, slot, tail = mo.slot_schedule([5, 9, 7, 1], 2)
    # heaviest first: 9, 7 | 5, 1; second slot: 5 goes to the replica that has 7, 1 to the one that has 9
    assert slot == [1, 0, 0, 1] and replica[1] != replica[2] and replica[0] == replica[2] and replica[3] == replica[1]
    assert tail == (9 + 5, 12)


def test_eq10_closed_form_equals_the_trie_count_difference():
    """Pins both sides of Eq. 10: the brute-force definition (trie with x minus trie without x) and the printed
    closed form agree for insertion in the middle, at either end, and into an empty microbatch."""
    import random
    from test_plan_oracle import random_tree
    from workloads import make_forest
    rng = random.Random(5)
    seen_middle = seen_end = 0
    for _ in range(40):
        fo = make_forest([random_tree(rng, rng.randint(2, 10), 12) for _ in range(rng.randint(1, 2))])
        trajs = sorted(mo.trajectory_tokens(fo))
        for _ in range(6):
            k = rng.randint(0, len(trajs) - 1)
            members = sorted(rng.sample(trajs, k))
            rest = [t for t in trajs if t not in members]
            x = rng.choice(rest)
            assert mo.delta_c(members, x) == mo.delta_c_eq10(members, x)
            if members:
                if members[0] < x < members[-1]:
                    seen_middle += 1
                else:
                    seen_end += 1
    assert seen_middle > 10 and seen_end > 10
    # hand-counted: members {ab, abc... } on explicit token tuples
    a, b, c = (1, 2, 3, 4), (1, 2, 5), (1, 2, 3, 9, 9)
    assert mo.delta_c([a, b], c) == 2 and mo.delta_c([], c) == 5 and mo.delta_c([b], a) == 2
