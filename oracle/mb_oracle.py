"""Oracle pieces for prefix-aware microbatch planning (Section 3.2, Eqs. 4-10).  TEST INFRASTRUCTURE ONLY.

The planner itself is a search with heuristics, so there is no single "right" plan to compare with.  What has a
plain definition is written out here and used to check the planner:

* ``trajectory_tokens``   every root-to-leaf trajectory as a tuple of canonical token ids (its token sequence,
                          since a compact token is one distinct prefix node);
* ``trie_cost``           the compact work of a set of trajectories: the number of distinct non-empty prefixes
                          (the unique token nodes of the merged trie, the definition behind Eq. 5);
* ``lcp``                 longest common prefix of two trajectories;
* ``best_contiguous``     brute force over all ways to cut a sequence of trajectories into K contiguous, capacity-
                          feasible groups: least total work, ties by least maximum single work (Eq. 9 and its
                          tie-break);
* ``slot_schedule``       the replica/slot assignment rule and the objective triple of Eq. 4;
* ``check_plan``          the guarantees every returned plan must have (exact coverage, capacity, K mod D = 0,
                          K / D microbatches per replica).

Pins (tests/test_oracle_mb.py): Eq. 5 and Eq. 6 against the trie count on random forests, the range-minimum rule
for pairwise LCP, hand-counted costs on the five-node tree.
"""
import itertools

import numpy as np

from .la_oracle import trajectories


def trajectory_tokens(forest):
    """List of tuples of canonical token ids, one per trajectory, in the order of la_oracle.trajectories."""
    ptr, rows = trajectories(forest)
    return [tuple(int(r) for r in rows[ptr[i]:ptr[i + 1]]) for i in range(len(ptr) - 1)]


def lcp(a, b):
    n = 0
    for x, y in zip(a, b):
        if x != y:
            break
        n += 1
    return n


def trie_cost(trajs):
    """Unique token nodes of the trie that merges the given trajectories."""
    nodes = set()
    for t in trajs:
        for i in range(1, len(t) + 1):
            nodes.add(t[:i])
    return len(nodes)


def interval_cost_eq5(trajs_sorted):
    """Eq. 5 on trajectories already in lexicographic (trie depth-first) order."""
    if not trajs_sorted:
        return 0
    c = len(trajs_sorted[0])
    for p, x in zip(trajs_sorted, trajs_sorted[1:]):
        c += len(x) - lcp(p, x)
    return c


def best_contiguous(trajs_sorted, K, T):
    """(total work, max single work) of the best cut into K contiguous non-empty groups with work <= T, or None."""
    n = len(trajs_sorted)
    best = None
    for cuts in itertools.combinations(range(1, n), K - 1):
        bounds = (0,) + cuts + (n,)
        works = [trie_cost(trajs_sorted[a:b]) for a, b in zip(bounds, bounds[1:])]
        if max(works) > T:
            continue
        key = (sum(works), max(works))
        if best is None or key < best:
            best = key
    return best


def slot_schedule(works, D):
    """Replica and slot of every microbatch: sort by work (heaviest first), every D consecutive ones form a slot,
    inside a slot the heavier microbatch goes to the replica with less cumulative work so far (ties: lower index).
    Returns (replica[K], slot[K], objective tail (sum_j max_d w, max_d sum_j w))."""
    works = np.asarray(works, dtype=np.int64)
    K = len(works)
    assert K % D == 0
    order = sorted(range(K), key=lambda i: (-works[i], i))
    load = [0] * D
    replica, slot = [0] * K, [0] * K
    slot_crit = 0
    for j in range(K // D):
        group = order[j * D:(j + 1) * D]
        free = sorted(range(D), key=lambda d: (load[d], d))
        for mb, d in zip(group, free):
            replica[mb], slot[mb] = d, j
        for mb in group:
            load[replica[mb]] += int(works[mb])
        slot_crit += int(max(works[mb] for mb in group))
    return replica, slot, (slot_crit, max(load))


def check_plan(trajs, mb_of_traj, replica, slot, D, T):
    """Asserts the guarantees of Section 3.2 "Plan selection and guarantees"; returns the objective triple J."""
    mb_of_traj = np.asarray(mb_of_traj)
    K = int(mb_of_traj.max()) + 1 if len(mb_of_traj) else 0
    assert len(mb_of_traj) == len(trajs) and mb_of_traj.min() >= 0          # exact coverage
    assert K % D == 0
    works = []
    for m in range(K):
        members = [trajs[i] for i in np.nonzero(mb_of_traj == m)[0]]
        assert members, "empty microbatch"
        w = trie_cost(members)
        assert w <= T, (m, w, T)
        works.append(w)
    per_replica = np.bincount(np.asarray(replica), minlength=D)
    assert (per_replica == K // D).all()
    for j in range(K // D):
        in_slot = [m for m in range(K) if slot[m] == j]
        assert len(in_slot) == D and sorted(replica[m] for m in in_slot) == list(range(D))
    slot_crit = sum(max(works[m] for m in range(K) if slot[m] == j) for j in range(K // D))
    load = [sum(works[m] for m in range(K) if replica[m] == d) for d in range(D)]
    return (sum(works), slot_crit, max(load)), works


def delta_c(members, x):
    """The compact-work increase that Eq. 10 gives in closed form, here from its definition: unique token nodes of the
    microbatch's trie with the candidate trajectory minus without it."""
    return trie_cost(list(members) + [x]) - trie_cost(list(members))


def delta_c_eq10(members_sorted, x):
    """Eq. 10 itself: members in lexicographic order, p / q the neighbours of x at its insertion position; a missing
    neighbour's terms are left out."""
    import bisect
    pos = bisect.bisect_left(members_sorted, x)
    p = members_sorted[pos - 1] if pos > 0 else None
    q = members_sorted[pos] if pos < len(members_sorted) else None
    d = len(x)
    if p is not None:
        d -= lcp(p, x)
    if q is not None:
        d -= lcp(x, q)
    if p is not None and q is not None:
        d += lcp(p, q)
    return d


def greedy_orders(trajs_sorted):
    """The four processing orders of the greedy as index lists into the lexicographically sorted trajectories:
    ascending, descending, descending length, descending unique-suffix score u(x) = |x| - max(LCP(p_x, x), LCP(x, q_x))
    with p_x, q_x the global neighbours (ties keep lexicographic order)."""
    n = len(trajs_sorted)
    asc = list(range(n))
    u = []
    for i, x in enumerate(trajs_sorted):
        left = lcp(trajs_sorted[i - 1], x) if i > 0 else 0
        right = lcp(x, trajs_sorted[i + 1]) if i + 1 < n else 0
        u.append(len(x) - max(left, right))
    return [asc, asc[::-1], sorted(asc, key=lambda i: -len(trajs_sorted[i])), sorted(asc, key=lambda i: -u[i])]


def greedy_place(trajs_sorted, order, T, best_fit):
    """Placement pass of the trie-aware greedy with the work increase taken from the trie count (delta_c): each
    trajectory goes to the capacity-feasible microbatch with the largest work after insertion (best-fit) or the
    largest shared amount |x| - delta (max-shared), the earliest on ties, else a new microbatch.
    Returns the steps [(trajectory index, microbatch, created, delta)]."""
    bins = []
    steps = []
    for i in order:
        x = trajs_sorted[i]
        best, best_key, best_d = None, -1, 0
        for b, members in enumerate(bins):
            work = trie_cost(members)
            d = delta_c(members, x)
            if work + d > T:
                continue
            key = work + d if best_fit else len(x) - d
            if key > best_key:
                best, best_key, best_d = b, key, d
        created = best is None
        if created:
            bins.append([])
            best, best_d = len(bins) - 1, len(x)
        bins[best].append(x)
        steps.append((i, best, int(created), best_d))
    return steps
