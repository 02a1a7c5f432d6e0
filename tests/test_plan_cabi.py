"""harts_la_plan (C++) against the pure-Python planner, bit for bit; error behaviour; exported symbols."""
import ctypes
import os
import random
import re

import numpy as np
import pytest

import paper_2608_28158_b200 as H
from oracle import plan_oracle as po
from workloads import make_forest, config_forest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def plan_of(fo, chunk=64):
    return H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, chunk)


def assert_same_plan(fo, chunk):
    mine, ref = plan_of(fo, chunk), po.plan_forest(fo, chunk)
    assert (mine.n_rounds, mine.n_rows, mine.n_replay, mine.n_seq, mine.n_slots) == \
           (ref.n_rounds, ref.C, ref.R, ref.n_seq, ref.n_slots)
    for name in po.Plan.FIELDS:
        a, b = getattr(mine, name), getattr(ref, name)
        if name == "seq_own_begin":
            a = a[:-1]
        if name == "rg_ptr" and len(b) == 1:
            a = a[:1]
        assert np.array_equal(a, b), name
    return mine


@pytest.mark.parametrize("name", ["cfg0", "cfg0b", "cfg1", "cfg2", "cfg3", "cfg4"])
def test_config_plans_bit_exact(name):
    p = assert_same_plan(config_forest(name), 64)
    if name == "cfg0":
        assert (p.n_rounds, p.C, p.R, p.n_seq, p.n_slots) == (2, 718, 36, 3, 2)


def random_tree(rng, max_nodes, max_len):
    n = rng.randint(1, max_nodes)
    par, off, ln = [-1], [0], [rng.randint(1, max_len)]
    for i in range(1, n):
        p = rng.randint(0, i - 1)
        par.append(p)
        off.append(rng.randint(1, ln[p]))
        ln.append(rng.randint(1, max_len))
    return par, off, ln


def test_random_forests_bit_exact():
    rng = random.Random(7)
    for _ in range(3000):
        B = rng.choice([1, 2, 4, 8, 64])
        trees = [random_tree(rng, rng.choice([3, 9, 30]), rng.choice([3, 3 * B + 1])) for _ in range(rng.randint(1, 4))]
        assert_same_plan(make_forest(trees), B)


def test_deep_chain_does_not_overflow_the_stack():
    # 20000 nested forks: every node forks one token before its parent's end
    n = 20000
    par = [-1] + list(range(n - 1))
    off = [0] + [2] * (n - 1)
    ln = [3] * n
    p = plan_of(make_forest([(par, off, ln)]), 64)
    assert p.n_rows == 3 * n and p.n_seq == n


def test_linear_time_scaling():
    import time
    rng = random.Random(3)

    def timed(n):
        trees = [random_tree(rng, n, 200)]
        fo = make_forest(trees)
        t0 = time.perf_counter()
        plan_of(fo, 64)
        return (time.perf_counter() - t0) / fo.n_nodes
    timed(2000)
    small = min(timed(20000) for _ in range(3))
    large = min(timed(200000) for _ in range(3))
    assert large < 6 * small      # per-node cost stays flat (allowing for cache effects and the sorts)


def _raw_plan(ptr, par, off, ln, chunk, out_null=False):
    arrs = [np.asarray(a, dtype=np.int32) for a in (ptr, par, off, ln)]
    h = ctypes.c_void_p()
    i32p = ctypes.POINTER(ctypes.c_int32)
    rc = H.lib.harts_la_plan(len(arrs[0]) - 1, *(a.ctypes.data_as(i32p) for a in arrs), chunk,
                             None if out_null else ctypes.byref(h))
    if h.value:
        H.lib.harts_la_plan_free(h)
    return rc


def test_malformed_forests_are_rejected():
    ok = ([0, 2], [-1, 0], [0, 3], [5, 4])
    assert _raw_plan(*ok, 64) == 0
    assert _raw_plan(*ok, 0) == -1                                   # chunk < 1
    assert _raw_plan(*ok, 64, out_null=True) == -1
    assert _raw_plan([0, 2], [-1, 0], [0, 6], [5, 4], 64) == -1      # fork offset past the parent's end
    assert _raw_plan([0, 2], [-1, 0], [0, 0], [5, 4], 64) == -1      # fork offset 0 on a child
    assert _raw_plan([0, 2], [-1, 1], [0, 3], [5, 4], 64) == -1      # parent not before the child
    assert _raw_plan([0, 2], [-1, 0], [0, 3], [5, 0], 64) == -1      # empty node
    assert _raw_plan([0, 2], [0, 0], [0, 3], [5, 4], 64) == -1       # root with a parent
    assert _raw_plan([0, 0], [], [], [], 64) == -1                   # empty tree
    assert H.harts_la_strerror(-3).startswith("unsupported")


def test_single_path_is_one_round():
    p = plan_of(make_forest([([-1, 0, 1], [0, 10, 7], [10, 7, 300])]), 64)
    assert (p.n_rounds, p.n_seq, p.n_replay, p.n_slots, p.n_chunks) == (1, 1, 0, 0, 5)
    assert p.row_of_token.tolist() == list(range(317))


def test_work_order_is_a_permutation_inside_every_round_longest_first():
    for name in ("cfg1", "cfg2", "cfg4"):
        p = plan_of(config_forest(name), 64)
        n = np.diff(p.seq_chunk_ptr)
        for r in range(p.n_rounds):
            lo, hi = int(p.round_seq_ptr[r]), int(p.round_seq_ptr[r + 1])
            order = p.seq_order[lo:hi]
            assert sorted(order.tolist()) == list(range(lo, hi))
            assert (np.diff(n[order]) <= 0).all()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "harts_la.h")).read()
    header += open(os.path.join(ROOT, "include", "harts_logp.h")).read()
    header += open(os.path.join(ROOT, "include", "harts_conv.h")).read()
    header += open(os.path.join(ROOT, "include", "harts_attn.h")).read()
    header += open(os.path.join(ROOT, "include", "harts_mb.h")).read()
    names = set(re.findall(r"\b(harts_(?:la|logp|conv|attn|mb)_\w+)\s*\(", header))
    assert {"harts_mb_plan", "harts_mb_plan_free", "harts_mb_plan_view", "harts_mb_extract"} <= names
    assert {"harts_attn_index", "harts_attn_fwd", "harts_attn_bwd"} <= names
    assert {"harts_conv_index", "harts_conv_fwd", "harts_conv_bwd", "harts_conv_scratch_bytes"} <= names
    assert {"harts_la_plan", "harts_la_fwd", "harts_la_bwd", "harts_logp_fwd", "harts_logp_bwd",
            "harts_logp_positions", "harts_logp_csr", "harts_logp_fwd_shard", "harts_logp_combine"} <= names
    for n in names:
        assert hasattr(H.lib, n), n


def test_expand_matches_the_oracles_semantic_map():
    """harts_la_expand (the trajectory-wise view behind the C ABI) against the oracle's own enumeration of the
    root-to-leaf trajectories and of the map m of Eq. 3: same trajectories, same order, same source tokens."""
    import random
    from oracle import la_oracle as lo
    from test_plan_oracle import random_tree
    rnd = random.Random(31)
    cases = [config_forest("cfg0"), config_forest("cfg0b"), config_forest("cfg1")]
    cases += [make_forest([random_tree(rnd, rnd.randint(1, 12), 30) for _ in range(rnd.randint(1, 4))]) for _ in range(200)]
    for fo in cases:
        lens, src = H.harts_la_expand(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len)
        ptr, rows = lo.trajectories(fo)
        assert np.array_equal(np.diff(ptr), lens) and np.array_equal(rows, src)
    with pytest.raises(H.HartsError):
        H.harts_la_expand([0, 2], [-1, 0], [0, 9], [3, 2])          # fork offset beyond the parent
