"""harts_conv_index (C ABI, host) against the oracle's predecessor table."""
import random

import numpy as np
import pytest

import paper_2608_28158_b200 as H
from oracle import conv_oracle as co
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _check(fo, rot):
    prev, nxt, cptr, crow = H.harts_conv_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot)
    pred = co.predecessors(fo)
    C = fo.n_tokens
    row = np.arange(C) if rot is None else np.asarray(rot, np.int64)
    want = np.where(pred >= 0, row[np.maximum(pred, 0)], -1)
    assert np.array_equal(prev[row], want)
    assert cptr[0] == 0 and cptr[-1] == C - fo.n_trees == len(crow)
    inv = np.empty(C, np.int64); inv[row] = np.arange(C)
    for r in range(C):                                # children of a row: exactly the tokens whose predecessor it is
        kids = crow[cptr[r]:cptr[r + 1]]
        assert inv[kids].tolist() == np.nonzero(pred == inv[r])[0].tolist()
        assert nxt[r] == (-1 if len(kids) == 0 else kids[0] if len(kids) == 1 else -2)


@pytest.mark.parametrize("name", ["cfg0", "cfg0b", "cfg1"])
def test_index_tables_of_the_configurations(name):
    fo = config_forest(name)
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    _check(fo, None)
    _check(fo, plan.row_of_token)


def test_index_tables_of_random_forests():
    rnd = random.Random(4)
    for _ in range(100):
        fo = make_forest([random_tree(rnd, 8, 12) for _ in range(rnd.randint(1, 3))])
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 4)
        _check(fo, plan.row_of_token)


def test_errors():
    with pytest.raises(H.HartsError):
        H.harts_conv_index([0, 2], [-1, 0], [0, 3], [2, 2])            # fork beyond the parent
    with pytest.raises(H.HartsError):
        H.harts_conv_index([0, 1], [-1], [0], [3], [0, 0, 1])          # not a permutation
    assert H.harts_conv_scratch_bytes(64, 4) == 2048 * 64 * 4 * 4
    with pytest.raises(H.HartsError):
        H.harts_conv_scratch_bytes(60, 4)
