"""harts_attn_index (C ABI, host): pieces, ancestor rows and descendant lists against the oracle's paths."""
import random

import numpy as np
import pytest

import paper_2608_28158_b200 as H
from oracle import attn_oracle as ao
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _check(fo, rot):
    ix = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot)
    C = fo.n_tokens
    row = np.arange(C) if rot is None else np.asarray(rot, np.int64)
    paths = ao.paths(fo)
    assert ix.n_rows == C and int(ix.piece_len.sum()) == C
    assert np.array_equal(ix.piece_row0, np.concatenate([[0], np.cumsum(ix.piece_len)[:-1]]))
    piece_of = np.repeat(np.arange(ix.n_pieces), ix.piece_len)
    for t in range(C):
        r = row[t]
        p = piece_of[r]
        seen = []
        for j in range(ix.anc_ptr[p], ix.anc_ptr[p + 1]):
            seen.extend(range(ix.anc_row0[j], ix.anc_row0[j] + ix.anc_len[j]))
        seen.extend(range(ix.piece_row0[p], r + 1))
        assert seen == row[paths[t]].tolist()                       # exactly the path, in order
    # descendants: q is listed under p iff p is among q's ancestors
    for p in range(ix.n_pieces):
        want = [q for q in range(ix.n_pieces) if p in _anc(ix, q)]
        assert ix.desc_piece[ix.desc_ptr[p]:ix.desc_ptr[p + 1]].tolist() == want
    # work lists: every tile of every piece once
    tiles = sorted((int(p), int(t)) for p in range(ix.n_pieces) for t in range((ix.piece_len[p] + 127) // 128))
    assert sorted(map(tuple, ix.q_item.reshape(-1, 2).tolist())) == tiles
    assert sorted(map(tuple, ix.kv_item.reshape(-1, 2).tolist())) == tiles


def _anc(ix, q):
    out, a = [], ix.piece_parent[q]
    while a >= 0:
        out.append(int(a)); a = ix.piece_parent[a]
    return out


@pytest.mark.parametrize("name", ["cfg0", "cfg0b"])
def test_index_of_the_small_configurations(name):
    fo = config_forest(name)
    plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64)
    _check(fo, None)
    _check(fo, plan.row_of_token)


def test_index_of_random_forests():
    rnd = random.Random(8)
    for _ in range(40):
        fo = make_forest([random_tree(rnd, 8, 12) for _ in range(rnd.randint(1, 3))])
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 4)
        _check(fo, plan.row_of_token)


def test_errors():
    with pytest.raises(H.HartsError):
        H.harts_attn_index([0, 2], [-1, 0], [0, 3], [2, 2])
    with pytest.raises(H.HartsError):
        H.harts_attn_index([0, 1], [-1], [0], [3], [0, 0, 1])
