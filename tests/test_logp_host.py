"""Host side of the log-probability step through the C ABI: positions and the row CSR against the oracle."""
import random

import numpy as np
import pytest

import paper_2608_28158_b200 as H
from oracle import logp_oracle as lo
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _positions(fo, tok, rot=None):
    return H.harts_logp_positions(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, tok, rot)


@pytest.mark.parametrize("name", ["cfg0", "cfg0b", "cfg1", "cfg2"])
def test_positions_equal_the_oracle(name):
    fo = config_forest(name)
    tok = np.random.default_rng(5).integers(0, 157184, fo.n_tokens).astype(np.int32)
    m, y, tp = _positions(fo, tok)
    m0, y0, tp0 = lo.positions(fo, tok)
    assert np.array_equal(m, m0) and np.array_equal(y, y0) and np.array_equal(tp, tp0)


def test_positions_random_forests_and_row_map():
    rnd = random.Random(11)
    for _ in range(300):
        fo = make_forest([random_tree(rnd, rnd.randint(1, 9), 40) for _ in range(rnd.randint(1, 3))])
        tok = np.arange(fo.n_tokens, dtype=np.int32) * 3 + 1
        m0, y0, tp0 = lo.positions(fo, tok)
        m, y, tp = _positions(fo, tok)
        assert np.array_equal(m, m0) and np.array_equal(y, y0) and np.array_equal(tp, tp0)
        plan = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 8)
        m2, y2, _ = _positions(fo, tok, plan.row_of_token)
        assert np.array_equal(m2, plan.row_of_token[m0]) and np.array_equal(y2, y0)


def test_csr_groups_positions_by_row_in_order():
    rng = np.random.default_rng(3)
    m = rng.integers(0, 50, 400).astype(np.int32)
    ptr, pos = H.harts_logp_csr(60, m)
    assert ptr[0] == 0 and ptr[-1] == 400 and len(ptr) == 61
    for c in range(60):
        assert pos[ptr[c]:ptr[c + 1]].tolist() == np.nonzero(m == c)[0].tolist()


def test_multiplicity_counts_the_trajectories_through_every_token():
    """Eq. 20 against the oracle (expansion of every trajectory) and two closed forms: a root token lies on every
    trajectory of its tree, and the multiplicities sum to the trajectory-wise token count."""
    rnd = random.Random(12)
    forests = [config_forest(n) for n in ("cfg0", "cfg0b", "cfg1")]
    forests += [make_forest([random_tree(rnd, rnd.randint(1, 12), 30) for _ in range(rnd.randint(1, 3))]) for _ in range(200)]
    for fo in forests:
        arrs = (fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len)
        want = lo.multiplicity(fo.n_tokens, fo)
        got = H.harts_logp_multiplicity(*arrs)
        assert np.array_equal(got, want)
        m0, _, tp0 = lo.positions(fo, np.zeros(fo.n_tokens, np.int32))
        assert int(got.sum()) == len(m0) + len(tp0) - 1      # non-terminal positions + one terminal per trajectory
        plan = H.harts_la_plan(*arrs, 8)
        phys = H.harts_logp_multiplicity(*arrs, row_of_token=plan.row_of_token, n_rows=fo.n_tokens + 3)
        assert np.array_equal(phys[plan.row_of_token], want) and int(phys.sum()) == int(want.sum())
    # five-node tree of cfg0: the root's 256 tokens are on all three trajectories
    fo = config_forest("cfg0")
    got = H.harts_logp_multiplicity(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len)
    assert set(got[:100].tolist()) == {3}


def test_errors():
    with pytest.raises(H.HartsError):
        H.harts_logp_csr(5, np.array([0, 5], np.int32))
    with pytest.raises(H.HartsError):
        H.harts_logp_positions([0, 2], [-1, 0], [0, 9], [4, 4], np.zeros(8, np.int32))   # fork beyond the parent
    ptr, pos = H.harts_logp_csr(3, np.zeros(0, np.int32))
    assert ptr.tolist() == [0, 0, 0, 0] and len(pos) == 0
    fo = config_forest("cfg0")
    with pytest.raises(H.HartsError):                       # fewer rows than compact tokens
        H.harts_logp_multiplicity(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, n_rows=10)
