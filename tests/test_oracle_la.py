"""Pins for the fp64 token-recurrence oracle (oracle/la_oracle.c): closed forms, the dense
decay-masked matmul form, finite differences, autograd of the dense form, the depth-first
compact evaluation, and invariance to how dO is split over copies of a shared row."""
import numpy as np
import pytest
import torch

from oracle import la_oracle as lo
from workloads import make_forest, config_forest, make_inputs, CONFIGS


def rand_traj(T, dk, dv, seed):
    rng = np.random.default_rng(seed)
    q = rng.normal(size=(T, dk)) / 4
    k = rng.normal(size=(T, dk)) / 4
    v = rng.normal(size=(T, dv))
    g = np.log(1 / (1 + np.exp(-rng.normal(1.0, 1.0, size=T))))
    dO = rng.normal(size=(T, dv))
    return q, k, v, g, dO


def dense_form(q, k, v, g):
    """O = ((Q K^T) * D) V with D_tj = exp(sum_{j<tau<=t} g_tau) for j <= t (textbook masked form)."""
    b = np.cumsum(g)
    D = np.tril(np.exp(b[:, None] - b[None, :]))
    return ((q @ k.T) * D) @ v


def test_closed_form_cumsum():
    # g = 0, d_k = d_v = 1, q = k = 1  =>  o = cumulative sum of v
    T = 257
    v = np.random.default_rng(0).normal(size=(T, 1))
    o = lo.traj_fwd(np.ones((T, 1)), np.ones((T, 1)), v, np.zeros(T))
    np.testing.assert_allclose(o[:, 0], np.cumsum(v[:, 0]), rtol=0, atol=1e-12)


def test_closed_form_geometric():
    # constant decay gamma: o_t = sum_j gamma^(t-j) v_j, checked against the O(T^2) sum
    T, gamma = 150, 0.9
    v = np.random.default_rng(1).normal(size=(T, 1))
    o = lo.traj_fwd(np.ones((T, 1)), np.ones((T, 1)), v, np.full(T, np.log(gamma)))
    ref = np.array([sum(gamma ** (t - j) * v[j, 0] for j in range(t + 1)) for t in range(T)])
    np.testing.assert_allclose(o[:, 0], ref, rtol=1e-12, atol=1e-12)
    # all-ones v: partial geometric series (1 - gamma^(t+1)) / (1 - gamma)
    o1 = lo.traj_fwd(np.ones((T, 1)), np.ones((T, 1)), np.ones((T, 1)), np.full(T, np.log(gamma)))
    np.testing.assert_allclose(o1[:, 0], (1 - gamma ** np.arange(1, T + 1)) / (1 - gamma), rtol=1e-12)


def test_outer_product_orientation():
    # one token: S = k^T v, o = q S = (q.k) v ; catches a transposed state or swapped k/v
    q = np.array([[1.0, 2.0, 3.0]])
    k = np.array([[0.5, -1.0, 2.0]])
    v = np.array([[7.0, 11.0]])
    o = lo.traj_fwd(q, k, v, np.array([-0.3]))
    np.testing.assert_allclose(o, (q @ k.T) * v, rtol=1e-14)


@pytest.mark.parametrize("T,dk,dv", [(1, 3, 2), (37, 5, 4), (203, 8, 16)])
def test_forward_equals_dense_form(T, dk, dv):
    q, k, v, g, _ = rand_traj(T, dk, dv, T)
    np.testing.assert_allclose(lo.traj_fwd(q, k, v, g), dense_form(q, k, v, g), rtol=1e-10, atol=1e-11)


@pytest.mark.parametrize("T,dk,dv", [(1, 2, 2), (23, 3, 2), (205, 4, 3)])
def test_backward_equals_autograd_of_dense_form(T, dk, dv):
    q, k, v, g, dO = rand_traj(T, dk, dv, 100 + T)
    tq, tk, tv, tg = (torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (q, k, v, g))
    b = torch.cumsum(tg, 0)
    D = torch.tril(torch.exp(b[:, None] - b[None, :]))
    o = ((tq @ tk.T) * D) @ tv
    (o * torch.tensor(dO)).sum().backward()
    dq, dk_, dv_, dg = lo.traj_bwd(q, k, v, g, dO)
    for mine, ref in ((dq, tq.grad), (dk_, tk.grad), (dv_, tv.grad), (dg, tg.grad)):
        np.testing.assert_allclose(mine, ref.numpy(), rtol=1e-9, atol=1e-10)


def test_backward_finite_differences():
    T, dk, dv = 11, 3, 2
    q, k, v, g, dO = rand_traj(T, dk, dv, 7)
    dq, dk_, dv_, dg = lo.traj_bwd(q, k, v, g, dO)

    def loss():
        return float((lo.traj_fwd(q, k, v, g) * dO).sum())

    h = 1e-6
    for x, gx in ((q, dq), (k, dk_), (v, dv_), (g, dg)):
        it = np.nditer(x, flags=["multi_index"])
        for _ in it:
            i = it.multi_index
            old = x[i]
            x[i] = old + h
            up = loss()
            x[i] = old - h
            dn = loss()
            x[i] = old
            assert abs((up - dn) / (2 * h) - gx[i]) < 1e-7, (i, (up - dn) / (2 * h), gx[i])


def small_forest():
    # root (10 tokens) with a fork inside it (at 4), two forks at its end, a grandchild fork inside a child
    par = [-1, 0, 0, 0, 2, 2]
    off = [0, 4, 10, 10, 3, 5]
    ln = [10, 6, 5, 7, 4, 2]
    return make_forest([(par, off, ln), ([-1], [0], [5])])


def test_trajectories_map():
    fo = small_forest()
    ptr, rows = lo.trajectories(fo)
    # leaves: node1 (4+6), node3 (10+7), node4 (10+3+4), node5 = end of node2 is continued by node5 (off 5 == len 5)
    lens = np.diff(ptr).tolist()
    assert lens == [10, 17, 17, 17, 5]
    assert rows[ptr[0]:ptr[1]].tolist() == [0, 1, 2, 3] + list(range(10, 16))
    # node4 forks at offset 3 of node2 (tokens 16..20): path = root(0..9) + node2[0:3] + node4
    assert rows[ptr[2]:ptr[3]].tolist() == list(range(10)) + [16, 17, 18] + list(range(28, 32))
    assert rows[ptr[3]:ptr[4]].tolist() == list(range(10)) + list(range(16, 21)) + [32, 33]
    assert rows[ptr[4]:ptr[5]].tolist() == list(range(34, 39))


def test_forest_matches_compact_dfs_and_copies_agree():
    fo = small_forest()
    inp = make_inputs(fo.n_tokens, 2, 3, 4, "fp32", 5)
    res = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"])
    dfs = lo.compact_dfs_fwd(fo, inp["q"], inp["k"], inp["v"], inp["g"])
    assert res["copy_gap"] < 1e-12
    np.testing.assert_allclose(res["o"], dfs, rtol=1e-12, atol=1e-13)


def test_cfg0_compact_equals_trajectorywise():
    fo = config_forest("cfg0")
    cfg = CONFIGS["cfg0"]
    inp = make_inputs(fo.n_tokens, cfg["H"], cfg["dk"], cfg["dv"], cfg["dtype"], cfg["seed"])
    res = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"])
    assert res["S"] == 1074 and fo.n_tokens == 718
    assert res["copy_gap"] < 1e-12
    np.testing.assert_allclose(res["o"], lo.compact_dfs_fwd(fo, inp["q"], inp["k"], inp["v"], inp["g"]),
                               rtol=1e-12, atol=1e-13)


def test_forest_gradients_by_finite_differences_on_shared_prefix():
    fo = small_forest()
    inp = {n: x.double().numpy() for n, x in make_inputs(fo.n_tokens, 1, 2, 2, "fp32", 9).items()}
    res = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])

    def loss():
        return float((lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"])["o"] * inp["dO"]).sum())

    h = 1e-6
    rng = np.random.default_rng(0)
    for name, gname in (("q", "dq"), ("k", "dk"), ("v", "dv"), ("g", "dg")):
        x = inp[name]
        # rows 0..3 are shared by all five trajectories of the first tree, 16..18 by two
        for row in [0, 3, 5, 12, 17, 20, 29, 33, 36]:
            idx = (row, 0) + ((int(rng.integers(x.shape[2])),) if x.ndim == 3 else ())
            old = x[idx]
            x[idx] = old + h
            up = loss()
            x[idx] = old - h
            dn = loss()
            x[idx] = old
            assert abs((up - dn) / (2 * h) - res[gname][idx]) < 1e-6, (name, idx)


def test_gradients_do_not_depend_on_how_dO_is_split():
    # all of dO_c on the first copy instead of dO_c / multiplicity on each: same compact gradients
    fo = small_forest()
    inp = {n: x.double().numpy() for n, x in make_inputs(fo.n_tokens, 1, 3, 2, "fp32", 11).items()}
    res = lo.forest_eval(fo, inp["q"], inp["k"], inp["v"], inp["g"], inp["dO"])
    ptr, rows = res["traj_ptr"], res["traj_rows"]
    acc = {n: np.zeros_like(res[n]) for n in ("dq", "dk", "dv", "dg")}
    seen = set()
    for x in range(len(ptr) - 1):
        r = rows[ptr[x]:ptr[x + 1]]
        dO = np.stack([inp["dO"][c, 0] if c not in seen else np.zeros(2) for c in r])
        seen.update(r.tolist())
        dq, dk_, dv_, dg = lo.traj_bwd(inp["q"][r, 0], inp["k"][r, 0], inp["v"][r, 0], inp["g"][r, 0], dO)
        np.add.at(acc["dq"][:, 0], r, dq)
        np.add.at(acc["dk"][:, 0], r, dk_)
        np.add.at(acc["dv"][:, 0], r, dv_)
        np.add.at(acc["dg"][:, 0], r, dg)
    for n in acc:
        np.testing.assert_allclose(acc[n], res[n], rtol=1e-10, atol=1e-12)
