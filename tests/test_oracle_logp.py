"""Pins of the log-probability oracle (Eqs. 17, 19, 20) against things fixed outside it."""
import numpy as np
import torch

from oracle import logp_oracle as lo
from workloads import config_forest, make_forest


def _rand(C, V, P, seed):
    rng = np.random.default_rng(seed)
    z = rng.normal(0, 2, (C, V))
    m = rng.integers(0, C, P)
    y = rng.integers(0, V, P)
    g = rng.normal(0, 1, P) * (rng.random(P) < 0.7)
    return z, m, y, g


def test_uniform_logits_closed_form():
    # all logits equal: lambda = -log V whatever the target, gradient = g (onehot - 1/V)
    C, V = 3, 17
    z = np.full((C, V), 1.25)
    m = np.array([0, 2, 2, 2]); y = np.array([5, 0, 16, 0]); g = np.array([1.0, 2.0, -0.5, 0.25])
    lam, lse = lo.mapped_logp(z, m, y)
    assert np.allclose(lam, -np.log(V), atol=1e-14)
    assert np.allclose(lse, 1.25 + np.log(V), atol=1e-14)
    dz = lo.mapped_logp_grad(z, m, y, g)
    want = np.zeros((C, V))
    want[0] = -1.0 / V; want[0, 5] += 1.0
    want[2] = -(2.0 - 0.5 + 0.25) / V; want[2, 0] += 2.25; want[2, 16] += -0.5
    assert np.allclose(dz, want, atol=1e-14)
    assert not dz[1].any()                      # a row no position maps to gets no gradient


def test_two_word_vocabulary_is_a_logistic():
    # V = 2: lambda for word 1 is log sigmoid(z1 - z0); d lambda / d z1 = 1 - sigmoid = sigmoid(z0 - z1)
    z = np.array([[0.3, -1.1], [2.0, 2.5]])
    m = np.array([0, 1]); y = np.array([1, 1])
    lam, _ = lo.mapped_logp(z, m, y)
    d = z[:, 1] - z[:, 0]
    assert np.allclose(lam, -np.log1p(np.exp(-d)), atol=1e-14)
    dz = lo.mapped_logp_grad(z, m, y, np.ones(2))
    sig = 1 / (1 + np.exp(-d))
    assert np.allclose(dz[:, 1], 1 - sig, atol=1e-14) and np.allclose(dz[:, 0], -(1 - sig), atol=1e-14)


def test_equals_torch_log_softmax_on_expanded_rows_with_autograd():
    # the semantic definition: expand to one row per position, library log_softmax, autograd through the copy
    z, m, y, g = _rand(11, 53, 40, 0)
    lam, _ = lo.mapped_logp(z, m, y)
    zt = torch.tensor(z, requires_grad=True)
    expanded = zt.index_select(0, torch.tensor(m))
    lam_t = torch.log_softmax(expanded, dim=1).gather(1, torch.tensor(y)[:, None])[:, 0]
    assert np.allclose(lam, lam_t.detach().numpy(), atol=1e-12)
    assert np.allclose(lam, lo.expanded_logp(z, m, y), atol=1e-12)
    (lam_t * torch.tensor(g)).sum().backward()
    assert np.allclose(lo.mapped_logp_grad(z, m, y, g), zt.grad.numpy(), atol=1e-12)


def test_gradient_by_central_differences():
    z, m, y, g = _rand(4, 9, 12, 1)
    dz = lo.mapped_logp_grad(z, m, y, g)
    h = 1e-6
    for c in range(4):
        for v in range(9):
            zp = z.copy(); zp[c, v] += h
            zm = z.copy(); zm[c, v] -= h
            fd = (np.dot(lo.mapped_logp(zp, m, y)[0], g) - np.dot(lo.mapped_logp(zm, m, y)[0], g)) / (2 * h)
            assert abs(fd - dz[c, v]) < 1e-8


def test_gradient_rows_sum_to_zero_and_shift_invariance():
    z, m, y, g = _rand(6, 31, 25, 2)
    dz = lo.mapped_logp_grad(z, m, y, g)
    assert np.allclose(dz.sum(axis=1), 0, atol=1e-13)
    shift = np.linspace(-3, 3, 6)[:, None]
    assert np.allclose(lo.mapped_logp(z + shift, m, y)[0], lo.mapped_logp(z, m, y)[0], atol=1e-12)
    assert np.allclose(lo.mapped_logp_grad(z + shift, m, y, g), dz, atol=1e-12)
    assert np.all(lo.mapped_logp(z, m, y)[0] < 0)                  # a log-probability


def test_shared_row_sums_independent_contributions():
    # two positions on one compact row with different targets and weights: not "one gradient times a count"
    z = np.array([[0.0, 1.0, 2.0]])
    p = np.exp(z[0]) / np.exp(z[0]).sum()
    dz = lo.mapped_logp_grad(z, np.array([0, 0]), np.array([0, 2]), np.array([3.0, -1.0]))
    assert np.allclose(dz[0], np.array([3.0, 0.0, -1.0]) - 2.0 * p, atol=1e-14)


def test_positions_of_the_five_node_tree():
    # root 256; A(128) and X(44) continue at the root's end; B(90) continues X; C(200) forks at offset 100.
    # Trajectories: root+A (384), root+X+B (390), root[:100]+C (300): 1074 positions, 3 of them terminal.
    f = config_forest("cfg0")
    C = f.n_tokens
    tok = np.arange(C) + 1000                                     # id = canonical index + 1000
    m, y, ptr = lo.positions(f, tok)
    assert ptr.tolist() == [0, 383, 383 + 389, 383 + 389 + 299]
    assert len(m) == 1074 - 3
    base = f.token_base()                                         # nodes in input order: root, A, X, B, C
    # the root's last token (canonical 255) is followed by A's first token in one trajectory, X's in another
    at = np.nonzero(m == 255)[0]
    assert sorted(y[at].tolist()) == [1000 + base[1], 1000 + base[2]]
    # canonical token 99 (offset 99 of the root) is followed by root[100] twice and by C's first token once
    at = np.nonzero(m == 99)[0]
    assert sorted(y[at].tolist()) == sorted([1100, 1100, 1000 + base[4]])
    # inside a node the next token is the next canonical token
    inner = np.nonzero(m == base[3] + 5)[0]
    assert y[inner].tolist() == [1000 + base[3] + 6]
    q = lo.multiplicity(C, f)
    assert q[:100].tolist() == [3] * 100 and q[100:256].tolist() == [2] * 156 and q[256:].tolist() == [1] * (C - 256)
    assert q.sum() == 1074


def test_positions_single_token_trajectory_has_none():
    f = make_forest([([-1], [0], [1])])
    m, y, ptr = lo.positions(f, np.array([7]))
    assert len(m) == 0 and ptr.tolist() == [0, 0]
