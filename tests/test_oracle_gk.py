"""Pins of the per-channel-decay oracle (the Diag(gamma) term of Eq. 1, Section 2.2) against things it does not
compute itself: the scalar-gate oracle when all channels decay alike, a closed form, the dense per-channel
decay-masked form evaluated with library routines (and its fp64 autograd), central finite differences."""
import numpy as np
import torch

from oracle import gk_oracle as go
from oracle import la_oracle as lo
from workloads import config_forest, make_forest


def _rand(C, H, dk, dv, seed):
    rng = np.random.default_rng(seed)
    q, k = rng.normal(size=(2, C, H, dk)) / np.sqrt(dk)
    v, dO = rng.normal(size=(2, C, H, dv))
    g = -np.log1p(np.exp(-rng.normal(3.0, 1.0, size=(C, H, dk))))        # logsigmoid(N(3,1))
    return q, k, v, g, dO


def test_equal_channels_reduce_to_the_scalar_gate_oracle():
    fo = config_forest("cfg0b")
    q, k, v, g, dO = _rand(fo.n_tokens, 2, 5, 3, 0)
    g = np.repeat(g[:, :, :1], 5, axis=2)
    a = go.forest_eval(fo, q, k, v, g, dO)
    b = lo.forest_eval(fo, q, k, v, g[:, :, 0], dO)
    assert a["copy_gap"] < 1e-12
    for n in ("o", "dq", "dk", "dv"):
        np.testing.assert_allclose(a[n], b[n], rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(a["dg"].sum(axis=2), b["dg"], rtol=1e-11, atol=1e-13)   # the scalar gate feeds every channel


def test_closed_form_constant_gates_two_channels():
    # d_v = 1, q = k = 1, v = 1, channel i decays by gamma_i per token: o_t = sum_i sum_{j<=t} gamma_i^(t-j)
    T, gam = 12, np.array([0.5, 0.9])
    o = go.traj_fwd(np.ones((T, 2)), np.ones((T, 2)), np.ones((T, 1)), np.tile(np.log(gam), (T, 1)))
    want = np.array([sum((1 - gi ** (t + 1)) / (1 - gi) for gi in gam) for t in range(T)])
    np.testing.assert_allclose(o[:, 0], want, rtol=1e-13)
    # a channel with g = -inf-like forgets everything but the current token; the other with g = 0 is a cumulative sum
    o = go.traj_fwd(np.ones((T, 2)), np.ones((T, 2)), np.arange(1.0, T + 1)[:, None], np.tile([-700.0, 0.0], (T, 1)))
    np.testing.assert_allclose(o[:, 0], np.arange(1.0, T + 1) + np.cumsum(np.arange(1.0, T + 1)), rtol=1e-13)


def _dense(q, k, v, g):
    """o_t = sum_{j<=t} (sum_i q_t[i] k_j[i] exp(B_t[i] - B_j[i])) v_j with B the running sum of g: one trajectory."""
    B = torch.cumsum(g, dim=0)
    decay = torch.exp(B[:, None, :] - B[None, :, :])                       # [t, j, i]
    A = torch.einsum("ti,ji,tji->tj", q, k, decay)
    A = A * torch.tril(torch.ones_like(A))
    return A @ v


def test_dense_per_channel_form_and_its_autograd():
    T, dk, dv = 37, 6, 4
    q, k, v, g, dO = (torch.tensor(a[:, 0], dtype=torch.float64, requires_grad=True) for a in _rand(T, 1, dk, dv, 3))
    o = _dense(q, k, v, g)
    (o * dO.detach()).sum().backward()
    args = [a.detach().numpy() for a in (q, k, v, g)]
    np.testing.assert_allclose(go.traj_fwd(*args), o.detach().numpy(), rtol=1e-11, atol=1e-13)
    for mine, ref in zip(go.traj_bwd(*args, dO.detach().numpy()), (q.grad, k.grad, v.grad, g.grad)):
        np.testing.assert_allclose(mine, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_finite_differences_on_a_shared_prefix_forest():
    fo = make_forest([([-1, 0, 0, 1], [0, 3, 5, 2], [5, 4, 2, 3])])
    q, k, v, g, dO = _rand(fo.n_tokens, 1, 3, 2, 7)
    ref = go.forest_eval(fo, q, k, v, g, dO)
    loss = lambda *a: float((go.forest_eval(fo, *a)["o"] * dO).sum())  # noqa: E731
    rng = np.random.default_rng(1)
    for name, idx in (("dq", 0), ("dk", 1), ("dv", 2), ("dg", 3)):
        args = [q, k, v, g]
        for _ in range(6):
            pos = tuple(int(rng.integers(n)) for n in args[idx].shape)
            hi, lo_ = [a.copy() for a in args], [a.copy() for a in args]
            hi[idx][pos] += 1e-6
            lo_[idx][pos] -= 1e-6
            fd = (loss(*hi) - loss(*lo_)) / 2e-6
            assert abs(fd - ref[name][pos]) <= 1e-7 * max(1.0, abs(fd)), (name, pos, fd, ref[name][pos])
