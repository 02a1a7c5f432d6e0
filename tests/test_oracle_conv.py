"""Pins of the tree-aware causal convolution oracle against library conv1d on expanded trajectories."""
import random

import numpy as np
import torch

from oracle import conv_oracle as co
from oracle.la_oracle import trajectories
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _expanded_conv(forest, x, W):
    """Library definition: every trajectory on its own, zero left padding, depthwise conv1d."""
    ptr, rows = trajectories(forest)
    xt = torch.tensor(x, requires_grad=True)
    Wt = torch.tensor(W, requires_grad=True)
    D, w = W.shape
    outs = []
    for i in range(len(ptr) - 1):
        seq = xt.index_select(0, torch.tensor(rows[ptr[i]:ptr[i + 1]]))            # [L, D]
        y = torch.nn.functional.conv1d(seq.t()[None], Wt[:, None, :], padding=w - 1, groups=D)[0, :, :seq.shape[0]]
        outs.append(y.t())
    return xt, Wt, torch.cat(outs), rows


def test_equals_conv1d_on_every_trajectory_and_copies_agree():
    rnd = random.Random(2)
    rng = np.random.default_rng(2)
    for w in (2, 3, 4):
        fo = make_forest([random_tree(rnd, 7, 9) for _ in range(2)])
        x = rng.normal(size=(fo.n_tokens, 5)); W = rng.normal(size=(5, w))
        y = co.conv_fwd(fo, x, W)
        _, _, y_exp, rows = _expanded_conv(fo, x, W)
        assert np.allclose(y[rows], y_exp.detach().numpy(), atol=1e-12)           # every copy of a shared token


def test_backward_equals_autograd_through_the_expansion():
    rnd = random.Random(3)
    rng = np.random.default_rng(3)
    fo = make_forest([random_tree(rnd, 8, 7) for _ in range(2)])
    x = rng.normal(size=(fo.n_tokens, 4)); W = rng.normal(size=(4, 4)); dy = rng.normal(size=x.shape)
    xt, Wt, y_exp, rows = _expanded_conv(fo, x, W)
    # the compact loss sum_t <dy_t, y_t> counts every compact token once: weight its first copy only
    first = np.zeros(len(rows), bool)
    first[np.unique(rows, return_index=True)[1]] = True
    (y_exp * torch.tensor(dy[rows] * first[:, None])).sum().backward()
    dx, dW = co.conv_bwd(fo, x, W, dy)
    assert np.allclose(dx, xt.grad.numpy(), atol=1e-12) and np.allclose(dW, Wt.grad.numpy(), atol=1e-12)


def test_identity_and_shift_filters_on_the_five_node_tree():
    fo = config_forest("cfg0")
    x = np.arange(fo.n_tokens, dtype=np.float64)[:, None] + 1.0
    W = np.zeros((1, 4)); W[0, 3] = 1.0
    assert np.array_equal(co.conv_fwd(fo, x, W), x)                                # last tap = the token itself
    W = np.zeros((1, 4)); W[0, 2] = 1.0                                            # one step back
    y = co.conv_fwd(fo, x, W)[:, 0]
    base = fo.token_base()
    assert y[0] == 0 and y[5] == x[4, 0]
    assert y[base[1]] == x[255, 0] and y[base[2]] == x[255, 0]                     # A and X follow the root's end
    assert y[base[4]] == x[99, 0]                                                  # C forks after root offset 100
    assert y[base[3]] == x[base[2] + 43, 0]                                        # B follows X's last token
    W = np.zeros((1, 4)); W[0, 0] = 1.0                                            # three steps back, across a fork
    y = co.conv_fwd(fo, x, W)[:, 0]
    assert y[base[4] + 1] == x[98, 0] and y[base[4] + 3] == x[base[4], 0] and y[2] == 0


def test_central_differences():
    rnd = random.Random(5)
    rng = np.random.default_rng(5)
    fo = make_forest([random_tree(rnd, 5, 5)])
    x = rng.normal(size=(fo.n_tokens, 2)); W = rng.normal(size=(2, 3)); dy = rng.normal(size=x.shape)
    dx, dW = co.conv_bwd(fo, x, W, dy)
    f = lambda x_, W_: float((co.conv_fwd(fo, x_, W_) * dy).sum())  # noqa: E731
    h = 1e-6
    for idx in [(0, 0), (fo.n_tokens - 1, 1), (fo.n_tokens // 2, 0)]:
        xp, xm = x.copy(), x.copy(); xp[idx] += h; xm[idx] -= h
        assert abs((f(xp, W) - f(xm, W)) / (2 * h) - dx[idx]) < 1e-7
    for idx in [(0, 0), (1, 2), (0, 1)]:
        Wp, Wm = W.copy(), W.copy(); Wp[idx] += h; Wm[idx] -= h
        assert abs((f(x, Wp) - f(x, Wm)) / (2 * h) - dW[idx]) < 1e-7
