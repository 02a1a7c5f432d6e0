"""Pins of the compact-token attention oracle (Section 3.4, Eqs. 21-22) against library attention per trajectory."""
import random

import numpy as np
import torch

from oracle import attn_oracle as ao
from oracle.la_oracle import trajectories
from workloads import config_forest, make_forest
from test_plan_oracle import random_tree


def _rand(fo, Hq, Hkv, d, seed):
    rng = np.random.default_rng(seed)
    C = fo.n_tokens
    return (rng.normal(size=(C, Hq, d)), rng.normal(size=(C, Hkv, d)), rng.normal(size=(C, Hkv, d)),
            rng.normal(size=(C, Hq, d)))


def _sdpa_per_trajectory(fo, q, k, v, scale):
    """Library definition: every root-to-leaf trajectory alone, causal scaled_dot_product_attention."""
    ptr, rows = trajectories(fo)
    qt, kt, vt = (torch.tensor(a, requires_grad=True) for a in (q, k, v))
    G = q.shape[1] // k.shape[1]
    outs = []
    for i in range(len(ptr) - 1):
        idx = torch.tensor(rows[ptr[i]:ptr[i + 1]])
        qs = qt.index_select(0, idx).transpose(0, 1)                     # [Hq, L, d]
        ks = kt.index_select(0, idx).transpose(0, 1).repeat_interleave(G, 0)
        vs = vt.index_select(0, idx).transpose(0, 1).repeat_interleave(G, 0)
        o = torch.nn.functional.scaled_dot_product_attention(qs, ks, vs, is_causal=True, scale=scale)
        outs.append(o.transpose(0, 1))
    return qt, kt, vt, torch.cat(outs), rows


def test_forward_and_backward_equal_causal_sdpa_on_every_trajectory():
    rnd = random.Random(1)
    for Hq, Hkv in ((2, 2), (4, 2)):
        fo = make_forest([random_tree(rnd, 7, 9) for _ in range(2)])
        q, k, v, dO = _rand(fo, Hq, Hkv, 8, 3)
        scale = 0.3
        o, lse = ao.attn_fwd(fo, q, k, v, scale)
        qt, kt, vt, o_exp, rows = _sdpa_per_trajectory(fo, q, k, v, scale)
        assert np.allclose(o[rows], o_exp.detach().numpy(), atol=1e-12)          # every copy of a shared token
        first = np.zeros(len(rows), bool)
        first[np.unique(rows, return_index=True)[1]] = True                      # the compact loss counts a token once
        (o_exp * torch.tensor(dO[rows] * first[:, None, None])).sum().backward()
        dq, dk, dv = ao.attn_bwd(fo, q, k, v, dO, scale)
        assert np.allclose(dq, qt.grad.numpy(), atol=1e-11)
        assert np.allclose(dk, kt.grad.numpy(), atol=1e-11) and np.allclose(dv, vt.grad.numpy(), atol=1e-11)


def test_branch_view_is_bottom_right_aligned():
    # branch C of the five-node tree: h = 100 ancestors (root[:100]), l = 200 own tokens
    fo = config_forest("cfg0")
    base = fo.token_base()
    paths = ao.paths(fo)
    h, l = 100, 200
    mask = ao.branch_view_mask(h, l)
    kv_view = np.concatenate([np.arange(100), np.arange(base[4], base[4] + l)])  # ancestors then own tokens
    for i in (0, 1, 57, 199):
        assert np.array_equal(kv_view[mask[i]], paths[base[4] + i])
    assert mask.shape == (l, h + l) and mask[0].sum() == h + 1 and mask[-1].all()
    # a top-left alignment would let query 0 see only one key
    assert not np.array_equal(mask, np.tril(np.ones((l, h + l), bool)))


def test_equal_keys_give_the_running_mean_and_one_token_returns_v():
    fo = config_forest("cfg0")
    C = fo.n_tokens
    rng = np.random.default_rng(0)
    q = rng.normal(size=(C, 1, 4)); v = rng.normal(size=(C, 1, 4))
    k = np.ones((C, 1, 4))
    o, lse = ao.attn_fwd(fo, q, k, v, 0.5)
    paths = ao.paths(fo)
    for t in (0, 5, 300, C - 1):
        assert np.allclose(o[t, 0], v[paths[t], 0].mean(axis=0), atol=1e-13)
        assert np.isclose(lse[t, 0], 0.5 * q[t, 0].sum() + np.log(len(paths[t])))
    one = make_forest([([-1], [0], [1])])
    o1, _ = ao.attn_fwd(one, q[:1], k[:1], v[:1], 1.0)
    assert np.allclose(o1, v[:1])


def test_central_differences():
    rnd = random.Random(7)
    fo = make_forest([random_tree(rnd, 5, 4)])
    q, k, v, dO = _rand(fo, 2, 1, 3, 9)
    dq, dk, dv = ao.attn_bwd(fo, q, k, v, dO, 0.7)
    f = lambda q_, k_, v_: float((ao.attn_fwd(fo, q_, k_, v_, 0.7)[0] * dO).sum())  # noqa: E731
    h = 1e-6
    C = fo.n_tokens
    for idx in [(0, 0, 0), (C - 1, 1, 2), (C // 2, 0, 1)]:
        qp, qm = q.copy(), q.copy(); qp[idx] += h; qm[idx] -= h
        assert abs((f(qp, k, v) - f(qm, k, v)) / (2 * h) - dq[idx]) < 1e-7
    for idx in [(0, 0, 0), (C - 1, 0, 2), (C // 2, 0, 1)]:
        kp, km = k.copy(), k.copy(); kp[idx] += h; km[idx] -= h
        assert abs((f(q, kp, v) - f(q, km, v)) / (2 * h) - dk[idx]) < 1e-7
        vp, vm = v.copy(), v.copy(); vp[idx] += h; vm[idx] -= h
        assert abs((f(q, k, vp) - f(q, k, vm)) / (2 * h) - dv[idx]) < 1e-7


def test_key_row_gradients_equal_the_full_backward_rows():
    """attn_bwd_key_row (one key row from the definition, used for full-size checks) against attn_bwd, which is
    pinned above by autograd: a root row with many descendants, a fork row, a leaf row; MHA and GQA."""
    import random
    from test_plan_oracle import random_tree
    from workloads import make_attn_inputs, make_forest
    rnd = random.Random(21)
    fo = make_forest([random_tree(rnd, 7, 9) for _ in range(2)])
    for Hq, Hkv in ((2, 2), (4, 2)):
        inp = {n: x.double().numpy() for n, x in make_attn_inputs(fo.n_tokens, Hq, Hkv, 8, "fp32", 3).items()}
        _, dk, dv = ao.attn_bwd(fo, inp["q"], inp["k"], inp["v"], inp["dO"], 0.3)
        for s in (0, 1, fo.n_tokens // 2, fo.n_tokens - 1):
            dk_s, dv_s = ao.attn_bwd_key_row(fo, inp["q"], inp["k"], inp["v"], inp["dO"], 0.3, s)
            np.testing.assert_allclose(dk_s, dk[s], rtol=1e-10, atol=1e-13)
            np.testing.assert_allclose(dv_s, dv[s], rtol=1e-10, atol=1e-13)
    assert len(ao.descendants(fo, 0)) > 5
