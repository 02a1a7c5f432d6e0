"""GPU parity of attention on compact tokens (Section 3.4, Eqs. 21-22) through the C ABI against the fp64 oracle.

Tolerances (bf16 inputs, fp32 accumulation, P rounded to bf16 before P.V): o relative Frobenius <= 5e-3, lse
<= 2e-3 absolute (fp32 sum of bf16-rounded probabilities); gradients <= 1e-2 relative Frobenius."""
import math
import random

import numpy as np
import pytest
import torch

import paper_2608_28158_b200 as H
from oracle import attn_oracle as ao
from workloads import config_forest, make_attn_inputs, make_forest
from test_plan_oracle import random_tree

pytestmark = pytest.mark.gpu
D = 128
SCALE = 1.0 / math.sqrt(D)


def _rel(a, b):
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30))


def _setup(fo, Hq, Hkv, seed, use_plan=True):
    C = fo.n_tokens
    inp = make_attn_inputs(C, Hq, Hkv, D, "bf16", seed)
    rot = None
    if use_plan:
        rot = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).row_of_token
    index = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot).upload()
    rows = torch.arange(C) if rot is None else torch.as_tensor(rot.astype(np.int64))
    phys = {}
    for n, x in inp.items():
        t = torch.empty_like(x); t[rows] = x; phys[n] = t.cuda()
    return inp, phys, index, rows.cuda()


def _forward(phys, index):
    o = torch.full_like(phys["q"], float("nan"))
    lse = torch.full(phys["q"].shape[:2], float("nan"), device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    H.harts_attn_fwd(index, phys["q"], phys["k"], phys["v"], o, lse, SCALE, dev_status=status)
    H.harts_la_check(status)
    return o, lse


@pytest.mark.parametrize("name,Hq,Hkv", [("cfg0", 1, 1), ("cfg0b", 2, 2), ("cfg0b", 4, 2)])
def test_forward_small_trees(name, Hq, Hkv):
    fo = config_forest(name)
    inp, phys, index, rows = _setup(fo, Hq, Hkv, 1)
    o, lse = _forward(phys, index)
    o_ref, lse_ref = ao.attn_fwd(fo, inp["q"].double().numpy(), inp["k"].double().numpy(), inp["v"].double().numpy(), SCALE)
    assert _rel(o[rows].double().cpu().numpy(), o_ref) <= 5e-3
    assert np.abs(lse[rows].double().cpu().numpy() - lse_ref).max() <= 2e-3


def test_forward_bushy_random_forest_without_a_row_map():
    rnd = random.Random(6)
    fo = make_forest([random_tree(rnd, 9, 300) for _ in range(3)] + [([-1], [0], [1])])
    for use_plan in (False, True):
        inp, phys, index, rows = _setup(fo, 2, 1, 2, use_plan)
        o, lse = _forward(phys, index)
        o_ref, lse_ref = ao.attn_fwd(fo, inp["q"].double().numpy(), inp["k"].double().numpy(), inp["v"].double().numpy(), SCALE)
        assert _rel(o[rows].double().cpu().numpy(), o_ref) <= 5e-3
        assert np.abs(lse[rows].double().cpu().numpy() - lse_ref).max() <= 2e-3


def test_forward_cfg1_sampled_queries():
    fo = config_forest("cfg1")
    inp, phys, index, rows = _setup(fo, 4, 4, 3)
    o, lse = _forward(phys, index)
    tok = np.unique(np.concatenate([np.linspace(0, fo.n_tokens - 1, 40).astype(np.int64), fo.token_base()[:-1],
                                    fo.token_base()[1:] - 1]))
    o_ref, lse_ref = ao.attn_fwd(fo, inp["q"].double().numpy(), inp["k"].double().numpy(), inp["v"].double().numpy(), SCALE,
                                 tokens=tok)
    got = o[rows].double().cpu().numpy()
    assert _rel(got[tok], o_ref[tok]) <= 5e-3
    assert np.abs(lse[rows].double().cpu().numpy()[tok] - lse_ref[tok]).max() <= 2e-3
    assert bool(torch.isfinite(o.float()).all()) and bool(torch.isfinite(lse).all())


def _backward(phys, index, o, lse):
    dq = torch.full_like(phys["q"], float("nan")); dk = torch.full_like(phys["k"], float("nan"))
    dv = torch.full_like(phys["v"], float("nan"))
    delta = torch.empty(phys["q"].shape[:2], device="cuda")
    status = torch.zeros(4, dtype=torch.int32, device="cuda")
    H.harts_attn_bwd(index, phys["q"], phys["k"], phys["v"], o, lse, phys["dO"], dq, dk, dv, delta, SCALE, dev_status=status)
    H.harts_la_check(status)
    return dq, dk, dv


def _check_backward(fo, Hq, Hkv, seed, use_plan=True):
    inp, phys, index, rows = _setup(fo, Hq, Hkv, seed, use_plan)
    o, lse = _forward(phys, index)
    dq, dk, dv = _backward(phys, index, o, lse)
    ref = ao.attn_bwd(fo, *(inp[n].double().numpy() for n in ("q", "k", "v", "dO")), SCALE)
    errs = [_rel(x[rows].double().cpu().numpy(), r) for x, r in zip((dq, dk, dv), ref)]
    assert max(errs) <= 1e-2, errs
    return errs


@pytest.mark.parametrize("name,Hq,Hkv", [("cfg0", 1, 1), ("cfg0b", 2, 2), ("cfg0b", 4, 2)])
def test_backward_small_trees(name, Hq, Hkv):
    _check_backward(config_forest(name), Hq, Hkv, 4)


def test_backward_bushy_random_forest():
    rnd = random.Random(6)
    fo = make_forest([random_tree(rnd, 9, 300) for _ in range(3)] + [([-1], [0], [1])])
    _check_backward(fo, 2, 1, 5, use_plan=False)
    _check_backward(fo, 2, 2, 5, use_plan=True)


def test_full_size_sampled_queries_and_invariants():
    """The benchmark's workload (cfg2, 16 heads): o, lse and dq of sampled queries against the oracle one by one;
    dv through an identity that holds at any size (every softmax row sums to 1, so sum_s dv_s = sum_t dO_t)."""
    fo = config_forest("cfg2")
    Hq = Hkv = 16
    inp = make_attn_inputs(fo.n_tokens, Hq, Hkv, D, "bf16", 90, device="cuda")
    rot = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).row_of_token
    index = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot).upload()
    rows = torch.as_tensor(rot.astype(np.int64)).cuda()
    phys = {}
    for n, x in inp.items():
        t = torch.empty_like(x); t[rows] = x; phys[n] = t
    o, lse = _forward(phys, index)
    dq, dk, dv = _backward(phys, index, o, lse)
    tok = np.unique(np.concatenate([np.linspace(0, fo.n_tokens - 1, 12).astype(np.int64), fo.token_base()[1:4] - 1]))
    heads = [0, 7, 15]
    cpu = {n: x[:, heads].double().cpu().numpy() for n, x in inp.items()}
    o_ref, lse_ref = ao.attn_fwd(fo, cpu["q"], cpu["k"], cpu["v"], SCALE, tokens=tok)
    dq_ref, _, _ = ao.attn_bwd(fo, cpu["q"], cpu["k"], cpu["v"], cpu["dO"], SCALE, tokens=tok)
    pick = lambda x: x[rows][:, heads].double().cpu().numpy()[tok]  # noqa: E731
    assert _rel(pick(o), o_ref[tok]) <= 5e-3
    assert np.abs(pick(lse) - lse_ref[tok]).max() <= 2e-3
    assert _rel(pick(dq), dq_ref[tok]) <= 1e-2
    total_dv = dv.double().sum(dim=0).cpu().numpy()
    total_dO = inp["dO"].double().sum(dim=0).cpu().numpy()
    assert _rel(total_dv, total_dO) <= 5e-3
    assert all(bool(torch.isfinite(x.float()).all()) for x in (o, dq, dk, dv))
    # dk and dv of sampled KEY rows, each summed over all the queries that see it: the last token of a forking node
    # with about a thousand descendants on several branches, and a row near the end of a leaf
    base = fo.token_base()
    n_children = np.zeros(len(fo.node_len), np.int64)
    for t in range(fo.n_trees):
        lo_ = int(fo.tree_node_ptr[t])
        par = fo.tree(t)[0]
        for i in range(1, len(par)):
            n_children[lo_ + par[i]] += 1
    forks = [(abs(len(ao.descendants(fo, int(base[n + 1]) - 1)) - 1000), int(base[n + 1]) - 1)
             for n in range(len(fo.node_len)) if n_children[n] >= 2]
    leaf = next(n for n in range(len(fo.node_len)) if n_children[n] == 0 and fo.node_len[n] > 8)
    key_rows = [min(forks)[1], int(base[leaf + 1]) - 3]
    kheads = [0, 15]
    cpu2 = {n: x[:, kheads].double().cpu().numpy() for n, x in inp.items()}
    for s_ in key_rows:
        dk_ref, dv_ref = ao.attn_bwd_key_row(fo, cpu2["q"], cpu2["k"], cpu2["v"], cpu2["dO"], SCALE, s_)
        r = int(rot[s_])
        got_dk = dk[r][kheads].double().cpu().numpy()
        got_dv = dv[r][kheads].double().cpu().numpy()
        print("key row", s_, "descendants", len(ao.descendants(fo, s_)), _rel(got_dk, dk_ref), _rel(got_dv, dv_ref))
        assert _rel(got_dk, dk_ref) <= 1e-2 and _rel(got_dv, dv_ref) <= 1e-2


def test_many_short_pieces():
    """The first 120 nodes of a cfg4 tree: branches of 1..63 tokens forking off chunk boundaries, i.e. more than a
    hundred pieces much shorter than a tile, ragged everywhere.  Forward and dq on sampled tokens, dk and dv in full."""
    par, off, ln = (a[:120].tolist() for a in config_forest("cfg4").tree(0))     # a prefix of the nodes is a tree
    fo = make_forest([(par, off, ln)])
    Hq, Hkv = 2, 1
    inp, phys, index, rows = _setup(fo, Hq, Hkv, 11)
    assert index.n_pieces > 100
    o, lse = _forward(phys, index)
    dq, dk, dv = _backward(phys, index, o, lse)
    tok = np.unique(np.concatenate([np.linspace(0, fo.n_tokens - 1, 60).astype(np.int64), fo.token_base()[1:40] - 1]))
    cpu = {n: x.double().numpy() for n, x in inp.items()}
    o_ref, lse_ref = ao.attn_fwd(fo, cpu["q"], cpu["k"], cpu["v"], SCALE, tokens=tok)
    dq_ref, _, _ = ao.attn_bwd(fo, cpu["q"], cpu["k"], cpu["v"], cpu["dO"], SCALE, tokens=tok)
    pick = lambda x: x[rows].double().cpu().numpy()[tok]  # noqa: E731
    assert _rel(pick(o), o_ref[tok]) <= 5e-3 and np.abs(pick(lse) - lse_ref[tok]).max() <= 2e-3
    assert _rel(pick(dq), dq_ref[tok]) <= 1e-2
    # dk, dv against the full oracle on this tree (a few seconds)
    _, dk_ref, dv_ref = ao.attn_bwd(fo, cpu["q"], cpu["k"], cpu["v"], cpu["dO"], SCALE)
    assert _rel(dk[rows].double().cpu().numpy(), dk_ref) <= 1e-2
    assert _rel(dv[rows].double().cpu().numpy(), dv_ref) <= 1e-2


@pytest.mark.parametrize("seed", [2052, 3017])
def test_forward_rescale_waits_for_the_previous_tile(seed):
    """Two random forests on which an early version rescaled O (a row whose maximum jumps by more than 2^8 late in
    the walk) while the previous tile's P.V MMAs were still accumulating into it: one wrong row in thousands."""
    rnd = random.Random(seed)
    max_len = rnd.choice([5, 70, 200, 700])
    fo = make_forest([random_tree(rnd, rnd.randint(1, 10), max_len) for _ in range(rnd.randint(1, 4))])
    rnd.choice([1, 2, 3])
    Hkv = rnd.choice([1, 2]); Hq = Hkv * rnd.choice([1, 2])
    inp = make_attn_inputs(fo.n_tokens, Hq, Hkv, D, "bf16", seed % 1000)
    use_plan = rnd.random() < 0.7
    rot = H.harts_la_plan(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, 64).row_of_token if use_plan else None
    index = H.harts_attn_index(fo.tree_node_ptr, fo.node_parent, fo.node_fork_off, fo.node_len, rot).upload()
    rows = torch.arange(fo.n_tokens) if rot is None else torch.as_tensor(np.asarray(rot).astype(np.int64))
    phys = {}
    for n, x in inp.items():
        t = torch.empty_like(x); t[rows] = x; phys[n] = t.cuda()
    o, lse = _forward(phys, index)
    o_ref, lse_ref = ao.attn_fwd(fo, inp["q"].double().numpy(), inp["k"].double().numpy(), inp["v"].double().numpy(), SCALE)
    got = o[rows.cuda()].double().cpu().numpy()
    assert np.abs(got - o_ref).max() <= 0.05                   # no single row off (the relative norm alone would hide one)
    assert _rel(got, o_ref) <= 5e-3


def test_repeated_runs_are_bit_identical_with_a_wide_query_group():
    """Forward and dQ have a fixed summation order, so repeated launches must agree bit for bit.  With eight query
    heads per key/value head and many partial query tiles, an early version let a fast warp's arrival for tile n+1
    count towards tile n (one barrier for both S buffers) and now and then ran P.V on a tile another warp had not
    written yet; such a run differs from the others."""
    rnd = random.Random(7 * 7919 + 128)
    fo = make_forest([random_tree(rnd, rnd.randint(3, 30), rnd.choice([300, 1500, 4000])) for _ in range(rnd.randint(1, 3))])
    Hq, Hkv = 8, 1
    inp, phys, index, rows = _setup(fo, Hq, Hkv, 128)
    phys["q"] = (phys["q"].float() * 6.0).to(torch.bfloat16)          # sharp rows: the running maximum jumps late
    o0, lse0 = _forward(phys, index)
    assert bool(torch.isfinite(o0.float()).all()) and bool(torch.isfinite(lse0).all())
    dq0, _, _ = _backward(phys, index, o0, lse0)
    for _ in range(250):                  # the early version failed about once in 250 launches of this case
        o, lse = _forward(phys, index)
        assert torch.equal(o, o0) and torch.equal(lse, lse0)
    for _ in range(20):
        dq, _, _ = _backward(phys, index, o0, lse0)
        assert torch.equal(dq, dq0)
    # and the result is the right one, on sampled queries
    tok = np.array(sorted(rnd.sample(range(fo.n_tokens), 16)))
    cpu = {n: x[:, [0] if n in ("k", "v") else [0, Hq - 1]].double().numpy() for n, x in inp.items()}
    cpu["q"] = (inp["q"].float() * 6.0).to(torch.bfloat16)[:, [0, Hq - 1]].double().numpy()
    cpu["k"] = np.repeat(cpu["k"], 2, axis=1); cpu["v"] = np.repeat(cpu["v"], 2, axis=1)
    o_ref, lse_ref = ao.attn_fwd(fo, cpu["q"], cpu["k"], cpu["v"], SCALE, tokens=tok)
    got = o0[rows][:, [0, Hq - 1]].double().cpu().numpy()[tok]
    assert np.abs(got - o_ref[tok]).max() <= 0.06


def test_degenerate_forests_have_closed_forms():
    """One token: o = v, lse = scale q.k, dq = dk = 0, dv = dO.  A chain of one-token nodes (every token its own
    piece, each the child of the previous one) is plain causal attention over the chain."""
    fo = make_forest([([-1], [0], [1])])
    inp, phys, index, rows = _setup(fo, 2, 1, 11)
    o, lse = _forward(phys, index)
    dq, dk, dv = _backward(phys, index, o, lse)
    assert torch.equal(o, phys["v"].expand(-1, 2, -1))
    want = (phys["q"].float() * phys["k"].float()).sum(-1) * SCALE
    assert float((lse - want).abs().max()) <= 1e-5
    assert float(dq.float().abs().max()) == 0.0 and float(dk.float().abs().max()) <= 1e-6
    assert _rel(dv.double().cpu().numpy(), phys["dO"].double().sum(dim=1, keepdim=True).cpu().numpy()) <= 4e-3

    n = 70                                                  # more than one 64-row tile of one-token pieces
    fo = make_forest([([-1] + list(range(n - 1)), [0] + [1] * (n - 1), [1] * n)])
    inp, phys, index, rows = _setup(fo, 2, 2, 12)
    o, lse = _forward(phys, index)
    dq, dk, dv = _backward(phys, index, o, lse)
    q, k, v, dO = (inp[x].float().cuda().transpose(0, 1).requires_grad_(x != "dO") for x in ("q", "k", "v", "dO"))
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True, scale=SCALE)
    ref.backward(dO)
    pick = lambda x: x[rows].float().transpose(0, 1)     # noqa: E731
    assert _rel(pick(o).cpu().numpy(), ref.detach().cpu().numpy()) <= 5e-3
    for got, want_ in ((dq, q.grad), (dk, k.grad), (dv, v.grad)):
        assert _rel(pick(got).cpu().numpy(), want_.cpu().numpy()) <= 1e-2
