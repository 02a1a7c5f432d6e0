"""fp64 oracle of full attention on compact tokens (Section 3.4 "Full attention on compact tokens", Section 4.2
"MLA execution with asymmetric packed Q/KV views", Eqs. 21-22).  TEST INFRASTRUCTURE ONLY.

Every compact token t has one query; it attends to the keys/values of its true ancestors and of itself (the
tokens on the path from the root of its tree to t), which is what the packed view of Eq. 21 with the
bottom-right alignment of Eq. 22 expresses branch by branch: a branch with h ancestor tokens and l own tokens
has l queries and h+l keys, and query i sees key j iff j <= h + i.

    o_t = sum_{s in path(t)} softmax_s(scale * q_t . k_s) v_s          (per query head; GQA: kv head = head // G)

Backward of L = sum_t <dO_t, o_t>: the standard softmax-attention gradients, with dk/dv of a shared ancestor
summing the contributions of every descendant on every branch (the gather's backward of Section 3.4).

Pins (tests/test_oracle_attn.py): torch scaled_dot_product_attention (causal) on every expanded trajectory with
autograd through the expansion, the Eq. 22 mask on a branch view, equal-keys closed form, central differences.
"""
import numpy as np

from .conv_oracle import predecessors


def _path(pred, t):
    chain = []
    a = t
    while a >= 0:
        chain.append(a)
        a = pred[a]
    return np.asarray(chain[::-1], np.int64)


def paths(forest):
    """path[t] = canonical indices of the tokens t attends to, root first, t last."""
    pred = predecessors(forest)
    return [_path(pred, t) for t in range(forest.n_tokens)]


def attn_fwd(forest, q, k, v, scale, tokens=None):
    """q [C,Hq,d], k,v [C,Hkv,d] canonical order -> (o [C,Hq,d], lse [C,Hq]) in fp64; lse in natural log units.
    tokens: compute only these queries (the other rows of the result stay zero)."""
    q, k, v = (np.asarray(a, np.float64) for a in (q, k, v))
    C, Hq, d = q.shape
    G = Hq // k.shape[1]
    o = np.zeros((C, Hq, v.shape[2]))
    lse = np.zeros((C, Hq))
    pred = predecessors(forest)
    for t in (range(C) if tokens is None else tokens):
        t = int(t)
        path = _path(pred, t)
        for h in range(Hq):
            s = scale * (k[path, h // G] @ q[t, h])
            m = s.max()
            e = np.exp(s - m)
            lse[t, h] = m + np.log(e.sum())
            o[t, h] = (e / e.sum()) @ v[path, h // G]
    return o, lse


def attn_bwd(forest, q, k, v, dO, scale, tokens=None):
    """(dq, dk, dv) of sum_t <dO_t, o_t>.  tokens: only these queries (dq rows of the others stay zero; dk, dv then
    hold the contributions of these queries alone)."""
    q, k, v, dO = (np.asarray(a, np.float64) for a in (q, k, v, dO))
    C, Hq, d = q.shape
    G = Hq // k.shape[1]
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    pred = predecessors(forest)
    for t in (range(C) if tokens is None else tokens):
        t = int(t)
        path = _path(pred, t)
        for h in range(Hq):
            hk = h // G
            s = scale * (k[path, hk] @ q[t, h])
            p = np.exp(s - s.max())
            p /= p.sum()
            dv[path, hk] += np.outer(p, dO[t, h])
            dp = v[path, hk] @ dO[t, h]
            ds = p * (dp - np.dot(p, dp))
            dq[t, h] = scale * (ds @ k[path, hk])
            dk[path, hk] += scale * np.outer(ds, q[t, h])
    return dq, dk, dv


def branch_view_mask(h, l):
    """Eq. 22: l queries against h + l keys, query i sees key j iff j <= h + i."""
    i = np.arange(l)[:, None]
    j = np.arange(h + l)[None, :]
    return j <= h + i


def descendants(forest, s):
    """Canonical indices of every token whose path contains token s (s itself included), ascending."""
    pred = predecessors(forest)
    inside = np.zeros(forest.n_tokens, bool)
    inside[s] = True
    for t in range(s + 1, forest.n_tokens):       # canonical order puts a token after its predecessor
        p = pred[t]
        if p >= 0 and inside[p]:
            inside[t] = True
    return np.nonzero(inside)[0]


def attn_bwd_key_row(forest, q, k, v, dO, scale, s):
    """dk[s], dv[s] ([Hkv, d] each) written out from the definition for ONE key row: the sum, over every query t
    that sees s (its descendants on every branch, and s itself) and every query head of the group, of
        dv_s += p_t(s) dO_t,      dk_s += scale * p_t(s) (dO_t . v_s - sum_r p_t(r) dO_t . v_r) q_t
    with p_t the softmax of t's scores over its own path.  Same arithmetic as attn_bwd restricted to one row, so that
    a shared ancestor of thousands of queries can be checked at full problem size."""
    q, k, v, dO = (np.asarray(a, np.float64) for a in (q, k, v, dO))
    Hq, Hkv = q.shape[1], k.shape[1]
    G = Hq // Hkv
    dk_s, dv_s = np.zeros((Hkv, k.shape[2])), np.zeros((Hkv, v.shape[2]))
    pred = predecessors(forest)
    for t in descendants(forest, s):
        path = _path(pred, int(t))
        at = int(np.nonzero(path == s)[0][0])
        for h in range(Hq):
            hk = h // G
            sc = scale * (k[path, hk] @ q[t, h])
            p = np.exp(sc - sc.max())
            p /= p.sum()
            dp = v[path, hk] @ dO[t, h]
            dv_s[hk] += p[at] * dO[t, h]
            dk_s[hk] += scale * p[at] * (dp[at] - np.dot(p, dp)) * q[t, h]
    return dk_s, dv_s
