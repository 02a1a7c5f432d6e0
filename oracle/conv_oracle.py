"""fp64 oracle of the tree-aware causal convolution that precedes the linear-attention core (Section 4.2,
"KDA state reuse and causal convolution").  TEST INFRASTRUCTURE ONLY.

The convolution is depthwise (one filter of width w per channel) and causal along a TRAJECTORY: the history of
a compact token is its true ancestors in the rollout tree, never whatever happens to sit before it in the packed
layout, and positions before the start of the trajectory contribute zero.  With taps indexed like a library
conv1d (the last tap multiplies the current token),

    y_t[c] = sum_{i=0}^{w-1} W[c, w-1-i] * x_{anc_i(t)}[c],     anc_0(t) = t, anc_{i+1}(t) = predecessor of anc_i(t).

Every compact token has ONE output (its ancestors are the same in every trajectory through it), and its input
gradient collects the contributions of all its descendants within w-1 steps, on every branch.

Pins (tests/test_oracle_conv.py): torch conv1d on every expanded trajectory, autograd through the expansion,
identity and shift filters, central differences, agreement of all copies of a shared token.
"""
import numpy as np


def predecessors(forest):
    """pred[t] = canonical index of the token before t on its trajectory, -1 at the start of a root."""
    base = forest.token_base()
    pred = np.arange(-1, forest.n_tokens - 1, dtype=np.int64)           # inside a node: the previous token
    for t in range(forest.n_trees):
        lo = int(forest.tree_node_ptr[t])
        par, off, ln = (a.tolist() for a in forest.tree(t))
        for i in range(len(par)):
            first = base[lo + i]
            pred[first] = -1 if par[i] < 0 else base[lo + par[i]] + off[i] - 1
    return pred


def conv_fwd(forest, x, W):
    """x [C, D] canonical order, W [D, w] -> y [C, D] (fp64)."""
    x = np.asarray(x, np.float64)
    W = np.asarray(W, np.float64)
    w = W.shape[1]
    pred = predecessors(forest)
    y = np.zeros_like(x)
    for t in range(x.shape[0]):
        a = t
        for i in range(w):
            if a < 0:
                break
            y[t] += W[:, w - 1 - i] * x[a]
            a = pred[a]
    return y


def conv_bwd(forest, x, W, dy):
    """Gradients of sum_t <dy_t, y_t>: (dx [C, D], dW [D, w])."""
    x = np.asarray(x, np.float64)
    W = np.asarray(W, np.float64)
    dy = np.asarray(dy, np.float64)
    w = W.shape[1]
    pred = predecessors(forest)
    dx = np.zeros_like(x)
    dW = np.zeros_like(W)
    for t in range(x.shape[0]):
        a = t
        for i in range(w):
            if a < 0:
                break
            dx[a] += W[:, w - 1 - i] * dy[t]
            dW[:, w - 1 - i] += dy[t] * x[a]
            a = pred[a]
    return dx, dW
