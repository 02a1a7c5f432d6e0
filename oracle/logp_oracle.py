"""fp64 oracle of the compact-to-semantic log-probability (Section "Preserving RL and MoE semantics
without expansion", Eqs. 17 and 19).  TEST INFRASTRUCTURE ONLY: imported by tests, the smoke check and
the CPU-baseline leg of the benchmark, never by the product path.

What it computes, written out from the definitions:

* ``positions``      the set P of non-terminal semantic positions of a forest in original batch order
                     (trajectory by trajectory), each with m(s) = the compact token it reuses and
                     y_s = the next token of the same trajectory;
* ``mapped_logp``    Eq. 17: lambda_s = z[m(s), y_s] - log sum_v exp z[m(s), v];
* ``mapped_logp_grad`` Eq. 19 with grad_z lambda_s = onehot(y_s) - softmax(z_{m(s)}): the contributions of
                     all positions that share a compact row are summed one by one;
* ``expanded_logp``  the direct restoration the section argues against (copy the C rows into S rows, full
                     log-softmax on each): used as the semantic definition the mapped form must equal.

Pins (tests/test_oracle_logp.py): uniform-logit and two-word closed forms, torch log_softmax + autograd on
the expanded rows, central finite differences, zero row sums and shift invariance of the gradient, and the
hand-counted positions of the five-node example tree.
"""
import numpy as np

from .la_oracle import trajectories


def positions(forest, token_id):
    """Non-terminal semantic positions of every trajectory, in original batch order.

    token_id: int array [C], the vocabulary id of every compact token in canonical order.
    Returns (m, y, pos_ptr): m[s] = canonical compact token of position s, y[s] = id of the token that
    follows it in the same trajectory, pos_ptr [n_traj+1] = where each trajectory's positions start."""
    token_id = np.asarray(token_id)
    traj_ptr, traj_rows = trajectories(forest)
    m, y, ptr = [], [], [0]
    for x in range(len(traj_ptr) - 1):
        rows = traj_rows[traj_ptr[x]:traj_ptr[x + 1]]
        for i in range(len(rows) - 1):              # the last token of a trajectory has no next token
            m.append(int(rows[i]))
            y.append(int(token_id[rows[i + 1]]))
        ptr.append(len(m))
    return np.asarray(m, np.int64), np.asarray(y, np.int64), np.asarray(ptr, np.int64)


def row_logsumexp(z):
    """log sum_v exp z[c, v] for every compact row, straight from the definition (fp64)."""
    z = np.asarray(z, np.float64)
    assert np.all(np.abs(z) < 600.0), "direct exp would overflow; logits are expected to be O(10)"
    return np.log(np.sum(np.exp(z), axis=1))


def mapped_logp(z, m, y):
    """Eq. 17.  z [C,V], m,y [P] -> (lambda [P], lse [C])."""
    z = np.asarray(z, np.float64)
    lse = row_logsumexp(z)
    lam = np.empty(len(m))
    for s in range(len(m)):
        lam[s] = z[m[s], y[s]] - lse[m[s]]
    return lam, lse


def mapped_logp_grad(z, m, y, g):
    """Eq. 19: dz[c] = sum over positions s with m(s)=c of g[s] * (onehot(y_s) - softmax(z_c)).
    g[s] = dL/dlambda_s (zero where the action mask drops the position)."""
    z = np.asarray(z, np.float64)
    C, V = z.shape
    lse = row_logsumexp(z)
    dz = np.zeros((C, V))
    for s in range(len(m)):
        c = m[s]
        dz[c] -= g[s] * np.exp(z[c] - lse[c])
        dz[c, y[s]] += g[s]
    return dz


def expanded_logp(z, m, y):
    """Direct restoration: one expanded logit row per position, full log-softmax on each."""
    z = np.asarray(z, np.float64)
    lam = np.empty(len(m))
    for s in range(len(m)):
        row = z[m[s]].copy()                         # the S x V copy the mapped form avoids
        lam[s] = (row - np.log(np.sum(np.exp(row))))[y[s]]
    return lam


def multiplicity(C, forest):
    """Eq. 20: q_c = number of semantic positions (terminal ones included) that map to compact token c."""
    _, traj_rows = trajectories(forest)
    return np.bincount(traj_rows, minlength=C).astype(np.int64)
