"""Seeded rollout-tree generators for the five benchmark configurations.

A forest is stored as flat node arrays.  Node ``i`` of a tree has a parent
(tree-local index, -1 for the root), the offset inside the parent at which it
forks (1..len(parent); a fork at ``len(parent)`` is a fork at the parent's
end) and a token count.  A parent always precedes its children.  The canonical
token order is: trees in order, nodes in input order, tokens in order.

Only shapes are produced here; nothing in this file plans, chunks or evaluates
the recurrence.
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass

import numpy as np

_DATA_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "data")


@dataclass
class Forest:
    tree_node_ptr: np.ndarray  # int32 [n_trees + 1]
    node_parent: np.ndarray    # int32 [n_nodes], tree-local, -1 = root
    node_fork_off: np.ndarray  # int32 [n_nodes], 0 for roots
    node_len: np.ndarray       # int32 [n_nodes], >= 1

    @property
    def n_trees(self) -> int:
        return len(self.tree_node_ptr) - 1

    @property
    def n_nodes(self) -> int:
        return len(self.node_len)

    @property
    def n_tokens(self) -> int:
        return int(self.node_len.sum())

    def tree(self, t: int):
        lo, hi = int(self.tree_node_ptr[t]), int(self.tree_node_ptr[t + 1])
        return (self.node_parent[lo:hi], self.node_fork_off[lo:hi], self.node_len[lo:hi])

    def subset(self, tree_ids) -> "Forest":
        return make_forest([tuple(a.tolist() for a in self.tree(t)) for t in tree_ids])

    def token_base(self) -> np.ndarray:
        """Canonical index of the first token of every node, int64 [n_nodes + 1]."""
        out = np.zeros(self.n_nodes + 1, dtype=np.int64)
        np.cumsum(self.node_len, out=out[1:])
        return out

    def to_json(self) -> dict:
        return {
            "tree_node_ptr": self.tree_node_ptr.tolist(),
            "node_parent": self.node_parent.tolist(),
            "node_fork_off": self.node_fork_off.tolist(),
            "node_len": self.node_len.tolist(),
        }

    @staticmethod
    def from_json(d: dict) -> "Forest":
        return Forest(*(np.asarray(d[k], dtype=np.int32) for k in
                        ("tree_node_ptr", "node_parent", "node_fork_off", "node_len")))


def make_forest(trees) -> Forest:
    """trees: iterable of (parent[], fork_off[], len[]) per tree."""
    ptr, par, off, ln = [0], [], [], []
    for p, o, l in trees:
        assert len(p) == len(o) == len(l) and len(p) >= 1
        par += list(p)
        off += list(o)
        ln += list(l)
        ptr.append(len(par))
    i32 = lambda x: np.asarray(x, dtype=np.int32)  # noqa: E731
    return Forest(i32(ptr), i32(par), i32(off), i32(ln))


# --------------------------------------------------------------------------------------
# Per-tree counts used by the rejection windows (shape statistics only).
# --------------------------------------------------------------------------------------
def tree_counts(par, off, ln):
    """(compact tokens, trajectory-wise tokens, leaves) of one tree."""
    n = len(par)
    start = [0] * n
    ends_at_tail = [False] * n
    for i in range(1, n):
        start[i] = start[par[i]] + off[i]
        if off[i] == ln[par[i]]:
            ends_at_tail[par[i]] = True
    c = int(sum(ln))
    s = 0
    leaves = 0
    for v in range(n):
        if not ends_at_tail[v]:      # the node's own end is a trajectory end
            s += start[v] + ln[v]
            leaves += 1
    return c, s, leaves


# --------------------------------------------------------------------------------------
# Fixed trees (configuration 0 and its variant)
# --------------------------------------------------------------------------------------
def _cfg0():
    #        root  A    X    B   C
    par = [-1, 0, 0, 2, 0]
    off = [0, 256, 256, 44, 100]
    ln = [256, 128, 44, 90, 200]
    return [(par, off, ln)]


def _cfg0b():
    # X gets a second leaf so that position 300 is a real fork inside a chunk
    par = [-1, 0, 0, 2, 0, 2]
    off = [0, 256, 256, 44, 100, 44]
    ln = [256, 128, 44, 90, 200, 50]
    return [(par, off, ln)]


# --------------------------------------------------------------------------------------
# Random trees
# --------------------------------------------------------------------------------------
def _lognormal_len(rng, mu, sigma, lo, hi):
    return int(np.clip(np.round(rng.lognormal(mu, sigma)), lo, hi))


def _cfg1(seed=1, c_window=(14000, 18000)):
    rng = np.random.default_rng(seed)
    while True:
        depth = int(rng.integers(1, 5))
        par, off, ln = [-1], [0], [_lognormal_len(rng, np.log(512), 0.8, 16, 4096)]
        frontier = [0]
        for _ in range(depth - 1):
            nxt = []
            for v in frontier:
                for _ in range(int(rng.integers(1, 4))):
                    par.append(v)
                    ln.append(_lognormal_len(rng, np.log(512), 0.8, 16, 4096))
                    off.append(int(rng.integers(1, ln[v] + 1)))
                    nxt.append(len(par) - 1)
            frontier = nxt
        if c_window[0] <= sum(ln) <= c_window[1]:
            return [(par, off, ln)]


def _draw_agentic_tree(rng, c_max):
    root = int(rng.integers(8192, 16385))
    depth = int(rng.integers(2, 7))          # node levels including the root
    par, ln, total = [-1], [root], root
    frontier = [0]
    for _ in range(depth - 1):
        nxt = []
        for v in frontier:
            for _ in range(int(rng.integers(1, 5))):
                length = _lognormal_len(rng, np.log(1500), 1.0, 32, 16384)
                par.append(v)
                ln.append(length)
                total += length
                nxt.append(len(par) - 1)
                if total > c_max:
                    return None
        frontier = nxt
    off = [0] + [ln[p] for p in par[1:]]     # turns fork at the parent's end
    return par, off, ln


def _agentic(seed, n_trees, c_window=(12000, 20000), ratio_window=(5.4, 5.9)):
    rng = np.random.default_rng(seed)
    out = []
    while len(out) < n_trees:
        t = _draw_agentic_tree(rng, c_window[1])
        if t is None:
            continue
        c, s, _ = tree_counts(*t)
        if c < c_window[0] or not (ratio_window[0] <= s / c <= ratio_window[1]):
            continue
        out.append(t)
    return out


def _cfg4(seed=4, n_trees=64, root_len=2048, fanout=16, levels=3, chunk=64):
    rng = np.random.default_rng(seed)
    out = []
    for _ in range(n_trees):
        par, off, ln, start = [-1], [0], [root_len], [0]
        frontier = [0]
        for _ in range(levels - 1):
            nxt = []
            for v in frontier:
                for _ in range(fanout):
                    length = int(rng.integers(1, 64))
                    while True:
                        o = int(rng.integers(1, ln[v] + 1))
                        if (start[v] + o) % chunk != 0:
                            break
                    par.append(v)
                    off.append(o)
                    ln.append(length)
                    start.append(start[v] + o)
                    nxt.append(len(par) - 1)
            frontier = nxt
        out.append((par, off, ln))
    return out


# name -> (heads, d_k, d_v, dtype, chunk, seed, builder or stored file)
CONFIGS = {
    "cfg0":  dict(H=1, dk=64, dv=64, dtype="fp32", chunk=64, seed=0, build=_cfg0),
    "cfg0b": dict(H=1, dk=64, dv=64, dtype="fp32", chunk=64, seed=0, build=_cfg0b),
    "cfg1":  dict(H=4, dk=128, dv=128, dtype="bf16", chunk=64, seed=1, build=_cfg1),
    "cfg2":  dict(H=16, dk=128, dv=128, dtype="bf16", chunk=64, seed=2, stored="cfg2_trees.json",
                  build=lambda: _agentic(2, 8)),
    "cfg3":  dict(H=32, dk=128, dv=128, dtype="bf16", chunk=64, seed=3, stored="cfg3_trees.json",
                  build=lambda: _agentic(3, 32)),
    "cfg4":  dict(H=16, dk=128, dv=128, dtype="bf16", chunk=64, seed=4, build=_cfg4),
}


def config_forest(name: str) -> Forest:
    """The forest of a named configuration.  The rejection-sampled forests of
    cfg2/cfg3 take minutes to draw, so their node arrays are stored beside this
    file (written by ``python -m workloads.trees --write``)."""
    cfg = CONFIGS[name]
    stored = cfg.get("stored")
    if stored:
        path = os.path.join(_DATA_DIR, stored)
        if os.path.exists(path):
            with open(path) as f:
                return Forest.from_json(json.load(f))
    return make_forest(cfg["build"]())


if __name__ == "__main__":
    import sys
    import time

    if "--write" in sys.argv:
        os.makedirs(_DATA_DIR, exist_ok=True)
        for name, cfg in CONFIGS.items():
            if not cfg.get("stored"):
                continue
            t0 = time.time()
            forest = make_forest(cfg["build"]())
            with open(os.path.join(_DATA_DIR, cfg["stored"]), "w") as f:
                json.dump(forest.to_json(), f)
            print(name, "nodes", forest.n_nodes, "tokens", forest.n_tokens, "sec", round(time.time() - t0, 1))
    else:
        for name in CONFIGS:
            fo = config_forest(name)
            c = s = 0
            for t in range(fo.n_trees):
                ci, si, _ = tree_counts(*(a.tolist() for a in fo.tree(t)))
                c += ci
                s += si
            print(name, "trees", fo.n_trees, "nodes", fo.n_nodes, "C", c, "S", s, "S/C", round(s / c, 3))
