// Trajectory-wise view of a forest (the conventional execution that Section 5 compares with): every root-to-leaf
// trajectory on its own, with the compact token each of its positions maps to (the map m of Eq. 3).
#include <cstdint>
#include <vector>

#include "../../include/harts_la.h"

extern "C" int32_t harts_la_expand(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                   const int32_t* node_fork_off, const int32_t* node_len, int64_t cap_traj,
                                   int64_t cap_tokens, int32_t* traj_len, int64_t* src_token, int64_t* n_traj,
                                   int64_t* n_tokens) {
    if (n_trees < 1 || !tree_node_ptr || !node_parent || !node_fork_off || !node_len || !n_traj || !n_tokens)
        return HARTS_EINVAL;
    if (tree_node_ptr[0] != 0) return HARTS_EINVAL;
    const int32_t n_nodes = tree_node_ptr[n_trees];
    std::vector<int64_t> base(static_cast<size_t>(n_nodes) + 1, 0);      // canonical index of a node's first token
    std::vector<int64_t> depth(n_nodes, 0);                              // tokens on the path before the node
    std::vector<char> continued(n_nodes, 0);                             // a child forks at the node's very end
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        if (hi <= lo) return HARTS_EINVAL;
        for (int32_t i = lo; i < hi; ++i) {
            if (node_len[i] < 1) return HARTS_EINVAL;
            base[i + 1] = base[i] + node_len[i];
            if (i == lo) {
                if (node_parent[i] != -1) return HARTS_EINVAL;
                continue;
            }
            const int32_t p = node_parent[i];
            if (p < 0 || lo + p >= i || node_fork_off[i] < 1 || node_fork_off[i] > node_len[lo + p]) return HARTS_EINVAL;
            depth[i] = depth[lo + p] + node_fork_off[i];
            if (node_fork_off[i] == node_len[lo + p]) continued[lo + p] = 1;
        }
    }
    // a trajectory ends in every node that no child continues from its last token
    int64_t traj = 0, tokens = 0;
    const bool fill = traj_len != nullptr || src_token != nullptr;
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t leaf = lo; leaf < hi; ++leaf) {
            if (continued[leaf]) continue;
            const int64_t len = depth[leaf] + node_len[leaf];
            if (fill) {
                if (!traj_len || !src_token || traj >= cap_traj || tokens + len > cap_tokens) return HARTS_EINVAL;
                if (len > INT32_MAX) return HARTS_EINVAL;
                traj_len[traj] = static_cast<int32_t>(len);
                // walk up from the leaf, writing each node's used tokens at its place on the path
                int32_t node = leaf;
                int64_t upto = node_len[leaf];
                while (true) {
                    int64_t* dst = src_token + tokens + depth[node];
                    for (int64_t j = 0; j < upto; ++j) dst[j] = base[node] + j;
                    if (node_parent[node] < 0) break;
                    upto = node_fork_off[node];
                    node = lo + node_parent[node];
                }
            }
            ++traj;
            tokens += len;
        }
    }
    *n_traj = traj;
    *n_tokens = tokens;
    return HARTS_OK;
}
