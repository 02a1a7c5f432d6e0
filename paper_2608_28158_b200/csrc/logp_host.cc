// Host side of the compact-to-semantic log-probability (Section 3.5, Eqs. 17 and 19): the list of
// non-terminal semantic positions with their compact row m(s) and target y_s, and the grouping of
// positions by row that the backward sums over.
#include <cstdint>
#include <utility>
#include <vector>

#include "../../include/harts_logp.h"

namespace {

// Same admissibility rules as the planner: parents precede children, fork offsets lie in 1..len(parent).
bool forest_ok(int32_t n_trees, const int32_t* ptr, const int32_t* par, const int32_t* off, const int32_t* len,
               int64_t* n_tokens) {
    if (n_trees < 0 || !ptr || ptr[0] != 0) return false;
    int64_t total = 0;
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = ptr[t], hi = ptr[t + 1];
        if (hi <= lo) return false;
        for (int32_t i = lo; i < hi; ++i) {
            if (len[i] < 1) return false;
            if (i == lo) {
                if (par[i] != -1 || off[i] != 0) return false;
            } else {
                if (par[i] < 0 || par[i] >= i - lo) return false;
                if (off[i] < 1 || off[i] > len[lo + par[i]]) return false;
            }
            total += len[i];
        }
    }
    if (total >= INT32_MAX) return false;
    *n_tokens = total;
    return true;
}

}  // namespace

extern "C" int32_t harts_logp_positions(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                        const int32_t* node_fork_off, const int32_t* node_len,
                                        const int32_t* row_of_token, const int32_t* token_id, int64_t cap, int32_t* m,
                                        int32_t* y, int64_t* traj_pos_ptr, int64_t* n_pos, int64_t* n_traj) {
    if (!node_parent || !node_fork_off || !node_len || !n_pos || !n_traj) return HARTS_EINVAL;
    if ((m == nullptr) != (y == nullptr)) return HARTS_EINVAL;
    int64_t C = 0;
    if (!forest_ok(n_trees, tree_node_ptr, node_parent, node_fork_off, node_len, &C)) return HARTS_EINVAL;
    const int32_t n_nodes = n_trees ? tree_node_ptr[n_trees] : 0;
    std::vector<int64_t> base(n_nodes + 1, 0);            // canonical index of each node's first token
    for (int32_t i = 0; i < n_nodes; ++i) base[i + 1] = base[i] + node_len[i];
    std::vector<int64_t> start(n_nodes, 0);               // tokens of the trajectory that precede the node
    std::vector<char> continued(n_nodes, 0);              // a child starts exactly at the node's end
    int64_t P = 0, T = 0;
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t i = lo + 1; i < hi; ++i) {
            const int32_t p = lo + node_parent[i];
            start[i] = start[p] + node_fork_off[i];
            if (node_fork_off[i] == node_len[p]) continued[p] = 1;
        }
        for (int32_t i = lo; i < hi; ++i)
            if (!continued[i]) { P += start[i] + node_len[i] - 1; ++T; }
    }
    *n_pos = P;
    *n_traj = T;
    if (!m) return HARTS_OK;
    if (cap < P || !token_id) return HARTS_EINVAL;
    if (P >= INT32_MAX) return HARTS_EINVAL;              // position ids are int32 in the row CSR

    std::vector<int32_t> chain;
    int64_t s = 0, x = 0;
    auto row = [&](int64_t canon) { return row_of_token ? row_of_token[canon] : static_cast<int32_t>(canon); };
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t leaf = lo; leaf < hi; ++leaf) {
            if (continued[leaf]) continue;
            chain.clear();
            for (int32_t v = leaf; v >= lo; v = (v == lo ? -1 : lo + node_parent[v])) chain.push_back(v);
            if (traj_pos_ptr) traj_pos_ptr[x] = s;
            ++x;
            // walk root -> leaf; node chain[j] contributes its first `upto` tokens
            int64_t prev = -1;                            // canonical index of the previous token of the path
            for (size_t j = chain.size(); j-- > 0;) {
                const int32_t v = chain[j];
                const int32_t upto = (j == 0) ? node_len[v] : node_fork_off[chain[j - 1]];
                for (int32_t o = 0; o < upto; ++o) {
                    const int64_t cur = base[v] + o;
                    if (prev >= 0) {
                        m[s] = row(prev);
                        y[s] = token_id[cur];
                        ++s;
                    }
                    prev = cur;
                }
            }
        }
    }
    if (traj_pos_ptr) traj_pos_ptr[x] = s;
    return s == P ? HARTS_OK : HARTS_EINTERNAL;
}

extern "C" int32_t harts_logp_csr(int32_t n_rows, int64_t n_pos, const int32_t* m, int32_t* row_pos_ptr,
                                  int32_t* row_pos) {
    if (n_rows < 0 || n_pos < 0 || n_pos >= INT32_MAX || !row_pos_ptr || (n_pos && (!m || !row_pos)))
        return HARTS_EINVAL;
    for (int64_t s = 0; s < n_pos; ++s)
        if (m[s] < 0 || m[s] >= n_rows) return HARTS_EINVAL;
    for (int32_t c = 0; c <= n_rows; ++c) row_pos_ptr[c] = 0;
    for (int64_t s = 0; s < n_pos; ++s) ++row_pos_ptr[m[s] + 1];
    for (int32_t c = 0; c < n_rows; ++c) row_pos_ptr[c + 1] += row_pos_ptr[c];
    std::vector<int32_t> fill(row_pos_ptr, row_pos_ptr + n_rows);
    for (int64_t s = 0; s < n_pos; ++s) row_pos[fill[m[s]]++] = static_cast<int32_t>(s);
    return HARTS_OK;
}

extern "C" int32_t harts_logp_multiplicity(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                           const int32_t* node_fork_off, const int32_t* node_len,
                                           const int32_t* row_of_token, int64_t n_rows, int32_t* mult) {
    if (!node_parent || !node_fork_off || !node_len || !mult) return HARTS_EINVAL;
    int64_t C = 0;
    if (!forest_ok(n_trees, tree_node_ptr, node_parent, node_fork_off, node_len, &C)) return HARTS_EINVAL;
    if (n_rows < C) return HARTS_EINVAL;
    if (row_of_token)
        for (int64_t c = 0; c < C; ++c)
            if (row_of_token[c] < 0 || row_of_token[c] >= n_rows) return HARTS_EINVAL;
    const int32_t n_nodes = n_trees ? tree_node_ptr[n_trees] : 0;
    for (int64_t r = 0; r < n_rows; ++r) mult[r] = 0;
    std::vector<int64_t> base(n_nodes + 1, 0);
    for (int32_t i = 0; i < n_nodes; ++i) base[i + 1] = base[i] + node_len[i];
    // through[i]: trajectories that contain node i's first token.  Children come after their parent, so one reverse
    // sweep sees every child before its parent.  add[o] of a node: trajectories that leave it right after its token
    // o - 1 (children forking at offset o; at o = len also the node's own end if no child continues it).
    std::vector<int64_t> through(n_nodes, 0);
    std::vector<std::vector<std::pair<int32_t, int64_t>>> forks(n_nodes);   // (fork offset, trajectories) per parent
    for (int32_t t = n_trees - 1; t >= 0; --t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t i = hi - 1; i >= lo; --i) {
            auto& f = forks[i];
            bool continued = false;
            int64_t total = 0;
            for (auto& e : f) {
                continued = continued || e.first == node_len[i];
                total += e.second;
            }
            if (!continued) total += 1;                   // the node's end is a trajectory end
            through[i] = total;
            if (total >= INT32_MAX) return HARTS_EINVAL;
            // tokens o = len-1 .. 0: a token at offset o is on every trajectory that leaves at an offset > o
            std::vector<int64_t> leave(node_len[i] + 1, 0);
            for (auto& e : f) leave[e.first] += e.second;
            if (!continued) leave[node_len[i]] += 1;
            int64_t run = 0;
            for (int32_t o = node_len[i] - 1; o >= 0; --o) {
                run += leave[o + 1];
                const int64_t canon = base[i] + o;
                mult[row_of_token ? row_of_token[canon] : canon] = static_cast<int32_t>(run);
            }
            if (i > lo) forks[lo + node_parent[i]].emplace_back(node_fork_off[i], total);
            std::vector<std::pair<int32_t, int64_t>>().swap(f);
        }
    }
    return HARTS_OK;
}
