// Host side of the tree-aware causal convolution (Section 4.2): predecessor and successor tables in physical rows.
#include <cstdint>
#include <vector>

#include "../../include/harts_conv.h"

extern "C" int32_t harts_conv_index(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                    const int32_t* node_fork_off, const int32_t* node_len,
                                    const int32_t* row_of_token, int32_t* prev_row, int32_t* next_row,
                                    int32_t* child_ptr, int32_t* child_row) {
    if (n_trees < 0 || !tree_node_ptr || !node_parent || !node_fork_off || !node_len || !prev_row || !next_row || !child_ptr)
        return HARTS_EINVAL;
    if (tree_node_ptr[0] != 0) return HARTS_EINVAL;
    const int32_t n_nodes = tree_node_ptr[n_trees];
    std::vector<int64_t> base(n_nodes + 1, 0);
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        if (hi <= lo) return HARTS_EINVAL;
        for (int32_t i = lo; i < hi; ++i) {
            if (node_len[i] < 1) return HARTS_EINVAL;
            if (i == lo ? (node_parent[i] != -1 || node_fork_off[i] != 0)
                        : (node_parent[i] < 0 || node_parent[i] >= i - lo || node_fork_off[i] < 1 ||
                           node_fork_off[i] > node_len[lo + node_parent[i]]))
                return HARTS_EINVAL;
            base[i + 1] = base[i] + node_len[i];
        }
    }
    const int64_t C = base[n_nodes];
    if (C >= INT32_MAX) return HARTS_EINVAL;
    if (C - n_trees > 0 && !child_row) return HARTS_EINVAL;
    auto row = [&](int64_t canon) { return row_of_token ? row_of_token[canon] : static_cast<int32_t>(canon); };
    if (row_of_token) {                               // must be a permutation of 0..C-1
        std::vector<char> seen(C, 0);
        for (int64_t c = 0; c < C; ++c) {
            const int32_t r = row_of_token[c];
            if (r < 0 || r >= C || seen[r]) return HARTS_EINVAL;
            seen[r] = 1;
        }
    }
    // canonical predecessor of every token, then the same in physical rows
    std::vector<int64_t> pred(C);
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t i = lo; i < hi; ++i) {
            pred[base[i]] = i == lo ? -1 : base[lo + node_parent[i]] + node_fork_off[i] - 1;
            for (int64_t c = base[i] + 1; c < base[i + 1]; ++c) pred[c] = c - 1;
        }
    }
    for (int64_t r = 0; r <= C; ++r) child_ptr[r] = 0;
    for (int64_t c = 0; c < C; ++c) {
        prev_row[row(c)] = pred[c] < 0 ? -1 : row(pred[c]);
        if (pred[c] >= 0) ++child_ptr[row(pred[c]) + 1];
    }
    for (int64_t r = 0; r < C; ++r) child_ptr[r + 1] += child_ptr[r];
    std::vector<int32_t> fill(child_ptr, child_ptr + C);
    for (int64_t c = 0; c < C; ++c)                   // canonical order of the children of one row
        if (pred[c] >= 0) child_row[fill[row(pred[c])]++] = row(c);
    for (int64_t r = 0; r < C; ++r) {
        const int32_t n = child_ptr[r + 1] - child_ptr[r];
        next_row[r] = n == 0 ? -1 : (n == 1 ? child_row[child_ptr[r]] : -2);
    }
    return HARTS_OK;
}
