// Host index for attention on compact tokens (Section 3.4, Eqs. 21-22): pieces of the tree in physical rows, their
// ancestor rows and descendant pieces, and the work lists of the forward (query tiles) and backward (key tiles).
#include <algorithm>
#include <cstdint>
#include <numeric>
#include <vector>

#include "../../include/harts_attn.h"

namespace {
constexpr int TILE = 128;
}

extern "C" int32_t harts_attn_index(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                    const int32_t* node_fork_off, const int32_t* node_len,
                                    const int32_t* row_of_token, int64_t cap_words, int32_t* blob, int64_t* n_words) {
    if (n_trees < 0 || !tree_node_ptr || !node_parent || !node_fork_off || !node_len || !n_words) return HARTS_EINVAL;
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
    auto row = [&](int64_t canon) { return row_of_token ? row_of_token[canon] : static_cast<int32_t>(canon); };
    if (row_of_token) {
        std::vector<char> seen(C, 0);
        for (int64_t c = 0; c < C; ++c) {
            const int32_t r = row_of_token[c];
            if (r < 0 || r >= C || seen[r]) return HARTS_EINVAL;
            seen[r] = 1;
        }
    }
    // predecessor and number of successors of every physical row
    std::vector<int32_t> prev(C), n_child(C, 0);
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        for (int32_t i = lo; i < hi; ++i) {
            const int64_t p0 = i == lo ? -1 : base[lo + node_parent[i]] + node_fork_off[i] - 1;
            prev[row(base[i])] = p0 < 0 ? -1 : row(p0);
            for (int64_t c = base[i] + 1; c < base[i + 1]; ++c) prev[row(c)] = row(c - 1);
        }
    }
    for (int64_t r = 0; r < C; ++r)
        if (prev[r] >= 0) ++n_child[prev[r]];
    // pieces: row r continues the piece of row r-1 iff r-1 is its predecessor and r is r-1's only successor
    std::vector<int32_t> piece_of(C), p_row0, p_len, p_parent;
    for (int64_t r = 0; r < C; ++r) {
        const bool cont = r > 0 && prev[r] == r - 1 && n_child[r - 1] == 1;
        if (!cont) {
            p_row0.push_back(static_cast<int32_t>(r));
            p_len.push_back(0);
        }
        piece_of[r] = static_cast<int32_t>(p_row0.size()) - 1;
        ++p_len.back();
    }
    const int32_t P = static_cast<int32_t>(p_row0.size());
    p_parent.resize(P);
    for (int32_t p = 0; p < P; ++p) {
        const int32_t a = prev[p_row0[p]];
        p_parent[p] = a < 0 ? -1 : piece_of[a];
        // the predecessor must close its piece, so that ancestors are whole pieces
        if (a >= 0 && a != p_row0[p_parent[p]] + p_len[p_parent[p]] - 1) return HARTS_EINTERNAL;
    }
    // ancestor runs (root first, physically adjacent pieces merged) and descendant lists
    std::vector<int32_t> anc_ptr(P + 1, 0), anc_row0, anc_len, desc_ptr(P + 1, 0), desc_piece;
    std::vector<int64_t> anc_total(P, 0), desc_total(P, 0);
    std::vector<int32_t> chain;
    std::vector<std::vector<int32_t>> desc(P);
    for (int32_t p = 0; p < P; ++p) {
        chain.clear();
        for (int32_t a = p_parent[p]; a >= 0; a = p_parent[a]) chain.push_back(a);
        for (size_t j = chain.size(); j-- > 0;) {
            const int32_t a = chain[j];
            desc[a].push_back(p);
            desc_total[a] += p_len[p];
            anc_total[p] += p_len[a];
            if (!anc_row0.empty() && static_cast<int32_t>(anc_row0.size()) > anc_ptr[p] &&
                anc_row0.back() + anc_len.back() == p_row0[a])
                anc_len.back() += p_len[a];
            else {
                anc_row0.push_back(p_row0[a]);
                anc_len.push_back(p_len[a]);
            }
        }
        anc_ptr[p + 1] = static_cast<int32_t>(anc_row0.size());
    }
    for (int32_t p = 0; p < P; ++p) {
        desc_piece.insert(desc_piece.end(), desc[p].begin(), desc[p].end());
        desc_ptr[p + 1] = static_cast<int32_t>(desc_piece.size());
    }
    // work lists, most work first (stable, so the order is reproducible)
    struct Item { int32_t piece, tile; int64_t work; };
    std::vector<Item> qi, ki;
    for (int32_t p = 0; p < P; ++p)
        for (int32_t t = 0; t * TILE < p_len[p]; ++t) {
            const int64_t q_rows = std::min<int64_t>(TILE, p_len[p] - (int64_t)t * TILE);
            qi.push_back({p, t, q_rows * (anc_total[p] + std::min<int64_t>(p_len[p], (int64_t)(t + 1) * TILE))});
            ki.push_back({p, t, q_rows * (desc_total[p] + p_len[p] - (int64_t)t * TILE)});
        }
    auto by_work = [](const Item& a, const Item& b) { return a.work > b.work; };
    std::stable_sort(qi.begin(), qi.end(), by_work);
    std::stable_sort(ki.begin(), ki.end(), by_work);

    const std::vector<int32_t>* arrays[] = {&p_row0, &p_len, &p_parent, &anc_ptr, &anc_row0, &anc_len, &desc_ptr,
                                            &desc_piece};
    int64_t total = HARTS_ATTN_HEADER_WORDS;
    int64_t offs[10];
    for (int i = 0; i < 8; ++i) {
        offs[i] = total;
        total += (static_cast<int64_t>(arrays[i]->size()) + 3) & ~int64_t(3);      // 16-byte aligned starts
    }
    offs[8] = total;
    total += (2 * static_cast<int64_t>(qi.size()) + 3) & ~int64_t(3);
    offs[9] = total;
    total += (2 * static_cast<int64_t>(ki.size()) + 3) & ~int64_t(3);
    if (total >= INT32_MAX) return HARTS_EINVAL;
    *n_words = total;
    if (!blob) return HARTS_OK;
    if (cap_words < total) return HARTS_EINVAL;
    std::fill(blob, blob + total, 0);
    blob[0] = static_cast<int32_t>(C);
    blob[1] = P;
    blob[2] = static_cast<int32_t>(anc_row0.size());
    blob[3] = static_cast<int32_t>(desc_piece.size());
    blob[4] = static_cast<int32_t>(qi.size());
    blob[5] = static_cast<int32_t>(ki.size());
    blob[6] = static_cast<int32_t>(total);
    for (int i = 0; i < 10; ++i) blob[8 + i] = static_cast<int32_t>(offs[i]);
    for (int i = 0; i < 8; ++i) std::copy(arrays[i]->begin(), arrays[i]->end(), blob + offs[i]);
    for (size_t i = 0; i < qi.size(); ++i) {
        blob[offs[8] + 2 * i] = qi[i].piece;
        blob[offs[8] + 2 * i + 1] = qi[i].tile;
    }
    for (size_t i = 0; i < ki.size(); ++i) {
        blob[offs[9] + 2 * i] = ki[i].piece;
        blob[offs[9] + 2 * i + 1] = ki[i].tile;
    }
    return HARTS_OK;
}
