// Host-side minimum-call planner (paper Section 3.3, Algorithm 1) and compact physical layout
// (Section 4.2).  Integer work only; everything is iterative (explicit stacks) so that deep
// continuation chains cannot overflow the call stack.
//
// Pipeline: node forest -> segment tree per rollout tree (maximal fork-free token paths) ->
// T_pre / T_in (Eqs. 11-14) -> recovery of sequences, rounds, state sources and replay spans ->
// global ordering of sequences, physical rows, slots and the backward CSR tables.
#include "plan.h"

#include <algorithm>
#include <cstring>
#include <new>

namespace harts {
namespace {

struct Piece {
    int32_t node;  // tree-local node
    int32_t lo, hi;
};

struct Seg {
    int64_t s, e;          // absolute token positions [s, e)
    int32_t piece_begin;   // into pieces
    int32_t piece_count;
    int32_t parent;        // segment index, -1 for the root
    int32_t child_begin;   // into child_list
    int32_t child_count;
    int32_t t_pre, t_in;
};

struct SeqTmp {
    int32_t round;         // 1-based
    int64_t start;         // start anchor
    int32_t producer;      // temporary index of the producing sequence, -1 = zero state
    int32_t chunk;         // chunk index in the producer
    int32_t replay_from;   // segment at whose end this sequence forks, -1 for a root sequence
    int32_t tree;
    int32_t seg_base;      // tree's first segment in the global segment array
    int64_t first_token;   // canonical index of the first own token
    std::vector<int32_t> segs;   // tree-local segment ids, chain order
};

inline int64_t anchor(int64_t p, int64_t B) { return B * (p / B); }  // Eq. 2

struct TreeBuilder {
    const int32_t *par, *off, *len;
    int32_t n;
    std::vector<int32_t> kid_ptr, kids;   // children of every node, sorted by (fork offset, input order)
    std::vector<Seg> segs;
    std::vector<Piece> pieces;
    std::vector<int32_t> child_list;

    void group_children() {
        kid_ptr.assign(n + 1, 0);
        for (int32_t i = 1; i < n; i++) kid_ptr[par[i] + 1]++;
        for (int32_t i = 0; i < n; i++) kid_ptr[i + 1] += kid_ptr[i];
        kids.resize(n > 0 ? n - 1 : 0);
        std::vector<int32_t> fill(kid_ptr.begin(), kid_ptr.end() - 1);
        for (int32_t i = 1; i < n; i++) kids[fill[par[i]]++] = i;
        for (int32_t v = 0; v < n; v++)
            std::stable_sort(kids.begin() + kid_ptr[v], kids.begin() + kid_ptr[v + 1],
                             [&](int32_t a, int32_t b) { return off[a] < off[b]; });
    }

    void build() {
        group_children();
        // kid: index into kids of the first child of `node` that forks after offset lo
        struct Item { int32_t node, lo, kid; int64_t abs_lo; int32_t parent, slot; };
        std::vector<Item> stack;
        stack.push_back({0, 0, kid_ptr[0], 0, -1, -1});
        while (!stack.empty()) {
            Item it = stack.back();
            stack.pop_back();
            int32_t idx = (int32_t)segs.size();
            if (it.slot >= 0) child_list[it.slot] = idx;
            Seg sg{it.abs_lo, it.abs_lo, (int32_t)pieces.size(), 0, it.parent, 0, 0, 0, 0};
            int32_t node = it.node, lo = it.lo, a = it.kid;
            // (child node, offset, first kid) of the fork that ends this segment
            struct Child { int32_t node, lo, kid; };
            std::vector<Child> ch;
            for (;;) {
                int32_t hi = a < kid_ptr[node + 1] ? off[kids[a]] : len[node];
                pieces.push_back({node, lo, hi});
                sg.piece_count++;
                sg.e += hi - lo;
                int32_t b = a;
                while (b < kid_ptr[node + 1] && off[kids[b]] == hi) b++;
                int32_t forked = b - a;
                if (hi < len[node]) {            // fork inside the node: its own continuation comes first
                    ch.push_back({node, hi, b});
                    for (int32_t j = a; j < b; j++) ch.push_back({kids[j], 0, kid_ptr[kids[j]]});
                    break;
                }
                if (forked == 1) {               // single child at the node's end: same segment
                    node = kids[a];
                    lo = 0;
                    a = kid_ptr[node];
                    continue;
                }
                for (int32_t j = a; j < b; j++) ch.push_back({kids[j], 0, kid_ptr[kids[j]]});
                break;
            }
            sg.child_begin = (int32_t)child_list.size();
            sg.child_count = (int32_t)ch.size();
            child_list.resize(child_list.size() + ch.size(), -1);
            segs.push_back(sg);
            for (int32_t j = (int32_t)ch.size() - 1; j >= 0; j--)
                stack.push_back({ch[j].node, ch[j].lo, ch[j].kid, sg.e, idx, sg.child_begin + j});
        }
    }

    // Algorithm 1, first pass.  Parents are created before their children, so a reverse sweep is
    // a valid post-order.  h_o = max over the other children comes from the two largest T_pre.
    void call_counts(int64_t B) {
        for (int32_t v = (int32_t)segs.size() - 1; v >= 0; v--) {
            Seg& sg = segs[v];
            if (sg.child_count == 0) {
                sg.t_pre = sg.t_in = 1;   // Eq. 12
                continue;
            }
            int32_t big = 0, second = 0, big_count = 0;
            for (int32_t j = 0; j < sg.child_count; j++) {
                int32_t t = segs[child_list[sg.child_begin + j]].t_pre;
                if (t > big) { second = big; big = t; big_count = 1; }
                else if (t == big) big_count++;
                else if (t > second) second = t;
            }
            int32_t best = INT32_MAX;
            for (int32_t j = 0; j < sg.child_count; j++) {
                const Seg& o = segs[child_list[sg.child_begin + j]];
                int32_t h = (o.t_pre == big && big_count == 1) ? second : big;
                best = std::min(best, std::max(o.t_in, 1 + h));   // Eq. 13
            }
            sg.t_in = best;
            sg.t_pre = (sg.e < anchor(sg.s, B) + B) ? big : best;   // Eq. 14 with Eq. 11
        }
    }
};

}  // namespace

int32_t build_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                   const int32_t* node_fork_off, const int32_t* node_len, int32_t chunk, Plan& P) {
    if (n_trees < 1 || !tree_node_ptr || !node_parent || !node_fork_off || !node_len || chunk < 1)
        return HARTS_EINVAL;
    if (tree_node_ptr[0] != 0) return HARTS_EINVAL;
    const int64_t B = chunk;
    int64_t total_tokens = 0;
    for (int32_t t = 0; t < n_trees; t++) {
        int32_t lo = tree_node_ptr[t], hi = tree_node_ptr[t + 1];
        if (hi <= lo) return HARTS_EINVAL;
        for (int32_t i = lo; i < hi; i++) {
            int32_t p = node_parent[i];
            if (node_len[i] < 1) return HARTS_EINVAL;
            if (i == lo) {
                if (p != -1 || node_fork_off[i] != 0) return HARTS_EINVAL;
            } else {
                if (p < 0 || p >= i - lo) return HARTS_EINVAL;
                if (node_fork_off[i] < 1 || node_fork_off[i] > node_len[lo + p]) return HARTS_EINVAL;
            }
            total_tokens += node_len[i];
        }
    }
    if (total_tokens >= INT32_MAX) return HARTS_EINVAL;
    const int32_t n_nodes = tree_node_ptr[n_trees];
    std::vector<int64_t> token_base(n_nodes + 1, 0);
    for (int32_t i = 0; i < n_nodes; i++) token_base[i + 1] = token_base[i] + node_len[i];

    // ---- per tree: segments, call counts, recovery -------------------------------------------
    std::vector<Seg> all_segs;
    std::vector<Piece> all_pieces;        // node index made global
    std::vector<SeqTmp> seqs;
    int64_t replay_total = 0;
    int32_t n_rounds = 0;
    for (int32_t t = 0; t < n_trees; t++) {
        int32_t lo = tree_node_ptr[t];
        TreeBuilder tb;
        tb.par = node_parent + lo;
        tb.off = node_fork_off + lo;
        tb.len = node_len + lo;
        tb.n = tree_node_ptr[t + 1] - lo;
        tb.build();
        tb.call_counts(B);
        n_rounds = std::max(n_rounds, tb.segs[0].t_pre);

        const int32_t seg_base = (int32_t)all_segs.size();
        const int32_t piece_base = (int32_t)all_pieces.size();
        auto first_token_of = [&](int32_t v) {
            const Piece& pc = tb.pieces[tb.segs[v].piece_begin];
            return token_base[lo + pc.node] + pc.lo;
        };

        // recovery (Algorithm 1, procedure Recover), iterative
        struct Frame { int32_t v; bool ready; int32_t k_round, r, seq; };
        std::vector<Frame> stack;
        const int32_t root_seq = (int32_t)seqs.size();
        seqs.push_back(SeqTmp{1, 0, -1, 0, -1, t, seg_base, first_token_of(0), {}});
        stack.push_back({0, true, tb.segs[0].t_pre, 1, root_seq});
        while (!stack.empty()) {
            Frame f = stack.back();
            stack.pop_back();
            seqs[f.seq].segs.push_back(f.v);
            const Seg& sg = tb.segs[f.v];
            if (sg.child_count == 0) continue;
            if (sg.child_count >= 2) replay_total += (int64_t)(sg.child_count - 1) * (sg.e % B);  // Eq. 15
            const int64_t a_v = anchor(sg.s, B), b_v = anchor(sg.e, B);
            const bool same = f.ready && sg.e < a_v + B;
            const int32_t delta = same ? 0 : 1;
            const int32_t k_side = f.k_round - delta;
            int32_t over = 0;
            for (int32_t j = 0; j < sg.child_count; j++)
                over += tb.segs[tb.child_list[sg.child_begin + j]].t_pre > k_side;
            int32_t direct = -1;
            for (int32_t j = 0; j < sg.child_count && direct < 0; j++) {
                int32_t o = tb.child_list[sg.child_begin + j];
                int32_t budget = same ? tb.segs[o].t_pre : tb.segs[o].t_in;
                if (budget <= f.k_round && over - (tb.segs[o].t_pre > k_side ? 1 : 0) == 0) direct = o;
            }
            if (direct < 0) return HARTS_EINTERNAL;
            stack.push_back({direct, same, f.k_round, f.r, f.seq});
            for (int32_t j = 0; j < sg.child_count; j++) {
                int32_t u = tb.child_list[sg.child_begin + j];
                if (u == direct) continue;
                SeqTmp q;
                q.tree = t;
                q.seg_base = seg_base;
                q.replay_from = f.v;
                q.first_token = first_token_of(u);
                if (same) {          // launched in round r from the open sequence's own initial state
                    q.round = f.r;
                    q.start = seqs[f.seq].start;
                    q.producer = seqs[f.seq].producer;
                    q.chunk = seqs[f.seq].chunk;
                } else {             // S_{b_v} is requested from the open sequence; next round
                    q.round = f.r + 1;
                    q.start = b_v;
                    q.producer = f.seq;
                    q.chunk = (int32_t)((b_v - seqs[f.seq].start) / B);
                    if (q.chunk < 1) return HARTS_EINTERNAL;
                }
                int32_t id = (int32_t)seqs.size();
                seqs.push_back(std::move(q));
                stack.push_back({u, true, k_side, f.r + delta, id});
            }
        }
        for (const Seg& s : tb.segs) {
            Seg g = s;
            g.piece_begin += piece_base;
            all_segs.push_back(g);
        }
        for (const Piece& p : tb.pieces) all_pieces.push_back({p.node + lo, p.lo, p.hi});
    }

    // ---- global sequence order: (round, canonical index of the first own token) ---------------
    const int32_t n_seq = (int32_t)seqs.size();
    std::vector<int32_t> order(n_seq), new_index(n_seq);
    for (int32_t i = 0; i < n_seq; i++) order[i] = i;
    std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
        if (seqs[a].round != seqs[b].round) return seqs[a].round < seqs[b].round;
        return seqs[a].first_token < seqs[b].first_token;
    });
    for (int32_t i = 0; i < n_seq; i++) new_index[order[i]] = i;

    const int32_t C = (int32_t)total_tokens;
    P.chunk = chunk;
    P.n_rounds = n_rounds;
    P.n_rows = C;
    P.n_replay = (int32_t)replay_total;
    P.n_seq = n_seq;
    P.row_of_token.assign(C, -1);
    P.round_seq_ptr.assign(n_rounds + 1, 0);
    P.seq_tree.resize(n_seq);
    P.seq_own_begin.resize(n_seq + 1);
    P.seq_own_len.resize(n_seq);
    P.seq_start_pos.resize(n_seq);
    P.seq_init_slot.assign(n_seq, -1);
    P.seq_replay_ptr.assign(n_seq + 1, 0);
    P.replay_row.clear();
    P.replay_row.reserve((size_t)replay_total);

    // physical rows
    int32_t row = 0;
    for (int32_t i = 0; i < n_seq; i++) {
        const SeqTmp& q = seqs[order[i]];
        P.round_seq_ptr[q.round]++;
        P.seq_tree[i] = q.tree;
        P.seq_start_pos[i] = (int32_t)q.start;
        P.seq_own_begin[i] = row;
        for (int32_t v : q.segs) {
            const Seg& sg = all_segs[q.seg_base + v];
            for (int32_t p = 0; p < sg.piece_count; p++) {
                const Piece& pc = all_pieces[sg.piece_begin + p];
                int64_t base = token_base[pc.node];
                for (int32_t o = pc.lo; o < pc.hi; o++) P.row_of_token[base + o] = row++;
            }
        }
        P.seq_own_len[i] = row - P.seq_own_begin[i];
    }
    P.seq_own_begin[n_seq] = row;
    if (row != C) return HARTS_EINTERNAL;
    for (int32_t r = 0; r < n_rounds; r++) P.round_seq_ptr[r + 1] += P.round_seq_ptr[r];

    // replay rows: absolute positions [start, s_first) along the ancestor path, in path order
    std::vector<int32_t> rev;
    for (int32_t i = 0; i < n_seq; i++) {
        const SeqTmp& q = seqs[order[i]];
        const Seg& first = all_segs[q.seg_base + q.segs[0]];
        int64_t need = first.s - q.start;
        if (need < 0 || need >= B || q.start % B != 0) return HARTS_EINTERNAL;
        rev.clear();
        int32_t v = q.replay_from;
        while (need > 0) {
            if (v < 0) return HARTS_EINTERNAL;
            const Seg& sg = all_segs[q.seg_base + v];
            for (int32_t p = sg.piece_count - 1; p >= 0 && need > 0; p--) {
                const Piece& pc = all_pieces[sg.piece_begin + p];
                int64_t base = token_base[pc.node];
                for (int32_t o = pc.hi - 1; o >= pc.lo && need > 0; o--, need--)
                    rev.push_back(P.row_of_token[base + o]);
            }
            v = sg.parent;
        }
        for (auto it = rev.rbegin(); it != rev.rend(); ++it) P.replay_row.push_back(*it);
        P.seq_replay_ptr[i + 1] = (int32_t)P.replay_row.size();
    }
    if ((int64_t)P.replay_row.size() != replay_total) return HARTS_EINTERNAL;

    // slots: unique (producer, chunk) pairs, numbered in (producer sequence, chunk) order
    std::vector<std::pair<int32_t, int32_t>> wanted;
    for (int32_t i = 0; i < n_seq; i++) {
        const SeqTmp& q = seqs[order[i]];
        if (q.producer >= 0) wanted.push_back({new_index[q.producer], q.chunk});
    }
    std::sort(wanted.begin(), wanted.end());
    wanted.erase(std::unique(wanted.begin(), wanted.end()), wanted.end());
    const int32_t n_slots = (int32_t)wanted.size();
    P.n_slots = n_slots;
    P.seq_req_ptr.assign(n_seq + 1, 0);
    P.slot_chunk.resize(n_slots);
    for (int32_t s = 0; s < n_slots; s++) {
        P.seq_req_ptr[wanted[s].first + 1]++;
        P.slot_chunk[s] = wanted[s].second;
    }
    for (int32_t i = 0; i < n_seq; i++) P.seq_req_ptr[i + 1] += P.seq_req_ptr[i];
    P.slot_cons_ptr.assign(n_slots + 1, 0);
    for (int32_t i = 0; i < n_seq; i++) {
        const SeqTmp& q = seqs[order[i]];
        if (q.producer < 0) continue;
        auto key = std::make_pair(new_index[q.producer], q.chunk);
        int32_t s = (int32_t)(std::lower_bound(wanted.begin(), wanted.end(), key) - wanted.begin());
        P.seq_init_slot[i] = s;
        P.slot_cons_ptr[s + 1]++;
    }
    for (int32_t s = 0; s < n_slots; s++) P.slot_cons_ptr[s + 1] += P.slot_cons_ptr[s];
    P.slot_cons_seq.resize(P.slot_cons_ptr[n_slots]);
    {
        std::vector<int32_t> fill(P.slot_cons_ptr.begin(), P.slot_cons_ptr.end() - 1);
        for (int32_t i = 0; i < n_seq; i++)
            if (P.seq_init_slot[i] >= 0) P.slot_cons_seq[fill[P.seq_init_slot[i]]++] = i;
    }

    // chunk counts
    P.seq_chunk_ptr.assign(n_seq + 1, 0);
    for (int32_t i = 0; i < n_seq; i++) {
        int64_t virt = (int64_t)(P.seq_replay_ptr[i + 1] - P.seq_replay_ptr[i]) + P.seq_own_len[i];
        P.seq_chunk_ptr[i + 1] = P.seq_chunk_ptr[i] + (int32_t)((virt + B - 1) / B);
    }
    P.n_chunks = P.seq_chunk_ptr[n_seq];

    // replay-gradient CSR: for every replayed physical row the replay entries that read it
    {
        const int32_t R = P.n_replay;
        P.rg_row.clear();
        P.rg_ptr.assign(1, 0);
        P.rg_entry.resize(R);
        if ((int64_t)R * 16 > C) {
            // many replay entries: counting sort by the row they read (stable: one row's entries stay in entry order)
            std::vector<int32_t> first(C + 1, 0);
            for (int32_t e = 0; e < R; e++) first[P.replay_row[e] + 1]++;
            for (int32_t r = 0; r < C; r++) {
                if (first[r + 1]) {
                    if (!P.rg_row.empty()) P.rg_ptr.push_back(first[r]);
                    P.rg_row.push_back(r);
                }
                first[r + 1] += first[r];
            }
            for (int32_t e = 0; e < R; e++) P.rg_entry[first[P.replay_row[e]]++] = e;
        } else {
            for (int32_t e = 0; e < R; e++) P.rg_entry[e] = e;
            std::stable_sort(P.rg_entry.begin(), P.rg_entry.end(),
                             [&](int32_t a, int32_t b) { return P.replay_row[a] < P.replay_row[b]; });
            for (int32_t e = 0; e < R; e++) {
                int32_t r = P.replay_row[P.rg_entry[e]];
                if (P.rg_row.empty() || P.rg_row.back() != r) {
                    if (!P.rg_row.empty()) P.rg_ptr.push_back(e);
                    P.rg_row.push_back(r);
                }
            }
        }
        if (R > 0) P.rg_ptr.push_back(R);
        P.n_rg_rows = (int32_t)P.rg_row.size();
    }
    // work order: inside every round the sequences by decreasing chunk count (longest chains start first)
    P.seq_order.resize(n_seq);
    for (int32_t i = 0; i < n_seq; i++) P.seq_order[i] = i;
    for (int32_t r = 0; r < n_rounds; r++)
        std::stable_sort(P.seq_order.begin() + P.round_seq_ptr[r], P.seq_order.begin() + P.round_seq_ptr[r + 1],
                         [&](int32_t a, int32_t b) {
                             return P.seq_chunk_ptr[a + 1] - P.seq_chunk_ptr[a] > P.seq_chunk_ptr[b + 1] - P.seq_chunk_ptr[b];
                         });
    P.pack();
    return HARTS_OK;
}

// ---- flat blob: every device table, each start 16-byte aligned -------------------------------
void Plan::pack() {
    const std::vector<int32_t>* arrays[N_DEVICE_TABLES] = {
        &seq_own_begin, &seq_init_slot, &seq_replay_ptr, &replay_row, &seq_req_ptr, &slot_chunk,
        &seq_chunk_ptr, &slot_cons_ptr, &slot_cons_seq, &rg_row, &rg_ptr, &rg_entry, &seq_order};
    size_t words = 0;
    for (int i = 0; i < N_DEVICE_TABLES; i++) {
        table_offset[i] = words;
        words += (arrays[i]->size() + 3) / 4 * 4;
        if (arrays[i]->empty()) words += 4;   // keep every table pointer valid and distinct
    }
    blob.assign(words, 0);
    for (int i = 0; i < N_DEVICE_TABLES; i++)
        if (!arrays[i]->empty())
            std::memcpy(blob.data() + table_offset[i], arrays[i]->data(), arrays[i]->size() * sizeof(int32_t));
}

void Plan::tables(const void* dev_blob, harts_la_tables_t* t) const {
    const int32_t* base = static_cast<const int32_t*>(dev_blob);
    t->chunk = chunk;
    t->n_rows = n_rows;
    t->n_replay = n_replay;
    t->n_seq = n_seq;
    t->n_slots = n_slots;
    t->n_chunks = n_chunks;
    t->n_rg_rows = n_rg_rows;
    t->seq_own_begin = base + table_offset[0];
    t->seq_init_slot = base + table_offset[1];
    t->seq_replay_ptr = base + table_offset[2];
    t->replay_row = base + table_offset[3];
    t->seq_req_ptr = base + table_offset[4];
    t->slot_chunk = base + table_offset[5];
    t->seq_chunk_ptr = base + table_offset[6];
    t->slot_cons_ptr = base + table_offset[7];
    t->slot_cons_seq = base + table_offset[8];
    t->rg_row = base + table_offset[9];
    t->rg_ptr = base + table_offset[10];
    t->rg_entry = base + table_offset[11];
    t->seq_order = base + table_offset[12];
}

}  // namespace harts

// ---- C ABI: planning ---------------------------------------------------------------------------
struct harts_la_plan {
    harts::Plan p;
};

extern "C" {

int32_t harts_la_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                      const int32_t* node_fork_off, const int32_t* node_len, int32_t chunk,
                      harts_la_plan_t** out) {
    if (!out) return HARTS_EINVAL;
    *out = nullptr;
    try {
        harts_la_plan_t* h = new (std::nothrow) harts_la_plan_t();
        if (!h) return HARTS_ENOMEM;
        int32_t rc = harts::build_plan(n_trees, tree_node_ptr, node_parent, node_fork_off, node_len, chunk, h->p);
        if (rc != HARTS_OK) {
            delete h;
            return rc;
        }
        *out = h;
        return HARTS_OK;
    } catch (const std::bad_alloc&) {
        return HARTS_ENOMEM;
    } catch (...) {
        return HARTS_EINTERNAL;
    }
}

void harts_la_plan_free(harts_la_plan_t* plan) { delete plan; }

int32_t harts_la_plan_view(const harts_la_plan_t* plan, harts_la_plan_view_t* v) {
    if (!plan || !v) return HARTS_EINVAL;
    const harts::Plan& p = plan->p;
    v->chunk = p.chunk;
    v->n_rounds = p.n_rounds;
    v->n_rows = p.n_rows;
    v->n_replay = p.n_replay;
    v->n_seq = p.n_seq;
    v->n_slots = p.n_slots;
    v->n_chunks = p.n_chunks;
    v->n_rg_rows = p.n_rg_rows;
    v->row_of_token = p.row_of_token.data();
    v->round_seq_ptr = p.round_seq_ptr.data();
    v->seq_tree = p.seq_tree.data();
    v->seq_own_begin = p.seq_own_begin.data();
    v->seq_own_len = p.seq_own_len.data();
    v->seq_start_pos = p.seq_start_pos.data();
    v->seq_init_slot = p.seq_init_slot.data();
    v->seq_replay_ptr = p.seq_replay_ptr.data();
    v->replay_row = p.replay_row.data();
    v->seq_req_ptr = p.seq_req_ptr.data();
    v->slot_chunk = p.slot_chunk.data();
    v->seq_chunk_ptr = p.seq_chunk_ptr.data();
    v->slot_cons_ptr = p.slot_cons_ptr.data();
    v->slot_cons_seq = p.slot_cons_seq.data();
    v->rg_row = p.rg_row.data();
    v->rg_ptr = p.rg_ptr.data();
    v->rg_entry = p.rg_entry.data();
    v->seq_order = p.seq_order.data();
    return HARTS_OK;
}

int32_t harts_la_plan_device_bytes(const harts_la_plan_t* plan, size_t* bytes) {
    if (!plan || !bytes) return HARTS_EINVAL;
    *bytes = plan->p.blob.size() * sizeof(int32_t);
    return HARTS_OK;
}

int32_t harts_la_plan_tables(const harts_la_plan_t* plan, const void* dev_blob, harts_la_tables_t* out) {
    if (!plan || !dev_blob || !out || (reinterpret_cast<uintptr_t>(dev_blob) & 15)) return HARTS_EINVAL;
    plan->p.tables(dev_blob, out);
    return HARTS_OK;
}

const harts::Plan* harts_la_plan_internal(const harts_la_plan_t* plan) { return plan ? &plan->p : nullptr; }

}  // extern "C"
