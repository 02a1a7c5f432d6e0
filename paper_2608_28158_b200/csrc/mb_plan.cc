// Prefix-aware microbatch planning and schedule construction (Section 3.2, Eqs. 4-10), host side.
//
// Readings where the section leaves room (also listed in the design notes):
//  * "lexicographic order" is a depth-first order of the forest (see harts_mb.h); the adjacent-LCP identities
//    (Eqs. 5, 6 and the range-minimum rule) hold in any depth-first order of the trie;
//  * sampled K for N > 512: all values if there are at most 32, else both ends, the 16 smallest, and 14 spread evenly;
//  * greedy: "eliminate small microbatches" = repeatedly try to re-place all members of the lightest microbatch into
//    others (max-shared destination, all or nothing); "align K to D" = split off the single trajectory whose removal
//    into a microbatch of its own costs least, until K mod D = 0;
//  * the slot schedule sorts microbatches by work, heaviest first.
#include <algorithm>
#include <cstdint>
#include <limits>
#include <new>
#include <set>
#include <vector>

#include "../../include/harts_mb.h"

namespace {

using i64 = int64_t;
constexpr int N_EXACT = 512, Q_MAX = 32, B_REF = 3, H_WIN = 8;

struct Traj {
    int leaf, len;
    std::vector<std::pair<int, int>> path;        // (global node, tokens used of it), root first
};

// Lengths, adjacent LCPs and O(1) interval work / pairwise LCP of the trajectories in lexicographic order.
struct Costs {
    int N = 0;
    std::vector<int> len, L;                      // L[i] = LCP(x_{i-1}, x_i), L[0] = 0
    std::vector<i64> plen, pL;                    // prefix sums
    std::vector<std::vector<int>> sparse;         // range-minimum table over L
    void build() {
        N = static_cast<int>(len.size());
        plen.assign(N + 1, 0);
        pL.assign(N + 1, 0);
        for (int i = 0; i < N; ++i) {
            plen[i + 1] = plen[i] + len[i];
            pL[i + 1] = pL[i] + L[i];
        }
        sparse.assign(1, L);
        for (int k = 1; (1 << k) <= N; ++k) {
            const auto& prev = sparse.back();
            std::vector<int> cur(N - (1 << k) + 1);
            for (int i = 0; i + (1 << k) <= N; ++i) cur[i] = std::min(prev[i], prev[i + (1 << (k - 1))]);
            sparse.push_back(std::move(cur));
        }
    }
    i64 W(int a, int b) const { return plen[b + 1] - plen[a] - (pL[b + 1] - pL[a + 1]); }      // interval a..b
    int lcp(int a, int b) const {                 // a < b: minimum of L[a+1..b]
        int lo = a + 1, n = b - a, k = 0;
        while ((2 << k) <= n) ++k;
        return std::min(sparse[k][lo], sparse[k][b + 1 - (1 << k)]);
    }
};

// A grouping: members of every microbatch as sorted lexicographic indices.
struct Grouping {
    std::vector<std::vector<int>> mb;
    int source = HARTS_MB_NATURAL;
    bool refined = false;
};
i64 work_of(const Costs& c, const std::vector<int>& m) {
    i64 w = 0;
    for (size_t i = 0; i < m.size(); ++i) w += c.len[m[i]] - (i ? c.lcp(m[i - 1], m[i]) : 0);
    return w;
}
i64 total_work(const Costs& c, const Grouping& g) {
    i64 t = 0;
    for (const auto& m : g.mb) t += work_of(c, m);
    return t;
}
Grouping from_cuts(const std::vector<int>& starts, int N, int source) {      // starts: first index of every interval
    Grouping g;
    g.source = source;
    for (size_t k = 0; k < starts.size(); ++k) {
        const int a = starts[k], b = k + 1 < starts.size() ? starts[k + 1] : N;
        std::vector<int> m(b - a);
        for (int i = a; i < b; ++i) m[i - a] = i;
        g.mb.push_back(std::move(m));
    }
    return g;
}
bool contiguous(const Grouping& g, std::vector<int>* starts) {
    std::vector<std::pair<int, int>> iv;
    for (const auto& m : g.mb) {
        if (m.back() - m.front() + 1 != static_cast<int>(m.size())) return false;
        iv.push_back({m.front(), m.back()});
    }
    std::sort(iv.begin(), iv.end());
    if (starts) {
        starts->clear();
        for (auto& p : iv) starts->push_back(p.first);
    }
    return true;
}

// ---- natural partition: cut intervals heavier than T at the lowest adjacent-LCP valley ------------------------------
void natural_split(const Costs& c, i64 T, int a, int b, std::vector<int>& starts) {
    if (c.W(a, b) <= T) {
        starts.push_back(a);
        return;
    }
    int best = -1;
    i64 best_max = 0, best_diff = 0;
    int best_l = std::numeric_limits<int>::max();
    for (int t = a + 1; t <= b; ++t) {
        const i64 wl = c.W(a, t - 1), wr = c.W(t, b);
        const i64 mx = std::max(wl, wr), df = wl > wr ? wl - wr : wr - wl;
        if (c.L[t] < best_l || (c.L[t] == best_l && (mx < best_max || (mx == best_max && df < best_diff)))) {
            best = t;
            best_l = c.L[t];
            best_max = mx;
            best_diff = df;
        }
    }
    natural_split(c, T, a, best - 1, starts);
    natural_split(c, T, best, b, starts);
}

// ---- exact search over contiguous partitions (Eq. 9) for every k <= K_max at once ------------------------------------
// F[k][e]: least total work of the first e trajectories in k microbatches; ties by the lighter heaviest microbatch.
struct ExactDP {
    int N, Kmax;
    std::vector<std::vector<i64>> F, M;
    std::vector<std::vector<int>> from;
    static constexpr i64 INF = std::numeric_limits<i64>::max() / 4;
    ExactDP(const Costs& c, i64 T, int Kmax_) : N(c.N), Kmax(Kmax_) {
        F.assign(Kmax + 1, std::vector<i64>(N + 1, INF));
        M.assign(Kmax + 1, std::vector<i64>(N + 1, INF));
        from.assign(Kmax + 1, std::vector<int>(N + 1, -1));
        F[0][0] = 0;
        M[0][0] = 0;
        // first feasible start of an interval that ends at e-1 (W(s, e-1) shrinks as s moves right)
        std::vector<int> first(N + 1, 0);
        for (int e = 1, s = 0; e <= N; ++e) {
            while (c.W(s, e - 1) > T) ++s;
            first[e] = s;
        }
        for (int k = 1; k <= Kmax; ++k)
            for (int e = k; e <= N; ++e)
                for (int s = std::max(first[e], k - 1); s < e; ++s) {
                    if (F[k - 1][s] >= INF) continue;
                    const i64 w = c.W(s, e - 1), f = F[k - 1][s] + w, mx = std::max(M[k - 1][s], w);
                    if (f < F[k][e] || (f == F[k][e] && mx < M[k][e])) {
                        F[k][e] = f;
                        M[k][e] = mx;
                        from[k][e] = s;
                    }
                }
    }
    bool feasible(int k) const { return k <= Kmax && F[k][N] < INF; }
    Grouping plan(int k) const {
        std::vector<int> starts(k);
        for (int e = N, j = k; j >= 1; --j) {
            starts[j - 1] = from[j][e];
            e = from[j][e];
        }
        return from_cuts(starts, N, HARTS_MB_EXACT);
    }
};

// ---- merge / split evolution of the natural partition towards a target K (contiguous throughout) --------------------
bool evolve(const Costs& c, i64 T, std::vector<int> starts, int target, Grouping* out) {
    const int N = c.N;
    auto end_of = [&](size_t k) { return (k + 1 < starts.size() ? starts[k + 1] : N) - 1; };
    while (static_cast<int>(starts.size()) > target) {           // merge the feasible neighbours that save most
        int best = -1;
        i64 best_save = -1;
        for (size_t k = 0; k + 1 < starts.size(); ++k) {
            if (c.W(starts[k], end_of(k + 1)) > T) continue;
            const i64 save = c.L[starts[k + 1]];                 // Eq. 6
            if (save > best_save) {
                best_save = save;
                best = static_cast<int>(k);
            }
        }
        if (best < 0) return false;
        starts.erase(starts.begin() + best + 1);
    }
    while (static_cast<int>(starts.size()) < target) {           // split where it costs least
        int best_t = -1, best_l = std::numeric_limits<int>::max();
        for (size_t k = 0; k < starts.size(); ++k)
            for (int t = starts[k] + 1; t <= end_of(k); ++t)
                if (c.L[t] < best_l) {
                    best_l = c.L[t];
                    best_t = t;
                }
        if (best_t < 0) return false;
        starts.insert(std::upper_bound(starts.begin(), starts.end(), best_t), best_t);
    }
    *out = from_cuts(starts, N, HARTS_MB_EVOLVED);
    return true;
}

// ---- trie-aware greedy placement (Eq. 10) ------------------------------------------------------------------------------
struct Bin {
    std::set<int> members;
    i64 work = 0;
};
// exact work increase of inserting x (Eq. 10) and the amount it shares
i64 insert_delta(const Costs& c, const Bin& b, int x) {
    auto it = b.members.lower_bound(x);
    const bool has_q = it != b.members.end(), has_p = it != b.members.begin();
    const int q = has_q ? *it : -1, p = has_p ? *std::prev(it) : -1;
    i64 d = c.len[x];
    if (has_p) d -= c.lcp(p, x);
    if (has_q) d -= c.lcp(x, q);
    if (has_p && has_q) d += c.lcp(p, q);
    return d;
}
// the same with one member left out of the microbatch (skip < 0: nobody); x itself is never counted as a neighbour
i64 insert_delta_without(const Costs& c, const Bin& b, int x, int skip) {
    auto hi = b.members.upper_bound(x);
    while (hi != b.members.end() && *hi == skip) ++hi;
    auto lo = b.members.lower_bound(x);
    int p = -1;
    while (lo != b.members.begin()) {
        --lo;
        if (*lo != skip) {
            p = *lo;
            break;
        }
    }
    const int q = hi != b.members.end() ? *hi : -1;
    i64 d = c.len[x];
    if (p >= 0) d -= c.lcp(p, x);
    if (q >= 0) d -= c.lcp(x, q);
    if (p >= 0 && q >= 0) d += c.lcp(p, q);
    return d;
}
void bin_insert(const Costs& c, Bin& b, int x) {
    b.work += insert_delta(c, b, x);
    b.members.insert(x);
}
void bin_erase(const Costs& c, Bin& b, int x) {
    b.members.erase(x);
    b.work -= insert_delta(c, b, x);
}

// One placement step as the greedy saw it: trajectory x went to microbatch dest (a new one when created == 1) with
// work increase delta (Eq. 10).
struct GreedyStep {
    int x, dest, created;
    i64 delta;
};
// The placement pass of the greedy: every trajectory, in the given order, goes to the capacity-feasible microbatch
// with the largest work after insertion (best-fit) or the largest shared amount |x| - delta (max-shared); ties go to
// the earliest microbatch; a new microbatch is opened when none fits.
void greedy_place(const Costs& c, i64 T, const std::vector<int>& order, bool best_fit, std::vector<Bin>& bins,
                  std::vector<GreedyStep>* trace) {
    for (int x : order) {
        int best = -1;
        i64 best_key = -1, best_delta = 0;
        for (size_t k = 0; k < bins.size(); ++k) {
            const i64 d = insert_delta(c, bins[k], x);
            if (bins[k].work + d > T) continue;
            const i64 key = best_fit ? bins[k].work + d : c.len[x] - d;     // work after insertion | shared amount
            if (key > best_key) {
                best_key = key;
                best_delta = d;
                best = static_cast<int>(k);
            }
        }
        const bool created = best < 0;
        if (created) {
            bins.emplace_back();
            best = static_cast<int>(bins.size()) - 1;
            best_delta = c.len[x];
        }
        bin_insert(c, bins[best], x);
        if (trace) trace->push_back({x, best, created ? 1 : 0, best_delta});
    }
}
// The four processing orders: ascending and descending lexicographic, descending length, descending unique-suffix
// score u(x) = |x| - max(LCP with the global predecessor, LCP with the global successor); stable.
std::vector<std::vector<int>> greedy_orders(const Costs& c) {
    const int N = static_cast<int>(c.len.size());
    std::vector<std::vector<int>> orders(4, std::vector<int>(N));
    for (int i = 0; i < N; ++i) orders[0][i] = i, orders[1][i] = N - 1 - i, orders[2][i] = i, orders[3][i] = i;
    std::stable_sort(orders[2].begin(), orders[2].end(), [&](int a, int b) { return c.len[a] > c.len[b]; });
    std::vector<int> uniq(N);
    for (int i = 0; i < N; ++i) uniq[i] = c.len[i] - std::max(c.L[i], i + 1 < N ? c.L[i + 1] : 0);
    std::stable_sort(orders[3].begin(), orders[3].end(), [&](int a, int b) { return uniq[a] > uniq[b]; });
    return orders;
}

bool greedy_plan(const Costs& c, i64 T, int D, const std::vector<int>& order, bool best_fit, Grouping* out) {
    std::vector<Bin> bins;
    greedy_place(c, T, order, best_fit, bins, nullptr);
    // eliminate small microbatches: re-place all members of the lightest one (max-shared destination), all or nothing
    while (bins.size() > 1) {
        size_t lightest = 0;
        for (size_t k = 1; k < bins.size(); ++k)
            if (bins[k].work < bins[lightest].work) lightest = k;
        std::vector<Bin> trial = bins;
        trial.erase(trial.begin() + lightest);
        bool ok = true;
        for (int x : bins[lightest].members) {
            int best = -1;
            i64 best_shared = -1;
            for (size_t k = 0; k < trial.size(); ++k) {
                const i64 d = insert_delta(c, trial[k], x);
                if (trial[k].work + d > T) continue;
                if (c.len[x] - d > best_shared) {
                    best_shared = c.len[x] - d;
                    best = static_cast<int>(k);
                }
            }
            if (best < 0) {
                ok = false;
                break;
            }
            bin_insert(c, trial[best], x);
        }
        if (!ok) break;
        bins.swap(trial);
    }
    // align K to D: split off the single trajectory whose own microbatch costs least extra
    while (bins.size() % D != 0) {
        int best_bin = -1, best_x = -1;
        i64 best_inc = std::numeric_limits<i64>::max();
        for (size_t k = 0; k < bins.size(); ++k) {
            if (bins[k].members.size() < 2) continue;
            for (int x : bins[k].members) {
                const i64 inc = c.len[x] - insert_delta_without(c, bins[k], x, -1);      // own microbatch minus what it frees
                if (inc < best_inc) {
                    best_inc = inc;
                    best_bin = static_cast<int>(k);
                    best_x = x;
                }
            }
        }
        if (best_bin < 0) return false;
        bin_erase(c, bins[best_bin], best_x);
        bins.emplace_back();
        bin_insert(c, bins.back(), best_x);
    }
    out->mb.clear();
    out->source = HARTS_MB_GREEDY;
    for (auto& b : bins) out->mb.emplace_back(b.members.begin(), b.members.end());
    return true;
}

// ---- local refinement ---------------------------------------------------------------------------------------------------
// Boundary refinement of a contiguous plan: every cut may move up to H_WIN positions; two sweeps at most.
bool refine_boundaries(const Costs& c, i64 T, std::vector<int>& starts) {
    const int N = c.N;
    bool any = false;
    for (int sweep = 0; sweep < 2; ++sweep) {
        bool changed = false;
        for (size_t k = 1; k < starts.size(); ++k) {
            const int a = starts[k - 1], b = (k + 1 < starts.size() ? starts[k + 1] : N) - 1, cur = starts[k];
            i64 best_sum = c.W(a, cur - 1) + c.W(cur, b), best_max = std::max(c.W(a, cur - 1), c.W(cur, b));
            int best = cur;
            for (int t = std::max(a + 1, cur - H_WIN); t <= std::min(b, cur + H_WIN); ++t) {
                const i64 wl = c.W(a, t - 1), wr = c.W(t, b);
                if (wl > T || wr > T) continue;
                if (wl + wr < best_sum || (wl + wr == best_sum && std::max(wl, wr) < best_max)) {
                    best_sum = wl + wr;
                    best_max = std::max(wl, wr);
                    best = t;
                }
            }
            if (best != cur) {
                starts[k] = best;
                changed = any = true;
            }
        }
        if (!changed) break;
    }
    return any;
}

// Sparse repair: at most four single moves or swaps between microbatches that are close in lexicographic order.
bool sparse_repair(const Costs& c, i64 T, Grouping& g) {
    const int N = c.N;
    std::vector<Bin> bins(g.mb.size());
    std::vector<int> of(N);
    for (size_t k = 0; k < g.mb.size(); ++k)
        for (int x : g.mb[k]) {
            bin_insert(c, bins[k], x);
            of[x] = static_cast<int>(k);
        }
    bool any = false;
    for (int iter = 0; iter < 4; ++iter) {
        i64 best_gain = 0;
        int mv_x = -1, mv_to = -1, sw_x = -1, sw_y = -1;
        for (int x = 0; x < N; ++x) {                       // moves out of non-singleton microbatches
            const int A = of[x];
            if (bins[A].members.size() < 2) continue;
            for (int y = std::max(0, x - H_WIN); y <= std::min(N - 1, x + H_WIN); ++y) {
                const int B = of[y];
                if (B == A) continue;
                const i64 d = insert_delta(c, bins[B], x);
                if (bins[B].work + d > T) continue;
                const i64 gain = insert_delta_without(c, bins[A], x, -1) - d;      // freed in A minus added in B
                if (gain > best_gain) {
                    best_gain = gain;
                    mv_x = x;
                    mv_to = B;
                }
            }
        }
        if (mv_x < 0) {                                      // no improving move: try swaps
            for (int x = 0; x < N; ++x)
                for (int y = x + 1; y <= std::min(N - 1, x + H_WIN); ++y) {
                    const int A = of[x], B = of[y];
                    if (A == B) continue;
                    const i64 a_new = bins[A].work - insert_delta_without(c, bins[A], x, -1) +
                                      insert_delta_without(c, bins[A], y, x);
                    const i64 b_new = bins[B].work - insert_delta_without(c, bins[B], y, -1) +
                                      insert_delta_without(c, bins[B], x, y);
                    if (a_new > T || b_new > T) continue;
                    const i64 gain = (bins[A].work + bins[B].work) - (a_new + b_new);
                    if (gain > best_gain) {
                        best_gain = gain;
                        sw_x = x;
                        sw_y = y;
                    }
                }
        }
        if (mv_x >= 0) {
            bin_erase(c, bins[of[mv_x]], mv_x);
            bin_insert(c, bins[mv_to], mv_x);
            of[mv_x] = mv_to;
        } else if (sw_x >= 0) {
            const int A = of[sw_x], B = of[sw_y];
            bin_erase(c, bins[A], sw_x);
            bin_erase(c, bins[B], sw_y);
            bin_insert(c, bins[A], sw_y);
            bin_insert(c, bins[B], sw_x);
            of[sw_x] = B;
            of[sw_y] = A;
        } else {
            break;
        }
        any = true;
    }
    if (any)
        for (size_t k = 0; k < g.mb.size(); ++k) g.mb[k].assign(bins[k].members.begin(), bins[k].members.end());
    return any;
}

// ---- replica / slot assignment and Eq. 4 ----------------------------------------------------------------------------------
struct Schedule {
    std::vector<i64> work;
    std::vector<int> replica, slot;
    i64 J[3] = {0, 0, 0};
};
Schedule schedule(const Costs& c, const Grouping& g, int D) {
    Schedule s;
    const int K = static_cast<int>(g.mb.size());
    s.work.resize(K);
    for (int k = 0; k < K; ++k) s.work[k] = work_of(c, g.mb[k]);
    std::vector<int> order(K);
    for (int k = 0; k < K; ++k) order[k] = k;
    std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return s.work[a] > s.work[b]; });
    std::vector<i64> load(D, 0);
    s.replica.assign(K, 0);
    s.slot.assign(K, 0);
    for (int j = 0; j < K / D; ++j) {
        std::vector<int> free(D);
        for (int d = 0; d < D; ++d) free[d] = d;
        std::stable_sort(free.begin(), free.end(), [&](int a, int b) { return load[a] < load[b]; });
        i64 heaviest = 0;
        for (int u = 0; u < D; ++u) {
            const int m = order[j * D + u];
            s.replica[m] = free[u];
            s.slot[m] = j;
            heaviest = std::max(heaviest, s.work[m]);
        }
        for (int u = 0; u < D; ++u) load[free[u]] += s.work[order[j * D + u]];
        s.J[1] += heaviest;
    }
    for (i64 w : s.work) s.J[0] += w;
    s.J[2] = *std::max_element(load.begin(), load.end());
    return s;
}
bool better(const i64 (&a)[3], const i64 (&b)[3]) {
    for (int i = 0; i < 3; ++i)
        if (a[i] != b[i]) return a[i] < b[i];
    return false;
}

}  // namespace

struct harts_mb_plan {
    std::vector<int32_t> tree_node_ptr, node_parent, node_fork_off, node_len;
    std::vector<Traj> traj;
    std::vector<int32_t> traj_leaf, traj_len, traj_lcp, traj_mb, mb_replica, mb_slot;
    std::vector<int64_t> mb_work;
    harts_mb_view_t view{};
};

namespace {

bool forest_ok(int32_t n_trees, const int32_t* ptr, const int32_t* par, const int32_t* off, const int32_t* len) {
    if (n_trees < 0 || !ptr || !par || !off || !len || ptr[0] != 0) return false;
    for (int32_t t = 0; t < n_trees; ++t) {
        const int32_t lo = ptr[t], hi = ptr[t + 1];
        if (hi <= lo) return false;
        for (int32_t i = lo; i < hi; ++i) {
            if (len[i] < 1) return false;
            if (i == lo ? (par[i] != -1 || off[i] != 0)
                        : (par[i] < 0 || par[i] >= i - lo || off[i] < 1 || off[i] > len[lo + par[i]]))
                return false;
        }
    }
    return true;
}

// Trajectories in depth-first order (explicit stack: trees may be deep chains).
void enumerate(const harts_mb_plan_t& p, int32_t n_trees, std::vector<Traj>& out) {
    const auto& ptr = p.tree_node_ptr;
    const auto& par = p.node_parent;
    const auto& off = p.node_fork_off;
    const auto& len = p.node_len;
    const int n_nodes = ptr[n_trees];
    std::vector<std::vector<int>> kids(n_nodes);
    std::vector<char> continued(n_nodes, 0);
    for (int t = 0; t < n_trees; ++t)
        for (int i = ptr[t] + 1; i < ptr[t + 1]; ++i) {
            const int q = ptr[t] + par[i];
            kids[q].push_back(i);
            if (off[i] == len[q]) continued[q] = 1;
        }
    for (auto& k : kids) std::stable_sort(k.begin(), k.end(), [&](int a, int b) { return off[a] < off[b]; });
    std::vector<int> root_of(n_nodes);
    for (int t = 0; t < n_trees; ++t)
        for (int i = ptr[t]; i < ptr[t + 1]; ++i) root_of[i] = ptr[t];
    for (int t = 0; t < n_trees; ++t) {
        std::vector<std::pair<int, size_t>> stack;
        stack.push_back({ptr[t], size_t(0)});
        while (!stack.empty()) {
            auto& top = stack.back();
            const int v = top.first;
            if (top.second < kids[v].size()) {
                const int child = kids[v][top.second++];
                stack.push_back({child, size_t(0)});
                continue;
            }
            if (!continued[v]) {
                Traj tr;
                tr.leaf = v;
                int node = v, upto = len[v];
                while (true) {
                    tr.path.push_back({node, upto});
                    if (node == root_of[node]) break;
                    upto = off[node];
                    node = root_of[node] + par[node];
                }
                std::reverse(tr.path.begin(), tr.path.end());
                tr.len = 0;
                for (auto& e : tr.path) tr.len += e.second;
                out.push_back(std::move(tr));
            }
            stack.pop_back();
        }
    }
}
int path_lcp(const Traj& a, const Traj& b) {
    int n = 0;
    for (size_t i = 0; i < a.path.size() && i < b.path.size(); ++i) {
        if (a.path[i].first != b.path[i].first) break;
        n += std::min(a.path[i].second, b.path[i].second);
        if (a.path[i].second != b.path[i].second) break;
    }
    return n;
}

int32_t build(harts_mb_plan_t& p, int32_t n_trees, int32_t D, i64 T) {
    enumerate(p, n_trees, p.traj);
    const int N = static_cast<int>(p.traj.size());
    if (N < D) return HARTS_EINVAL;
    Costs c;
    c.len.resize(N);
    c.L.assign(N, 0);
    for (int i = 0; i < N; ++i) {
        c.len[i] = p.traj[i].len;
        if (c.len[i] > T) return HARTS_EINVAL;
        if (i) c.L[i] = path_lcp(p.traj[i - 1], p.traj[i]);
    }
    c.build();

    std::vector<Grouping> cands;
    std::vector<int> nat;
    natural_split(c, T, 0, N - 1, nat);
    const int K0 = static_cast<int>(nat.size());
    Grouping natural = from_cuts(nat, N, HARTS_MB_NATURAL);
    if (K0 % D == 0) cands.push_back(natural);
    const i64 G = c.W(0, N - 1);
    const int Kmin = D * static_cast<int>(std::max<i64>(1, (G + T * D - 1) / (T * D)));
    const int Kmax = std::max(Kmin, std::min(D * ((K0 + D - 1) / D), D * (N / D)));
    std::vector<int> ks;
    for (int K = Kmin; K <= Kmax; K += D) ks.push_back(K);
    const size_t n_base_begin = cands.size();
    if (N <= N_EXACT) {
        ExactDP dp(c, T, std::min(Kmax, N));
        for (int K : ks)
            if (K <= N && dp.feasible(K)) cands.push_back(dp.plan(K));
    } else {
        std::vector<int> pick;
        if (static_cast<int>(ks.size()) <= Q_MAX) {
            pick = ks;
        } else {
            std::set<int> chosen{ks.front(), ks.back()};
            for (int i = 0; i < 16; ++i) chosen.insert(ks[i]);
            for (int i = 0; i < 14; ++i) chosen.insert(ks[16 + (ks.size() - 17) * (i + 1) / 15]);
            pick.assign(chosen.begin(), chosen.end());
        }
        for (int K : pick) {
            Grouping g;
            if (K <= N && evolve(c, T, nat, K, &g)) cands.push_back(std::move(g));
        }
    }
    const size_t n_base_end = cands.size();

    // greedy: four processing orders x two placement policies, one candidate (fewest microbatches, then least work)
    const std::vector<std::vector<int>> orders = greedy_orders(c);
    bool have_greedy = false;
    Grouping greedy;
    i64 greedy_work = 0;
    for (const auto& order : orders)
        for (int policy = 0; policy < 2; ++policy) {
            Grouping g;
            if (!greedy_plan(c, T, D, order, policy == 0, &g)) continue;
            const i64 w = total_work(c, g);
            if (!have_greedy || g.mb.size() < greedy.mb.size() || (g.mb.size() == greedy.mb.size() && w < greedy_work)) {
                greedy = std::move(g);
                greedy_work = w;
                have_greedy = true;
            }
        }
    if (have_greedy) cands.push_back(greedy);

    // local refinement of the anchors; refined plans join the comparison, the plans they came from stay in it
    std::vector<size_t> anchors;
    if (N <= N_EXACT) {
        if (have_greedy) anchors.push_back(cands.size() - 1);
    } else {
        const int gk = have_greedy ? static_cast<int>(greedy.mb.size()) : -1;
        auto add = [&](size_t i) {
            if (std::find(anchors.begin(), anchors.end(), i) == anchors.end() && anchors.size() < B_REF) anchors.push_back(i);
        };
        if (have_greedy) add(cands.size() - 1);
        if (n_base_end > n_base_begin) {
            size_t lowest = n_base_begin, closest = n_base_begin;
            for (size_t i = n_base_begin; i < n_base_end; ++i) {
                if (total_work(c, cands[i]) < total_work(c, cands[lowest])) lowest = i;
                if (std::abs(static_cast<int>(cands[i].mb.size()) - gk) < std::abs(static_cast<int>(cands[closest].mb.size()) - gk))
                    closest = i;
            }
            add(lowest);
            add(closest);
        }
    }
    for (size_t a : anchors) {
        Grouping g = cands[a];
        bool changed = false;
        std::vector<int> starts;
        if (contiguous(g, &starts) && refine_boundaries(c, T, starts)) {
            const int src = g.source;
            g = from_cuts(starts, N, src);
            changed = true;
        }
        changed = sparse_repair(c, T, g) || changed;
        if (changed) {
            g.refined = true;
            cands.push_back(std::move(g));
        }
    }

    // schedule every candidate and keep the best under Eq. 4 (earlier candidate on ties)
    int best = -1;
    Schedule best_s;
    int n_valid = 0;
    for (size_t i = 0; i < cands.size(); ++i) {
        const int K = static_cast<int>(cands[i].mb.size());
        if (K % D != 0 || K == 0) continue;
        Schedule s = schedule(c, cands[i], D);
        if (*std::max_element(s.work.begin(), s.work.end()) > T) continue;
        ++n_valid;
        if (best < 0 || better(s.J, best_s.J)) {
            best = static_cast<int>(i);
            best_s = std::move(s);
        }
    }
    if (best < 0) return HARTS_EINVAL;       // no grouping with K mod D = 0 fits (e.g. too few trajectories)
    const Grouping& g = cands[best];
    const int K = static_cast<int>(g.mb.size());
    p.traj_leaf.resize(N);
    p.traj_len = c.len;
    p.traj_lcp = c.L;
    p.traj_mb.assign(N, -1);
    for (int i = 0; i < N; ++i) p.traj_leaf[i] = p.traj[i].leaf;
    for (int k = 0; k < K; ++k)
        for (int x : g.mb[k]) p.traj_mb[x] = k;
    p.mb_work = best_s.work;
    p.mb_replica = best_s.replica;
    p.mb_slot = best_s.slot;
    harts_mb_view_t& v = p.view;
    v.n_traj = N;
    v.n_mb = K;
    v.D = D;
    v.source = g.source;
    v.refined = g.refined ? 1 : 0;
    v.natural_mb = K0;
    v.n_candidates = n_valid;
    v.T = T;
    for (int i = 0; i < 3; ++i) v.J[i] = best_s.J[i];
    v.total_work_all = G;
    v.natural_work = total_work(c, natural);
    return HARTS_OK;
}

}  // namespace

extern "C" int32_t harts_mb_plan(int32_t n_trees, const int32_t* tree_node_ptr, const int32_t* node_parent,
                                 const int32_t* node_fork_off, const int32_t* node_len, int32_t D, int64_t T,
                                 harts_mb_plan_t** out) {
    if (!out || D < 1 || T < 1 || n_trees < 1) return HARTS_EINVAL;
    if (!forest_ok(n_trees, tree_node_ptr, node_parent, node_fork_off, node_len)) return HARTS_EINVAL;
    harts_mb_plan_t* p = new (std::nothrow) harts_mb_plan_t;
    if (!p) return HARTS_ENOMEM;
    int32_t rc;
    try {
        const int n_nodes = tree_node_ptr[n_trees];
        p->tree_node_ptr.assign(tree_node_ptr, tree_node_ptr + n_trees + 1);
        p->node_parent.assign(node_parent, node_parent + n_nodes);
        p->node_fork_off.assign(node_fork_off, node_fork_off + n_nodes);
        p->node_len.assign(node_len, node_len + n_nodes);
        rc = build(*p, n_trees, D, T);
    } catch (const std::bad_alloc&) {
        rc = HARTS_ENOMEM;
    }
    if (rc != HARTS_OK) {
        delete p;
        return rc;
    }
    harts_mb_view_t& v = p->view;
    v.traj_leaf = p->traj_leaf.data();
    v.traj_len = p->traj_len.data();
    v.traj_lcp = p->traj_lcp.data();
    v.traj_mb = p->traj_mb.data();
    v.mb_work = p->mb_work.data();
    v.mb_replica = p->mb_replica.data();
    v.mb_slot = p->mb_slot.data();
    *out = p;
    return HARTS_OK;
}

extern "C" int32_t harts_mb_greedy_trace(const harts_mb_plan_t* plan, int32_t order, int32_t policy, int32_t cap,
                                         int32_t* step_traj, int32_t* step_mb, int32_t* step_created,
                                         int64_t* step_delta, int32_t* n_steps) {
    if (!plan || order < 0 || order > 3 || policy < 0 || policy > 1 || !n_steps) return HARTS_EINVAL;
    try {
        const int N = static_cast<int>(plan->traj_len.size());
        Costs c;
        c.len.assign(plan->traj_len.begin(), plan->traj_len.end());
        c.L.assign(plan->traj_lcp.begin(), plan->traj_lcp.end());
        c.build();
        std::vector<Bin> bins;
        std::vector<GreedyStep> trace;
        greedy_place(c, plan->view.T, greedy_orders(c)[order], policy == 0, bins, &trace);
        *n_steps = N;
        if (!step_traj && !step_mb && !step_created && !step_delta) return HARTS_OK;
        if (cap < N || !step_traj || !step_mb || !step_created || !step_delta) return HARTS_EINVAL;
        for (int i = 0; i < N; ++i) {
            step_traj[i] = trace[i].x;
            step_mb[i] = trace[i].dest;
            step_created[i] = trace[i].created;
            step_delta[i] = trace[i].delta;
        }
    } catch (const std::bad_alloc&) {
        return HARTS_ENOMEM;
    }
    return HARTS_OK;
}

extern "C" void harts_mb_plan_free(harts_mb_plan_t* plan) { delete plan; }

extern "C" int32_t harts_mb_plan_view(const harts_mb_plan_t* plan, harts_mb_view_t* out) {
    if (!plan || !out) return HARTS_EINVAL;
    *out = plan->view;
    return HARTS_OK;
}

extern "C" int32_t harts_mb_extract(const harts_mb_plan_t* plan, int32_t mb, int32_t cap_trees, int32_t cap_nodes,
                                    int32_t* tree_node_ptr, int32_t* node_parent, int32_t* node_fork_off,
                                    int32_t* node_len, int32_t* node_src, int32_t* n_trees, int32_t* n_nodes) {
    if (!plan || !n_trees || !n_nodes || mb < 0 || mb >= plan->view.n_mb) return HARTS_EINVAL;
    const int total_nodes = static_cast<int>(plan->node_len.size());
    std::vector<int> extent(total_nodes, 0);            // tokens of every node that some trajectory of the microbatch uses
    for (int i = 0; i < plan->view.n_traj; ++i)
        if (plan->traj_mb[i] == mb)
            for (auto& e : plan->traj[i].path) extent[e.first] = std::max(extent[e.first], e.second);
    int trees = 0, nodes = 0;
    const int T_in = static_cast<int>(plan->tree_node_ptr.size()) - 1;
    for (int t = 0; t < T_in; ++t) {
        if (extent[plan->tree_node_ptr[t]] == 0) continue;
        ++trees;
        for (int i = plan->tree_node_ptr[t]; i < plan->tree_node_ptr[t + 1]; ++i) nodes += extent[i] > 0;
    }
    *n_trees = trees;
    *n_nodes = nodes;
    if (!tree_node_ptr && !node_parent && !node_fork_off && !node_len) return HARTS_OK;
    if (!tree_node_ptr || !node_parent || !node_fork_off || !node_len || cap_trees < trees || cap_nodes < nodes)
        return HARTS_EINVAL;
    std::vector<int> local(total_nodes, -1);
    int tt = 0, nn = 0;
    tree_node_ptr[0] = 0;
    for (int t = 0; t < T_in; ++t) {
        const int lo = plan->tree_node_ptr[t];
        if (extent[lo] == 0) continue;
        const int first = nn;
        for (int i = lo; i < plan->tree_node_ptr[t + 1]; ++i) {
            if (extent[i] == 0) continue;
            local[i] = nn - first;
            node_parent[nn] = i == lo ? -1 : local[lo + plan->node_parent[i]];
            node_fork_off[nn] = plan->node_fork_off[i];
            node_len[nn] = extent[i];
            if (node_src) node_src[nn] = i;
            ++nn;
        }
        tree_node_ptr[++tt] = nn;
    }
    return HARTS_OK;
}
