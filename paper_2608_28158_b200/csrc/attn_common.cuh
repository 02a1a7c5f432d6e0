// Shared by the attention kernels: the device view of the host index and the walk over the key tiles of a
// query tile (ancestor rows first, then the piece's own rows up to the diagonal, Eq. 22).
#pragma once
#include <cstdint>

namespace harts {
namespace attn {

constexpr int BQ = 128, BK = 64, D = 128;
constexpr int NO_DIAG = -(1 << 28);

struct Index {
    const int32_t *piece_row0, *piece_len, *anc_ptr, *anc_row0, *anc_len, *desc_ptr, *desc_piece, *q_item, *kv_item;
    int n_q_items, n_kv_items;
};
inline Index make_index(const int32_t* hi, const int32_t* di) {
    Index ix;
    ix.piece_row0 = di + hi[8];
    ix.piece_len = di + hi[9];
    ix.anc_ptr = di + hi[11];
    ix.anc_row0 = di + hi[12];
    ix.anc_len = di + hi[13];
    ix.desc_ptr = di + hi[14];
    ix.desc_piece = di + hi[15];
    ix.q_item = di + hi[16];
    ix.kv_item = di + hi[17];
    ix.n_q_items = hi[4];
    ix.n_kv_items = hi[5];
    return ix;
}

// The t-th key tile of an item: rows [row, row + n_valid), and the diagonal shift (key column j is visible to
// query row i iff j + shift <= i; NO_DIAG for ancestor rows).
struct KvTile {
    int row, n_valid, shift;
};

template <int W>
struct TileWalkT {      // enumerates the key tiles (W rows) of one item in order; run data is read once per run, not per tile
    const Index& ix;
    int run0, run, run_end, off, own_row0, own_end, q0, cur_row0, cur_len;
    bool in_own;
    __device__ TileWalkT(const Index& ix_, int piece, int qt) : ix(ix_) {
        run0 = run = ix.anc_ptr[piece];
        run_end = ix.anc_ptr[piece + 1];
        off = 0;
        own_row0 = ix.piece_row0[piece];
        q0 = qt * BQ;
        own_end = min(ix.piece_len[piece], q0 + BQ);      // own rows up to the end of the query tile
        in_own = run == run_end;
        cur_row0 = cur_len = 0;
        if (!in_own) {
            cur_row0 = ix.anc_row0[run];
            cur_len = ix.anc_len[run];
        }
    }
    __device__ int count() const {          // number of tiles next() will deliver from a fresh walk
        int n = (own_end + W - 1) / W;
        for (int r = run0; r < run_end; r++) n += (ix.anc_len[r] + W - 1) / W;
        return n;
    }
    __device__ bool next(KvTile& t) {
        if (!in_own) {
            t.row = cur_row0 + off;
            t.n_valid = min(W, cur_len - off);
            t.shift = NO_DIAG;
            off += W;
            if (off >= cur_len) {
                off = 0;
                if (++run == run_end) {
                    in_own = true;
                } else {
                    cur_row0 = ix.anc_row0[run];
                    cur_len = ix.anc_len[run];
                }
            }
            return true;
        }
        if (off >= own_end) return false;
        t.row = own_row0 + off;
        t.n_valid = min(W, own_end - off);
        t.shift = off - q0;
        off += W;
        return true;
    }
};
using TileWalk = TileWalkT<BK>;

// The query tiles (64 rows) that see the key tile `kt` (128 rows) of a piece: for every query head of the group,
// the rest of the piece from the key tile's first row on (causal inside), then all rows of every descendant piece.
// Key row i is seen by query column j iff jmin(i) <= j < n_valid, with jmin(i) = max(0, i - lead) for own tiles
// (lead = first query row of the tile minus first key row of the key tile) and 0 for descendants.
struct QTile {
    int row, n_valid, lead, head;       // lead < 0: descendant piece (no diagonal)
};
struct QWalk {
    const Index& ix;
    int piece, k0, own_len, own_row0, G, head0, g, off, d, d_end, cur_len, cur_row0;
    bool in_own;
    __device__ QWalk(const Index& ix_, int piece_, int kt, int hk, int G_) : ix(ix_), piece(piece_), G(G_) {
        k0 = kt * 128;
        own_len = ix.piece_len[piece];
        own_row0 = ix.piece_row0[piece];
        head0 = hk * G;
        d_end = ix.desc_ptr[piece + 1];
        start_head(0);
    }
    __device__ void start_head(int g_) {
        g = g_;
        in_own = true;
        off = k0;
        d = ix.desc_ptr[piece];
    }
    __device__ int count() const {
        int n = (own_len - k0 + 63) / 64;
        for (int e = ix.desc_ptr[piece]; e < d_end; e++) n += (ix.piece_len[ix.desc_piece[e]] + 63) / 64;
        return n * G;
    }
    __device__ bool next(QTile& t) {
        while (true) {
            if (g >= G) return false;
            if (in_own) {
                if (off < own_len) {
                    t.row = own_row0 + off;
                    t.n_valid = min(64, own_len - off);
                    t.lead = off - k0;
                    t.head = head0 + g;
                    off += 64;
                    return true;
                }
                in_own = false;
                off = 0;
                if (d < d_end) {
                    cur_len = ix.piece_len[ix.desc_piece[d]];
                    cur_row0 = ix.piece_row0[ix.desc_piece[d]];
                }
            }
            if (d < d_end) {
                t.row = cur_row0 + off;
                t.n_valid = min(64, cur_len - off);
                t.lead = -1;
                t.head = head0 + g;
                off += 64;
                if (off >= cur_len) {
                    off = 0;
                    if (++d < d_end) {
                        cur_len = ix.piece_len[ix.desc_piece[d]];
                        cur_row0 = ix.piece_row0[ix.desc_piece[d]];
                    }
                }
                return true;
            }
            start_head(g + 1);
        }
    }
};

}  // namespace attn
}  // namespace harts
