// Tensor-core backward of the packed chunkwise call for bf16, d_k = d_v = 128, chunk 64: one fused
// kernel that walks a sequence's chunks in reverse and emits dq, dk, dv, dg and the gradient of the
// sequence's initial state (the hand-off into the sequence that produced it, Section 3.4).
//
// One CTA per (sequence, head).  dS (gradient w.r.t. the state at the END of the current chunk) lives
// in tensor memory for the whole walk, lane i (0..127) = row i of dS, columns = d_v.  Per chunk
// (b_t running sum of g, n last row, w_j = e^{b_n-b_j}, D_tj = e^{b_t-b_j}[j<=t], dO~_t = e^{b_t} dO_t):
//     A  = Q K^T,  dA = dO V^T                               (t on lanes 0..63)
//     P  = A .* D, dP = dA .* D                              bf16 tiles, rows past the end zeroed
//     dq^T = K^T dP^T + S_c dO~^T                            (lanes = d_k, columns = t)
//     dk^T = Q^T dP   + w .* (dS V^T)                        two accumulators, combined in the epilogue
//     dv^T = dO^T P   + w .* (dS^T K^T)                      two accumulators
//     dg_t = sum_{tau>=t} (q.dq - k.dk) + e^{b_n} <S_c, dS> + sum_j k_j . (w_j dS v_j)
//     dS  <- e^{b_n} dS + Q^T dO~                            accumulate in tensor memory
// where dS includes, at an exported boundary, the initial-state gradients of every sequence that
// started there (read from the scratch area, where those sequences' calls left them).
// S_c comes from the chunk-state workspace written by the forward ([d_k][d_v] bf16 per chunk-head).
// Gradients of replayed rows go to the scratch area (fp32) and are folded into their ancestor rows by
// the replay-reduce kernel.  Full chunks (all 64 rows own rows, nearly all of them) take the matrix-fragment epilogue
// (tcgen05.ld 16x256b, ldmatrix / stmatrix transposing, swizzled staging panels, TMA stores).  Every wait is bounded; one that runs out sets the status word and a CTA-wide latch, and the
// CTA leaves its loops at the end of the chunk, drains what it has in flight, releases tensor memory and returns.
#include "kernels.h"
#include "tc_common.cuh"

namespace harts {

int32_t make_row_map(CUtensorMap* map, const void* base, int64_t rows, int32_t H);
int32_t make_state_map(CUtensorMap* map, const void* base, int64_t n);
int32_t make_out_map(CUtensorMap* map, const void* base, int64_t rows, int32_t H);
int sm_count();

namespace {

using namespace tc;



constexpr int BT = 64, D = 128;
constexpr int NC = 512;                       // 16 compute warps: warp w works on tensor-memory lanes 32(w&3)..+31 and
                                              // on column group w>>2 (a quarter of every accumulator)
constexpr int NT = NC + 64;                   // plus one warp whose first lane issues every TMA and MMA, and one
                                              // that prepares row data and finishes dg (off the issuing thread's path)
constexpr int TILE = BT * D * 2;              // 16 KB
constexpr int PANEL = BT * 128;               // 8 KB
constexpr int S_PANEL = D * 128;              // 16 KB
constexpr float LOG2E = 1.4426950408889634f;

constexpr int COL_DS = 0, COL_A = 128, COL_DA = 192, COL_DQ = 256, COL_DK = 320, COL_DV = 384, TMEM_COLS = 512;

struct Smem {
    static constexpr int q = 0, k = TILE, v = 2 * TILE, dO = 3 * TILE, dOs = 4 * TILE, p = 5 * TILE,
                         dp = 5 * TILE + PANEL, s = 5 * TILE + 2 * PANEL, ds = s + 2 * S_PANEL,
                         stage_dq = ds + 2 * S_PANEL, stage_dk = stage_dq + TILE, stage_dv = stage_dk + TILE,
                         misc = stage_dv + TILE;       // stage_*: outputs of a full chunk, [row][feature], for TMA stores
    static constexpr int bytes = misc + 4096;
};
struct RowData {             // per-chunk row quantities, double-buffered (the next chunk's are prepared in the tail)
    float b2[BT];            // running log-decay in log2 units
    float eb[BT];            // e^{b_t} on rows with an output, 0 elsewhere
    float w[BT];             // e^{b_n - b_t}
    int code[BT];            // physical row (>= 0 own), -2 - row (replayed), -1 (past the end)
    float gamma;             // e^{b_n}
    float pad[3];            // keeps the second buffer 16-byte aligned (vector loads of b2)
};
struct SeqInfo {
    int own_begin, n_replay, n_virtual, n_chunks, replay_base, init_slot, req_lo, req_hi, chunk_base;
};
struct Misc {
    RowData rows[2];
    float red[NC / 32][16];  // per-warp partial sums of q.dq - k.dk (warp w covers rows 16(w>>2)..+15)
    float gred[NC / 32];
    uint32_t tmem;
    uint64_t bar_tiles, bar_tiles2, bar_a, bar_o, bar_o2, bar_o3, bar_qk_read, bar_exit;
    int dead;                // latch: a wait of this CTA ran out, the walk is being abandoned
    int item;                // all rounds in one launch: the work item thread 0 drew
    int head;
    SeqInfo seq;
};

__device__ __forceinline__ SeqInfo seq_info(const harts_la_tables_t& tb, int seq) {
    SeqInfo s;
    s.own_begin = tb.seq_own_begin[seq];
    int own_len = tb.seq_own_begin[seq + 1] - s.own_begin;
    s.replay_base = tb.seq_replay_ptr[seq];
    s.n_replay = tb.seq_replay_ptr[seq + 1] - s.replay_base;
    s.n_virtual = s.n_replay + own_len;
    s.n_chunks = (s.n_virtual + BT - 1) / BT;
    s.init_slot = tb.seq_init_slot[seq];
    s.req_lo = tb.seq_req_ptr[seq];
    s.req_hi = tb.seq_req_ptr[seq + 1];
    s.chunk_base = tb.seq_chunk_ptr[seq];
    return s;
}

// Sum over the 32 lanes of a warp for each of 16 per-lane values; lane l returns the total of z[l & 15].
__device__ __forceinline__ float warp_transpose_reduce16(float (&z)[16], int lane) {
#pragma unroll
    for (int s = 8; s >= 1; s >>= 1) {
        const bool upper = (lane & s) != 0;
#pragma unroll
        for (int i = 0; i < s; i++) {
            float send = upper ? z[i] : z[i + s];
            float keep = upper ? z[i + s] : z[i];
            z[i] = keep + __shfl_xor_sync(0xffffffffu, send, s);
        }
    }
    return z[0] + __shfl_xor_sync(0xffffffffu, z[0], 16);
}

// ---- partial chunks (a ragged tail, or chunk 0 of a sequence that replays ancestor rows) ------------------------------
// Epilogue for this thread's feature index L and its 16 rows, in three parts that follow the three commits of the MMA
// batch (dk, dv, dq: the longest part first, so that little is left after the last MMA).  qk[e] holds q[t][L] (low
// half) and k[t][L] (high half) as bf16 bits, read from the tiles before the batch so that the tiles can be reloaded
// while the epilogue runs.  The outputs are staged in shared memory ([row][feature], plain layout); the compute warps
// copy the valid rows out after the epilogue (own rows to the outputs, replayed rows, staged in fp32, to the scratch).
__device__ __forceinline__ void epilogue_dq(const RowData& m, unsigned char* smem, uint32_t tm_lane, int grp, int L, int H,
                                            int h, const uint32_t (&qk)[16], __nv_bfloat16* dq, float (&z)[16]) {
    const int t0 = grp * 16;
    uint32_t xq[16];
    tmem_ld16(tm_lane + COL_DQ + t0, xq);
    tmem_ld_wait();
#pragma unroll
    for (int e = 0; e < 16; e++) {
        const int t = t0 + e;
        const float dqv = __uint_as_float(xq[e]);
        const float qv = __uint_as_float(qk[e] << 16);
        z[e] += (m.code[t] != -1) ? qv * dqv : 0.f;
        // replayed rows have no dq; their row of this staging tile holds one half of their fp32 dk (epilogue_dk)
        if (m.code[t] >= -1)
            *reinterpret_cast<__nv_bfloat16*>(smem + Smem::stage_dq + t * 256 + L * 2) = __float2bfloat16_rn(dqv);
    }
}

__device__ __forceinline__ void epilogue_dk(const RowData& m, unsigned char* smem, uint32_t tm_lane, int grp, int L, int H,
                                            int h, int replay_base, const uint32_t (&qk)[16], __nv_bfloat16* dk_,
                                            float* rk, float (&z)[16], float& g_part) {
    const int t0 = grp * 16;
    uint32_t xi[16], xe[16];
    tmem_ld16(tm_lane + COL_DK + t0, xi);
    tmem_ld16(tm_lane + COL_A + t0, xe);
    tmem_ld_wait();
#pragma unroll
    for (int e = 0; e < 16; e++) {
        const int t = t0 + e;
        const float kv = __uint_as_float(qk[e] & 0xffff0000u);
        const float inter = m.w[t] * __uint_as_float(xe[e]);
        const float dkv = __uint_as_float(xi[e]) + inter;
        const bool row_ok = m.code[t] != -1;
        z[e] = row_ok ? -kv * dkv : 0.f;
        g_part += row_ok ? kv * inter : 0.f;
        // replayed rows (chunk 0 only) keep fp32: features 0..63 in the row's 256 bytes of the dk staging tile,
        // 64..127 in its row of the dq staging tile (replayed rows have no dq); every operand tile is still being read
        if (m.code[t] < -1)
            *reinterpret_cast<float*>(smem + (L < 64 ? Smem::stage_dk : Smem::stage_dq) + t * 256 + (L & 63) * 4) = dkv;
        else
            *reinterpret_cast<__nv_bfloat16*>(smem + Smem::stage_dk + t * 256 + L * 2) = __float2bfloat16_rn(dkv);
    }
}

__device__ __forceinline__ void epilogue_dv(const RowData& m, unsigned char* smem, uint32_t tm_lane, int grp, int L, int H,
                                            int h, int replay_base, __nv_bfloat16* dv_, float* rv) {
    const int t0 = grp * 16;
    uint32_t xi[16], xe[16];
    tmem_ld16(tm_lane + COL_DV + t0, xi);
    tmem_ld16(tm_lane + COL_DA + t0, xe);
    tmem_ld_wait();
#pragma unroll
    for (int e = 0; e < 16; e++) {
        const int t = t0 + e;
        const float dvv = __uint_as_float(xi[e]) + m.w[t] * __uint_as_float(xe[e]);
        *reinterpret_cast<__nv_bfloat16*>(smem + Smem::stage_dv + t * 256 + L * 2) = __float2bfloat16_rn(dvv);
        // replayed rows: fp32 over the bf16 copy of dS, which no MMA reads once the dk and dv groups are done
        if (m.code[t] < -1) *reinterpret_cast<float*>(smem + Smem::ds + t * 512 + L * 4) = dvv;
    }
}

// ---- full chunks: the epilogue in matrix-fragment layout -------------------------------------------------------------
// All 64 rows of the chunk are own rows.  A warp covers 32 features (its tensor-memory lane quarter) x 16 rows t (its
// column group); tcgen05.ld hands every thread 16 values as fragments of 8x8 matrices: features f = m + 8 fa
// (m = lane >> 2, fa = 0..3), rows t = t0 + 8 ta + 2 c + {0, 1} (c = lane & 3, ta = 0, 1).  q and k arrive in the same
// layout by ldmatrix (transposing), the outputs leave by stmatrix (transposing) into 128-byte-swizzled [row][64
// features] panels that TMA stores pick up: no 2-byte shared-memory accesses and no transposed reads.
struct Frag {
    uint32_t q[2][4], k[2][4];      // [ta][fa], two bf16 per register: rows t, t + 1
};
// value index -> (fa, ta, low/high row of the pair) for register r of load l (l = 0: lanes +0, l = 1: lanes +16)
__device__ __forceinline__ float frag_elem(const uint32_t (&f)[2][4], int l, int r) {
    const uint32_t pair = f[r >> 2][2 * l + ((r >> 1) & 1)];
    return __uint_as_float((r & 1) ? (pair & 0xffff0000u) : (pair << 16));
}
__device__ __forceinline__ uint32_t frag_addr(uint32_t tile, int lane, int Lq, int t0, int ta) {
    const int f = Lq + 8 * (lane >> 3), t = t0 + 8 * ta + (lane & 7);
    return tile + (f >> 6) * PANEL + sw128_chunk(t, (f & 63) >> 3);
}
__device__ __forceinline__ void frag_store(uint32_t stage, int lane, int Lq, int t0, const float (&val)[2][8]) {
#pragma unroll
    for (int ta = 0; ta < 2; ta++) {
        uint32_t pk[4];
#pragma unroll
        for (int fa = 0; fa < 4; fa++) {
            const int l = fa >> 1, r = 4 * ta + 2 * (fa & 1);
            pk[fa] = pack_bf16(val[l][r], val[l][r + 1]);
        }
        stmatrix_x4_trans(frag_addr(stage, lane, Lq, t0, ta), pk);
    }
}

// ONE_LAUNCH: all rounds in one launch (work items drawn from `ticket`, hand-off gradients published
// and awaited through `ds0_flags`); otherwise one round per launch and neither pointer is looked at.
template <bool ONE_LAUNCH>
__global__ void __launch_bounds__(NT, 1)
tc_bwd_kernel(const harts_la_tables_t tb, int seq_lo, int n_items, int H, const __grid_constant__ CUtensorMap map_q,
              const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_cs,
              const __grid_constant__ CUtensorMap map_dq, const __grid_constant__ CUtensorMap map_dk,
              const __grid_constant__ CUtensorMap map_dv, const __nv_bfloat16* __restrict__ q,
              const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ g,
              const __nv_bfloat16* __restrict__ dO, __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk_,
              __nv_bfloat16* __restrict__ dv_, float* __restrict__ dg, float* __restrict__ ds0, float* __restrict__ rk,
              float* __restrict__ rv, float* __restrict__ rg, int* status, const int32_t* gate, int* ds0_flags,
              int* ticket, const RoundOrder rounds) {
    if (gate_closed(gate)) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    unsigned char* sQ = smem + Smem::q;
    unsigned char* sK = smem + Smem::k;
    unsigned char* sV = smem + Smem::v;
    unsigned char* sDO = smem + Smem::dO;
    unsigned char* sDOs = smem + Smem::dOs;
    unsigned char* sP = smem + Smem::p;
    unsigned char* sDP = smem + Smem::dp;
    unsigned char* sS = smem + Smem::s;
    unsigned char* sDS = smem + Smem::ds;
    Misc& m = *reinterpret_cast<Misc*>(smem + Smem::misc);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_compute = warp < NC / 32;
    const bool is_issuer = tid == NC;              // first lane of the issuing warp
    const bool is_aux = warp == NC / 32 + 1;       // row data of the next chunk, dg of the finished one
    const int grp = warp >> 2;                    // column group (compute warps)
    const int L = (warp & 3) * 32 + lane;         // tensor-memory lane = feature index (or row t) of this thread
    const size_t state_elems = (size_t)D * D;

    if (tid == 0) {
        mbar_init(&m.bar_tiles, 1);
        mbar_init(&m.bar_tiles2, 1);
        mbar_init(&m.bar_a, 1);
        mbar_init(&m.bar_o, 1);
        mbar_init(&m.bar_o2, 1);
        mbar_init(&m.bar_o3, 1);
        mbar_init(&m.bar_qk_read, NC / 32);
        mbar_init(&m.bar_exit, 1);
        m.dead = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc<TMEM_COLS>(&m.tmem);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = m.tmem;
    const uint32_t tm_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);

    // Persistent CTAs: work item = (sequence, head); items are ordered longest sequence first and dealt to the CTAs
    // in a snake pattern, so that every CTA gets a similar amount of work.
    uint32_t ph_tiles = 0, ph_a = 0, ph_o = 0;
    bool tiles_pending = false, gave_up = false;   // tiles_pending is kept by the issuing thread only
    const int G = gridDim.x;
    for (int tier = 0;; tier++) {
    int item, seq_pos;
    if constexpr (ONE_LAUNCH) {
        // all rounds in one launch: whichever CTA is free draws the next item; the order is last round first, and
        // inside a round the plan's order (longest sequence first)
        if (tid == 0) m.item = atomicAdd(ticket, 1);
        __syncthreads();
        item = m.item;
        __syncthreads();
        if (item >= n_items) break;
        int j = item / H;
        seq_pos = -1;
        for (int r = rounds.n - 1; r >= 0 && seq_pos < 0; r--) {
            const int cnt = rounds.ptr[r + 1] - rounds.ptr[r];
            if (j < cnt) seq_pos = rounds.ptr[r] + j;
            else j -= cnt;
        }
    } else {
        if (tier * G >= n_items) break;
        item = (tier & 1) ? tier * G + (G - 1 - (int)blockIdx.x) : tier * G + (int)blockIdx.x;
        if (item >= n_items) continue;
        seq_pos = seq_lo + item / H;
    }
    const int seq = tb.seq_order ? tb.seq_order[seq_pos] : seq_pos;
    // the item's record lives in shared memory and is read where it is needed: held in registers over the whole walk it
    // would push the kernel over its register budget
    __syncthreads();                               // the previous item's last readers of the record are through
    if (tid == 0) {
        m.seq = seq_info(tb, seq);
        m.head = item % H;
    }
    __syncthreads();
    const SeqInfo& s = m.seq;
    const int h = *(volatile int*)&m.head;
    if (is_compute) {   // dS = 0: nothing follows the last chunk
        uint32_t zero[32];
#pragma unroll
        for (int i = 0; i < 32; i++) zero[i] = 0u;
        tmem_st32(tm_lane + COL_DS + grp * 32, zero);
        tmem_st_wait();
    }

    const uint32_t aQ = smem_u32(sQ), aK = smem_u32(sK), aV = smem_u32(sV), aDO = smem_u32(sDO), aDOs = smem_u32(sDOs),
                   aP = smem_u32(sP), aDP = smem_u32(sDP), aS = smem_u32(sS), aDS = smem_u32(sDS);
    constexpr uint32_t I_KK64 = instr_desc(128, 64, 0, 0);
    constexpr uint32_t I_MK64 = instr_desc(128, 64, 1, 0);
    constexpr uint32_t I_MM64 = instr_desc(128, 64, 1, 1);
    constexpr uint32_t I_MM128 = instr_desc(128, 128, 1, 1);

    // loop-invariant operand descriptors (k-step 0); "k" = contraction dimension contiguous, "m" = the other one
    const uint64_t dQk = desc_kmajor_base(aQ), dKk = desc_kmajor_base(aK), dVk = desc_kmajor_base(aV),
                   dDOk_hi = desc_kmajor_base(aDO - PANEL),   // rows 64..127 of this operand are the dO tile
                   dDOsk = desc_kmajor_base(aDOs), dDPk = desc_kmajor_base(aDP), dDSk = desc_kmajor_base(aDS);
    const uint64_t dQm = desc_mnmajor_base<BT>(aQ), dKm = desc_mnmajor_base<BT>(aK), dDOm = desc_mnmajor_base<BT>(aDO),
                   dDOsm = desc_mnmajor_base<BT>(aDOs), dPm = desc_mnmajor_base<BT>(aP),
                   dDPm = desc_mnmajor_base<BT>(aDP), dDSm = desc_mnmajor_base<D>(aDS);
    const uint64_t dSk = desc_kmajor_base(aS);

    // The tiles of a chunk travel on two barriers, in the order in which the chunk needs them: the chunk state and
    // dO first (the dS pass starts on them), then q, k, v (the A / dA MMAs, which run under that pass).  They are
    // requested as soon as the previous chunk's MMAs are done (the epilogue works from registers and tensor memory
    // only), so the loads overlap the epilogue, and the second half of them the dS pass.
    auto issue_tiles = [&](int c, bool tiles) {
        int row0 = s.own_begin - s.n_replay + c * BT;
        int idx = (s.chunk_base + c) * H + h;
        tiles_pending = true;
        mbar_expect_tx(&m.bar_tiles, (tiles ? TILE : 0) + 2 * S_PANEL);
        if (tiles)
            for (int p = 0; p < 2; p++) tma_load_3d(sDO + p * PANEL, &map_do, p * 64, h, row0, &m.bar_tiles);
        tma_load_3d(sS, &map_cs, 0, 0, idx, &m.bar_tiles);
        tma_load_3d(sS + S_PANEL, &map_cs, 64, 0, idx, &m.bar_tiles);
        mbar_expect_tx(&m.bar_tiles2, tiles ? 3 * TILE : 0);
        if (tiles)
            for (int p = 0; p < 2; p++) {
                tma_load_3d(sV + p * PANEL, &map_v, p * 64, h, row0, &m.bar_tiles2);
                tma_load_3d(sQ + p * PANEL, &map_q, p * 64, h, row0, &m.bar_tiles2);
                tma_load_3d(sK + p * PANEL, &map_k, p * 64, h, row0, &m.bar_tiles2);
            }
    };
    // Row codes and g of chunk c for rows `lane` and `lane + 32` (the auxiliary warp prepares a chunk's row data on its own).
    auto load_rows = [&](int c, int (&code)[2], float (&gv)[2]) {
#pragma unroll
        for (int r = 0; r < 2; r++) {
            code[r] = -1;
            gv[r] = 0.f;
            int vr = c * BT + lane + 32 * r;
            if (c >= 0 && vr < s.n_virtual) {
                int row = vr < s.n_replay ? tb.replay_row[s.replay_base + vr] : s.own_begin + (vr - s.n_replay);
                code[r] = vr < s.n_replay ? -2 - row : row;
                gv[r] = g[(size_t)row * H + h];
            }
        }
    };
    auto store_rows = [&](RowData& rd, const int (&code)[2], const float (&gv)[2]) {
        float x0 = gv[0], x1 = gv[1];
#pragma unroll
        for (int o_ = 1; o_ < 32; o_ <<= 1) {
            float y0 = __shfl_up_sync(0xffffffffu, x0, o_), y1 = __shfl_up_sync(0xffffffffu, x1, o_);
            if (lane >= o_) {
                x0 += y0;
                x1 += y1;
            }
        }
        x1 += __shfl_sync(0xffffffffu, x0, 31);
        const float bn = __shfl_sync(0xffffffffu, x1, 31);
        const float b[2] = {x0, x1};
#pragma unroll
        for (int r = 0; r < 2; r++) {
            int t = lane + 32 * r;
            rd.code[t] = code[r];
            rd.b2[t] = b[r] * LOG2E;
            rd.eb[t] = code[r] >= 0 ? ex2(b[r] * LOG2E) : 0.f;     // rows without an output carry no dO
            rd.w[t] = ex2((bn - b[r]) * LOG2E);
        }
        if (lane == 0) rd.gamma = ex2(bn * LOG2E);
    };

    const bool gather_first = s.n_replay > 0;
    int next_req = s.req_hi - 1;
    // chunk index of the next exported boundary on the way down (kept in a register: no global load per chunk)
    int next_boundary = next_req >= s.req_lo ? tb.slot_chunk[next_req] : -1;
    int aux_req = next_req, aux_boundary = next_boundary;    // the auxiliary warp's own walk over the boundaries
    if (is_issuer) issue_tiles(s.n_chunks - 1, !(gather_first && s.n_chunks == 1));
    int nx_code[2];
    float nx_g[2];
    if (is_aux) {
        load_rows(s.n_chunks - 1, nx_code, nx_g);
        store_rows(m.rows[0], nx_code, nx_g);
    }
    int cur = 0;

    tc_fence_before();
    __syncthreads();                              // row data of the first chunk visible
    tc_fence_after();

    // Two block-wide barriers per chunk: (A) before the MMA batch, (B) at the end of the epilogue.  After (B) the
    // compute warps go straight on to the next chunk, while the issuing thread sends the staged outputs off and the
    // auxiliary warp finishes dg for the chunk just done.
    for (int c = s.n_chunks - 1; c >= 0; c--, cur ^= 1) {
        const bool gathered = c == 0 && gather_first;
        // all 64 rows are own rows: outputs leave through staged TMA stores
        const bool full = !gathered && (c + 1) * BT <= s.n_virtual;
        const RowData& rd = m.rows[cur];
        if (gathered) {
            for (int e = tid; e < BT * 16; e += NT) {
                int row = e >> 4, ch = e & 15, code = rd.code[row];
                uint4 zero = make_uint4(0, 0, 0, 0), kq = zero, vq = zero, qq = zero, dq4 = zero;
                if (code != -1) {
                    int r = code >= 0 ? code : -2 - code;
                    size_t off = ((size_t)r * H + h) * D + ch * 8;
                    kq = *reinterpret_cast<const uint4*>(k + off);
                    vq = *reinterpret_cast<const uint4*>(v + off);
                    if (code >= 0) {
                        qq = *reinterpret_cast<const uint4*>(q + off);
                        dq4 = *reinterpret_cast<const uint4*>(dO + off);
                    }
                }
                uint32_t dst = (ch >> 3) * PANEL + sw128_chunk(row, ch & 7);
                *reinterpret_cast<uint4*>(sQ + dst) = qq;
                *reinterpret_cast<uint4*>(sK + dst) = kq;
                *reinterpret_cast<uint4*>(sV + dst) = vq;
                *reinterpret_cast<uint4*>(sDO + dst) = dq4;
            }
            fence_async_smem();
            __syncthreads();
        }
        const bool got_tiles = mbar_wait(&m.bar_tiles, ph_tiles, status, &m.dead);
        // ---- A = Q K^T on lanes 0..63, dA = dO V^T on lanes 64..127 (rows 0..63 of that operand are unused) ----------
        if (is_issuer) {
            if (mbar_wait(&m.bar_tiles2, ph_tiles, status, &m.dead) && got_tiles) tiles_pending = false;
            tc_fence_after();
#pragma unroll
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_A, dQk + kstep_kmajor<BT>(ks), dKk + kstep_kmajor<BT>(ks), I_KK64, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_DA, dDOk_hi + kstep_kmajor<BT>(ks), dVk + kstep_kmajor<BT>(ks), I_KK64, ks > 0);
            mma_commit(&m.bar_a);
            tma_store_wait_read();                // the previous chunk's output stores have left the staging tiles
        }
        if (got_tiles) ph_tiles ^= 1;
        if (is_aux) {
            load_rows(c - 1, nx_code, nx_g);              // next chunk's rows and g, in flight during this chunk
            if (aux_boundary == c + 1) {                  // the boundary this chunk's dS pass is crossing
                aux_req--;
                aux_boundary = aux_req >= s.req_lo ? tb.slot_chunk[aux_req] : -1;
            }
            if (ONE_LAUNCH && aux_boundary == c) {
                // all rounds in one launch: the next chunk crosses an exported boundary; the sequences that started
                // there may still be running elsewhere.  Waited for here, a chunk ahead and off the compute warps' path;
                // barrier (B) hands the result on.
                for (int u = tb.slot_cons_ptr[aux_req] + lane; u < tb.slot_cons_ptr[aux_req + 1]; u += 32)
                    flag_wait(ds0_flags + (size_t)tb.slot_cons_seq[u] * H + h, status, &m.dead);
                __syncwarp();
            }
        }
        float g_part = 0.f;                       // this thread's share of <S_{c+1}, dS_{c+1}>
        uint32_t qk[16];                          // q[t][L] | k[t][L] << 16 of this thread's 16 rows (bf16 bits)
        if (is_compute) {
            // ---- dS pass: add hand-off gradients, bf16 operand copy, <S_c, dS>, pre-scale by gamma -----------------
            {
                const bool boundary = next_boundary == c + 1;
                // one launch per round: all consumers' gradients were summed into the first consumer's buffer by
                // handoff_reduce; all rounds in one launch: they are summed here, in the same order
                const int cons_lo = boundary ? tb.slot_cons_ptr[next_req] : 0;
                const int cons_all = boundary ? tb.slot_cons_ptr[next_req + 1] : 0;
                const int cons_hi = ONE_LAUNCH ? cons_all : min(cons_all, cons_lo + 1);
                const float gamma = rd.gamma;
                float dot = 0.f;
                const int blk = grp;
                uint32_t x[32];
                tmem_ld32(tm_lane + COL_DS + blk * 32, x);
                // dO~ = e^{b_t} dO (zero on rows without an output): two 16-byte vectors per thread
                for (int e = tid; e < BT * 16; e += NC) {
                    uint32_t off = e * 16;
                    float sc = rd.eb[(off % PANEL) >> 7];
                    uint4 raw = *reinterpret_cast<const uint4*>(sDO + off);
                    __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
                    for (int e2 = 0; e2 < 4; e2++) {
                        float2 f = __bfloat1622float2(h2[e2]);
                        h2[e2] = sc != 0.f ? __floats2bfloat162_rn(f.x * sc, f.y * sc) : __floats2bfloat162_rn(0.f, 0.f);
                    }
                    *reinterpret_cast<uint4*>(sDOs + off) = raw;
                }
                tmem_ld_wait();
                if (cons_lo < cons_hi) {
                    const size_t in_state = (size_t)L * D + blk * 32;
                    const float4* first = reinterpret_cast<const float4*>(
                        ds0 + ((size_t)tb.slot_cons_seq[cons_lo] * H + h) * state_elems + in_state);
#pragma unroll
                    for (int i4 = 0; i4 < 8; i4++) {
                        float4 a;
                        if constexpr (ONE_LAUNCH) {       // written during this launch by other CTAs: read past L1
                            a = __ldcg(first + i4);
                            for (int u = cons_lo + 1; u < cons_hi; u++) {
                                const float4 b4 = __ldcg(reinterpret_cast<const float4*>(
                                    ds0 + ((size_t)tb.slot_cons_seq[u] * H + h) * state_elems + in_state) + i4);
                                a.x += b4.x; a.y += b4.y; a.z += b4.z; a.w += b4.w;
                            }
                        } else {
                            a = first[i4];
                        }
                        x[i4 * 4 + 0] = __float_as_uint(__uint_as_float(x[i4 * 4 + 0]) + a.x);
                        x[i4 * 4 + 1] = __float_as_uint(__uint_as_float(x[i4 * 4 + 1]) + a.y);
                        x[i4 * 4 + 2] = __float_as_uint(__uint_as_float(x[i4 * 4 + 2]) + a.z);
                        x[i4 * 4 + 3] = __float_as_uint(__uint_as_float(x[i4 * 4 + 3]) + a.w);
                    }
                }
#pragma unroll
                for (int v4 = 0; v4 < 4; v4++) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(x[v4 * 8 + 0]), __uint_as_float(x[v4 * 8 + 1]));
                    pk.y = pack_bf16(__uint_as_float(x[v4 * 8 + 2]), __uint_as_float(x[v4 * 8 + 3]));
                    pk.z = pack_bf16(__uint_as_float(x[v4 * 8 + 4]), __uint_as_float(x[v4 * 8 + 5]));
                    pk.w = pack_bf16(__uint_as_float(x[v4 * 8 + 6]), __uint_as_float(x[v4 * 8 + 7]));
                    int col = blk * 32 + v4 * 8;
                    *reinterpret_cast<uint4*>(sDS + (col >> 6) * S_PANEL + sw128_chunk(L, (col & 63) >> 3)) = pk;
                }
                // <S_c[i][:], dS[i][:]> over this thread's 32 columns: row i = L of the state tile, four 16-byte chunks
#pragma unroll
                for (int v4 = 0; v4 < 4; v4++) {
                    int col = blk * 32 + v4 * 8;
                    uint4 raw = *reinterpret_cast<const uint4*>(sS + (col >> 6) * S_PANEL + sw128_chunk(L, (col & 63) >> 3));
                    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw);
#pragma unroll
                    for (int e2 = 0; e2 < 4; e2++) {
                        float2 f = __bfloat1622float2(h2[e2]);
                        dot += f.x * __uint_as_float(x[v4 * 8 + 2 * e2]) + f.y * __uint_as_float(x[v4 * 8 + 2 * e2 + 1]);
                    }
                }
#pragma unroll
                for (int i = 0; i < 32; i++) x[i] = __float_as_uint(__uint_as_float(x[i]) * gamma);
                tmem_st32(tm_lane + COL_DS + blk * 32, x);     // awaited at the end of the masking pass
                if (boundary) {
                    next_req--;
                    next_boundary = next_req >= s.req_lo ? tb.slot_chunk[next_req] : -1;
                }
                g_part = gamma * dot;
            }
            // ---- P = A .* decay (lanes 0..63), dP = dA .* decay (lanes 64..127): 16 columns of one of them per thread ------
            mbar_wait(&m.bar_a, ph_a, status, &m.dead);
            tc_fence_after();
            {
                const bool is_p = (warp & 3) < 2;
                const int t = L & 63;
                unsigned char* dst = is_p ? sP : sDP;
                if (grp * 16 > ((warp & 1) * 32 + 31)) {
                    // this warp's 32 rows x 16 columns lie entirely above the diagonal
                    *reinterpret_cast<uint4*>(dst + sw128_chunk(t, grp * 2)) = make_uint4(0, 0, 0, 0);
                    *reinterpret_cast<uint4*>(dst + sw128_chunk(t, grp * 2 + 1)) = make_uint4(0, 0, 0, 0);
                } else {
                const float bt = rd.b2[t];
                // replay rows and rows past the end have no dO and no q: nothing is visible to them (limit = -1)
                const int limit = rd.code[t] >= 0 ? t : -1;
                uint32_t xa[16];
                tmem_ld16(tm_lane + (is_p ? COL_A : COL_DA) + grp * 16, xa);
                // the 16 column decays with four 16-byte loads; no load or branch under the per-element condition
                float bj[16];
#pragma unroll
                for (int v = 0; v < 4; v++)
                    *reinterpret_cast<float4*>(bj + 4 * v) = *reinterpret_cast<const float4*>(rd.b2 + grp * 16 + 4 * v);
                tmem_ld_wait();
#pragma unroll
                for (int v4 = 0; v4 < 2; v4++) {
                    float ya[8];
#pragma unroll
                    for (int e = 0; e < 8; e++) {
                        const int j = grp * 16 + v4 * 8 + e;
                        const float y = __uint_as_float(xa[v4 * 8 + e]) * ex2(bt - bj[v4 * 8 + e]);
                        ya[e] = j <= limit ? y : 0.f;      // a select: above the diagonal the product may be inf or NaN
                    }
                    *reinterpret_cast<uint4*>(dst + sw128_chunk(t, grp * 2 + v4)) =
                        make_uint4(pack_bf16(ya[0], ya[1]), pack_bf16(ya[2], ya[3]), pack_bf16(ya[4], ya[5]),
                                   pack_bf16(ya[6], ya[7]));
                }
                }
            }
            tmem_st_wait();
            fence_async_smem();
        }
        ph_a ^= 1;
        tc_fence_before();
        __syncthreads();                          // (A) all operand tiles and the scaled dS are in place
        tc_fence_after();
        const bool next_tiles = !(c - 1 == 0 && gather_first);
        if (is_issuer) {
            // Order of the three groups: the one with the longest epilogue first, the shortest last, so that little is
            // left to do once the last MMA is done.
            // dk^T: Q^T dP   |   dS V^T (into the columns A occupied)
#pragma unroll
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_DK, dQm + kstep_mnmajor(ks), dDPm + kstep_mnmajor(ks), I_MM64, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_A, dDSk + kstep_kmajor<D>(ks), dVk + kstep_kmajor<BT>(ks), I_KK64, ks > 0);
            mma_commit(&m.bar_o);
            // dv^T: dO^T P   |   dS^T K^T (into the columns dA occupied)
#pragma unroll
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_DV, dDOm + kstep_mnmajor(ks), dPm + kstep_mnmajor(ks), I_MM64, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_DA, dDSm + kstep_mnmajor(ks), dKk + kstep_kmajor<BT>(ks), I_MK64, ks > 0);
            mma_commit(&m.bar_o2);
            // dq^T = K^T dP^T + S_c dO~^T
#pragma unroll
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_DQ, dKm + kstep_mnmajor(ks), dDPk + kstep_kmajor<BT>(ks), I_MK64, ks > 0);
#pragma unroll
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_DQ, dSk + kstep_kmajor<D>(ks), dDOsk + kstep_kmajor<BT>(ks), I_KK64, true);
            // dS += Q^T dO~   (dS was pre-scaled by e^{b_n})
#pragma unroll
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_DS, dQm + kstep_mnmajor(ks), dDOsm + kstep_mnmajor(ks), I_MM128, true);
            mma_commit(&m.bar_o3);
            // every tile is free once these are done: the epilogue works from registers and tensor memory
            mbar_wait(&m.bar_o3, ph_o, status, &m.dead);
            mbar_wait(&m.bar_qk_read, ph_o, status, &m.dead);      // every compute warp has taken its q and k values
            if (c > 0) issue_tiles(c - 1, next_tiles);
        }
        if (is_aux && c > 0) store_rows(m.rows[cur ^ 1], nx_code, nx_g);   // visible to the others at barrier (B)
        if (is_compute) {
            if (full) {
                const int c4 = lane & 3, Lq = (warp & 3) * 32, t0 = grp * 16;
                Frag fr;
#pragma unroll
                for (int ta = 0; ta < 2; ta++) {
                    ldmatrix_x4_trans(frag_addr(aQ, lane, Lq, t0, ta), fr.q[ta]);
                    ldmatrix_x4_trans(frag_addr(aK, lane, Lq, t0, ta), fr.k[ta]);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&m.bar_qk_read);
                // e^{b_n - b_t} of this thread's four rows: t0 + 2c, +1, t0 + 8 + 2c, +1
                const float2 wlo = *reinterpret_cast<const float2*>(rd.w + t0 + 2 * c4);
                const float2 whi = *reinterpret_cast<const float2*>(rd.w + t0 + 8 + 2 * c4);
                const float wv[4] = {wlo.x, wlo.y, whi.x, whi.y};
                float zf[4] = {0.f, 0.f, 0.f, 0.f};              // q.dq - k.dk over this thread's features, per row
                float val[2][8];
                uint32_t xi[2][8], xe[2][8];
                // ---- dk -----------------------------------------------------------------------------------------------
                mbar_wait(&m.bar_o, ph_o, status, &m.dead);
                tc_fence_after();
#pragma unroll
                for (int l = 0; l < 2; l++) {
                    tmem_ld_frag16(tm_lane + ((uint32_t)(16 * l) << 16) + COL_DK + t0, xi[l]);
                    tmem_ld_frag16(tm_lane + ((uint32_t)(16 * l) << 16) + COL_A + t0, xe[l]);
                }
                tmem_ld_wait();
#pragma unroll
                for (int l = 0; l < 2; l++)
#pragma unroll
                    for (int r = 0; r < 8; r++) {
                        const int ti = 2 * (r >> 2) + (r & 1);
                        const float kv = frag_elem(fr.k, l, r);
                        const float inter = wv[ti] * __uint_as_float(xe[l][r]);
                        const float dkv = __uint_as_float(xi[l][r]) + inter;
                        zf[ti] -= kv * dkv;
                        g_part += kv * inter;
                        val[l][r] = dkv;
                    }
                frag_store(smem_u32(smem + Smem::stage_dk), lane, Lq, t0, val);
#pragma unroll
                for (int o_ = 16; o_ > 0; o_ >>= 1) g_part += __shfl_xor_sync(0xffffffffu, g_part, o_);
                if (lane == 0) m.gred[warp] = g_part;
                // ---- dv -----------------------------------------------------------------------------------------------
                mbar_wait(&m.bar_o2, ph_o, status, &m.dead);
                tc_fence_after();
#pragma unroll
                for (int l = 0; l < 2; l++) {
                    tmem_ld_frag16(tm_lane + ((uint32_t)(16 * l) << 16) + COL_DV + t0, xi[l]);
                    tmem_ld_frag16(tm_lane + ((uint32_t)(16 * l) << 16) + COL_DA + t0, xe[l]);
                }
                tmem_ld_wait();
#pragma unroll
                for (int l = 0; l < 2; l++)
#pragma unroll
                    for (int r = 0; r < 8; r++)
                        val[l][r] = __uint_as_float(xi[l][r]) + wv[2 * (r >> 2) + (r & 1)] * __uint_as_float(xe[l][r]);
                frag_store(smem_u32(smem + Smem::stage_dv), lane, Lq, t0, val);
                // ---- dq -----------------------------------------------------------------------------------------------
                mbar_wait(&m.bar_o3, ph_o, status, &m.dead);
                tc_fence_after();
#pragma unroll
                for (int l = 0; l < 2; l++) tmem_ld_frag16(tm_lane + ((uint32_t)(16 * l) << 16) + COL_DQ + t0, xi[l]);
                tmem_ld_wait();
#pragma unroll
                for (int l = 0; l < 2; l++)
#pragma unroll
                    for (int r = 0; r < 8; r++) {
                        const float dqv = __uint_as_float(xi[l][r]);
                        zf[2 * (r >> 2) + (r & 1)] += frag_elem(fr.q, l, r) * dqv;
                        val[l][r] = dqv;
                    }
                frag_store(smem_u32(smem + Smem::stage_dq), lane, Lq, t0, val);
                // rows are shared by the eight threads with the same c: sum over them, then one writer per row
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    zf[i] += __shfl_xor_sync(0xffffffffu, zf[i], 4);
                    zf[i] += __shfl_xor_sync(0xffffffffu, zf[i], 8);
                    zf[i] += __shfl_xor_sync(0xffffffffu, zf[i], 16);
                }
                if (lane < 4) {
                    m.red[warp][2 * c4] = zf[0];
                    m.red[warp][2 * c4 + 1] = zf[1];
                    m.red[warp][8 + 2 * c4] = zf[2];
                    m.red[warp][8 + 2 * c4 + 1] = zf[3];
                }
            } else {
            // q[t][L], k[t][L] of this thread's 16 rows, for the dg terms (read while the first MMAs run; after this
            // the epilogue does not touch the tiles, which are reloaded as soon as the MMAs are done)
            {
                const uint32_t qk_base = (L >> 6) * PANEL + (L & 7) * 2;
                const uint32_t cL = (L & 63) >> 3;
#pragma unroll
                for (int e = 0; e < 16; e++) {
                    const int t = grp * 16 + e;
                    const uint32_t off = qk_base + t * 128 + ((cL ^ (uint32_t)(t & 7)) << 4);
                    qk[e] = (uint32_t)*reinterpret_cast<const unsigned short*>(sQ + off) |
                            ((uint32_t)*reinterpret_cast<const unsigned short*>(sK + off) << 16);
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(&m.bar_qk_read);
            }
            // ---- epilogue in three parts, each as soon as its accumulators are complete -------------------------------
            float z[16];
            mbar_wait(&m.bar_o, ph_o, status, &m.dead);
            tc_fence_after();
            epilogue_dk(rd, smem, tm_lane, grp, L, H, h, s.replay_base, qk, dk_, rk, z, g_part);
#pragma unroll
            for (int o_ = 16; o_ > 0; o_ >>= 1) g_part += __shfl_xor_sync(0xffffffffu, g_part, o_);
            if (lane == 0) m.gred[warp] = g_part;
            mbar_wait(&m.bar_o2, ph_o, status, &m.dead);
            tc_fence_after();
            epilogue_dv(rd, smem, tm_lane, grp, L, H, h, s.replay_base, dv_, rv);
            mbar_wait(&m.bar_o3, ph_o, status, &m.dead);
            tc_fence_after();
            epilogue_dq(rd, smem, tm_lane, grp, L, H, h, qk, dq, z);
            const float row_total = warp_transpose_reduce16(z, lane);
            if (lane < 16) m.red[warp][lane] = row_total;
            }
            if (full) fence_async_smem();
        }
        ph_o ^= 1;
        tc_fence_before();
        gave_up = __syncthreads_or(m.dead) != 0;  // (B) staged outputs, partial sums and the next chunk's row data visible
        tc_fence_after();
        if (gave_up) break;
        if (is_compute && !full) {
            // partial chunk: the staged rows leave with 16-byte stores, own rows to the outputs (bf16), replayed rows
            // to the scratch (fp32); rows past the end go nowhere
            for (int e = tid; e < BT * 16 * 3; e += NC) {
                const int which = e / (BT * 16), t = (e / 16) % BT, j = e % 16, code = rd.code[t];
                if (code < 0) continue;
                __nv_bfloat16* out = which == 0 ? dq : (which == 1 ? dk_ : dv_);
                const int stage = which == 0 ? Smem::stage_dq : (which == 1 ? Smem::stage_dk : Smem::stage_dv);
                *reinterpret_cast<uint4*>(out + ((size_t)code * H + h) * D + j * 8) =
                    *reinterpret_cast<const uint4*>(smem + stage + t * 256 + j * 16);
            }
            if (gathered)
                for (int e = tid; e < BT * 32 * 2; e += NC) {
                    const int which = e / (BT * 32), t = (e / 32) % BT, j = e % 32;
                    if (rd.code[t] >= -1) continue;
                    float* out = which == 0 ? rk : rv;
                    const int src = which == 1 ? Smem::ds + t * 512 + j * 16
                                               : (j < 16 ? Smem::stage_dk : Smem::stage_dq) + t * 256 + (j & 15) * 16;
                    *reinterpret_cast<float4*>(out + ((size_t)(s.replay_base + t) * H + h) * D + j * 4) =
                        *reinterpret_cast<const float4*>(smem + src);
                }
        }
        if (is_issuer && full) {
            int row0 = s.own_begin - s.n_replay + c * BT;
            for (int p = 0; p < 2; p++) {         // the staging tiles of a full chunk are swizzled [row][64] panels
                tma_store_3d(&map_dq, smem + Smem::stage_dq + p * PANEL, p * 64, h, row0);
                tma_store_3d(&map_dk, smem + Smem::stage_dk + p * PANEL, p * 64, h, row0);
                tma_store_3d(&map_dv, smem + Smem::stage_dv + p * PANEL, p * 64, h, row0);
            }
            tma_store_commit();
        }
        if (is_aux) {
            // dg_t = sum_{tau >= t} r_tau + <S_{c+1}, dS_{c+1}>, rows `lane` and `lane + 32` per thread of this warp
            auto row_sum = [&](int t) {
                const int g4 = (t >> 4) * 4, e = t & 15;
                return m.red[g4][e] + m.red[g4 + 1][e] + m.red[g4 + 2][e] + m.red[g4 + 3][e];
            };
            float lo = row_sum(lane), hi = row_sum(lane + 32);
#pragma unroll
            for (int o_ = 1; o_ < 32; o_ <<= 1) {
                float y0 = __shfl_down_sync(0xffffffffu, lo, o_), y1 = __shfl_down_sync(0xffffffffu, hi, o_);
                if (lane + o_ < 32) {
                    lo += y0;
                    hi += y1;
                }
            }
            float G = __shfl_sync(0xffffffffu, hi, 0);     // total of rows 32..63
            float Gs = 0.f;
#pragma unroll
            for (int w_ = 0; w_ < NC / 32; w_++) Gs += m.gred[w_];
            const float val[2] = {lo + G + Gs, hi + Gs};
#pragma unroll
            for (int r = 0; r < 2; r++) {
                int t = lane + 32 * r, code = rd.code[t];
                if (code >= 0) dg[(size_t)code * H + h] = val[r];
                else if (code < -1) rg[(size_t)(s.replay_base + t) * H + h] = val[r];
            }
        }
    }
    if (gave_up) break;
    // gradient w.r.t. the initial state: the hand-off into the producing sequence
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (is_compute && s.init_slot >= 0) {
        float* dst = ds0 + ((size_t)seq * H + h) * state_elems + (size_t)L * D;
        uint32_t x[32];
        tmem_ld32(tm_lane + COL_DS + grp * 32, x);
        tmem_ld_wait();
#pragma unroll
        for (int i4 = 0; i4 < 8; i4++)
            reinterpret_cast<float4*>(dst + grp * 32)[i4] =
                make_float4(__uint_as_float(x[i4 * 4]), __uint_as_float(x[i4 * 4 + 1]), __uint_as_float(x[i4 * 4 + 2]),
                            __uint_as_float(x[i4 * 4 + 3]));
        if (ONE_LAUNCH) __threadfence();           // this thread's part, before the flag that follows the barrier below
    }
    if (ONE_LAUNCH && s.init_slot >= 0) {           // publish: the gradient of this sequence's initial state is in place
        if (!__syncthreads_or(m.dead) && tid == 0) flag_set(ds0_flags + (size_t)seq * H + h);
    }
    }   // work items
    const bool abandoned = __syncthreads_or(m.dead) != 0;
    if (abandoned && is_issuer) {                  // let copies and MMAs in flight finish (bounded)
        if (tiles_pending) {
            mbar_wait_drain(&m.bar_tiles, ph_tiles);
            mbar_wait_drain(&m.bar_tiles2, ph_tiles);
        }
        mma_commit(&m.bar_exit);
        mbar_wait_drain(&m.bar_exit, 0);
    }
    if (is_issuer) tma_store_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc<TMEM_COLS>(tmem);
}

}  // namespace

int32_t tc_bwd(const BwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (int32_t rc0 = handoff_reduce(a); rc0 != HARTS_OK) return rc0;
    CUtensorMap mq, mk, mv, mdo, mcs, mdq, mdk, mdv;
    int32_t rc;
    if ((rc = make_row_map(&mq, a.q, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, a.k, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, a.v, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdo, a.dO, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_state_map(&mcs, a.chunk_states, (int64_t)a.tb.n_chunks * a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdq, a.dq, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdk, a.dk_, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdv, a.dv_, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(tc_bwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    ScratchLayout sl = scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    int n = (a.seq_hi - a.seq_lo) * a.H;
    int grid = n < sm_count() ? n : sm_count();
    tc_bwd_kernel<false><<<grid, NT, Smem::bytes + 1024, a.stream>>>(
        a.tb, a.seq_lo, n, a.H, mq, mk, mv, mdo, mcs, mdq, mdk, mdv, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
        (const __nv_bfloat16*)a.v, a.g, (const __nv_bfloat16*)a.dO, (__nv_bfloat16*)a.dq, (__nv_bfloat16*)a.dk_,
        (__nv_bfloat16*)a.dv_, a.dg, (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
        (float*)(base + sl.rg), a.dev_status, status_gate(a.flags, a.dev_status), nullptr, nullptr, RoundOrder{});
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}


// All rounds of a plan in ONE launch: the persistent CTAs draw the (sequence, head) items from a ticket counter, last
// round first.  A sequence publishes a flag once its initial-state gradient is in the scratch area; a sequence that
// exported a boundary waits (its auxiliary warp does, one chunk ahead) for the flags of all the sequences that started
// there and sums their gradients itself, in the order handoff_reduce uses.  Those sequences sit in later rounds and
// hold smaller tickets, and a ticket is only ever held by a running CTA: they are running or done whether or not the
// whole grid is resident, so an ordinary launch cannot deadlock.  `flags`: caller-owned DEVICE array of n_seq * H
// int32, `ticket`: one int32; both zeroed here on the stream.  rounds: the plan's round table (sequences of round r =
// [ptr[r], ptr[r+1])).
int32_t tc_bwd_fused(const BwdArgs& a, int* flags, int* ticket, const RoundOrder& rounds) {
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    if (n == 0) return HARTS_OK;
    if (rounds.n < 1 || rounds.ptr[0] != a.seq_lo || rounds.ptr[rounds.n] != a.seq_hi) return HARTS_EINVAL;
    // offered while a CTA gets few items, where the idle tail of every round is what one launch saves (cfg1: 0.55 ->
    // 0.35 ms; cfg2, 7.5 items per CTA: 1.85 -> 1.72 ms); with many items per CTA it loses (cfg3: 12.05 -> 12.45 ms;
    // cfg4, 1,800 short items per CTA whose hand-off sums then run inside the walk: 42 -> 62 ms)
    if (n > ONE_LAUNCH_ITEMS_PER_CTA * sm_count()) return HARTS_EUNSUPPORTED;
    CUtensorMap mq, mk, mv, mdo, mcs, mdq, mdk, mdv;
    int32_t rc;
    if ((rc = make_row_map(&mq, a.q, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, a.k, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, a.v, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdo, a.dO, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_state_map(&mcs, a.chunk_states, (int64_t)a.tb.n_chunks * a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdq, a.dq, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdk, a.dk_, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdv, a.dv_, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(tc_bwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    if (cudaMemsetAsync(flags, 0, (size_t)a.tb.n_seq * a.H * sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    if (cudaMemsetAsync(ticket, 0, sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    ScratchLayout sl = scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    const int grid = n < sm_count() ? n : sm_count();
    tc_bwd_kernel<true><<<grid, NT, Smem::bytes + 1024, a.stream>>>(
        a.tb, a.seq_lo, n, a.H, mq, mk, mv, mdo, mcs, mdq, mdk, mdv, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
        (const __nv_bfloat16*)a.v, a.g, (const __nv_bfloat16*)a.dO, (__nv_bfloat16*)a.dq, (__nv_bfloat16*)a.dk_,
        (__nv_bfloat16*)a.dv_, a.dg, (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
        (float*)(base + sl.rg), a.dev_status, status_gate(a.flags, a.dev_status), flags, ticket, rounds);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
