// Tensor-core forward of the packed chunkwise call (Eq. 16) for bf16, d_k = d_v = 128, chunk 64.
//
// One CTA per (sequence, head) walks the chunks in order.  The recurrent state lives in tensor
// memory for the whole walk: lane i (0..127) holds row i of S (S[i][j'] for all j' in its 128 fp32
// columns).  Per chunk (b_t = running sum of g, n = last row, w_j = e^{b_n-b_j}):
//     A     = Q K^T                      tcgen05, M=128 (rows 64..127 unused) N=64  K=128
//     P     = A .* e^{b_t-b_j} [j<=t]    registers -> bf16 tile in shared memory
//     O1^T  = V^T P^T                    tcgen05, M=128 (d_v) N=64 (t) K=64 (j)
//     O2^T  = S_c^T Q^T                  tcgen05, M=128 N=64 K=128, S_c as bf16 tile [d_k][d_v]
//     o_t   = O1 + e^{b_t} O2            epilogue, own rows only
//     S     = e^{b_n} S + (w .* K)^T V   tcgen05 accumulate, M=128 N=128 K=64
// q/k/v tiles arrive by TMA as 128-byte-swizzled panels; the first chunk of a replay-started
// sequence is gathered row by row instead (replay rows come from arbitrary ancestor rows).  The
// start-of-chunk state goes to the chunk-state workspace (bf16, [d_k][d_v] per chunk-head) by TMA
// store, and to its slot (fp32, [d_k][d_v]) when the plan requests that boundary.
// Every wait is bounded; a wait that runs out sets the status word and a CTA-wide latch: the CTA leaves its loops at
// the next chunk boundary, waits (bounded) for what it still has in flight, releases tensor memory and returns.
#include "kernels.h"
#include "tc_common.cuh"

namespace harts {
namespace {

using namespace tc;

constexpr int BT = 64, D = 128;
constexpr int NT = 256;                       // 8 warps: warp w works on tensor-memory lanes 32(w&3)..+31, column half w>>2
constexpr int TILE = BT * D * 2;              // 16 KB: two panels of [64][64] bf16
constexpr int PANEL = BT * 128;               // 8 KB
constexpr int S_PANEL = D * 128;              // 16 KB: [128][64] bf16
constexpr float LOG2E = 1.4426950408889634f;

// tensor-memory columns
constexpr int COL_S = 0, COL_A = 128, COL_O1 = 192, TMEM_COLS = 256;

struct Smem {
    static constexpr int q = 0, k = TILE, v = 2 * TILE, p = 3 * TILE, s = 3 * TILE + PANEL,
                         stage = 3 * TILE + PANEL + 2 * S_PANEL,       // outputs of a full chunk, [row][feature]
                         misc = stage + TILE;
    static constexpr int bytes = misc + 2048;
};
struct SeqInfo {
    int own_begin, n_replay, n_virtual, n_chunks, replay_base, init_slot, req_lo, req_hi, chunk_base;
};
struct Misc {
    float part[BT];      // per-warp partial running sums of g
    float b2[BT];        // running log-decay, in log2 units
    float eb[BT];        // e^{b_t}
    float w[BT];         // e^{b_n - b_t}
    int code[BT];        // physical row (>= 0 own), -2 - row (replay), -1 (past the end)
    float gamma;
    uint32_t tmem;
    uint64_t bar_tma, bar_a, bar_o, bar_exit;
    int dead;            // latch: a wait of this CTA ran out, the walk is being abandoned
    int item;            // all rounds in one launch: the work item thread 0 drew
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

// Asks the L2 for what the NEXT work item of this CTA reads first: its initial state and the rows of its first chunk
// (q, k, v).  Out of line, so that it does not weigh on the kernel's register allocation; called once per item, while
// the item's last chunk waits for its MMAs.
__device__ __noinline__ void prefetch_item(const harts_la_tables_t& tb, int seq_lo, int item, int H, const float* slots,
                                           const __nv_bfloat16* q, const __nv_bfloat16* k, const __nv_bfloat16* v) {
    const int sp = seq_lo + item / H, h = item % H;
    const int seq = tb.seq_order ? tb.seq_order[sp] : sp;
    const int own_begin = tb.seq_own_begin[seq], own_len = tb.seq_own_begin[seq + 1] - own_begin;
    const int replay_base = tb.seq_replay_ptr[seq], n_replay = tb.seq_replay_ptr[seq + 1] - replay_base;
    const int init_slot = tb.seq_init_slot[seq];
    const int tid = threadIdx.x;
    if (init_slot >= 0) {
        const char* st = reinterpret_cast<const char*>(slots + ((size_t)init_slot * H + h) * (size_t)(D * D));
        for (int p = tid; p < D * D * 4 / 128; p += NT) asm volatile("prefetch.global.L2 [%0];" ::"l"(st + p * 128));
    }
    const int n_rows = min(BT, n_replay + own_len);
    for (int p = tid; p < n_rows * 2; p += NT) {
        const int vr = p >> 1;
        const int r = vr < n_replay ? tb.replay_row[replay_base + vr] : own_begin + (vr - n_replay);
        const size_t off = (((size_t)r * H + h) * D) * 2 + (p & 1) * 128;
        asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(k) + off));
        asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(v) + off));
        if (vr >= n_replay) asm volatile("prefetch.global.L2 [%0];" ::"l"(reinterpret_cast<const char*>(q) + off));
    }
}

// out of line: the wait loop's registers (timer values, counters) must not weigh on the kernel's allocation
__device__ __noinline__ void wait_for_slot(const int* flag, int* status, int* dead) { flag_wait(flag, status, dead); }

// ONE_LAUNCH: all rounds in one launch (work items drawn from `ticket`, sequences wait on `slot_flags`);
// otherwise one round per launch, items dealt statically, and neither pointer is looked at.
template <bool ONE_LAUNCH>
__global__ void __launch_bounds__(NT, 2)
tc_fwd_kernel(const harts_la_tables_t tb, int seq_lo, int n_items, int H, const __grid_constant__ CUtensorMap map_q,
              const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
              const __grid_constant__ CUtensorMap map_cs, const __grid_constant__ CUtensorMap map_o,
              const __nv_bfloat16* __restrict__ q,
              const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ g,
              __nv_bfloat16* __restrict__ o, float* __restrict__ slots, int store_states, int* status,
              const int32_t* gate, int* slot_flags, int* ticket) {
    if (gate_closed(gate)) return;
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    unsigned char* sQ = smem + Smem::q;
    unsigned char* sK = smem + Smem::k;
    unsigned char* sV = smem + Smem::v;
    unsigned char* sP = smem + Smem::p;
    unsigned char* sS = smem + Smem::s;
    unsigned char* sO = smem + Smem::stage;
    Misc& m = *reinterpret_cast<Misc*>(smem + Smem::misc);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int grp = warp >> 2;                    // column half
    const int L = (warp & 3) * 32 + lane;         // tensor-memory lane of this thread
    const size_t state_elems = (size_t)D * D;

    if (tid == 0) {
        mbar_init(&m.bar_tma, 1);
        mbar_init(&m.bar_a, 1);
        mbar_init(&m.bar_o, 1);
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
    uint32_t ph_tma = 0, ph_a = 0, ph_o = 0;
    bool tma_pending = false, gave_up = false;     // tma_pending is kept by thread 0 only
    const int G = gridDim.x;
    for (int tier = 0;; tier++) {
    int item;
    if constexpr (ONE_LAUNCH) {      // items are drawn in order (round by round) by whichever CTA is free
        if (tid == 0) m.item = atomicAdd(ticket, 1);
        __syncthreads();
        item = m.item;
        __syncthreads();
        if (item >= n_items) break;
    } else {
        if (tier * G >= n_items) break;
        item = (tier & 1) ? tier * G + (G - 1 - (int)blockIdx.x) : tier * G + (int)blockIdx.x;
        if (item >= n_items) continue;
    }
    SeqInfo s_own;
    if constexpr (ONE_LAUNCH) {
        if (tid == 0) {
            const int sp = seq_lo + item / H;
            m.seq = seq_info(tb, tb.seq_order ? tb.seq_order[sp] : sp);
            m.head = item % H;
        }
        __syncthreads();
    } else {
        const int sp = seq_lo + item / H;
        s_own = seq_info(tb, tb.seq_order ? tb.seq_order[sp] : sp);
    }
    const SeqInfo& s = ONE_LAUNCH ? const_cast<const SeqInfo&>(m.seq) : s_own;
    const int h = ONE_LAUNCH ? *(volatile int*)&m.head : item % H;
    if (ONE_LAUNCH && s.init_slot >= 0) {
        // all rounds in one launch: the producer of this sequence's initial state may still be running elsewhere
        if (tid == 0) wait_for_slot(slot_flags + (size_t)s.init_slot * H + h, status, &m.dead);
        __syncthreads();
    }
    // initial state into tensor memory: lane i = L holds S[i][:]
    {
        const float* src = s.init_slot < 0 ? nullptr : slots + ((size_t)s.init_slot * H + h) * state_elems + (size_t)L * D;
        for (int blk = 2 * grp; blk < 2 * grp + 2; blk++) {
            uint32_t x[32];
#pragma unroll
            for (int i4 = 0; i4 < 8; i4++) {
                // one launch: the slot was written during this launch by another CTA (read past L1); one launch per
                // round: siblings that start from the same slot on this SM find it in L1
                float4 a = !src ? make_float4(0.f, 0.f, 0.f, 0.f)
                           : ONE_LAUNCH ? __ldcg(reinterpret_cast<const float4*>(src + blk * 32) + i4)
                                        : reinterpret_cast<const float4*>(src + blk * 32)[i4];
                x[i4 * 4 + 0] = __float_as_uint(a.x);
                x[i4 * 4 + 1] = __float_as_uint(a.y);
                x[i4 * 4 + 2] = __float_as_uint(a.z);
                x[i4 * 4 + 3] = __float_as_uint(a.w);
            }
            tmem_st32(tm_lane + COL_S + blk * 32, x);
        }
        tmem_st_wait();
    }

    const uint32_t aQ = smem_u32(sQ), aK = smem_u32(sK), aV = smem_u32(sV), aP = smem_u32(sP), aS = smem_u32(sS);
    constexpr uint32_t IDESC_A = instr_desc(128, 64, 0, 0);    // Q (K-major) x K (K-major)
    constexpr uint32_t IDESC_O1 = instr_desc(128, 64, 1, 0);   // V^T (MN-major) x P (K-major)
    constexpr uint32_t IDESC_O2 = instr_desc(128, 64, 1, 0);   // S^T from the [d_k][d_v] tile (MN-major) x Q (K-major)
    constexpr uint32_t IDESC_S = instr_desc(128, 128, 1, 1);   // K~^T (MN-major) x V (MN-major)

    auto issue_tma = [&](int c) {
        int row0 = s.own_begin - s.n_replay + c * BT;
        tma_pending = true;
        mbar_expect_tx(&m.bar_tma, 3 * TILE);
        for (int p = 0; p < 2; p++) {
            tma_load_3d(sQ + p * PANEL, &map_q, p * 64, h, row0, &m.bar_tma);
            tma_load_3d(sK + p * PANEL, &map_k, p * 64, h, row0, &m.bar_tma);
            tma_load_3d(sV + p * PANEL, &map_v, p * 64, h, row0, &m.bar_tma);
        }
    };

    const bool gather_first = s.n_replay > 0;
    int next_req = s.req_lo;
    // chunk index of the next requested boundary (kept in a register: no global load per chunk)
    int next_boundary = next_req < s.req_hi ? tb.slot_chunk[next_req] : -1;
    if (!gather_first && tid == 0) issue_tma(0);

    // row codes and g of a chunk, loaded one chunk ahead (during the previous epilogue)
    auto row_code = [&](int c, int& code, float& gv) {
        code = -1;
        gv = 0.f;
        int vr = c * BT + tid;
        if (tid < BT && c < s.n_chunks && vr < s.n_virtual) {
            int r = vr < s.n_replay ? tb.replay_row[s.replay_base + vr] : s.own_begin + (vr - s.n_replay);
            code = vr < s.n_replay ? -2 - r : r;
            gv = g[(size_t)r * H + h];
        }
    };
    float gval;
    int my_code;
    row_code(0, my_code, gval);

    for (int c = 0; c < s.n_chunks; c++) {
        if (tid == 0) tma_store_wait_read();      // the previous chunk's state store has left sS
        tc_fence_before();
        gave_up = __syncthreads_or(m.dead) != 0;  // (1) epilogue of the previous chunk is over everywhere
        tc_fence_after();
        if (gave_up) break;
        if (tid < BT) {
            m.code[tid] = my_code;
            float x = gval;                       // inclusive scan inside each of the two warps
#pragma unroll
            for (int o_ = 1; o_ < 32; o_ <<= 1) {
                float y = __shfl_up_sync(0xffffffffu, x, o_);
                if (lane >= o_) x += y;
            }
            m.part[tid] = x;
        }
        if (c == 0 && gather_first) {
            __syncthreads();
            for (int e = tid; e < BT * 16; e += NT) {
                int row = e >> 4, ch = e & 15, code = m.code[row];
                uint4 zero = make_uint4(0, 0, 0, 0), kq = zero, vq = zero, qq = zero;
                if (code != -1) {
                    int r = code >= 0 ? code : -2 - code;
                    size_t off = ((size_t)r * H + h) * D + ch * 8;
                    kq = *reinterpret_cast<const uint4*>(k + off);
                    vq = *reinterpret_cast<const uint4*>(v + off);
                    if (code >= 0) qq = *reinterpret_cast<const uint4*>(q + off);
                }
                uint32_t dst = (ch >> 3) * PANEL + sw128_chunk(row, ch & 7);
                *reinterpret_cast<uint4*>(sQ + dst) = qq;
                *reinterpret_cast<uint4*>(sK + dst) = kq;
                *reinterpret_cast<uint4*>(sV + dst) = vq;
            }
            fence_async_smem();
        }
        __syncthreads();                          // (2) codes, gathered tiles, partial sums visible
        if (tid < BT) {
            float first_half_total = m.part[31];
            float b = m.part[tid] + (tid >= 32 ? first_half_total : 0.f);
            float bn = m.part[63] + first_half_total;
            m.b2[tid] = b * LOG2E;
            m.eb[tid] = ex2(b * LOG2E);
            m.w[tid] = ex2((bn - b) * LOG2E);
            if (tid == 0) m.gamma = ex2(bn * LOG2E);
        }
        if (!(c == 0 && gather_first)) {
            if (mbar_wait(&m.bar_tma, ph_tma, status, &m.dead)) {
                ph_tma ^= 1;
                tma_pending = false;
            }
        }
        // ---- A = Q K^T ----------------------------------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_A, desc_kmajor<BT>(aQ, ks), desc_kmajor<BT>(aK, ks), IDESC_A, ks > 0);
            mma_commit(&m.bar_a);
        }
        __syncthreads();                          // (3) b2 / eb / w / gamma visible
        // ---- state pass: S_c^T -> bf16 operand tile (+ slot), S^T <- gamma S^T ----------------------------
        {
            const bool export_slot = next_boundary == c;
            float* slot_dst = export_slot ? slots + ((size_t)next_req * H + h) * state_elems + (size_t)L * D : nullptr;
            const float gamma = m.gamma;
            for (int blk = 2 * grp; blk < 2 * grp + 2; blk++) {
                uint32_t x[32];
                tmem_ld32(tm_lane + COL_S + blk * 32, x);
                tmem_ld_wait();
                if (slot_dst) {
#pragma unroll
                    for (int i4 = 0; i4 < 8; i4++)
                        reinterpret_cast<float4*>(slot_dst + blk * 32)[i4] =
                            make_float4(__uint_as_float(x[i4 * 4]), __uint_as_float(x[i4 * 4 + 1]),
                                        __uint_as_float(x[i4 * 4 + 2]), __uint_as_float(x[i4 * 4 + 3]));
                }
#pragma unroll
                for (int v4 = 0; v4 < 4; v4++) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(x[v4 * 8 + 0]), __uint_as_float(x[v4 * 8 + 1]));
                    pk.y = pack_bf16(__uint_as_float(x[v4 * 8 + 2]), __uint_as_float(x[v4 * 8 + 3]));
                    pk.z = pack_bf16(__uint_as_float(x[v4 * 8 + 4]), __uint_as_float(x[v4 * 8 + 5]));
                    pk.w = pack_bf16(__uint_as_float(x[v4 * 8 + 6]), __uint_as_float(x[v4 * 8 + 7]));
                    int col = blk * 32 + v4 * 8;           // first of 8 consecutive j'
                    *reinterpret_cast<uint4*>(sS + (col >> 6) * S_PANEL + sw128_chunk(L, (col & 63) >> 3)) = pk;
                }
#pragma unroll
                for (int i = 0; i < 32; i++) x[i] = __float_as_uint(__uint_as_float(x[i]) * gamma);
                tmem_st32(tm_lane + COL_S + blk * 32, x);
            }
            tmem_st_wait();
            if (export_slot) {
                if (ONE_LAUNCH) __threadfence();           // this thread's part of the slot, before the flag below
                next_req++;
                next_boundary = next_req < s.req_hi ? tb.slot_chunk[next_req] : -1;
            }
            fence_async_smem();
        }
        // ---- P = A .* decay (warps 0,1)  |  K <- w .* K (warps 2,3) ------------------------------------------
        mbar_wait(&m.bar_a, ph_a, status, &m.dead);
        ph_a ^= 1;
        tc_fence_after();
        if ((warp & 3) < 2) {
            const int t = L;
            const float bt = m.b2[t];
            {
                const int half = grp;
                uint32_t x[32];
                tmem_ld32(tm_lane + COL_A + half * 32, x);
                tmem_ld_wait();
#pragma unroll
                for (int v4 = 0; v4 < 4; v4++) {
                    // the eight column decays with two 16-byte loads; no load or branch under the per-element condition
                    float bj[8];
                    *reinterpret_cast<float4*>(bj) = *reinterpret_cast<const float4*>(m.b2 + half * 32 + v4 * 8);
                    *reinterpret_cast<float4*>(bj + 4) = *reinterpret_cast<const float4*>(m.b2 + half * 32 + v4 * 8 + 4);
                    float y[8];
#pragma unroll
                    for (int e = 0; e < 8; e++) {
                        const int j = half * 32 + v4 * 8 + e;
                        const float p = __uint_as_float(x[v4 * 8 + e]) * ex2(bt - bj[e]);
                        y[e] = j <= t ? p : 0.f;           // a select: above the diagonal the product may be inf or NaN
                    }
                    uint4 pk = make_uint4(pack_bf16(y[0], y[1]), pack_bf16(y[2], y[3]), pack_bf16(y[4], y[5]),
                                          pack_bf16(y[6], y[7]));
                    *reinterpret_cast<uint4*>(sP + sw128_chunk(t, half * 4 + v4)) = pk;
                }
            }
        } else {
            for (int e = ((warp & 3) - 2) * 32 + lane + 64 * grp; e < BT * 16; e += 128) {
                uint32_t off = e * 16;
                float wj = m.w[(off % PANEL) >> 7];
                uint4 raw = *reinterpret_cast<uint4*>(sK + off);
                __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw);
#pragma unroll
                for (int e2 = 0; e2 < 4; e2++) {
                    float2 f = __bfloat1622float2(h2[e2]);
                    h2[e2] = __floats2bfloat162_rn(f.x * wj, f.y * wj);
                }
                *reinterpret_cast<uint4*>(sK + off) = raw;
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();                          // (4) P, scaled K, S operand tile and scaled S^T are in place
        tc_fence_after();
        // ---- O1^T, O2^T, state update --------------------------------------------------------------------
        if (tid == 0) {
            // the slot written during this chunk's state pass (every thread fenced its part before barrier (4))
            if (ONE_LAUNCH && next_req > s.req_lo && tb.slot_chunk[next_req - 1] == c)
                flag_set(slot_flags + (size_t)(next_req - 1) * H + h);
            if (store_states) {
                int idx = (s.chunk_base + c) * H + h;
                tma_store_3d(&map_cs, sS, 0, 0, idx);
                tma_store_3d(&map_cs, sS + S_PANEL, 64, 0, idx);
                tma_store_commit();
            }
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_O1, desc_mnmajor<BT>(aV, ks), desc_kmajor<BT>(aP, ks), IDESC_O1, ks > 0);
            for (int ks = 0; ks < 8; ks++)
                mma_ss(tmem + COL_A, desc_mnmajor<D>(aS, ks), desc_kmajor<BT>(aQ, ks), IDESC_O2, ks > 0);
            for (int ks = 0; ks < 4; ks++)
                mma_ss(tmem + COL_S, desc_mnmajor<BT>(aK, ks), desc_mnmajor<BT>(aV, ks), IDESC_S, true);
            mma_commit(&m.bar_o);
        }
        if constexpr (!ONE_LAUNCH) {
            if (c == s.n_chunks - 1) {                      // the next item of this CTA (snake order), if there is one
                const int nt = tier + 1;
                const int nxt = (nt & 1) ? nt * G + (G - 1 - (int)blockIdx.x) : nt * G + (int)blockIdx.x;
                if (nxt < n_items) prefetch_item(tb, seq_lo, nxt, H, slots, q, k, v);
            }
        }
        mbar_wait(&m.bar_o, ph_o, status, &m.dead);
        ph_o ^= 1;
        tc_fence_after();
        if (tid == 0 && c + 1 < s.n_chunks) issue_tma(c + 1);   // tiles are free: every MMA that read them is done
        row_code(c + 1, my_code, gval);
        // ---- epilogue: o_t = O1 + e^{b_t} O2, lane = output column j', 32 rows per column half ---------------
        const bool full = !(c == 0 && gather_first) && (c + 1) * BT <= s.n_virtual;
        {
            const int t0 = grp * 32;
            uint32_t x1[32], x2[32];
            tmem_ld32(tm_lane + COL_O1 + t0, x1);
            tmem_ld32(tm_lane + COL_A + t0, x2);
            tmem_ld_wait();
            if (full) {            // all 64 rows are own rows: stage [row][feature] for one TMA store
                float ebt[32];
#pragma unroll
                for (int i4 = 0; i4 < 8; i4++) {
                    float4 e4 = reinterpret_cast<const float4*>(m.eb + t0)[i4];
                    ebt[i4 * 4 + 0] = e4.x;
                    ebt[i4 * 4 + 1] = e4.y;
                    ebt[i4 * 4 + 2] = e4.z;
                    ebt[i4 * 4 + 3] = e4.w;
                }
#pragma unroll
                for (int e = 0; e < 32; e++) {
                    int t = t0 + e;
                    float val = __fmaf_rn(ebt[e], __uint_as_float(x2[e]), __uint_as_float(x1[e]));
                    *reinterpret_cast<__nv_bfloat16*>(sO + t * 256 + L * 2) = __float2bfloat16_rn(val);
                }
                fence_async_smem();
            } else {
#pragma unroll
                for (int e = 0; e < 32; e++) {
                    int t = t0 + e, code = m.code[t];
                    if (code >= 0) {
                        float val = __fmaf_rn(m.eb[t], __uint_as_float(x2[e]), __uint_as_float(x1[e]));
                        o[((size_t)code * H + h) * D + L] = __float2bfloat16_rn(val);
                    }
                }
            }
        }
        if (full) {
            tc_fence_before();
            __syncthreads();                      // (5) staged outputs complete
            if (tid == 0) {
                tma_store_3d(&map_o, sO, 0, h, s.own_begin - s.n_replay + c * BT);
                tma_store_commit();
            }
        }
    }
    if (gave_up) break;
    }   // work items
    if (__syncthreads_or(m.dead) && tid == 0) {   // abandoned: let copies and MMAs in flight finish (bounded)
        if (tma_pending) mbar_wait_drain(&m.bar_tma, ph_tma);
        mma_commit(&m.bar_exit);
        mbar_wait_drain(&m.bar_exit, 0);
    }
    if (tid == 0) tma_store_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc<TMEM_COLS>(tmem);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// [rows][H][128] bf16 tensor, box = 64 rows x 1 head x 64 columns
int32_t make_row_map(CUtensorMap* map, const void* base, int64_t rows, int32_t H) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HARTS_ECUDA;
    cuuint64_t dims[3] = {128, (cuuint64_t)H, (cuuint64_t)rows};
    cuuint64_t strides[2] = {256, (cuuint64_t)H * 256};
    cuuint32_t box[3] = {64, 1, 64}, es[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HARTS_OK : HARTS_ECUDA;
}

// [n][128][128] bf16 states, box = 1 state x 128 rows x 64 columns
int32_t make_state_map(CUtensorMap* map, const void* base, int64_t n) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HARTS_ECUDA;
    cuuint64_t dims[3] = {128, 128, (cuuint64_t)(n < 1 ? 1 : n)};
    cuuint64_t strides[2] = {256, 32768};
    cuuint32_t box[3] = {64, 128, 1}, es[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HARTS_OK : HARTS_ECUDA;
}

// [rows][H][128] bf16 output tensor, box = 64 rows x 1 head x 128 columns, plain (unswizzled) rows
int32_t make_out_map(CUtensorMap* map, const void* base, int64_t rows, int32_t H) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return HARTS_ECUDA;
    cuuint64_t dims[3] = {128, (cuuint64_t)H, (cuuint64_t)rows};
    cuuint64_t strides[2] = {256, (cuuint64_t)H * 256};
    cuuint32_t box[3] = {128, 1, 64}, es[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? HARTS_OK : HARTS_ECUDA;
}

int sm_count() {
    static int n = [] {
        int dev = 0, v = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v < 1)
            v = 148;
        return v;
    }();
    return n;
}

int32_t tc_supported(int32_t dtype, int32_t dk, int32_t dv) { return dtype == HARTS_BF16 && dk == 128 && dv == 128; }

int32_t tc_fwd(const FwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    CUtensorMap mq, mk, mv, mcs, mo;
    int32_t rc;
    if ((rc = make_row_map(&mq, a.q, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, a.k, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, a.v, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    const void* cs = a.chunk_states ? a.chunk_states : a.q;   // a valid address for the (unused) map
    if ((rc = make_state_map(&mcs, cs, a.chunk_states ? (int64_t)a.tb.n_chunks * a.H : 1)) != HARTS_OK) return rc;
    if ((rc = make_out_map(&mo, a.o, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(tc_fwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    int n = (a.seq_hi - a.seq_lo) * a.H;
    int grid = n < 2 * sm_count() ? n : 2 * sm_count();
    tc_fwd_kernel<false><<<grid, NT, Smem::bytes + 1024, a.stream>>>(
        a.tb, a.seq_lo, n, a.H, mq, mk, mv, mcs, mo, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
        (const __nv_bfloat16*)a.v, a.g, (__nv_bfloat16*)a.o, a.slots, a.chunk_states != nullptr, a.dev_status,
        status_gate(a.flags, a.dev_status), nullptr, nullptr);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}


// All rounds of a plan in ONE launch: sequences [seq_lo, seq_hi) span several rounds (they are numbered round by
// round), the persistent CTAs draw the work items in that order from a ticket counter, and a sequence that starts from
// an exported state waits for the flag its producer sets after writing the slot (which it does when it passes the
// boundary, not at its end).  A waiting item's producer sits in an earlier round, so it holds a smaller ticket -- and a
// ticket is only ever held by a CTA that is running: the producer is running or done whether or not every CTA of the
// grid is resident, so an ordinary launch cannot deadlock (a CTA that is not yet resident holds no ticket and nobody
// waits for it).  Which CTA computes an item does not change its arithmetic: the results equal those of one launch
// per round bit for bit.  `flags`: caller-owned DEVICE array of n_slots * H int32, `ticket`: one int32; both zeroed
// here on the stream.
int32_t tc_fwd_fused(const FwdArgs& a, int* flags, int* ticket) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    CUtensorMap mq, mk, mv, mcs, mo;
    int32_t rc;
    if ((rc = make_row_map(&mq, a.q, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, a.k, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, a.v, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    const void* cs = a.chunk_states ? a.chunk_states : a.q;
    if ((rc = make_state_map(&mcs, cs, a.chunk_states ? (int64_t)a.tb.n_chunks * a.H : 1)) != HARTS_OK) return rc;
    if ((rc = make_out_map(&mo, a.o, a.tb.n_rows, a.H)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(tc_fwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    // Offered while a CTA gets few items (at most ONE_LAUNCH_ITEMS_PER_CTA on average): there the idle tail of every
    // round, about one item long, is what one launch saves (cfg1, one item per CTA: forward 0.38 -> 0.26 ms; cfg2, 3.7
    // items per CTA: 1.24 -> 1.03 ms).  With many items per CTA nothing is left to gain (cfg3, 28 items per CTA: 5.98
    // against 6.03 ms) and the per-item flag traffic costs (cfg4, 900 short items per CTA: 16.7 against 18.0 ms).
    if ((int64_t)(a.seq_hi - a.seq_lo) * a.H > (int64_t)ONE_LAUNCH_ITEMS_PER_CTA * 2 * sm_count()) return HARTS_EUNSUPPORTED;
    if (a.tb.n_slots > 0 &&
        cudaMemsetAsync(flags, 0, (size_t)a.tb.n_slots * a.H * sizeof(int), a.stream) != cudaSuccess)
        return HARTS_ECUDA;
    if (cudaMemsetAsync(ticket, 0, sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    int n = (a.seq_hi - a.seq_lo) * a.H;
    int grid = n < 2 * sm_count() ? n : 2 * sm_count();
    tc_fwd_kernel<true><<<grid, NT, Smem::bytes + 1024, a.stream>>>(
        a.tb, a.seq_lo, n, a.H, mq, mk, mv, mcs, mo, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k,
        (const __nv_bfloat16*)a.v, a.g, (__nv_bfloat16*)a.o, a.slots, a.chunk_states != nullptr, a.dev_status,
        status_gate(a.flags, a.dev_status), flags, ticket);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
