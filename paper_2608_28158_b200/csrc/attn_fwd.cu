// Forward of full attention on compact tokens (Section 3.4, Eqs. 21-22) for bf16, head dimension 128, on tcgen05.
//
// One work item = (piece, tile of 128 query rows, query head).  The CTA walks the key/value rows that tile sees --
// the piece's ancestor rows (all visible), then the piece's own rows up to the diagonal (Eq. 22) -- in tiles of 64:
//     S = Q K^T            tcgen05.mma, operands in shared memory (TMA, 128-byte swizzle), S in tensor memory
//     P = exp2(S - m)      four warps, one query row per thread; P goes back to tensor memory as bf16 over S
//     O += P V             tcgen05.mma with P as the tensor-memory operand
// with the running maximum m raised only when a row's maximum grows by more than 2^8 (the values of P stay
// representable and O is rescaled rarely).  K/V tiles are double-buffered; two CTAs share an SM, so one CTA's
// softmax overlaps the other's MMAs.  Every wait is bounded.
#include "kernels.h"
#include "tc_common.cuh"

#include "../../include/harts_attn.h"
#include "attn_common.cuh"

namespace harts {

int32_t make_row_map(CUtensorMap* map, const void* base, int64_t rows, int32_t H);
int sm_count();

namespace {

using namespace tc;

using namespace attn;
constexpr int NS = 128;                 // softmax threads (4 warps), thread = query row = tensor-memory lane
constexpr int NT = NS + 64;             // plus one warp whose first lane issues the MMAs and one whose first lane issues the TMA loads
constexpr int Q_BYTES = BQ * D * 2;     // 32 KB: two panels [128 rows][64 columns]
constexpr int KV_BYTES = BK * D * 2;    // 16 KB: two panels [64 rows][64 columns]
constexpr int COL_S = 0, COL_O = 128, TMEM_COLS = 256;     // S / P of tile n at COL_S + 64 (n & 1)
constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
constexpr float RAISE = 8.f;            // the reference maximum follows the row maximum in steps of at least 2^8

struct Smem {
    static constexpr int q = 0, k0 = Q_BYTES, v0 = k0 + 2 * KV_BYTES, misc = v0 + 2 * KV_BYTES;
    static constexpr int bytes = misc + 256;
};
struct Misc {
    uint64_t bar_q, bar_k[2], bar_v[2], bar_kfree[2], bar_vfree[2], bar_s[2], bar_p[2], bar_pv, bar_o, bar_exit;
    int dead;        // latch: a wait of this CTA ran out, the CTA is abandoning its work
    uint32_t tmem;
};

__global__ void __launch_bounds__(NT, 2)
attn_fwd_kernel(Index ix, int Hq, int G, float scale_log2, const __grid_constant__ CUtensorMap map_q,
                const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                const __grid_constant__ CUtensorMap map_o, __nv_bfloat16* __restrict__ o, float* __restrict__ lse,
                int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    unsigned char* sQ = smem + Smem::q;
    Misc& m = *reinterpret_cast<Misc*>(smem + Smem::misc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_softmax = warp < NS / 32;
    const bool is_issuer = tid == NS, is_producer = tid == NS + 32;

    if (tid == 0) {
        mbar_init(&m.bar_q, 1);
        for (int st = 0; st < 2; st++) {
            mbar_init(&m.bar_k[st], 1);
            mbar_init(&m.bar_v[st], 1);
            mbar_init(&m.bar_kfree[st], 1);
            mbar_init(&m.bar_vfree[st], 1);
        }
        mbar_init(&m.bar_s[0], 1);
        mbar_init(&m.bar_s[1], 1);
        mbar_init(&m.bar_p[0], NS / 32);
        mbar_init(&m.bar_p[1], NS / 32);
        mbar_init(&m.bar_pv, 1);
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

    constexpr uint32_t I_S = instr_desc(BQ, BK, 0, 0);      // S[128 x 64] = Q (K-major) . K (K-major)
    constexpr uint32_t I_O = instr_desc(BQ, D, 0, 1);       // O[128 x 128] += P (tensor memory) . V (rows = keys)
    const uint32_t aQ = smem_u32(sQ);
    const uint64_t dQ = desc_kmajor_base(aQ);

    uint32_t tiles_done = 0;                     // key tiles this CTA has processed (the phase index of bar_pv)
    uint32_t ph_q = 0, ph_k[2] = {0, 0}, ph_v[2] = {0, 0}, ph_kfree[2] = {0, 0}, ph_vfree[2] = {0, 0}, ph_s[2] = {0, 0},
             ph_p[2] = {0, 0}, ph_o = 0;
    const int n_work = ix.n_q_items * Hq;
    // work items come most work first; dealt in a snake pattern (tier by tier, every second tier in reverse), so that no
    // CTA gets the largest item of every tier
    for (int tier = 0; tier * (int)gridDim.x < n_work; tier++) {
        const int w = tier * (int)gridDim.x + ((tier & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x);
        if (w >= n_work) continue;
        const int item = w / Hq, h = w % Hq, hk = h / G;
        const int piece = ix.q_item[2 * item], qt = ix.q_item[2 * item + 1];
        const int q_row0 = ix.piece_row0[piece] + qt * BQ;
        const int q_valid = min(BQ, ix.piece_len[piece] - qt * BQ);

        if (is_producer) {
            // ---- TMA producer: the Q tile, then the key/value tiles two stages deep ---------------------------------
            TileWalk lw(ix, piece, qt);
            KvTile lt;
            mbar_expect_tx(&m.bar_q, Q_BYTES);
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++)
                    tma_load_3d(sQ + p * (Q_BYTES / 2) + r * (Q_BYTES / 4), &map_q, p * 64, h, q_row0 + r * 64, &m.bar_q);
            for (int n = 0; lw.next(lt); n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int stage = n & 1;
                unsigned char* sK = smem + Smem::k0 + stage * KV_BYTES;
                unsigned char* sV = smem + Smem::v0 + stage * KV_BYTES;
                // the K tile of a stage is free as soon as S of its previous tile is done, the V tile only after P V
                if (n >= 2) {
                    mbar_wait(&m.bar_kfree[stage], ph_kfree[stage], status, &m.dead);
                    ph_kfree[stage] ^= 1;
                }
                mbar_expect_tx(&m.bar_k[stage], KV_BYTES);
                for (int p = 0; p < 2; p++)
                    tma_load_3d(sK + p * (KV_BYTES / 2), &map_k, p * 64, hk, lt.row, &m.bar_k[stage]);
                if (n >= 2) {
                    mbar_wait(&m.bar_vfree[stage], ph_vfree[stage], status, &m.dead);
                    ph_vfree[stage] ^= 1;
                }
                mbar_expect_tx(&m.bar_v[stage], KV_BYTES);
                for (int p = 0; p < 2; p++)
                    tma_load_3d(sV + p * (KV_BYTES / 2), &map_v, p * 64, hk, lt.row, &m.bar_v[stage]);
            }
        }
        if (is_issuer) {
            // ---- MMA issue: this thread does nothing else, a tcgen05.mma holds it until the pipe has room ---------
            const int n_tiles = TileWalk(ix, piece, qt).count();
            auto issue_s = [&](int n) {                     // S(n) into buffer n & 1, from stage n & 1
                const int stage = n & 1;
                mbar_wait(&m.bar_k[stage], ph_k[stage], status, &m.dead);
                ph_k[stage] ^= 1;
                tc_fence_after();
                const uint64_t dK = desc_kmajor_base(smem_u32(smem + Smem::k0 + stage * KV_BYTES));
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ss(tmem + COL_S + stage * 64, dQ + kstep_kmajor<BQ>(ks), dK + kstep_kmajor<BK>(ks), I_S, ks > 0);
                mma_commit(&m.bar_s[stage]);
                if (n + 2 < n_tiles) mma_commit(&m.bar_kfree[stage]);     // the K tile will be refilled
            };
            mbar_wait(&m.bar_q, ph_q, status, &m.dead);
            ph_q ^= 1;
            issue_s(0);
            for (int n = 0; n < n_tiles; n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int stage = n & 1;
                // S of tile n+1 goes to the other buffer and runs under the softmax of tile n (its K stage was freed
                // by the P V MMAs of tile n-1, which precede it in the pipe)
                if (n + 1 < n_tiles) issue_s(n + 1);
                // O += P V for tile n as soon as the softmax warps have written P.  One barrier per S buffer: a warp that
                // is done with tile n may already work on tile n+1 (its S is complete) and arrive for it, and that
                // arrival must not count for tile n.
                mbar_wait(&m.bar_p[stage], ph_p[stage], status, &m.dead);
                ph_p[stage] ^= 1;
                mbar_wait(&m.bar_v[stage], ph_v[stage], status, &m.dead);
                ph_v[stage] ^= 1;
                tc_fence_after();
                const uint64_t dV = desc_mnmajor_base<BK>(smem_u32(smem + Smem::v0 + stage * KV_BYTES));
#pragma unroll
                for (int ks = 0; ks < 4; ks++)
                    mma_ts(tmem + COL_O, tmem + COL_S + stage * 64 + ks * 8, dV + kstep_mnmajor(ks), I_O, n > 0 || ks > 0);
                mma_commit(&m.bar_pv);                                    // one phase per tile, in order
                if (n + 2 < n_tiles) mma_commit(&m.bar_vfree[stage]);     // the V tile will be refilled
                if (n + 1 == n_tiles) mma_commit(&m.bar_o);
            }
        }

        float m_ref = -INFINITY, l_sum = 0.f;
        if (is_softmax) {
            TileWalk walk(ix, piece, qt);
            KvTile t;
            const int i = tid;                                // query row inside the tile
            int n = 0;
            while (walk.next(t)) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int b = n & 1;
                mbar_wait_warp(&m.bar_s[b], ph_s[b], status, &m.dead);
                ph_s[b] ^= 1;
                tc_fence_after();
                const int limit = min(t.n_valid, t.shift == NO_DIAG ? BK : i - t.shift + 1);   // visible: j < limit
                // the whole row of S in registers; hidden columns become -inf (exp2 gives 0), only in tiles that have some
                uint32_t x[BK];
                tmem_ld32(tm_lane + COL_S + b * 64, x);
                tmem_ld32(tm_lane + COL_S + b * 64 + 32, x + 32);
                tmem_ld_wait();
                if (!__all_sync(0xffffffffu, limit >= BK)) {
#pragma unroll
                    for (int e = 0; e < BK; e++)
                        if (e >= limit) x[e] = __float_as_uint(-INFINITY);
                }
                // row maximum (three-input max: 32 instructions for 64 values)
                float mx = __uint_as_float(x[0]);
#pragma unroll
                for (int e = 1; e + 1 < BK; e += 2) mx = max3(mx, __uint_as_float(x[e]), __uint_as_float(x[e + 1]));
                mx = fmaxf(mx, __uint_as_float(x[BK - 1])) * scale_log2;
                // raise the reference only by big steps; the whole warp decides together whether O must be rescaled
                const bool raise = mx > m_ref + RAISE || m_ref == -INFINITY;
                if (__any_sync(0xffffffffu, raise && n > 0)) {
                    // O is about to be read and rewritten: the P V MMAs of the previous tile must be done.  S of this tile
                    // was issued before them (it has its own buffer), so its completion does not say so; bar_pv does.  Its
                    // phase index is the running tile count; this warp is never more than one phase behind (P V of this tile
                    // cannot be issued before this warp arrives on bar_p), so the parity alone identifies the phase.
                    mbar_wait_warp(&m.bar_pv, (tiles_done - 1) & 1, status, &m.dead);
                    tc_fence_after();
                    const float m_new = raise ? mx : m_ref;
                    const float alpha = m_new == -INFINITY ? 1.f : ex2(m_ref - m_new);   // m_ref = -inf: O and l are still 0
                    l_sum *= alpha;
#pragma unroll
                    for (int c = 0; c < 4; c++) {
                        uint32_t y[32];
                        tmem_ld32(tm_lane + COL_O + c * 32, y);
                        tmem_ld_wait();
#pragma unroll
                        for (int e = 0; e < 32; e++) y[e] = __float_as_uint(__uint_as_float(y[e]) * alpha);
                        tmem_st32(tm_lane + COL_O + c * 32, y);
                    }
                    m_ref = m_new;
                } else if (raise) {
                    m_ref = mx;                               // first tile: nothing accumulated yet
                }
                // P = exp2(s - m_ref), written over S as bf16 pairs; four independent partial sums
                const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
                float part[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int c = 0; c < 2; c++) {
                    uint32_t pk[16];
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        const float p0 = ex2(fmaf(__uint_as_float(x[c * 32 + e]), scale_log2, neg_m));
                        const float p1 = ex2(fmaf(__uint_as_float(x[c * 32 + e + 1]), scale_log2, neg_m));
                        pk[e >> 1] = pack_bf16(p0, p1);
                        part[(e >> 1) & 3] += p0 + p1;
                    }
                    tmem_st16(tm_lane + COL_S + b * 64 + c * 16, pk);
                }
                l_sum += (part[0] + part[1]) + (part[2] + part[3]);
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&m.bar_p[b]);
                n++;
                tiles_done++;
            }
            // ---- epilogue: O / l -> bf16, lse ----------------------------------------------------------------------
            mbar_wait_warp(&m.bar_o, ph_o, status, &m.dead);
            tc_fence_after();
            const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
            const bool full = q_valid == BQ;
            if (i < q_valid) lse[(size_t)(q_row0 + i) * Hq + h] = (m_ref + log2f(l_sum)) * LN2;
#pragma unroll
            for (int c = 0; c < 4; c++) {
                uint32_t x[32];
                tmem_ld32(tm_lane + COL_O + c * 32, x);
                tmem_ld_wait();
#pragma unroll
                for (int v4 = 0; v4 < 4; v4++) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(x[v4 * 8 + 0]) * inv, __uint_as_float(x[v4 * 8 + 1]) * inv);
                    pk.y = pack_bf16(__uint_as_float(x[v4 * 8 + 2]) * inv, __uint_as_float(x[v4 * 8 + 3]) * inv);
                    pk.z = pack_bf16(__uint_as_float(x[v4 * 8 + 4]) * inv, __uint_as_float(x[v4 * 8 + 5]) * inv);
                    pk.w = pack_bf16(__uint_as_float(x[v4 * 8 + 6]) * inv, __uint_as_float(x[v4 * 8 + 7]) * inv);
                    const int col = c * 32 + v4 * 8;
                    if (full)       // staged over the Q tile in the swizzled panel layout, for TMA stores
                        *reinterpret_cast<uint4*>(sQ + (col >> 6) * (Q_BYTES / 2) + sw128_chunk(i, (col & 63) >> 3)) = pk;
                    else if (i < q_valid)
                        *reinterpret_cast<uint4*>(o + ((size_t)(q_row0 + i) * Hq + h) * D + col) = pk;
                }
            }
            if (full) fence_async_smem();
        }
        ph_o ^= 1;
        tc_fence_before();
        if (__syncthreads_or(m.dead)) break;                                      // O staged; tensor memory and Q tile free for the next item
        tc_fence_after();
        if (is_issuer && q_valid == BQ) {
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++)
                    tma_store_3d(&map_o, sQ + p * (Q_BYTES / 2) + r * (Q_BYTES / 4), p * 64, h, q_row0 + r * 64);
            tma_store_commit();
            tma_store_wait_read();                            // the Q tile is reloaded right away
        }
        __syncthreads();
    }
    if (__syncthreads_or(m.dead)) {               // abandoned: let the loads and MMAs in flight finish (bounded)
        if (is_issuer) {
            mma_commit(&m.bar_exit);
            mbar_wait_drain(&m.bar_exit, 0);
        }
        drain_delay();
    }
    if (is_issuer) tma_store_wait_all();
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc<TMEM_COLS>(tmem);
}

}  // namespace

int32_t attn_index_ok(const int32_t* host_index) {
    return host_index && host_index[0] >= 0 && host_index[6] >= HARTS_ATTN_HEADER_WORDS ? HARTS_OK : HARTS_EINVAL;
}

int32_t attn_fwd_launch(const int32_t* hi, const int32_t* di, const void* q, const void* k, const void* v, void* o,
                        float* lse, int Hq, int Hkv, float scale, int32_t* status, cudaStream_t st) {
    const int n_rows = hi[0];
    if (n_rows == 0 || hi[4] == 0) return HARTS_OK;
    CUtensorMap mq, mk, mv, mo;
    int32_t rc;
    if ((rc = make_row_map(&mq, q, n_rows, Hq)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, k, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, v, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mo, o, n_rows, Hq)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(attn_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const Index ix = make_index(hi, di);
    const long long n_work = (long long)ix.n_q_items * Hq;
    const int grid = (int)(n_work < 2LL * sm_count() ? n_work : 2LL * sm_count());
    attn_fwd_kernel<<<grid, NT, Smem::bytes + 1024, st>>>(ix, Hq, Hq / Hkv, scale * LOG2E, mq, mk, mv, mo,
                                                         (__nv_bfloat16*)o, lse, status);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
