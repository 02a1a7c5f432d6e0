// dK / dV of attention on compact tokens (Section 3.4: the ancestor-KV gather's backward sums every consumer into the
// ancestor's unique compact activation) for bf16, head dimension 128, on tcgen05.
//
// One work item = (piece, tile of 128 key rows, kv head).  Key rows sit on the tensor-memory lanes; the CTA keeps the
// K and V tiles in shared memory and streams every query tile (64 rows) that sees them: the rest of the key tile's
// own piece (causal inside the tile, Eq. 22), then all rows of all descendant pieces, for each query head of the GQA
// group.  Per query tile:
//     S^T = K Q^T,  dP^T = V dO^T            operands in shared memory, results in tensor memory
//     P^T = exp2(S^T - lse_q),  dS^T = P^T (dP^T - delta_q)     one key row per thread; bf16 back over S^T / dP^T
//     dV += P^T dO,  dK += dS^T Q            A operand from tensor memory, Q / dO tiles read row-major as B
// dK and dV of the tile are complete when the walk ends and are written once.  Every wait is bounded.
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

constexpr int NS = 256, NT = NS + 64;     // 8 element-wise warps: warp w and w + 4 share a lane quarter and split the columns
constexpr int BKV = 128, BQT = 64;
constexpr int KV_TILE = BKV * D * 2;      // 32 KB: two panels [128 rows][64 columns]
constexpr int Q_TILE = BQT * D * 2;       // 16 KB: two panels [64 rows][64 columns]
constexpr int STAGES = 4;
constexpr float LOG2E = 1.4426950408889634f;
constexpr int COL_DV = 256, COL_DK = 384, TMEM_COLS = 512;   // S^T at 128 b, dP^T at 128 b + 64

struct Smem {
    static constexpr int k = 0, v = KV_TILE, q0 = 2 * KV_TILE, do0 = q0 + STAGES * Q_TILE, vec = do0 + STAGES * Q_TILE,
                         misc = vec + 2 * 2 * BQT * 4;
    static constexpr int bytes = misc + 256;
};
struct Misc {
    uint64_t bar_kv, bar_q[STAGES], bar_s[2], bar_p[2], bar_free[STAGES], bar_o, bar_exit;
    int dead;        // latch: a wait of this CTA ran out, the CTA is abandoning its work
    uint32_t tmem;
};

__global__ void __launch_bounds__(NT, 1)
attn_dkv_kernel(Index ix, int Hq, int Hkv, int G, float scale, const __grid_constant__ CUtensorMap map_q,
                const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_k,
                const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_dk,
                const __grid_constant__ CUtensorMap map_dv, const float* __restrict__ lse,
                const float* __restrict__ delta, __nv_bfloat16* __restrict__ dk_, __nv_bfloat16* __restrict__ dv_,
                int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    unsigned char* sK = smem + Smem::k;
    unsigned char* sV = smem + Smem::v;
    float* sVec = reinterpret_cast<float*>(smem + Smem::vec);       // [2 buffers][lse2 | delta][64]
    Misc& m = *reinterpret_cast<Misc*>(smem + Smem::misc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_softmax = warp < NS / 32, is_issuer = tid == NS, is_producer = tid == NS + 32;
    if (tid == 0) {
        mbar_init(&m.bar_kv, 1);
        for (int s = 0; s < STAGES; s++) { mbar_init(&m.bar_q[s], 1); mbar_init(&m.bar_free[s], 1); }
        for (int b = 0; b < 2; b++) { mbar_init(&m.bar_s[b], 1); mbar_init(&m.bar_p[b], NS / 32); }
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
    constexpr uint32_t I_ST = instr_desc(BKV, BQT, 0, 0);   // [128 keys x 64 queries] = (K | V) . (Q | dO), all K-major
    constexpr uint32_t I_ACC = instr_desc(BKV, D, 0, 1);    // [128 keys x 128] += (P^T | dS^T) (tensor memory) . (dO | Q)
    const uint64_t dKd = desc_kmajor_base(smem_u32(sK)), dVd = desc_kmajor_base(smem_u32(sV));
    const float scale_log2 = scale * LOG2E;

    uint32_t ph_kv = 0, ph_q[STAGES] = {}, ph_free[STAGES] = {}, ph_s[2] = {0, 0}, ph_p[2] = {0, 0}, ph_o = 0;
    const int n_work = ix.n_kv_items * Hkv;
    // work items come most work first; dealt in a snake pattern (tier by tier, every second tier in reverse), so that no
    // CTA gets the largest item of every tier
    for (int tier = 0; tier * (int)gridDim.x < n_work; tier++) {
        const int w = tier * (int)gridDim.x + ((tier & 1) ? (int)gridDim.x - 1 - (int)blockIdx.x : (int)blockIdx.x);
        if (w >= n_work) continue;
        const int item = w / Hkv, hk = w % Hkv;
        const int piece = ix.kv_item[2 * item], kt = ix.kv_item[2 * item + 1];
        const int kv_row0 = ix.piece_row0[piece] + kt * BKV;
        const int kv_valid = min(BKV, ix.piece_len[piece] - kt * BKV);

        if (is_producer) {
            // ---- TMA producer: the K and V tiles, then the query / dO tiles STAGES deep -----------------------------
            QWalk lw(ix, piece, kt, hk, G);
            QTile lt;
            mbar_expect_tx(&m.bar_kv, 2 * KV_TILE);
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++) {
                    tma_load_3d(sK + p * (KV_TILE / 2) + r * (KV_TILE / 4), &map_k, p * 64, hk, kv_row0 + r * 64, &m.bar_kv);
                    tma_load_3d(sV + p * (KV_TILE / 2) + r * (KV_TILE / 4), &map_v, p * 64, hk, kv_row0 + r * 64, &m.bar_kv);
                }
            for (int n = 0; lw.next(lt); n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int stage = n % STAGES;
                if (n >= STAGES) {
                    mbar_wait(&m.bar_free[stage], ph_free[stage], status, &m.dead);
                    ph_free[stage] ^= 1;
                }
                unsigned char* sQ = smem + Smem::q0 + stage * Q_TILE;
                unsigned char* sDO = smem + Smem::do0 + stage * Q_TILE;
                mbar_expect_tx(&m.bar_q[stage], 2 * Q_TILE);
                for (int p = 0; p < 2; p++) {
                    tma_load_3d(sQ + p * (Q_TILE / 2), &map_q, p * 64, lt.head, lt.row, &m.bar_q[stage]);
                    tma_load_3d(sDO + p * (Q_TILE / 2), &map_do, p * 64, lt.head, lt.row, &m.bar_q[stage]);
                }
            }
        }
        if (is_issuer) {
            // ---- MMA issue: this thread does nothing else, a tcgen05.mma holds it until the pipe has room ---------
            const int n_tiles = QWalk(ix, piece, kt, hk, G).count();
            auto issue_s = [&](int n) {      // S^T(n), dP^T(n) into buffer n & 1
                const int stage = n % STAGES, b = n & 1;
                mbar_wait(&m.bar_q[stage], ph_q[stage], status, &m.dead);
                ph_q[stage] ^= 1;
                tc_fence_after();
                const uint64_t dQ = desc_kmajor_base(smem_u32(smem + Smem::q0 + stage * Q_TILE));
                const uint64_t dDO = desc_kmajor_base(smem_u32(smem + Smem::do0 + stage * Q_TILE));
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ss(tmem + b * 128, dKd + kstep_kmajor<BKV>(ks), dQ + kstep_kmajor<BQT>(ks), I_ST, ks > 0);
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ss(tmem + b * 128 + 64, dVd + kstep_kmajor<BKV>(ks), dDO + kstep_kmajor<BQT>(ks), I_ST, ks > 0);
                mma_commit(&m.bar_s[b]);
            };
            mbar_wait(&m.bar_kv, ph_kv, status, &m.dead);
            ph_kv ^= 1;
            issue_s(0);
            for (int n = 0; n < n_tiles; n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                if (n + 1 < n_tiles) issue_s(n + 1);
                const int stage = n % STAGES, b = n & 1;
                mbar_wait(&m.bar_p[b], ph_p[b], status, &m.dead);
                ph_p[b] ^= 1;
                tc_fence_after();
                const uint64_t dDOm = desc_mnmajor_base<BQT>(smem_u32(smem + Smem::do0 + stage * Q_TILE));
                const uint64_t dQm = desc_mnmajor_base<BQT>(smem_u32(smem + Smem::q0 + stage * Q_TILE));
#pragma unroll
                for (int ks = 0; ks < 4; ks++)
                    mma_ts(tmem + COL_DV, tmem + b * 128 + (ks >> 1) * 32 + (ks & 1) * 8, dDOm + kstep_mnmajor(ks), I_ACC, n > 0 || ks > 0);
#pragma unroll
                for (int ks = 0; ks < 4; ks++)
                    mma_ts(tmem + COL_DK, tmem + b * 128 + 64 + (ks >> 1) * 32 + (ks & 1) * 8, dQm + kstep_mnmajor(ks), I_ACC, n > 0 || ks > 0);
                if (n + STAGES < n_tiles) mma_commit(&m.bar_free[stage]);
                if (n + 1 == n_tiles) mma_commit(&m.bar_o);
            }
        }
        if (is_softmax) {
            QWalk walk(ix, piece, kt, hk, G), ahead(ix, piece, kt, hk, G);
            QTile t, ta;
            const int i = tid & 127, c = tid >> 7;             // key row inside the tile, and which 32 of the 64 query columns
            const bool row_ok = i < kv_valid;
            // per-column lse (log2 units) and delta of a query tile: thread j < 64 fetches lse, thread 64 + j delta;
            // fetched one tile ahead, handed over through shared memory
            auto fetch = [&](const QTile& qt) -> float {              // threads 0..127 only
                const int j = tid & 63;
                if (tid >= 128) return 0.f;
                if (j >= qt.n_valid) return tid < 64 ? INFINITY : 0.f;    // columns past the end: probability 0
                const size_t at = (size_t)(qt.row + j) * Hq + qt.head;
                return tid < 64 ? lse[at] * LOG2E : delta[at];
            };
            bool more_ahead = ahead.next(ta);
            float pre = more_ahead ? fetch(ta) : 0.f;
            if (tid < 128) sVec[(tid >> 6) * BQT + (tid & 63)] = pre;            // buffer 0
            asm volatile("bar.sync 1, 256;" ::: "memory");
            for (int n = 0; walk.next(t); n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int b = n & 1;
                more_ahead = more_ahead && ahead.next(ta);
                if (more_ahead) pre = fetch(ta);              // in flight during this tile
                mbar_wait_warp(&m.bar_s[b], ph_s[b], status, &m.dead);
                ph_s[b] ^= 1;
                tc_fence_after();
                const float* vl = sVec + b * 2 * BQT;
                const float* vd = vl + BQT;
                // visible columns of key row i: jmin <= j < n_valid
                const int jmin = !row_ok ? BQT : (t.lead < 0 ? 0 : max(0, i - t.lead));
                {
                    uint32_t xs[32], xp[32], pp[16], pd[16];
                    tmem_ld32(tm_lane + b * 128 + c * 32, xs);
                    tmem_ld32(tm_lane + b * 128 + 64 + c * 32, xp);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; e += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(vl + c * 32 + e);
                        const float4 d4 = *reinterpret_cast<const float4*>(vd + c * 32 + e);
                        const float ls[4] = {l4.x, l4.y, l4.z, l4.w}, dl[4] = {d4.x, d4.y, d4.z, d4.w};
                        float p[4], ds[4];
#pragma unroll
                        for (int u = 0; u < 4; u++) {
                            const int j = c * 32 + e + u;
                            p[u] = j >= jmin ? ex2(fmaf(__uint_as_float(xs[e + u]), scale_log2, -ls[u])) : 0.f;
                            ds[u] = p[u] * (__uint_as_float(xp[e + u]) - dl[u]) * scale;
                        }
                        pp[e >> 1] = pack_bf16(p[0], p[1]);
                        pp[(e >> 1) + 1] = pack_bf16(p[2], p[3]);
                        pd[e >> 1] = pack_bf16(ds[0], ds[1]);
                        pd[(e >> 1) + 1] = pack_bf16(ds[2], ds[3]);
                    }
                    tmem_st16(tm_lane + b * 128 + c * 32, pp);          // over this warp's own half (the other warp may still read its half)
                    tmem_st16(tm_lane + b * 128 + 64 + c * 32, pd);
                }
                tmem_st_wait();
                tc_fence_before();
                if (more_ahead && tid < 128) sVec[((b ^ 1) * 2 + (tid >> 6)) * BQT + (tid & 63)] = pre;
                asm volatile("bar.sync 1, 256;" ::: "memory");      // next tile's vectors visible; this tile's reads done
                if (lane == 0) mbar_arrive(&m.bar_p[b]);
            }
            // ---- epilogue: dV, dK -> bf16 ---------------------------------------------------------------------------
            mbar_wait_warp(&m.bar_o, ph_o, status, &m.dead);
            tc_fence_after();
            const bool full = kv_valid == BKV;
#pragma unroll
            for (int which = 0; which < 2; which++) {
                unsigned char* stage_buf = which ? sK : sV;              // the K / V tiles are no longer needed
                __nv_bfloat16* out = which ? dk_ : dv_;
#pragma unroll
                for (int cc = 0; cc < 2; cc++) {
                    const int c4 = c * 2 + cc;
                    uint32_t x[32];
                    tmem_ld32(tm_lane + (which ? COL_DK : COL_DV) + c4 * 32, x);
                    tmem_ld_wait();
#pragma unroll
                    for (int v4 = 0; v4 < 4; v4++) {
                        uint4 pk;
                        pk.x = pack_bf16(__uint_as_float(x[v4 * 8 + 0]), __uint_as_float(x[v4 * 8 + 1]));
                        pk.y = pack_bf16(__uint_as_float(x[v4 * 8 + 2]), __uint_as_float(x[v4 * 8 + 3]));
                        pk.z = pack_bf16(__uint_as_float(x[v4 * 8 + 4]), __uint_as_float(x[v4 * 8 + 5]));
                        pk.w = pack_bf16(__uint_as_float(x[v4 * 8 + 6]), __uint_as_float(x[v4 * 8 + 7]));
                        const int col = c4 * 32 + v4 * 8;
                        if (full)
                            *reinterpret_cast<uint4*>(stage_buf + (col >> 6) * (KV_TILE / 2) + sw128_chunk(i, (col & 63) >> 3)) = pk;
                        else if (row_ok)
                            *reinterpret_cast<uint4*>(out + ((size_t)(kv_row0 + i) * Hkv + hk) * D + col) = pk;
                    }
                }
            }
            if (full) fence_async_smem();
        }
        ph_o ^= 1;
        tc_fence_before();
        if (__syncthreads_or(m.dead)) break;
        tc_fence_after();
        if (is_issuer && kv_valid == BKV) {
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++) {
                    tma_store_3d(&map_dv, sV + p * (KV_TILE / 2) + r * (KV_TILE / 4), p * 64, hk, kv_row0 + r * 64);
                    tma_store_3d(&map_dk, sK + p * (KV_TILE / 2) + r * (KV_TILE / 4), p * 64, hk, kv_row0 + r * 64);
                }
            tma_store_commit();
            tma_store_wait_read();
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

int32_t attn_dkv_launch(const Index& ix, int n_rows, const void* q, const void* k, const void* v, const float* lse,
                        const void* dO, const float* delta, void* dk_, void* dv_, int Hq, int Hkv, float scale,
                        int32_t* status, cudaStream_t st) {
    CUtensorMap mq, mdo, mk, mv, mdk, mdv;
    int32_t rc;
    if ((rc = make_row_map(&mq, q, n_rows, Hq)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdo, dO, n_rows, Hq)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, k, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, v, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdk, dk_, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdv, dv_, n_rows, Hkv)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(attn_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Smem::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const long long n_work = (long long)ix.n_kv_items * Hkv;
    const int grid = (int)(n_work < sm_count() ? n_work : sm_count());
    attn_dkv_kernel<<<grid, NT, Smem::bytes + 1024, st>>>(ix, Hq, Hkv, Hq / Hkv, scale, mq, mdo, mk, mv, mdk, mdv, lse,
                                                          delta, (__nv_bfloat16*)dk_, (__nv_bfloat16*)dv_, status);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
