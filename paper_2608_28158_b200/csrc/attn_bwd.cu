// Backward of full attention on compact tokens (Section 3.4, Eqs. 21-22) for bf16, head dimension 128, on tcgen05.
//
// Three kernels, no atomics, fixed summation orders:
//   delta_kernel   delta_t = <dO_t, o_t> per (row, head);
//   dq_kernel      one work item = (piece, tile of 128 query rows, query head); walks the key tiles the queries see,
//                  exactly like the forward:  S = Q K^T,  dP = dO V^T,  P = exp2(S - lse),  dS = P (dP - delta),
//                  dQ += dS K  (dS goes back to tensor memory over S as the A operand);
//   dkv_kernel     one work item = (piece, tile of 128 key rows, kv head); walks every query tile that sees those
//                  keys -- the rest of its own piece (causal) and all rows of all descendant pieces, for every query
//                  head of the group -- with everything transposed so that key rows sit on the tensor-memory lanes:
//                  S^T = K Q^T,  dP^T = V dO^T,  dV += P^T dO,  dK += dS^T Q.
//                  The gradient of a shared ancestor's K/V is thus accumulated on chip over all its descendants and
//                  written once: this replaces the scatter-add of the gather's backward.
// S/dP live in two tensor-memory buffers, so the MMAs of tile n+1 run under the element-wise pass of tile n.
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
constexpr int Q_BYTES = BQ * D * 2;       // 32 KB
constexpr float LOG2E = 1.4426950408889634f;

__global__ void __launch_bounds__(256) delta_kernel(const __nv_bfloat16* __restrict__ o,
                                                    const __nv_bfloat16* __restrict__ dO, float* __restrict__ delta,
                                                    long long n) {       // n = rows * Hq; one warp per (row, head)
    const long long w = (blockIdx.x * 256LL + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= n) return;
    const uint2 a = reinterpret_cast<const uint2*>(o + w * D)[lane], b = reinterpret_cast<const uint2*>(dO + w * D)[lane];
    const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
    const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
    float s = 0.f;
#pragma unroll
    for (int e = 0; e < 2; e++) {
        const float2 x = __bfloat1622float2(pa[e]), y = __bfloat1622float2(pb[e]);
        s = fmaf(x.x, y.x, fmaf(x.y, y.y, s));
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
    if (lane == 0) delta[w] = s;
}

// ------------------------------------------------------------------------------------------------------------------
// dQ: key tiles of 128 rows, so that every MMA has N = 128 (the N = 64 shape is bound by operand reads, not by the
// tensor pipe).  Tensor memory: S in two buffers (S of tile n+1 runs under the element-wise pass of tile n), dP, dQ.
// ------------------------------------------------------------------------------------------------------------------
constexpr int BKW = 128;                       // key rows per tile
constexpr int KW_BYTES = BKW * D * 2;          // 32 KB: two panels [128 rows][64 columns]
constexpr int KST = 3;                         // K stages (a K tile is held from S to dQ); V has two (held for dP only)
struct SmemQ {
    static constexpr int q = 0, dO = Q_BYTES, k0 = 2 * Q_BYTES, v0 = k0 + KST * KW_BYTES, misc = v0 + 2 * KW_BYTES;
    static constexpr int bytes = misc + 256;
};
struct MiscQ {
    uint64_t bar_q, bar_k[KST], bar_v[2], bar_kfree[KST], bar_vfree[2], bar_s, bar_dpfree, bar_p[2], bar_o, bar_exit;
    int dead;        // latch: a wait of this CTA ran out, the CTA is abandoning its work
    uint32_t tmem;
};
constexpr int COL_DP = 256, COL_DQ = 384, TMEM_Q = 512;     // S of tile n at 128 (n & 1)
using WalkW = TileWalkT<BKW>;

__global__ void __launch_bounds__(NT, 1)
attn_dq_kernel(Index ix, int Hq, int G, float scale, const __grid_constant__ CUtensorMap map_q,
               const __grid_constant__ CUtensorMap map_do, const __grid_constant__ CUtensorMap map_k,
               const __grid_constant__ CUtensorMap map_v, const __grid_constant__ CUtensorMap map_dq,
               const float* __restrict__ lse, const float* __restrict__ delta, __nv_bfloat16* __restrict__ dq,
               int* status) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);
    unsigned char* sQ = smem + SmemQ::q;
    unsigned char* sDO = smem + SmemQ::dO;
    MiscQ& m = *reinterpret_cast<MiscQ*>(smem + SmemQ::misc);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool is_softmax = warp < NS / 32, is_issuer = tid == NS, is_producer = tid == NS + 32;
    if (tid == 0) {
        mbar_init(&m.bar_q, 1);
        for (int st = 0; st < KST; st++) {
            mbar_init(&m.bar_k[st], 1);
            mbar_init(&m.bar_kfree[st], 1);
        }
        for (int st = 0; st < 2; st++) {
            mbar_init(&m.bar_v[st], 1);
            mbar_init(&m.bar_vfree[st], 1);
        }
        mbar_init(&m.bar_s, 1);
        mbar_init(&m.bar_dpfree, NS / 32);
        mbar_init(&m.bar_p[0], NS / 32);
        mbar_init(&m.bar_p[1], NS / 32);
        mbar_init(&m.bar_o, 1);
        mbar_init(&m.bar_exit, 1);
        m.dead = 0;
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc<TMEM_Q>(&m.tmem);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = m.tmem;
    const uint32_t tm_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    constexpr uint32_t I_S = instr_desc(BQ, BKW, 0, 0);    // [128 x 128] = (Q | dO) (K-major) . (K | V) (K-major)
    constexpr uint32_t I_DQ = instr_desc(BQ, D, 0, 1);     // dQ[128 x 128] += dS (tensor memory) . K (rows = keys)
    const uint64_t dQd = desc_kmajor_base(smem_u32(sQ)), dDOd = desc_kmajor_base(smem_u32(sDO));
    const float scale_log2 = scale * LOG2E;

    uint32_t ph_q = 0, ph_k[KST] = {}, ph_v[2] = {0, 0}, ph_kfree[KST] = {}, ph_vfree[2] = {0, 0}, ph_s = 0, ph_p[2] = {0, 0},
             ph_dpfree = 0, ph_o = 0;
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
            // ---- TMA producer: Q and dO tiles, then K and V tiles two deep (released separately) --------------------
            WalkW lw(ix, piece, qt);
            KvTile lt;
            mbar_expect_tx(&m.bar_q, 2 * Q_BYTES);
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++) {
                    tma_load_3d(sQ + p * (Q_BYTES / 2) + r * (Q_BYTES / 4), &map_q, p * 64, h, q_row0 + r * 64, &m.bar_q);
                    tma_load_3d(sDO + p * (Q_BYTES / 2) + r * (Q_BYTES / 4), &map_do, p * 64, h, q_row0 + r * 64, &m.bar_q);
                }
            for (int n = 0; lw.next(lt); n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int stage = n & 1, kst = n % KST;
                unsigned char* sK = smem + SmemQ::k0 + kst * KW_BYTES;
                unsigned char* sV = smem + SmemQ::v0 + stage * KW_BYTES;
                if (n >= KST) {
                    mbar_wait(&m.bar_kfree[kst], ph_kfree[kst], status, &m.dead);         // released after dQ of tile n - KST
                    ph_kfree[kst] ^= 1;
                }
                mbar_expect_tx(&m.bar_k[kst], KW_BYTES);
                for (int p = 0; p < 2; p++)
                    for (int r = 0; r < 2; r++)
                        tma_load_3d(sK + p * (KW_BYTES / 2) + r * (KW_BYTES / 4), &map_k, p * 64, hk, lt.row + r * 64, &m.bar_k[kst]);
                if (n >= 2) {
                    mbar_wait(&m.bar_vfree[stage], ph_vfree[stage], status, &m.dead);     // released after dP of tile n - 2
                    ph_vfree[stage] ^= 1;
                }
                mbar_expect_tx(&m.bar_v[stage], KW_BYTES);
                for (int p = 0; p < 2; p++)
                    for (int r = 0; r < 2; r++)
                        tma_load_3d(sV + p * (KW_BYTES / 2) + r * (KW_BYTES / 4), &map_v, p * 64, hk, lt.row + r * 64, &m.bar_v[stage]);
            }
        }
        if (is_issuer) {
            // ---- MMA issue: this thread does nothing else, a tcgen05.mma holds it until the pipe has room ---------
            const int n_tiles = WalkW(ix, piece, qt).count();
            auto issue_s = [&](int n) {      // S(n) into buffer n & 1
                const int stage = n & 1, kst = n % KST;
                mbar_wait(&m.bar_k[kst], ph_k[kst], status, &m.dead);
                ph_k[kst] ^= 1;
                tc_fence_after();
                const uint64_t dK = desc_kmajor_base(smem_u32(smem + SmemQ::k0 + kst * KW_BYTES));
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ss(tmem + stage * 128, dQd + kstep_kmajor<BQ>(ks), dK + kstep_kmajor<BKW>(ks), I_S, ks > 0);
            };
            auto issue_dp = [&](int n) {     // dP(n); its commit also covers S(n), issued before it
                const int stage = n & 1;
                mbar_wait(&m.bar_v[stage], ph_v[stage], status, &m.dead);
                ph_v[stage] ^= 1;
                tc_fence_after();
                const uint64_t dV = desc_kmajor_base(smem_u32(smem + SmemQ::v0 + stage * KW_BYTES));
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ss(tmem + COL_DP, dDOd + kstep_kmajor<BQ>(ks), dV + kstep_kmajor<BKW>(ks), I_S, ks > 0);
                mma_commit(&m.bar_s);
                if (n + 2 < n_tiles) mma_commit(&m.bar_vfree[stage]);
            };
            mbar_wait(&m.bar_q, ph_q, status, &m.dead);
            ph_q ^= 1;
            issue_s(0);
            issue_dp(0);
            for (int n = 0; n < n_tiles; n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int stage = n & 1;
                // S(n+1) and dP(n+1) run under the element-wise pass of tile n: S has a second buffer, and the pass
                // takes dP(n) into registers first and says so
                if (n + 1 < n_tiles) {
                    issue_s(n + 1);
                    mbar_wait(&m.bar_dpfree, ph_dpfree, status, &m.dead);
                    ph_dpfree ^= 1;
                    tc_fence_after();
                    issue_dp(n + 1);
                }
                // dS(n) written, S(n) read.  One barrier per S buffer: a warp that is done with tile n may already work
                // on tile n+1 (its S and dP are complete) and arrive for it, and that arrival must not count for tile n.
                mbar_wait(&m.bar_p[stage], ph_p[stage], status, &m.dead);
                ph_p[stage] ^= 1;
                tc_fence_after();
                const uint64_t dKm = desc_mnmajor_base<BKW>(smem_u32(smem + SmemQ::k0 + (n % KST) * KW_BYTES));
#pragma unroll
                for (int ks = 0; ks < 8; ks++)
                    mma_ts(tmem + COL_DQ, tmem + stage * 128 + (ks >> 2) * 64 + (ks & 3) * 8, dKm + kstep_mnmajor(ks), I_DQ,
                           n > 0 || ks > 0);
                if (n + KST < n_tiles) mma_commit(&m.bar_kfree[n % KST]);
                if (n + 1 == n_tiles) mma_commit(&m.bar_o);
            }
        }
        if (is_softmax) {
            WalkW walk(ix, piece, qt);
            KvTile t;
            const int i = tid & 127, c = tid >> 7;           // query row, and which 64 of a tile's 128 key columns
            const bool row_ok = i < q_valid;
            // rows past the end of the piece: lse = +inf makes every probability 0
            const float lse2 = row_ok ? lse[(size_t)(q_row0 + i) * Hq + h] * LOG2E : INFINITY;
            const float dl = row_ok ? delta[(size_t)(q_row0 + i) * Hq + h] : 0.f;
            for (int n = 0; walk.next(t); n++) {
                if (*(volatile int*)&m.dead) break;       // a wait ran out: abandon the item
                const int b = n & 1;
                mbar_wait_warp(&m.bar_s, ph_s, status, &m.dead);
                ph_s ^= 1;
                tc_fence_after();
                const int limit = min(t.n_valid, t.shift == NO_DIAG ? BKW : i - t.shift + 1);
                // dP of this thread's 64 columns into registers, so that the buffer can take dP of the next tile
                uint32_t xp[64];
                tmem_ld32(tm_lane + COL_DP + c * 64, xp);
                tmem_ld32(tm_lane + COL_DP + c * 64 + 32, xp + 32);
                tmem_ld_wait();
                tc_fence_before();
                __syncwarp();
                const bool last_tile = walk.in_own && walk.off >= walk.own_end;     // no dP follows the last tile
                if (lane == 0 && !last_tile) mbar_arrive(&m.bar_dpfree);
#pragma unroll
                for (int cc = 0; cc < 2; cc++) {
                    const int j0 = c * 64 + cc * 32;
                    uint32_t xs[32], pk[16];
                    tmem_ld32(tm_lane + b * 128 + j0, xs);
                    tmem_ld_wait();
#pragma unroll
                    for (int e = 0; e < 32; e += 2) {
                        float ds[2];
#pragma unroll
                        for (int u = 0; u < 2; u++) {
                            const float p = j0 + e + u < limit ? ex2(fmaf(__uint_as_float(xs[e + u]), scale_log2, -lse2)) : 0.f;
                            ds[u] = p * (__uint_as_float(xp[cc * 32 + e + u]) - dl) * scale;
                        }
                        pk[e >> 1] = pack_bf16(ds[0], ds[1]);
                    }
                    // over this thread's own half of S (columns it has already read)
                    tmem_st16(tm_lane + b * 128 + c * 64 + cc * 16, pk);
                }
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&m.bar_p[b]);
            }
            // ---- epilogue: dQ -> bf16 ------------------------------------------------------------------------------
            mbar_wait_warp(&m.bar_o, ph_o, status, &m.dead);
            tc_fence_after();
            const bool full = q_valid == BQ;
#pragma unroll
            for (int cc = 0; cc < 2; cc++) {
                const int c4 = c * 2 + cc;
                uint32_t x[32];
                tmem_ld32(tm_lane + COL_DQ + c4 * 32, x);
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
                        *reinterpret_cast<uint4*>(sQ + (col >> 6) * (Q_BYTES / 2) + sw128_chunk(i, (col & 63) >> 3)) = pk;
                    else if (row_ok)
                        *reinterpret_cast<uint4*>(dq + ((size_t)(q_row0 + i) * Hq + h) * D + col) = pk;
                }
            }
            if (full) fence_async_smem();
        }
        ph_o ^= 1;
        tc_fence_before();
        if (__syncthreads_or(m.dead)) break;
        tc_fence_after();
        if (is_issuer && q_valid == BQ) {
            for (int p = 0; p < 2; p++)
                for (int r = 0; r < 2; r++)
                    tma_store_3d(&map_dq, sQ + p * (Q_BYTES / 2) + r * (Q_BYTES / 4), p * 64, h, q_row0 + r * 64);
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
    if (warp == 0) tmem_dealloc<TMEM_Q>(tmem);
}

}  // namespace

int32_t attn_dkv_launch(const Index& ix, int n_rows, const void* q, const void* k, const void* v, const float* lse,
                        const void* dO, const float* delta, void* dk_, void* dv_, int Hq, int Hkv, float scale,
                        int32_t* status, cudaStream_t st);

int32_t attn_bwd_launch(const int32_t* hi, const int32_t* di, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, const void* dO, void* dq, void* dk_, void* dv_, float* delta,
                        int Hq, int Hkv, float scale, int32_t* status, cudaStream_t st) {
    const int n_rows = hi[0];
    if (n_rows == 0 || hi[4] == 0) return HARTS_OK;
    const long long n = (long long)n_rows * Hq;
    delta_kernel<<<(unsigned)((n * 32 + 255) / 256), 256, 0, st>>>((const __nv_bfloat16*)o, (const __nv_bfloat16*)dO,
                                                                  delta, n);
    CUtensorMap mq, mdo, mk, mv, mdq;
    int32_t rc;
    if ((rc = make_row_map(&mq, q, n_rows, Hq)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdo, dO, n_rows, Hq)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mk, k, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mv, v, n_rows, Hkv)) != HARTS_OK) return rc;
    if ((rc = make_row_map(&mdq, dq, n_rows, Hq)) != HARTS_OK) return rc;
    if (cudaFuncSetAttribute(attn_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SmemQ::bytes + 1024) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const Index ix = make_index(hi, di);
    const long long n_work = (long long)ix.n_q_items * Hq;
    const int grid = (int)(n_work < sm_count() ? n_work : sm_count());
    attn_dq_kernel<<<grid, NT, SmemQ::bytes + 1024, st>>>(ix, Hq, Hq / Hkv, scale, mq, mdo, mk, mv, mdq, lse, delta,
                                                         (__nv_bfloat16*)dq, status);
    if (cudaGetLastError() != cudaSuccess) return HARTS_ECUDA;
    return attn_dkv_launch(ix, n_rows, q, k, v, lse, dO, delta, dk_, dv_, Hq, Hkv, scale, status, st);
}

}  // namespace harts
