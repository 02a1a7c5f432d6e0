// Per-channel-decay recurrence (the Diag(gamma) term of Eq. 1, Section 2.2) for bf16 tensors with d_k = d_v = 128:
// the same packed chunkwise call (Eq. 16), plan tables, slots, chunk states and scratch layout as la_gk.cu, with
// every dense product of a chunk on the tensor cores (warp-level mma.sync.m16n8k16, bf16 operands, fp32
// accumulation) and the running state S (forward) / its gradient dS (backward) held in the accumulator registers of
// the CTA's eight warps for the whole walk over a sequence.  What cannot be a dense product stays on the CUDA cores
// in fp32: the decay-dependent pair sums
//     A_tj      = sum_i q_t[i] k_j[i] e^{b_t[i]-b_j[i]}                          (j <= t)
//     dq_t[i]  += sum_{j<=t} dA_tj k_j[i] e^{b_t[i]-b_j[i]},   dk_j[i] += sum_{t>=j} dA_tj q_t[i] e^{b_t[i]-b_j[i]}
// for t and j in the same 16-row block of the chunk; pairs in different blocks become dense products too, through
// operands anchored at the first row of t's block (see scores_*).  Every exponent is a difference of running sums that
// is <= 0 for log-decays g <= 0: no gate value can overflow.  The operands that carry a decay (q~ = q e^{b_t},
// k~ = k e^{b_n-b_j}, the anchored operands, the scores A, the states) are rounded to bf16 as in the scalar-gate
// tensor-core kernels.
//
// Shared-memory tiles of bf16 are row-major with the 16-byte pieces of a row XOR-ed by (row & 7), so that ldmatrix
// (plain and transposed) is free of bank conflicts.
#include "kernels.h"
#include "tc_common.cuh"

namespace harts {

int sm_count();

namespace {

constexpr int BT = 64;      // chunk rows
constexpr int D = 128;      // d_k = d_v
constexpr int NT = 512;     // threads: 16 warps
constexpr int NW = NT / 32;
constexpr float LOG2E = 1.4426950408889634f;

// ---- shared-memory addressing ---------------------------------------------------------------------------------------
// [rows][128] bf16 (256-byte rows) and [rows][64] bf16 (128-byte rows); c16 = index of the 16-byte piece in the row
__device__ __forceinline__ uint32_t sw256(int r, int c16) { return (uint32_t)(r * 256 + ((c16 ^ (r & 7)) << 4)); }
__device__ __forceinline__ uint32_t sw128(int r, int c16) { return (uint32_t)(r * 128 + ((c16 ^ (r & 7)) << 4)); }
__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void ldsm4(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void ldsm4t(uint32_t (&r)[4], uint32_t addr) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr) : "memory");
}
__device__ __forceinline__ void mma16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// 2^x by the special-function unit; the running log-decays are kept in log2 units so that no multiply precedes it
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Fragment loaders.  `tile` is the shared-memory address of a swizzled tile, PITCH its row pitch in bytes.
// A operand (16 x 16) of a matrix stored [m][k]: rows m0.., columns k0..
template <int PITCH>
__device__ __forceinline__ void frag_a(uint32_t (&a)[4], uint32_t tile, int m0, int k0, int lane) {
    const int r = m0 + (lane & 7) + ((lane >> 3) & 1) * 8, c = (k0 >> 3) + (lane >> 4);
    ldsm4(a, tile + (PITCH == 256 ? sw256(r, c) : sw128(r, c)));
}
// A operand (16 x 16) of the TRANSPOSE of a matrix stored [k][m]: A[m][k] = stored[k][m]
template <int PITCH>
__device__ __forceinline__ void frag_a_t(uint32_t (&a)[4], uint32_t tile, int m0, int k0, int lane) {
    const int r = k0 + (lane & 7) + (lane >> 4) * 8, c = (m0 >> 3) + ((lane >> 3) & 1);
    ldsm4t(a, tile + (PITCH == 256 ? sw256(r, c) : sw128(r, c)));
}
// B operands of TWO adjacent n-tiles (n0.., n0+8..) for one k-step, matrix stored [k][n]: b[0],b[1] -> tile n0;
// b[2],b[3] -> tile n0+8
template <int PITCH>
__device__ __forceinline__ void frag_b_kn(uint32_t (&b)[4], uint32_t tile, int k0, int n0, int lane) {
    const int r = k0 + (lane & 7) + ((lane >> 3) & 1) * 8, c = (n0 >> 3) + (lane >> 4);
    ldsm4t(b, tile + (PITCH == 256 ? sw256(r, c) : sw128(r, c)));
}
// the same for a matrix stored [n][k] (B = stored^T)
template <int PITCH>
__device__ __forceinline__ void frag_b_nk(uint32_t (&b)[4], uint32_t tile, int k0, int n0, int lane) {
    const int r = n0 + (lane & 7) + (lane >> 4) * 8, c = (k0 >> 3) + ((lane >> 3) & 1);
    ldsm4(b, tile + (PITCH == 256 ? sw256(r, c) : sw128(r, c)));
}

struct SeqInfo {
    int own_begin, n_replay, n_virtual, n_chunks, replay_base, init_slot, req_lo, req_hi, chunk_base;
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

// row codes of chunk c: physical row >= 0 (own), -2 - row (replayed), -1 (past the end)
__device__ __forceinline__ void load_codes(const harts_la_tables_t& tb, const SeqInfo& s, int c, int* srow) {
    const int tid = threadIdx.x;
    if (tid < BT) {
        const int vr = c * BT + tid;
        int code = -1;
        if (vr < s.n_virtual)
            code = vr < s.n_replay ? -2 - tb.replay_row[s.replay_base + vr] : s.own_begin + (vr - s.n_replay);
        srow[tid] = code;
    }
}

// One [BT][128] bf16 tile of a [rows, H, 128] tensor into a swizzled tile, 16 bytes at a time.  need_own: only rows
// with an output are taken (q, dO); otherwise every valid row (k, v).  Rows that are not taken become zero.
__device__ __forceinline__ void load_tile_bf16(const __nv_bfloat16* src, int H, int h, const int* srow, bool need_own,
                                               unsigned char* dst) {
    constexpr int N = BT * 16 / NT;
    uint4 buf[N];
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 4, c16 = p & 15, code = srow[t];
        const bool take = need_own ? code >= 0 : code != -1;
        const int r = code >= 0 ? code : -2 - code;
        buf[u] = take ? *reinterpret_cast<const uint4*>(src + ((size_t)r * H + h) * D + c16 * 8) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 4, c16 = p & 15;
        *reinterpret_cast<uint4*>(dst + sw256(t, c16)) = buf[u];
    }
}

// g of the chunk's valid rows (fp32 [rows, H, 128]) into sB [BT][128] in log2 units (g * log2 e), zero elsewhere
__device__ __forceinline__ void load_g(const float* gk, int H, int h, const int* srow, float* sB) {
    constexpr int N = BT * 32 / NT;
    float4 buf[N];
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 5, c4 = p & 31, code = srow[t];
        const int r = code >= 0 ? code : -2 - code;
        buf[u] = code != -1 ? *reinterpret_cast<const float4*>(gk + ((size_t)r * H + h) * D + c4 * 4)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT;
        reinterpret_cast<float4*>(sB)[p] = make_float4(buf[u].x * LOG2E, buf[u].y * LOG2E, buf[u].z * LOG2E, buf[u].w * LOG2E);
    }
}

// Asks the L2 for the rows of chunk c of a [rows, H, 128] tensor (the chunk after the one being worked on: its global
// loads then find their lines in the L2 instead of waiting for HBM).  Chunks >= 1 hold own rows only, which are
// consecutive: virtual row vr is physical row own_begin - n_replay + vr.
template <typename T>
__device__ __forceinline__ void prefetch_rows(const T* base, int H, int h, const SeqInfo& s, int c) {
    constexpr int LINES = D * (int)sizeof(T) / 128;              // 128-byte lines per row and head
    for (int p = threadIdx.x; p < BT * LINES; p += NT) {
        const int vr = c * BT + p / LINES;
        if (vr < s.n_virtual) {
            const char* addr = reinterpret_cast<const char*>(base + ((size_t)(s.own_begin - s.n_replay + vr) * H + h) * D) +
                               (p % LINES) * 128;
            asm volatile("prefetch.global.L2 [%0];" ::"l"(addr));
        }
    }
}

// running sum over the rows, per channel: four threads per channel (16 rows each, scanned in registers), joined through
// sTmp[4][128]
__device__ __forceinline__ void cumsum_rows(float* sB, float* sTmp) {
    const int tid = threadIdx.x, i = tid & (D - 1), part = tid >> 7;
    float x[16];
#pragma unroll
    for (int u = 0; u < 16; u++) x[u] = sB[(part * 16 + u) * D + i];
#pragma unroll
    for (int u = 1; u < 16; u++) x[u] += x[u - 1];
    sTmp[part * D + i] = x[15];
    __syncthreads();
    float base = 0.f;
    for (int pp = 0; pp < part; pp++) base += sTmp[pp * D + i];
#pragma unroll
    for (int u = 0; u < 16; u++) sB[(part * 16 + u) * D + i] = x[u] + base;
    __syncthreads();
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

// ---- the scores A_tj = sum_i q_t[i] k_j[i] e^{b_t[i]-b_j[i]} (j <= t), bf16 into sP ([BT][BT], swizzled) --------------
// The chunk is cut into four blocks of 16 rows.  With a_I = b at the first row of block I (log-decays are <= 0, so b
// only falls along the rows):
//   j in an EARLIER block than t (block I):  e^{b_t-b_j} = e^{b_t-a_I} e^{a_I-b_j}, both exponents <= 0, so the block of
//     scores is the dense product of q^_t = q_t e^{b_t-a_I} and k^(I)_j = k_j e^{a_I-b_j} (tensor cores);
//   j in the SAME block as t: the exponent difference is taken directly (CUDA cores, fp32), as no anchor inside the
//     block bounds both factors.
// anchored operands: sQa [64][128] (row t anchored at its own block), sKa: k^(1) rows 0..15, k^(2) rows 0..31, k^(3)
// rows 0..47 stored one after the other (row offsets 0, 16, 48)
__device__ __forceinline__ int ka_row0(int I) { return I == 1 ? 0 : (I == 2 ? 16 : 48); }

__device__ __forceinline__ void anchored_operands(const unsigned char* sQ, const unsigned char* sK, const float* sB,
                                                  unsigned char* sQa, unsigned char* sKa) {
    // 64 rows of q^ and 16 + 32 + 48 = 96 rows of k^(I): 160 rows x 16 pieces
    for (int p = threadIdx.x; p < 160 * 16; p += NT) {
        const int rr = p >> 4, c16 = p & 15;
        int src_row, anchor_row, dst_row;
        bool is_q;
        if (rr < 64) { is_q = true; src_row = rr; anchor_row = rr & ~15; dst_row = rr; }
        else {
            is_q = false;
            const int r2 = rr - 64, I = r2 < 16 ? 1 : (r2 < 48 ? 2 : 3);
            src_row = r2 - ka_row0(I); anchor_row = 16 * I; dst_row = r2;
        }
        uint4 x = *reinterpret_cast<const uint4*>((is_q ? sQ : sK) + sw256(src_row, c16));
        uint32_t* w = reinterpret_cast<uint32_t*>(&x);
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const int i = c16 * 8 + e * 2;
            const float2 bs = *reinterpret_cast<const float2*>(sB + src_row * D + i);
            const float2 ba = *reinterpret_cast<const float2*>(sB + anchor_row * D + i);
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]));
            // q^: e^{b_t - a_I};  k^(I): e^{a_I - b_j}
            const float e0 = is_q ? ex2(bs.x - ba.x) : ex2(ba.x - bs.x);
            const float e1 = is_q ? ex2(bs.y - ba.y) : ex2(ba.y - bs.y);
            w[e] = pack2(f.x * e0, f.y * e1);
        }
        // the local row index of a k^(I) sub-tile is dst_row - its row offset; the offsets are multiples of 8, so the
        // swizzle of the stacked tile equals that of the sub-tile
        *reinterpret_cast<uint4*>((is_q ? sQa : sKa) + sw256(dst_row, c16)) = x;
    }
}

// Pairs INSIDE a 16-row block: with the same anchor a_I (b at the block's first row) the key factor e^{a_I-b_j} is >= 1
// and grows to e^{a_I - b_{16I+15}} at the block's last row.  While that total decay of a block stays below 2^MILD_LOG2
// in every channel (bf16 and fp32 hold 2^127), the block on the diagonal is a dense product too: q^ (anchored at its
// block, as above) against k_j e^{a_I-b_j} for the keys of the same block, masked to j <= t afterwards -- the entries
// right of the diagonal are finite and thrown away.  A chunk in which any block decays faster takes the exact CUDA-core
// path for its diagonal blocks instead (one decision per chunk, the same for the whole CTA).
constexpr float MILD_LOG2 = 100.f;

__device__ __forceinline__ bool chunk_is_mild(const float* sB) {
    const int i = threadIdx.x & (D - 1), blk = threadIdx.x >> 7;       // 512 threads: 4 blocks x 128 channels
    const float fall = sB[16 * blk * D + i] - sB[(16 * blk + 15) * D + i];
    return __syncthreads_or(!(fall <= MILD_LOG2)) == 0;                  // also false for a NaN gate
}

// keys anchored at their OWN block: sKd[j] = k_j .* 2^{a_I(j) - b_j}  (bf16 [64][128], swizzled)
__device__ __forceinline__ void diag_operand(const unsigned char* sK, const float* sB, unsigned char* sKd) {
    for (int p = threadIdx.x; p < BT * 16; p += NT) {
        const int j = p >> 4, c16 = p & 15, a_row = j & ~15;
        uint4 x = *reinterpret_cast<const uint4*>(sK + sw256(j, c16));
        uint32_t* w = reinterpret_cast<uint32_t*>(&x);
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const int i = c16 * 8 + e * 2;
            const float2 bs = *reinterpret_cast<const float2*>(sB + j * D + i);
            const float2 ba = *reinterpret_cast<const float2*>(sB + a_row * D + i);
            const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]));
            w[e] = pack2(f.x * ex2(ba.x - bs.x), f.y * ex2(ba.y - bs.y));
        }
        *reinterpret_cast<uint4*>(sKd + sw256(j, c16)) = x;
    }
}

// blocks left of the diagonal: warp -> row block I = warp & 3, 16-column tile J = warp >> 2; with `diag` (a mild chunk)
// the warps with J == I take the block on the diagonal from the keys anchored at their own block
__device__ __forceinline__ void scores_off_diagonal(uint32_t aQa, uint32_t aKa, unsigned char* sP, int warp, int lane,
                                                    bool diag = false, uint32_t aKd = 0) {
    const int I = warp & 3, g = lane >> 2, tq = lane & 3;
    if (diag && (warp >> 2) == I) {
        float acc[2][4];
#pragma unroll
        for (int x = 0; x < 2; x++) acc[x][0] = acc[x][1] = acc[x][2] = acc[x][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ks++) {
            uint32_t a[4], b[4];
            frag_a<256>(a, aQa, 16 * I, ks * 16, lane);
            frag_b_nk<256>(b, aKd, ks * 16, 16 * I, lane);
            mma16816(acc[0], a, b[0], b[1]);
            mma16816(acc[1], a, b[2], b[3]);
        }
#pragma unroll
        for (int x = 0; x < 2; x++) {
            const int jc = 8 * x + 2 * tq, col = 16 * I + jc;           // jc, g: column and row inside the block
            const float v0 = jc <= g ? acc[x][0] : 0.f, v1 = jc + 1 <= g ? acc[x][1] : 0.f;
            const float v2 = jc <= g + 8 ? acc[x][2] : 0.f, v3 = jc + 1 <= g + 8 ? acc[x][3] : 0.f;
            *reinterpret_cast<uint32_t*>(sP + sw128(16 * I + g, col >> 3) + (col & 7) * 2) = pack2(v0, v1);
            *reinterpret_cast<uint32_t*>(sP + sw128(16 * I + g + 8, col >> 3) + (col & 7) * 2) = pack2(v2, v3);
        }
        return;
    }
    for (int J = warp >> 2; J < I; J += NW / 4) {
        float acc[2][4];
#pragma unroll
        for (int x = 0; x < 2; x++) acc[x][0] = acc[x][1] = acc[x][2] = acc[x][3] = 0.f;
#pragma unroll
        for (int ks = 0; ks < 8; ks++) {
            uint32_t a[4], b[4];
            frag_a<256>(a, aQa, 16 * I, ks * 16, lane);
            frag_b_nk<256>(b, aKa, ks * 16, ka_row0(I) + 16 * J, lane);
            mma16816(acc[0], a, b[0], b[1]);
            mma16816(acc[1], a, b[2], b[3]);
        }
#pragma unroll
        for (int x = 0; x < 2; x++) {
            const int col = 16 * J + 8 * x + 2 * tq;
            *reinterpret_cast<uint32_t*>(sP + sw128(16 * I + g, col >> 3) + (col & 7) * 2) = pack2(acc[x][0], acc[x][1]);
            *reinterpret_cast<uint32_t*>(sP + sw128(16 * I + g + 8, col >> 3) + (col & 7) * 2) = pack2(acc[x][2], acc[x][3]);
        }
    }
}

// one-step decay factors 2^{b_t - b_{t-1}} of the rows 1..63 of a chunk (fp32 [BT][128]; row 0 is not used: the factors
// serve pairs inside a 16-row block only)
__device__ __forceinline__ void step_factors(const float* sB, float* sR) {
    for (int p = threadIdx.x; p < BT * 32; p += NT) {
        const int t = p >> 5, c4 = p & 31;
        if (t == 0) continue;
        const float4 hi = *reinterpret_cast<const float4*>(sB + t * D + c4 * 4);
        const float4 lo = *reinterpret_cast<const float4*>(sB + (t - 1) * D + c4 * 4);
        *reinterpret_cast<float4*>(sR + t * D + c4 * 4) = make_float4(ex2(hi.x - lo.x), ex2(hi.y - lo.y), ex2(hi.z - lo.z), ex2(hi.w - lo.w));
    }
}

// diagonal blocks: one warp per row t, every lane takes 4 channels of all (at most 16) pairs of the row, walking j from t
// down with the decay as a running product of the one-step factors (x_{t,j-1} = x_{t,j} r_j: every factor <= 1, no
// exponential per pair); the warp sums the lanes with a transposed reduction, lanes 0..15 then hold A[t][16 I + lane]
// (zero right of the diagonal)
__device__ __forceinline__ void scores_diagonal(const unsigned char* sQ, const unsigned char* sK, const float* sR,
                                                unsigned char* sP, int warp, int lane) {
    for (int t = warp; t < BT; t += NW) {
        const int j_lo = t & ~15;
        const uint2 qraw = *reinterpret_cast<const uint2*>(sQ + sw256(t, lane >> 1) + (lane & 1) * 8);
        const float2 q01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qraw.x));
        const float2 q23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qraw.y));
        float4 qx = make_float4(q01.x, q01.y, q23.x, q23.y);          // q_t .* x_{t,j}, j walking down from t
        float z[16];
#pragma unroll
        for (int u = 15; u >= 0; u--) {
            const int j = j_lo + u;
            float acc = 0.f;
            if (j <= t) {
                const uint2 kraw = *reinterpret_cast<const uint2*>(sK + sw256(j, lane >> 1) + (lane & 1) * 8);
                const float2 k01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kraw.x));
                const float2 k23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kraw.y));
                acc = qx.x * k01.x + qx.y * k01.y + qx.z * k23.x + qx.w * k23.y;
                if (u > 0) {
                    const float4 r = *reinterpret_cast<const float4*>(sR + j * D + lane * 4);
                    qx.x *= r.x; qx.y *= r.y; qx.z *= r.z; qx.w *= r.w;
                }
            }
            z[u] = acc;
        }
        const float total = warp_transpose_reduce16(z, lane);
        const float other = __shfl_down_sync(0xffffffffu, total, 1);
        if (lane < 16 && !(lane & 1)) {
            const int col = j_lo + lane;
            *reinterpret_cast<uint32_t*>(sP + sw128(t, col >> 3) + (col & 7) * 2) = pack2(total, other);
        }
    }
}

// q <- q .* e^{b_t} and k <- k .* e^{b_n - b_t} written to (possibly other) swizzled tiles
__device__ __forceinline__ void scale_qk(const unsigned char* sQ, const unsigned char* sK, const float* sB,
                                         unsigned char* dQ, unsigned char* dK) {
#pragma unroll
    for (int u = 0; u < BT * 16 / NT; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 4, c16 = p & 15;
        const uint32_t off = sw256(t, c16);
        uint4 qv = *reinterpret_cast<const uint4*>(sQ + off), kv = *reinterpret_cast<const uint4*>(sK + off);
        uint32_t* qw = reinterpret_cast<uint32_t*>(&qv);
        uint32_t* kw = reinterpret_cast<uint32_t*>(&kv);
#pragma unroll
        for (int e = 0; e < 4; e++) {
            const int i = c16 * 8 + e * 2;
            const float2 bt = *reinterpret_cast<const float2*>(sB + t * D + i);
            const float2 bn = *reinterpret_cast<const float2*>(sB + (BT - 1) * D + i);
            const float2 qf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qw[e]));
            const float2 kf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kw[e]));
            qw[e] = pack2(qf.x * ex2(bt.x), qf.y * ex2(bt.y));
            kw[e] = pack2(kf.x * ex2(bn.x - bt.x), kf.y * ex2(bn.y - bt.y));
        }
        *reinterpret_cast<uint4*>(dQ + off) = qv;
        *reinterpret_cast<uint4*>(dK + off) = kv;
    }
}

// The state fragments of a warp: rows 16 * (warp & 7) + g and + g + 8 (g = lane / 4), columns
// 64 * (warp >> 3) + 8 * n + 2 * (lane % 4) + {0, 1} of n-tile n: st[n][0..1] = row g, st[n][2..3] = row g + 8.
struct Shared {
    static constexpr int q = 0, k = 16384, v = 32768;          // bf16 [64][128]
    static constexpr int p = 49152;                             // bf16 [64][64]
    static constexpr int sb = 57344;                            // bf16 [128][128]: the state as an MMA operand
    static constexpr int b = 90112;                             // fp32 [64][128]: running log-decay (log2 units)
    static constexpr int qa = 122880;                           // bf16 [64][128]: q anchored at its 16-row block
    static constexpr int ka = qa + 16384;                       // bf16 [96][128]: k anchored at blocks 1, 2, 3
    static constexpr int r = ka + 96 * 256;                     // fp32 [64][128]: one-step decay factors
    static constexpr int tmp = r + 32768;                       // fp32 [4][128]
    static constexpr int row = tmp + 2048;                      // int  [64]
    static constexpr int fwd_bytes = row + 256;
};

// state fragments -> bf16 operand tile (swizzled [128][128])
__device__ __forceinline__ void state_to_operand(const float (&st)[8][4], unsigned char* sSb, int warp, int lane) {
    const int g = lane >> 2, tq = lane & 3, r0 = (warp & 7) * 16 + g, c0 = (warp >> 3) * 8;
#pragma unroll
    for (int n = 0; n < 8; n++) {
        *reinterpret_cast<uint32_t*>(sSb + sw256(r0, c0 + n) + tq * 4) = pack2(st[n][0], st[n][1]);
        *reinterpret_cast<uint32_t*>(sSb + sw256(r0 + 8, c0 + n) + tq * 4) = pack2(st[n][2], st[n][3]);
    }
}
// state fragments <-> fp32 [128][128] in global memory (slots, initial-state gradients)
// PAST_L1: the data was written during this launch by another CTA
template <bool ADD, bool PAST_L1>
__device__ __forceinline__ void state_from_global(float (&st)[8][4], const float* src, int warp, int lane) {
    const int g = lane >> 2, tq = lane & 3, r0 = (warp & 7) * 16 + g, c0 = (warp >> 3) * 64 + tq * 2;
#pragma unroll
    for (int n = 0; n < 8; n++) {
        const float2* p_lo = reinterpret_cast<const float2*>(src + (size_t)r0 * D + c0 + n * 8);
        const float2* p_hi = reinterpret_cast<const float2*>(src + (size_t)(r0 + 8) * D + c0 + n * 8);
        const float2 lo = PAST_L1 ? __ldcg(p_lo) : *p_lo;
        const float2 hi = PAST_L1 ? __ldcg(p_hi) : *p_hi;
        if (ADD) { st[n][0] += lo.x; st[n][1] += lo.y; st[n][2] += hi.x; st[n][3] += hi.y; }
        else { st[n][0] = lo.x; st[n][1] = lo.y; st[n][2] = hi.x; st[n][3] = hi.y; }
    }
}
__device__ __forceinline__ void state_to_global(const float (&st)[8][4], float* dst, int warp, int lane) {
    const int g = lane >> 2, tq = lane & 3, r0 = (warp & 7) * 16 + g, c0 = (warp >> 3) * 64 + tq * 2;
#pragma unroll
    for (int n = 0; n < 8; n++) {
        *reinterpret_cast<float2*>(dst + (size_t)r0 * D + c0 + n * 8) = make_float2(st[n][0], st[n][1]);
        *reinterpret_cast<float2*>(dst + (size_t)(r0 + 8) * D + c0 + n * 8) = make_float2(st[n][2], st[n][3]);
    }
}
// st <- Diag(2^{b_n}) st + X^T Y over the chunk's 64 rows: X stored [row][128] (its transpose is the A operand), Y
// stored [row][128]
__device__ __forceinline__ void state_update(float (&st)[8][4], const float* sB, uint32_t aX, uint32_t aY, int warp, int lane) {
    const int g = lane >> 2, r0 = (warp & 7) * 16, c0 = (warp >> 3) * 64;
    const float g_lo = ex2(sB[(BT - 1) * D + r0 + g]), g_hi = ex2(sB[(BT - 1) * D + r0 + g + 8]);
#pragma unroll
    for (int n = 0; n < 8; n++) {
        st[n][0] *= g_lo; st[n][1] *= g_lo; st[n][2] *= g_hi; st[n][3] *= g_hi;
    }
#pragma unroll
    for (int ks = 0; ks < 4; ks++) {
        uint32_t a[4];
        frag_a_t<256>(a, aX, r0, ks * 16, lane);
#pragma unroll
        for (int n2 = 0; n2 < 4; n2++) {
            uint32_t b[4];
            frag_b_kn<256>(b, aY, ks * 16, c0 + n2 * 16, lane);
            mma16816(st[2 * n2], a, b[0], b[1]);
            mma16816(st[2 * n2 + 1], a, b[2], b[3]);
        }
    }
}
// swizzled bf16 [rows][128] tile -> plain row-major global memory ([rows][128] contiguous), 16 bytes per thread and step
template <int ROWS>
__device__ __forceinline__ void tile_to_global(const unsigned char* tile, __nv_bfloat16* dst) {
    for (int p = threadIdx.x; p < ROWS * 16; p += NT)
        reinterpret_cast<uint4*>(dst)[p] = *reinterpret_cast<const uint4*>(tile + sw256(p >> 4, p & 15));
}

// ONE_LAUNCH: the grid covers the sequences of ALL rounds (numbered round by round).  Every CTA draws its work item
// from `ticket`, so an item is only ever held by a running CTA; a sequence that starts from an exported state waits for
// the flag its producer (an earlier round, a smaller ticket, hence running or done) sets after writing the slot.
// Otherwise: one launch per round, item = block index, no flags.
template <bool ONE_LAUNCH>
__global__ void __launch_bounds__(NT, 1)
gk_mma_fwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const __nv_bfloat16* __restrict__ q,
                  const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ gk,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ slots, __nv_bfloat16* __restrict__ chunk_states,
                  const int32_t* gate, int* status, int* slot_flags, int* ticket) {
    if (gate_closed(gate)) return;
    __shared__ int s_item, s_dead;
    extern __shared__ __align__(1024) unsigned char sm[];
    unsigned char *sQ = sm + Shared::q, *sK = sm + Shared::k, *sV = sm + Shared::v, *sP = sm + Shared::p,
                  *sSb = sm + Shared::sb, *sQa = sm + Shared::qa, *sKa = sm + Shared::ka;
    float* sB = reinterpret_cast<float*>(sm + Shared::b);
    float* sR = reinterpret_cast<float*>(sm + Shared::r);
    float* sTmp = reinterpret_cast<float*>(sm + Shared::tmp);
    int* srow = reinterpret_cast<int*>(sm + Shared::row);
    const uint32_t aQ = s_u32(sQ), aK = s_u32(sK), aV = s_u32(sV), aP = s_u32(sP), aSb = s_u32(sSb);

    // blocks are handed to the SMs in index order: with the plan's order (longest sequence of the round first) the long
    // walks start first and the short ones fill the tail
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    int item = blockIdx.x;
    if constexpr (ONE_LAUNCH) {
        if (tid == 0) {
            s_item = atomicAdd(ticket, 1);
            s_dead = 0;
        }
        __syncthreads();
        item = s_item;
    }
    const int seq_pos = seq_lo + item / H, h = item % H;
    const int seq = tb.seq_order ? tb.seq_order[seq_pos] : seq_pos;
    const int mb = warp & 3, nq = warp >> 2;          // this warp's 16-row block and 32-column quarter of [64][128] products
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)D * D;

    float st[8][4];
    if (s.init_slot < 0) {
#pragma unroll
        for (int n = 0; n < 8; n++) st[n][0] = st[n][1] = st[n][2] = st[n][3] = 0.f;
    } else {
        if constexpr (ONE_LAUNCH) {
            if (tid == 0) tc::flag_wait(slot_flags + (size_t)s.init_slot * H + h, status, &s_dead);
            if (__syncthreads_or(s_dead)) return;      // the wait ran out (status word set): give the walk up
        }
        state_from_global<false, ONE_LAUNCH>(st, slots + ((size_t)s.init_slot * H + h) * state_elems, warp, lane);
    }

    int next_req = s.req_lo;
    for (int c = 0; c < s.n_chunks; c++) {
        __syncthreads();                                   // the previous chunk's readers of every tile are through
        load_codes(tb, s, c, srow);
        __syncthreads();
        load_tile_bf16(k, H, h, srow, false, sK);
        load_tile_bf16(q, H, h, srow, true, sQ);
        load_tile_bf16(v, H, h, srow, false, sV);
        load_g(gk, H, h, srow, sB);
        if (c + 1 < s.n_chunks) {
            prefetch_rows(k, H, h, s, c + 1);
            prefetch_rows(q, H, h, s, c + 1);
            prefetch_rows(v, H, h, s, c + 1);
            prefetch_rows(gk, H, h, s, c + 1);
        }
        // start-of-chunk state: operand copy, kept for the backward, exported when the plan requests this boundary
        state_to_operand(st, sSb, warp, lane);
        const bool exported = next_req < s.req_hi && tb.slot_chunk[next_req] == c;
        if (exported) {
            state_to_global(st, slots + ((size_t)next_req * H + h) * state_elems, warp, lane);
            if (ONE_LAUNCH) __threadfence();               // this thread's part of the slot, before the flag below
            next_req++;
        }
        __syncthreads();
        if (ONE_LAUNCH && exported && tid == 0) tc::flag_set(slot_flags + (size_t)(next_req - 1) * H + h);
        if (chunk_states) tile_to_global<D>(sSb, chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems);
        cumsum_rows(sB, sTmp);
        const bool mild = chunk_is_mild(sB);
        unsigned char* sKd = reinterpret_cast<unsigned char*>(sR);        // the two are never needed in the same chunk
        if (mild) diag_operand(sK, sB, sKd);
        else step_factors(sB, sR);
        anchored_operands(sQ, sK, sB, sQa, sKa);
        __syncthreads();
        if (!mild) scores_diagonal(sQ, sK, sR, sP, warp, lane);
        scores_off_diagonal(s_u32(sQa), s_u32(sKa), sP, warp, lane, mild, s_u32(sKd));
        __syncthreads();
        scale_qk(sQ, sK, sB, sQ, sK);
        __syncthreads();
        // ---- o = P V + q~ S_c : warp -> rows 16 * mb, columns 32 * nq ----------------------------------------------
        {
            const int m0 = mb * 16, n_base = nq * 32;
            float acc[4][4];
#pragma unroll
            for (int n = 0; n < 4; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            for (int ks = 0; ks <= mb; ks++) {              // P is zero right of the diagonal block
                uint32_t a[4];
                frag_a<128>(a, aP, m0, ks * 16, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    uint32_t b[4];
                    frag_b_kn<256>(b, aV, ks * 16, n_base + n2 * 16, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
#pragma unroll
            for (int ks = 0; ks < 8; ks++) {
                uint32_t a[4];
                frag_a<256>(a, aQ, m0, ks * 16, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    uint32_t b[4];
                    frag_b_kn<256>(b, aSb, ks * 16, n_base + n2 * 16, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
            const int c_lo = srow[m0 + g], c_hi = srow[m0 + g + 8];
#pragma unroll
            for (int n = 0; n < 4; n++) {
                const int col = n_base + n * 8 + tq * 2;
                if (c_lo >= 0) *reinterpret_cast<uint32_t*>(o + ((size_t)c_lo * H + h) * D + col) = pack2(acc[n][0], acc[n][1]);
                if (c_hi >= 0) *reinterpret_cast<uint32_t*>(o + ((size_t)c_hi * H + h) * D + col) = pack2(acc[n][2], acc[n][3]);
            }
        }
        // ---- S <- Diag(e^{b_n}) S + k~^T V ---------------------------------------------------------------------------
        state_update(st, sB, aK, aV, warp, lane);
    }
}

// ---- backward ---------------------------------------------------------------------------------------------------------
// With dS the gradient of the state at the END of the chunk on entry, dA_tj = dO_t . v_j, ew_j = e^{b_n-b_j}:
//   dq_t[i] = e^{b_t[i]} (dO_t S_c^T)[i] + sum_{j<=t} dA_tj k_j[i] e^{b_t[i]-b_j[i]}
//   dk_j[i] = ew_j[i] (v_j dS^T)[i]      + sum_{t>=j} dA_tj q_t[i] e^{b_t[i]-b_j[i]}
//   dv_j    = sum_{t>=j} A_tj dO_t + (k_j .* ew_j) dS
//   dg_t[i] = sum_{tau>=t} (q_tau[i] dq_tau[i] - k_tau[i] dk_tau[i]) + e^{b_n[i]} <S_c[i,:], dS[i,:]> + sum_j k_j[i] ew_j[i] (v_j dS^T)[i]
//   dS     <- Diag(e^{b_n}) dS + (q .* e^{b})^T dO
// The pair sums are split like the scores of the forward: pairs in different 16-row blocks through the anchored
// operands (for dk the factor e^{a_I-b_j} of block I multiplies the product of dA's block with q^ afterwards, so one
// set of anchors serves both), pairs inside a block on the CUDA cores, one thread per (channel, half of the rows).
struct SharedB {
    static constexpr int q = 0, k = 16384, v = 32768, dO = 49152;    // bf16 [64][128]
    static constexpr int b = 65536;                                     // fp32 [64][128]
    static constexpr int sc = 98304;                                    // bf16 [128][128] S_c; later fp32 [64][128] dq
    static constexpr int dsb = 131072;                                  // bf16 [128][128] dS as an MMA operand
    static constexpr int qa = 163840;                                   // bf16 [64][128] anchored q  } later fp32
    static constexpr int ka = qa + 16384;                               // bf16 [96][128] anchored k  } [64][128] dk
    static constexpr int p = ka + 96 * 256;                             // bf16 [64][64] scores
    static constexpr int dab = p + 8192;                                // bf16 [64][64] dA
    static constexpr int dad = dab + 8192;                              // fp32 [64][16] dA, diagonal blocks
    static constexpr int tmp = dad + 4096;                              // fp32 [4][128]
    static constexpr int rowdot = tmp + 2048;                           // fp32 [2][128]
    static constexpr int gi = rowdot + 1024;                            // fp32 [4][128]
    static constexpr int row = gi + 2048;                               // int [64]
    static constexpr int bytes = row + 256;
};
static_assert(SharedB::bytes <= 232448, "backward tiles do not fit in shared memory");

// plain row-major [128][128] bf16 in global memory -> swizzled tile
__device__ __forceinline__ void global_to_tile128(const __nv_bfloat16* src, unsigned char* tile) {
    uint4 buf[D * 16 / NT];
#pragma unroll
    for (int u = 0; u < D * 16 / NT; u++) buf[u] = reinterpret_cast<const uint4*>(src)[threadIdx.x + u * NT];
#pragma unroll
    for (int u = 0; u < D * 16 / NT; u++) {
        const int p = threadIdx.x + u * NT;
        *reinterpret_cast<uint4*>(tile + sw256(p >> 4, p & 15)) = buf[u];
    }
}

__device__ __forceinline__ float2 ld_bf2(const unsigned char* tile, int r, int col) {      // [r][col], [r][col+1]; col even
    return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(tile + sw256(r, col >> 3) + (col & 7) * 2));
}


// ONE_LAUNCH: the grid covers the sequences of all rounds; every CTA draws its item from `ticket` (last round first,
// inside a round the plan's order).  A sequence publishes a flag once its initial-state gradient is in the scratch area;
// a sequence that exported a boundary waits for the flags of all sequences that started there (later rounds, smaller
// tickets, hence running or done) and sums their gradients itself in the order handoff_reduce uses.
template <bool ONE_LAUNCH>
__global__ void __launch_bounds__(NT, 1)
gk_mma_bwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const __nv_bfloat16* __restrict__ q,
                  const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ gk,
                  const __nv_bfloat16* __restrict__ dO, __nv_bfloat16* __restrict__ dq, __nv_bfloat16* __restrict__ dk_,
                  __nv_bfloat16* __restrict__ dv_, float* __restrict__ dgk, const __nv_bfloat16* __restrict__ chunk_states,
                  float* __restrict__ ds0, float* __restrict__ rk, float* __restrict__ rv, float* __restrict__ rg,
                  const int32_t* gate, int* status, int* ds0_flags, int* ticket, const RoundOrder rounds) {
    if (gate_closed(gate)) return;
    __shared__ int s_item, s_dead;
    extern __shared__ __align__(1024) unsigned char sm[];
    unsigned char *sQ = sm + SharedB::q, *sK = sm + SharedB::k, *sV = sm + SharedB::v, *sDO = sm + SharedB::dO,
                  *sSc = sm + SharedB::sc, *sdSb = sm + SharedB::dsb, *sQa = sm + SharedB::qa, *sKa = sm + SharedB::ka,
                  *sP = sm + SharedB::p, *sdAb = sm + SharedB::dab;
    float* sB = reinterpret_cast<float*>(sm + SharedB::b);
    float* sR = reinterpret_cast<float*>(sm + SharedB::sc);        // one-step decay factors, after S_c is dead
    float* sDQ = reinterpret_cast<float*>(sm + SharedB::sc);       // after the step factors are dead
    float* sDK = reinterpret_cast<float*>(sm + SharedB::qa);       // after the anchored operands are dead
    float* sdAd = reinterpret_cast<float*>(sm + SharedB::dad);
    float* sTmp = reinterpret_cast<float*>(sm + SharedB::tmp);
    float* sRowdot = reinterpret_cast<float*>(sm + SharedB::rowdot);
    float* sGi = reinterpret_cast<float*>(sm + SharedB::gi);
    int* srow = reinterpret_cast<int*>(sm + SharedB::row);
    const uint32_t aQ = s_u32(sQ), aK = s_u32(sK), aV = s_u32(sV), aDO = s_u32(sDO), aSc = s_u32(sSc), adSb = s_u32(sdSb),
                   aQa = s_u32(sQa), aKa = s_u32(sKa), aP = s_u32(sP), adAb = s_u32(sdAb);

    // blocks are handed to the SMs in index order: with the plan's order (longest sequence of the round first) the long
    // walks start first and the short ones fill the tail
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    int seq_pos = seq_lo + blockIdx.x / H, h = blockIdx.x % H;
    if constexpr (ONE_LAUNCH) {
        if (tid == 0) {
            s_item = atomicAdd(ticket, 1);
            s_dead = 0;
        }
        __syncthreads();
        int j = s_item / H;
        h = s_item % H;
        seq_pos = -1;
        for (int r = rounds.n - 1; r >= 0 && seq_pos < 0; r--) {      // last round first
            const int cnt = rounds.ptr[r + 1] - rounds.ptr[r];
            if (j < cnt) seq_pos = rounds.ptr[r] + j;
            else j -= cnt;
        }
    }
    const int seq = tb.seq_order ? tb.seq_order[seq_pos] : seq_pos;
    const int mb = warp & 3, nq = warp >> 2;          // this warp's 16-row block and 32-column quarter of [64][128] products
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)D * D;

    float ds[8][4];                                   // dS, laid out over the warps like the forward's state
#pragma unroll
    for (int n = 0; n < 8; n++) ds[n][0] = ds[n][1] = ds[n][2] = ds[n][3] = 0.f;

    int next_req = s.req_hi - 1;                      // slots of this sequence are ordered by chunk index
    for (int c = s.n_chunks - 1; c >= 0; c--) {
        __syncthreads();                              // the previous chunk's readers of every tile are through
        // gradient arriving at boundary c+1 from the sequences that started there: one launch per round -- summed into
        // the first consumer's buffer by handoff_reduce; all rounds in one launch -- awaited and summed here, same order
        if (next_req >= s.req_lo && tb.slot_chunk[next_req] == c + 1) {
            const int cons_lo = tb.slot_cons_ptr[next_req], cons_hi = tb.slot_cons_ptr[next_req + 1];
            if constexpr (ONE_LAUNCH) {
                for (int u = cons_lo + tid; u < cons_hi; u += NT)
                    tc::flag_wait(ds0_flags + (size_t)tb.slot_cons_seq[u] * H + h, status, &s_dead);
                if (__syncthreads_or(s_dead)) return;      // a wait ran out (status word set): give the walk up
            }
            if (cons_lo < cons_hi) {
                if constexpr (ONE_LAUNCH) {
                    float a[8][4];
                    state_from_global<false, true>(a, ds0 + ((size_t)tb.slot_cons_seq[cons_lo] * H + h) * state_elems, warp, lane);
                    for (int u = cons_lo + 1; u < cons_hi; u++)
                        state_from_global<true, true>(a, ds0 + ((size_t)tb.slot_cons_seq[u] * H + h) * state_elems, warp, lane);
#pragma unroll
                    for (int n = 0; n < 8; n++) {
                        ds[n][0] += a[n][0]; ds[n][1] += a[n][1]; ds[n][2] += a[n][2]; ds[n][3] += a[n][3];
                    }
                } else {
                    state_from_global<true, false>(ds, ds0 + ((size_t)tb.slot_cons_seq[cons_lo] * H + h) * state_elems, warp, lane);
                }
            }
            next_req--;
        }
        load_codes(tb, s, c, srow);
        __syncthreads();
        load_tile_bf16(k, H, h, srow, false, sK);
        load_tile_bf16(q, H, h, srow, true, sQ);
        load_tile_bf16(v, H, h, srow, false, sV);
        load_tile_bf16(dO, H, h, srow, true, sDO);
        load_g(gk, H, h, srow, sB);
        global_to_tile128(chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems, sSc);
        if (c >= 1) {      // the next chunk of the walk (chunk 0 of a sequence with replayed rows is not consecutive)
            if (c - 1 >= 1 || s.n_replay == 0) {
                prefetch_rows(k, H, h, s, c - 1);
                prefetch_rows(q, H, h, s, c - 1);
                prefetch_rows(v, H, h, s, c - 1);
                prefetch_rows(dO, H, h, s, c - 1);
                prefetch_rows(gk, H, h, s, c - 1);
            }
            const char* st = reinterpret_cast<const char*>(chunk_states + ((size_t)(s.chunk_base + c - 1) * H + h) * state_elems);
            for (int p = tid; p < D * D * 2 / 128; p += NT) asm volatile("prefetch.global.L2 [%0];" ::"l"(st + p * 128));
        }
        state_to_operand(ds, sdSb, warp, lane);
        __syncthreads();
        cumsum_rows(sB, sTmp);
        const bool mild = chunk_is_mild(sB);          // diagonal blocks as dense products too (see chunk_is_mild)
        const int r_lo = 16 * mb + g, r_hi = r_lo + 8;            // this thread's rows in the [64][128] products
        // ---- dA = dO V^T, iq = dO S_c^T, ik = V dS^T, <S_c, dS> per channel -------------------------------------------
        float iq[4][4], ik[4][4];
        {
            float da[2][4];
#pragma unroll
            for (int n = 0; n < 4; n++) {
                iq[n][0] = iq[n][1] = iq[n][2] = iq[n][3] = 0.f;
                ik[n][0] = ik[n][1] = ik[n][2] = ik[n][3] = 0.f;
            }
#pragma unroll
            for (int n = 0; n < 2; n++) da[n][0] = da[n][1] = da[n][2] = da[n][3] = 0.f;
#pragma unroll
            for (int ks = 0; ks < 8; ks++) {
                uint32_t a[4], b[4];
                frag_a<256>(a, aDO, 16 * mb, ks * 16, lane);
                frag_b_nk<256>(b, aV, ks * 16, 16 * nq, lane);          // dA: columns (keys) 16 * nq ..
                mma16816(da[0], a, b[0], b[1]);
                mma16816(da[1], a, b[2], b[3]);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    frag_b_nk<256>(b, aSc, ks * 16, 32 * nq + 16 * n2, lane);
                    mma16816(iq[2 * n2], a, b[0], b[1]);
                    mma16816(iq[2 * n2 + 1], a, b[2], b[3]);
                }
                frag_a<256>(a, aV, 16 * mb, ks * 16, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    frag_b_nk<256>(b, adSb, ks * 16, 32 * nq + 16 * n2, lane);
                    mma16816(ik[2 * n2], a, b[0], b[1]);
                    mma16816(ik[2 * n2 + 1], a, b[2], b[3]);
                }
            }
            // dA: bf16 copy for the block products, fp32 copy of the diagonal 16-blocks for the pair sums
#pragma unroll
            for (int n = 0; n < 2; n++) {
                const int col = 16 * nq + 8 * n + 2 * tq;
                // the bf16 copy serves products that sum over j <= t (or t >= j) only: zero right of the diagonal
                const bool dg_blk = nq == mb;
                const int jc = (col & 15), tr = g;                       // column and row inside the diagonal block
                const float m0 = !dg_blk || jc <= tr ? da[n][0] : 0.f, m1 = !dg_blk || jc + 1 <= tr ? da[n][1] : 0.f;
                const float m2 = !dg_blk || jc <= tr + 8 ? da[n][2] : 0.f, m3 = !dg_blk || jc + 1 <= tr + 8 ? da[n][3] : 0.f;
                *reinterpret_cast<uint32_t*>(sdAb + sw128(r_lo, col >> 3) + (col & 7) * 2) = pack2(m0, m1);
                *reinterpret_cast<uint32_t*>(sdAb + sw128(r_hi, col >> 3) + (col & 7) * 2) = pack2(m2, m3);
                if (nq == mb) {
                    *reinterpret_cast<float2*>(sdAd + r_lo * 16 + (col & 15)) = make_float2(da[n][0], da[n][1]);
                    *reinterpret_cast<float2*>(sdAd + r_hi * 16 + (col & 15)) = make_float2(da[n][2], da[n][3]);
                }
            }
        }
        {   // <S_c[i,:], dS[i,:]> over this warp's 64 columns of its 16 state rows i (the two column halves meet later)
            const int i0 = (warp & 7) * 16 + g, c0 = (warp >> 3) * 64 + tq * 2;
            float d_lo = 0.f, d_hi = 0.f;
#pragma unroll
            for (int n = 0; n < 8; n++) {
                const float2 s_lo = ld_bf2(sSc, i0, c0 + n * 8), s_hi = ld_bf2(sSc, i0 + 8, c0 + n * 8);
                d_lo += s_lo.x * ds[n][0] + s_lo.y * ds[n][1];
                d_hi += s_hi.x * ds[n][2] + s_hi.y * ds[n][3];
            }
            d_lo += __shfl_xor_sync(0xffffffffu, d_lo, 1); d_lo += __shfl_xor_sync(0xffffffffu, d_lo, 2);
            d_hi += __shfl_xor_sync(0xffffffffu, d_hi, 1); d_hi += __shfl_xor_sync(0xffffffffu, d_hi, 2);
            if (tq == 0) { sRowdot[(warp >> 3) * D + i0] = d_lo; sRowdot[(warp >> 3) * D + i0 + 8] = d_hi; }
        }
        // inter-chunk parts at the fragment positions: iq <- e^{b_t} iq, ik <- ew ik, and sum_j k_j ew_j ik_j per channel
#pragma unroll
        for (int n = 0; n < 4; n++) {
            const int col = 32 * nq + 8 * n + 2 * tq;
            const float2 b_lo = *reinterpret_cast<const float2*>(sB + r_lo * D + col);
            const float2 b_hi = *reinterpret_cast<const float2*>(sB + r_hi * D + col);
            const float2 b_n = *reinterpret_cast<const float2*>(sB + (BT - 1) * D + col);
            const float2 k_lo = ld_bf2(sK, r_lo, col), k_hi = ld_bf2(sK, r_hi, col);
            iq[n][0] *= ex2(b_lo.x); iq[n][1] *= ex2(b_lo.y); iq[n][2] *= ex2(b_hi.x); iq[n][3] *= ex2(b_hi.y);
            ik[n][0] *= ex2(b_n.x - b_lo.x); ik[n][1] *= ex2(b_n.y - b_lo.y);
            ik[n][2] *= ex2(b_n.x - b_hi.x); ik[n][3] *= ex2(b_n.y - b_hi.y);
            float g0 = k_lo.x * ik[n][0] + k_hi.x * ik[n][2], g1 = k_lo.y * ik[n][1] + k_hi.y * ik[n][3];
#pragma unroll
            for (int o = 4; o <= 16; o <<= 1) {
                g0 += __shfl_xor_sync(0xffffffffu, g0, o);
                g1 += __shfl_xor_sync(0xffffffffu, g1, o);
            }
            if (g == 0) *reinterpret_cast<float2*>(sGi + mb * D + col) = make_float2(g0, g1);
        }
        // ---- scores and the anchored operands ------------------------------------------------------------------------
        anchored_operands(sQ, sK, sB, sQa, sKa);
        __syncthreads();                              // S_c is dead from here on; dA and the anchored operands are visible
        unsigned char* sKd = sSc;                     // keys anchored at their own block, over the dead S_c tile
        const uint32_t aKd = aSc;
        if (mild) {
            diag_operand(sK, sB, sKd);
            __syncthreads();
        } else {
            step_factors(sB, sR);                     // over the dead S_c tile as well; read after the next barrier
        }
        scores_off_diagonal(aQa, aKa, sP, warp, lane, mild, aKd);
        // ---- pairs in different blocks -------------------------------------------------------------------------------
        if (mb >= 1 || mild) {   // dq: rows of block mb against the keys of the blocks before it (and, in a mild
                                 // chunk, of its own block: dA is zero right of the diagonal), anchored at block mb
            float acc[4][4];
#pragma unroll
            for (int n = 0; n < 4; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            for (int ks = 0; ks < mb + (mild ? 1 : 0); ks++) {
                uint32_t a[4], b[4];
                frag_a<128>(a, adAb, 16 * mb, 16 * ks, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    if (ks < mb) frag_b_kn<256>(b, aKa, ka_row0(mb) + 16 * ks, 32 * nq + 16 * n2, lane);
                    else frag_b_kn<256>(b, aKd, 16 * mb, 32 * nq + 16 * n2, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
#pragma unroll
            for (int n = 0; n < 4; n++) {
                const int col = 32 * nq + 8 * n + 2 * tq;
                const float2 b_lo = *reinterpret_cast<const float2*>(sB + r_lo * D + col);
                const float2 b_hi = *reinterpret_cast<const float2*>(sB + r_hi * D + col);
                const float2 an = *reinterpret_cast<const float2*>(sB + 16 * mb * D + col);
                iq[n][0] += ex2(b_lo.x - an.x) * acc[n][0]; iq[n][1] += ex2(b_lo.y - an.y) * acc[n][1];
                iq[n][2] += ex2(b_hi.x - an.x) * acc[n][2]; iq[n][3] += ex2(b_hi.y - an.y) * acc[n][3];
            }
        }
        // dk: keys of block mb against the queries of block I (in a mild chunk also I = mb: the factor e^{a_I-b_j} is then
        // >= 1 but bounded), anchored at block I
        for (int I = mild ? mb : mb + 1; I < 4; I++) {
            float acc[4][4];
#pragma unroll
            for (int n = 0; n < 4; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            uint32_t a[4], b[4];
            frag_a_t<128>(a, adAb, 16 * mb, 16 * I, lane);
#pragma unroll
            for (int n2 = 0; n2 < 2; n2++) {
                frag_b_kn<256>(b, aQa, 16 * I, 32 * nq + 16 * n2, lane);
                mma16816(acc[2 * n2], a, b[0], b[1]);
                mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
            }
#pragma unroll
            for (int n = 0; n < 4; n++) {
                const int col = 32 * nq + 8 * n + 2 * tq;
                const float2 b_lo = *reinterpret_cast<const float2*>(sB + r_lo * D + col);
                const float2 b_hi = *reinterpret_cast<const float2*>(sB + r_hi * D + col);
                const float2 an = *reinterpret_cast<const float2*>(sB + 16 * I * D + col);
                ik[n][0] += ex2(an.x - b_lo.x) * acc[n][0]; ik[n][1] += ex2(an.y - b_lo.y) * acc[n][1];
                ik[n][2] += ex2(an.x - b_hi.x) * acc[n][2]; ik[n][3] += ex2(an.y - b_hi.y) * acc[n][3];
            }
        }
        __syncthreads();                              // the anchored operands are dead, the step factors visible
        if (!mild) scores_diagonal(sQ, sK, sR, sP, warp, lane);
#pragma unroll
        for (int n = 0; n < 4; n++) {
            const int col = 32 * nq + 8 * n + 2 * tq;
            *reinterpret_cast<float2*>(sDK + r_lo * D + col) = make_float2(ik[n][0], ik[n][1]);
            *reinterpret_cast<float2*>(sDK + r_hi * D + col) = make_float2(ik[n][2], ik[n][3]);
        }
        __syncthreads();                              // the step factors / own-block keys are dead
#pragma unroll
        for (int n = 0; n < 4; n++) {
            const int col = 32 * nq + 8 * n + 2 * tq;
            *reinterpret_cast<float2*>(sDQ + r_lo * D + col) = make_float2(iq[n][0], iq[n][1]);
            *reinterpret_cast<float2*>(sDQ + r_hi * D + col) = make_float2(iq[n][2], iq[n][3]);
        }
        __syncthreads();

        // ---- pairs inside a 16-block and dg: thread = (channel i, 16-row block blk) --------------------------------------
        {
            const int i = tid & (D - 1), blk = tid >> 7, t0 = 16 * blk;
            float total = 0.f;                            // sum of q dq - k dk over this thread's rows
            if (!mild) {
                // rows ascending; xr[u] = 2^{b_t - b_u} as a running product of the one-step factors (one exponential per
                // row instead of one per pair; every factor <= 1), the same factor for dq and dk
                float dk_acc[16], kf[16], xr[16];
#pragma unroll
                for (int u = 0; u < 16; u++) {
                    dk_acc[u] = 0.f;
                    kf[u] = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sK + sw256(t0 + u, i >> 3) + (i & 7) * 2));
                }
                float b_prev = 0.f;
#pragma unroll
                for (int tt = 0; tt < 16; tt++) {
                    const int t = t0 + tt;
                    const float qt = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sQ + sw256(t, i >> 3) + (i & 7) * 2));
                    const float bt = sB[t * D + i];
                    const float r = ex2(bt - b_prev);
                    b_prev = bt;
                    xr[tt] = 1.f;
                    float dq_acc = 0.f;
#pragma unroll
                    for (int u = 0; u <= tt; u++) {
                        if (u < tt) xr[u] *= r;
                        const float x = sdAd[t * 16 + u] * xr[u];
                        dq_acc += x * kf[u];
                        dk_acc[u] += x * qt;
                    }
                    sDQ[t * D + i] += dq_acc;
                }
#pragma unroll
                for (int tt = 0; tt < 16; tt++) sDK[(t0 + tt) * D + i] += dk_acc[tt];
            }
            // sum of q dq - k dk over this thread's rows
#pragma unroll 4
            for (int tt = 0; tt < 16; tt++) {
                const int t = t0 + tt;
                const float qt = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sQ + sw256(t, i >> 3) + (i & 7) * 2));
                const float kt = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sK + sw256(t, i >> 3) + (i & 7) * 2));
                total += qt * sDQ[t * D + i] - kt * sDK[t * D + i];
            }
            sTmp[blk * D + i] = total;
            __syncthreads();
            // dg_t = suffix over the rows + <S_{c+1}[i,:], dS[i,:]> = e^{b_n} <S_c, dS> + sum_j k_j ew_j ik_j
            float suffix = ex2(sB[(BT - 1) * D + i]) * (sRowdot[i] + sRowdot[D + i]) + sGi[i] + sGi[D + i] + sGi[2 * D + i] +
                           sGi[3 * D + i];
            for (int b2 = 3; b2 > blk; b2--) suffix += sTmp[b2 * D + i];
            for (int t = t0 + 15; t >= t0; t--) {
                const int code = srow[t];
                if (code == -1) continue;
                const float qt = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sQ + sw256(t, i >> 3) + (i & 7) * 2));
                const float kt = __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(sK + sw256(t, i >> 3) + (i & 7) * 2));
                suffix += qt * sDQ[t * D + i] - kt * sDK[t * D + i];
                if (code >= 0) dgk[((size_t)code * H + h) * D + i] = suffix;
                else rg[((size_t)(s.replay_base + t) * H + h) * D + i] = suffix;     // replayed rows sit in chunk 0
            }
        }
        __syncthreads();
        // ---- dq, dk out: own rows as bf16, replayed rows' dk in fp32 to the scratch -------------------------------------
#pragma unroll
        for (int u = 0; u < BT * 16 / NT; u++) {
            const int p = tid + u * NT, t = p >> 4, c16 = p & 15, code = srow[t];
            if (code == -1) continue;
            const float4 q0 = *reinterpret_cast<const float4*>(sDQ + t * D + c16 * 8), q1 = *reinterpret_cast<const float4*>(sDQ + t * D + c16 * 8 + 4);
            const float4 k0 = *reinterpret_cast<const float4*>(sDK + t * D + c16 * 8), k1 = *reinterpret_cast<const float4*>(sDK + t * D + c16 * 8 + 4);
            if (code >= 0) {
                const size_t off = ((size_t)code * H + h) * D + c16 * 8;
                *reinterpret_cast<uint4*>(dq + off) = make_uint4(pack2(q0.x, q0.y), pack2(q0.z, q0.w), pack2(q1.x, q1.y), pack2(q1.z, q1.w));
                *reinterpret_cast<uint4*>(dk_ + off) = make_uint4(pack2(k0.x, k0.y), pack2(k0.z, k0.w), pack2(k1.x, k1.y), pack2(k1.z, k1.w));
            } else {
                float* dst = rk + ((size_t)(s.replay_base + t) * H + h) * D + c16 * 8;
                *reinterpret_cast<float4*>(dst) = k0;
                *reinterpret_cast<float4*>(dst + 4) = k1;
            }
        }
        scale_qk(sQ, sK, sB, sQ, sK);                 // q~, k~ over the raw tiles, which nobody reads any more
        __syncthreads();
        // ---- dv_j = sum_{t>=j} A_tj dO_t + k~_j dS : warp -> rows 16 * mb, columns 32 * nq -------------------------------
        {
            float acc[4][4];
#pragma unroll
            for (int n = 0; n < 4; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            for (int ks = mb; ks < 4; ks++) {             // A_tj = 0 for t < j
                uint32_t a[4], b[4];
                frag_a_t<128>(a, aP, 16 * mb, 16 * ks, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    frag_b_kn<256>(b, aDO, 16 * ks, 32 * nq + 16 * n2, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
#pragma unroll
            for (int ks = 0; ks < 8; ks++) {
                uint32_t a[4], b[4];
                frag_a<256>(a, aK, 16 * mb, 16 * ks, lane);
#pragma unroll
                for (int n2 = 0; n2 < 2; n2++) {
                    frag_b_kn<256>(b, adSb, 16 * ks, 32 * nq + 16 * n2, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
            const int c_lo = srow[r_lo], c_hi = srow[r_hi];
#pragma unroll
            for (int n = 0; n < 4; n++) {
                const int col = 32 * nq + 8 * n + 2 * tq;
                if (c_lo >= 0) *reinterpret_cast<uint32_t*>(dv_ + ((size_t)c_lo * H + h) * D + col) = pack2(acc[n][0], acc[n][1]);
                else if (c_lo < -1) *reinterpret_cast<float2*>(rv + ((size_t)(s.replay_base + r_lo) * H + h) * D + col) = make_float2(acc[n][0], acc[n][1]);
                if (c_hi >= 0) *reinterpret_cast<uint32_t*>(dv_ + ((size_t)c_hi * H + h) * D + col) = pack2(acc[n][2], acc[n][3]);
                else if (c_hi < -1) *reinterpret_cast<float2*>(rv + ((size_t)(s.replay_base + r_hi) * H + h) * D + col) = make_float2(acc[n][2], acc[n][3]);
            }
        }
        // ---- dS <- Diag(e^{b_n}) dS + q~^T dO ---------------------------------------------------------------------------
        state_update(ds, sB, aQ, aDO, warp, lane);
    }
    if (s.init_slot >= 0) {
        state_to_global(ds, ds0 + ((size_t)seq * H + h) * state_elems, warp, lane);
        if constexpr (ONE_LAUNCH) {
            __threadfence();                           // this thread's part, before the flag that follows the barrier
            __syncthreads();
            if (tid == 0) tc::flag_set(ds0_flags + (size_t)seq * H + h);
        }
    }
}

}  // namespace

int32_t gk_mma_supported(int32_t dtype, int32_t dk, int32_t dv) { return dtype == HARTS_BF16 && dk == D && dv == D; }

int32_t gk_mma_fwd(const FwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (cudaFuncSetAttribute(gk_mma_fwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, Shared::fwd_bytes) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    gk_mma_fwd_kernel<false><<<n, NT, Shared::fwd_bytes, a.stream>>>(
        a.tb, a.seq_lo, a.H, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.g,
        (__nv_bfloat16*)a.o, a.slots, (__nv_bfloat16*)a.chunk_states, status_gate(a.flags, a.dev_status), a.dev_status,
        nullptr, nullptr);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

int32_t gk_mma_bwd(const BwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (cudaFuncSetAttribute(gk_mma_bwd_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SharedB::bytes) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    const GkScratchLayout sl = gk_scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    gk_mma_bwd_kernel<false><<<n, NT, SharedB::bytes, a.stream>>>(
        a.tb, a.seq_lo, a.H, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.g,
        (const __nv_bfloat16*)a.dO, (__nv_bfloat16*)a.dq, (__nv_bfloat16*)a.dk_, (__nv_bfloat16*)a.dv_, a.dg,
        (const __nv_bfloat16*)a.chunk_states, (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
        (float*)(base + sl.rg), status_gate(a.flags, a.dev_status), a.dev_status, nullptr, nullptr, RoundOrder{});
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

// All rounds in one launch per pass (sequences [seq_lo, seq_hi) = the whole plan).  flags: n_slots * H (forward) or
// n_seq * H (backward) int32 on the device, ticket: one int32; both zeroed here on the stream.  Offered while the
// problem has few items per SM, like the scalar-gate forms; HARTS_EUNSUPPORTED otherwise.
int32_t gk_mma_fwd_all(const FwdArgs& a, int* flags, int* ticket) {
    const int64_t n = (int64_t)(a.seq_hi - a.seq_lo) * a.H;
    if (n == 0) return HARTS_OK;
    if (n > (int64_t)ONE_LAUNCH_ITEMS_PER_CTA * sm_count()) return HARTS_EUNSUPPORTED;
    if (cudaFuncSetAttribute(gk_mma_fwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, Shared::fwd_bytes) !=
        cudaSuccess)
        return HARTS_ECUDA;
    if (a.tb.n_slots > 0 &&
        cudaMemsetAsync(flags, 0, (size_t)a.tb.n_slots * a.H * sizeof(int), a.stream) != cudaSuccess)
        return HARTS_ECUDA;
    if (cudaMemsetAsync(ticket, 0, sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    gk_mma_fwd_kernel<true><<<(int)n, NT, Shared::fwd_bytes, a.stream>>>(
        a.tb, a.seq_lo, a.H, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.g,
        (__nv_bfloat16*)a.o, a.slots, (__nv_bfloat16*)a.chunk_states, status_gate(a.flags, a.dev_status), a.dev_status,
        flags, ticket);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

int32_t gk_mma_bwd_all(const BwdArgs& a, int* flags, int* ticket, const RoundOrder& rounds) {
    const int64_t n = (int64_t)(a.seq_hi - a.seq_lo) * a.H;
    if (n == 0) return HARTS_OK;
    if (rounds.n < 1 || rounds.ptr[0] != a.seq_lo || rounds.ptr[rounds.n] != a.seq_hi) return HARTS_EINVAL;
    if (n > (int64_t)ONE_LAUNCH_ITEMS_PER_CTA * sm_count()) return HARTS_EUNSUPPORTED;
    if (cudaFuncSetAttribute(gk_mma_bwd_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SharedB::bytes) !=
        cudaSuccess)
        return HARTS_ECUDA;
    if (cudaMemsetAsync(flags, 0, (size_t)a.tb.n_seq * a.H * sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    if (cudaMemsetAsync(ticket, 0, sizeof(int), a.stream) != cudaSuccess) return HARTS_ECUDA;
    const GkScratchLayout sl = gk_scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    gk_mma_bwd_kernel<true><<<(int)n, NT, SharedB::bytes, a.stream>>>(
        a.tb, a.seq_lo, a.H, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.g,
        (const __nv_bfloat16*)a.dO, (__nv_bfloat16*)a.dq, (__nv_bfloat16*)a.dk_, (__nv_bfloat16*)a.dv_, a.dg,
        (const __nv_bfloat16*)a.chunk_states, (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
        (float*)(base + sl.rg), status_gate(a.flags, a.dev_status), a.dev_status, flags, ticket, rounds);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
