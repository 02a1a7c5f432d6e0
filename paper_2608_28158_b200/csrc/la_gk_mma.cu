// Per-channel-decay recurrence (the Diag(gamma) term of Eq. 1, Section 2.2) for bf16 tensors with d_k = d_v = 128:
// the same packed chunkwise call (Eq. 16), plan tables, slots, chunk states and scratch layout as la_gk.cu, with
// every dense product of a chunk on the tensor cores (warp-level mma.sync.m16n8k16, bf16 operands, fp32
// accumulation) and the running state S (forward) / its gradient dS (backward) held in the accumulator registers of
// the CTA's eight warps for the whole walk over a sequence.  What cannot be a dense product stays on the CUDA cores
// in fp32: the decay-dependent pair sums
//     A_tj      = sum_i q_t[i] k_j[i] e^{b_t[i]-b_j[i]}                          (j <= t)
//     dq_t[i]  += sum_{j<=t} dA_tj k_j[i] e^{b_t[i]-b_j[i]},   dk_j[i] += sum_{t>=j} dA_tj q_t[i] e^{b_t[i]-b_j[i]}
// whose exponents are differences of running sums inside the chunk and never positive (no factorisation of
// e^{b_t} e^{-b_j}: no overflow for any gate).  The operands that carry a decay (q~ = q e^{b_t}, k~ = k e^{b_n-b_j},
// the scores A, the states) are rounded to bf16 as in the scalar-gate tensor-core kernels.
//
// Shared-memory tiles of bf16 are row-major with the 16-byte pieces of a row XOR-ed by (row & 7), so that ldmatrix
// (plain and transposed) is free of bank conflicts.
#include "kernels.h"

namespace harts {
namespace {

constexpr int BT = 64;      // chunk rows
constexpr int D = 128;      // d_k = d_v
constexpr int NT = 256;     // threads: 8 warps

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
    uint4 buf[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 4, c16 = p & 15, code = srow[t];
        const bool take = need_own ? code >= 0 : code != -1;
        const int r = code >= 0 ? code : -2 - code;
        buf[u] = take ? *reinterpret_cast<const uint4*>(src + ((size_t)r * H + h) * D + c16 * 8) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < 4; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 4, c16 = p & 15;
        *reinterpret_cast<uint4*>(dst + sw256(t, c16)) = buf[u];
    }
}

// g of the chunk's valid rows (fp32 [rows, H, 128]) into sB [BT][128], zero elsewhere
__device__ __forceinline__ void load_g(const float* gk, int H, int h, const int* srow, float* sB) {
    float4 buf[8];
#pragma unroll
    for (int u = 0; u < 8; u++) {
        const int p = threadIdx.x + u * NT, t = p >> 5, c4 = p & 31, code = srow[t];
        const int r = code >= 0 ? code : -2 - code;
        buf[u] = code != -1 ? *reinterpret_cast<const float4*>(gk + ((size_t)r * H + h) * D + c4 * 4)
                            : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 8; u++) {
        const int p = threadIdx.x + u * NT;
        reinterpret_cast<float4*>(sB)[p] = buf[u];
    }
}

// running sum over the rows, per channel: two threads per channel (rows 0..31 and 32..63), joined through sTmp[128]
__device__ __forceinline__ void cumsum_rows(float* sB, float* sTmp) {
    const int tid = threadIdx.x, i = tid & (D - 1), half = tid >> 7;
    float acc = 0.f;
    for (int t = half * 32; t < half * 32 + 32; t++) {
        acc += sB[t * D + i];
        sB[t * D + i] = acc;
    }
    if (half == 0) sTmp[i] = acc;
    __syncthreads();
    if (half == 1) {
        const float base = sTmp[i];
        for (int t = 32; t < BT; t++) sB[t * D + i] += base;
    }
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
            const float e0 = is_q ? __expf(bs.x - ba.x) : __expf(ba.x - bs.x);
            const float e1 = is_q ? __expf(bs.y - ba.y) : __expf(ba.y - bs.y);
            w[e] = pack2(f.x * e0, f.y * e1);
        }
        // the local row index of a k^(I) sub-tile is dst_row - its row offset; the offsets are multiples of 8, so the
        // swizzle of the stacked tile equals that of the sub-tile
        *reinterpret_cast<uint4*>((is_q ? sQa : sKa) + sw256(dst_row, c16)) = x;
    }
}

// blocks left of the diagonal: warp -> row block I = warp & 3, every second 16-column tile
__device__ __forceinline__ void scores_off_diagonal(uint32_t aQa, uint32_t aKa, unsigned char* sP, int warp, int lane) {
    const int I = warp & 3, g = lane >> 2, tq = lane & 3;
    for (int J = warp >> 2; J < I; J += 2) {
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

// diagonal blocks: one warp per row t, every lane takes 4 channels of all (at most 16) pairs of the row, the warp sums
// them with a transposed reduction; lanes 0..15 then hold A[t][16 I + lane] (zero right of the diagonal)
__device__ __forceinline__ void scores_diagonal(const unsigned char* sQ, const unsigned char* sK, const float* sB,
                                                unsigned char* sP, int warp, int lane) {
    for (int t = warp; t < BT; t += NT / 32) {
        const int j_lo = t & ~15;
        const uint2 qraw = *reinterpret_cast<const uint2*>(sQ + sw256(t, lane >> 1) + (lane & 1) * 8);
        const float4 bt = *reinterpret_cast<const float4*>(sB + t * D + lane * 4);
        const float2 q01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qraw.x));
        const float2 q23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&qraw.y));
        float z[16];
#pragma unroll
        for (int u = 0; u < 16; u++) {
            const int j = j_lo + u;
            float acc = 0.f;
            if (j <= t) {
                const uint2 kraw = *reinterpret_cast<const uint2*>(sK + sw256(j, lane >> 1) + (lane & 1) * 8);
                const float4 bj = *reinterpret_cast<const float4*>(sB + j * D + lane * 4);
                const float2 k01 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kraw.x));
                const float2 k23 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&kraw.y));
                acc = q01.x * k01.x * __expf(bt.x - bj.x);
                acc += q01.y * k01.y * __expf(bt.y - bj.y);
                acc += q23.x * k23.x * __expf(bt.z - bj.z);
                acc += q23.y * k23.y * __expf(bt.w - bj.w);
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
    for (int u = 0; u < 4; u++) {
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
            qw[e] = pack2(qf.x * __expf(bt.x), qf.y * __expf(bt.y));
            kw[e] = pack2(kf.x * __expf(bn.x - bt.x), kf.y * __expf(bn.y - bt.y));
        }
        *reinterpret_cast<uint4*>(dQ + off) = qv;
        *reinterpret_cast<uint4*>(dK + off) = kv;
    }
}

// The state fragments of a warp: rows 16*warp + g and + g + 8 (g = lane / 4), columns 8*n + 2*(lane % 4) + {0, 1} of
// n-tile n: st[n][0..1] = row g, st[n][2..3] = row g + 8.
struct Shared {
    static constexpr int q = 0, k = 16384, v = 32768;          // bf16 [64][128]
    static constexpr int p = 49152;                             // bf16 [64][64]
    static constexpr int sb = 57344;                            // bf16 [128][128]: the state as an MMA operand
    static constexpr int b = 90112;                             // fp32 [64][128]: running log-decay
    static constexpr int tmp = 122880;                          // fp32 [128]
    static constexpr int row = tmp + 512;                       // int  [64]
    static constexpr int qa = 124928;                           // bf16 [64][128]: q anchored at its 16-row block
    static constexpr int ka = qa + 16384;                       // bf16 [96][128]: k anchored at blocks 1, 2, 3
    static constexpr int fwd_bytes = ka + 96 * 256;
};

// state fragments -> bf16 operand tile (swizzled [128][128])
__device__ __forceinline__ void state_to_operand(const float (&st)[16][4], unsigned char* sSb, int warp, int lane) {
    const int g = lane >> 2, tq = lane & 3, r0 = warp * 16 + g;
#pragma unroll
    for (int n = 0; n < 16; n++) {
        *reinterpret_cast<uint32_t*>(sSb + sw256(r0, n) + tq * 4) = pack2(st[n][0], st[n][1]);
        *reinterpret_cast<uint32_t*>(sSb + sw256(r0 + 8, n) + tq * 4) = pack2(st[n][2], st[n][3]);
    }
}
// swizzled bf16 [rows][128] tile -> plain row-major global memory ([rows][128] contiguous), 16 bytes per thread and step
template <int ROWS>
__device__ __forceinline__ void tile_to_global(const unsigned char* tile, __nv_bfloat16* dst) {
    for (int p = threadIdx.x; p < ROWS * 16; p += NT)
        reinterpret_cast<uint4*>(dst)[p] = *reinterpret_cast<const uint4*>(tile + sw256(p >> 4, p & 15));
}

__global__ void __launch_bounds__(NT, 1)
gk_mma_fwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const __nv_bfloat16* __restrict__ q,
                  const __nv_bfloat16* __restrict__ k, const __nv_bfloat16* __restrict__ v, const float* __restrict__ gk,
                  __nv_bfloat16* __restrict__ o, float* __restrict__ slots, __nv_bfloat16* __restrict__ chunk_states,
                  const int32_t* gate) {
    if (gate_closed(gate)) return;
    extern __shared__ __align__(1024) unsigned char sm[];
    unsigned char *sQ = sm + Shared::q, *sK = sm + Shared::k, *sV = sm + Shared::v, *sP = sm + Shared::p,
                  *sSb = sm + Shared::sb;
    float* sB = reinterpret_cast<float*>(sm + Shared::b);
    float* sTmp = reinterpret_cast<float*>(sm + Shared::tmp);
    int* srow = reinterpret_cast<int*>(sm + Shared::row);
    unsigned char *sQa = sm + Shared::qa, *sKa = sm + Shared::ka;
    const uint32_t aQ = s_u32(sQ), aK = s_u32(sK), aV = s_u32(sV), aP = s_u32(sP), aSb = s_u32(sSb);

    const int seq = seq_lo + blockIdx.x / H, h = blockIdx.x % H;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, tq = lane & 3;
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)D * D;

    float st[16][4];                       // S rows 16*warp + g (+8), all 128 columns
    if (s.init_slot < 0) {
#pragma unroll
        for (int n = 0; n < 16; n++) st[n][0] = st[n][1] = st[n][2] = st[n][3] = 0.f;
    } else {
        const float* src = slots + ((size_t)s.init_slot * H + h) * state_elems;
#pragma unroll
        for (int n = 0; n < 16; n++) {
            const float2 lo = *reinterpret_cast<const float2*>(src + (size_t)(warp * 16 + g) * D + n * 8 + tq * 2);
            const float2 hi = *reinterpret_cast<const float2*>(src + (size_t)(warp * 16 + g + 8) * D + n * 8 + tq * 2);
            st[n][0] = lo.x; st[n][1] = lo.y; st[n][2] = hi.x; st[n][3] = hi.y;
        }
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
        // start-of-chunk state: operand copy, kept for the backward, exported when the plan requests this boundary
        state_to_operand(st, sSb, warp, lane);
        if (next_req < s.req_hi && tb.slot_chunk[next_req] == c) {
            float* dst = slots + ((size_t)next_req * H + h) * state_elems;
#pragma unroll
            for (int n = 0; n < 16; n++) {
                *reinterpret_cast<float2*>(dst + (size_t)(warp * 16 + g) * D + n * 8 + tq * 2) = make_float2(st[n][0], st[n][1]);
                *reinterpret_cast<float2*>(dst + (size_t)(warp * 16 + g + 8) * D + n * 8 + tq * 2) = make_float2(st[n][2], st[n][3]);
            }
            next_req++;
        }
        __syncthreads();
        if (chunk_states) tile_to_global<D>(sSb, chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems);
        cumsum_rows(sB, sTmp);
        anchored_operands(sQ, sK, sB, sQa, sKa);
        scores_diagonal(sQ, sK, sB, sP, warp, lane);
        __syncthreads();
        scores_off_diagonal(s_u32(sQa), s_u32(sKa), sP, warp, lane);
        scale_qk(sQ, sK, sB, sQ, sK);
        __syncthreads();
        // ---- o = P V + q~ S_c : warp -> rows 16*(warp & 3), columns 64*(warp >> 2) ---------------------------------
        {
            const int m0 = (warp & 3) * 16, n_base = (warp >> 2) * 64;
            float acc[8][4];
#pragma unroll
            for (int n = 0; n < 8; n++) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
            for (int ks = 0; ks <= (warp & 3); ks++) {      // P is zero right of the diagonal block
                uint32_t a[4];
                frag_a<128>(a, aP, m0, ks * 16, lane);
#pragma unroll
                for (int n2 = 0; n2 < 4; n2++) {
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
                for (int n2 = 0; n2 < 4; n2++) {
                    uint32_t b[4];
                    frag_b_kn<256>(b, aSb, ks * 16, n_base + n2 * 16, lane);
                    mma16816(acc[2 * n2], a, b[0], b[1]);
                    mma16816(acc[2 * n2 + 1], a, b[2], b[3]);
                }
            }
            const int c_lo = srow[m0 + g], c_hi = srow[m0 + g + 8];
#pragma unroll
            for (int n = 0; n < 8; n++) {
                const int col = n_base + n * 8 + tq * 2;
                if (c_lo >= 0) *reinterpret_cast<uint32_t*>(o + ((size_t)c_lo * H + h) * D + col) = pack2(acc[n][0], acc[n][1]);
                if (c_hi >= 0) *reinterpret_cast<uint32_t*>(o + ((size_t)c_hi * H + h) * D + col) = pack2(acc[n][2], acc[n][3]);
            }
        }
        // ---- S <- Diag(e^{b_n}) S + k~^T V : warp -> state rows 16*warp .. ------------------------------------------
        {
            const float g_lo = __expf(sB[(BT - 1) * D + warp * 16 + g]), g_hi = __expf(sB[(BT - 1) * D + warp * 16 + g + 8]);
#pragma unroll
            for (int n = 0; n < 16; n++) {
                st[n][0] *= g_lo; st[n][1] *= g_lo; st[n][2] *= g_hi; st[n][3] *= g_hi;
            }
#pragma unroll
            for (int ks = 0; ks < 4; ks++) {
                uint32_t a[4];
                frag_a_t<256>(a, aK, warp * 16, ks * 16, lane);
#pragma unroll
                for (int n2 = 0; n2 < 8; n2++) {
                    uint32_t b[4];
                    frag_b_kn<256>(b, aV, ks * 16, n2 * 16, lane);
                    mma16816(st[2 * n2], a, b[0], b[1]);
                    mma16816(st[2 * n2 + 1], a, b[2], b[3]);
                }
            }
        }
    }
}

}  // namespace

int32_t gk_mma_supported(int32_t dtype, int32_t dk, int32_t dv) { return dtype == HARTS_BF16 && dk == D && dv == D; }

int32_t gk_mma_fwd(const FwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (cudaFuncSetAttribute(gk_mma_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, Shared::fwd_bytes) !=
        cudaSuccess)
        return HARTS_ECUDA;
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    gk_mma_fwd_kernel<<<n, NT, Shared::fwd_bytes, a.stream>>>(
        a.tb, a.seq_lo, a.H, (const __nv_bfloat16*)a.q, (const __nv_bfloat16*)a.k, (const __nv_bfloat16*)a.v, a.g,
        (__nv_bfloat16*)a.o, a.slots, (__nv_bfloat16*)a.chunk_states, status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
