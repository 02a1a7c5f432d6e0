// fp32-FMA kernels for the packed chunkwise call (Eq. 16): the path for fp32 inputs and the
// on-device cross-check for the tensor-core kernels.  One CTA per (sequence, head) walks the
// sequence's chunks in order; everything inside a chunk lives in shared memory.
//
// Chunk formulas (derived from the token recurrence S_t = e^{g_t} S_{t-1} + k_t^T v_t,
// o_t = q_t S_t; b_t is the running sum of g inside the chunk, n its last row):
//   A_tj = (q_t . k_j) e^{b_t - b_j}  (j <= t),   o_t = e^{b_t} q_t S_c + sum_j A_tj v_j
//   S_{c+1} = e^{b_n} S_c + sum_j e^{b_n - b_j} k_j^T v_j
// backward (dS is the gradient w.r.t. the state at the END of the chunk on entry):
//   dA_tj = (dO_t . v_j) e^{b_t - b_j}  (j <= t)
//   dq_t = e^{b_t} dO_t S_c^T + sum_j dA_tj k_j
//   dk_j = sum_t dA_tj q_t + e^{b_n - b_j} v_j dS^T
//   dv_j = sum_t A_tj dO_t + e^{b_n - b_j} k_j dS
//   dg_t = sum_{tau >= t} (q_tau . dq_tau - k_tau . dk_tau) + <S_{c+1}, dS>
//   dS  <- e^{b_n} dS + sum_t e^{b_t} q_t^T dO_t            (gradient at the START of the chunk)
// A sequence's virtual rows are its replay rows (gathered by physical row id, state update only,
// Section 3.4 "Round-wise execution") followed by its own rows; chunk c covers virtual rows
// [64c, 64c+64).
#include "kernels.h"

namespace harts {
namespace {

constexpr int BT = 64;
constexpr int NT = 256;

template <typename T> __device__ __forceinline__ float to_f(T x);
template <> __device__ __forceinline__ float to_f<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Shared-memory index swizzles: both "lanes walk a row" and "lanes walk a column" stay (nearly)
// bank-conflict free.
template <int D> __device__ __forceinline__ int tix(int t, int i) { return t * D + (i ^ (t & 31)); }

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

// physical row of virtual row j (or -1 past the end); own = produces an output
__device__ __forceinline__ int virtual_row(const harts_la_tables_t& tb, const SeqInfo& s, int j, bool& own) {
    own = false;
    if (j >= s.n_virtual) return -1;
    if (j < s.n_replay) return tb.replay_row[s.replay_base + j];
    own = true;
    return s.own_begin + (j - s.n_replay);
}

// Loads one chunk: row ids, k/v (all valid rows), q and dO (own rows only, zero otherwise), and
// the in-chunk running sum of g.  Rows past the end are zero with g = 0.
template <typename T, int DK, int DV, bool BWD>
__device__ void load_chunk(const harts_la_tables_t& tb, const SeqInfo& s, int c, int h, int H, const T* q,
                           const T* k, const T* v, const float* g, const T* dO, T* sq, T* sk, T* sv, T* sdo,
                           float* sb, int* srow) {
    const int tid = threadIdx.x;
    if (tid < BT) {
        bool own;
        int r = virtual_row(tb, s, c * BT + tid, own);
        srow[tid] = r < 0 ? -1 : (own ? r : -2 - r);          // replay rows are stored as -2 - row
        sb[tid] = r < 0 ? 0.f : g[(size_t)r * H + h];
    }
    __syncthreads();
    for (int e = tid; e < BT * DK; e += NT) {
        int t = e / DK, i = e % DK, code = srow[t];
        int r = code >= 0 ? code : -2 - code;
        sk[tix<DK>(t, i)] = code == -1 ? from_f<T>(0.f) : k[((size_t)r * H + h) * DK + i];
        sq[tix<DK>(t, i)] = code >= 0 ? q[((size_t)r * H + h) * DK + i] : from_f<T>(0.f);
    }
    for (int e = tid; e < BT * DV; e += NT) {
        int t = e / DV, j = e % DV, code = srow[t];
        int r = code >= 0 ? code : -2 - code;
        sv[tix<DV>(t, j)] = code == -1 ? from_f<T>(0.f) : v[((size_t)r * H + h) * DV + j];
        if (BWD) sdo[tix<DV>(t, j)] = code >= 0 ? dO[((size_t)r * H + h) * DV + j] : from_f<T>(0.f);
    }
    if (tid == 0) {
        float acc = 0.f;
        for (int t = 0; t < BT; t++) {
            acc += sb[t];
            sb[t] = acc;
        }
    }
    __syncthreads();
}

template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) fma_fwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const T* q,
                                                     const T* k, const T* v, const float* g, T* o, float* slots,
                                                     T* chunk_states, const int32_t* gate) {
    if (gate_closed(gate)) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sS = reinterpret_cast<float*>(smem_raw);       // [DK][DV]
    float* sA = sS + DK * DV;                             // [BT][BT+1]
    float* sb = sA + BT * (BT + 1);                       // [BT]
    int* srow = reinterpret_cast<int*>(sb + BT);          // [BT]
    T* sq = reinterpret_cast<T*>(srow + BT);              // [BT][DK]
    T* sk = sq + BT * DK;
    T* sv = sk + BT * DK;                                 // [BT][DV]

    const int seq = seq_lo + blockIdx.x / H, h = blockIdx.x % H;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)DK * DV;

    for (int e = tid; e < DK * DV; e += NT)
        sS[tix<DV>(e / DV, e % DV)] = s.init_slot < 0 ? 0.f : slots[((size_t)s.init_slot * H + h) * state_elems + e];
    __syncthreads();

    int next_req = s.req_lo;
    for (int c = 0; c < s.n_chunks; c++) {
        load_chunk<T, DK, DV, false>(tb, s, c, h, H, q, k, v, g, nullptr, sq, sk, sv, nullptr, sb, srow);
        // start-of-chunk state: kept for the backward; exported when the plan requests this boundary
        if (chunk_states) {
            T* dst = chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems;
            for (int e = tid; e < DK * DV; e += NT) dst[e] = from_f<T>(sS[tix<DV>(e / DV, e % DV)]);
        }
        if (next_req < s.req_hi && tb.slot_chunk[next_req] == c) {
            float* dst = slots + ((size_t)next_req * H + h) * state_elems;
            for (int e = tid; e < DK * DV; e += NT) dst[e] = sS[tix<DV>(e / DV, e % DV)];
            next_req++;
        }
        // A = (Q K^T) .* decay, lower triangle
        for (int r = 0; r < 4; r++) {
            int t = ty * 4 + r;
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int i = 0; i < DK; i++) {
                float qv = to_f(sq[tix<DK>(t, i)]);
#pragma unroll
                for (int cc = 0; cc < 4; cc++) acc[cc] += qv * to_f(sk[tix<DK>(tx + 16 * cc, i)]);
            }
#pragma unroll
            for (int cc = 0; cc < 4; cc++) {
                int j = tx + 16 * cc;
                sA[t * (BT + 1) + j] = j <= t ? acc[cc] * __expf(sb[t] - sb[j]) : 0.f;
            }
        }
        __syncthreads();
        // o = e^{b_t} q S_c + A v
        for (int r = 0; r < 4; r++) {
            int t = ty * 4 + r;
            int code = srow[t];
            if (code < 0) continue;
            float acc[DV / 16], acc2[DV / 16];
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) acc[cc] = acc2[cc] = 0.f;
            for (int i = 0; i < DK; i++) {
                float qv = to_f(sq[tix<DK>(t, i)]);
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc[cc] += qv * sS[tix<DV>(i, tx + 16 * cc)];
            }
            for (int j = 0; j <= t; j++) {
                float a = sA[t * (BT + 1) + j];
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc2[cc] += a * to_f(sv[tix<DV>(j, tx + 16 * cc)]);
            }
            float eb = __expf(sb[t]);
            T* dst = o + ((size_t)code * H + h) * DV;
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) dst[tx + 16 * cc] = from_f<T>(eb * acc[cc] + acc2[cc]);
        }
        __syncthreads();
        // S <- e^{b_n} S + sum_j e^{b_n - b_j} k_j^T v_j
        {
            float bn = sb[BT - 1];
            float acc[DK / 16][DV / 16];
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) acc[ri][cj] = 0.f;
            for (int j = 0; j < BT; j++) {
                float w = __expf(bn - sb[j]);
                float kv[DK / 16];
#pragma unroll
                for (int ri = 0; ri < DK / 16; ri++) kv[ri] = w * to_f(sk[tix<DK>(j, ty + 16 * ri)]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    float vv = to_f(sv[tix<DV>(j, tx + 16 * cj)]);
#pragma unroll
                    for (int ri = 0; ri < DK / 16; ri++) acc[ri][cj] += kv[ri] * vv;
                }
            }
            float gam = __expf(bn);
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    int e = tix<DV>(ty + 16 * ri, tx + 16 * cj);
                    sS[e] = gam * sS[e] + acc[ri][cj];
                }
        }
        __syncthreads();
    }
}

template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) fma_bwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const T* q,
                                                     const T* k, const T* v, const float* g, const T* dO, T* dq,
                                                     T* dk_, T* dv_, float* dg, const T* chunk_states,
                                                     float* ds0, float* rk, float* rv, float* rg, const int32_t* gate) {
    if (gate_closed(gate)) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sS = reinterpret_cast<float*>(smem_raw);       // S_c           [DK][DV]
    float* sdS = sS + DK * DV;                            // dS            [DK][DV]
    float* sP = sdS + DK * DV;                            // A             [BT][BT+1]
    float* sdP = sP + BT * (BT + 1);                      // dA            [BT][BT+1]
    float* sb = sdP + BT * (BT + 1);                      // [BT]
    float* sr = sb + BT;                                  // q.dq - k.dk per row [BT]
    float* sred = sr + BT;                                // [8] block reduction
    int* srow = reinterpret_cast<int*>(sred + 8);         // [BT]
    T* sq = reinterpret_cast<T*>(srow + BT);
    T* sk = sq + BT * DK;
    T* sv = sk + BT * DK;
    T* sdo = sv + BT * DV;

    const int seq = seq_lo + blockIdx.x / H, h = blockIdx.x % H;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)DK * DV;

    for (int e = tid; e < DK * DV; e += NT) sdS[e] = 0.f;
    __syncthreads();

    int next_req = s.req_hi - 1;     // slots of this sequence are ordered by chunk index
    for (int c = s.n_chunks - 1; c >= 0; c--) {
        // gradient arriving at boundary c+1 from the sequences that started there
        if (next_req >= s.req_lo && tb.slot_chunk[next_req] == c + 1) {
            // all consumers' gradients were summed into the first consumer's buffer by handoff_reduce
            if (tb.slot_cons_ptr[next_req] < tb.slot_cons_ptr[next_req + 1]) {
                const float* src = ds0 + ((size_t)tb.slot_cons_seq[tb.slot_cons_ptr[next_req]] * H + h) * state_elems;
                for (int e = tid; e < DK * DV; e += NT) sdS[tix<DV>(e / DV, e % DV)] += src[e];
            }
            next_req--;
        }
        load_chunk<T, DK, DV, true>(tb, s, c, h, H, q, k, v, g, dO, sq, sk, sv, sdo, sb, srow);
        {
            const T* src = chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems;
            for (int e = tid; e < DK * DV; e += NT) sS[tix<DV>(e / DV, e % DV)] = to_f(src[e]);
        }
        if (tid < BT) sr[tid] = 0.f;
        // A and dA, decay-masked lower triangles
        for (int r = 0; r < 4; r++) {
            int t = ty * 4 + r;
            float acc[4] = {0.f, 0.f, 0.f, 0.f}, dacc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int i = 0; i < DK; i++) {
                float qv = to_f(sq[tix<DK>(t, i)]);
#pragma unroll
                for (int cc = 0; cc < 4; cc++) acc[cc] += qv * to_f(sk[tix<DK>(tx + 16 * cc, i)]);
            }
            for (int j = 0; j < DV; j++) {
                float dov = to_f(sdo[tix<DV>(t, j)]);
#pragma unroll
                for (int cc = 0; cc < 4; cc++) dacc[cc] += dov * to_f(sv[tix<DV>(tx + 16 * cc, j)]);
            }
#pragma unroll
            for (int cc = 0; cc < 4; cc++) {
                int j = tx + 16 * cc;
                float w = j <= t ? __expf(sb[t] - sb[j]) : 0.f;
                sP[t * (BT + 1) + j] = acc[cc] * w;
                sdP[t * (BT + 1) + j] = dacc[cc] * w;
            }
        }
        __syncthreads();
        const float bn = sb[BT - 1];
        float g_inter = 0.f;      // this thread's share of sum_j k_j . dk_j(inter)
        // dq and dk: rows ty*4+r, columns tx + 16*cc
        for (int r = 0; r < 4; r++) {
            int t = ty * 4 + r;
            int code = srow[t];
            if (code == -1) continue;
            float aq[DK / 16], ak[DK / 16], ai[DK / 16];
#pragma unroll
            for (int cc = 0; cc < DK / 16; cc++) aq[cc] = ak[cc] = ai[cc] = 0.f;
            for (int j = 0; j < DV; j++) {
                float dov = to_f(sdo[tix<DV>(t, j)]), vv = to_f(sv[tix<DV>(t, j)]);
#pragma unroll
                for (int cc = 0; cc < DK / 16; cc++) {
                    int i = tx + 16 * cc;
                    aq[cc] += dov * sS[tix<DV>(i, j)];
                    ai[cc] += vv * sdS[tix<DV>(i, j)];
                }
            }
            float eb = __expf(sb[t]), ew = __expf(bn - sb[t]);
#pragma unroll
            for (int cc = 0; cc < DK / 16; cc++) {
                aq[cc] *= eb;
                ai[cc] *= ew;
            }
            for (int j = 0; j <= t; j++) {
                float w = sdP[t * (BT + 1) + j];
#pragma unroll
                for (int cc = 0; cc < DK / 16; cc++) aq[cc] += w * to_f(sk[tix<DK>(j, tx + 16 * cc)]);
            }
            for (int u = t; u < BT; u++) {
                float w = sdP[u * (BT + 1) + t];
#pragma unroll
                for (int cc = 0; cc < DK / 16; cc++) ak[cc] += w * to_f(sq[tix<DK>(u, tx + 16 * cc)]);
            }
            float rsum = 0.f;
#pragma unroll
            for (int cc = 0; cc < DK / 16; cc++) {
                int i = tx + 16 * cc;
                float qv = to_f(sq[tix<DK>(t, i)]), kv = to_f(sk[tix<DK>(t, i)]);
                float dkv = ak[cc] + ai[cc];
                rsum += qv * aq[cc] - kv * dkv;
                g_inter += kv * ai[cc];
                if (code >= 0) {
                    dq[((size_t)code * H + h) * DK + i] = from_f<T>(aq[cc]);
                    dk_[((size_t)code * H + h) * DK + i] = from_f<T>(dkv);
                } else {
                    rk[((size_t)(s.replay_base + c * BT + t) * H + h) * DK + i] = dkv;   // replay rows sit in chunk 0
                }
            }
            // the 16 threads of a row are one half of a warp: fixed-order butterfly, one writer (no atomics)
            const unsigned half_mask = 0xffffu << (tid & 16);
#pragma unroll
            for (int o_ = 8; o_ > 0; o_ >>= 1) rsum += __shfl_xor_sync(half_mask, rsum, o_);
            if (tx == 0) sr[t] = rsum;
        }
        // dv
        for (int r = 0; r < 4; r++) {
            int t = ty * 4 + r;
            int code = srow[t];
            if (code == -1) continue;
            float av[DV / 16], ai[DV / 16];
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) av[cc] = ai[cc] = 0.f;
            for (int i = 0; i < DK; i++) {
                float kv = to_f(sk[tix<DK>(t, i)]);
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) ai[cc] += kv * sdS[tix<DV>(i, tx + 16 * cc)];
            }
            float ew = __expf(bn - sb[t]);
            for (int u = t; u < BT; u++) {
                float w = sP[u * (BT + 1) + t];
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) av[cc] += w * to_f(sdo[tix<DV>(u, tx + 16 * cc)]);
            }
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) {
                int j = tx + 16 * cc;
                float val = av[cc] + ew * ai[cc];
                if (code >= 0) dv_[((size_t)code * H + h) * DV + j] = from_f<T>(val);
                else rv[((size_t)(s.replay_base + c * BT + t) * H + h) * DV + j] = val;
            }
        }
        // <S_{c+1}, dS> = e^{b_n} <S_c, dS> + sum_j k_j . dk_j(inter)
        {
            float part = 0.f;
            for (int e = tid; e < DK * DV; e += NT) part += sS[e] * sdS[e];
            part = __expf(bn) * part + g_inter;
            for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
            if (tid % 32 == 0) sred[tid / 32] = part;
        }
        __syncthreads();
        if (tid < BT) {
            float G = 0.f;
            for (int w = 0; w < NT / 32; w++) G += sred[w];
            float suffix = 0.f;
            for (int u = tid; u < BT; u++) suffix += sr[u];
            int code = srow[tid];
            if (code >= 0) dg[(size_t)code * H + h] = suffix + G;
            else if (code < -1) rg[(size_t)(s.replay_base + c * BT + tid) * H + h] = suffix + G;
        }
        // dS <- e^{b_n} dS + sum_t e^{b_t} q_t^T dO_t
        {
            float acc[DK / 16][DV / 16];
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) acc[ri][cj] = 0.f;
            for (int t = 0; t < BT; t++) {
                float w = __expf(sb[t]);
                float qv[DK / 16];
#pragma unroll
                for (int ri = 0; ri < DK / 16; ri++) qv[ri] = w * to_f(sq[tix<DK>(t, ty + 16 * ri)]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    float dov = to_f(sdo[tix<DV>(t, tx + 16 * cj)]);
#pragma unroll
                    for (int ri = 0; ri < DK / 16; ri++) acc[ri][cj] += qv[ri] * dov;
                }
            }
            float gam = __expf(bn);
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    int e = tix<DV>(ty + 16 * ri, tx + 16 * cj);
                    sdS[e] = gam * sdS[e] + acc[ri][cj];
                }
        }
        __syncthreads();
    }
    if (s.init_slot >= 0) {
        float* dst = ds0 + ((size_t)seq * H + h) * state_elems;
        for (int e = tid; e < DK * DV; e += NT) dst[e] = sdS[tix<DV>(e / DV, e % DV)];
    }
}

// dk/dv/dg of a replayed row += the contributions of every sequence that replayed it (summed in table order).  A group
// of (DK + DV) / 4 threads serves one (row, head): every thread owns four consecutive channels of dk or dv (16-byte
// loads of the fp32 contributions), the group's first thread the scalar dg as well.
template <typename T>
__device__ __forceinline__ void add4(T* p, const float4& a);
template <>
__device__ __forceinline__ void add4<float>(float* p, const float4& a) {
    float4 x = *reinterpret_cast<float4*>(p);
    x.x += a.x; x.y += a.y; x.z += a.z; x.w += a.w;
    *reinterpret_cast<float4*>(p) = x;
}
template <>
__device__ __forceinline__ void add4<__nv_bfloat16>(__nv_bfloat16* p, const float4& a) {
    uint2 raw = *reinterpret_cast<uint2*>(p);
    __nv_bfloat162* h2 = reinterpret_cast<__nv_bfloat162*>(&raw);
    float2 lo = __bfloat1622float2(h2[0]), hi = __bfloat1622float2(h2[1]);
    h2[0] = __floats2bfloat162_rn(lo.x + a.x, lo.y + a.y);
    h2[1] = __floats2bfloat162_rn(hi.x + a.z, hi.y + a.w);
    *reinterpret_cast<uint2*>(p) = raw;
}

template <typename T>
__global__ void replay_reduce_kernel(harts_la_tables_t tb, int H, int DK, int DV, T* dk_, T* dv_, float* dg,
                                     const float* rk, const float* rv, const float* rg, int n_items) {
    const int per = (DK + DV) / 4;
    const int item = blockIdx.x * (blockDim.x / per) + threadIdx.x / per, part = threadIdx.x % per;
    if (item >= n_items) return;
    const int m = item / H, h = item % H;
    const int row = tb.rg_row[m];
    const int lo = tb.rg_ptr[m], hi = tb.rg_ptr[m + 1];
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (part * 4 < DK) {
        const int i = part * 4;
        for (int e = lo; e < hi; e++) {
            const float4 x = *reinterpret_cast<const float4*>(rk + ((size_t)tb.rg_entry[e] * H + h) * DK + i);
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
        add4<T>(dk_ + ((size_t)row * H + h) * DK + i, acc);
    } else {
        const int j = part * 4 - DK;
        for (int e = lo; e < hi; e++) {
            const float4 x = *reinterpret_cast<const float4*>(rv + ((size_t)tb.rg_entry[e] * H + h) * DV + j);
            acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
        }
        add4<T>(dv_ + ((size_t)row * H + h) * DV + j, acc);
    }
    if (part == 0) {
        float g = 0.f;
        for (int e = lo; e < hi; e++) g += rg[(size_t)tb.rg_entry[e] * H + h];
        dg[(size_t)row * H + h] += g;
    }
}

template <typename T, int DK, int DV>
constexpr size_t fwd_smem() {
    return sizeof(float) * (DK * DV + BT * (BT + 1) + BT) + sizeof(int) * BT + sizeof(T) * (2 * BT * DK + BT * DV);
}
template <typename T, int DK, int DV>
constexpr size_t bwd_smem() {
    return sizeof(float) * (2 * DK * DV + 2 * BT * (BT + 1) + 2 * BT + 8) + sizeof(int) * BT +
           sizeof(T) * (2 * BT * DK + 2 * BT * DV);
}

template <typename T, int DK, int DV>
int32_t launch_fwd(const FwdArgs& a) {
    auto kern = fma_fwd_kernel<T, DK, DV>;
    constexpr size_t smem = fwd_smem<T, DK, DV>();
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return HARTS_ECUDA;
    int n = (a.seq_hi - a.seq_lo) * a.H;
    kern<<<n, NT, smem, a.stream>>>(a.tb, a.seq_lo, a.H, (const T*)a.q, (const T*)a.k, (const T*)a.v, a.g, (T*)a.o,
                                    a.slots, (T*)a.chunk_states, status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

template <typename T, int DK, int DV>
int32_t launch_bwd(const BwdArgs& a) {
    auto kern = fma_bwd_kernel<T, DK, DV>;
    constexpr size_t smem = bwd_smem<T, DK, DV>();
    static_assert(smem <= 232448, "backward tile does not fit in shared memory");
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return HARTS_ECUDA;
    int n = (a.seq_hi - a.seq_lo) * a.H;
    ScratchLayout sl = scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    kern<<<n, NT, smem, a.stream>>>(a.tb, a.seq_lo, a.H, (const T*)a.q, (const T*)a.k, (const T*)a.v, a.g,
                                    (const T*)a.dO, (T*)a.dq, (T*)a.dk_, (T*)a.dv_, a.dg, (const T*)a.chunk_states,
                                    (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
                                    (float*)(base + sl.rg), status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace

int32_t fma_supported(int32_t dtype, int32_t dk, int32_t dv) {
    if (dtype == HARTS_FP32) return dk == 64 && dv == 64;
    if (dtype == HARTS_BF16) return (dk == 64 && dv == 64) || (dk == 128 && dv == 128);
    return 0;
}

int32_t fma_fwd(const FwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (a.dtype == HARTS_FP32 && a.dk == 64 && a.dv == 64) return launch_fwd<float, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 64 && a.dv == 64) return launch_fwd<__nv_bfloat16, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 128 && a.dv == 128) return launch_fwd<__nv_bfloat16, 128, 128>(a);
    return HARTS_EUNSUPPORTED;
}

// Sums the initial-state gradients of all sequences that started from one exported boundary (Section 3.4: several
// consumers of one boundary tensor are summed) into the first consumer's buffer, for the boundaries that the
// sequences [seq_lo, seq_hi) exported: a bandwidth-bound pass, in consumer order (deterministic), so that the
// backward kernels add one tensor per boundary instead of walking the consumer list under their own latency.
__global__ void __launch_bounds__(256) handoff_reduce_kernel(const harts_la_tables_t tb, int seq_lo, int seq_hi, int H,
                                                             int elems, float* __restrict__ ds0, const int32_t* gate) {
    if (gate_closed(gate)) return;
    const int slot = blockIdx.x;
    if (slot < tb.seq_req_ptr[seq_lo] || slot >= tb.seq_req_ptr[seq_hi]) return;
    const int c0 = tb.slot_cons_ptr[slot], c1 = tb.slot_cons_ptr[slot + 1];
    if (c1 - c0 < 2) return;
    const int h = blockIdx.y;
    float4* dst = reinterpret_cast<float4*>(ds0 + ((size_t)tb.slot_cons_seq[c0] * H + h) * elems);
    for (int e = blockIdx.z * 256 + threadIdx.x; e < elems / 4; e += gridDim.z * 256) {
        float4 acc = dst[e];
        int u = c0 + 1;
        for (; u + 3 < c1; u += 4) {              // four independent loads in flight
            float4 v[4];
#pragma unroll
            for (int i = 0; i < 4; i++)
                v[i] = reinterpret_cast<const float4*>(ds0 + ((size_t)tb.slot_cons_seq[u + i] * H + h) * elems)[e];
#pragma unroll
            for (int i = 0; i < 4; i++) {
                acc.x += v[i].x; acc.y += v[i].y; acc.z += v[i].z; acc.w += v[i].w;
            }
        }
        for (; u < c1; u++) {
            const float4 v = reinterpret_cast<const float4*>(ds0 + ((size_t)tb.slot_cons_seq[u] * H + h) * elems)[e];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
        }
        dst[e] = acc;
    }
}

int32_t handoff_reduce(const BwdArgs& a) {
    if (a.tb.n_slots == 0 || a.seq_hi == a.seq_lo) return HARTS_OK;
    ScratchLayout sl = scratch_layout(a.tb, a.H, a.dk, a.dv);
    float* ds0 = reinterpret_cast<float*>(static_cast<char*>(a.scratch) + sl.ds0);
    const int elems = a.dk * a.dv;
    dim3 grid(a.tb.n_slots, a.H, (elems / 4 + 1023) / 1024);
    handoff_reduce_kernel<<<grid, 256, 0, a.stream>>>(a.tb, a.seq_lo, a.seq_hi, a.H, elems, ds0,
                                                      status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

int32_t fma_bwd(const BwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (int32_t rc = handoff_reduce(a); rc != HARTS_OK) return rc;
    if (a.dtype == HARTS_FP32 && a.dk == 64 && a.dv == 64) return launch_bwd<float, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 64 && a.dv == 64) return launch_bwd<__nv_bfloat16, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 128 && a.dv == 128) return launch_bwd<__nv_bfloat16, 128, 128>(a);
    return HARTS_EUNSUPPORTED;
}

int32_t replay_reduce(const harts_la_tables_t& tb, void* dk_, void* dv_, float* dg, const void* scratch, int32_t H,
                      int32_t dk, int32_t dv, int32_t dtype, cudaStream_t stream) {
    if (tb.n_rg_rows == 0) return HARTS_OK;
    ScratchLayout sl = scratch_layout(tb, H, dk, dv);
    const char* base = static_cast<const char*>(scratch);
    const float* rk = (const float*)(base + sl.rk);
    const float* rv = (const float*)(base + sl.rv);
    const float* rg = (const float*)(base + sl.rg);
    const int n = tb.n_rg_rows * H, per = (dk + dv) / 4, threads = 256;
    if ((dk + dv) % 4 != 0 || dk % 4 != 0 || threads % per != 0) return HARTS_EUNSUPPORTED;
    const int blocks = (n + threads / per - 1) / (threads / per);
    if (dtype == HARTS_FP32)
        replay_reduce_kernel<float><<<blocks, threads, 0, stream>>>(tb, H, dk, dv, (float*)dk_, (float*)dv_, dg, rk, rv, rg, n);
    else
        replay_reduce_kernel<__nv_bfloat16><<<blocks, threads, 0, stream>>>(tb, H, dk, dv, (__nv_bfloat16*)dk_,
                                                                            (__nv_bfloat16*)dv_, dg, rk, rv, rg, n);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
