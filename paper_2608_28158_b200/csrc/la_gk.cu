// Packed chunkwise call (Eq. 16) for the recurrence with a PER-CHANNEL decay, the Diag(gamma) term of Eq. 1
// (Section 2.2):   S_t = Diag(e^{g_t}) S_{t-1} + k_t^T v_t,   o_t = q_t S_t,   g_t in R^{d_k}.
// Same plan, slots, replay rows, chunk states and hand-off gradients as the scalar-gate kernels; only the chunk
// arithmetic differs.  fp32 arithmetic on the CUDA cores, one CTA per (sequence, head), everything of a chunk in
// shared memory.  With b_t[i] the running sum of g[.][i] inside the chunk and n its last row:
//   A_tj   = sum_i q_t[i] k_j[i] e^{b_t[i] - b_j[i]}                    (j <= t; every exponent <= 0, no factorisation
//                                                                       of e^{b_t} e^{-b_j}, hence no overflow for any gate)
//   o_t    = (q_t .* e^{b_t}) S_c + sum_{j<=t} A_tj v_j
//   S_{c+1} = Diag(e^{b_n}) S_c + sum_j (k_j .* e^{b_n - b_j})^T v_j
// backward (dS = gradient w.r.t. the state at the END of the chunk on entry, dA_tj = dO_t . v_j):
//   dq_t[i] = e^{b_t[i]} (dO_t S_c^T)[i] + sum_{j<=t} dA_tj k_j[i] e^{b_t[i]-b_j[i]}
//   dk_j[i] = e^{b_n[i]-b_j[i]} (v_j dS^T)[i] + sum_{t>=j} dA_tj q_t[i] e^{b_t[i]-b_j[i]}
//   dv_j    = sum_{t>=j} A_tj dO_t + (k_j .* e^{b_n-b_j}) dS
//   dg_t[i] = sum_{tau>=t} (q_tau[i] dq_tau[i] - k_tau[i] dk_tau[i]) + <S_{c+1}[i,:], dS[i,:]>
//   dS     <- Diag(e^{b_n}) dS + sum_t (q_t .* e^{b_t})^T dO_t
// In the backward a pair of threads owns one key channel i for the decay-dependent sums, so that every
// e^{b_t[i]-b_j[i]} is evaluated once and serves dq and dk alike.
#include "kernels.h"

namespace harts {
namespace {

constexpr int BT = 64;
constexpr int NT = 256;
constexpr int N_PAIRS = BT * (BT + 1) / 2;

template <typename T> __device__ __forceinline__ float to_f(T x);
template <> __device__ __forceinline__ float to_f<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// [rows][D] tiles with the column index rotated by the row, so that "lanes walk a row" and "lanes walk a column"
// both spread over the banks
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

// One [BT][D] tile of a [rows, H, D] tensor into shared memory: every thread fetches its 16-byte pieces first (all in
// flight together), then scatters them element by element into the rotated layout.  need_own: only rows with an
// output are taken (q, dO); otherwise every valid row (k, v).  Rows that are not taken become zero.
template <typename T, int D, bool ROTATED, typename Dst>
__device__ __forceinline__ void load_tile(const T* src, int H, int h, const int* srow, bool need_own, Dst* dst) {
    constexpr int VE = 16 / sizeof(T);                    // elements per piece
    constexpr int PER_ROW = D / VE;
    constexpr int N = BT * PER_ROW / NT;                  // pieces per thread
    static_assert(BT * PER_ROW % NT == 0, "tile does not divide over the threads");
    uint4 buf[N];
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT, t = p / PER_ROW, part = p % PER_ROW, code = srow[t];
        const bool take = need_own ? code >= 0 : code != -1;
        const int r = code >= 0 ? code : -2 - code;
        buf[u] = take ? *reinterpret_cast<const uint4*>(src + ((size_t)r * H + h) * D + part * VE) : make_uint4(0, 0, 0, 0);
    }
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int p = threadIdx.x + u * NT, t = p / PER_ROW, part = p % PER_ROW;
        const T* el = reinterpret_cast<const T*>(&buf[u]);
#pragma unroll
        for (int x = 0; x < VE; x++) {
            const int i = part * VE + x;
            dst[ROTATED ? tix<D>(t, i) : t * D + i] = static_cast<Dst>(el[x]);
        }
    }
}

// A [DK][DV] state from global memory (plain layout) into the rotated shared-memory layout, or back.
template <typename Src, typename Dst, int DK, int DV, bool ADD>
__device__ __forceinline__ void load_state(const Src* src, Dst* dst) {
    constexpr int VE = 16 / sizeof(Src);
    constexpr int N = DK * DV / VE / NT;
    uint4 buf[N];
#pragma unroll
    for (int u = 0; u < N; u++) buf[u] = reinterpret_cast<const uint4*>(src)[threadIdx.x + u * NT];
#pragma unroll
    for (int u = 0; u < N; u++) {
        const int e0 = (threadIdx.x + u * NT) * VE;
        const Src* el = reinterpret_cast<const Src*>(&buf[u]);
#pragma unroll
        for (int x = 0; x < VE; x++) {
            const int e = e0 + x, idx = tix<DV>(e / DV, e % DV);
            if (ADD) dst[idx] += static_cast<Dst>(el[x]);
            else dst[idx] = static_cast<Dst>(el[x]);
        }
    }
}
template <typename Dst, int DK, int DV>
__device__ __forceinline__ void store_state(const float* sS, Dst* dst) {
    constexpr int VE = 16 / sizeof(Dst);
    for (int p = threadIdx.x; p < DK * DV / VE; p += NT) {
        uint4 out;
        Dst* el = reinterpret_cast<Dst*>(&out);
#pragma unroll
        for (int x = 0; x < VE; x++) {
            const int e = p * VE + x;
            el[x] = from_f<Dst>(sS[tix<DV>(e / DV, e % DV)]);
        }
        reinterpret_cast<uint4*>(dst)[p] = out;
    }
}

// Loads one chunk: row codes (physical row >= 0 own, -2 - row replayed, -1 past the end), k/v of all valid rows, q and
// dO of own rows (zero elsewhere), and the per-channel running sum of g (rows past the end add nothing).
template <typename T, int DK, int DV, bool BWD>
__device__ void load_chunk(const harts_la_tables_t& tb, const SeqInfo& s, int c, int h, int H, const T* q, const T* k,
                           const T* v, const float* gk, const T* dO, T* sq, T* sk, T* sv, T* sdo, float* sb, int* srow) {
    const int tid = threadIdx.x;
    if (tid < BT) {
        const int vr = c * BT + tid;
        int code = -1;
        if (vr < s.n_virtual)
            code = vr < s.n_replay ? -2 - tb.replay_row[s.replay_base + vr] : s.own_begin + (vr - s.n_replay);
        srow[tid] = code;
    }
    __syncthreads();
    load_tile<T, DK, true>(k, H, h, srow, false, sk);
    load_tile<T, DK, true>(q, H, h, srow, true, sq);
    load_tile<float, DK, false>(gk, H, h, srow, false, sb);
    load_tile<T, DV, true>(v, H, h, srow, false, sv);
    if (BWD) load_tile<T, DV, true>(dO, H, h, srow, true, sdo);
    __syncthreads();
    if (tid < DK) {
        float acc = 0.f;
        for (int t = 0; t < BT; t++) {
            acc += sb[t * DK + tid];
            sb[t * DK + tid] = acc;
        }
    }
    __syncthreads();
}

// A_tj = sum_i q_t[i] k_j[i] e^{b_t[i]-b_j[i]} for j <= t (and, in the backward, dA_tj = dO_t . v_j) into [BT][BT]
template <typename T, int DK, int DV, bool BWD>
__device__ void intra_scores(const T* sq, const T* sk, const T* sv, const T* sdo, const float* sb, float* sA, float* sdA) {
    const int tid = threadIdx.x, lane = tid & 31;
    for (int p = tid; p < N_PAIRS; p += NT) {
        int t = (int)((sqrtf(8.f * p + 1.f) - 1.f) * 0.5f);
        while ((t + 1) * (t + 2) / 2 <= p) t++;
        while (t * (t + 1) / 2 > p) t--;
        const int j = p - t * (t + 1) / 2;
        float acc = 0.f;
        for (int ii = 0; ii < DK; ii++) {
            const int i = (ii + lane) & (DK - 1);          // lanes start at different channels: no bank conflicts
            acc += to_f(sq[tix<DK>(t, i)]) * to_f(sk[tix<DK>(j, i)]) * __expf(sb[t * DK + i] - sb[j * DK + i]);
        }
        sA[t * BT + j] = acc;
        if (BWD) {
            float d = 0.f;
            for (int jj0 = 0; jj0 < DV; jj0++) {
                const int jj = (jj0 + lane) & (DV - 1);
                d += to_f(sdo[tix<DV>(t, jj)]) * to_f(sv[tix<DV>(j, jj)]);
            }
            sdA[t * BT + j] = d;
        }
    }
}

// q_t <- q_t .* e^{b_t},  k_j <- k_j .* e^{b_n - b_j}   (in the tiles' own type, as the scalar-gate kernels do for K)
template <typename T, int DK>
__device__ void scale_qk(T* sq, T* sk, const float* sb) {
    for (int e = threadIdx.x; e < BT * DK; e += NT) {
        const int t = e / DK, i = e % DK;
        const float bt = sb[t * DK + i], bn = sb[(BT - 1) * DK + i];
        sq[tix<DK>(t, i)] = from_f<T>(to_f(sq[tix<DK>(t, i)]) * __expf(bt));
        sk[tix<DK>(t, i)] = from_f<T>(to_f(sk[tix<DK>(t, i)]) * __expf(bn - bt));
    }
}

template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) gk_fwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const T* q, const T* k,
                                                    const T* v, const float* gk, T* o, float* slots, T* chunk_states,
                                                    const int32_t* gate) {
    if (gate_closed(gate)) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sS = reinterpret_cast<float*>(smem_raw);       // [DK][DV], column index rotated by the row
    float* sb = sS + DK * DV;                             // [BT][DK] running log-decay per channel
    float* sA = sb + BT * DK;                             // [BT][BT]
    int* srow = reinterpret_cast<int*>(sA + BT * BT);     // [BT]
    T* sq = reinterpret_cast<T*>(srow + BT);
    T* sk = sq + BT * DK;
    T* sv = sk + BT * DK;

    const int seq = seq_lo + blockIdx.x / H, h = blockIdx.x % H;
    const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
    const SeqInfo s = seq_info(tb, seq);
    const size_t state_elems = (size_t)DK * DV;

    if (s.init_slot < 0)
        for (int e = tid; e < DK * DV; e += NT) sS[e] = 0.f;
    else
        load_state<float, float, DK, DV, false>(slots + ((size_t)s.init_slot * H + h) * state_elems, sS);
    __syncthreads();

    int next_req = s.req_lo;
    for (int c = 0; c < s.n_chunks; c++) {
        load_chunk<T, DK, DV, false>(tb, s, c, h, H, q, k, v, gk, nullptr, sq, sk, sv, nullptr, sb, srow);
        // start-of-chunk state: kept for the backward; exported when the plan requests this boundary
        if (chunk_states) {
            store_state<T, DK, DV>(sS, chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems);
        }
        if (next_req < s.req_hi && tb.slot_chunk[next_req] == c) {
            store_state<float, DK, DV>(sS, slots + ((size_t)next_req * H + h) * state_elems);
            next_req++;
        }
        intra_scores<T, DK, DV, false>(sq, sk, sv, nullptr, sb, sA, nullptr);
        __syncthreads();
        scale_qk<T, DK>(sq, sk, sb);
        __syncthreads();
        // o_t = q~_t S_c + sum_{j<=t} A_tj v_j : rows ty*4+r, columns tx + 16*cc
        for (int r = 0; r < 4; r++) {
            const int t = ty * 4 + r, code = srow[t];
            if (code < 0) continue;
            float acc[DV / 16];
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) acc[cc] = 0.f;
            for (int i = 0; i < DK; i++) {
                const float qv = to_f(sq[tix<DK>(t, i)]);
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc[cc] += qv * sS[tix<DV>(i, tx + 16 * cc)];
            }
            for (int j = 0; j <= t; j++) {
                const float a = sA[t * BT + j];
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc[cc] += a * to_f(sv[tix<DV>(j, tx + 16 * cc)]);
            }
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) o[((size_t)code * H + h) * DV + tx + 16 * cc] = from_f<T>(acc[cc]);
        }
        __syncthreads();
        // S <- Diag(e^{b_n}) S + k~^T v
        {
            float acc[DK / 16][DV / 16];
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) acc[ri][cj] = 0.f;
            for (int j = 0; j < BT; j++) {
                float kv[DK / 16];
#pragma unroll
                for (int ri = 0; ri < DK / 16; ri++) kv[ri] = to_f(sk[tix<DK>(j, ty + 16 * ri)]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    const float vv = to_f(sv[tix<DV>(j, tx + 16 * cj)]);
#pragma unroll
                    for (int ri = 0; ri < DK / 16; ri++) acc[ri][cj] += kv[ri] * vv;
                }
            }
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++) {
                const float gam = __expf(sb[(BT - 1) * DK + ty + 16 * ri]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    const int e = tix<DV>(ty + 16 * ri, tx + 16 * cj);
                    sS[e] = gam * sS[e] + acc[ri][cj];
                }
            }
        }
        __syncthreads();
    }
}

template <typename T, int DK, int DV>
constexpr size_t gk_fwd_smem() {
    return sizeof(float) * (DK * DV + BT * DK + BT * BT) + sizeof(int) * BT + sizeof(T) * (2 * BT * DK + BT * DV);
}

template <typename T, int DK, int DV>
int32_t launch_gk_fwd(const FwdArgs& a) {
    auto kern = gk_fwd_kernel<T, DK, DV>;
    constexpr size_t smem = gk_fwd_smem<T, DK, DV>();
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return HARTS_ECUDA;
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    kern<<<n, NT, smem, a.stream>>>(a.tb, a.seq_lo, a.H, (const T*)a.q, (const T*)a.k, (const T*)a.v, a.g, (T*)a.o,
                                    a.slots, (T*)a.chunk_states, status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace

namespace {

template <typename T, int DK, int DV>
__global__ void __launch_bounds__(NT) gk_bwd_kernel(harts_la_tables_t tb, int seq_lo, int H, const T* q, const T* k,
                                                    const T* v, const float* gk, const T* dO, T* dq, T* dk_, T* dv_,
                                                    float* dgk, const T* chunk_states, float* ds0, float* rk, float* rv,
                                                    float* rg, const int32_t* gate) {
    if (gate_closed(gate)) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* sdS = reinterpret_cast<float*>(smem_raw);      // dS   [DK][DV], column index rotated by the row
    float* sb = sdS + DK * DV;                            // [BT][DK]
    float* sA = sb + BT * DK;                             // A    [BT][BT]
    float* sdA = sA + BT * BT;                            // dA   [BT][BT]
    int* srow = reinterpret_cast<int*>(sdA + BT * BT);    // [BT]
    T* sS = reinterpret_cast<T*>(srow + BT);              // S_c  [DK][DV] in the run dtype (as the forward stored it)
    T* sq = sS + DK * DV;
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
        // gradient arriving at boundary c+1 from the sequences that started there (summed into the first consumer's
        // buffer by handoff_reduce)
        if (next_req >= s.req_lo && tb.slot_chunk[next_req] == c + 1) {
            if (tb.slot_cons_ptr[next_req] < tb.slot_cons_ptr[next_req + 1]) {
                load_state<float, float, DK, DV, true>(
                    ds0 + ((size_t)tb.slot_cons_seq[tb.slot_cons_ptr[next_req]] * H + h) * state_elems, sdS);
            }
            next_req--;
        }
        load_chunk<T, DK, DV, true>(tb, s, c, h, H, q, k, v, gk, dO, sq, sk, sv, sdo, sb, srow);
        {
            load_state<T, T, DK, DV, false>(chunk_states + ((size_t)(s.chunk_base + c) * H + h) * state_elems, sS);
        }
        intra_scores<T, DK, DV, true>(sq, sk, sv, sdo, sb, sA, sdA);
        __syncthreads();
        // ---- two threads per key channel i (lanes 2i, 2i+1): dq, dk, dg of the chunk, rows in reverse.  Thread hh of the
        //      pair takes the state columns jj = hh (mod 2) of the two row-dots and the rows j = hh (mod 2) of the
        //      decay-dependent sums, so that it alone accumulates dk_j for its rows; partial sums meet by shuffles.
        if (tid < 2 * DK) {
            const int i = tid >> 1, hh = tid & 1;
            const unsigned pair_mask = 0x3u << ((tid & 31) & ~1);
            const float bn = sb[(BT - 1) * DK + i];
            float dk_acc[BT / 2];                          // rows j = 2 * jh + hh
#pragma unroll
            for (int jh = 0; jh < BT / 2; jh++) dk_acc[jh] = 0.f;
            float rowdot = 0.f;                            // <S_c[i,:], dS[i,:]>
            for (int jj = hh; jj < DV; jj += 2) rowdot += to_f(sS[tix<DV>(i, jj)]) * sdS[tix<DV>(i, jj)];
            rowdot += __shfl_xor_sync(pair_mask, rowdot, 1);
            float suffix = 0.f, g_inter = 0.f;
#pragma unroll
            for (int t = BT - 1; t >= 0; t--) {
                const int code = srow[t];
                if (code == -1) continue;                  // past the end: nothing there (the same for the whole CTA)
                float iq = 0.f, ik = 0.f;                  // (dO_t S_c^T)[i], (v_t dS^T)[i]
                for (int jj = hh; jj < DV; jj += 2) {
                    iq += to_f(sdo[tix<DV>(t, jj)]) * to_f(sS[tix<DV>(i, jj)]);
                    ik += to_f(sv[tix<DV>(t, jj)]) * sdS[tix<DV>(i, jj)];
                }
                const float bt = sb[t * DK + i];
                const float qt = to_f(sq[tix<DK>(t, i)]), kt = to_f(sk[tix<DK>(t, i)]);
                float dq_acc = 0.f;
#pragma unroll
                for (int jh = 0; 2 * jh <= t; jh++) {
                    const int j = 2 * jh + hh;
                    if (j <= t) {
                        const float x = sdA[t * BT + j] * __expf(bt - sb[j * DK + i]);   // one exponential for dq and dk
                        dq_acc += x * to_f(sk[tix<DK>(j, i)]);
                        dk_acc[jh] += x * qt;
                    }
                }
                iq += __shfl_xor_sync(pair_mask, iq, 1);
                ik += __shfl_xor_sync(pair_mask, ik, 1);
                dq_acc += __shfl_xor_sync(pair_mask, dq_acc, 1);
                // row t has received all its contributions (rows >= t are done); its owner is thread t mod 2 of the pair
                const float dk_intra = __shfl_sync(pair_mask, dk_acc[t >> 1], ((tid & 31) & ~1) + (t & 1));
                const float ew = __expf(bn - bt);
                const float dqv = dq_acc + __expf(bt) * iq;
                const float dkv = dk_intra + ew * ik;
                g_inter += kt * ew * ik;
                suffix += qt * dqv - kt * dkv;
                if (hh == 0) {
                    if (code >= 0) {
                        const size_t off = ((size_t)code * H + h) * DK + i;
                        dq[off] = from_f<T>(dqv);
                        dk_[off] = from_f<T>(dkv);
                        dgk[off] = suffix;
                    } else {                               // replayed rows sit in chunk 0: virtual row = t
                        const size_t off = ((size_t)(s.replay_base + t) * H + h) * DK + i;
                        rk[off] = dkv;
                        rg[off] = suffix;
                    }
                }
            }
            // every row of the chunk also gets <S_{c+1}[i,:], dS[i,:]> = e^{b_n[i]} <S_c[i,:], dS[i,:]> + sum_j k_j[i] dk_j(inter)[i]
            const float G = __expf(bn) * rowdot + g_inter;
            if (hh == 0)
                for (int t = 0; t < BT; t++) {
                    const int code = srow[t];
                    if (code >= 0) dgk[((size_t)code * H + h) * DK + i] += G;
                    else if (code < -1) rg[((size_t)(s.replay_base + t) * H + h) * DK + i] += G;
                }
        }
        __syncthreads();
        scale_qk<T, DK>(sq, sk, sb);
        __syncthreads();
        // ---- dv_j = sum_{t>=j} A_tj dO_t + k~_j dS : rows ty*4+r, columns tx + 16*cc ---------------------------------
        for (int r = 0; r < 4; r++) {
            const int j = ty * 4 + r, code = srow[j];
            if (code == -1) continue;
            float acc[DV / 16];
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) acc[cc] = 0.f;
            for (int i = 0; i < DK; i++) {
                const float kv = to_f(sk[tix<DK>(j, i)]);
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc[cc] += kv * sdS[tix<DV>(i, tx + 16 * cc)];
            }
            for (int t = j; t < BT; t++) {
                const float a = sA[t * BT + j];
#pragma unroll
                for (int cc = 0; cc < DV / 16; cc++) acc[cc] += a * to_f(sdo[tix<DV>(t, tx + 16 * cc)]);
            }
#pragma unroll
            for (int cc = 0; cc < DV / 16; cc++) {
                const int jj = tx + 16 * cc;
                if (code >= 0) dv_[((size_t)code * H + h) * DV + jj] = from_f<T>(acc[cc]);
                else rv[((size_t)(s.replay_base + j) * H + h) * DV + jj] = acc[cc];
            }
        }
        __syncthreads();
        // ---- dS <- Diag(e^{b_n}) dS + q~^T dO --------------------------------------------------------------------------
        {
            float acc[DK / 16][DV / 16];
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++)
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) acc[ri][cj] = 0.f;
            for (int t = 0; t < BT; t++) {
                float qv[DK / 16];
#pragma unroll
                for (int ri = 0; ri < DK / 16; ri++) qv[ri] = to_f(sq[tix<DK>(t, ty + 16 * ri)]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    const float dov = to_f(sdo[tix<DV>(t, tx + 16 * cj)]);
#pragma unroll
                    for (int ri = 0; ri < DK / 16; ri++) acc[ri][cj] += qv[ri] * dov;
                }
            }
#pragma unroll
            for (int ri = 0; ri < DK / 16; ri++) {
                const float gam = __expf(sb[(BT - 1) * DK + ty + 16 * ri]);
#pragma unroll
                for (int cj = 0; cj < DV / 16; cj++) {
                    const int e = tix<DV>(ty + 16 * ri, tx + 16 * cj);
                    sdS[e] = gam * sdS[e] + acc[ri][cj];
                }
            }
        }
        __syncthreads();
    }
    if (s.init_slot >= 0) {
        store_state<float, DK, DV>(sdS, ds0 + ((size_t)seq * H + h) * state_elems);
    }
}

// dk/dv/dg of a replayed row += the contributions of every sequence that replayed it (Section 4.2: the gather's
// backward sums all consumers into the unique producer row); dg is a vector over the key channels here.
template <typename T>
__global__ void gk_replay_reduce_kernel(harts_la_tables_t tb, int H, int DK, int DV, T* dk_, T* dv_, float* dgk,
                                        const float* rk, const float* rv, const float* rg) {
    const int m = blockIdx.x / H, h = blockIdx.x % H;
    const int row = tb.rg_row[m];
    const int lo = tb.rg_ptr[m], hi = tb.rg_ptr[m + 1];
    for (int i = threadIdx.x; i < 2 * DK + DV; i += blockDim.x) {
        float acc = 0.f;
        if (i < DK) {
            for (int e = lo; e < hi; e++) acc += rk[((size_t)tb.rg_entry[e] * H + h) * DK + i];
            T* p = dk_ + ((size_t)row * H + h) * DK + i;
            *p = from_f<T>(to_f(*p) + acc);
        } else if (i < DK + DV) {
            const int j = i - DK;
            for (int e = lo; e < hi; e++) acc += rv[((size_t)tb.rg_entry[e] * H + h) * DV + j];
            T* p = dv_ + ((size_t)row * H + h) * DV + j;
            *p = from_f<T>(to_f(*p) + acc);
        } else {
            const int c = i - DK - DV;
            for (int e = lo; e < hi; e++) acc += rg[((size_t)tb.rg_entry[e] * H + h) * DK + c];
            dgk[((size_t)row * H + h) * DK + c] += acc;
        }
    }
}

template <typename T, int DK, int DV>
constexpr size_t gk_bwd_smem() {
    return sizeof(float) * (DK * DV + BT * DK + 2 * BT * BT) + sizeof(int) * BT +
           sizeof(T) * (DK * DV + 2 * BT * DK + 2 * BT * DV);
}

template <typename T, int DK, int DV>
int32_t launch_gk_bwd(const BwdArgs& a) {
    auto kern = gk_bwd_kernel<T, DK, DV>;
    constexpr size_t smem = gk_bwd_smem<T, DK, DV>();
    static_assert(smem <= 232448, "backward tile does not fit in shared memory");
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return HARTS_ECUDA;
    const int n = (a.seq_hi - a.seq_lo) * a.H;
    const GkScratchLayout sl = gk_scratch_layout(a.tb, a.H, a.dk, a.dv);
    char* base = static_cast<char*>(a.scratch);
    kern<<<n, NT, smem, a.stream>>>(a.tb, a.seq_lo, a.H, (const T*)a.q, (const T*)a.k, (const T*)a.v, a.g,
                                    (const T*)a.dO, (T*)a.dq, (T*)a.dk_, (T*)a.dv_, a.dg, (const T*)a.chunk_states,
                                    (float*)(base + sl.ds0), (float*)(base + sl.rk), (float*)(base + sl.rv),
                                    (float*)(base + sl.rg), status_gate(a.flags, a.dev_status));
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace

// dtype / head dimensions served: fp32 with d = 64, bf16 with d = 64 or 128 (d_k = d_v)
int32_t gk_supported(int32_t dtype, int32_t dk, int32_t dv) {
    if (dtype == HARTS_FP32) return dk == 64 && dv == 64;
    if (dtype == HARTS_BF16) return (dk == 64 && dv == 64) || (dk == 128 && dv == 128);
    return 0;
}

int32_t gk_fwd(const FwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (gk_mma_supported(a.dtype, a.dk, a.dv) && !(a.flags & HARTS_FLAG_FMA_KERNELS)) return gk_mma_fwd(a);
    if (a.dtype == HARTS_FP32 && a.dk == 64 && a.dv == 64) return launch_gk_fwd<float, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 64 && a.dv == 64) return launch_gk_fwd<__nv_bfloat16, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 128 && a.dv == 128) return launch_gk_fwd<__nv_bfloat16, 128, 128>(a);
    return HARTS_EUNSUPPORTED;
}

int32_t gk_bwd(const BwdArgs& a) {
    if (a.seq_hi == a.seq_lo) return HARTS_OK;
    if (int32_t rc = handoff_reduce(a); rc != HARTS_OK) return rc;     // ds0 sits at the same place in both layouts
    if (gk_mma_supported(a.dtype, a.dk, a.dv) && !(a.flags & HARTS_FLAG_FMA_KERNELS)) return gk_mma_bwd(a);
    if (a.dtype == HARTS_FP32 && a.dk == 64 && a.dv == 64) return launch_gk_bwd<float, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 64 && a.dv == 64) return launch_gk_bwd<__nv_bfloat16, 64, 64>(a);
    if (a.dtype == HARTS_BF16 && a.dk == 128 && a.dv == 128) return launch_gk_bwd<__nv_bfloat16, 128, 128>(a);
    return HARTS_EUNSUPPORTED;
}

int32_t gk_replay_reduce(const harts_la_tables_t& tb, void* dk_, void* dv_, float* dgk, const void* scratch, int32_t H,
                         int32_t dk, int32_t dv, int32_t dtype, cudaStream_t stream) {
    if (tb.n_rg_rows == 0) return HARTS_OK;
    const GkScratchLayout sl = gk_scratch_layout(tb, H, dk, dv);
    const char* base = static_cast<const char*>(scratch);
    const float* rk = (const float*)(base + sl.rk);
    const float* rv = (const float*)(base + sl.rv);
    const float* rg = (const float*)(base + sl.rg);
    const int n = tb.n_rg_rows * H;
    if (dtype == HARTS_FP32)
        gk_replay_reduce_kernel<float><<<n, 128, 0, stream>>>(tb, H, dk, dv, (float*)dk_, (float*)dv_, dgk, rk, rv, rg);
    else
        gk_replay_reduce_kernel<__nv_bfloat16><<<n, 128, 0, stream>>>(tb, H, dk, dv, (__nv_bfloat16*)dk_,
                                                                      (__nv_bfloat16*)dv_, dgk, rk, rv, rg);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

}  // namespace harts
