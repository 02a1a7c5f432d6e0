// Compact-to-semantic log-probability kernels (Section 3.5, Eqs. 17 and 19) for sm_100a.
//
// Both passes are streaming scans over the compact logit rows and are bound by HBM bandwidth:
//   forward   reads  n_rows*V elements once (online max / sum-exp per row), then n_pos 1-element gathers;
//   backward  reads  n_rows*V elements and writes n_rows*V elements (rows without an active position are
//             zero-filled without being read), then patches the <= n_pos target columns.
// One CTA owns one row at a time (rows dealt round-robin over a grid of a few CTAs per SM), every thread
// keeps several 16-byte loads in flight, and all reductions run in a fixed order, so results are
// deterministic.  There is no tensor-core work here: nothing in the step is a contraction.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/harts_logp.h"

namespace {

constexpr int NT = 256;            // threads per CTA
constexpr int UNROLL = 4;          // 16-byte loads in flight per thread
constexpr float LOG2E = 1.4426950408889634f;
constexpr float LN2 = 0.6931471805599453f;

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <typename T> struct Elem;
template <> struct Elem<float> {
    static constexpr int PER_VEC = 4;
    static __device__ __forceinline__ void unpack(const uint4& u, float* x) {
        x[0] = __uint_as_float(u.x); x[1] = __uint_as_float(u.y);
        x[2] = __uint_as_float(u.z); x[3] = __uint_as_float(u.w);
    }
    static __device__ __forceinline__ uint4 pack(const float* x) {
        return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
    }
    static __device__ __forceinline__ float load(const float* p) { return *p; }
    static __device__ __forceinline__ void store(float* p, float v) { *p = v; }
};
template <> struct Elem<__nv_bfloat16> {
    static constexpr int PER_VEC = 8;
    static __device__ __forceinline__ void unpack(const uint4& u, float* x) {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ uint32_t pack2(float lo, float hi) {
        uint32_t r;
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
        return r;
    }
    static __device__ __forceinline__ uint4 pack(const float* x) {
        return make_uint4(pack2(x[0], x[1]), pack2(x[2], x[3]), pack2(x[4], x[5]), pack2(x[6], x[7]));
    }
    static __device__ __forceinline__ float load(const __nv_bfloat16* p) { return __bfloat162float(*p); }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// Running (max, sum of exp(x - max)) pair; `ml` caches max*log2(e) (0 while max is still -inf).
struct MaxSum {
    float mx, ml, sum;
    __device__ __forceinline__ void init() { mx = -INFINITY; ml = 0.f; sum = 0.f; }
    __device__ __forceinline__ void raise(float cand) {
        if (cand > mx) {
            sum = (mx == -INFINITY) ? 0.f : sum * ex2(ml - cand * LOG2E);
            mx = cand;
            ml = cand * LOG2E;
        }
    }
    __device__ __forceinline__ void add(float x) { sum += ex2(fmaf(x, LOG2E, -ml)); }
    __device__ __forceinline__ void merge(float omx, float osum) {
        if (omx == -INFINITY) return;
        if (mx == -INFINITY) { mx = omx; ml = omx * LOG2E; sum = osum; return; }
        const float M = fmaxf(mx, omx);
        sum = sum * ex2((mx - M) * LOG2E) + osum * ex2((omx - M) * LOG2E);
        mx = M;
        ml = M * LOG2E;
    }
};

// Elements of a row before the first 16-byte boundary (all of the row if it is shorter).
template <typename T>
__device__ __forceinline__ int head_elems(const T* row, int V) {
    const int mis = static_cast<int>(reinterpret_cast<uintptr_t>(row) & 15);
    const int h = ((16 - mis) & 15) / static_cast<int>(sizeof(T));
    return h < V ? h : V;
}

// ---------------------------------------------------------------------------------------------------
// Forward: per-row max and sum-exp in one pass.
// ---------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) lse_kernel(const T* __restrict__ z, int n_rows, int V, int64_t ld,
                                                 float* __restrict__ lse, float* __restrict__ row_max,
                                                 float* __restrict__ row_sum) {
    constexpr int EPV = Elem<T>::PER_VEC;
    __shared__ float s_mx[NT / 32], s_sum[NT / 32];
    const int tid = threadIdx.x;
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        const T* zr = z + static_cast<int64_t>(row) * ld;
        const int head = head_elems(zr, V);
        const int nvec = (V - head) / EPV;
        const int tail0 = head + nvec * EPV;
        const uint4* zv = reinterpret_cast<const uint4*>(zr + head);
        MaxSum acc;
        acc.init();
        if (tid < head) { const float x = Elem<T>::load(zr + tid); acc.raise(x); acc.add(x); }
        if (tid < V - tail0) { const float x = Elem<T>::load(zr + tail0 + tid); acc.raise(x); acc.add(x); }
        int i = tid;
        for (; i + (UNROLL - 1) * NT < nvec; i += UNROLL * NT) {
            uint4 u[UNROLL];
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) u[k] = __ldcs(zv + i + k * NT);
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) {
                float x[EPV];
                Elem<T>::unpack(u[k], x);
                float lm = x[0];
#pragma unroll
                for (int e = 1; e < EPV; ++e) lm = fmaxf(lm, x[e]);
                acc.raise(lm);
#pragma unroll
                for (int e = 0; e < EPV; ++e) acc.add(x[e]);
            }
        }
        for (; i < nvec; i += NT) {
            float x[EPV];
            Elem<T>::unpack(__ldcs(zv + i), x);
            float lm = x[0];
#pragma unroll
            for (int e = 1; e < EPV; ++e) lm = fmaxf(lm, x[e]);
            acc.raise(lm);
#pragma unroll
            for (int e = 0; e < EPV; ++e) acc.add(x[e]);
        }
        // fixed-order reduction: butterfly inside the warp, then warp 0 over the warps
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) {
            const float omx = __shfl_xor_sync(0xffffffffu, acc.mx, d);
            const float osum = __shfl_xor_sync(0xffffffffu, acc.sum, d);
            acc.merge(omx, osum);
        }
        if ((tid & 31) == 0) { s_mx[tid >> 5] = acc.mx; s_sum[tid >> 5] = acc.sum; }
        __syncthreads();
        if (tid == 0) {
            MaxSum tot;
            tot.init();
            for (int w = 0; w < NT / 32; ++w) tot.merge(s_mx[w], s_sum[w]);
            if (lse) lse[row] = tot.mx + lg2(tot.sum) * LN2;     // -inf for a row of -inf only
            if (row_max) { row_max[row] = tot.mx; row_sum[row] = tot.sum; }
        }
        __syncthreads();
    }
}

// lambda_s = z[m(s), y_s] - lse[m(s)]  (lse given), or the shard's target logit (lse == nullptr).
template <typename T>
__global__ void __launch_bounds__(NT) gather_kernel(const T* __restrict__ z, int n_rows, int V, int64_t ld,
                                                    int v_begin, int64_t n_pos, const int32_t* __restrict__ m,
                                                    const int32_t* __restrict__ y, int V_total,
                                                    const float* __restrict__ lse, float* __restrict__ out,
                                                    int32_t* status) {
    for (int64_t s = blockIdx.x * static_cast<int64_t>(NT) + threadIdx.x; s < n_pos;
         s += static_cast<int64_t>(gridDim.x) * NT) {
        const int c = m[s], yy = y[s];
        float r = 0.f;
        if (c < 0 || c >= n_rows || yy < 0 || yy >= V_total) {
            if (status && atomicCAS(status, 0, HARTS_EINVAL) == 0) status[1] = static_cast<int32_t>(s);
        } else {
            const int col = yy - v_begin;
            if (col >= 0 && col < V) {
                r = Elem<T>::load(z + static_cast<int64_t>(c) * ld + col);
                if (lse) r -= lse[c];
            }
        }
        out[s] = r;
    }
}

__global__ void __launch_bounds__(NT) combine_rows_kernel(int n_shards, int n_rows, const float* __restrict__ row_max,
                                                          const float* __restrict__ row_sum, float* __restrict__ lse) {
    const int c = blockIdx.x * NT + threadIdx.x;
    if (c >= n_rows) return;
    MaxSum tot;
    tot.init();
    for (int k = 0; k < n_shards; ++k)
        tot.merge(row_max[static_cast<int64_t>(k) * n_rows + c], row_sum[static_cast<int64_t>(k) * n_rows + c]);
    lse[c] = tot.mx + lg2(tot.sum) * LN2;
}

__global__ void __launch_bounds__(NT) combine_pos_kernel(int n_shards, int n_rows, int64_t n_pos,
                                                         const int32_t* __restrict__ m,
                                                         const float* __restrict__ target,
                                                         const float* __restrict__ lse, float* __restrict__ lambda) {
    const int64_t s = blockIdx.x * static_cast<int64_t>(NT) + threadIdx.x;
    if (s >= n_pos) return;
    float t = 0.f;
    for (int k = 0; k < n_shards; ++k) t += target[static_cast<int64_t>(k) * n_pos + s];
    const int c = m[s];
    lambda[s] = (c >= 0 && c < n_rows) ? t - lse[c] : 0.f;
}

// ---------------------------------------------------------------------------------------------------
// Backward: dz[c, :] = -w_c softmax(z_c) + sum_s g_s onehot(y_s),  w_c = sum of g_s over the row's positions.
// ---------------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(NT) dz_kernel(const T* __restrict__ z, int n_rows, int V, int64_t ld,
                                                const int32_t* __restrict__ y, const int32_t* __restrict__ row_pos_ptr,
                                                const int32_t* __restrict__ row_pos, const float* __restrict__ lse,
                                                const float* __restrict__ g, T* __restrict__ dz, int64_t lddz,
                                                int v_begin, int V_total, int32_t* status) {
    constexpr int EPV = Elem<T>::PER_VEC;
    __shared__ float s_w;
    __shared__ int s_active;
    const int tid = threadIdx.x;
    for (int row = blockIdx.x; row < n_rows; row += gridDim.x) {
        const int p0 = row_pos_ptr[row], p1 = row_pos_ptr[row + 1];
        if (tid == 0) {                       // the row's weight, summed in CSR order by one thread
            float w = 0.f;
            int active = 0;
            for (int p = p0; p < p1; ++p) {
                const float gs = g[row_pos[p]];
                w += gs;
                active |= (gs != 0.f);
            }
            s_w = w;
            s_active = active;
        }
        __syncthreads();
        const float w = s_w;
        const bool active = s_active != 0;
        const T* zr = z + static_cast<int64_t>(row) * ld;
        T* dr = dz + static_cast<int64_t>(row) * lddz;
        // the vector body follows dz's alignment; z is read with the same element offsets
        const int head = head_elems(dr, V);
        const int nvec = (V - head) / EPV;
        const int tail0 = head + nvec * EPV;
        const bool z_aligned = ((reinterpret_cast<uintptr_t>(zr + head) & 15) == 0);
        uint4* dv = reinterpret_cast<uint4*>(dr + head);
        if (!active) {
            if (tid < head) Elem<T>::store(dr + tid, 0.f);
            if (tid < V - tail0) Elem<T>::store(dr + tail0 + tid, 0.f);
            for (int i = tid; i < nvec; i += NT) __stcs(dv + i, make_uint4(0u, 0u, 0u, 0u));
        } else {
            const float nl = -lse[row] * LOG2E;
            const float nw = -w;
            if (tid < head) Elem<T>::store(dr + tid, nw * ex2(fmaf(Elem<T>::load(zr + tid), LOG2E, nl)));
            if (tid < V - tail0)
                Elem<T>::store(dr + tail0 + tid, nw * ex2(fmaf(Elem<T>::load(zr + tail0 + tid), LOG2E, nl)));
            if (z_aligned) {
                const uint4* zv = reinterpret_cast<const uint4*>(zr + head);
                int i = tid;
                for (; i + (UNROLL - 1) * NT < nvec; i += UNROLL * NT) {
                    uint4 u[UNROLL];
#pragma unroll
                    for (int k = 0; k < UNROLL; ++k) u[k] = __ldcs(zv + i + k * NT);
#pragma unroll
                    for (int k = 0; k < UNROLL; ++k) {
                        float x[EPV];
                        Elem<T>::unpack(u[k], x);
#pragma unroll
                        for (int e = 0; e < EPV; ++e) x[e] = nw * ex2(fmaf(x[e], LOG2E, nl));
                        __stcs(dv + i + k * NT, Elem<T>::pack(x));
                    }
                }
                for (; i < nvec; i += NT) {
                    float x[EPV];
                    Elem<T>::unpack(__ldcs(zv + i), x);
#pragma unroll
                    for (int e = 0; e < EPV; ++e) x[e] = nw * ex2(fmaf(x[e], LOG2E, nl));
                    __stcs(dv + i, Elem<T>::pack(x));
                }
            } else {                          // z and dz rows are aligned differently: element loads
                for (int i = tid; i < nvec; i += NT) {
                    float x[EPV];
#pragma unroll
                    for (int e = 0; e < EPV; ++e)
                        x[e] = nw * ex2(fmaf(Elem<T>::load(zr + head + i * EPV + e), LOG2E, nl));
                    __stcs(dv + i, Elem<T>::pack(x));
                }
            }
            __syncthreads();                  // the row is written before its target columns are patched
            for (int j = tid; j < p1 - p0; j += NT) {
                const int s = row_pos[p0 + j];
                const int yy = y[s];
                if (yy < 0 || yy >= V_total) {
                    if (status && atomicCAS(status, 0, HARTS_EINVAL) == 0) status[1] = s;
                    continue;
                }
                const int col = yy - v_begin;
                if (col < 0 || col >= V) continue;
                float hit = 0.f;              // all positions of this row with the same target, in CSR order
                for (int p = p0; p < p1; ++p) {
                    const int s2 = row_pos[p];
                    if (y[s2] == yy) hit += g[s2];
                }
                Elem<T>::store(dr + col, hit + nw * ex2(fmaf(Elem<T>::load(zr + col), LOG2E, nl)));
            }
        }
        __syncthreads();                      // s_w / s_active are rewritten for the next row
    }
}

int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    }
    return n;
}

int row_grid(int n_rows) {
    const int cap = sm_count() * 8;           // 8 CTAs of 256 threads fill an SM
    return n_rows < cap ? n_rows : cap;
}

int pos_grid(int64_t n_pos) {
    const int64_t want = (n_pos + NT - 1) / NT;
    const int64_t cap = static_cast<int64_t>(sm_count()) * 8;
    return static_cast<int>(want < cap ? want : cap);
}

bool elem_aligned(const void* p, int dtype) {
    return (reinterpret_cast<uintptr_t>(p) & (dtype == HARTS_BF16 ? 1 : 3)) == 0;
}

int32_t launched() { return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA; }

int32_t fwd_common(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int32_t v_begin,
                   int32_t V_total, int64_t n_pos, const int32_t* m, const int32_t* y, float* lse, float* row_max,
                   float* row_sum, float* out, int32_t* dev_status, void* stream) {
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    if (n_rows < 0 || V < 1 || ldz < V || n_pos < 0 || v_begin < 0 || V_total < V) return HARTS_EINVAL;
    if (n_rows && (!z || !elem_aligned(z, dtype))) return HARTS_EINVAL;
    if (n_pos && (!m || !y || !out)) return HARTS_EINVAL;
    if (dev_status && (reinterpret_cast<uintptr_t>(dev_status) & 3)) return HARTS_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_rows) {
        if (dtype == HARTS_BF16)
            lse_kernel<__nv_bfloat16><<<row_grid(n_rows), NT, 0, st>>>(static_cast<const __nv_bfloat16*>(z), n_rows, V,
                                                                       ldz, lse, row_max, row_sum);
        else
            lse_kernel<float><<<row_grid(n_rows), NT, 0, st>>>(static_cast<const float*>(z), n_rows, V, ldz, lse,
                                                               row_max, row_sum);
    }
    if (n_pos) {
        if (dtype == HARTS_BF16)
            gather_kernel<__nv_bfloat16><<<pos_grid(n_pos), NT, 0, st>>>(static_cast<const __nv_bfloat16*>(z), n_rows,
                                                                         V, ldz, v_begin, n_pos, m, y, V_total, lse,
                                                                         out, dev_status);
        else
            gather_kernel<float><<<pos_grid(n_pos), NT, 0, st>>>(static_cast<const float*>(z), n_rows, V, ldz, v_begin,
                                                                 n_pos, m, y, V_total, lse, out, dev_status);
    }
    return launched();
}

}  // namespace

extern "C" int32_t harts_logp_fwd(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int64_t n_pos,
                                  const int32_t* m, const int32_t* y, float* lse, float* lambda, int32_t* dev_status,
                                  void* stream) {
    if (n_rows > 0 && !lse) return HARTS_EINVAL;
    return fwd_common(z, dtype, n_rows, V, ldz, 0, V, n_pos, m, y, lse, nullptr, nullptr, lambda, dev_status, stream);
}

extern "C" int32_t harts_logp_fwd_shard(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz,
                                        int32_t v_begin, int64_t n_pos, const int32_t* m, const int32_t* y,
                                        float* row_max, float* row_sum, float* target, int32_t* dev_status,
                                        void* stream) {
    if (n_rows > 0 && (!row_max || !row_sum)) return HARTS_EINVAL;
    if (V < 1 || v_begin < 0 || v_begin > INT32_MAX - V) return HARTS_EINVAL;
    // targets are only required to be valid vocabulary ids; which shard holds them is decided per position
    return fwd_common(z, dtype, n_rows, V, ldz, v_begin, INT32_MAX, n_pos, m, y, nullptr, row_max, row_sum, target,
                      dev_status, stream);
}

extern "C" int32_t harts_logp_combine(int32_t n_shards, int32_t n_rows, int64_t n_pos, const int32_t* m,
                                      const float* row_max, const float* row_sum, const float* target, float* lse,
                                      float* lambda, void* stream) {
    if (n_shards < 1 || n_rows < 0 || n_pos < 0) return HARTS_EINVAL;
    if (n_rows && (!row_max || !row_sum || !lse)) return HARTS_EINVAL;
    if (n_pos && (!m || !target || !lambda || !lse)) return HARTS_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_rows) combine_rows_kernel<<<(n_rows + NT - 1) / NT, NT, 0, st>>>(n_shards, n_rows, row_max, row_sum, lse);
    if (n_pos)
        combine_pos_kernel<<<static_cast<unsigned>((n_pos + NT - 1) / NT), NT, 0, st>>>(n_shards, n_rows, n_pos, m,
                                                                                         target, lse, lambda);
    return launched();
}

extern "C" int32_t harts_logp_bwd(const void* z, int32_t dtype, int32_t n_rows, int32_t V, int64_t ldz, int64_t n_pos,
                                  const int32_t* y, const int32_t* row_pos_ptr, const int32_t* row_pos,
                                  const float* lse, const float* g, void* dz, int64_t lddz, int32_t v_begin,
                                  int32_t V_total, int32_t* dev_status, void* stream) {
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return HARTS_EUNSUPPORTED;
    if (n_rows < 0 || V < 1 || ldz < V || lddz < V || n_pos < 0 || v_begin < 0 || V_total < V ||
        v_begin > V_total - V)
        return HARTS_EINVAL;
    if (n_rows == 0) return HARTS_OK;
    if (!z || !dz || !lse || !row_pos_ptr || !elem_aligned(z, dtype) || !elem_aligned(dz, dtype) || z == dz)
        return HARTS_EINVAL;
    if (n_pos && (!y || !row_pos || !g)) return HARTS_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == HARTS_BF16)
        dz_kernel<__nv_bfloat16><<<row_grid(n_rows), NT, 0, st>>>(
            static_cast<const __nv_bfloat16*>(z), n_rows, V, ldz, y, row_pos_ptr, row_pos, lse, g,
            static_cast<__nv_bfloat16*>(dz), lddz, v_begin, V_total, dev_status);
    else
        dz_kernel<float><<<row_grid(n_rows), NT, 0, st>>>(static_cast<const float*>(z), n_rows, V, ldz, y, row_pos_ptr,
                                                          row_pos, lse, g, static_cast<float*>(dz), lddz, v_begin,
                                                          V_total, dev_status);
    return launched();
}
