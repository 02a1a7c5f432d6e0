// Tree-aware depthwise causal convolution on compact tokens (Section 4.2, "KDA state reuse and causal
// convolution") for sm_100a: forward, and backward (dx, dW).
//
// Both passes are HBM-bound streams: a thread owns 8 channels (one 16-byte vector of bf16), keeps its filter taps
// in registers and walks a strip of consecutive rows with the w-1 neighbouring rows it needs in a register window,
// so every row of x and dy leaves HBM once; only where the packed order is not the trajectory order (a branch or
// sequence start, a fork) does it follow the index tables, and those rows come from L2.  The rows of the walk are
// prefetched eight iterations ahead with cp.async into per-thread shared-memory slots, so the bytes in flight do
// not cost registers (the backward holds 32 taps and 32 dW accumulators per thread).  Algorithmic bytes per row: forward 2*D*e, backward 3*D*e.  No contraction, no tensor cores.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>
#include <vector>

#include "../../include/harts_conv.h"

namespace {

constexpr int NT = 256;
constexpr int MAX_W = 4;
constexpr int MAX_PARTIALS = 2048;         // per-channel partial sums of dW (slots of the scratch)

template <typename T> struct Vec8;
template <> struct Vec8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* f) {
        const uint4 u = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float* f) {
        uint32_t r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r[i]) : "f"(f[2 * i + 1]), "f"(f[2 * i]));
        *reinterpret_cast<uint4*>(p) = make_uint4(r[0], r[1], r[2], r[3]);
    }
};
template <> struct Vec8<float> {
    static __device__ __forceinline__ void load(const float* p, float* f) {
        const float4 a = reinterpret_cast<const float4*>(p)[0], b = reinterpret_cast<const float4*>(p)[1];
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
    static __device__ __forceinline__ void store(float* p, const float* f) {
        reinterpret_cast<float4*>(p)[0] = make_float4(f[0], f[1], f[2], f[3]);
        reinterpret_cast<float4*>(p)[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
};

// Thread layout shared by the kernels: cx = channel group inside the CTA (CX groups), ry = row lane (NT / CX rows
// per CTA step).  taps[i][e] = W[8g + e][w-1-i]: the weight of the i-th ancestor.
struct Lane {
    int g, ry, RY;
    bool active;
};
__device__ __forceinline__ Lane lane_of(int CX, int groups) {
    Lane l;
    l.RY = NT / CX;
    l.g = blockIdx.y * CX + threadIdx.x % CX;
    l.ry = threadIdx.x / CX;
    l.active = l.g < groups;
    return l;
}
template <int W_>
__device__ __forceinline__ void load_taps(const float* __restrict__ W, int g, float (&taps)[W_][8]) {
#pragma unroll
    for (int e = 0; e < 8; ++e)
#pragma unroll
        for (int i = 0; i < W_; ++i) taps[i][e] = W[(size_t)(8 * g + e) * W_ + (W_ - 1 - i)];
}

// 8 channels of one row, kept in the storage format until they are used.
template <typename T> struct Raw;
template <> struct Raw<__nv_bfloat16> {
    uint4 u;
    __device__ __forceinline__ void load(const __nv_bfloat16* p) { u = *reinterpret_cast<const uint4*>(p); }
    __device__ __forceinline__ void zero() { u = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void get(float* f) const {
        const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct Raw<float> {
    float4 a, b;
    __device__ __forceinline__ void load(const float* p) {
        a = reinterpret_cast<const float4*>(p)[0];
        b = reinterpret_cast<const float4*>(p)[1];
    }
    __device__ __forceinline__ void zero() { a = b = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void get(float* f) const {
        f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
    }
};

// Register-free prefetch: a thread copies the rows it will need a few iterations ahead into its own slots of a
// shared-memory ring with cp.async (nobody else reads them, so no barrier is needed, only wait_group).
template <typename T> struct Ring { static constexpr int DEPTH = sizeof(T) == 2 ? 8 : 4; };
template <typename T>
__device__ __forceinline__ void ring_fetch(Raw<T>* slot, const T* src) {
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(slot));
#pragma unroll
    for (int i = 0; i < static_cast<int>(sizeof(Raw<T>)) / 16; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 16 * i), "l"(reinterpret_cast<const char*>(src) + 16 * i)
                     : "memory");
}
__device__ __forceinline__ void ring_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void ring_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

constexpr int STRIP = 128;   // consecutive rows one thread walks with its sliding window

// Forward.  A thread walks a strip of consecutive rows upwards and keeps the last w-1 rows in registers: as long
// as a row's predecessor is the row before it (inside a sequence) the window just shifts and the row costs one
// 16-byte load; where the chain breaks (first row of a strip, of a sequence, of a branch) the window is rebuilt by
// following prev_row, from L2.
template <typename T, int W_>
__global__ void __launch_bounds__(NT, 3) conv_fwd_kernel(const T* __restrict__ x, const float* __restrict__ W,
                                                         const int32_t* __restrict__ prev, T* __restrict__ y,
                                                         int n_rows, int D, int CX) {
    const Lane l = lane_of(CX, D / 8);
    if (!l.active) return;
    constexpr int DEPTH = Ring<T>::DEPTH;
    extern __shared__ __align__(16) unsigned char ring_raw[];
    Raw<T>* ring_x = reinterpret_cast<Raw<T>*>(ring_raw) + threadIdx.x;          // [DEPTH][NT] slots of this thread
    float taps[W_][8];
    load_taps<W_>(W, l.g, taps);
    const size_t col = 8 * (size_t)l.g;
    for (int strip = blockIdx.x * l.RY + l.ry; strip * STRIP < n_rows; strip += gridDim.x * l.RY) {
        const int r0 = strip * STRIP, r1 = min(n_rows, r0 + STRIP);
        Raw<T> h[W_ - 1];                                  // h[i] = x of the (i+1)-th ancestor of the current row
#pragma unroll
        for (int k = 0; k < DEPTH; ++k) {                  // prologue of the ring: the first DEPTH rows of the strip
            if (r0 + k < r1) ring_fetch(ring_x + k * NT, x + (size_t)(r0 + k) * D + col);
            ring_commit();
        }
        int pv_next = prev[r0];
        for (int k = 0, r = r0; r < r1; ++k, ++r) {
            {
                const int slot = k % DEPTH;
                ring_wait<DEPTH - 1>();                    // row r has landed
                Raw<T> xs[1] = {ring_x[slot * NT]};
                if (r + DEPTH < r1) ring_fetch(ring_x + slot * NT, x + (size_t)(r + DEPTH) * D + col);
                ring_commit();
                const int pv[1] = {pv_next};
                if (r + 1 < r1) pv_next = prev[r + 1];
                constexpr int u = 0;
                if (pv[u] != r - 1 || r == r0) {           // chain break: rebuild the window from the true ancestors
                    int a = pv[u];
#pragma unroll
                    for (int i = 0; i < W_ - 1; ++i) {
                        if (a >= 0) {
                            h[i].load(x + (size_t)a * D + col);
                            a = prev[a];
                        } else {
                            h[i].zero();
                        }
                    }
                }
                float acc[8], f[8];
                xs[u].get(f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = taps[0][e] * f[e];
#pragma unroll
                for (int i = 0; i < W_ - 1; ++i) {
                    h[i].get(f);
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[e] = fmaf(taps[i + 1][e], f[e], acc[e]);
                }
                Vec8<T>::store(y + (size_t)r * D + col, acc);
#pragma unroll
                for (int i = W_ - 2; i > 0; --i) h[i] = h[i - 1];
                h[0] = xs[u];
            }
        }
        ring_wait<0>();
    }
}

// Backward.  dx_a = taps[0] dy_a + sum over descendants t at distance i <= w-1 of taps[i] dy_t, and
// dW[:, w-1-i] += x_a * (sum of dy over the descendants at distance i): both need, per row a, its own x and dy
// and the dy of its descendants.  A thread walks a strip downwards with the dy of the next w-1 rows in registers;
// where row a's descendants are exactly the rows a+1 .. a+w-1 (a plain chain inside a sequence: next_row says so)
// the row costs two 16-byte loads, otherwise the successor lists are followed, from L2, children in CSR order.
template <typename T, int W_>
__global__ void __launch_bounds__(NT, 2) conv_bwd_kernel(const T* __restrict__ x, const float* __restrict__ W,
                                                         const T* __restrict__ dy, const int32_t* __restrict__ next_row,
                                                         const int32_t* __restrict__ child_ptr,
                                                         const int32_t* __restrict__ child_row, T* __restrict__ dx,
                                                         float* __restrict__ partial, int n_rows, int D, int CX) {
    const Lane l = lane_of(CX, D / 8);
    if (!l.active) return;
    constexpr int DEPTH = Ring<T>::DEPTH;
    extern __shared__ __align__(16) unsigned char ring_raw[];
    Raw<T>* ring_x = reinterpret_cast<Raw<T>*>(ring_raw) + threadIdx.x;          // [DEPTH][NT] slots of this thread
    Raw<T>* ring_g = ring_x + DEPTH * NT;
    float taps[W_][8], dw[W_][8];
    load_taps<W_>(W, l.g, taps);
#pragma unroll
    for (int i = 0; i < W_; ++i)
#pragma unroll
        for (int e = 0; e < 8; ++e) dw[i][e] = 0.f;
    const size_t col = 8 * (size_t)l.g;
    for (int strip = blockIdx.x * l.RY + l.ry; strip * STRIP < n_rows; strip += gridDim.x * l.RY) {
        const int r0 = strip * STRIP, r1 = min(n_rows, r0 + STRIP);
        Raw<T> d[W_ - 1];                                  // d[i] = dy of row r + 1 + i (valid while `run` says so)
        int run = 0;                                       // plain-chain links known below the current row
        // prologue of the ring: the first DEPTH rows of the walk (top of the strip downwards)
#pragma unroll
        for (int k = 0; k < DEPTH; ++k) {
            const int r = r1 - 1 - k;
            if (r >= r0) {
                ring_fetch(ring_x + k * NT, x + (size_t)r * D + col);
                ring_fetch(ring_g + k * NT, dy + (size_t)r * D + col);
            }
            ring_commit();
        }
        int nx_next = next_row[r1 - 1];
        for (int k = 0, r = r1 - 1; r >= r0; ++k, --r) {
            {
                const int slot = k % DEPTH;
                ring_wait<DEPTH - 1>();                    // the oldest group, i.e. row r, has landed
                const Raw<T> xs_r = ring_x[slot * NT], gs_r = ring_g[slot * NT];
                const int rn = r - DEPTH;                  // refill the slot with the row DEPTH iterations ahead
                if (rn >= r0) {
                    ring_fetch(ring_x + slot * NT, x + (size_t)rn * D + col);
                    ring_fetch(ring_g + slot * NT, dy + (size_t)rn * D + col);
                }
                ring_commit();
                const int nx_r = nx_next;
                if (r > r0) nx_next = next_row[r - 1];
                Raw<T> xs[1] = {xs_r}, gs[1] = {gs_r};
                const int nx[1] = {nx_r};
                constexpr int u = 0;
                float xf[8], g0[8], acc[8], f[8];
                xs[u].get(xf);
                gs[u].get(g0);
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    acc[e] = taps[0][e] * g0[e];
                    dw[0][e] = fmaf(xf[e], g0[e], dw[0][e]);
                }
                run = (nx[u] == r + 1 && r != r1 - 1) ? min(run + 1, W_ - 1) : 0;   // the strip's top row has no window
                if (run == W_ - 1) {                       // descendants are rows r+1 .. r+w-1, all in registers
#pragma unroll
                    for (int i = 0; i < W_ - 1; ++i) {
                        d[i].get(f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            acc[e] = fmaf(taps[i + 1][e], f[e], acc[e]);
                            dw[i + 1][e] = fmaf(xf[e], f[e], dw[i + 1][e]);
                        }
                    }
                } else {
                    for (int p1 = child_ptr[r]; p1 < child_ptr[r + 1]; ++p1) {
                        const int c1 = child_row[p1];
                        Vec8<T>::load(dy + (size_t)c1 * D + col, f);
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            acc[e] = fmaf(taps[1][e], f[e], acc[e]);
                            dw[1][e] = fmaf(xf[e], f[e], dw[1][e]);
                        }
                        if (W_ > 2)
                            for (int p2 = child_ptr[c1]; p2 < child_ptr[c1 + 1]; ++p2) {
                                const int c2 = child_row[p2];
                                Vec8<T>::load(dy + (size_t)c2 * D + col, f);
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    acc[e] = fmaf(taps[W_ > 2 ? 2 : 0][e], f[e], acc[e]);
                                    dw[W_ > 2 ? 2 : 0][e] = fmaf(xf[e], f[e], dw[W_ > 2 ? 2 : 0][e]);
                                }
                                if (W_ > 3)
                                    for (int p3 = child_ptr[c2]; p3 < child_ptr[c2 + 1]; ++p3) {
                                        const int c3 = child_row[p3];
                                        Vec8<T>::load(dy + (size_t)c3 * D + col, f);
#pragma unroll
                                        for (int e = 0; e < 8; ++e) {
                                            acc[e] = fmaf(taps[W_ > 3 ? 3 : 0][e], f[e], acc[e]);
                                            dw[W_ > 3 ? 3 : 0][e] = fmaf(xf[e], f[e], dw[W_ > 3 ? 3 : 0][e]);
                                        }
                                    }
                            }
                    }
                }
                Vec8<T>::store(dx + (size_t)r * D + col, acc);
#pragma unroll
                for (int i = W_ - 2; i > 0; --i) d[i] = d[i - 1];
                d[0] = gs[u];
            }
        }
        ring_wait<0>();
    }
    // partial[slot][channel][tap], slot = (blockIdx.x, ry)
    float* dst = partial + ((size_t)(blockIdx.x * l.RY + l.ry) * D + col) * W_;
#pragma unroll
    for (int e = 0; e < 8; ++e)
#pragma unroll
        for (int i = 0; i < W_; ++i) dst[e * W_ + (W_ - 1 - i)] = dw[i][e];
}

__global__ void __launch_bounds__(NT) conv_dw_reduce_kernel(const float* __restrict__ partial, int slots, int n,
                                                            float* __restrict__ dW) {
    const int i = blockIdx.x * NT + threadIdx.x;
    if (i >= n) return;
    float s = 0.f;
    for (int b = 0; b < slots; ++b) s += partial[(size_t)b * n + i];
    dW[i] = s;
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

struct Shape {
    int CX, RY;
    dim3 grid;
};
Shape shape_of(int n_rows, int D, int max_slots) {
    Shape s;
    const int groups = D / 8;
    s.CX = 1;
    while (s.CX < groups && s.CX < NT) s.CX <<= 1;      // a power of two, so that it divides NT
    s.RY = NT / s.CX;
    const int gy = (groups + s.CX - 1) / s.CX;
    const int strips = (n_rows + STRIP - 1) / STRIP;
    int gx = (strips + s.RY - 1) / s.RY;
    const int fill = (sm_count() * 8 + gy - 1) / gy;     // enough CTAs for eight per SM
    if (gx > fill) gx = fill;
    if (max_slots && gx * s.RY > max_slots) gx = max_slots / s.RY;
    if (gx < 1) gx = 1;
    s.grid = dim3(gx, gy);
    return s;
}

bool args_ok(const void* a, const void* b, int32_t n_rows, int32_t D, int32_t w, int32_t dtype) {
    if (dtype != HARTS_FP32 && dtype != HARTS_BF16) return false;
    if (n_rows < 0 || D < 8 || (D & 7) || w < 2 || w > MAX_W) return false;
    if ((reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(b)) & 15) return false;
    return true;
}

template <typename T>
void launch_fwd(const Shape& s, cudaStream_t st, const void* x, const float* W, const int32_t* prev, void* y, int n,
                int D, int w) {
    const T* xx = static_cast<const T*>(x);
    T* yy = static_cast<T*>(y);
    constexpr size_t ring_bytes = (size_t)Ring<T>::DEPTH * NT * sizeof(Raw<T>);          // 32 KB
    if (w == 2) conv_fwd_kernel<T, 2><<<s.grid, NT, ring_bytes, st>>>(xx, W, prev, yy, n, D, s.CX);
    if (w == 3) conv_fwd_kernel<T, 3><<<s.grid, NT, ring_bytes, st>>>(xx, W, prev, yy, n, D, s.CX);
    if (w == 4) conv_fwd_kernel<T, 4><<<s.grid, NT, ring_bytes, st>>>(xx, W, prev, yy, n, D, s.CX);
}
template <typename T>
void launch_bwd(const Shape& s, cudaStream_t st, const void* x, const float* W, const void* dy, const int32_t* prev,
                const int32_t* cp, const int32_t* cr, void* dx, float* partial, int n, int D, int w) {
    const T *xx = static_cast<const T*>(x), *gg = static_cast<const T*>(dy);
    T* dd = static_cast<T*>(dx);
    constexpr size_t ring_bytes = 2 * (size_t)Ring<T>::DEPTH * NT * sizeof(Raw<T>);      // 64 KB
    cudaFuncSetAttribute(conv_bwd_kernel<T, 2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_bytes);
    cudaFuncSetAttribute(conv_bwd_kernel<T, 3>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_bytes);
    cudaFuncSetAttribute(conv_bwd_kernel<T, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)ring_bytes);
    if (w == 2) conv_bwd_kernel<T, 2><<<s.grid, NT, ring_bytes, st>>>(xx, W, gg, prev, cp, cr, dd, partial, n, D, s.CX);
    if (w == 3) conv_bwd_kernel<T, 3><<<s.grid, NT, ring_bytes, st>>>(xx, W, gg, prev, cp, cr, dd, partial, n, D, s.CX);
    if (w == 4) conv_bwd_kernel<T, 4><<<s.grid, NT, ring_bytes, st>>>(xx, W, gg, prev, cp, cr, dd, partial, n, D, s.CX);
}

}  // namespace

extern "C" int32_t harts_conv_fwd(const void* x, const float* W, const int32_t* prev_row, void* y, int32_t n_rows,
                                  int32_t D, int32_t w, int32_t dtype, void* stream) {
    if (!args_ok(x, y, n_rows, D, w, dtype)) return dtype > 1 || dtype < 0 ? HARTS_EUNSUPPORTED : HARTS_EINVAL;
    if (n_rows == 0) return HARTS_OK;
    if (!x || !y || !W || !prev_row || x == y) return HARTS_EINVAL;
    const Shape s = shape_of(n_rows, D, 0);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (dtype == HARTS_BF16) launch_fwd<__nv_bfloat16>(s, st, x, W, prev_row, y, n_rows, D, w);
    else launch_fwd<float>(s, st, x, W, prev_row, y, n_rows, D, w);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}

extern "C" int32_t harts_conv_scratch_bytes(int32_t D, int32_t w, size_t* bytes) {
    if (!bytes || D < 8 || (D & 7) || w < 2 || w > MAX_W) return HARTS_EINVAL;
    *bytes = (size_t)MAX_PARTIALS * D * w * sizeof(float);
    return HARTS_OK;
}

extern "C" int32_t harts_conv_bwd(const void* x, const float* W, const void* dy, const int32_t* next_row,
                                  const int32_t* child_ptr, const int32_t* child_row, void* dx, float* dW,
                                  void* scratch, int32_t n_rows, int32_t D, int32_t w, int32_t dtype, void* stream) {
    if (!args_ok(x, dx, n_rows, D, w, dtype)) return dtype > 1 || dtype < 0 ? HARTS_EUNSUPPORTED : HARTS_EINVAL;
    if (!dW || !scratch || (reinterpret_cast<uintptr_t>(scratch) & 15) || (reinterpret_cast<uintptr_t>(dy) & 15))
        return HARTS_EINVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (n_rows == 0) return cudaMemsetAsync(dW, 0, (size_t)D * w * sizeof(float), st) == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
    if (!x || !W || !dy || !next_row || !child_ptr || !child_row || !dx || dx == dy || dx == x) return HARTS_EINVAL;
    const Shape s = shape_of(n_rows, D, MAX_PARTIALS);
    float* partial = static_cast<float*>(scratch);
    if (dtype == HARTS_BF16)
        launch_bwd<__nv_bfloat16>(s, st, x, W, dy, next_row, child_ptr, child_row, dx, partial, n_rows, D, w);
    else
        launch_bwd<float>(s, st, x, W, dy, next_row, child_ptr, child_row, dx, partial, n_rows, D, w);
    const int n = D * w;
    conv_dw_reduce_kernel<<<(n + NT - 1) / NT, NT, 0, st>>>(partial, (int)s.grid.x * s.RY, n, dW);
    return cudaGetLastError() == cudaSuccess ? HARTS_OK : HARTS_ECUDA;
}
