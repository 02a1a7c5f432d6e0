// Internal launch interface between the C ABI (api.cu) and the kernel files.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstddef>
#include <cstdint>

#include "../../include/harts_la.h"

namespace harts {

struct FwdArgs {
    harts_la_tables_t tb;
    int32_t seq_lo, seq_hi;
    const void *q, *k, *v;
    const float* g;
    void* o;
    float* slots;
    void* chunk_states;
    int32_t H, dk, dv, dtype;
    uint32_t flags;
    int32_t* dev_status;
    cudaStream_t stream;
};

struct BwdArgs {
    harts_la_tables_t tb;
    int32_t seq_lo, seq_hi;
    const void *q, *k, *v;
    const float* g;
    const void* dO;
    void *dq, *dk_, *dv_;
    float* dg;
    const void* chunk_states;
    void* scratch;
    int32_t H, dk, dv, dtype;
    uint32_t flags;
    int32_t* dev_status;
    cudaStream_t stream;
};

// Byte offsets inside the backward scratch buffer (each region 256-byte aligned).
struct ScratchLayout {
    size_t ds0;    // [n_seq, H, dk, dv] fp32: gradient w.r.t. each sequence's initial state
    size_t rk;     // [n_replay, H, dk] fp32: dk of replayed rows
    size_t rv;     // [n_replay, H, dv] fp32
    size_t rg;     // [n_replay, H] fp32
    size_t total;
};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline ScratchLayout scratch_layout(const harts_la_tables_t& tb, int32_t H, int32_t dk, int32_t dv) {
    ScratchLayout s;
    size_t off = 0;
    s.ds0 = off;
    off = align_up(off + (size_t)tb.n_seq * H * dk * dv * sizeof(float), 256);
    s.rk = off;
    off = align_up(off + (size_t)tb.n_replay * H * dk * sizeof(float), 256);
    s.rv = off;
    off = align_up(off + (size_t)tb.n_replay * H * dv * sizeof(float), 256);
    s.rg = off;
    off = align_up(off + (size_t)tb.n_replay * H * sizeof(float), 256);
    s.total = off < 256 ? 256 : off;
    return s;
}

// With HARTS_FLAG_CHECK_TABLES the kernels of a call run only while the status word is still zero: check_tables (a
// validation kernel ahead of them on the stream) records a bad index there, and nothing is dereferenced after it.
inline const int32_t* status_gate(uint32_t flags, const int32_t* dev_status) {
    return (flags & HARTS_FLAG_CHECK_TABLES) ? dev_status : nullptr;
}
#ifdef __CUDACC__
__device__ __forceinline__ bool gate_closed(const int32_t* gate) {     // called by every thread of the CTA
    if (!gate) return false;
    __shared__ int closed;
    if (threadIdx.x == 0) closed = *reinterpret_cast<const volatile int32_t*>(gate);
    __syncthreads();
    return closed != 0;
}
#endif
int32_t check_tables(const harts_la_tables_t& tb, int32_t seq_lo, int32_t seq_hi, int32_t* dev_status, cudaStream_t stream);

// The same for the per-channel-decay calls: the replay-row gradient of g is a vector over the key channels.
struct GkScratchLayout {
    size_t ds0, rk, rv, rg, total;     // rg: [n_replay, H, dk] fp32
};
inline GkScratchLayout gk_scratch_layout(const harts_la_tables_t& tb, int32_t H, int32_t dk, int32_t dv) {
    GkScratchLayout s;
    size_t off = 0;
    s.ds0 = off;
    off = align_up(off + (size_t)tb.n_seq * H * dk * dv * sizeof(float), 256);
    s.rk = off;
    off = align_up(off + (size_t)tb.n_replay * H * dk * sizeof(float), 256);
    s.rv = off;
    off = align_up(off + (size_t)tb.n_replay * H * dv * sizeof(float), 256);
    s.rg = off;
    off = align_up(off + (size_t)tb.n_replay * H * dk * sizeof(float), 256);
    s.total = off < 256 ? 256 : off;
    return s;
}

int32_t gk_supported(int32_t dtype, int32_t dk, int32_t dv);
int32_t gk_fwd(const FwdArgs& a);      // FwdArgs::g / BwdArgs::g, ::dg point to [rows, H, dk] arrays here
int32_t gk_bwd(const BwdArgs& a);
// bf16, d_k = d_v = 128: the dense products on the tensor cores (la_gk_mma.cu); taken unless HARTS_FLAG_FMA_KERNELS
int32_t gk_mma_supported(int32_t dtype, int32_t dk, int32_t dv);
int32_t gk_mma_fwd(const FwdArgs& a);
int32_t gk_mma_bwd(const BwdArgs& a);
int32_t gk_replay_reduce(const harts_la_tables_t& tb, void* dk_, void* dv_, float* dgk, const void* scratch, int32_t H,
                         int32_t dk, int32_t dv, int32_t dtype, cudaStream_t stream);

int32_t fma_supported(int32_t dtype, int32_t dk, int32_t dv);
int32_t fma_fwd(const FwdArgs& a);
int32_t fma_bwd(const BwdArgs& a);
int32_t tc_supported(int32_t dtype, int32_t dk, int32_t dv);
int32_t tc_fwd(const FwdArgs& a);
int32_t tc_fwd_fused(const FwdArgs& a, int* flags, int* ticket);     // all rounds in one launch

// Flags for the one-launch forms, kept behind the chunk states in the chunk-state workspace: one int32 per
// (slot, head) for the forward, one per (sequence, head) for the backward.
inline size_t chunk_state_payload(const harts_la_tables_t& tb, int32_t H, int32_t dk, int32_t dv, size_t elem) {
    return align_up((size_t)tb.n_chunks * H * dk * dv * elem, 256);
}
// flags of the one-launch forms: n_slots * H (forward), n_seq * H (backward), then one ticket counter each
inline size_t fused_flag_count(const harts_la_tables_t& tb, int32_t H) { return ((size_t)tb.n_slots + tb.n_seq) * H; }
inline size_t fused_flag_bytes(const harts_la_tables_t& tb, int32_t H) {
    return align_up((fused_flag_count(tb, H) + 2) * sizeof(int32_t), 256);
}
// the plan's round table by value (kernel argument): sequences of round r (0-based) = [ptr[r], ptr[r + 1])
constexpr int MAX_FUSED_ROUNDS = 32;
constexpr int ONE_LAUNCH_ITEMS_PER_CTA = 8;    // the one-launch forms are offered up to this many items per resident CTA
struct RoundOrder {
    int n;
    int ptr[MAX_FUSED_ROUNDS + 1];
};
int32_t gk_mma_fwd_all(const FwdArgs& a, int* flags, int* ticket);     // all rounds in one launch (la_gk_mma.cu)
int32_t gk_mma_bwd_all(const BwdArgs& a, int* flags, int* ticket, const RoundOrder& rounds);
int32_t tc_bwd(const BwdArgs& a);
int32_t tc_bwd_fused(const BwdArgs& a, int* flags, int* ticket, const RoundOrder& rounds);   // all rounds in one launch
int32_t handoff_reduce(const BwdArgs& a);
int32_t replay_reduce(const harts_la_tables_t& tb, void* dk_, void* dv_, float* dg, const void* scratch, int32_t H,
                      int32_t dk, int32_t dv, int32_t dtype, cudaStream_t stream);

}  // namespace harts
