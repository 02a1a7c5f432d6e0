// Backward of all rounds with the scratch area in a fixed device array owned by the library, for callers
// that cannot hand in (or create) a scratch buffer.  Nothing here allocates: the array is part of the
// loaded module, and its device address is looked up once per device.
#include <mutex>

#include "kernels.h"
#include "plan.h"

namespace {

// Every GPU that loads the library holds this array until the process exits.
constexpr size_t STATIC_SCRATCH_BYTES = HARTS_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
std::mutex g_mutex;
void* g_scratch_addr[MAX_DEVICES] = {};   // device address of g_static_scratch on each device, once looked up

// In host code the array's name only stands for the symbol; the address a kernel can use comes from the runtime,
// separately for every device.
int32_t static_scratch_address(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return HARTS_ECUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return HARTS_ECUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return HARTS_OK;
}

}  // namespace

extern "C" int32_t harts_la_bwd_static(const harts_la_plan_t* plan, const void* dev_blob, const void* q, const void* k,
                                       const void* v, const float* g, const void* dO, void* dq, void* dk_, void* dv_,
                                       float* dg, const void* chunk_states, int32_t H, int32_t dk, int32_t dv,
                                       int32_t dtype, uint32_t flags, int32_t* dev_status, void* stream) {
    const harts::Plan* p = harts_la_plan_internal(plan);
    if (!p) return HARTS_EINVAL;
    harts_la_tables_t tb;
    int32_t rc = harts_la_plan_tables(plan, dev_blob, &tb);
    if (rc != HARTS_OK) return rc;
    if (H < 1 || dk < 1 || dv < 1) return HARTS_EINVAL;
    if (harts::scratch_layout(tb, H, dk, dv).total > STATIC_SCRATCH_BYTES) return HARTS_ESCRATCH;
    void* scratch = nullptr;
    if ((rc = static_scratch_address(&scratch)) != HARTS_OK) return rc;
    // Every scratch entry that the backward reads (initial-state gradients of consumer sequences, gradients of
    // replayed rows) is written earlier in the same call, so nothing has to be cleared between calls.
    for (int32_t r = p->n_rounds; r >= 1; r--) {
        rc = harts_la_bwd_seqs(&tb, p->round_seq_ptr[r - 1], p->round_seq_ptr[r], q, k, v, g, dO, dq, dk_, dv_, dg,
                               chunk_states, scratch, H, dk, dv, dtype, flags, dev_status, stream);
        if (rc != HARTS_OK) return rc;
    }
    return harts_la_bwd_finish(&tb, dk_, dv_, dg, scratch, H, dk, dv, dtype, stream);
}
