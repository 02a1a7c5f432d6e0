// C entry points of attention on compact tokens: argument checks and launches.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/harts_attn.h"

namespace harts {
int32_t attn_fwd_launch(const int32_t* hi, const int32_t* di, const void* q, const void* k, const void* v, void* o,
                        float* lse, int Hq, int Hkv, float scale, int32_t* status, cudaStream_t st);
int32_t attn_bwd_launch(const int32_t* hi, const int32_t* di, const void* q, const void* k, const void* v,
                        const void* o, const float* lse, const void* dO, void* dq, void* dk_, void* dv_, float* delta,
                        int Hq, int Hkv, float scale, int32_t* status, cudaStream_t st);
}  // namespace harts

namespace {
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int32_t check_common(const int32_t* hi, const int32_t* di, int32_t Hq, int32_t Hkv, int32_t d, float scale,
                     int32_t dtype) {
    if (!hi || !di || hi[0] < 0 || hi[6] < HARTS_ATTN_HEADER_WORDS || !aligned16(di)) return HARTS_EINVAL;
    if (dtype != HARTS_BF16 || d != 128) return HARTS_EUNSUPPORTED;
    if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || !(scale > 0.f)) return HARTS_EINVAL;
    return HARTS_OK;
}
}  // namespace

extern "C" int32_t harts_attn_fwd(const int32_t* host_index, const int32_t* dev_index, const void* q, const void* k,
                                  const void* v, void* o, float* lse, int32_t Hq, int32_t Hkv, int32_t d, float scale,
                                  int32_t dtype, int32_t* dev_status, void* stream) {
    int32_t rc = check_common(host_index, dev_index, Hq, Hkv, d, scale, dtype);
    if (rc != HARTS_OK) return rc;
    if (host_index[0] == 0) return HARTS_OK;
    if (!q || !k || !v || !o || !lse || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o))
        return HARTS_EINVAL;
    return harts::attn_fwd_launch(host_index, dev_index, q, k, v, o, lse, Hq, Hkv, scale, dev_status,
                                  static_cast<cudaStream_t>(stream));
}

extern "C" int32_t harts_attn_bwd(const int32_t* host_index, const int32_t* dev_index, const void* q, const void* k,
                                  const void* v, const void* o, const float* lse, const void* dO, void* dq, void* dk_,
                                  void* dv_, float* delta, int32_t Hq, int32_t Hkv, int32_t d, float scale,
                                  int32_t dtype, int32_t* dev_status, void* stream) {
    int32_t rc = check_common(host_index, dev_index, Hq, Hkv, d, scale, dtype);
    if (rc != HARTS_OK) return rc;
    if (host_index[0] == 0) return HARTS_OK;
    if (!q || !k || !v || !o || !lse || !dO || !dq || !dk_ || !dv_ || !delta) return HARTS_EINVAL;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || !aligned16(dO) || !aligned16(dq) ||
        !aligned16(dk_) || !aligned16(dv_))
        return HARTS_EINVAL;
    return harts::attn_bwd_launch(host_index, dev_index, q, k, v, o, lse, dO, dq, dk_, dv_, delta, Hq, Hkv, scale,
                                  dev_status, static_cast<cudaStream_t>(stream));
}
