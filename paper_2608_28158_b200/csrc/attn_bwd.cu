// Backward of attention on compact tokens -- placeholder until the kernels land.
#include "kernels.h"
#include "../../include/harts_attn.h"
namespace harts {
int32_t attn_bwd_launch(const int32_t*, const int32_t*, const void*, const void*, const void*, const void*,
                        const float*, const void*, void*, void*, void*, float*, int, int, float, int32_t*,
                        cudaStream_t) {
    return HARTS_EUNSUPPORTED;
}
}  // namespace harts
