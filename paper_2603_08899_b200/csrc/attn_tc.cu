// Tensor-core (tcgen05 + TMA) tree attention -- placeholder until the kernel lands.
#include "common.cuh"

namespace confu {

bool tc_attention_supported(const confu_dims&) { return false; }

cudaError_t launch_attention_tc(const Ctx*, const confu_dims&, const void*, const void*, const void*, int64_t,
                                const int64_t*, const int32_t*, const void*, const void*, const void*, void*, void*,
                                float*, int32_t*, cudaStream_t)
{
    return cudaErrorNotSupported;
}

}  // namespace confu
