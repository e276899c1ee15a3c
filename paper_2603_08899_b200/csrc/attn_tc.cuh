// Declarations shared by the tensor-core attention kernel (attn_tc.cu) and the kernels that merge
// its split-KV partial results (combine.cu).
#pragma once

#include "common.cuh"

namespace confu {
namespace tc {

constexpr int kD = 128;

struct Params {
    confu_dims d;
    SlotMap map;         // packed pool (seq_start) or paged pool (block table, pages of 128 slots = one key tile)
    const int32_t* prefix_len;
    const void* plan;
    float* partials;
    __nv_bfloat16* out;
    float* lse;
    int32_t* status;
    int n_mt;            // M tiles in use (R > 32 ? 2 : 1)
    int n_rg;            // groups of 64 query rows (R > 64 ? 2 : 1); a pair = (sequence, kv head, row group)
    int G;
    float c;             // sm_scale * log2(e)
    unsigned long long wait_ns;   // limit of every wait on an mbarrier (wall clock)
    const float* k_scale;         // E4M3 cache: value = code * scale[kv head] (device, [Hkv]); unused otherwise
    const float* v_scale;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Enqueues the merge of the partial results that the attention launch with the same parameters
// left in prm.partials (pairs whose key tiles were split over several CTAs).
cudaError_t launch_combine(const Params& prm, int sm_count, cudaStream_t st);

}  // namespace tc
}  // namespace confu
