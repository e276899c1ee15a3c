// confu_tree_accept_static: the acceptance step for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a serving engine whose
// memory pool owns the whole device, in a plugin that is handed streams but no allocator, or in a
// latency-critical loop where an allocation would synchronise the device.  confu_tree_accept asks
// such a caller for a workspace it has no means to provide.  This variant keeps the row-statistics
// scratch in a fixed array that is part of the loaded library image instead, so the caller passes
// inputs and outputs only.
//
// The array lives in every CUDA context that loads the library until the process exits
// (kStaticScratchBytes per device), all calls share it, and it keeps whatever the last call left
// there.  Nothing in it has to start at zero: every entry the walk kernel reads has been written
// by the statistics kernel of the same call.  Two calls that overlap on the GPU (different streams,
// or different host threads) race on it; serialise them.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int kStaticMaxRows = 4096;                                  // B * T of one call
constexpr size_t kStaticScratchBytes = (size_t)2 * kStaticMaxRows * 16 * 16;   // 2 matrices x rows x 16 chunks x 16 B = 2 MiB

static __device__ __align__(256) unsigned char g_accept_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

// The array's name is only a handle on the host; the address the kernels need comes from the
// runtime, per device, with that device current.  Done once per device, on the first call.
cudaError_t scratch_address(void** out)
{
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_accept_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace

extern "C" {

size_t confu_tree_accept_static_max_rows(void) { return (size_t)kStaticMaxRows; }

int confu_tree_accept_static(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                             const void* target_logits, const void* draft_logits, const int32_t* tokens,
                             const int32_t* parent, const int32_t* con_owner, const float* uniforms,
                             float temperature, int32_t sibling_mode, int32_t* accept_len, int32_t* path,
                             int32_t* next_token, int32_t* future_row, int32_t* counters, int32_t* status,
                             void* stream)
{
    if (B < 0 || T <= 0 || C < 0 || V <= 0) return CONFU_ERR_SHAPE;
    if (logit_dtype != CONFU_BF16 && logit_dtype != CONFU_F32) return CONFU_ERR_ARG;
    if ((sibling_mode & ~CONFU_ACCEPT_LAZY) != 0 && (sibling_mode & ~CONFU_ACCEPT_LAZY) != 1) return CONFU_ERR_ARG;
    if (!(temperature >= 0.f)) return CONFU_ERR_ARG;
    if (T > CONFU_MAX_TREE || C > CONFU_MAX_TREE || V > 262144) return CONFU_ERR_UNSUPPORTED;
    // the fixed scratch holds the statistics of at most kStaticMaxRows logit rows per matrix
    if ((int64_t)B * T > kStaticMaxRows) return CONFU_ERR_WORKSPACE;
    if (B == 0) return CONFU_OK;
    if (!target_logits || !tokens || !parent || !accept_len || !path || !next_token) return CONFU_ERR_ARG;
    if (C > 0 && !con_owner) return CONFU_ERR_ARG;
    if (temperature > 0.f && (!draft_logits || !uniforms)) return CONFU_ERR_ARG;
    if ((reinterpret_cast<uintptr_t>(target_logits) & 15u) || (reinterpret_cast<uintptr_t>(draft_logits) & 15u))
        return CONFU_ERR_ALIGN;
    if (confu::accept_workspace_bytes(B, T, V) > kStaticScratchBytes) return CONFU_ERR_WORKSPACE;
    void* scratch = nullptr;
    if (scratch_address(&scratch) != cudaSuccess) return CONFU_ERR_CUDA;
    cudaError_t e = confu::launch_accept(nullptr, B, T, C, V, logit_dtype, target_logits, draft_logits, tokens, parent,
                                         con_owner, uniforms, temperature, sibling_mode, accept_len, path, next_token,
                                         future_row, counters, scratch, status, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : CONFU_ERR_CUDA;
}

}  // extern "C"
