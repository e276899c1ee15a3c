// KV compaction of the accepted path: cache[P + k] <- cache[P + path[k]], k = 1..accept_len, for
// every layer and for K and V, in place.
//
// In-place safety without a snapshot: node ids are topologically numbered (parent < child), so
// path[k] >= k, the sources path[1] < path[2] < ... are increasing, and destination k can only
// coincide with a source of an EARLIER step (path[j] = k needs j <= k).  Each thread owns one
// 16-byte column of the row and walks k upwards in batches (all loads of a batch before its
// stores), so within a thread every source is read before any step at or after it overwrites
// that slot, and different threads never touch each other's columns.
//
// That argument needs path[0] = 0 < path[1] < ... < path[a] < T and a <= CONFU_MAX_DEPTH.  A path
// that breaks it (a stale or corrupted buffer) is not followed: the sequence gets the status code
// CONFU_ST_BAD_PATH, nothing of it is copied and its new prefix length is prefix_len + 1 (the root
// only).  Every thread checks the path itself (at most 64 cached loads), so no thread copies a row
// of a path another thread would have refused.
#include "common.cuh"

namespace confu {

constexpr int kCompactBatch = 8;

__global__ void __launch_bounds__(128) compact_kernel(int n_layers, int T, int64_t row_vecs, void* const* __restrict__ k_layers,
                                                      void* const* __restrict__ v_layers,
                                                      const SlotMap map,
                                                      const int32_t* __restrict__ prefix_len,
                                                      const int32_t* __restrict__ accept_len,
                                                      const int32_t* __restrict__ path,
                                                      int32_t* __restrict__ new_prefix_len,
                                                      int32_t* __restrict__ status)
{
    const int b = blockIdx.z, layer = blockIdx.y >> 1, kv = blockIdx.y & 1;
    const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int32_t* pth = path + (size_t)b * kPathLen;
    int a = accept_len[b];
    bool ok = a >= 0 && a <= CONFU_MAX_DEPTH && pth[0] == 0;
    if (ok) {
        int before = 0;
        for (int k = 1; k <= a; ++k) {
            const int node = pth[k];
            ok = ok && node > before && node < T;
            before = node;
        }
    }
    if (!ok) a = 0;
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
        if (new_prefix_len) new_prefix_len[b] = prefix_len[b] + a + 1;
        if (!ok && status) status[b] = CONFU_ST_BAD_PATH;
    }
    if (a == 0 || col >= row_vecs) return;
    uint4* pool = reinterpret_cast<uint4*>(kv ? v_layers[layer] : k_layers[layer]);
    const int64_t root = prefix_len[b];              // the root's slot, counted from the sequence's first
    for (int k0 = 1; k0 <= a; k0 += kCompactBatch) {
        uint4 buf[kCompactBatch];
#pragma unroll
        for (int j = 0; j < kCompactBatch; ++j)
            if (k0 + j <= a) buf[j] = pool[pool_slot(map, b, root + pth[k0 + j]) * row_vecs + col];
#pragma unroll
        for (int j = 0; j < kCompactBatch; ++j)
            if (k0 + j <= a) pool[pool_slot(map, b, root + k0 + j) * row_vecs + col] = buf[j];
    }
    (void)n_layers;
}

// cache[seq_start[b] + prefix_len[b] + r] = rows[b][r]  (K and V of the step's own query rows)
__global__ void __launch_bounds__(128) append_kernel(int R, int64_t row_vecs, const uint4* __restrict__ k_rows,
                                                     const uint4* __restrict__ v_rows, uint4* __restrict__ k_cache,
                                                     uint4* __restrict__ v_cache, const SlotMap map,
                                                     const int32_t* __restrict__ prefix_len)
{
    const int r = blockIdx.x, b = blockIdx.y, kv = blockIdx.z;
    const uint4* src = (kv ? v_rows : k_rows) + ((size_t)b * R + r) * row_vecs;
    uint4* dst = (kv ? v_cache : k_cache) + (size_t)pool_slot(map, b, (int64_t)prefix_len[b] + r) * row_vecs;
    for (int64_t c = threadIdx.x; c < row_vecs; c += blockDim.x) dst[c] = src[c];
}

// E4M3 cache: cache[...][g][d] = e4m3(rows[b][r][g][d] / scale[g]) (quotient in fp32, round to nearest even,
// saturating at 448).  One thread per 16 output bytes.
__global__ void __launch_bounds__(128) append_fp8_kernel(int R, int Hkv, int D, const __nv_bfloat16* __restrict__ k_rows,
                                                         const __nv_bfloat16* __restrict__ v_rows, uint8_t* __restrict__ k_cache,
                                                         uint8_t* __restrict__ v_cache, const SlotMap map,
                                                         const int32_t* __restrict__ prefix_len,
                                                         const float* __restrict__ k_scale, const float* __restrict__ v_scale)
{
    const int r = blockIdx.x, b = blockIdx.y, kv = blockIdx.z;
    const int row_elems = Hkv * D;
    const __nv_bfloat16* src = (kv ? v_rows : k_rows) + ((size_t)b * R + r) * row_elems;
    uint8_t* dst = (kv ? v_cache : k_cache) + (size_t)pool_slot(map, b, (int64_t)prefix_len[b] + r) * row_elems;
    const float* scale = kv ? v_scale : k_scale;
    for (int i = threadIdx.x * 16; i < row_elems; i += blockDim.x * 16) {
        const float s = scale[i / D];
        uint32_t w[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            float x[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) x[j] = __bfloat162float(src[i + 4 * q + j]) / s;
            uint32_t word;
            asm("{\n\t.reg .b16 lo, hi;\n\t"
                "cvt.rn.satfinite.e4m3x2.f32 lo, %2, %1;\n\t"
                "cvt.rn.satfinite.e4m3x2.f32 hi, %4, %3;\n\t"
                "mov.b32 %0, {lo, hi};\n\t}"
                : "=r"(word)
                : "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]));
            w[q] = word;
        }
        *reinterpret_cast<uint4*>(dst + i) = make_uint4(w[0], w[1], w[2], w[3]);
    }
}

cudaError_t launch_append_fp8(int B, int R, int Hkv, int D, const void* k_rows, const void* v_rows, void* k_cache,
                              void* v_cache, const SlotMap& map, const int32_t* prefix_len, const float* k_scale,
                              const float* v_scale, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    append_fp8_kernel<<<dim3(R, B, 2), 128, 0, st>>>(R, Hkv, D, (const __nv_bfloat16*)k_rows, (const __nv_bfloat16*)v_rows,
                                                     (uint8_t*)k_cache, (uint8_t*)v_cache, map, prefix_len, k_scale, v_scale);
    return cudaGetLastError();
}

cudaError_t launch_append(int B, int R, int64_t row_bytes, const void* k_rows, const void* v_rows, void* k_cache,
                          void* v_cache, const SlotMap& map, const int32_t* prefix_len, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    append_kernel<<<dim3(R, B, 2), 128, 0, st>>>(R, row_bytes / 16, (const uint4*)k_rows, (const uint4*)v_rows,
                                                 (uint4*)k_cache, (uint4*)v_cache, map, prefix_len);
    return cudaGetLastError();
}

cudaError_t launch_compact(const Ctx*, int B, int T, int n_layers, int64_t row_bytes, void* const* k_layers,
                           void* const* v_layers, const SlotMap& map, const int32_t* prefix_len,
                           const int32_t* accept_len, const int32_t* path, int32_t* new_prefix_len,
                           int32_t* status, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const int64_t row_vecs = row_bytes / 16;
    // with no layers there is still new_prefix_len to write: one block row does it
    dim3 grid((unsigned)((row_vecs + 127) / 128), (unsigned)(n_layers > 0 ? 2 * n_layers : 1), (unsigned)B);
    if (n_layers == 0) {
        compact_kernel<<<dim3(1, 1, B), 128, 0, st>>>(0, T, 0, k_layers, v_layers, map, prefix_len, accept_len, path,
                                                       new_prefix_len, status);
    } else {
        compact_kernel<<<grid, 128, 0, st>>>(n_layers, T, row_vecs, k_layers, v_layers, map, prefix_len, accept_len,
                                             path, new_prefix_len, status);
    }
    return cudaGetLastError();
}

}  // namespace confu
