// Shared declarations of the CUDA library (not used by the CPU oracle).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "confu.h"

namespace confu {

constexpr int kMaxRows = CONFU_MAX_ROWS;        // R = T + C <= 128
constexpr int kMaxTree = CONFU_MAX_TREE;        // T <= 64: one 64-bit word of visible tree slots per row
constexpr int kGroupRows = 64;                  // query rows the tensor-core kernel handles per pass over a pair's keys
constexpr int kPathLen = CONFU_MAX_DEPTH + 1;
constexpr int kTileKeys = 128;                  // keys per attention tile (tensor-core path)

// ---------------------------------------------------------------------------
// Plan buffer (device).  Built once per step by plan_kernel, read by every layer.
//   PlanHeader
//   uint64 mask[B][128]       bit j < T of mask[b][r]: row r sees the slot of tree row j.  (A contemplate
//                             row also sees its own slot and no other contemplate row's: not stored.)
//   int32  bad[B]             non-zero: malformed tree, sequence skipped
//   int32  tiles[B]           key tiles of one (sequence, kv head) pair, soft-prompt tile included
//   int64  tile_base[B + 1]   position of sequence b's first (sequence, kv head) stretch on the flat cost line (exclusive scan)
//   int32  seg_begin[kPlanMaxCtas + 1]   CTA c of the tensor-core kernel walks segs[seg_begin[c] .. seg_begin[c+1])
//   SegDesc segs[B * Hkv * 2 + kPlanMaxCtas]   the runs of key tiles, one pair at a time, of every CTA in walking order
//
// The split-KV work is balanced on a "cost line": every (sequence, kv head) pair takes
// tiles + kPairOverheadTiles consecutive positions (the overhead stands for loading Q, draining
// the pipeline and writing the output once per pair), pairs in (sequence, head) order.  The line is
// cut into n equal shares; share c covers positions [c*N/n, (c+1)*N/n); position q of a pair means
// key tile q - kPairOverheadTiles, so a share that ends inside a pair's overhead zone takes none of
// its tiles.  With n_rg groups of 64 query rows (n_rg = 1 or 2) there are n = n_ctas / n_rg shares and
// CTA c * n_rg + rg walks share c for row group rg: the CTAs of a share read the same K/V tiles at
// about the same time, so that only the first read of a tile goes to DRAM.
// ---------------------------------------------------------------------------
constexpr int kPairOverheadTiles = 4;
struct PlanHeader {
    int32_t B, Hkv, T, C, S, R;
    int32_t n_ctas;            // work units of the tensor-core attention launch: CTAs (<= SM count) or CTA pairs
    int32_t paired;            // 1: the runs are listed per CTA pair (two-SM kernel), 0: per CTA
    int64_t n_tiles;           // length N of the cost line
};

// One run of key tiles of one pair inside a CTA's share of the cost line.
constexpr int kPlanMaxCtas = 256;
struct alignas(16) SegDesc {
    int32_t b, g_rg;           // sequence; kv head | group of 64 query rows << 16
    int32_t t0, t1;            // tiles [t0, t1) of the pair
    int32_t nt, P;             // tiles of the pair (soft-prompt tile included); prefix length
    int32_t part_slot;         // -1: the run covers the whole pair; else the CTA's partial slot
    int32_t pad0;
    int64_t slot0;             // packed pool: the sequence's first slot
    int64_t pad1;
};
static_assert(sizeof(SegDesc) == 48, "SegDesc is read as three 16-byte words");

struct PlanView {
    PlanHeader* hdr;
    uint64_t* mask;
    int32_t* bad;
    int32_t* tiles;
    int64_t* tile_base;
    int32_t* seg_begin;
    SegDesc* segs;
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline size_t plan_bytes(int B, int Hkv)
{
    size_t n = align_up(sizeof(PlanHeader), 256);
    n += align_up((size_t)B * kMaxRows * sizeof(uint64_t), 256);
    n += align_up((size_t)B * sizeof(int32_t), 256);
    n += align_up((size_t)B * sizeof(int32_t), 256);
    n += align_up((size_t)(B + 1) * sizeof(int64_t), 256);
    n += align_up((size_t)(kPlanMaxCtas + 1) * sizeof(int32_t), 256);
    n += align_up(((size_t)B * Hkv * 2 + kPlanMaxCtas) * sizeof(SegDesc), 256);
    return n;
}

__host__ __device__ inline PlanView plan_view(void* base, int B)
{
    char* p = (char*)base;
    PlanView v;
    v.hdr = (PlanHeader*)p;                  p += align_up(sizeof(PlanHeader), 256);
    v.mask = (uint64_t*)p;                   p += align_up((size_t)B * kMaxRows * sizeof(uint64_t), 256);
    v.bad = (int32_t*)p;                     p += align_up((size_t)B * sizeof(int32_t), 256);
    v.tiles = (int32_t*)p;                   p += align_up((size_t)B * sizeof(int32_t), 256);
    v.tile_base = (int64_t*)p;               p += align_up((size_t)(B + 1) * sizeof(int64_t), 256);
    v.seg_begin = (int32_t*)p;               p += align_up((size_t)(kPlanMaxCtas + 1) * sizeof(int32_t), 256);
    v.segs = (SegDesc*)p;
    return v;
}

// Split-KV partial of the tensor-core path: per CTA two slots of M_MAX rows x (D fp32 + max + sum).
constexpr int kPartRows = 256;                  // 2 M-tiles of 128 rows
constexpr int kPartD = 128;
__host__ __device__ inline size_t partial_slot_bytes()
{
    return (size_t)kPartRows * kPartD * sizeof(float) + (size_t)kPartRows * 2 * sizeof(float);
}

// Where sequence b's slot s (0 = first prefix token) lives in a layer's pool: behind seq_start[b]
// in a packed pool, or in page block_table[b][s / 128] of a paged pool (pages of kTileKeys slots).
struct SlotMap {
    const int64_t* seq_start;
    const int32_t* block_table;    // [B][max_pages] page ids, or nullptr for a packed pool
    int32_t max_pages;
};
__device__ __forceinline__ int64_t pool_slot(const SlotMap& m, int b, int64_t s)
{
    if (m.block_table) return (int64_t)m.block_table[(size_t)b * m.max_pages + (s >> 7)] * kTileKeys + (s & (kTileKeys - 1));
    return m.seq_start[b] + s;
}

struct Ctx {
    int device;
    int sm_count;
    void* workspace;
    size_t workspace_bytes;
    const int32_t* block_table;    // paged pools when set (confu_set_paging)
    int32_t max_pages;
    cudaError_t last_error;
    const float* k_scale;          // E4M3 caches: per-kv-head scales (confu_set_kv_scales)
    const float* v_scale;
    int attention_path;            // CONFU_ATTENTION_* (confu_set_option)
    unsigned long long wait_ns;    // limit of the bounded waits inside the kernels
};

// A function attribute (the opt-in to more than 48 KB of dynamic shared memory) belongs to a
// device, not to the process: run `fn` once for every device that comes along as the current one.
struct OncePerDevice {
    static constexpr int kMaxDevices = 64;
    bool done[kMaxDevices] = {};
    template <typename F> cudaError_t run(F fn)
    {
        int dev = -1;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
        if (done[dev]) return cudaSuccess;
        e = fn();
        if (e == cudaSuccess) done[dev] = true;
        return e;
    }
};

// ---------------------------------------------------------------------------
// element access
// ---------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T> __device__ __forceinline__ T from_f32(float x);
template <> __device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---------------------------------------------------------------------------
// fast exponent and packed fp32 arithmetic
// ---------------------------------------------------------------------------
__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// Packed fp32 pairs (one 64-bit register): the FMA pipe takes two lanes per instruction.
__device__ __forceinline__ uint64_t f2_pack(float a, float b)
{
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& a, float& b) { asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v)); }
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c)
{
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b)
{
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// ---------------------------------------------------------------------------
// launchers (defined in the .cu files)
// ---------------------------------------------------------------------------
cudaError_t launch_plan(const Ctx* ctx, const confu_dims& d, const int64_t* seq_start, const int32_t* prefix_len,
                        const int32_t* parent, const int32_t* con_owner, void* plan, int32_t* status, bool paired,
                        cudaStream_t st);

cudaError_t launch_attention_generic(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                     const void* v_cache, const SlotMap& map, const int32_t* prefix_len,
                                     const void* k_soft, const void* v_soft, const void* plan, void* out,
                                     float* lse, cudaStream_t st);

cudaError_t launch_accept(const Ctx* ctx, int B, int T, int C, int V, int logit_dtype, const void* tl,
                          const void* dl, const int32_t* tokens, const int32_t* parent, const int32_t* con_owner,
                          const float* uniforms, float temperature, int sibling_mode, int32_t* accept_len,
                          int32_t* path, int32_t* next_token, int32_t* future_row, int32_t* counters,
                          void* workspace, int32_t* status, cudaStream_t st);
size_t accept_workspace_bytes(int B, int T, int V);

cudaError_t launch_accept_match(int B, int T, int C, int V, int logit_dtype, const void* tl, const int32_t* tokens,
                                const int32_t* parent, const int32_t* con_owner, const float* uniforms,
                                float temperature, int32_t* accept_len, int32_t* path, int32_t* next_token,
                                int32_t* future_row, int32_t* counters, int32_t* status, cudaStream_t st);

cudaError_t launch_compact(const Ctx* ctx, int B, int T, int n_layers, int64_t row_bytes, void* const* k_layers,
                           void* const* v_layers, const SlotMap& map, const int32_t* prefix_len,
                           const int32_t* accept_len, const int32_t* path, int32_t* new_prefix_len,
                           int32_t* status, cudaStream_t st);

cudaError_t launch_con_embedding(int B, int H_in, int H_out, int n_expert, int k_expert, int dtype, const void* hidden,
                                 const void* router_w, const void* router_b, const void* experts, int renormalize,
                                 void* out, int32_t* sel, float* gate, int32_t* status, cudaStream_t st);

cudaError_t launch_append(int B, int R, int64_t row_bytes, const void* k_rows, const void* v_rows, void* k_cache,
                          void* v_cache, const SlotMap& map, const int32_t* prefix_len, cudaStream_t st);

}  // namespace confu
