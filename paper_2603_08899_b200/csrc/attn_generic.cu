// Generic tree attention: one CTA per (row, query head, sequence), CUDA-core fp32 math.
// Serves every dtype / head-dim / group size the tensor-core path does not take, and is the
// simplest statement of the masked online softmax on the GPU.
//
// Key order seen by a row: [soft-prompt entries (contemplate rows only)] [prefix slots] [tree
// slots allowed by the row's ancestor bitmask].
#include "common.cuh"

namespace confu {

template <typename T, int D>
__global__ void __launch_bounds__(128) attention_generic_kernel(
    confu_dims dm, const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
    const SlotMap map, const int32_t* __restrict__ prefix_len, const T* __restrict__ ks,
    const T* __restrict__ vs, const void* plan_raw, T* __restrict__ out, float* __restrict__ lse)
{
    constexpr int NT = 128;
    const int r = blockIdx.x, h = blockIdx.y, b = blockIdx.z;
    const int R = dm.T + dm.C, Hq = dm.Hq, Hkv = dm.Hkv, g = h / (Hq / Hkv);
    PlanView pv = plan_view(const_cast<void*>(plan_raw), dm.B);
    const int tid = threadIdx.x;
    T* orow = out + (((size_t)b * R + r) * Hq + h) * D;
    if (pv.bad[b]) {
        if (tid < D) orow[tid] = from_f32<T>(0.f);
        if (lse && tid == 0) lse[((size_t)b * R + r) * Hq + h] = 0.f;
        return;
    }
    const uint64_t mask = pv.mask[(size_t)b * kMaxRows + r];
    const int64_t P = prefix_len[b];
    const int S_vis = (r >= dm.T) ? dm.S : 0;
    const int64_t n = S_vis + P + R;
    const float scale = dm.sm_scale != 0.f ? dm.sm_scale : rsqrtf((float)D);

    __shared__ float s_q[D];
    __shared__ float s_p[NT];
    __shared__ float s_red[NT / 32];
    __shared__ float s_bcast[2];

    if (tid < D) s_q[tid] = to_f32(q[(((size_t)b * R + r) * Hq + h) * D + tid]) * scale;
    __syncthreads();

    float m_run = -INFINITY, l_run = 0.f, acc = 0.f;     // acc: output dim `tid` (tid < D)

    for (int64_t c0 = 0; c0 < n; c0 += NT) {
        const int64_t i = c0 + tid;
        float s = -INFINITY;
        if (i < n) {
            const T* kp;
            bool vis;
            if (i < S_vis) { kp = ks + ((size_t)i * Hkv + g) * D; vis = true; }
            else {
                const int64_t slot = i - S_vis;
                const int64_t j = slot - P;              // >= 0: the slot of query row j
                vis = j < 0 || (j < dm.T ? (int)((mask >> j) & 1ull) : (j == r));
                kp = kc + ((size_t)pool_slot(map, b, slot) * Hkv + g) * D;
            }
            if (vis) {
                float a = 0.f;
#pragma unroll 8
                for (int dd = 0; dd < D; ++dd) a = fmaf(s_q[dd], to_f32(kp[dd]), a);
                s = a;
            }
        }
        // block max
        float wm = warp_max(s);
        if ((tid & 31) == 0) s_red[tid >> 5] = wm;
        __syncthreads();
        if (tid == 0) {
            float cm = fmaxf(fmaxf(s_red[0], s_red[1]), fmaxf(s_red[2], s_red[3]));
            const float m_new = fmaxf(m_run, cm);
            s_bcast[0] = m_new;
        }
        __syncthreads();
        const float m_new = s_bcast[0];
        if (m_new == -INFINITY) { __syncthreads(); continue; }      // nothing visible yet
        const float alpha = (m_run == -INFINITY) ? 0.f : expf(m_run - m_new);
        const float p = (s == -INFINITY) ? 0.f : expf(s - m_new);
        s_p[tid] = p;
        float ws = warp_sum(p);
        __syncthreads();                       // s_red reads above are done, s_p visible below
        if ((tid & 31) == 0) s_red[tid >> 5] = ws;
        __syncthreads();
        l_run = l_run * alpha + (s_red[0] + s_red[1] + s_red[2] + s_red[3]);
        m_run = m_new;
        if (tid < D) {
            acc *= alpha;
            const int cnt = (int)((n - c0) < NT ? (n - c0) : NT);
            for (int j = 0; j < cnt; ++j) {
                const float pj = s_p[j];
                if (pj == 0.f) continue;
                const int64_t ii = c0 + j;
                const T* vp = (ii < S_vis) ? vs + ((size_t)ii * Hkv + g) * D
                                           : vc + ((size_t)pool_slot(map, b, ii - S_vis) * Hkv + g) * D;
                acc = fmaf(pj, to_f32(vp[tid]), acc);
            }
        }
        __syncthreads();
    }
    if (tid < D) orow[tid] = from_f32<T>(acc / l_run);
    if (lse && tid == 0) lse[((size_t)b * R + r) * Hq + h] = m_run + logf(l_run);
}

template <typename T>
static cudaError_t launch_t(const confu_dims& d, const void* q, const void* kc, const void* vc,
                            const SlotMap& map, const int32_t* prefix_len, const void* ks, const void* vs,
                            const void* plan, void* out, float* lse, cudaStream_t st)
{
    dim3 grid(d.T + d.C, d.Hq, d.B);
    if (d.B == 0) return cudaSuccess;
    if (d.D == 64)
        attention_generic_kernel<T, 64><<<grid, 128, 0, st>>>(d, (const T*)q, (const T*)kc, (const T*)vc, map,
                                                              prefix_len, (const T*)ks, (const T*)vs, plan, (T*)out, lse);
    else
        attention_generic_kernel<T, 128><<<grid, 128, 0, st>>>(d, (const T*)q, (const T*)kc, (const T*)vc, map,
                                                               prefix_len, (const T*)ks, (const T*)vs, plan, (T*)out, lse);
    return cudaGetLastError();
}

cudaError_t launch_attention_generic(const Ctx*, const confu_dims& d, const void* q, const void* k_cache,
                                     const void* v_cache, const SlotMap& map, const int32_t* prefix_len,
                                     const void* k_soft, const void* v_soft, const void* plan, void* out,
                                     float* lse, cudaStream_t st)
{
    if (d.kv_dtype == CONFU_F32)
        return launch_t<float>(d, q, k_cache, v_cache, map, prefix_len, k_soft, v_soft, plan, out, lse, st);
    return launch_t<__nv_bfloat16>(d, q, k_cache, v_cache, map, prefix_len, k_soft, v_soft, plan, out, lse, st);
}

}  // namespace confu
