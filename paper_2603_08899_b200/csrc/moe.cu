// Contemplate-token embedding as a mixture of expert embeddings: router linear layer on the hidden
// state of the most recently accepted token, softmax over the experts, the k largest scores, sum of
// the chosen experts' embeddings weighted by their gating scores.
//
// One CTA per sequence.  The router is n_expert dot products of length H_in: a warp per expert,
// lanes striding the hidden dimension with 16-byte loads, fp32 accumulation; the router matrix is
// the same for every sequence and stays in L2.  The softmax and the selection (k rounds of a warp
// argmax, the lower index on equal scores) run in one warp; the output is written 16 bytes per
// thread.  A few hundred KB per sequence: the kernel is bound by latency, not by bandwidth.
//
// A non-finite router score (a NaN or an infinity in the hidden state or the router) makes the
// scores of the sequence meaningless: the sequence's output row is written as zeros, its selection
// as experts 0..k-1 with gate 0, and status[b] (optional) gets CONFU_ST_NONFINITE.  The selected
// indices are clamped to the table whatever the scores are, so no input value can send a load or a
// store out of bounds.
#include "common.cuh"

namespace confu {

constexpr int kMoeThreads = 256;
constexpr int kMoeMaxExperts = 1024;
constexpr int kMoeMaxK = 32;

template <typename T> struct Vec16;
template <> struct Vec16<__nv_bfloat16> { static constexpr int n = 8; };
template <> struct Vec16<float> { static constexpr int n = 4; };

template <typename T>
__device__ __forceinline__ void load_vec(const T* p, float (&x)[Vec16<T>::n])
{
    if constexpr (sizeof(T) == 2) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            x[2 * j] = __uint_as_float(w[j] << 16);
            x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
        }
    } else {
        const float4 v = *reinterpret_cast<const float4*>(p);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
    }
}

template <typename T>
__global__ void __launch_bounds__(kMoeThreads) con_embedding_kernel(
    int H_in, int H_out, int n_expert, int k_expert, const T* __restrict__ hidden, const T* __restrict__ router_w,
    const T* __restrict__ router_b, const T* __restrict__ experts, int renormalize, T* __restrict__ out,
    int32_t* __restrict__ sel, float* __restrict__ gate, int32_t* __restrict__ status)
{
    constexpr int kVec = Vec16<T>::n;
    __shared__ float s_score[kMoeMaxExperts];
    __shared__ int s_sel[kMoeMaxK];
    __shared__ float s_w[kMoeMaxK];
    __shared__ int s_bad;
    const int b = blockIdx.x, tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const T* h = hidden + (size_t)b * H_in;
    const bool vec_in = H_in % kVec == 0, vec_out = H_out % kVec == 0;

    if (tid == 0) s_bad = 0;
    __syncthreads();
    // ---- router logits ----
    for (int e = warp; e < n_expert; e += kMoeThreads / 32) {
        const T* w = router_w + (size_t)e * H_in;
        float acc = 0.f;
        if (vec_in) {
            for (int i = lane * kVec; i < H_in; i += 32 * kVec) {
                float x[kVec], y[kVec];
                load_vec(h + i, x);
                load_vec(w + i, y);
#pragma unroll
                for (int j = 0; j < kVec; ++j) acc = fmaf(x[j], y[j], acc);
            }
        } else {
            for (int i = lane; i < H_in; i += 32) acc = fmaf(to_f32(h[i]), to_f32(w[i]), acc);
        }
        acc = warp_sum(acc);
        if (lane == 0) {
            const float sc = acc + (router_b ? to_f32(router_b[e]) : 0.f);
            s_score[e] = sc;
            if (!(fabsf(sc) <= 3.0e38f)) s_bad = 1;
        }
    }
    __syncthreads();
    if (s_bad) {
        T* o = out + (size_t)b * H_out;
        for (int j = tid; j < H_out; j += kMoeThreads) o[j] = from_f32<T>(0.f);
        if (tid < k_expert) {
            if (sel) sel[(size_t)b * k_expert + tid] = tid;
            if (gate) gate[(size_t)b * k_expert + tid] = 0.f;
        }
        if (tid == 0 && status) status[b] = CONFU_ST_NONFINITE;
        return;
    }

    // ---- softmax and the k largest scores (one warp) ----
    if (warp == 0) {
        float m = -INFINITY;
        for (int e = lane; e < n_expert; e += 32) m = fmaxf(m, s_score[e]);
        m = warp_max(m);
        float z = 0.f;
        for (int e = lane; e < n_expert; e += 32) {
            const float p = __expf(s_score[e] - m);
            s_score[e] = p;
            z += p;
        }
        z = warp_sum(z);
        const float inv_z = 1.f / z;
        __syncwarp();
        float wsum = 0.f;
        for (int k = 0; k < k_expert; ++k) {
            float bv = -1.f;                     // scores are >= 0; a taken expert is marked -1
            int be = INT_MAX;
            for (int e = lane; e < n_expert; e += 32) {
                const float p = s_score[e];
                if (p > bv) { bv = p; be = e; }                  // ascending e: the lower index wins a tie
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
                const int oe = __shfl_xor_sync(0xffffffffu, be, o);
                if (ov > bv || (ov == bv && oe < be)) { bv = ov; be = oe; }
            }
            be = min(max(be, 0), n_expert - 1);       // finite scores always give an index; never trust that for an address
            if (lane == 0) {
                s_sel[k] = be;
                s_w[k] = bv * inv_z;
                s_score[be] = -1.f;
            }
            wsum += bv * inv_z;
            __syncwarp();
        }
        if (renormalize && lane < k_expert) s_w[lane] = s_w[lane] / wsum;
        __syncwarp();
        if (lane < k_expert) {
            if (sel) sel[(size_t)b * k_expert + lane] = s_sel[lane];
            if (gate) gate[(size_t)b * k_expert + lane] = s_w[lane];
        }
    }
    __syncthreads();

    // ---- weighted sum of the chosen embeddings ----
    T* o = out + (size_t)b * H_out;
    if (vec_out) {
        for (int j = tid * kVec; j < H_out; j += kMoeThreads * kVec) {
            float acc[kVec];
#pragma unroll
            for (int i = 0; i < kVec; ++i) acc[i] = 0.f;
            for (int k = 0; k < k_expert; ++k) {
                float x[kVec];
                load_vec(experts + (size_t)s_sel[k] * H_out + j, x);
                const float w = s_w[k];
#pragma unroll
                for (int i = 0; i < kVec; ++i) acc[i] = fmaf(w, x[i], acc[i]);
            }
#pragma unroll
            for (int i = 0; i < kVec; ++i) o[j + i] = from_f32<T>(acc[i]);
        }
    } else {
        for (int j = tid; j < H_out; j += kMoeThreads) {
            float acc = 0.f;
            for (int k = 0; k < k_expert; ++k) acc = fmaf(s_w[k], to_f32(experts[(size_t)s_sel[k] * H_out + j]), acc);
            o[j] = from_f32<T>(acc);
        }
    }
}

cudaError_t launch_con_embedding(int B, int H_in, int H_out, int n_expert, int k_expert, int dtype, const void* hidden,
                                 const void* router_w, const void* router_b, const void* experts, int renormalize,
                                 void* out, int32_t* sel, float* gate, int32_t* status, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    if (dtype == CONFU_F32)
        con_embedding_kernel<float><<<B, kMoeThreads, 0, st>>>(H_in, H_out, n_expert, k_expert, (const float*)hidden,
                                                               (const float*)router_w, (const float*)router_b,
                                                               (const float*)experts, renormalize, (float*)out, sel, gate, status);
    else
        con_embedding_kernel<__nv_bfloat16><<<B, kMoeThreads, 0, st>>>(
            H_in, H_out, n_expert, k_expert, (const __nv_bfloat16*)hidden, (const __nv_bfloat16*)router_w,
            (const __nv_bfloat16*)router_b, (const __nv_bfloat16*)experts, renormalize, (__nv_bfloat16*)out, sel, gate, status);
    return cudaGetLastError();
}

}  // namespace confu
