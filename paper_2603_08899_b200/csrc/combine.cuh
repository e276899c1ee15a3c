// The merge of the split-KV partial results of one output row by one warp, shared by the kernel that
// merges after the attention launch (combine.cu) and by the attention kernel that merges inside its
// own launch (attn_tc2.cu).
#pragma once

#include "attn_tc.cuh"

namespace confu {
namespace tc {

// Output row (b, r, head g * G + hl) and its lse as zeros, by one warp: what a sequence with a
// malformed tree gets (the same as on the generic path).
__device__ __forceinline__ void zero_row(const Params& prm, int b, int g, int r, int hl, int lane)
{
    const int R = prm.d.T + prm.d.C, Hq = prm.d.Hq;
    if (r >= R) return;
    const int h = g * prm.G + hl;
    reinterpret_cast<uint2*>(prm.out + (((size_t)b * R + r) * Hq + h) * kD)[lane] = make_uint2(0u, 0u);
    if (prm.lse && lane == 0) prm.lse[((size_t)b * R + r) * Hq + h] = 0.f;
}

// The merge of one output row by one warp, in two steps so that a caller can work out what there is
// to do (plan data only) before the partial results exist.
struct MergeJob {
    int kind;                 // 0: nothing to do (no such row, or one CTA covered the pair and wrote it), 1: zeros, 2: merge
    int b, g, r, hl;          // the output row: sequence, kv head, query row, head inside the GQA group
    int row;                  // row of the partial slots
    int c_first, c_last;      // first and last CTA (or CTA pair) that walked the pair; every n_rg-th in between did too
};

// Row `lane_row` (0..127) of M tile t of pair (sequence, kv head, row group).
__device__ __forceinline__ MergeJob merge_job(const Params& prm, const PlanView& pv, int pair, int t, int lane_row)
{
    MergeJob j;
    j.kind = 0;
    // pairs: sequence major, then kv head, then row group
    const int per_seq = prm.d.Hkv * prm.n_rg;
    const int b = pair / per_seq, g = (pair % per_seq) / prm.n_rg, rg = pair % prm.n_rg;
    const int G = prm.G, R = prm.d.T + prm.d.C;
    j.b = b;
    j.g = g;
    j.r = kGroupRows * rg + 32 * t + lane_row / G;
    j.hl = lane_row % G;
    j.row = t * 128 + lane_row;
    j.c_first = j.c_last = 0;
    if (t >= prm.n_mt || lane_row >= 32 * G || j.r >= R) return j;
    const int nt = pv.tiles[b];
    if (nt == 0) {                                      // malformed tree: no CTA worked on the pair; its rows read 0
        j.kind = 1;
        return j;
    }
    const int64_t N = pv.hdr->n_tiles, n = pv.hdr->n_ctas / prm.n_rg;
    // key tile q of (sequence, kv head) sits at position F + q of the cost line; position x belongs to lane
    // floor(((x + 1) * n - 1) / N) of the n lanes, and row group rg of lane c is walked by CTA c * n_rg + rg
    const int64_t F = pv.tile_base[b] + (int64_t)g * (nt + kPairOverheadTiles) + kPairOverheadTiles;
    j.c_first = (int)(((F + 1) * n - 1) / N) * prm.n_rg + rg;
    j.c_last = (int)(((F + nt) * n - 1) / N) * prm.n_rg + rg;
    if (j.c_first != j.c_last) j.kind = 2;              // else one CTA covered the pair and wrote the output itself
    return j;
}

// The row's partial results (one per CTA that walked the pair) merged in CTA order.  The parts' maxima
// and sums are taken one per lane; with at most 16 parts every load of the row is in flight at once
// (one round trip to L2), with more the rows of eight parts at a time.  The order of every sum is
// fixed by the part index alone, so the result does not depend on the run.  Partial results are read
// past L1: they were written by other SMs, possibly inside this very launch.
__device__ __forceinline__ void merge_run(const Params& prm, const MergeJob& j, int lane)
{
    if (j.kind == 0) return;
    if (j.kind == 1) {
        zero_row(prm, j.b, j.g, j.r, j.hl, lane);
        return;
    }
    const int R = prm.d.T + prm.d.C, Hq = prm.d.Hq, row = j.row;
    const int c_first = j.c_first, c_last = j.c_last, n_rg = prm.n_rg;
    const int n_parts = (c_last - c_first) / n_rg + 1;
    const size_t slot_floats = partial_slot_bytes() / sizeof(float);
    auto slot_of = [&](int p) {                         // part p of the pair: the partial slot of the p-th CTA that walked it
        const int cta = c_first + p * n_rg;
        return prm.partials + (size_t)(2 * cta + (cta < c_last ? 1 : 0)) * slot_floats;
    };
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float M = -INFINITY, L = 0.f;
    if (n_parts <= 16) {
        float m = -INFINITY, l = 0.f;
        if (lane < n_parts) {
            const float* ml = slot_of(lane) + (size_t)kPartRows * kPartD;
            m = __ldcg(ml + row);
            l = __ldcg(ml + kPartRows + row);
        }
        float4 v[16];
#pragma unroll
        for (int k = 0; k < 16; ++k)
            v[k] = k < n_parts ? __ldcg(reinterpret_cast<const float4*>(slot_of(k) + (size_t)row * kPartD) + lane)
                               : make_float4(0.f, 0.f, 0.f, 0.f);
        M = warp_max(m);
        const float w = (m == -INFINITY) ? 0.f : ex2(m - M);
        L = warp_sum(w * l);
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const float wk = __shfl_sync(0xffffffffu, w, k);              // 0 past the last part
            acc.x = fmaf(wk, v[k].x, acc.x); acc.y = fmaf(wk, v[k].y, acc.y);
            acc.z = fmaf(wk, v[k].z, acc.z); acc.w = fmaf(wk, v[k].w, acc.w);
        }
    } else {
        for (int p = lane; p < n_parts; p += 32) M = fmaxf(M, __ldcg(slot_of(p) + (size_t)kPartRows * kPartD + row));
        M = warp_max(M);
        for (int p0 = 0; p0 < n_parts; p0 += 32) {
            float w = 0.f, wl = 0.f;                    // this lane's part of the group: weight, weight * sum
            if (p0 + lane < n_parts) {
                const float* ml = slot_of(p0 + lane) + (size_t)kPartRows * kPartD;
                const float m = __ldcg(ml + row);
                w = (m == -INFINITY) ? 0.f : ex2(m - M);
                wl = w * __ldcg(ml + kPartRows + row);
            }
            L += warp_sum(wl);
            const int n_grp = min(32, n_parts - p0);
            for (int q0 = 0; q0 < n_grp; q0 += 8) {
                float4 v[8];
                float wq[8];
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    wq[k] = __shfl_sync(0xffffffffu, w, (q0 + k) & 31);      // 0 past the last part
                    v[k] = q0 + k < n_grp ? __ldcg(reinterpret_cast<const float4*>(slot_of(p0 + q0 + k) + (size_t)row * kPartD) + lane)
                                          : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) {
                    acc.x = fmaf(wq[k], v[k].x, acc.x); acc.y = fmaf(wq[k], v[k].y, acc.y);
                    acc.z = fmaf(wq[k], v[k].z, acc.z); acc.w = fmaf(wq[k], v[k].w, acc.w);
                }
            }
        }
    }
    const float inv_l = 1.f / L;
    const int h = j.g * prm.G + j.hl;
    __nv_bfloat16* orow = prm.out + (((size_t)j.b * R + j.r) * Hq + h) * kD;
    uint2 pkt;
    pkt.x = pack_bf16(acc.x * inv_l, acc.y * inv_l);
    pkt.y = pack_bf16(acc.z * inv_l, acc.w * inv_l);
    reinterpret_cast<uint2*>(orow)[lane] = pkt;
    if (prm.lse && lane == 0) prm.lse[((size_t)j.b * R + j.r) * Hq + h] = (M + log2f(L)) * 0.6931471805599453f;
}

__device__ __forceinline__ void merge_row(const Params& prm, const PlanView& pv, int pair, int t, int lane_row, int lane)
{
    merge_run(prm, merge_job(prm, pv, pair, t, lane_row), lane);
}

}  // namespace tc
}  // namespace confu
