// Step-level planning kernel: tree validation, ancestor bitmasks, split-KV tile counts.
//
// Mask rule (tree attention over a token tree, with one contemplate token hung on a node's
// branch): a tree row sees itself and its ancestors; a contemplate row sees itself, its owner
// and the owner's ancestors.  Bit j < T of mask[b][r] says "row r sees the slot of tree row j";
// that a contemplate row sees its own slot (and no other contemplate row's) is implied.
#include "common.cuh"

namespace confu {

__global__ void __launch_bounds__(256) plan_kernel(confu_dims d, int units, int paired, const int64_t* __restrict__ seq_start,
                                                   const int32_t* __restrict__ prefix_len,
                                                   const int32_t* __restrict__ parent,
                                                   const int32_t* __restrict__ con_owner, void* plan_raw,
                                                   int32_t* status)
{
    const int B = d.B, T = d.T, C = d.C, R = d.T + d.C;
    PlanView pv = plan_view(plan_raw, B);
    __shared__ int s_bad[2];
    __shared__ uint64_t s_mask[2][kMaxTree];
    const int grp = threadIdx.x >> 7, r = threadIdx.x & 127;     // two sequences at a time, one thread per row

    for (int b0 = 0; b0 < B; b0 += 2) {
        const int b = b0 + grp;
        if (r == 0) s_bad[grp] = 0;
        __syncthreads();
        if (b < B) {
            const int32_t* par = parent + (size_t)b * T;
            int code = 0;
            if (r < T) {
                const int p = par[r];
                if (r == 0 ? (p != -1) : (p < 0 || p >= r)) code = CONFU_ST_BAD_PARENT;
            } else if (r < R) {
                const int o = con_owner[(size_t)b * C + (r - T)];
                if (o < 0 || o >= T) code = CONFU_ST_BAD_OWNER;
            }
            if (code) atomicMax(&s_bad[grp], code == CONFU_ST_BAD_PARENT ? 2 : 1);
        }
        __syncthreads();
        if (b < B && r < T) {
            // a tree row sees itself and its ancestors
            const int32_t* par = parent + (size_t)b * T;
            uint64_t m = 1ull << r;
            if (!s_bad[grp]) {
                int a = par[r];
                for (int it = 0; it < T && a >= 0; ++it) { m |= 1ull << a; a = par[a]; }
            }
            s_mask[grp][r] = m;
        }
        __syncthreads();
        if (b < B) {
            const int bad = s_bad[grp];
            uint64_t m = 0;
            if (r < T) m = s_mask[grp][r];
            else if (r < R && !bad) m = s_mask[grp][con_owner[(size_t)b * C + (r - T)]];   // owner and its ancestors (+ its own slot, implied)
            pv.mask[(size_t)b * kMaxRows + r] = m;
            if (r == 0) {
                const int code = bad == 2 ? CONFU_ST_BAD_PARENT : (bad == 1 ? CONFU_ST_BAD_OWNER : 0);
                pv.bad[b] = code;
                if (code && status) status[b] = code;
                const int64_t keys = (int64_t)prefix_len[b] + R;
                pv.tiles[b] = code ? 0 : (int32_t)((keys + kTileKeys - 1) / kTileKeys) + (d.S > 0 ? 1 : 0);
            }
        }
        __syncthreads();
    }
    __shared__ int s_count[kPlanMaxCtas + 1];
    if (threadIdx.x == 0) {
        int64_t acc = 0;
        for (int b = 0; b < B; ++b) {
            pv.tile_base[b] = acc;
            // one stretch of the line per (sequence, kv head); its groups of 64 query rows are walked side by side
            if (pv.tiles[b] > 0) acc += (int64_t)(pv.tiles[b] + kPairOverheadTiles) * d.Hkv;
        }
        pv.tile_base[B] = acc;
        PlanHeader h;
        h.B = B; h.Hkv = d.Hkv; h.T = T; h.C = C; h.S = d.S; h.R = R;
        h.n_tiles = acc;
        // The line is cut into `lanes` shares; CTA lane * n_rg + rg walks the lane's share for row group rg,
        // so the CTAs of a lane read the same K/V tiles at about the same time (the second read hits L2).
        const int n_rg0 = (R + kGroupRows - 1) / kGroupRows;
        int cap = units < kPlanMaxCtas ? units : kPlanMaxCtas;
        int lanes = cap / n_rg0;
        if ((int64_t)lanes > acc) lanes = (int)acc;
        h.n_ctas = lanes * n_rg0;
        h.paired = paired;
        *pv.hdr = h;
    }
    __syncthreads();
    // The runs of key tiles of every CTA of the tensor-core attention kernel, worked out once per step
    // instead of by every role of every CTA of every layer: thread c walks CTA c's share of the cost
    // line, first to count its runs, then (behind a prefix sum) to write them down.
    const int n_rg = (R + kGroupRows - 1) / kGroupRows;
    const int64_t N = pv.hdr->n_tiles;
    const int n_ctas = pv.hdr->n_ctas, n_lanes = n_ctas / n_rg;
    for (int pass = 0; pass < 2; ++pass) {
        const int c = threadIdx.x;
        if (c < n_ctas) {
            const int lane = c / n_rg, rg = c % n_rg;
            int64_t f = (int64_t)lane * N / n_lanes;
            const int64_t f1 = (int64_t)(lane + 1) * N / n_lanes;
            int n = 0;
            SegDesc* out = pv.segs + (pass ? s_count[c] : 0);
            int lo = 0;
            while (f < f1) {
                while (lo + 1 < B && pv.tile_base[lo + 1] <= f) ++lo;         // the sequence position f falls into
                const int nt = pv.tiles[lo];
                const int cost = nt + kPairOverheadTiles;
                const int64_t local = f - pv.tile_base[lo];
                const int pos = (int)(local % cost);
                const int64_t room = f1 - f;
                const int take = (int)((int64_t)(cost - pos) <= room ? cost - pos : room);
                f += take;
                const int t0 = pos > kPairOverheadTiles ? pos - kPairOverheadTiles : 0;
                const int t1 = pos + take > kPairOverheadTiles ? pos + take - kPairOverheadTiles : 0;
                if (t1 <= t0) continue;                    // the share ended inside this pair's overhead zone
                if (pass) {
                    SegDesc d;
                    d.b = lo;
                    d.g_rg = (int)(local / cost) | (rg << 16);       // the stretches of a sequence are in kv-head order
                    d.t0 = t0;
                    d.t1 = t1;
                    d.nt = nt;
                    d.P = prefix_len[lo];
                    d.part_slot = (t0 == 0 && t1 == nt) ? -1 : 2 * c + (t1 < nt ? 1 : 0);
                    d.pad0 = 0;
                    d.slot0 = seq_start ? seq_start[lo] : 0;
                    d.pad1 = 0;
                    out[n] = d;
                }
                ++n;
            }
            if (!pass) s_count[c] = n;
        }
        __syncthreads();
        if (!pass && threadIdx.x == 0) {
            int acc = 0;
            for (int c2 = 0; c2 < n_ctas; ++c2) { const int n = s_count[c2]; s_count[c2] = acc; acc += n; }
            s_count[n_ctas] = acc;
            for (int c2 = 0; c2 <= n_ctas; ++c2) pv.seg_begin[c2] = s_count[c2];
        }
        __syncthreads();
    }
}

cudaError_t launch_plan(const Ctx* ctx, const confu_dims& d, const int64_t* seq_start, const int32_t* prefix_len,
                        const int32_t* parent, const int32_t* con_owner, void* plan, int32_t* status, bool paired,
                        cudaStream_t st)
{
    // work units of the attention launch the plan is for: one CTA per SM, or one CTA pair per two SMs
    const int units = paired ? ctx->sm_count / 2 : ctx->sm_count;
    plan_kernel<<<1, 256, 0, st>>>(d, units, paired ? 1 : 0, seq_start, prefix_len, parent, con_owner, plan, status);
    return cudaGetLastError();
}

}  // namespace confu
