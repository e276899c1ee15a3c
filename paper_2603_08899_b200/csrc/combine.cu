// Merge of the split-KV partial results of the tensor-core attention kernel: a pair (sequence, kv
// head, row group) whose key tiles were walked by several CTAs has one unnormalised partial (O, m,
// l) per CTA; these kernels combine them into the output rows.
#include "combine.cuh"

namespace confu {
namespace tc {

// Merge of the split-KV partials of one (sequence, kv head) pair, in CTA order (deterministic).
// One block per (pair, M tile, 32 rows); a warp takes a row at a time (four rows in all), lane i the
// row's columns 4i..4i+3, so partial rows are read and output rows written as whole 512- and
// 256-byte lines.
__global__ void __launch_bounds__(256) combine_kernel(const Params prm)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the attention kernel has completed
    const PlanView pv = plan_view(const_cast<void*>(prm.plan), prm.d.B);
    const int pair = blockIdx.x, t = blockIdx.y;
    // pairs: sequence major, then kv head, then row group
    const int per_seq = prm.d.Hkv * prm.n_rg;
    const int b = pair / per_seq, g = (pair % per_seq) / prm.n_rg, rg = pair % prm.n_rg;
    const int nt = pv.tiles[b];
    if (t >= prm.n_mt) return;
    const int G = prm.G, R = prm.d.T + prm.d.C, Hq = prm.d.Hq;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (nt == 0) {                                      // malformed tree: no CTA worked on the pair; its rows read 0
        for (int lane_row = blockIdx.z * 32 + warp; lane_row < min(32 * G, (int)blockIdx.z * 32 + 32); lane_row += 8)
            zero_row(prm, b, g, kGroupRows * rg + 32 * t + lane_row / G, lane_row % G, lane);
        return;
    }
    const int64_t N = pv.hdr->n_tiles, n = pv.hdr->n_ctas / prm.n_rg;
    // key tile q of (sequence, kv head) sits at position F + q of the cost line; position x belongs to lane
    // floor(((x + 1) * n - 1) / N) of the n lanes, and row group rg of lane c is walked by CTA c * n_rg + rg
    const int64_t F = pv.tile_base[b] + (int64_t)g * (nt + kPairOverheadTiles) + kPairOverheadTiles;
    const int c_first = (int)(((F + 1) * n - 1) / N) * prm.n_rg + rg, c_last = (int)(((F + nt) * n - 1) / N) * prm.n_rg + rg;
    if (c_first == c_last) return;                      // one CTA covered the pair and wrote the output itself
    const size_t slot_floats = partial_slot_bytes() / sizeof(float);
    for (int lane_row = blockIdx.z * 32 + warp; lane_row < min(32 * G, (int)blockIdx.z * 32 + 32); lane_row += 8) {
        const int r = kGroupRows * rg + 32 * t + lane_row / G, hl = lane_row % G;
        if (r >= R) break;
        const int row = t * 128 + lane_row;
        float M = -INFINITY;
        for (int cta = c_first; cta <= c_last; cta += prm.n_rg) {
            const float* slot = prm.partials + (size_t)(2 * cta + (cta < c_last ? 1 : 0)) * slot_floats;
            M = fmaxf(M, slot[(size_t)kPartRows * kPartD + row]);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float L = 0.f;
        for (int cta = c_first; cta <= c_last; cta += prm.n_rg) {
            const float* slot = prm.partials + (size_t)(2 * cta + (cta < c_last ? 1 : 0)) * slot_floats;
            const float m = slot[(size_t)kPartRows * kPartD + row];
            const float w = (m == -INFINITY) ? 0.f : ex2(m - M);
            L += w * slot[(size_t)kPartRows * kPartD + kPartRows + row];
            const float4 v = reinterpret_cast<const float4*>(slot + (size_t)row * kPartD)[lane];
            acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
        }
        const float inv_l = 1.f / L;
        const int h = g * G + hl;
        __nv_bfloat16* orow = prm.out + (((size_t)b * R + r) * Hq + h) * kD;
        uint2 pkt;
        pkt.x = pack_bf16(acc.x * inv_l, acc.y * inv_l);
        pkt.y = pack_bf16(acc.z * inv_l, acc.w * inv_l);
        reinterpret_cast<uint2*>(orow)[lane] = pkt;
        if (prm.lse && lane == 0) prm.lse[((size_t)b * R + r) * Hq + h] = (M + log2f(L)) * 0.6931471805599453f;
    }
}

// The same merge for pairs spread over many CTAs (long prefixes in a small batch: more CTAs than
// pairs).  One block per (pair, M tile, 16 rows), one warp per row; the parts' maxima and weights are
// taken 32 parts at a time, one per lane, and the rows of eight parts are in flight together.  The
// order of every sum is fixed by the part index alone, so the result does not depend on the run.
constexpr int kCombineRowsPerBlock = 16;
__global__ void __launch_bounds__(32 * kCombineRowsPerBlock) combine_wide_kernel(const Params prm)
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next kernel may start its prologue
    asm volatile("griddepcontrol.wait;" ::: "memory");      // the attention kernel has completed
    const PlanView pv = plan_view(const_cast<void*>(prm.plan), prm.d.B);
    merge_row(prm, pv, blockIdx.x, blockIdx.y, blockIdx.z * kCombineRowsPerBlock + (threadIdx.x >> 5), threadIdx.x & 31);
}

cudaError_t launch_combine(const Params& prm, int sm_count, cudaStream_t st)
{
    // few pairs for the machine (each spread over several CTAs): the merge that is parallel over parts
    const int n_pairs = prm.d.B * prm.d.Hkv * prm.n_rg;
    // a programmatic dependent of the attention kernel: scheduled while that one drains, waits at its top
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.stream = st;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    if (sm_count >= 2 * n_pairs) {
        cfg.gridDim = dim3((unsigned)n_pairs, (unsigned)prm.n_mt, 128 / kCombineRowsPerBlock);
        cfg.blockDim = dim3(32 * kCombineRowsPerBlock);
        return cudaLaunchKernelEx(&cfg, combine_wide_kernel, prm);
    }
    cfg.gridDim = dim3((unsigned)n_pairs, (unsigned)prm.n_mt, 4);
    cfg.blockDim = dim3(256);
    return cudaLaunchKernelEx(&cfg, combine_kernel, prm);
}

}  // namespace tc
}  // namespace confu
