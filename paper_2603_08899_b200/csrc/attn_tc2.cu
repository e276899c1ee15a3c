// Tensor-core tree attention on CTA pairs: the two-SM form of tcgen05.mma (cta_group::2).
//
// Two CTAs of a cluster (two neighbouring SMs) work on one (sequence, kv head, row group) at a time.
// The 256 query rows that share the kv head (64 rows x 4 heads of the GQA group) are one M = 256
// operand: rows 0-127 (query rows 0-31 of the group) live in CTA 0, rows 128-255 in CTA 1.  Per
// 128-key tile
//     S = Q K^T      one M256 N128 K16 instruction per 16 head dims: each CTA supplies its 128 rows of
//                    Q and 64 of the 128 keys, and receives its 128 rows of S in its own tensor memory
//     P = exp2(S c - m)   one thread per row, bf16, into a tensor-memory buffer of its own
//     O += P V       A = P from tensor memory, B = V: each CTA supplies 64 of the 128 head dims
// so every K and V byte is fetched once per CTA pair, each SM reads half of the B operands from
// its shared memory, and each SM carries ONE chain S -> softmax -> P -> P V.  With one chain per SM
// tensor memory has room for two S buffers and two P buffers: Q K^T of tile g + 1 is issued before
// P V of tile g, so the softmax warps always find their next S waiting and the tensor pipe works
// on Q K^T while they compute exponentials.
//
// Roles per CTA (384 threads): warps 0-3 softmax of the even key tiles of the CTA's walk, warps 4-7
// of the odd ones (the same 128 rows, one thread of each set per row: the two sets run half a tile
// out of phase, so that one loads, masks and stores while the other keeps the exponential unit
// busy; the row's reference maximum is handed from tile to tile through shared memory); warp 8 TMA producer (its own half of every tile, plain loads); warp 9 tensor
// memory allocation and, in CTA 0, the one thread that issues every MMA of the pair; warp 10 the
// relay: it waits for this CTA's loads, zeroes the rows of a V tile that lie past the sequence's
// last slot, and tells CTA 0's issuing thread (remote mbarrier arrive) that this CTA's half of
// the stage is ready.  The issuing thread's commits arrive on the barriers of both CTAs.
//
// Every wait is bounded; a wait that runs out raises the abort flag of both CTAs, all roles leave,
// tensor memory is released and CONFU_ST_TIMEOUT is reported.  No load carries a multicast
// qualifier and every tensor map covers memory of this GPU only.
#include "tc_walk.cuh"

namespace confu {
namespace tc {
namespace pair {

constexpr int kThreads = 384;
constexpr int kStages = 4;                          // ring of stages; stage h = [K of key tile h | V of key tile h - kVLag]
constexpr int kVLag = 2;                            // Q K^T runs about two tiles ahead of P V: a stage's K and V are used at about the same time
constexpr int kQBufs = 1;                           // Q buffers (the next run's Q lands while this run's output rows are written)
constexpr int kKHalf = 64 * 128;                    // this CTA's 64 keys x one 64-wide half of the head dim
constexpr int kKBytes = 2 * kKHalf;                 // 16 KB
constexpr int kVBytes = kTileKeys * 128;            // 128 keys x this CTA's 64 head dims: 16 KB
constexpr int kStageBytes = kKBytes + kVBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256, kColP = 384;   // S0 S1 | O | P0 P1 (P: 64 columns of bf16 pairs)
constexpr float kRescaleThreshold = 8.f;

struct SharedStorage {
    alignas(1024) uint8_t q[kQBufs][kTileBytes];    // this CTA's 128 query rows, two 64-wide halves
    alignas(1024) uint8_t kv[kStages][kStageBytes];
    alignas(16) float4 xpose[8][32 * 8];            // per softmax warp: 32 x 32 fp32 transpose tile of the epilogue
    alignas(8) uint2 xref[2][128];                  // [set][row]: {tile tag, the row's reference maximum as of that tile}
    float xsum[2][128], xm[2][128];                 // [set][row]: the two threads of a row swap sums and references at the end of a run
    alignas(8) uint64_t q_full[kQBufs], q_ready[kQBufs], q_empty[kQBufs];
    uint64_t kv_full[kStages], kv_ready[kStages], kv_empty[kStages];
    uint64_t s_full[2], s_free[2], p_full[2], o_done;
    uint64_t x_bar[4];                              // per pair of softmax warps (same rows): both have written xsum
    uint32_t tmem_base;
    int abort;
};

// ------------------------------------------------------------------------------------ cluster PTX
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// address of the same shared-memory object in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(const void* p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
// Arrival on a barrier of a CTA of the pair (an address from map_to_cta).  What the arrival orders is
// tensor-memory traffic (tcgen05.wait / fence before it) and completed TMA copies, not generic-proxy
// data: the default scope is enough, and a cluster-scope release costs ~1000 cycles here.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void store_remote_u32(uint32_t cluster_addr, uint32_t v)
{
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ void cluster_sync_all()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ bool mbar_try_wait_pair(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  On expiry the abort flags of both CTAs are raised.
__device__ __forceinline__ bool wait_c(SharedStorage& sh, uint64_t* bar, uint32_t parity, unsigned long long limit_ns)
{
    if (mbar_try_wait_pair(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
    volatile int* abort = &sh.abort;
    for (uint32_t it = 1;; ++it) {
        if (mbar_try_wait_pair(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort) return false;
            if (global_ns() - t0 > limit_ns) {
                *abort = 1;
                store_remote_u32(map_to_cta(&sh.abort, cluster_ctarank() ^ 1u), 1u);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void raise_abort(SharedStorage& sh)
{
    *(volatile int*)&sh.abort = 1;
    store_remote_u32(map_to_cta(&sh.abort, cluster_ctarank() ^ 1u), 1u);
}
constexpr uint32_t kSpinLimit = 1u << 22;           // polls of a shared-memory flag before a role gives up (~0.1 s)

// The same for a whole warp: every lane leaves with the same answer, so that the warp-wide
// instructions behind the wait (tcgen05.ld / st, __syncwarp) are never reached by a part of the warp.
__device__ __forceinline__ bool wait_warp(SharedStorage& sh, uint64_t* bar, uint32_t parity, unsigned long long limit_ns)
{
    return __all_sync(0xffffffffu, wait_c(sh, bar, parity, limit_ns));
}

// commit of everything the issuing thread has issued so far, arriving on the barrier at this offset in both CTAs
__device__ __forceinline__ void commit_both(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"((uint16_t)3)
                 : "memory");
}
// D[tmem] (+)= A[smem] * B[smem], M = 256 over the CTA pair
__device__ __forceinline__ void mma2_ss(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "mov.b64 da, {%1, %5};\n\tmov.b64 db, {%2, %5};\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], da, db, %3, {%6, %6, %6, %6, %6, %6, %6, %6}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(acc), "r"(kDescHi), "r"(0u)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma2_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t idesc, uint32_t acc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "mov.b64 db, {%2, %5};\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], db, %3, {%6, %6, %6, %6, %6, %6, %6, %6}, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(idesc), "r"(acc), "r"(kDescHi), "r"(0u)
        : "memory");
}
// bf16 x bf16 -> fp32, M = 256 (both CTAs), N = 128; B K-major (Q K^T) or MN-major (P V)
constexpr uint32_t kIdescQK2 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
constexpr uint32_t kIdescPV2 = kIdescQK2 | (1u << 16);

// ------------------------------------------------------------------------------------ roles
struct TileRef {
    int g, z;                          // kv head, first slot (row) of the tile
    bool soft;
    bool present;                      // false: no tile (before the first, behind the last)
};

// This CTA's half of every stage: 64 of the tile's keys (K, both 64-wide halves of the head dim) and 64
// of the head dims of all 128 keys of the tile before (V); at the start of a run its 128 rows of Q.
__device__ void producer_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t rank,
                              const CUtensorMap* q_map, const CUtensorMap* k_map, const CUtensorMap* v_map,
                              const CUtensorMap* ks_map, const CUtensorMap* vs_map)
{
    Walker w(pv, prm, blockIdx.x >> 1);
    const int n_total = (int)(w.end - w.cur);
    Segment s;
    uint32_t g = 0, seg = 0;
    const int R = prm.d.T + prm.d.C;
    const uint32_t q_box_bytes = 32u * prm.G * 128u;
    TileRef hist[kVLag];               // the tiles of the last kVLag stages, oldest first: hist[0]'s V travels with this stage's K
#pragma unroll
    for (int i = 0; i < kVLag; ++i) hist[i].present = false;
    auto fill = [&](const TileRef* cur) -> bool {
        const uint32_t st = g % kStages;
        const bool have_v = hist[0].present;
        if (!wait_c(sh, &sh.kv_empty[st], ((g / kStages) & 1) ^ 1, prm.wait_ns)) return false;
        mbar_arrive_expect_tx(&sh.kv_full[st], (cur ? kKBytes : 0) + (have_v ? kVBytes : 0));
        if (cur) {
            const CUtensorMap* m = cur->soft ? ks_map : k_map;
            tma_load_3d(sh.kv[st], m, &sh.kv_full[st], 0, cur->g, cur->z + 64 * (int)rank);
            tma_load_3d(sh.kv[st] + kKHalf, m, &sh.kv_full[st], 64, cur->g, cur->z + 64 * (int)rank);
        }
        if (have_v) {
            const CUtensorMap* m = hist[0].soft ? vs_map : v_map;
            tma_load_3d(sh.kv[st] + kKBytes, m, &sh.kv_full[st], 64 * (int)rank, hist[0].g, hist[0].z);
        }
#pragma unroll
        for (int i = 0; i + 1 < kVLag; ++i) hist[i] = hist[i + 1];
        if (cur) hist[kVLag - 1] = *cur;
        else hist[kVLag - 1].present = false;
        ++g;
        return true;
    };
    while (w.next(s)) {
        for (int t = s.t0; t < s.t1; ++t) {
            TileRef cur;
            cur.present = true;
            cur.g = s.g;
            cur.soft = t >= s.nkt;
            cur.z = cur.soft ? 0
                  : prm.map.block_table ? prm.map.block_table[(size_t)s.b * prm.map.max_pages + t] * kTileKeys
                                        : (int)(s.slot0 + (int64_t)t * kTileKeys);
            if (!fill(&cur)) return;
            if (t == s.t0) {
                const uint32_t qb = seg % kQBufs;
                if (!wait_c(sh, &sh.q_empty[qb], ((seg / kQBufs) & 1) ^ 1, prm.wait_ns)) return;
                mbar_arrive_expect_tx(&sh.q_full[qb], 2u * q_box_bytes);
                for (int kb = 0; kb < 2; ++kb)
                    tma_load_3d(sh.q[qb] + kb * kHalfTile, q_map, &sh.q_full[qb], kb * 64, s.g * prm.G,
                                s.b * R + kGroupRows * s.rg + 32 * (int)rank);
            }
        }
        ++seg;
    }
    // kVLag more stages: they carry the V tiles of the last key tiles (a stage may be empty when the
    // whole walk is shorter than kVLag tiles)
    for (int i = 0; i < (n_total > 0 ? kVLag : 0); ++i)
        if (!fill(nullptr)) return;
}

// Waits for this CTA's loads of every stage (and of every run's Q), zeroes the rows of a sequence's
// last V tile that lie past its last slot, and reports to the issuing thread in CTA 0.
__device__ void relay_role(SharedStorage& sh, const Params& prm, const PlanView& pv)
{
    Walker w(pv, prm, blockIdx.x >> 1);
    Segment s;
    const int R = prm.d.T + prm.d.C, lane = threadIdx.x & 31;
    uint32_t g = 0, seg = 0;
    int valid[kVLag];                  // ragged-row counts of the tiles of the last kVLag stages, oldest first (0: whole tile or no tile)
#pragma unroll
    for (int i = 0; i < kVLag; ++i) valid[i] = 0;
    bool any = false;
    auto run_stage = [&](bool have_cur, int cur_valid) -> bool {
        const uint32_t st = g % kStages;
        if (!wait_warp(sh, &sh.kv_full[st], (g / kStages) & 1, prm.wait_ns)) return false;
        if (valid[0] > 0) {
            const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
            for (int off = valid[0] * 128 + lane * 16; off < kVBytes; off += 32 * 16)
                *reinterpret_cast<uint4*>(sh.kv[st] + kKBytes + off) = zero;
            // generic-proxy stores that the other CTA's issuing threads hand to the tensor pipe: visible to the
            // async proxy, and (this rare case only) ordered at cluster scope before the arrival
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            asm volatile("fence.acq_rel.cluster;" ::: "memory");
        }
        __syncwarp();
        if (lane == 0) mbar_arrive_remote(map_to_cta(&sh.kv_ready[st], 0));
#pragma unroll
        for (int i = 0; i + 1 < kVLag; ++i) valid[i] = valid[i + 1];
        valid[kVLag - 1] = have_cur ? cur_valid : 0;
        any = any || have_cur;
        ++g;
        return true;
    };
    while (w.next(s)) {
        for (int tile = s.t0; tile < s.t1; ++tile) {
            if (!run_stage(true, ragged_rows(s, tile, R))) return;
            if (tile == s.t0) {
                const uint32_t qb = seg % kQBufs;
                if (!wait_warp(sh, &sh.q_full[qb], (seg / kQBufs) & 1, prm.wait_ns)) return;
                __syncwarp();
                if (lane == 0) mbar_arrive_remote(map_to_cta(&sh.q_ready[qb], 0));
            }
        }
        ++seg;
    }
    for (int i = 0; i < (any ? kVLag : 0); ++i)
        if (!run_stage(false, 0)) return;
}

// Two threads of CTA 0 issue the tensor-core work of the pair, each waiting only for what its own
// instructions need (the pipe takes instructions from both without loss), so that neither product
// waits behind a wake-up that belongs to the other:
//   qk_role   S[g & 1] = Q K^T of key tile g as soon as K has landed in both CTAs and the softmax
//             warps of both have read the S buffer's previous contents (tile g - 2) into registers;
//   pv_role   O += P V of key tile g as soon as V has landed and both CTAs have handed P over.
// A stage [K of tile h | V of tile h - kVLag] is free again when both threads' instructions on it have completed.
__device__ void qk_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t tmem)
{
    Walker w(pv, prm, blockIdx.x >> 1);
    Segment s;
    uint32_t g = 0, seg = 0;
    uint32_t q_lo[kQBufs];
    for (int i = 0; i < kQBufs; ++i) q_lo[i] = desc_lo(smem_u32(sh.q[i]), 16);
    const uint32_t k_lo0 = desc_lo(smem_u32(sh.kv[0]), 16);
    constexpr uint32_t kStageStep = kStageBytes >> 4;
    while (w.next(s)) {
        const int n_tiles = s.t1 - s.t0;
        for (int j = 0; j < n_tiles; ++j, ++g) {
            const uint32_t st = g % kStages;
            if (!wait_c(sh, &sh.kv_ready[st], (g / kStages) & 1, prm.wait_ns)) return;
            if (j == 0 && !wait_c(sh, &sh.q_ready[seg % kQBufs], (seg / kQBufs) & 1, prm.wait_ns)) return;
            if (!wait_c(sh, &sh.s_free[g & 1], ((g >> 1) & 1) ^ 1, prm.wait_ns)) return;
            tc_fence_after();
            // 8 steps of 16 head dims; step i sits in 64-wide half i / 4 at byte 32 (i % 4) of the swizzled row
            const uint32_t kl = k_lo0 + st * kStageStep, ql = q_lo[seg % kQBufs];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t q_off = ((uint32_t)(i >> 2) * kHalfTile + (uint32_t)(i & 3) * 32u) >> 4;
                const uint32_t k_off = ((uint32_t)(i >> 2) * kKHalf + (uint32_t)(i & 3) * 32u) >> 4;
                mma2_ss(tmem + kColS + (g & 1) * 128, ql + q_off, kl + k_off, kIdescQK2, i > 0 ? 1u : 0u);
            }
            commit_both(&sh.s_full[g & 1]);
            commit_both(&sh.kv_empty[st]);
            if (j + 1 == n_tiles) commit_both(&sh.q_empty[seg % kQBufs]);     // every Q K^T of this run has been issued
        }
        ++seg;
    }
    // the last kVLag stages carry no K tile: this thread has nothing to issue on them, but their release
    // counts its arrival too (the softmax threads wait for it before they rescale O)
    for (int i = 0; i < (g > 0 ? kVLag : 0); ++i, ++g) {
        if (!wait_c(sh, &sh.kv_ready[g % kStages], (g / kStages) & 1, prm.wait_ns)) return;
        commit_both(&sh.kv_empty[g % kStages]);
    }
}

__device__ void pv_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t tmem)
{
    Walker w(pv, prm, blockIdx.x >> 1);
    Segment s;
    uint32_t g = 0;
    const uint32_t v_lo0 = desc_lo(smem_u32(sh.kv[0] + kKBytes), 16);
    constexpr uint32_t kStageStep = kStageBytes >> 4;
    // the first kVLag stages carry no V tile: this thread has nothing to wait for on them
    for (int i = 0; i < kVLag; ++i) commit_both(&sh.kv_empty[i]);
    while (w.next(s)) {
        const int n_tiles = s.t1 - s.t0;
        for (int j = 0; j < n_tiles; ++j, ++g) {
            const uint32_t st = (g + kVLag) % kStages, pb = g & 1;      // V of tile g travels with K of tile g + kVLag
            if (!wait_c(sh, &sh.kv_ready[st], ((g + kVLag) / kStages) & 1, prm.wait_ns)) return;
            if (!wait_c(sh, &sh.p_full[pb], (g >> 1) & 1, prm.wait_ns)) return;
            tc_fence_after();
            // 8 steps of 16 keys (2048 B of the V tile and 8 tensor-memory columns of bf16 pairs each)
            const uint32_t vl = v_lo0 + st * kStageStep;
#pragma unroll
            for (int i = 0; i < 8; ++i)
                mma2_ts(tmem + kColO, tmem + kColP + pb * 64 + i * 8, vl + i * (2048u >> 4), kIdescPV2,
                        (j == 0 && i == 0) ? 0u : 1u);
            commit_both(&sh.kv_empty[st]);
            if (j + 1 == n_tiles) commit_both(&sh.o_done);
        }
    }
}

__device__ void softmax_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t tmem, uint32_t rank)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // set 0 (warps 0-3) takes the even key tiles of the CTA's walk, set 1 (warps 4-7) the odd ones; at
    // the end of a run set 0 writes head dims 0-63 of the output rows, set 1 head dims 64-127
    const int set = warp >> 2, wq = warp & 3;
    const int half = set;
    const int lane_row = wq * 32 + lane;                     // row of this CTA's 128 = tensor-memory lane
    const uint32_t lane_base = (uint32_t)(wq * 32) << 16;
    const int G = prm.G, T = prm.d.T, R = prm.d.T + prm.d.C, S = prm.d.S, Hq = prm.d.Hq;
    const int hl = lane_row % G;
    const float c = prm.c;
    const uint32_t buf = (uint32_t)set;                      // S and P buffer of this set's tiles
    const uint32_t p_full_leader = map_to_cta(&sh.p_full[buf], 0), s_free_leader = map_to_cta(&sh.s_free[buf], 0);
    const uint32_t s_addr = tmem + lane_base + kColS + buf * 128, p_addr = tmem + lane_base + kColP + buf * 64;
    const uint32_t ref_mine = smem_u32(&sh.xref[set][lane_row]), ref_theirs = smem_u32(&sh.xref[set ^ 1][lane_row]);

    Walker w(pv, prm, blockIdx.x >> 1);
    Segment s;
    uint32_t g = 0, seg = 0;
    while (w.next(s)) {
        const int r = kGroupRows * s.rg + 32 * (int)rank + lane_row / G;      // query row of this thread in this run
        const bool row_valid = lane_row < 32 * G && r < R;
        const uint64_t mask = row_valid ? pv.mask[(size_t)s.b * kMaxRows + r] : 0ull;
        // this thread's share of the row's sum of weights, relative to the reference maximum m_mine
        // (the row's reference as of the last tile this thread worked on)
        float m_mine = -INFINITY, l = 0.f;
        for (int tile = s.t0; tile < s.t1; ++tile, ++g) {
            if ((g & 1u) != (uint32_t)set) continue;
            if (!wait_warp(sh, &sh.s_full[buf], (g >> 1) & 1, prm.wait_ns)) return;
            tc_fence_after();
            uint32_t sv[128];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(s_addr + q4 * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[q4 * 32]));
            tc_wait_ld();
            // the scores sit in registers: the S buffer may take the tile after next
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(s_free_leader);
            const bool masked = tile >= s.nkt || (int64_t)(tile + 1) * kTileKeys > s.P;
            if (masked) {
                uint64_t lo, hi;
                visible_bits(s, tile, R, T, S, r, row_valid, mask, lo, hi);
#pragma unroll
                for (int j = 0; j < 64; ++j) {
                    if (!((lo >> j) & 1ull)) sv[j] = 0xff800000u;            // -inf
                    if (!((hi >> j) & 1ull)) sv[64 + j] = 0xff800000u;
                }
            }
            const float m_tile = max128(sv) * c;
            // The row's reference maximum is handed from tile to tile: the thread of the other set that
            // worked on tile g - 1 published it (tagged with its tile; bounded spin), this one publishes
            // the reference of tile g as soon as it is decided -- before any exponential.
            float m_ref = m_tile, m_prev = -INFINITY;
            bool move = false;
            if (tile != s.t0) {
                bool got = false;
                for (uint32_t it = 0; it < kSpinLimit; ++it) {
                    uint32_t tag, bits;
                    asm volatile("ld.volatile.shared.v2.u32 {%0, %1}, [%2];" : "=r"(tag), "=r"(bits) : "r"(ref_theirs) : "memory");
                    if (tag == g) { m_prev = __uint_as_float(bits); got = true; break; }
                    if ((it & 1023u) == 1023u && *(volatile int*)&sh.abort) break;
                }
                if (!__all_sync(0xffffffffu, got)) { raise_abort(sh); return; }
                move = m_tile - m_prev > kRescaleThreshold;                  // false when both are -inf (NaN)
                m_ref = move ? m_tile : m_prev;
            }
            asm volatile("st.volatile.shared.v2.u32 [%0], {%1, %2};" ::"r"(ref_mine), "r"(g + 1), "r"(__float_as_uint(m_ref)) : "memory");
            if (__any_sync(0xffffffffu, move)) {
                // O is being accumulated into by P V of the tile before, whose V travelled in stage g - 1 + kVLag:
                // that stage's release says it is done
                if (!wait_warp(sh, &sh.kv_empty[(g - 1 + kVLag) % kStages], ((g - 1 + kVLag) / kStages) & 1, prm.wait_ns)) return;
                tc_fence_after();
                const float alpha = move ? ex2(m_prev - m_ref) : 1.f;       // O so far is relative to m_prev
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t ov[32];
                    const uint32_t o_addr = tmem + lane_base + kColO + q4 * 32;
                    tmem_ld32(o_addr, ov);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
                    tmem_st32(o_addr, ov);
                }
            }
            // bring this thread's sum to the row's current reference
            if (m_ref != m_mine) {
                l = (m_mine == -INFINITY) ? 0.f : l * ex2(m_mine - m_ref);
                m_mine = m_ref;
            }
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            // the P buffer was last read by P V of tile g - 2, whose V travelled in stage g - 2 + kVLag
            if (g >= 2 && !wait_warp(sh, &sh.kv_empty[(g - 2 + kVLag) % kStages], ((g - 2 + kVLag) / kStages) & 1, prm.wait_ns)) return;
#pragma unroll
            for (int hh = 0; hh < 2; ++hh) {
                uint32_t pk[32];
                l += weights64(&sv[64 * hh], c, neg_m, pk);
                tmem_st32(p_addr + 32 * hh, pk);
            }
            tc_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_remote(p_full_leader);
        }
        // ---- end of the run: this thread's 64 head dims of the row of O ----
        if (!wait_warp(sh, &sh.o_done, seg & 1, prm.wait_ns)) return;
        tc_fence_after();
        // the row's sum of weights: the shares of the two threads of the row, each brought to the larger
        // (= the final) reference maximum (bounded wait, like every other)
        sh.xsum[set][lane_row] = l;
        sh.xm[set][lane_row] = m_mine;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.x_bar[wq]);
        if (!wait_warp(sh, &sh.x_bar[wq], seg & 1, prm.wait_ns)) return;
        const float m_oth = sh.xm[set ^ 1][lane_row], l_oth = sh.xsum[set ^ 1][lane_row];
        const float m_ref = fmaxf(m_mine, m_oth);
        const float l_row = (m_mine == -INFINITY ? 0.f : l * ex2(m_mine - m_ref)) + (m_oth == -INFINITY ? 0.f : l_oth * ex2(m_oth - m_ref));
        const int h = s.g * G + hl;
        float4* xp = sh.xpose[warp];
        const bool whole = s.part_slot < 0;
        const float inv_l = whole ? 1.f / l_row : 1.f;
        // Each 32-column chunk goes through the warp's transpose tile and leaves as whole rows in 16-byte
        // pieces: eight rows per instruction for the bf16 output, four for an fp32 partial.
        __nv_bfloat16* o_ptr[4];
        float* p_ptr = nullptr;
        if (whole) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const int lr = wq * 32 + 8 * kk + (lane >> 2);
                const int rk = kGroupRows * s.rg + 32 * (int)rank + lr / G;
                o_ptr[kk] = (lr < 32 * G && rk < R)
                                ? prm.out + (((size_t)s.b * R + rk) * Hq + s.g * G + lr % G) * kD + 8 * (lane & 3)
                                : nullptr;
            }
        } else {
            p_ptr = prm.partials + (size_t)s.part_slot * (partial_slot_bytes() / sizeof(float)) +
                    (size_t)(rank * 128 + wq * 32 + (lane >> 3)) * kPartD + 4 * (lane & 7);
        }
#pragma unroll 1
        for (int q4 = 2 * half; q4 < 2 * half + 2; ++q4) {
            uint32_t ov[32];
            tmem_ld32(tmem + lane_base + kColO + q4 * 32, ov);
            tc_wait_ld();
#pragma unroll
            for (int q = 0; q < 8; ++q)
                xp[lane * 8 + (q ^ (lane & 7))] =
                    make_float4(__uint_as_float(ov[4 * q]) * inv_l, __uint_as_float(ov[4 * q + 1]) * inv_l,
                                __uint_as_float(ov[4 * q + 2]) * inv_l, __uint_as_float(ov[4 * q + 3]) * inv_l);
            __syncwarp();
            if (whole) {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk) {
                    const int k = 8 * kk + (lane >> 2), q = 2 * (lane & 3);
                    const float4 a = xp[k * 8 + (q ^ (k & 7))], b2 = xp[k * 8 + ((q + 1) ^ (k & 7))];
                    if (o_ptr[kk])
                        *reinterpret_cast<uint4*>(o_ptr[kk] + q4 * 32) =
                            make_uint4(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w), pack_bf16(b2.x, b2.y), pack_bf16(b2.z, b2.w));
                }
            } else {
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const int k = 4 * kk + (lane >> 3);
                    *reinterpret_cast<float4*>(p_ptr + (size_t)(4 * kk) * kPartD + q4 * 32) = xp[k * 8 + ((lane & 7) ^ (k & 7))];
                }
            }
            __syncwarp();
        }
        if (half == 0) {
            if (whole) {
                if (row_valid && prm.lse)
                    prm.lse[((size_t)s.b * R + r) * Hq + h] = (m_ref + log2f(l_row)) * 0.6931471805599453f;
            } else {
                float* ml = prm.partials + (size_t)s.part_slot * (partial_slot_bytes() / sizeof(float)) + (size_t)kPartRows * kPartD;
                ml[rank * 128 + lane_row] = m_ref;
                ml[kPartRows + rank * 128 + lane_row] = l_row;
            }
        }
        // the P of the next run's first tile is only handed over after this point, which is what keeps
        // the tensor pipe from overwriting O before it has been read
        tc_fence_before();
        ++seg;
    }
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
attention_pair_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                      const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap ks_map,
                      const __grid_constant__ CUtensorMap vs_map, const Params prm)
{
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& sh = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5;
    const uint32_t rank = cluster_ctarank();

    if (threadIdx.x == 0) {
        for (int i = 0; i < kQBufs; ++i) {
            mbar_init(&sh.q_full[i], 1);
            mbar_init(&sh.q_ready[i], 2);
            mbar_init(&sh.q_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&sh.s_full[i], 1);
            mbar_init(&sh.s_free[i], 8);                    // one arrival per softmax warp of a set, both CTAs
            mbar_init(&sh.p_full[i], 8);
        }
        for (int i = 0; i < kStages; ++i) {
            mbar_init(&sh.kv_full[i], 1);
            mbar_init(&sh.kv_ready[i], 2);                  // the relay warps of both CTAs
            mbar_init(&sh.kv_empty[i], 2);                  // the commits of both issuing threads
        }
        mbar_init(&sh.o_done, 1);
        for (int i = 0; i < 4; ++i) mbar_init(&sh.x_bar[i], 2);
        sh.abort = 0;
        for (int i = 0; i < 2 * 128; ++i) (&sh.xref[0][0])[i] = make_uint2(0u, 0u);            // tag 0: no tile
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 9) {
        // tensor memory of both CTAs: the same warp of each issues the paired allocation
        asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // the other CTA's barriers exist before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // Everything above touches only this kernel's own shared and tensor memory, so it runs while the
    // kernel before this one in the stream drains.  From here on global memory is read and written:
    // every CTA waits until the kernels before this one have completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const PlanView pv = plan_view(const_cast<void*>(prm.plan), prm.d.B);
    // (both CTAs of a pair take the same way through the next two tests)
    const bool listed = (int)(blockIdx.x >> 1) < pv.hdr->n_ctas;
    const bool pair_plan = pv.hdr->paired == 1;             // the plan lists runs per CTA pair, not per CTA
    if (!pair_plan && blockIdx.x == 0 && prm.status)
        for (int b = threadIdx.x; b < prm.d.B; b += kThreads) prm.status[b] = CONFU_ST_BAD_PLAN;

    if (!listed || !pair_plan) {
        // nothing to do: straight to the teardown, which releases tensor memory
    } else if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        softmax_role(sh, prm, pv, tmem, rank);
    } else if (warp == 8) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if ((threadIdx.x & 31) == 0) producer_role(sh, prm, pv, rank, &q_map, &k_map, &v_map, &ks_map, &vs_map);
    } else if (warp == 9) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if ((threadIdx.x & 31) == 0 && rank == 0) qk_role(sh, prm, pv, tmem);
    } else if (warp == 10) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        relay_role(sh, prm, pv);
    } else if (warp == 11) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if ((threadIdx.x & 31) == 0 && rank == 0) pv_role(sh, prm, pv, tmem);
    }
    __syncwarp();
    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                                     // neither CTA leaves while the other may still reach into it
    if (sh.abort) {
        // give this CTA's copies that may still be in flight time to land before its shared memory goes away
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0 && rank == 0 && prm.status)
            for (int b = 0; b < prm.d.B; ++b) prm.status[b] = CONFU_ST_TIMEOUT;
        __syncthreads();
    }
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace pair

bool make_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t heads, uint32_t box_rows, uint32_t box_heads);

}  // namespace tc

bool pair_attention_supported(const confu_dims& d, int sm_count)
{
    const int G = d.Hq / d.Hkv;
    return d.kv_dtype == CONFU_BF16 && d.D == 128 && G <= 4 && d.S <= 128 && d.T + d.C > 32 && sm_count >= 4;
}

cudaError_t launch_attention_pair(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                  const void* v_cache, int64_t n_slots, const SlotMap& map,
                                  const int32_t* prefix_len, const void* k_soft, const void* v_soft, const void* plan,
                                  void* partials, void* out, float* lse, int32_t* status, cudaStream_t st)
{
    using namespace tc;
    using namespace tc::pair;
    const int R = d.T + d.C, G = d.Hq / d.Hkv;
    CUtensorMap q_map, k_map, v_map, ks_map, vs_map;
    // K: 64 keys x 64 head dims per box (this CTA's keys, one half of the head dim); V: 128 keys x 64 head dims
    bool ok = make_tile_map(&q_map, q, (uint64_t)d.B * R, d.Hq, 32, G) && make_tile_map(&k_map, k_cache, n_slots, d.Hkv, 64, 1) &&
              make_tile_map(&v_map, v_cache, n_slots, d.Hkv, kTileKeys, 1);
    if (d.S > 0) ok = ok && make_tile_map(&ks_map, k_soft, d.S, d.Hkv, 64, 1) && make_tile_map(&vs_map, v_soft, d.S, d.Hkv, kTileKeys, 1);
    else { ks_map = k_map; vs_map = v_map; }
    if (!ok) return cudaErrorInvalidValue;
    Params prm;
    prm.d = d;
    prm.map = map;
    prm.prefix_len = prefix_len;
    prm.plan = plan;
    prm.partials = (float*)partials;
    prm.out = (__nv_bfloat16*)out;
    prm.lse = lse;
    prm.status = status;
    prm.n_mt = 2;
    prm.n_rg = (R + kGroupRows - 1) / kGroupRows;
    prm.G = G;
    prm.c = (d.sm_scale != 0.f ? d.sm_scale : 1.f / sqrtf((float)d.D)) * 1.4426950408889634f;
    prm.wait_ns = ctx->wait_ns;
    prm.k_scale = prm.v_scale = nullptr;
    const size_t smem = sizeof(SharedStorage) + 1024;
    static OncePerDevice attr_done;
    {
        cudaError_t e = attr_done.run([&] {
            return cudaFuncSetAttribute(attention_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        });
        if (e != cudaSuccess) return e;
    }
    const int n_pairs = ctx->sm_count / 2;
    cudaLaunchAttribute attrs[1];
    attrs[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attrs[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(2 * n_pairs));
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = attrs;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attention_pair_kernel, q_map, k_map, v_map, ks_map, vs_map, prm);
    if (e != cudaSuccess) return e;
    return launch_combine(prm, n_pairs, st);
}

}  // namespace confu
