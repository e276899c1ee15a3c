// Tensor-core tree attention for sm_100a: TMA-staged bf16 K/V tiles, tcgen05.mma with TMEM
// accumulators, warp-specialised online softmax, stream-K split over the ragged batch.
//
// One persistent CTA per SM walks a contiguous range of the flat list of 128-key tiles of all
// (sequence, kv head) pairs.  For a pair the query block is the R rows x G heads that share the kv
// head: two M tiles of 128 rows (32 rows x G heads each, padded when G < 4).  Per key tile:
//     S_t = Q_t K^T           tcgen05.mma, A and B from shared memory (K-major, 128B swizzle)
//     P_t = exp2(S_t*c - m)   one thread per row: tcgen05.ld, mask (last tiles only), tcgen05.st as bf16
//                             over the S columns
//     O_t += P_t V            tcgen05.mma, A from TMEM, B = V tile in shared memory (MN-major)
// Each M tile has its own softmax warpgroup; the two run out of phase, so that while one computes
// exponentials the tensor pipe serves the other (P V, then the next Q K^T).  The tensor pipe holds
// about one instruction ahead of the issuing thread, so whatever that thread does between MMAs is
// idle pipe time: K/V travel in stages of [V of key tile g-1 | K of key tile g] with one full and
// one empty barrier each, which leaves the issuing thread three waits and three commits per key
// tile.  Prefix tiles need no mask; the ancestor bitmask (one 64-bit word per row, in a register) is applied only to
// the tiles that hold the tree slots, the ragged tail and the soft-prompt entries.  A range that
// does not cover a whole pair writes an unnormalised partial (O, m, l) that combine_kernel merges
// in a fixed order.
//
// The last key tile of a sequence reaches past its last slot, into slots that belong to another
// sequence, to an unused page tail or to memory nobody ever wrote.  Their scores are masked, so
// their weights are exactly 0, but 0 x NaN would still poison P V: a spare warp zeroes those rows
// of the V tile in shared memory before the tensor pipe reads them.  What such slots hold is
// therefore irrelevant.
//
// Every wait on an mbarrier is bounded (wall-clock limit); on expiry the CTA raises an abort flag,
// every role leaves its loop, tensor memory is released and CONFU_ST_TIMEOUT is reported.
#include "tc_walk.cuh"

namespace confu {

namespace tc {

constexpr int kThreads = 384;            // warps 0-3: softmax of M tile 0, 4-7: of M tile 1, 8: TMA, 9: MMA, 10: ragged tail of V
constexpr int kStages = 2;               // ring of stages; stage g = [V of the CTA's g-1st key tile | K of its g-th]
constexpr int kQBytes = 2 * kTileBytes;             // two M tiles
constexpr uint32_t kTmemCols = 512;                 // S0 | S1 | O0 | O1, 128 columns each; P_t overlays S_t
constexpr float kRescaleThreshold = 8.f;            // lazy rescale: move the reference max only past 2^8

struct SharedStorage {
    alignas(1024) uint8_t q[kQBytes];
    alignas(1024) uint8_t kv[kStages][2][kTileBytes];    // [stage][0: V tile, 1: K tile]
    alignas(8) uint64_t q_full, q_empty;
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t s_full[2], p_full[2], o_done[2];
    uint64_t v_fixed;                     // the rows of a V tile past the sequence's last slot have been zeroed
    uint32_t tmem_base;
    int abort;
    // per softmax warp: a 32 x 32 fp32 tile for turning "one thread per row" into whole-line stores;
    // the four floats (row, 4q .. 4q+3) sit at float4 index row * 8 + (q ^ (row & 7))
    alignas(16) float4 xpose[8][32 * 8];
};

// ------------------------------------------------------------------------------------ roles
// Key tiles of the CTA's share, all pairs together, are numbered g = 0..n-1 in walking order; stage
// g of the ring carries V of tile g-1 and K of tile g (stage 0 has no V, stage n no K).
struct TileRef {                       // where a key tile's K and V come from
    int g, z;                          // kv head, first slot (row) of the tile
    bool soft;                         // the soft-prompt tile
};

__device__ void producer_role(SharedStorage& sh, const Params& prm, const PlanView& pv, const CUtensorMap* q_map,
                              const CUtensorMap* k_map, const CUtensorMap* v_map, const CUtensorMap* ks_map,
                              const CUtensorMap* vs_map)
{
    Walker w(pv, prm, blockIdx.x);
    const int n_total = (int)(w.end - w.cur);                 // runs; every run has at least one tile
    Segment s;
    uint32_t stage = 0, seg = 0;       // running stage / pair counters
    const int R = prm.d.T + prm.d.C;
    const uint32_t q_box_bytes = 32u * prm.G * 128u;
    TileRef prev = {0, 0, false};
    bool have_prev = false;
    // fills stage `stage` with V of `prev` (if any) and K of `cur` (if any)
    auto fill = [&](const TileRef* cur) -> bool {
        const uint32_t st = stage % kStages;
        if (!mbar_wait(&sh.kv_empty[st], ((stage / kStages) & 1) ^ 1, &sh.abort, prm.wait_ns)) return false;
        mbar_arrive_expect_tx(&sh.kv_full[st], (have_prev ? kTileBytes : 0) + (cur ? kTileBytes : 0));
        if (have_prev) {
            const CUtensorMap* m = prev.soft ? vs_map : v_map;
            tma_load_3d(sh.kv[st][0], m, &sh.kv_full[st], 0, prev.g, prev.z);
            tma_load_3d(sh.kv[st][0] + kHalfTile, m, &sh.kv_full[st], 64, prev.g, prev.z);
        }
        if (cur) {
            const CUtensorMap* m = cur->soft ? ks_map : k_map;
            tma_load_3d(sh.kv[st][1], m, &sh.kv_full[st], 0, cur->g, cur->z);
            tma_load_3d(sh.kv[st][1] + kHalfTile, m, &sh.kv_full[st], 64, cur->g, cur->z);
        }
        ++stage;
        return true;
    };
    while (w.next(s)) {
        for (int t = s.t0; t < s.t1; ++t) {
            TileRef cur;
            cur.g = s.g;
            cur.soft = t >= s.nkt;
            // key tile t of a sequence is its slots 128 t .. 128 t + 127: one page of a paged pool
            cur.z = cur.soft ? 0
                  : prm.map.block_table ? prm.map.block_table[(size_t)s.b * prm.map.max_pages + t] * kTileKeys
                                        : (int)(s.slot0 + (int64_t)t * kTileKeys);
            // the stage first (it carries the previous pair's last V tile, which must not wait for
            // the Q buffer), then, at the start of a pair, its Q (both M tiles, two 64-wide halves each)
            if (!fill(&cur)) return;
            if (t == s.t0) {
                if (!mbar_wait(&sh.q_empty, (seg & 1) ^ 1, &sh.abort, prm.wait_ns)) return;
                mbar_arrive_expect_tx(&sh.q_full, 2u * prm.n_mt * q_box_bytes);
                for (int mt = 0; mt < prm.n_mt; ++mt)
                    for (int kb = 0; kb < 2; ++kb)
                        tma_load_3d(sh.q + (mt * 2 + kb) * kHalfTile, q_map, &sh.q_full, kb * 64, s.g * prm.G, s.b * R + kGroupRows * s.rg + 32 * mt);
            }
            prev = cur;
            have_prev = true;
        }
        ++seg;
    }
    if (n_total > 0 && !fill(nullptr)) return;
}

// One thread issues all tensor-core work.  Per stage g: P V of key tile g-1 for both M tiles (each
// as soon as its P is there), Q K^T of key tile g for both, then the stage is released.
template <bool kTwo>
__device__ void mma_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t tmem)
{
    constexpr int kMt = kTwo ? 2 : 1;
    Walker w(pv, prm, blockIdx.x);
    Segment s;
    uint32_t stage = 0, seg = 0;
    // descriptor low words: Q tiles (K-major); a stage's K tile (K-major) and V tile (MN-major, its
    // two 64-column halves kHalfTile apart) = stage 0's words + stage * stage size
    const uint32_t q_lo = desc_lo(smem_u32(sh.q), 16);
    const uint32_t v_lo0 = desc_lo(smem_u32(sh.kv[0][0]), kHalfTile), k_lo0 = desc_lo(smem_u32(sh.kv[0][1]), 16);
    constexpr uint32_t kTileStep = kTileBytes >> 4, kStageStep = 2 * kTileStep;

    // S_t = Q_t K^T: 8 steps of 16 head dims; step i sits in 64-column half i/4 at byte 32*(i%4) of the swizzled row
    auto issue_qk = [&](int t, uint32_t kl) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const uint32_t off = ((uint32_t)(i >> 2) * kHalfTile + (uint32_t)(i & 3) * 32u) >> 4;
            mma_ss(tmem + t * 128, q_lo + t * kTileStep + off, kl + off, kIdescQK, i > 0 ? 1u : 0u);
        }
        tc_commit(&sh.s_full[t]);
    };
    // O_t += P_t V: 8 steps of 16 keys (2048 B of the V tile and 8 TMEM columns of bf16 pairs each);
    // P sits in the first 64 columns of the S_t block
    auto issue_pv = [&](int t, uint32_t vl, bool first_of_segment) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            mma_ts(tmem + 256 + t * 128, tmem + t * 128 + i * 8, vl + i * (2048u >> 4), kIdescPV,
                   (first_of_segment && i == 0) ? 0u : 1u);
    };
    // one stage: P V of the previous key tile (if any), Q K^T of the current one (if any)
    bool have_prev = false, prev_first = false, prev_last = false, prev_ragged = false;
    uint32_t n_fix = 0;
    auto run_stage = [&](bool have_cur, bool cur_first, bool cur_last, bool cur_ragged) -> bool {
        const uint32_t st = stage % kStages;
        if (!mbar_wait(&sh.kv_full[st], (stage / kStages) & 1, &sh.abort, prm.wait_ns)) return false;
        if (have_cur && cur_first && !mbar_wait(&sh.q_full, seg & 1, &sh.abort, prm.wait_ns)) return false;
        // the V tile of a sequence's last key tile: wait until its rows past the last slot are zero
        if (have_prev && prev_ragged) {
            if (!mbar_wait(&sh.v_fixed, n_fix & 1, &sh.abort, prm.wait_ns)) return false;
            ++n_fix;
        }
        tc_fence_after();
        const uint32_t vl = v_lo0 + st * kStageStep, kl = k_lo0 + st * kStageStep;
#pragma unroll
        for (int t = 0; t < kMt; ++t) {
            if (have_prev) {
                // (At the start of a pair this P V overwrites the previous pair's O_t; the softmax
                // threads hand P over only after they have read that O_t out.)
                if (!mbar_wait(&sh.p_full[t], (stage - 1) & 1, &sh.abort, prm.wait_ns)) return false;
                tc_fence_after();
                issue_pv(t, vl, prev_first);
                if (prev_last) tc_commit(&sh.o_done[t]);
            }
            if (have_cur) issue_qk(t, kl);
        }
        tc_commit(&sh.kv_empty[st]);
        if (have_cur && cur_last) tc_commit(&sh.q_empty);               // last Q K^T of the pair has been issued
        ++stage;
        have_prev = have_cur;
        prev_first = cur_first;
        prev_last = cur_last;
        prev_ragged = cur_ragged;
        return true;
    };

    const int R = prm.d.T + prm.d.C;
    while (w.next(s)) {
        const int n_tiles = s.t1 - s.t0;
        for (int j = 0; j < n_tiles; ++j)
            if (!run_stage(true, j == 0, j + 1 == n_tiles, ragged_rows(s, s.t0 + j, R) > 0)) return;
        ++seg;
    }
    if (have_prev) run_stage(false, false, false, false);
}

// Follows the stages of the ring like the issuing thread does and, where a stage carries the V tile
// of a sequence's last key tile, zeroes the rows past the sequence's last slot (generic-proxy
// stores, made visible to the tensor pipe by a proxy fence) before it lets the issuing thread go on.
// It arrives on every stage's empty barrier, so a stage is never refilled before it has seen it.
__device__ void tail_role(SharedStorage& sh, const Params& prm, const PlanView& pv)
{
    Walker w(pv, prm, blockIdx.x);
    Segment s;
    const int R = prm.d.T + prm.d.C, lane = threadIdx.x & 31;
    uint32_t stage = 0;
    int prev_valid = 0;                 // > 0: the previous tile's V needs rows [prev_valid, 128) zeroed
    bool have_prev = false;
    auto run_stage = [&](int cur_valid) -> bool {
        const uint32_t st = stage % kStages;
        if (!mbar_wait(&sh.kv_full[st], (stage / kStages) & 1, &sh.abort, prm.wait_ns)) return false;
        if (have_prev && prev_valid > 0) {
            const uint4 zero = make_uint4(0u, 0u, 0u, 0u);
            for (int half = 0; half < 2; ++half)
                for (int off = prev_valid * 128 + lane * 16; off < kHalfTile; off += 32 * 16)
                    *reinterpret_cast<uint4*>(sh.kv[st][0] + half * kHalfTile + off) = zero;
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.v_fixed);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.kv_empty[st]);
        ++stage;
        have_prev = true;
        prev_valid = cur_valid;
        return true;
    };
    while (w.next(s))
        for (int tile = s.t0; tile < s.t1; ++tile)
            if (!run_stage(ragged_rows(s, tile, R))) return;
    if (have_prev) run_stage(0);
}

__device__ void softmax_role(SharedStorage& sh, const Params& prm, const PlanView& pv, uint32_t tmem, int t /*M tile*/)
{
    const int lane_row = threadIdx.x & 127;                 // row of the M tile = TMEM lane
    const int warp_in_wg = (threadIdx.x >> 5) & 3;
    const uint32_t lane_base = (uint32_t)(warp_in_wg * 32) << 16;
    const uint32_t s_addr = tmem + lane_base + t * 128;
    const uint32_t o_addr = tmem + lane_base + 256 + t * 128;
    const int G = prm.G, T = prm.d.T, R = prm.d.T + prm.d.C, S = prm.d.S, Hq = prm.d.Hq;
    const int hl = lane_row % G;
    const float c = prm.c;

    Walker w(pv, prm, blockIdx.x);
    Segment s;
    uint32_t n_s = 0, seg = 0;
    while (w.next(s)) {
        const int r = kGroupRows * s.rg + 32 * t + lane_row / G;            // query row of this thread in this pair
        const bool row_valid = lane_row < 32 * G && r < R;
        const uint64_t mask = row_valid ? pv.mask[(size_t)s.b * kMaxRows + r] : 0ull;
        float m_ref = -INFINITY, l = 0.f;
        for (int tile = s.t0; tile < s.t1; ++tile) {
            if (!mbar_wait(&sh.s_full[t], n_s & 1, &sh.abort, prm.wait_ns)) return;
            ++n_s;
            tc_fence_after();
            uint32_t sv[128];
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) tmem_ld32(s_addr + q4 * 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[q4 * 32]));
            tc_wait_ld();
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
            const float m_new = fmaxf(m_ref, max128(sv) * c);
            if (tile == s.t0) {
                m_ref = m_new;
            } else {
                const bool move = m_new - m_ref > kRescaleThreshold;         // false when both are -inf (NaN)
                if (__any_sync(0xffffffffu, move)) {
                    const float alpha = move ? ex2(m_ref - m_new) : 1.f;
                    if (move) { m_ref = m_new; l *= alpha; }
                    // S_full of this tile implies the previous PV of this M tile has completed
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t ov[32];
                        tmem_ld32(o_addr + q4 * 32, ov);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) ov[j] = __float_as_uint(__uint_as_float(ov[j]) * alpha);
                        tmem_st32(o_addr + q4 * 32, ov);
                    }
                }
            }
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            // P overlays the first 64 columns of S_t (all of S_t is in registers by now); masked
            // scores are -inf and get weight exactly 0
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t pk[32];
                l += weights64(&sv[64 * half], c, neg_m, pk);
                tmem_st32(s_addr + 32 * half, pk);
            }
            tc_wait_st();
            tc_fence_before();
            mbar_arrive(&sh.p_full[t]);
        }
        // ---- epilogue of this pair / range ----
        if (!mbar_wait(&sh.o_done[t], seg & 1, &sh.abort, prm.wait_ns)) return;
        tc_fence_after();
        // O_t leaves tensor memory one row per thread; written like that, every store instruction of a
        // warp would touch 32 different lines.  Each 32-column chunk goes through the warp's
        // shared-memory tile instead and is stored in 16-byte pieces that cover whole rows: eight
        // rows per instruction for the bf16 output (4 lanes x 16 B each), four for an fp32 partial.
        const int h = s.g * G + hl;
        const int lane = threadIdx.x & 31;
        float4* xp = sh.xpose[threadIdx.x >> 5];
        const bool whole = s.part_slot < 0;
        const float inv_l = whole ? 1.f / l : 1.f;
        // where this lane's pieces go: row 8 kk + lane / 4 of the warp's 32 (output), row 4 kk + lane / 8 (partial)
        __nv_bfloat16* o_ptr[4];
        float* p_ptr = nullptr;
        if (whole) {
#pragma unroll
            for (int kk = 0; kk < 4; ++kk) {
                const int lr = warp_in_wg * 32 + 8 * kk + (lane >> 2);
                const int rk = kGroupRows * s.rg + 32 * t + lr / G;
                o_ptr[kk] = (lr < 32 * G && rk < R)
                                ? prm.out + (((size_t)s.b * R + rk) * Hq + s.g * G + lr % G) * kD + 8 * (lane & 3)
                                : nullptr;
            }
        } else {
            p_ptr = prm.partials + (size_t)s.part_slot * (partial_slot_bytes() / sizeof(float)) +
                    (size_t)(t * 128 + warp_in_wg * 32 + (lane >> 3)) * kPartD + 4 * (lane & 7);
        }
#pragma unroll 1
        for (int q4 = 0; q4 < 4; ++q4) {
            uint32_t ov[32];
            tmem_ld32(o_addr + q4 * 32, ov);
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
                    const float4 a = xp[k * 8 + (q ^ (k & 7))], c = xp[k * 8 + ((q + 1) ^ (k & 7))];
                    if (o_ptr[kk])
                        *reinterpret_cast<uint4*>(o_ptr[kk] + q4 * 32) =
                            make_uint4(pack_bf16(a.x, a.y), pack_bf16(a.z, a.w), pack_bf16(c.x, c.y), pack_bf16(c.z, c.w));
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
        if (whole) {
            if (row_valid && prm.lse)
                prm.lse[((size_t)s.b * R + r) * Hq + h] = (m_ref + log2f(l)) * 0.6931471805599453f;
        } else {
            float* ml = prm.partials + (size_t)s.part_slot * (partial_slot_bytes() / sizeof(float)) + (size_t)kPartRows * kPartD;
            ml[t * 128 + lane_row] = m_ref;
            ml[kPartRows + t * 128 + lane_row] = l;
        }
        // the P of the next range's first tile is only handed over after this point, which is what
        // keeps the tensor pipe from overwriting O_t before it has been read
        tc_fence_before();
        ++seg;
    }
}

__global__ void __launch_bounds__(kThreads, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap q_map, const __grid_constant__ CUtensorMap k_map,
                    const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap ks_map,
                    const __grid_constant__ CUtensorMap vs_map, const Params prm)
{
    extern __shared__ uint8_t smem_raw[];
    SharedStorage& sh = *reinterpret_cast<SharedStorage*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int warp = threadIdx.x >> 5;

    if (threadIdx.x == 0) {
        mbar_init(&sh.q_full, 1);
        mbar_init(&sh.q_empty, 1);
        // a stage is free again when its MMAs have completed and the tail warp has seen it
        for (int i = 0; i < kStages; ++i) { mbar_init(&sh.kv_full[i], 1); mbar_init(&sh.kv_empty[i], 2); }
        mbar_init(&sh.v_fixed, 1);
        for (int t = 0; t < 2; ++t) {
            mbar_init(&sh.s_full[t], 1);
            mbar_init(&sh.p_full[t], 128);
            mbar_init(&sh.o_done[t], 1);
        }
        sh.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 9) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;
    // Everything above touches only this kernel's own shared and tensor memory, so it runs while the
    // kernel before this one in the stream drains.  From here on global memory is read and written:
    // every CTA waits until the kernels before this one have completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const PlanView pv = plan_view(const_cast<void*>(prm.plan), prm.d.B);

    if ((int)blockIdx.x >= pv.hdr->n_ctas) {
        // nothing to do: straight to the teardown, which releases tensor memory
    } else if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 224;");
        const int t = warp >> 2;
        if (t < prm.n_mt) softmax_role(sh, prm, pv, tmem, t);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 56;");
        if (warp == 8) {
            if ((threadIdx.x & 31) == 0) producer_role(sh, prm, pv, &q_map, &k_map, &v_map, &ks_map, &vs_map);
        } else if (warp == 9) {
            if ((threadIdx.x & 31) == 0) {
                if (prm.n_mt > 1) mma_role<true>(sh, prm, pv, tmem);
                else mma_role<false>(sh, prm, pv, tmem);
            }
        } else if (warp == 10) {
            tail_role(sh, prm, pv);
        }
        __syncwarp();
    }
    // ---- teardown ----
    tc_fence_before();
    __syncthreads();
    if (sh.abort) {
        // give copies that may still be in flight time to land before the CTA's shared memory goes away
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        if (threadIdx.x == 0 && prm.status)
            for (int b = 0; b < prm.d.B; ++b) prm.status[b] = CONFU_ST_TIMEOUT;
        __syncthreads();
    }
    if (warp == 9) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

// ------------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// [rows][heads][128] bf16 tensor, box = box_rows x box_heads x 64 elements, 128-byte swizzle
bool make_tile_map(CUtensorMap* map, const void* base, uint64_t rows, uint64_t heads, uint32_t box_rows,
                   uint32_t box_heads)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)kD, heads, rows};
    const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, heads * kD * 2};
    const cuuint32_t box[3] = {64, box_heads, box_rows};
    const cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace tc

bool tc_attention_supported(const confu_dims& d)
{
    const int G = d.Hq / d.Hkv;
    return d.kv_dtype == CONFU_BF16 && d.D == 128 && G <= 4 && d.S <= 128;
}

cudaError_t launch_attention_tc(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                const void* v_cache, int64_t n_slots, const SlotMap& map,
                                const int32_t* prefix_len, const void* k_soft, const void* v_soft, const void* plan,
                                void* partials, void* out, float* lse, int32_t* status, cudaStream_t st)
{
    using namespace tc;
    const int R = d.T + d.C, G = d.Hq / d.Hkv;
    CUtensorMap q_map, k_map, v_map, ks_map, vs_map;
    bool ok = make_tile_map(&q_map, q, (uint64_t)d.B * R, d.Hq, 32, G) && make_tile_map(&k_map, k_cache, n_slots, d.Hkv, kTileKeys, 1) &&
              make_tile_map(&v_map, v_cache, n_slots, d.Hkv, kTileKeys, 1);
    if (d.S > 0) ok = ok && make_tile_map(&ks_map, k_soft, d.S, d.Hkv, kTileKeys, 1) && make_tile_map(&vs_map, v_soft, d.S, d.Hkv, kTileKeys, 1);
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
    prm.n_mt = R > 32 ? 2 : 1;
    prm.n_rg = (R + kGroupRows - 1) / kGroupRows;
    prm.G = G;
    prm.c = (d.sm_scale != 0.f ? d.sm_scale : 1.f / sqrtf((float)d.D)) * 1.4426950408889634f;
    prm.wait_ns = ctx->wait_ns;
    prm.k_scale = prm.v_scale = nullptr;
    const size_t smem = sizeof(SharedStorage) + 1024;
    static OncePerDevice attr_done;
    {
        cudaError_t e = attr_done.run([&] {
            return cudaFuncSetAttribute(attention_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        });
        if (e != cudaSuccess) return e;
    }
    // Launched as a programmatic dependent of whatever precedes it in the stream: its CTAs may be
    // scheduled while the predecessor drains; the kernel sets up its barriers and tensor memory, then
    // waits (griddepcontrol.wait) for the predecessor's completion and memory flush before it touches
    // global memory.
    cudaLaunchAttribute pdl[1];
    pdl[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    pdl[0].val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)ctx->sm_count);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cfg.attrs = pdl;
    cfg.numAttrs = 1;
    cudaError_t e = cudaLaunchKernelEx(&cfg, attention_tc_kernel, q_map, k_map, v_map, ks_map, vs_map, prm);
    if (e != cudaSuccess) return e;
    return launch_combine(prm, ctx->sm_count, st);
}

}  // namespace confu
