// What the tensor-core attention kernels share about walking a CTA's share of the work: the runs of
// key tiles the plan lists per CTA (or per CTA pair), and which keys of a tile a query row may see.
#pragma once

#include "tc_ptx.cuh"

namespace confu {
namespace tc {

constexpr int kTileBytes = kTileKeys * kD * 2;      // one 128-key tile of K or V of one kv head: 32 KB
constexpr int kHalfTile = kTileBytes / 2;           // one 64-wide half of the head dim: [128 rows][128 B]

struct Segment {
    int b, g, rg;      // sequence, kv head, group of 64 query rows
    int t0, t1;        // tiles [t0, t1) of this pair
    int nt, nkt;       // tiles of the pair; key tiles (the soft-prompt tile, if any, is tile nkt)
    int64_t P;         // prefix length
    int64_t slot0;     // packed pool: the sequence's first slot
    int part_slot;     // -1: the range covers the whole pair, write the output directly
};

// A CTA's runs of key tiles come from the plan: one 48-byte descriptor each, in walking order.
struct Walker {
    const SegDesc* cur;
    const SegDesc* end;
    bool soft;
    __device__ Walker(const PlanView& v, const Params& p, int cta) : soft(p.d.S > 0)
    {
        cur = v.segs + v.seg_begin[cta];
        end = v.segs + v.seg_begin[cta + 1];
    }
    // Next run of key tiles of one pair inside the share; false when the share is used up.
    __device__ bool next(Segment& s)
    {
        if (cur >= end) return false;
        const uint4* q = reinterpret_cast<const uint4*>(cur);
        const uint4 w0 = __ldg(q), w1 = __ldg(q + 1), w2 = __ldg(q + 2);
        s.b = (int)w0.x;
        s.g = (int)(w0.y & 0xffffu);
        s.rg = (int)(w0.y >> 16);
        s.t0 = (int)w0.z;
        s.t1 = (int)w0.w;
        s.nt = (int)w1.x;
        s.nkt = s.nt - (soft ? 1 : 0);
        s.P = (int)w1.y;
        s.part_slot = (int)w1.z;
        s.slot0 = (int64_t)(((uint64_t)w2.y << 32) | w2.x);
        ++cur;
        return true;
    }
};

// Slots of key tile `tile` that belong to the sequence when the tile is its last key tile and
// reaches past its last slot (1..127); 0 for every other tile.
__device__ __forceinline__ int ragged_rows(const Segment& s, int tile, int R)
{
    if (tile != s.nkt - 1) return 0;
    return (int)((s.P + R) & (kTileKeys - 1));
}

// Which of the 128 keys of tile `t` may row r see.  lo: keys 0..63 of the tile, hi: 64..127.
__device__ __forceinline__ void visible_bits(const Segment& s, int t, int R, int T, int S, int r, bool row_valid,
                                             uint64_t mask, uint64_t& lo, uint64_t& hi)
{
    if (!row_valid) { lo = hi = ~0ull; return; }
    if (t >= s.nkt) {                          // soft-prompt tile: contemplate rows only, S entries
        const bool sees = r >= T;
        lo = sees ? (S >= 64 ? ~0ull : ((1ull << S) - 1)) : 0ull;
        hi = sees ? (S > 64 ? (S >= 128 ? ~0ull : ((1ull << (S - 64)) - 1)) : 0ull) : 0ull;
        return;
    }
    const int64_t off = s.P - (int64_t)t * kTileKeys;      // position of tree slot 0 inside this tile (may be < 0 or >= 128)
    // prefix part: keys [0, off)
    unsigned __int128 v = 0;
    if (off >= 128) v = ~(unsigned __int128)0;
    else if (off > 0) v = (((unsigned __int128)1) << off) - 1;
    // tree rows' slots: bit j of mask at position off + j; a contemplate row's own slot at off + r
    const unsigned __int128 m = (unsigned __int128)mask;
    if (off >= 0) { if (off < 128) v |= m << off; }
    else if (off > -64) v |= m >> (-off);
    if (r >= T) {
        const int64_t self = off + r;
        if (self >= 0 && self < 128) v |= ((unsigned __int128)1) << self;
    }
    (void)R;
    lo = (uint64_t)v;
    hi = (uint64_t)(v >> 64);
}

// max of 128 floats held as raw bits, as eight independent chains of three-input max
__device__ __forceinline__ float max128(const uint32_t (&sv)[128])
{
    float a[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        a[k] = fmaxf(__uint_as_float(sv[16 * k]), __uint_as_float(sv[16 * k + 1]));
#pragma unroll
        for (int j = 2; j < 16; j += 2)
            asm("max.f32 %0, %0, %1, %2;" : "+f"(a[k]) : "f"(__uint_as_float(sv[16 * k + j])), "f"(__uint_as_float(sv[16 * k + j + 1])));
    }
    return fmaxf(fmaxf(fmaxf(a[0], a[1]), fmaxf(a[2], a[3])), fmaxf(fmaxf(a[4], a[5]), fmaxf(a[6], a[7])));
}

// exp2(s*c - m) of 64 scores -> 32 packed bf16 pairs; returns their fp32 sum
__device__ __forceinline__ float weights64(const uint32_t* sv, float c, float neg_m, uint32_t (&pk)[32])
{
    uint64_t sum2 = f2_pack(0.f, 0.f);
    const uint64_t c2 = f2_pack(c, c), nm2 = f2_pack(neg_m, neg_m);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        float x0, x1;
        f2_unpack(f2_fma(f2_pack(__uint_as_float(sv[2 * j]), __uint_as_float(sv[2 * j + 1])), c2, nm2), x0, x1);
        const float p0 = ex2(x0), p1 = ex2(x1);
        sum2 = f2_add(sum2, f2_pack(p0, p1));
        pk[j] = pack_bf16(p0, p1);
    }
    float s0, s1;
    f2_unpack(sum2, s0, s1);
    return s0 + s1;
}

}  // namespace tc
}  // namespace confu
