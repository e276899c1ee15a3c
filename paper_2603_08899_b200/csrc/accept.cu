// Tree speculative-sampling acceptance.
//
//   row_stats_kernel   one streaming pass over every logit row of the target and draft matrices:
//                      per row chunk the running max, the sum of exp((x - max)/temperature) (online
//                      softmax), the lowest index of the max, and a non-finite flag.  HBM bound.
//   accept_walk_kernel one thread-block cluster of kWalkCluster CTAs per sequence: the sequential
//                      accept / reject walk.  After the k-th rejection at a node the target row is
//                      norm(max(p - q, 0)) applied k times; it is never materialised: each pass
//                      re-evaluates the k-level recursion per vocabulary entry from the two logit
//                      rows (L2 resident) and only the normalisers Z_1..Z_k are kept.  Every CTA of
//                      the cluster runs the same control flow on the same data; only the passes over
//                      the vocabulary are shared out (strip s to CTA s mod kWalkCluster), the strip
//                      sums being written into every CTA's shared memory before a cluster barrier.
//   match_walk_kernel  the sample-and-match rule, same cluster layout, no statistics kernel: at each
//                      node of the walked path the row's maximum, its softmax weights and the
//                      inverse CDF are computed on the spot, so only those rows are ever read.
#include <cooperative_groups.h>
#include <limits.h>

#include "common.cuh"

namespace confu {

constexpr int kStatChunksMax = 16;
constexpr int kWalkThreads = 512;
constexpr int kWalkCluster = 8;                           // CTAs per sequence (portable cluster size)
constexpr int kEpt = 8;                                   // vocabulary entries per thread per strip
constexpr int kStrip = kWalkThreads * kEpt;               // 4096
constexpr int kMaxStrips = 64;                            // V <= 262144
constexpr float kLog2e = 1.4426950408889634f;

struct RowStat {
    float m;        // max raw logit of the chunk
    float s;        // sum over the chunk of exp((x - m) / temperature)
    int32_t arg;    // lowest index of the max
    int32_t flag;   // 1: a non-finite logit was met
};

size_t accept_workspace_bytes(int B, int T, int /*V*/)
{
    return (size_t)2 * B * T * kStatChunksMax * sizeof(RowStat);
}

template <typename T>
__device__ __forceinline__ void load8(const T* __restrict__ row, int i0, int V, bool vec_ok, float (&x)[kEpt])
{
    if (vec_ok && i0 + kEpt <= V) {
        if constexpr (sizeof(T) == 2) {
            const uint4 v = *reinterpret_cast<const uint4*>(row + i0);
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                x[2 * j] = __uint_as_float(w[j] << 16);
                x[2 * j + 1] = __uint_as_float(w[j] & 0xffff0000u);
            }
        } else {
            const float4 a = *reinterpret_cast<const float4*>(row + i0);
            const float4 c = *reinterpret_cast<const float4*>(row + i0 + 4);
            x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w;
            x[4] = c.x; x[5] = c.y; x[6] = c.z; x[7] = c.w;
        }
    } else {
#pragma unroll
        for (int j = 0; j < kEpt; ++j) x[j] = (i0 + j < V) ? to_f32(row[i0 + j]) : -INFINITY;
    }
}

// ---------------------------------------------------------------------------------------------
// K3: row statistics
// ---------------------------------------------------------------------------------------------
// Eight bf16 logits (one 16-byte vector starting at index ib) folded into a thread's running
// statistics: maximum m, sum s of exp2((x - m) * k2), lowest index arg of the largest value bestv,
// non-finite flag.  Maximum and minimum are taken on packed bf16 pairs with NaN propagation, so one
// comparison of each against the finite range finds NaN and both infinities.
__device__ __forceinline__ void stats8_bf16(const uint4& v, int ib, float k2, float& m, float& s, float& bestv, int& arg,
                                            int& flag)
{
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    __nv_bfloat162 h[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) h[j] = *reinterpret_cast<const __nv_bfloat162*>(&w[j]);
    const __nv_bfloat162 mx2 = __hmax2_nan(__hmax2_nan(h[0], h[1]), __hmax2_nan(h[2], h[3]));
    const __nv_bfloat162 mn2 = __hmin2_nan(__hmin2_nan(h[0], h[1]), __hmin2_nan(h[2], h[3]));
    const float hi0 = __low2float(mx2), hi1 = __high2float(mx2), lo0 = __low2float(mn2), lo1 = __high2float(mn2);
    if (!(hi0 <= 3.0e38f && hi1 <= 3.0e38f && lo0 >= -3.0e38f && lo1 >= -3.0e38f)) flag = 1;
    const float cm = fmaxf(hi0, hi1);
    if (cm > bestv) {                                    // rare after the first vectors: find the first element equal to it
        bestv = cm;
#pragma unroll
        for (int j = 7; j >= 0; --j) {
            const float x = __uint_as_float((j & 1) ? (w[j >> 1] & 0xffff0000u) : (w[j >> 1] << 16));
            if (x == cm) arg = ib + j;
        }
    }
    if (cm > m) { s *= ex2((m - cm) * k2); m = cm; }
    const float nmk = -m * k2;
    uint64_t acc = f2_pack(0.f, 0.f);
    const uint64_t k22 = f2_pack(k2, k2), nmk2 = f2_pack(nmk, nmk);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        float x0, x1;
        f2_unpack(f2_fma(f2_pack(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xffff0000u)), k22, nmk2), x0, x1);
        acc = f2_add(acc, f2_pack(ex2(x0), ex2(x1)));
    }
    float a0, a1;
    f2_unpack(acc, a0, a1);
    s += a0 + a1;
}

template <typename T>
__global__ void __launch_bounds__(256) row_stats_kernel(const T* __restrict__ tl, const T* __restrict__ dl, int V,
                                                        int n_rows, int nch, int chunk_elems, float k2,
                                                        RowStat* __restrict__ stats)
{
    const int row = blockIdx.x, chunk = blockIdx.y, mat = blockIdx.z;
    const T* base = (mat == 0 ? tl : dl) + (size_t)row * V;
    const bool vec_ok = ((size_t)V * sizeof(T)) % 16 == 0;
    const int lo = chunk * chunk_elems, hi = min(V, lo + chunk_elems);
    const int tid = threadIdx.x;

    float m = -INFINITY, s = 0.f, bestv = -INFINITY;
    int arg = INT_MAX, flag = 0;

    for (int i0 = lo + tid * kEpt; i0 < hi; i0 += 256 * kEpt * 2) {
        float x[2][kEpt];
        const int i1 = i0 + 256 * kEpt;
        if constexpr (sizeof(T) == 2) {
            // bf16 rows, both 8-element vectors whole: packed path (about 4 instructions per logit)
            if (vec_ok && i1 + kEpt <= hi) {
                const uint4 v0 = *reinterpret_cast<const uint4*>(base + i0);
                const uint4 v1 = *reinterpret_cast<const uint4*>(base + i1);
                stats8_bf16(v0, i0, k2, m, s, bestv, arg, flag);
                stats8_bf16(v1, i1, k2, m, s, bestv, arg, flag);
                continue;
            }
        }
        load8(base, i0, hi, vec_ok, x[0]);
        if (i1 < hi) load8(base, i1, hi, vec_ok, x[1]);
#pragma unroll
        for (int u = 0; u < 2; ++u) {
            const int ib = u == 0 ? i0 : i1;
            if (ib >= hi) break;
            float lm = x[u][0];
#pragma unroll
            for (int j = 1; j < kEpt; ++j) lm = fmaxf(lm, x[u][j]);
            if (lm > m) { s *= exp2f((m - lm) * k2); m = lm; }
            float acc = 0.f;
#pragma unroll
            for (int j = 0; j < kEpt; ++j) {
                const float v = x[u][j];
                const bool in = ib + j < hi;
                if (in && !(fabsf(v) <= 3.0e38f)) flag = 1;
                acc += exp2f((v - m) * k2);                      // out-of-range entries are -inf -> 0
                if (v > bestv) { bestv = v; arg = ib + j; }
            }
            s += acc;
        }
    }
    // block reduction of (m, s), (bestv, arg), flag
    auto merge = [&](float m2, float s2, float v2, int a2, int f2) {
        const float mm = fmaxf(m, m2);
        const float c1 = (m == mm) ? 1.f : exp2f((m - mm) * k2);
        const float c2 = (m2 == mm) ? 1.f : exp2f((m2 - mm) * k2);
        s = s * c1 + s2 * c2;
        m = mm;
        if (v2 > bestv || (v2 == bestv && a2 < arg)) { bestv = v2; arg = a2; }
        flag |= f2;
    };
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const float s2 = __shfl_xor_sync(0xffffffffu, s, o);
        const float v2 = __shfl_xor_sync(0xffffffffu, bestv, o);
        const int a2 = __shfl_xor_sync(0xffffffffu, arg, o);
        const int f2 = __shfl_xor_sync(0xffffffffu, flag, o);
        merge(m2, s2, v2, a2, f2);
    }
    __shared__ float sm[8], ss[8], sv[8];
    __shared__ int sa[8], sf[8];
    if ((tid & 31) == 0) { sm[tid >> 5] = m; ss[tid >> 5] = s; sv[tid >> 5] = bestv; sa[tid >> 5] = arg; sf[tid >> 5] = flag; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 8; ++w) merge(sm[w], ss[w], sv[w], sa[w], sf[w]);
        RowStat r;
        r.m = m; r.s = s; r.arg = arg; r.flag = flag;
        stats[((size_t)mat * n_rows + row) * kStatChunksMax + chunk] = r;
    }
    (void)nch;
}

// ---------------------------------------------------------------------------------------------
// K4: the walk
// ---------------------------------------------------------------------------------------------
struct WalkShared {
    int code;
    int cur, len, k, nch, accepted, done, final_level;
    int path[kPathLen];
    int ch[kMaxTree];
    int xs[kMaxTree];          // rejected tokens at the current node
    float invZ[kMaxTree];      // 1 / Z_j
    float cs[kMaxTree];        // 1 / (1 - q_{j-1}(x_j))   (sibling_mode 1)
    float Mt, Md, invZt, invZd;
    int amax[kMaxTree];
    double strip[kMaxStrips];
    double warp_part[kMaxStrips][kWalkThreads / 32];
    double scan[kWalkThreads / 32];
    int pick;
    int pick_last;
    int tests, rejections;
    int strip_sel;
    double strip_off, target;
    // row maximum of match_walk_kernel: per warp, then per CTA of the cluster
    float red_m[kWalkThreads / 32], cl_m[kWalkCluster];
    int red_arg[kWalkThreads / 32], red_flag[kWalkThreads / 32], cl_arg[kWalkCluster], cl_flag[kWalkCluster];
    // maximum and sum of exponentials of two rows at once (statistics on demand)
    float red2_m[2][kWalkThreads / 32], red2_s[2][kWalkThreads / 32], cl2_m[2][kWalkCluster], cl2_s[2][kWalkCluster];
    int next;
    int cnt0, cnt1, below[64];     // children scan of the walk
    // closeness records: ratio tests (match rule: draws) within kBorderline of their threshold; the
    // last inverse-CDF draw: sum of all weights, running sums before and behind the chosen entry
    int border_tests, border_draw;
    double total, pick_lo, pick_hi;
};
constexpr double kBorderline = 1e-5;

// merged statistics of one row from its chunk partials (fixed order)
__device__ inline void merge_row(const RowStat* st, int nch, double inv_temp, float& M, double& Z, int& arg)
{
    float mm = -INFINITY;
    int a = INT_MAX;
    for (int c = 0; c < nch; ++c)
        if (st[c].m > mm) { mm = st[c].m; a = st[c].arg; }
    double z = 0.0;
    for (int c = 0; c < nch; ++c)
        if (st[c].m > -INFINITY) z += (double)st[c].s * exp(((double)st[c].m - (double)mm) * inv_temp);
    M = mm; Z = z; arg = a;
}

// Weight of vocabulary entry idx after `level` rejections at the current node:
//   level 0: p_0 = softmax(target)            level k: max(p_{k-1} - q_{k-1}, 0)  (unnormalised p_k)
__device__ __forceinline__ float weight_at(float tx, float dx, int idx, int level, int mode, const WalkShared& sh,
                                           float k2)
{
    float p = ex2((tx - sh.Mt) * k2) * sh.invZt;
    if (level == 0) return p;
    float q = ex2((dx - sh.Md) * k2) * sh.invZd;
    for (int j = 0; j + 1 < level; ++j) {
        const float pn = fmaxf(p - q, 0.f) * sh.invZ[j];
        if (mode == 1) q = (idx == sh.xs[j]) ? 0.f : q * sh.cs[j];
        p = pn;
    }
    return fmaxf(p - q, 0.f);
}

// fp32 sums of the weights of two runs of eight entries, i0 .. i0 + 7 and i1 .. i1 + 7 (i1 < 0: none),
// all loads issued before any weight is computed.  fp64 arithmetic is scarce on this part: everything
// above a thread's eight is summed in fp64.  A real call on purpose: a pass over the vocabulary runs
// its code once or twice, so what counts is how little code there is to fetch, and this body is the
// same for every strip, pass and level.
template <typename T>
__device__ __noinline__ float2 weight_sum8x2(const T* __restrict__ trow, const T* __restrict__ drow, int V, bool vec_ok,
                                             int i0, int i1, int level, int mode, const WalkShared& sh, float k2)
{
    float tx[2][kEpt], dx[2][kEpt];
    load8(trow, i0, V, vec_ok, tx[0]);
    if (level > 0) load8(drow, i0, V, vec_ok, dx[0]);
    if (i1 >= 0) {
        load8(trow, i1, V, vec_ok, tx[1]);
        if (level > 0) load8(drow, i1, V, vec_ok, dx[1]);
    }
    float2 acc = make_float2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < kEpt; ++j) acc.x += weight_at(tx[0][j], level > 0 ? dx[0][j] : 0.f, i0 + j, level, mode, sh, k2);
    if (i1 >= 0) {
#pragma unroll
        for (int j = 0; j < kEpt; ++j) acc.y += weight_at(tx[1][j], level > 0 ? dx[1][j] : 0.f, i1 + j, level, mode, sh, k2);
    }
    return acc;
}

// Inverse-CDF search inside one run of eight entries: `run` is the fp64 sum of all weights before
// entry i0.  Returns the first entry whose running sum exceeds the target (INT_MAX: none here);
// last = the highest entry of the eight with a positive weight (-1: none).
template <typename T>
__device__ __noinline__ int find8(const T* __restrict__ trow, const T* __restrict__ drow, int V, bool vec_ok, int i0,
                                  int level, int mode, const WalkShared& sh, float k2, double run, double target,
                                  int& last, double& lo, double& hi)
{
    float tx[kEpt], dx[kEpt];
    load8(trow, i0, V, vec_ok, tx);
    if (level > 0) load8(drow, i0, V, vec_ok, dx);
    int cand = INT_MAX;
    last = -1;
    lo = hi = 0.0;
#pragma unroll
    for (int j = 0; j < kEpt; ++j) {
        const float w = weight_at(tx[j], level > 0 ? dx[j] : 0.f, i0 + j, level, mode, sh, k2);
        const double before = run;
        run += (double)w;
        if (w > 0.f) last = i0 + j;
        if (cand == INT_MAX && run > target) { cand = i0 + j; lo = before; hi = run; }
    }
    return cand;
}

// Sum of weight_at(., level) over the vocabulary, strip by strip; fills sh.strip[] of every CTA of
// the cluster and returns the total to thread 0 (0 to the others).  CTA `rank` computes strips
// rank, rank + kWalkCluster, ...
template <typename T>
__device__ double full_pass(const T* __restrict__ trow, const T* __restrict__ drow, int V, bool vec_ok, int level,
                            int mode, WalkShared& sh, float k2)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, n_strips = (V + kStrip - 1) / kStrip;
#pragma unroll 1
    for (int st = rank; st < n_strips; st += 2 * kWalkCluster) {
        const int st1 = st + kWalkCluster < n_strips ? st + kWalkCluster : -1;
        const float2 a8 = weight_sum8x2(trow, drow, V, vec_ok, st * kStrip + tid * kEpt,
                                        st1 >= 0 ? st1 * kStrip + tid * kEpt : -1, level, mode, sh, k2);
        const double a0 = warp_sum((double)a8.x), a1 = warp_sum((double)a8.y);
        if ((tid & 31) == 0) {
            sh.warp_part[st][tid >> 5] = a0;
            if (st1 >= 0) sh.warp_part[st1][tid >> 5] = a1;
        }
    }
    __syncthreads();
    // every CTA has finished reading the strip sums of the previous pass: they may be overwritten
    cluster.sync();
    for (int i = tid; i < kMaxStrips * kWalkCluster; i += kWalkThreads) {
        const int st = i / kWalkCluster, peer = i % kWalkCluster;
        if (st < n_strips && st % kWalkCluster == rank) {
            double a = 0.0;
            for (int w = 0; w < kWalkThreads / 32; ++w) a += sh.warp_part[st][w];
            *cluster.map_shared_rank(&sh.strip[st], peer) = a;
        }
    }
    cluster.sync();
    double tot = 0.0;                    // thread 0 alone needs the total
    if (tid == 0)
        for (int st = 0; st < n_strips; ++st) tot += sh.strip[st];
    return tot;
}

// Inverse CDF in index order over weight_at(., level) using the strip sums of the last full_pass.
template <typename T>
__device__ int locate(const T* __restrict__ trow, const T* __restrict__ drow, int V, bool vec_ok, int level, int mode,
                      WalkShared& sh, float k2, double u, bool& borderline)
{
    const int tid = threadIdx.x, n_strips = (V + kStrip - 1) / kStrip;
    if (tid == 0) {
        double tot = 0.0;
        for (int s = 0; s < n_strips; ++s) tot += sh.strip[s];
        const double target = u * tot;
        double cum = 0.0;
        int sel = -1, last_nz = 0;
        for (int s = 0; s < n_strips; ++s) {
            if (sh.strip[s] > 0.0) last_nz = s;
            if (cum + sh.strip[s] > target) { sel = s; break; }
            cum += sh.strip[s];
        }
        if (sel < 0) {                      // rounding left no strip: take the last one that has mass
            sel = last_nz;
            cum = 0.0;
            for (int s = 0; s < sel; ++s) cum += sh.strip[s];
        }
        sh.strip_sel = sel; sh.strip_off = cum; sh.target = target; sh.total = tot;
        sh.pick = INT_MAX; sh.pick_last = -1;
    }
    __syncthreads();
    const int i0 = sh.strip_sel * kStrip + tid * kEpt;
    // the thread's eight weights, summed as in full_pass
    const double loc = (double)weight_sum8x2(trow, drow, V, vec_ok, i0, -1, level, mode, sh, k2).x;
    // block exclusive scan of loc (double): warp scan + warp totals
    double incl = loc;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double t = __shfl_up_sync(0xffffffffu, incl, o);
        if ((tid & 31) >= o) incl += t;
    }
    if ((tid & 31) == 31) sh.scan[tid >> 5] = incl;
    __syncthreads();
    double off = sh.strip_off;
    for (int wi = 0; wi < (tid >> 5); ++wi) off += sh.scan[wi];
    const double run = off + (incl - loc);
    int last;
    double lo, hi;
    const int cand = find8(trow, drow, V, vec_ok, i0, level, mode, sh, k2, run, sh.target, last, lo, hi);
    if (cand != INT_MAX) atomicMin(&sh.pick, cand);
    if (last >= 0) atomicMax(&sh.pick_last, last);
    __syncthreads();
    if (cand != INT_MAX && cand == sh.pick) { sh.pick_lo = lo; sh.pick_hi = hi; }
    __syncthreads();
    int res = sh.pick != INT_MAX ? sh.pick : (sh.pick_last >= 0 ? sh.pick_last : 0);
    // how close the draw came to an edge of the chosen entry's cell of the normalised CDF (a draw
    // that rounding pushed past the last cell counts as on the edge)
    if (sh.pick == INT_MAX) borderline = true;
    else {
        const double dlo = fabs(u - sh.pick_lo / sh.total), dhi = fabs(sh.pick_hi / sh.total - u);
        borderline = fmin(dlo, dhi) < kBorderline;
    }
    __syncthreads();
    return res;
}

template <typename T>
__device__ void max_pass(const T* __restrict__ trow, int V, bool vec_ok, WalkShared& sh, float& M, int& arg, int& flag);

// (m, s) <- merge of two (maximum, sum of 2^((x - maximum) k2)) pairs; an empty pair is (-inf, 0)
__device__ __forceinline__ void ms_merge(float& m, float& s, float om, float os, float k2)
{
    const float M = fmaxf(m, om);
    if (M == -INFINITY) { s = 0.f; return; }
    s = s * ex2((m - M) * k2) + os * ex2((om - M) * k2);
    m = M;
}

// Statistics on demand: maximum and sum of 2^((x - maximum) k2) of the target row and of the draft
// row of one node in a single pass over both (online softmax per thread, merged per warp, per CTA
// and over the cluster in a fixed order); flag: a non-finite logit in either row.
template <typename T>
__device__ void stats_pass(const T* __restrict__ trow, const T* __restrict__ drow, int V, bool vec_ok, WalkShared& sh,
                           float k2, float (&M)[2], double (&Z)[2], int& flag)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, n_strips = (V + kStrip - 1) / kStrip;
    float m[2] = {-INFINITY, -INFINITY}, s[2] = {0.f, 0.f};
    int f = 0;
    for (int st = rank; st < n_strips; st += kWalkCluster) {
        const int i0 = st * kStrip + tid * kEpt;
        float x[2][kEpt];
        load8(trow, i0, V, vec_ok, x[0]);
        load8(drow, i0, V, vec_ok, x[1]);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            float vm = -INFINITY;
#pragma unroll
            for (int j = 0; j < kEpt; ++j) {
                if (i0 + j < V) {
                    if (!(fabsf(x[r][j]) <= 3.0e38f)) f = 1;
                    vm = fmaxf(vm, x[r][j]);
                }
            }
            if (vm > m[r]) { s[r] *= ex2((m[r] - vm) * k2); m[r] = vm; }
            if (m[r] > -INFINITY) {
#pragma unroll
                for (int j = 0; j < kEpt; ++j) s[r] += ex2((x[r][j] - m[r]) * k2);      // padding is -inf: weight 0
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        f |= __shfl_xor_sync(0xffffffffu, f, o);
#pragma unroll
        for (int r = 0; r < 2; ++r) {
            const float om = __shfl_xor_sync(0xffffffffu, m[r], o), os = __shfl_xor_sync(0xffffffffu, s[r], o);
            // the same operand order in both partners, so that every lane ends with the same bits
            if ((tid & o) == 0) ms_merge(m[r], s[r], om, os, k2);
            else { float a = om, b = os; ms_merge(a, b, m[r], s[r], k2); m[r] = a; s[r] = b; }
        }
    }
    if ((tid & 31) == 0) {
        sh.red_flag[tid >> 5] = f;
        for (int r = 0; r < 2; ++r) { sh.red2_m[r][tid >> 5] = m[r]; sh.red2_s[r][tid >> 5] = s[r]; }
    }
    __syncthreads();
    cluster.sync();                      // every CTA has finished reading the previous exchange
    if (tid < kWalkCluster) {
        int bf = 0;
        float bm[2] = {-INFINITY, -INFINITY}, bs[2] = {0.f, 0.f};
        for (int w = 0; w < kWalkThreads / 32; ++w) {
            bf |= sh.red_flag[w];
            for (int r = 0; r < 2; ++r) ms_merge(bm[r], bs[r], sh.red2_m[r][w], sh.red2_s[r][w], k2);
        }
        *cluster.map_shared_rank(&sh.cl_flag[rank], tid) = bf;
        for (int r = 0; r < 2; ++r) {
            *cluster.map_shared_rank(&sh.cl2_m[r][rank], tid) = bm[r];
            *cluster.map_shared_rank(&sh.cl2_s[r][rank], tid) = bs[r];
        }
    }
    cluster.sync();
    flag = 0;
    for (int c = 0; c < kWalkCluster; ++c) flag |= sh.cl_flag[c];
    for (int r = 0; r < 2; ++r) {
        float mm = -INFINITY;
        for (int c = 0; c < kWalkCluster; ++c) mm = fmaxf(mm, sh.cl2_m[r][c]);
        double z = 0.0;
        for (int c = 0; c < kWalkCluster; ++c)
            if (sh.cl2_m[r][c] > -INFINITY) z += (double)sh.cl2_s[r][c] * exp2((double)(sh.cl2_m[r][c] - mm) * (double)k2);
        M[r] = mm;
        Z[r] = z;
    }
}

template <typename T>
__global__ void __launch_bounds__(kWalkThreads) accept_walk_kernel(
    int Tn, int C, int V, const T* __restrict__ tl, const T* __restrict__ dl, const int32_t* __restrict__ tokens,
    const int32_t* __restrict__ parent, const int32_t* __restrict__ con_owner, const float* __restrict__ uniforms,
    float temperature, int mode, int lazy, int nch, int n_rows, const RowStat* __restrict__ stats,
    int32_t* __restrict__ accept_len, int32_t* __restrict__ path, int32_t* __restrict__ next_token,
    int32_t* __restrict__ future_row, int32_t* __restrict__ counters, int32_t* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WalkShared& sh = *reinterpret_cast<WalkShared*>(smem_raw);
    const int b = blockIdx.x / kWalkCluster, tid = threadIdx.x;
    const bool writer = blockIdx.x % kWalkCluster == 0;            // the CTA of the cluster that writes the outputs
    const int32_t* par = parent + (size_t)b * Tn;
    const int32_t* tok = tokens + (size_t)b * Tn;
    const int32_t* own = con_owner ? con_owner + (size_t)b * C : nullptr;
    const bool greedy = !(temperature > 0.f);
    const RowStat* st_t = stats + ((size_t)0 * n_rows + (size_t)b * Tn) * kStatChunksMax;
    const RowStat* st_d = stats + ((size_t)1 * n_rows + (size_t)b * Tn) * kStatChunksMax;
    const bool vec_ok = ((size_t)V * sizeof(T)) % 16 == 0;

    if (tid == 0) sh.code = INT_MAX;
    __syncthreads();
    // ---- validation (lowest code wins, like a sequential check in code order) ----
    if (tid < Tn) {
        int code = INT_MAX;
        const int p = par[tid];
        if (tid == 0 ? (p != -1) : (p < 0 || p >= tid)) code = CONFU_ST_BAD_PARENT;
        else if (tok[tid] < 0 || tok[tid] >= V) code = CONFU_ST_BAD_TOKEN;
        else {
            if (!greedy && mode == 1 && tid > 0)
                for (int j = tid + 1; j < Tn; ++j)
                    if (par[j] == p && tok[j] == tok[tid]) code = CONFU_ST_DUP_SIBLING;
            if (code == INT_MAX && !lazy) {
                // (all flags are fetched before any is looked at: independent loads, one round trip)
                int f = 0;
                for (int c = 0; c < nch; ++c) {
                    f |= st_t[(size_t)tid * kStatChunksMax + c].flag;
                    if (!greedy) f |= st_d[(size_t)tid * kStatChunksMax + c].flag;
                }
                if (f) code = CONFU_ST_NONFINITE;
            }
        }
        if (code != INT_MAX) atomicMin(&sh.code, code);
    }
    if (tid < C) {
        const int o = own[tid];
        if (o < 0 || o >= Tn) atomicMin(&sh.code, (int)CONFU_ST_BAD_OWNER);
    }
    __syncthreads();
    int32_t* pth = path + (size_t)b * kPathLen;
    if (sh.code != INT_MAX) {
        if (writer && tid < kPathLen) pth[tid] = tid == 0 ? 0 : -1;
        if (writer && tid == 0) {
            accept_len[b] = 0; next_token[b] = -1;
            if (future_row) future_row[b] = -1;
            if (counters) { counters[4 * b] = 0; counters[4 * b + 1] = 0; counters[4 * b + 2] = 0; counters[4 * b + 3] = 0; }
            if (status) status[b] = sh.code;
        }
        return;
    }
    const double inv_temp = greedy ? 1.0 : 1.0 / (double)temperature;
    const float k2 = (float)inv_temp * kLog2e;

    if (tid == 0) { sh.cur = 0; sh.len = 0; sh.path[0] = 0; sh.tests = 0; sh.rejections = 0; sh.done = 0; sh.border_tests = 0; sh.border_draw = 0; }
    __syncthreads();

    int lazy_code = 0;                // statistics on demand: a non-finite logit in a row that was needed
    if (greedy && lazy) {
        // the same walk as below, node by node, with the argmax of a row computed when the first
        // child of a kept node comes up (every CTA of the cluster takes the same branches)
        if (tid == 0) { sh.k = 0; sh.cur = 0; sh.len = 0; }
        if (tid < Tn) sh.amax[tid] = -2;
        __syncthreads();
        unsigned long long keep = 1ull;
        for (int i = 1; i < Tn && !lazy_code; ++i) {
            const int pa = par[i];
            if (!((keep >> pa) & 1ull)) continue;
            if (sh.amax[pa] == -2) {
                float M; int a, flag;
                max_pass(tl + ((size_t)b * Tn + pa) * V, V, vec_ok, sh, M, a, flag);
                if (flag) { lazy_code = CONFU_ST_NONFINITE; break; }
                __syncthreads();
                if (tid == 0) sh.amax[pa] = a;
                __syncthreads();
            }
            if (tok[i] == sh.amax[pa]) keep |= 1ull << i;
        }
        if (!lazy_code) {
            // deepest kept node, lowest index on ties; its own row gives the next token
            int best = 0, best_depth = 0;
            for (int i = 1; i < Tn; ++i) {
                if (!((keep >> i) & 1ull)) continue;
                int d = 0;
                for (int a = i; a > 0; a = par[a]) ++d;
                if (d > best_depth) { best = i; best_depth = d; }
            }
            int a_best = sh.amax[best];
            if (a_best == -2) {
                float M; int flag;
                max_pass(tl + ((size_t)b * Tn + best) * V, V, vec_ok, sh, M, a_best, flag);
                if (flag) lazy_code = CONFU_ST_NONFINITE;
            }
            __syncthreads();
            if (tid == 0 && !lazy_code) {
                sh.len = best_depth;
                for (int a = best, k = best_depth; a >= 0; a = par[a], --k) sh.path[k] = a;
                sh.cur = best;
                if (writer) next_token[b] = a_best;
            }
            __syncthreads();
        }
    } else if (greedy) {
        if (tid < Tn) {
            float M; double Z; int a;
            merge_row(st_t + (size_t)tid * kStatChunksMax, nch, 1.0, M, Z, a);
            sh.amax[tid] = a;
        }
        __syncthreads();
        if (tid == 0) {
            unsigned long long keep = 1ull;
            int depth[kMaxTree];
            depth[0] = 0;
            int best = 0;
            for (int i = 1; i < Tn; ++i) {
                const int pa = par[i];
                depth[i] = depth[pa] + 1;
                if (!((keep >> pa) & 1ull)) continue;
                if (tok[i] == sh.amax[pa]) {
                    keep |= 1ull << i;
                    if (depth[i] > depth[best]) best = i;
                }
            }
            sh.len = depth[best];
            for (int a = best, k = sh.len; a >= 0; a = par[a], --k) sh.path[k] = a;
            sh.cur = best;
            if (writer) next_token[b] = sh.amax[best];
        }
        __syncthreads();
    } else {
        const double u0 = (double)uniforms[(size_t)b * Tn];
        for (;;) {
            // ---- set up the current node ----
            if (lazy) {
                // maximum and normaliser of the node's two rows, computed now
                __syncthreads();
                const T* rt = tl + ((size_t)b * Tn + sh.cur) * V;
                const T* rd = dl + ((size_t)b * Tn + sh.cur) * V;
                float M[2];
                double Z[2];
                int flag;
                stats_pass(rt, rd, V, vec_ok, sh, k2, M, Z, flag);
                if (flag) { lazy_code = CONFU_ST_NONFINITE; break; }
                __syncthreads();
                if (tid == 0) { sh.Mt = M[0]; sh.invZt = (float)(1.0 / Z[0]); sh.Md = M[1]; sh.invZd = (float)(1.0 / Z[1]); }
            }
            if (!lazy && tid < 32) {
                // chunk statistics of the node's two rows -> maximum and normaliser of each: lanes 0-15
                // take the target row's chunks, lanes 16-31 the draft row's; maxima and the fp64 sum
                // are reduced inside each half warp (a fixed order, the same in every CTA)
                __syncwarp();
                const int c = tid & 15;
                const RowStat* st = (tid < 16 ? st_t : st_d) + (size_t)sh.cur * kStatChunksMax;
                const float m = c < nch ? st[c].m : -INFINITY;
                const float sc = c < nch ? st[c].s : 0.f;
                float mm = m;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) mm = fmaxf(mm, __shfl_xor_sync(0xffffffffu, mm, o));
                double z = m > -INFINITY ? (double)sc * exp(((double)m - (double)mm) * inv_temp) : 0.0;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
                if (tid == 0) { sh.Mt = mm; sh.invZt = (float)(1.0 / z); }
                if (tid == 16) { sh.Md = mm; sh.invZd = (float)(1.0 / z); }
            }
            // children of the current node in increasing index: nodes 0-31 by the lanes of warp 0, 32-63
            // by warp 1, each child's place = the children before it
            if (tid < 2 * 32) {
                const int cur = sh.cur;
                const bool is_child = tid > cur && tid < Tn && par[tid] == cur;
                const unsigned mask = __ballot_sync(0xffffffffu, is_child);
                if (tid == 0) sh.cnt0 = __popc(mask);
                if (tid == 32) sh.cnt1 = __popc(mask);
                sh.below[tid] = __popc(mask & ((1u << (tid & 31)) - 1u)) | (is_child ? 0x100 : 0);
            }
            __syncthreads();
            if (tid < 2 * 32 && (sh.below[tid] & 0x100)) sh.ch[(sh.below[tid] & 0xff) + (tid >= 32 ? sh.cnt0 : 0)] = tid;
            if (tid == 0) { sh.nch = sh.cnt0 + sh.cnt1; sh.k = 0; sh.accepted = -1; }
            __syncthreads();
            const int cur = sh.cur;
            const T* trow = tl + ((size_t)b * Tn + cur) * V;
            const T* drow = dl + ((size_t)b * Tn + cur) * V;
            int final_level = 0;
            bool have_strips = false;
            for (int ci = 0; ci < sh.nch; ++ci) {
                const int c = sh.ch[ci];
                // ---- ratio test of child c (thread 0, double) ----
                if (tid == 0) {
                    const int x = tok[c];
                    const double u = (double)uniforms[(size_t)b * Tn + c];
                    double p = exp(((double)to_f32(trow[x]) - (double)sh.Mt) * inv_temp) * (double)sh.invZt;
                    double q = exp(((double)to_f32(drow[x]) - (double)sh.Md) * inv_temp) * (double)sh.invZd;
                    for (int j = 0; j < sh.k; ++j) {
                        const double pn = fmax(p - q, 0.0) * (double)sh.invZ[j];
                        if (mode == 1) q = (x == sh.xs[j]) ? 0.0 : q * (double)sh.cs[j];
                        p = pn;
                    }
                    const double ratio = (q == 0.0) ? (p > 0.0 ? INFINITY : 0.0) : p / q;
                    ++sh.tests;
                    if (fabs(ratio - u) < kBorderline) ++sh.border_tests;
                    if (u < ratio) sh.accepted = c;
                    else {
                        ++sh.rejections;
                        sh.xs[sh.k] = x;
                        const double rem = 1.0 - q;
                        sh.cs[sh.k] = rem > 0.0 ? (float)(1.0 / rem) : 0.f;
                        sh.done = (mode == 1 && !(rem > 0.0)) ? 1 : 0;      // q has no mass left: stop testing
                    }
                }
                __syncthreads();
                if (sh.accepted >= 0) break;
                // ---- rejection k+1: normaliser of the new residual ----
                const int level = sh.k + 1;
                const double Z = full_pass(trow, drow, V, vec_ok, level, mode, sh, k2);
                have_strips = true;
                final_level = level;
                if (tid == 0) {
                    if (Z > 0.0) { sh.invZ[sh.k] = (float)(1.0 / Z); sh.k = level; }
                    else { sh.done = 2; }                                    // no mass: fall back to the target row
                }
                __syncthreads();
                if (sh.done) break;
            }
            if (sh.accepted >= 0) {
                __syncthreads();
                if (tid == 0) {
                    if (sh.len + 1 > CONFU_MAX_DEPTH) sh.done = 3;
                    else { sh.path[++sh.len] = sh.accepted; sh.cur = sh.accepted; }
                }
                __syncthreads();
                if (sh.done == 3) break;
                continue;
            }
            // ---- final draw at this node ----
            if (sh.done == 2) { final_level = 0; have_strips = false; }
            if (!have_strips) full_pass(trow, drow, V, vec_ok, final_level, mode, sh, k2);
            bool borderline;
            const int pick = locate(trow, drow, V, vec_ok, final_level, mode, sh, k2, u0, borderline);
            if (tid == 0) sh.border_draw = borderline ? 1 : 0;
            if (writer && tid == 0) next_token[b] = pick;
            break;
        }
        __syncthreads();
        if (sh.done == 3) {              // path buffer exhausted
            if (writer && tid < kPathLen) pth[tid] = tid == 0 ? 0 : -1;
            if (writer && tid == 0) {
                accept_len[b] = 0; next_token[b] = -1;
                if (future_row) future_row[b] = -1;
                if (status) status[b] = CONFU_ST_TOO_DEEP;
            }
            return;
        }
        if (sh.done == 2 && writer && tid == 0 && status) status[b] = CONFU_ST_DEGENERATE;
    }
    if (lazy_code) {
        if (writer && tid < kPathLen) pth[tid] = tid == 0 ? 0 : -1;
        if (writer && tid == 0) {
            accept_len[b] = 0; next_token[b] = -1;
            if (future_row) future_row[b] = -1;
            if (counters) { counters[4 * b] = 0; counters[4 * b + 1] = 0; counters[4 * b + 2] = 0; counters[4 * b + 3] = 0; }
            if (status) status[b] = lazy_code;
        }
        return;
    }
    // ---- outputs ----
    if (writer && tid < kPathLen) pth[tid] = tid <= sh.len ? sh.path[tid] : -1;
    if (writer && tid == 0) {
        accept_len[b] = sh.len;
        if (future_row) {
            int fr = -1;
            for (int a = sh.cur; a >= 0 && fr < 0; a = par[a])
                for (int k = 0; k < C; ++k)
                    if (own[k] == a) { fr = Tn + k; break; }
            future_row[b] = fr;
        }
        if (counters) {
            counters[4 * b] = sh.tests; counters[4 * b + 1] = sh.rejections;
            counters[4 * b + 2] = sh.border_tests; counters[4 * b + 3] = sh.border_draw;
        }
    }
}

// ---------------------------------------------------------------------------------------------
// K4b: sample-and-match walk with statistics on demand
// ---------------------------------------------------------------------------------------------
// Largest logit of a row, its lowest index and a non-finite flag; every CTA of the cluster gets
// the same three values (strips shared out as in full_pass, partial results exchanged through
// distributed shared memory and merged in rank order).
template <typename T>
__device__ void max_pass(const T* __restrict__ trow, int V, bool vec_ok, WalkShared& sh, float& M, int& arg, int& flag)
{
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = (int)cluster.block_rank();
    const int tid = threadIdx.x, n_strips = (V + kStrip - 1) / kStrip;
    float m = -INFINITY;
    int a = INT_MAX, f = 0;
    for (int st = rank; st < n_strips; st += kWalkCluster) {
        const int i0 = st * kStrip + tid * kEpt;
        float x[kEpt];
        load8(trow, i0, V, vec_ok, x);
#pragma unroll
        for (int j = 0; j < kEpt; ++j) {
            if (i0 + j < V) {
                if (!(fabsf(x[j]) <= 3.0e38f)) f = 1;
                if (x[j] > m) { m = x[j]; a = i0 + j; }
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, o);
        const int oa = __shfl_xor_sync(0xffffffffu, a, o);
        f |= __shfl_xor_sync(0xffffffffu, f, o);
        if (om > m || (om == m && oa < a)) { m = om; a = oa; }
    }
    if ((tid & 31) == 0) { sh.red_m[tid >> 5] = m; sh.red_arg[tid >> 5] = a; sh.red_flag[tid >> 5] = f; }
    __syncthreads();
    // every CTA has finished reading the previous exchange: it may be overwritten
    cluster.sync();
    if (tid < kWalkCluster) {
        float bm = -INFINITY;
        int ba = INT_MAX, bf = 0;
        for (int w = 0; w < kWalkThreads / 32; ++w) {
            bf |= sh.red_flag[w];
            if (sh.red_m[w] > bm || (sh.red_m[w] == bm && sh.red_arg[w] < ba)) { bm = sh.red_m[w]; ba = sh.red_arg[w]; }
        }
        *cluster.map_shared_rank(&sh.cl_m[rank], tid) = bm;
        *cluster.map_shared_rank(&sh.cl_arg[rank], tid) = ba;
        *cluster.map_shared_rank(&sh.cl_flag[rank], tid) = bf;
    }
    cluster.sync();
    M = -INFINITY; arg = INT_MAX; flag = 0;
    for (int r = 0; r < kWalkCluster; ++r) {
        flag |= sh.cl_flag[r];
        if (sh.cl_m[r] > M || (sh.cl_m[r] == M && sh.cl_arg[r] < arg)) { M = sh.cl_m[r]; arg = sh.cl_arg[r]; }
    }
}

template <typename T>
__global__ void __launch_bounds__(kWalkThreads) match_walk_kernel(
    int Tn, int C, int V, const T* __restrict__ tl, const int32_t* __restrict__ tokens,
    const int32_t* __restrict__ parent, const int32_t* __restrict__ con_owner, const float* __restrict__ uniforms,
    float temperature, int32_t* __restrict__ accept_len, int32_t* __restrict__ path, int32_t* __restrict__ next_token,
    int32_t* __restrict__ future_row, int32_t* __restrict__ counters, int32_t* __restrict__ status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    WalkShared& sh = *reinterpret_cast<WalkShared*>(smem_raw);
    const int b = blockIdx.x / kWalkCluster, tid = threadIdx.x;
    const bool writer = blockIdx.x % kWalkCluster == 0;
    const int32_t* par = parent + (size_t)b * Tn;
    const int32_t* tok = tokens + (size_t)b * Tn;
    const int32_t* own = con_owner ? con_owner + (size_t)b * C : nullptr;
    const bool greedy = !(temperature > 0.f);
    const bool vec_ok = ((size_t)V * sizeof(T)) % 16 == 0;
    const float k2 = (greedy ? 1.f : 1.f / temperature) * kLog2e;
    int32_t* pth = path + (size_t)b * kPathLen;

    if (tid == 0) { sh.code = INT_MAX; sh.cur = 0; sh.len = 0; sh.path[0] = 0; sh.tests = 0; sh.accepted = 0; sh.done = 0; sh.next = -1; sh.border_tests = 0; }
    __syncthreads();
    if (tid < Tn) {
        const int p = par[tid];
        if (tid == 0 ? (p != -1) : (p < 0 || p >= tid)) atomicMin(&sh.code, (int)CONFU_ST_BAD_PARENT);
        else if (tok[tid] < 0 || tok[tid] >= V) atomicMin(&sh.code, (int)CONFU_ST_BAD_TOKEN);
    }
    if (tid < C) {
        const int o = own[tid];
        if (o < 0 || o >= Tn) atomicMin(&sh.code, (int)CONFU_ST_BAD_OWNER);
    }
    __syncthreads();
    int code = sh.code == INT_MAX ? 0 : sh.code;
    while (!code) {
        const int cur = sh.cur;
        const T* trow = tl + ((size_t)b * Tn + cur) * V;
        float M;
        int arg, flag;
        max_pass(trow, V, vec_ok, sh, M, arg, flag);
        if (flag) { code = CONFU_ST_NONFINITE; break; }
        int x = arg;
        bool borderline = false;
        if (!greedy) {
            // weights 2^((x - M) k2), unnormalised: the inverse CDF scales the uniform by their sum
            if (tid == 0) { sh.Mt = M; sh.invZt = 1.f; }
            __syncthreads();
            full_pass(trow, trow, V, vec_ok, 0, 0, sh, k2);
            x = locate(trow, trow, V, vec_ok, 0, 0, sh, k2, (double)uniforms[(size_t)b * Tn + cur], borderline);
        }
        if (tid == 0) {
            ++sh.tests;
            if (borderline) ++sh.border_tests;
            int hit = -1;
            for (int c = cur + 1; c < Tn; ++c)
                if (par[c] == cur && tok[c] == x) { hit = c; break; }
            if (hit < 0) { sh.next = x; sh.done = 1; }
            else if (sh.len + 1 > CONFU_MAX_DEPTH) sh.done = 3;
            else { sh.path[++sh.len] = hit; sh.cur = hit; ++sh.accepted; }
        }
        __syncthreads();
        if (sh.done == 3) code = CONFU_ST_TOO_DEEP;
        if (sh.done) break;
    }
    if (code) {
        if (writer && tid < kPathLen) pth[tid] = tid == 0 ? 0 : -1;
        if (writer && tid == 0) {
            accept_len[b] = 0; next_token[b] = -1;
            if (future_row) future_row[b] = -1;
            if (counters) { counters[4 * b] = 0; counters[4 * b + 1] = 0; counters[4 * b + 2] = 0; counters[4 * b + 3] = 0; }
            if (status) status[b] = code;
        }
        return;
    }
    if (writer && tid < kPathLen) pth[tid] = tid <= sh.len ? sh.path[tid] : -1;
    if (writer && tid == 0) {
        accept_len[b] = sh.len;
        next_token[b] = sh.next;
        if (future_row) {
            int fr = -1;
            for (int a = sh.cur; a >= 0 && fr < 0; a = par[a])
                for (int k = 0; k < C; ++k)
                    if (own[k] == a) { fr = Tn + k; break; }
            future_row[b] = fr;
        }
        if (counters) { counters[4 * b] = sh.tests; counters[4 * b + 1] = sh.accepted; counters[4 * b + 2] = sh.border_tests; counters[4 * b + 3] = 0; }
    }
}

template <typename T>
static cudaError_t launch_match_t(int B, int Tn, int C, int V, const void* tl, const int32_t* tokens,
                                  const int32_t* parent, const int32_t* con_owner, const float* uniforms,
                                  float temperature, int32_t* accept_len, int32_t* path, int32_t* next_token,
                                  int32_t* future_row, int32_t* counters, int32_t* status, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const size_t smem = sizeof(WalkShared);
    static OncePerDevice attr_done;          // (one per instantiation of this template)
    {
        cudaError_t e = attr_done.run([&] {
            return cudaFuncSetAttribute(match_walk_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        });
        if (e != cudaSuccess) return e;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)B * kWalkCluster);
    cfg.blockDim = dim3(kWalkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kWalkCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, match_walk_kernel<T>, Tn, C, V, (const T*)tl, tokens, parent, con_owner, uniforms,
                              temperature, accept_len, path, next_token, future_row, counters, status);
}

cudaError_t launch_accept_match(int B, int T, int C, int V, int logit_dtype, const void* tl, const int32_t* tokens,
                                const int32_t* parent, const int32_t* con_owner, const float* uniforms,
                                float temperature, int32_t* accept_len, int32_t* path, int32_t* next_token,
                                int32_t* future_row, int32_t* counters, int32_t* status, cudaStream_t st)
{
    if (logit_dtype == CONFU_F32)
        return launch_match_t<float>(B, T, C, V, tl, tokens, parent, con_owner, uniforms, temperature, accept_len, path,
                                     next_token, future_row, counters, status, st);
    return launch_match_t<__nv_bfloat16>(B, T, C, V, tl, tokens, parent, con_owner, uniforms, temperature, accept_len,
                                         path, next_token, future_row, counters, status, st);
}

template <typename T>
static cudaError_t launch_accept_t(int sm_count, int B, int Tn, int C, int V, const void* tl, const void* dl, const int32_t* tokens,
                                   const int32_t* parent, const int32_t* con_owner, const float* uniforms,
                                   float temperature, int mode_flags, int32_t* accept_len, int32_t* path,
                                   int32_t* next_token, int32_t* future_row, int32_t* counters, void* workspace,
                                   int32_t* status, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const int mode = mode_flags & 0xff, lazy = (mode_flags & CONFU_ACCEPT_LAZY) ? 1 : 0;
    const bool greedy = !(temperature > 0.f);
    const int n_rows = B * Tn;
    const int nmat = greedy ? 1 : 2;
    // enough CTAs to fill the machine a few times over, chunks a multiple of the vector width
    int nch = (sm_count * 8 + n_rows * nmat - 1) / (n_rows * nmat);
    nch = nch < 1 ? 1 : (nch > kStatChunksMax ? kStatChunksMax : nch);
    int chunk_elems = (V + nch - 1) / nch;
    chunk_elems = (chunk_elems + 15) / 16 * 16;
    nch = (V + chunk_elems - 1) / chunk_elems;
    const float k2 = (greedy ? 1.f : 1.f / temperature) * kLog2e;
    RowStat* stats = (RowStat*)workspace;
    cudaError_t e = cudaSuccess;
    if (!lazy) {
        row_stats_kernel<T><<<dim3(n_rows, nch, nmat), 256, 0, st>>>((const T*)tl, (const T*)dl, V, n_rows, nch,
                                                                     chunk_elems, k2, stats);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    const size_t smem = sizeof(WalkShared);
    static OncePerDevice attr_done;          // (one per instantiation of this template)
    e = attr_done.run([&] {
        return cudaFuncSetAttribute(accept_walk_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    });
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)B * kWalkCluster);
    cfg.blockDim = dim3(kWalkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kWalkCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, accept_walk_kernel<T>, Tn, C, V, (const T*)tl, (const T*)dl, tokens, parent, con_owner,
                              uniforms, temperature, mode, lazy, nch, n_rows, stats, accept_len, path, next_token, future_row,
                              counters, status);
}

// SM count of the current device, asked once per device (for callers without a context).
static cudaError_t current_sm_count(int& n)
{
    static int cached[OncePerDevice::kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= OncePerDevice::kMaxDevices) return cudaErrorInvalidDevice;
    if (!cached[dev]) {
        int v = 0;
        e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        cached[dev] = v;
    }
    n = cached[dev];
    return cudaSuccess;
}

cudaError_t launch_accept(const Ctx* ctx, int B, int T, int C, int V, int logit_dtype, const void* tl, const void* dl,
                          const int32_t* tokens, const int32_t* parent, const int32_t* con_owner,
                          const float* uniforms, float temperature, int sibling_mode, int32_t* accept_len,
                          int32_t* path, int32_t* next_token, int32_t* future_row, int32_t* counters,
                          void* workspace, int32_t* status, cudaStream_t st)
{
    int sm_count = ctx ? ctx->sm_count : 0;
    if (!ctx) {
        cudaError_t e = current_sm_count(sm_count);
        if (e != cudaSuccess) return e;
    }
    if (logit_dtype == CONFU_F32)
        return launch_accept_t<float>(sm_count, B, T, C, V, tl, dl, tokens, parent, con_owner, uniforms, temperature,
                                      sibling_mode, accept_len, path, next_token, future_row, counters, workspace,
                                      status, st);
    return launch_accept_t<__nv_bfloat16>(sm_count, B, T, C, V, tl, dl, tokens, parent, con_owner, uniforms, temperature,
                                          sibling_mode, accept_len, path, next_token, future_row, counters, workspace,
                                          status, st);
}

}  // namespace confu
