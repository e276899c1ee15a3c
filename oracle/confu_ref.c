/*
 * confu_ref.c -- fp64 CPU oracle for the ConFu tree-verification step.
 * TEST INFRASTRUCTURE ONLY: see confu_ref.h.  Plain C99 + OpenMP, no blocking,
 * no fusion, no reordering beyond what each definition states.
 */
#include "confu_ref.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ------------------------------------------------------------------ */
/* element access: widen bf16 / fp32 / fp64 exactly to double          */
/* ------------------------------------------------------------------ */
static double load_elem(const void* base, int dtype, int64_t i)
{
    if (dtype == CONFU_REF_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;
        float f;
        memcpy(&f, &bits, sizeof f);
        return (double)f;
    }
    if (dtype == CONFU_REF_F32) return (double)((const float*)base)[i];
    return ((const double*)base)[i];
}

int confu_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* ------------------------------------------------------------------ */
/* tree structure checks                                               */
/* ------------------------------------------------------------------ */
static int check_tree(const int32_t* parent, const int32_t* owner, int T, int C)
{
    if (parent[0] != -1) return CONFU_REF_ST_BAD_PARENT;
    for (int i = 1; i < T; ++i)
        if (parent[i] < 0 || parent[i] >= i) return CONFU_REF_ST_BAD_PARENT;
    for (int k = 0; k < C; ++k)
        if (owner[k] < 0 || owner[k] >= T) return CONFU_REF_ST_BAD_OWNER;
    return CONFU_REF_ST_OK;
}

/*
 * Visibility of tree slot j (0..R-1, the slot that holds row j's own key) from
 * query row r.  Tree row: itself and its ancestors.  Contemplate row: itself,
 * its owner and the owner's ancestors; never another contemplate row
 * (Fig. 3: one contemplate token after each draft token, mask adjusted so each
 * stays on its node's branch).
 */
static int tree_slot_visible(const int32_t* parent, const int32_t* owner, int T, int r, int j)
{
    if (j == r) return 1;
    if (j >= T) return 0;
    int a = (r < T) ? r : owner[r - T];
    while (a >= 0) {
        if (a == j) return 1;
        a = parent[a];
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* attention: one (b, r, h) output row, written from the definition    */
/* ------------------------------------------------------------------ */
static void attention_row(const confu_ref_dims* dm,
                          const void* q, const void* kc, const void* vc,
                          const int64_t* seq_start, const int32_t* prefix_len,
                          const void* ks, const void* vs,
                          const int32_t* parent, const int32_t* owner,
                          int b, int r, int h, double* out, double* lse)
{
    const int Hq = dm->Hq, Hkv = dm->Hkv, D = dm->D, T = dm->T, C = dm->C, S = dm->S;
    const int R = T + C, G = Hq / Hkv, g = h / G, dt = dm->dtype;
    const int64_t P = prefix_len[b], base = seq_start[b];
    const double scale = dm->sm_scale != 0.0 ? dm->sm_scale : 1.0 / sqrt((double)D);
    const int64_t n = (int64_t)S + P + R;
    const int32_t* par = parent + (int64_t)b * T;
    const int32_t* own = owner ? owner + (int64_t)b * C : NULL;
    const int64_t qoff = (((int64_t)b * R + r) * Hq + h) * D;

    double* score = (double*)malloc((size_t)n * sizeof(double));
    char* vis = (char*)malloc((size_t)n);

    /* which keys does row r see, and with what score */
    for (int64_t i = 0; i < n; ++i) {
        const void* kbase;
        int64_t koff;
        if (i < S) {                         /* soft-prompt entry i: contemplate rows only */
            vis[i] = (r >= T);
            kbase = ks; koff = ((int64_t)i * Hkv + g) * D;
        } else if (i < S + P) {              /* prefix slot: every row */
            vis[i] = 1;
            kbase = kc; koff = ((base + (i - S)) * Hkv + g) * D;
        } else {                             /* tree slot j */
            int j = (int)(i - S - P);
            vis[i] = (char)tree_slot_visible(par, own, T, r, j);
            kbase = kc; koff = ((base + P + j) * Hkv + g) * D;
        }
        if (!vis[i]) { score[i] = 0.0; continue; }
        double acc = 0.0;
        for (int d = 0; d < D; ++d)
            acc += load_elem(q, dt, qoff + d) * load_elem(kbase, dt, koff + d);
        score[i] = acc * scale;
    }
    double m = -INFINITY;
    for (int64_t i = 0; i < n; ++i) if (vis[i] && score[i] > m) m = score[i];
    double den = 0.0;
    for (int d = 0; d < D; ++d) out[d] = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        if (!vis[i]) continue;
        double w = exp(score[i] - m);
        den += w;
        const void* vbase;
        int64_t voff;
        if (i < S) { vbase = vs; voff = ((int64_t)i * Hkv + g) * D; }
        else       { vbase = vc; voff = ((base + (i - S)) * Hkv + g) * D; }
        for (int d = 0; d < D; ++d) out[d] += w * load_elem(vbase, dt, voff + d);
    }
    for (int d = 0; d < D; ++d) out[d] /= den;
    if (lse) *lse = m + log(den);
    free(score);
    free(vis);
}

static int attention_args_ok(const confu_ref_dims* dm)
{
    if (!dm) return 0;
    if (dm->B < 0 || dm->Hq <= 0 || dm->Hkv <= 0 || dm->D <= 0 || dm->T <= 0 || dm->C < 0 || dm->S < 0) return 0;
    if (dm->Hq % dm->Hkv) return 0;
    if (dm->dtype < CONFU_REF_BF16 || dm->dtype > CONFU_REF_F64) return 0;
    return 1;
}

int confu_ref_tree_attention(const confu_ref_dims* dm,
                             const void* q, const void* kc, const void* vc,
                             const int64_t* seq_start, const int32_t* prefix_len,
                             const void* ks, const void* vs,
                             const int32_t* parent, const int32_t* owner,
                             double* out, double* lse, int32_t* status)
{
    if (!attention_args_ok(dm)) return -1;
    const int B = dm->B, R = dm->T + dm->C, Hq = dm->Hq, D = dm->D;
    int* bad = (int*)calloc((size_t)(B > 0 ? B : 1), sizeof(int));
    for (int b = 0; b < B; ++b) {
        bad[b] = check_tree(parent + (int64_t)b * dm->T, owner ? owner + (int64_t)b * dm->C : NULL, dm->T, dm->C);
        if (status) status[b] = bad[b];
    }
    const int64_t total = (int64_t)B * R * Hq;
#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t it = 0; it < total; ++it) {
        int h = (int)(it % Hq);
        int r = (int)((it / Hq) % R);
        int b = (int)(it / ((int64_t)Hq * R));
        double* o = out + it * D;
        if (bad[b]) {
            for (int d = 0; d < D; ++d) o[d] = 0.0;
            if (lse) lse[it] = 0.0;
            continue;
        }
        attention_row(dm, q, kc, vc, seq_start, prefix_len, ks, vs, parent, owner, b, r, h, o, lse ? lse + it : NULL);
    }
    free(bad);
    return 0;
}

int confu_ref_tree_attention_rows(const confu_ref_dims* dm,
                                  const void* q, const void* kc, const void* vc,
                                  const int64_t* seq_start, const int32_t* prefix_len,
                                  const void* ks, const void* vs,
                                  const int32_t* parent, const int32_t* owner,
                                  int32_t n_sel, const int32_t* sel,
                                  double* out, double* lse)
{
    if (!attention_args_ok(dm) || n_sel < 0) return -1;
    const int R = dm->T + dm->C;
    for (int i = 0; i < n_sel; ++i) {
        int b = sel[3 * i], r = sel[3 * i + 1], h = sel[3 * i + 2];
        if (b < 0 || b >= dm->B || r < 0 || r >= R || h < 0 || h >= dm->Hq) return -1;
        if (check_tree(parent + (int64_t)b * dm->T, owner ? owner + (int64_t)b * dm->C : NULL, dm->T, dm->C)) return -1;
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int i = 0; i < n_sel; ++i)
        attention_row(dm, q, kc, vc, seq_start, prefix_len, ks, vs, parent, owner,
                      sel[3 * i], sel[3 * i + 1], sel[3 * i + 2],
                      out + (int64_t)i * dm->D, lse ? lse + i : NULL);
    return 0;
}

/* ------------------------------------------------------------------ */
/* acceptance                                                          */
/* ------------------------------------------------------------------ */

/* softmax(logits / temperature) of one row into dst[V]; returns 0 if a logit is non-finite */
static int softmax_row(const void* logits, int dtype, int64_t row, int V, double temperature, double* dst)
{
    double m = -INFINITY;
    int finite = 1;
    for (int v = 0; v < V; ++v) {
        double x = load_elem(logits, dtype, row * V + v);
        if (!isfinite(x)) finite = 0;
        dst[v] = x / temperature;
        if (dst[v] > m) m = dst[v];
    }
    if (!finite) return 0;
    double z = 0.0;
    for (int v = 0; v < V; ++v) { dst[v] = exp(dst[v] - m); z += dst[v]; }
    for (int v = 0; v < V; ++v) dst[v] /= z;
    return 1;
}

/* lowest index of the largest logit in one row; returns -1 if a logit is non-finite */
static int argmax_row(const void* logits, int dtype, int64_t row, int V)
{
    int best = 0;
    double bv = load_elem(logits, dtype, row * V);
    if (!isfinite(bv)) return -1;
    for (int v = 1; v < V; ++v) {
        double x = load_elem(logits, dtype, row * V + v);
        if (!isfinite(x)) return -1;
        if (x > bv) { bv = x; best = v; }
    }
    return best;
}

/*
 * Inverse CDF in index order on unnormalised weights: the smallest k whose
 * running sum exceeds u * total; if rounding leaves none, the largest k with
 * positive weight.  Also reports how close u came to an edge of the chosen cell
 * and the neighbouring positive-weight indices.
 */
static int inverse_cdf(const double* w, int V, double u, double* margin, int32_t* alt)
{
    double total = 0.0;
    for (int v = 0; v < V; ++v) total += w[v];
    const double target = u * total;
    double c = 0.0, lo = 0.0;
    int pick = -1;
    for (int v = 0; v < V; ++v) {
        lo = c;
        c += w[v];
        if (c > target) { pick = v; break; }
    }
    if (pick < 0) {
        for (int v = V - 1; v >= 0; --v) if (w[v] > 0.0) { pick = v; break; }
        if (pick < 0) pick = 0;
        lo = total - w[pick];
        c = total;
    }
    if (margin) {
        double dlo = u - lo / total, dhi = c / total - u;
        *margin = fabs(dlo) < fabs(dhi) ? fabs(dlo) : fabs(dhi);
    }
    if (alt) {
        alt[0] = alt[1] = -1;
        for (int v = pick - 1; v >= 0; --v) if (w[v] > 0.0) { alt[0] = v; break; }
        for (int v = pick + 1; v < V; ++v) if (w[v] > 0.0) { alt[1] = v; break; }
    }
    return pick;
}

static int future_row_of(const int32_t* parent, const int32_t* owner, int T, int C, int node)
{
    /* contemplate row of the last accepted node; if it has none, of its nearest ancestor that has */
    for (int a = node; a >= 0; a = parent[a])
        for (int k = 0; k < C; ++k)
            if (owner[k] == a) return T + k;
    return -1;
}

static void null_outputs(int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row)
{
    *accept_len = 0;
    path[0] = 0;
    for (int i = 1; i <= CONFU_REF_MAX_DEPTH; ++i) path[i] = -1;
    *next_token = -1;
    if (future_row) *future_row = -1;
}

static int accept_one(int T, int C, int V, int dtype,
                      const void* tl, const void* dl, int64_t row0,
                      const int32_t* tokens, const int32_t* parent, const int32_t* owner,
                      const double* uni, double temperature, int sibling_mode,
                      int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row,
                      int32_t* counters, double* ratio_margin, double* resample_margin, int32_t* alt_token)
{
    int32_t cnt[4] = {0, 0, 0, 0};
    double rmargin = INFINITY, smargin = INFINITY;
    int32_t alt[2] = {-1, -1};
    int st = CONFU_REF_ST_OK;
    int cur = 0, len = 0;
    /* statistics on demand: only the rows the walk needs are looked at (and checked) */
    const int lazy = (sibling_mode & CONFU_REF_ACCEPT_LAZY) != 0;
    sibling_mode &= ~CONFU_REF_ACCEPT_LAZY;

    null_outputs(accept_len, path, next_token, future_row);

    st = check_tree(parent, owner, T, C);
    if (!st)
        for (int i = 0; i < T; ++i)
            if (tokens[i] < 0 || tokens[i] >= V) { st = CONFU_REF_ST_BAD_TOKEN; break; }
    if (!st && temperature > 0.0 && sibling_mode == 1)
        for (int i = 1; i < T && !st; ++i)
            for (int j = i + 1; j < T; ++j)
                if (parent[i] == parent[j] && tokens[i] == tokens[j]) { st = CONFU_REF_ST_DUP_SIBLING; break; }
    if (!st && !lazy) {
        /* a non-finite logit anywhere in the rows the step is defined on is an input error */
        for (int i = 0; i < T && !st; ++i)
            for (int v = 0; v < V; ++v) {
                if (!isfinite(load_elem(tl, dtype, (row0 + i) * V + v))) { st = CONFU_REF_ST_NONFINITE; break; }
                if (temperature > 0.0 && !isfinite(load_elem(dl, dtype, (row0 + i) * V + v))) { st = CONFU_REF_ST_NONFINITE; break; }
            }
    }
    if (st) goto done;

    path[0] = 0;

    if (temperature <= 0.0) {
        /* greedy: a node is kept iff every edge on its root path carries the target's argmax
         * (ties: lowest token id); take the deepest kept node (ties: lowest node id). */
        int* keep = (int*)calloc((size_t)T, sizeof(int));
        int* depth = (int*)calloc((size_t)T, sizeof(int));
        int* amax = (int*)malloc((size_t)T * sizeof(int));
        for (int i = 0; i < T; ++i) amax[i] = -2;
        keep[0] = 1;
        int best = 0;
        for (int i = 1; i < T; ++i) {
            int pa = parent[i];
            depth[i] = depth[pa] + 1;
            if (!keep[pa]) continue;
            if (amax[pa] == -2) amax[pa] = argmax_row(tl, dtype, row0 + pa, V);
            if (amax[pa] == -1) { st = CONFU_REF_ST_NONFINITE; break; }
            keep[i] = (tokens[i] == amax[pa]);
            if (keep[i] && depth[i] > depth[best]) best = i;
        }
        len = depth[best];
        if (!st && len > CONFU_REF_MAX_DEPTH) st = CONFU_REF_ST_TOO_DEEP;
        if (!st) {
            for (int a = best, k = len; a >= 0; a = parent[a], --k) path[k] = a;
            cur = best;
            *next_token = argmax_row(tl, dtype, row0 + cur, V);
            if (*next_token < 0) st = CONFU_REF_ST_NONFINITE;
        }
        free(keep); free(depth); free(amax);
        if (st) { null_outputs(accept_len, path, next_token, future_row); goto done; }
    } else {
        double* p = (double*)malloc((size_t)V * sizeof(double));
        double* qd = (double*)malloc((size_t)V * sizeof(double));
        double* p_cur = (double*)malloc((size_t)V * sizeof(double));
        for (;;) {
            /* (with the check of all rows up front these two cannot fail) */
            if (!softmax_row(dl, dtype, row0 + cur, V, temperature, qd) ||
                !softmax_row(tl, dtype, row0 + cur, V, temperature, p_cur)) { st = CONFU_REF_ST_NONFINITE; break; }
            /* children of cur in increasing node index */
            int n_child = 0;
            for (int i = cur + 1; i < T; ++i) if (parent[i] == cur) ++n_child;
            if (n_child == 0) {            /* leaf: bonus token from the untouched target row */
                *next_token = inverse_cdf(p_cur, V, uni[0], &smargin, alt);
                break;
            }
            memcpy(p, p_cur, (size_t)V * sizeof(double));
            int accepted = -1, q_alive = 1;
            for (int c = cur + 1; c < T && q_alive; ++c) {
                if (parent[c] != cur) continue;
                const int x = tokens[c];
                const double u = uni[c];
                double ratio;
                if (qd[x] == 0.0) ratio = p[x] > 0.0 ? INFINITY : 0.0;
                else ratio = p[x] / qd[x];
                ++cnt[0];
                double mg = fabs(ratio - u);
                if (mg < rmargin) rmargin = mg;
                if (mg < 1e-5) ++cnt[2];
                if (u < ratio) { accepted = c; break; }
                /* rejected: residual  p <- norm(max(p - q, 0)) */
                ++cnt[1];
                double z = 0.0;
                for (int v = 0; v < V; ++v) { double d = p[v] - qd[v]; p[v] = d > 0.0 ? d : 0.0; z += p[v]; }
                if (z > 0.0) { for (int v = 0; v < V; ++v) p[v] /= z; }
                else { memcpy(p, p_cur, (size_t)V * sizeof(double)); st = CONFU_REF_ST_DEGENERATE; }
                if (sibling_mode == 1) {  /* drawn without replacement: drop x from q */
                    qd[x] = 0.0;
                    double zq = 0.0;
                    for (int v = 0; v < V; ++v) zq += qd[v];
                    if (zq > 0.0) { for (int v = 0; v < V; ++v) qd[v] /= zq; }
                    else q_alive = 0;
                }
            }
            if (accepted >= 0) {
                if (len + 1 > CONFU_REF_MAX_DEPTH) { st = CONFU_REF_ST_TOO_DEEP; break; }
                path[++len] = accepted;
                cur = accepted;
                continue;
            }
            *next_token = inverse_cdf(p, V, uni[0], &smargin, alt);
            break;
        }
        free(p); free(qd); free(p_cur);
        if (st == CONFU_REF_ST_TOO_DEEP || st == CONFU_REF_ST_NONFINITE) {      /* an error leaves no partial result */
            null_outputs(accept_len, path, next_token, future_row);
            memset(cnt, 0, sizeof cnt);
            goto done;
        }
        if (smargin < 1e-5) ++cnt[3];
    }
    *accept_len = len;
    if (future_row) *future_row = future_row_of(parent, owner, T, C, cur);

done:
    if (counters) memcpy(counters, cnt, sizeof cnt);
    if (ratio_margin) *ratio_margin = rmargin;
    if (resample_margin) *resample_margin = smargin;
    if (alt_token) { alt_token[0] = alt[0]; alt_token[1] = alt[1]; }
    return st;
}

int confu_ref_tree_accept(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                          const void* tl, const void* dl,
                          const int32_t* tokens, const int32_t* parent, const int32_t* owner,
                          const double* uniforms, double temperature, int32_t sibling_mode,
                          int32_t* accept_len, int32_t* path, int32_t* next_token,
                          int32_t* future_row, int32_t* counters,
                          double* ratio_margin, double* resample_margin, int32_t* alt_token,
                          int32_t* status)
{
    if (B < 0 || T <= 0 || C < 0 || V <= 0) return -1;
    if (logit_dtype < CONFU_REF_BF16 || logit_dtype > CONFU_REF_F64) return -1;
    if (!tl || !tokens || !parent || !accept_len || !path || !next_token) return -1;
    if (temperature > 0.0 && (!dl || !uniforms)) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int st = accept_one(T, C, V, logit_dtype, tl, dl, (int64_t)b * T,
                            tokens + (int64_t)b * T, parent + (int64_t)b * T,
                            owner ? owner + (int64_t)b * C : NULL,
                            uniforms ? uniforms + (int64_t)b * T : NULL, temperature, sibling_mode,
                            accept_len + b, path + (int64_t)b * (CONFU_REF_MAX_DEPTH + 1), next_token + b,
                            future_row ? future_row + b : NULL,
                            counters ? counters + 4 * (int64_t)b : NULL,
                            ratio_margin ? ratio_margin + b : NULL,
                            resample_margin ? resample_margin + b : NULL,
                            alt_token ? alt_token + 2 * (int64_t)b : NULL);
        if (status) status[b] = st;
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* acceptance, sample-and-match rule                                   */
/* ------------------------------------------------------------------ */
static int match_one(int T, int C, int V, int dtype, const void* tl, int64_t row0,
                     const int32_t* tokens, const int32_t* parent, const int32_t* owner,
                     const double* uni, double temperature,
                     int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row,
                     int32_t* counters, double* draw_margin, int32_t* alt_token)
{
    int32_t cnt[4] = {0, 0, 0, 0};
    double margin = INFINITY;
    int32_t alt[2] = {-1, -1};
    int cur = 0, len = 0;
    double* p = NULL;

    null_outputs(accept_len, path, next_token, future_row);
    int st = check_tree(parent, owner, T, C);
    if (!st)
        for (int i = 0; i < T; ++i)
            if (tokens[i] < 0 || tokens[i] >= V) { st = CONFU_REF_ST_BAD_TOKEN; break; }
    if (st) goto done;

    if (temperature > 0.0) p = (double*)malloc((size_t)V * sizeof(double));
    for (;;) {
        /* the token the target model itself emits after node cur */
        int x;
        if (temperature > 0.0) {
            if (!softmax_row(tl, dtype, row0 + cur, V, temperature, p)) { st = CONFU_REF_ST_NONFINITE; break; }
            double mg;
            x = inverse_cdf(p, V, uni[cur], &mg, alt);
            if (mg < margin) margin = mg;
            if (mg < 1e-5) ++cnt[2];
        } else {
            x = argmax_row(tl, dtype, row0 + cur, V);
            if (x < 0) { st = CONFU_REF_ST_NONFINITE; break; }
        }
        ++cnt[0];
        /* the draft token that matches it, if any (lowest node index) */
        int hit = -1;
        for (int c = cur + 1; c < T; ++c)
            if (parent[c] == cur && tokens[c] == x) { hit = c; break; }
        if (hit < 0) { *next_token = x; break; }
        if (len + 1 > CONFU_REF_MAX_DEPTH) { st = CONFU_REF_ST_TOO_DEEP; break; }
        path[++len] = hit;
        cur = hit;
        ++cnt[1];
    }
    free(p);
    if (st) { null_outputs(accept_len, path, next_token, future_row); memset(cnt, 0, sizeof cnt); goto done; }
    *accept_len = len;
    if (future_row) *future_row = future_row_of(parent, owner, T, C, cur);

done:
    if (counters) memcpy(counters, cnt, sizeof cnt);
    if (draw_margin) *draw_margin = margin;
    if (alt_token) { alt_token[0] = alt[0]; alt_token[1] = alt[1]; }
    return st;
}

int confu_ref_tree_accept_match(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                                const void* tl, const int32_t* tokens, const int32_t* parent,
                                const int32_t* owner, const double* uniforms, double temperature,
                                int32_t* accept_len, int32_t* path, int32_t* next_token,
                                int32_t* future_row, int32_t* counters, double* draw_margin,
                                int32_t* alt_token, int32_t* status)
{
    if (B < 0 || T <= 0 || C < 0 || V <= 0) return -1;
    if (logit_dtype < CONFU_REF_BF16 || logit_dtype > CONFU_REF_F64) return -1;
    if (!tl || !tokens || !parent || !accept_len || !path || !next_token) return -1;
    if (temperature > 0.0 && !uniforms) return -1;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int st = match_one(T, C, V, logit_dtype, tl, (int64_t)b * T, tokens + (int64_t)b * T,
                           parent + (int64_t)b * T, owner ? owner + (int64_t)b * C : NULL,
                           uniforms ? uniforms + (int64_t)b * T : NULL, temperature,
                           accept_len + b, path + (int64_t)b * (CONFU_REF_MAX_DEPTH + 1), next_token + b,
                           future_row ? future_row + b : NULL, counters ? counters + 4 * (int64_t)b : NULL,
                           draw_margin ? draw_margin + b : NULL, alt_token ? alt_token + 2 * (int64_t)b : NULL);
        if (status) status[b] = st;
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* 8-bit floating point cache entries (E4M3)                           */
/* ------------------------------------------------------------------ */
/*
 * E4M3 as the OCP 8-bit floating point specification defines it: 1 sign bit, 4 exponent bits (bias
 * 7), 3 mantissa bits; exponent 0 is subnormal (mantissa * 2^-9); there are no infinities; S.1111.111
 * is NaN; the largest magnitude is S.1111.110 = 448.
 */
static double e4m3_value(uint8_t c)
{
    const int sign = c >> 7, e = (c >> 3) & 15, m = c & 7;
    double v;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) v = ldexp((double)m, -9);
    else v = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -v : v;
}

int confu_ref_e4m3_decode(const uint8_t* src, int64_t n, double* dst)
{
    if (!src || !dst || n < 0) return -1;
    for (int64_t i = 0; i < n; ++i) dst[i] = e4m3_value(src[i]);
    return 0;
}

/*
 * The quantisation a cache entry goes through when it is written: x / scale in SINGLE precision (the
 * precision the decision is taken in on the device too), rounded to the nearest E4M3 value, ties to
 * the value with an even mantissa, magnitudes beyond 448 saturating to 448; NaN stays NaN.
 * Written as a search over the 127 non-negative finite codes: no bit tricks to get wrong.
 */
static uint8_t e4m3_code(float y)
{
    if (isnan(y)) return 0x7f;
    const uint8_t sign = signbit(y) ? 0x80 : 0x00;
    const double a = fabs((double)y);
    if (a >= 448.0) return (uint8_t)(sign | 0x7e);
    uint8_t best = 0;
    double best_d = INFINITY;
    for (int c = 0; c <= 0x7e; ++c) {
        const double d = fabs(e4m3_value((uint8_t)c) - a);
        /* codes ascend with their values: of two equally near neighbours the even code is the one with the even mantissa */
        if (d < best_d || (d == best_d && (c & 1) == 0)) { best_d = d; best = (uint8_t)c; }
    }
    return (uint8_t)(sign | best);
}

int confu_ref_e4m3_encode(const float* src, float scale, int64_t n, uint8_t* dst)
{
    if (!src || !dst || n < 0 || !(scale > 0.0f)) return -1;
    for (int64_t i = 0; i < n; ++i) dst[i] = e4m3_code(src[i] / scale);
    return 0;
}

/* ------------------------------------------------------------------ */
/* compaction                                                          */
/* ------------------------------------------------------------------ */
int confu_ref_kv_compact(int32_t B, int32_t n_layers, int64_t row_bytes,
                         void* const* k_layers, void* const* v_layers,
                         const int64_t* seq_start, const int32_t* prefix_len,
                         const int32_t* accept_len, const int32_t* path,
                         int32_t* new_prefix_len)
{
    if (B < 0 || n_layers < 0 || row_bytes <= 0) return -1;
    for (int b = 0; b < B; ++b) {
        const int a = accept_len[b];
        if (a < 0 || a > CONFU_REF_MAX_DEPTH) return -1;
        const int32_t* pth = path + (int64_t)b * (CONFU_REF_MAX_DEPTH + 1);
        const int64_t root = seq_start[b] + prefix_len[b];
        if (a > 0) {
            char* old = (char*)malloc((size_t)a * (size_t)row_bytes);
            for (int l = 0; l < n_layers; ++l)
                for (int kv = 0; kv < 2; ++kv) {
                    char* pool = (char*)(kv ? v_layers[l] : k_layers[l]);
                    /* snapshot every source row first: "old" means the cache before the call */
                    for (int k = 1; k <= a; ++k)
                        memcpy(old + (size_t)(k - 1) * row_bytes, pool + (root + pth[k]) * row_bytes, (size_t)row_bytes);
                    for (int k = 1; k <= a; ++k)
                        memcpy(pool + (root + k) * row_bytes, old + (size_t)(k - 1) * row_bytes, (size_t)row_bytes);
                }
            free(old);
        }
        if (new_prefix_len) new_prefix_len[b] = prefix_len[b] + a + 1;
    }
    return 0;
}

/* ------------------------------------------------------------------ */
/* contemplate-token embedding: mixture of expert embeddings           */
/* ------------------------------------------------------------------ */
int confu_ref_con_embedding(int32_t B, int32_t H_in, int32_t H_out, int32_t n_expert, int32_t k_expert,
                            int32_t dtype, const void* hidden, const void* router_w, const void* router_b,
                            const void* experts, int32_t renormalize,
                            double* out, int32_t* sel, double* gate, double* gap)
{
    if (B < 0 || H_in <= 0 || H_out <= 0 || n_expert <= 0 || k_expert <= 0 || k_expert > n_expert) return -1;
    if (dtype < CONFU_REF_BF16 || dtype > CONFU_REF_F64) return -1;
    if (!hidden || !router_w || !experts || !out) return -1;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        double* score = (double*)malloc((size_t)n_expert * sizeof(double));
        int* taken = (int*)calloc((size_t)n_expert, sizeof(int));
        /* router: a linear layer on the hidden state, then a softmax over the experts */
        double m = -INFINITY;
        for (int e = 0; e < n_expert; ++e) {
            double a = router_b ? load_elem(router_b, dtype, e) : 0.0;
            for (int i = 0; i < H_in; ++i)
                a += load_elem(router_w, dtype, (int64_t)e * H_in + i) * load_elem(hidden, dtype, (int64_t)b * H_in + i);
            score[e] = a;
            if (a > m) m = a;
        }
        double z = 0.0;
        for (int e = 0; e < n_expert; ++e) { score[e] = exp(score[e] - m); z += score[e]; }
        for (int e = 0; e < n_expert; ++e) score[e] /= z;
        /* the k_expert largest scores, largest first, the lower index on equal scores */
        double wsum = 0.0, kth = 0.0;
        for (int j = 0; j < H_out; ++j) out[(int64_t)b * H_out + j] = 0.0;
        int* pick = (int*)malloc((size_t)k_expert * sizeof(int));
        for (int k = 0; k < k_expert; ++k) {
            int best = -1;
            for (int e = 0; e < n_expert; ++e)
                if (!taken[e] && (best < 0 || score[e] > score[best])) best = e;
            taken[best] = 1;
            pick[k] = best;
            wsum += score[best];
            kth = score[best];
        }
        double next = -INFINITY;
        for (int e = 0; e < n_expert; ++e) if (!taken[e] && score[e] > next) next = score[e];
        /* weighted sum of the chosen experts' embeddings, weights = their gating scores */
        for (int k = 0; k < k_expert; ++k) {
            const double w = renormalize ? score[pick[k]] / wsum : score[pick[k]];
            if (sel) sel[(int64_t)b * k_expert + k] = pick[k];
            if (gate) gate[(int64_t)b * k_expert + k] = w;
            for (int j = 0; j < H_out; ++j)
                out[(int64_t)b * H_out + j] += w * load_elem(experts, dtype, (int64_t)pick[k] * H_out + j);
        }
        if (gap) gap[b] = k_expert < n_expert ? kth - next : INFINITY;
        free(score); free(taken); free(pick);
    }
    return 0;
}
