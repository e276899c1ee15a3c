/*
 * confu_ref.h -- fp64 CPU oracle for the ConFu tree-verification step.
 *
 * TEST INFRASTRUCTURE ONLY.  This code is the slow, plain, obviously-correct
 * statement of what the verification step computes.  It is used by the tests,
 * by the smoke check and by the benchmark's CPU-baseline leg; the product path
 * never calls it.  It shares no code, header, table or helper with the CUDA
 * library (the numeric values of the status codes are an interface and are
 * simply kept equal).
 *
 * Pins (tests marked "not gpu"): brute-force dense-mask attention, chain tree ==
 * causal attention (library SDPA), all-zero keys == mean of visible values,
 * identical draft/target == always accept, hand-computed two-token cases,
 * textbook linear speculative sampling on a chain, exact-rational resampling,
 * and a chi-square test of the emitted-token marginal against the target
 * distribution (with a power check on a deliberately broken variant).  The
 * closeness records of the acceptance walks (ratio_margin, resample_margin,
 * draw_margin, alt_token and the two "within 1e-5" counters) are pinned by
 * hand-computed cases, by cases planted inside and just outside the 1e-5 band,
 * and by exact-rational walks.  The E4M3 decode is pinned against a library conversion of all 256
 * codes and against hand-written values; the encode against the library conversion on random
 * values, hand-written ties, the saturation bound and the subnormal range.
 * The whole verify step on synthetic inputs has no published numbers:
 * beyond those pins, end-to-end parity is unpinned.
 *
 * All arithmetic is IEEE double.  bf16 / fp32 inputs are widened exactly.
 * All pointers are HOST pointers.
 */
#ifndef CONFU_REF_H
#define CONFU_REF_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { CONFU_REF_BF16 = 0, CONFU_REF_F32 = 1, CONFU_REF_F64 = 2 };

/* per-sequence status values (0 = ok) */
enum {
    CONFU_REF_ST_OK = 0,
    CONFU_REF_ST_BAD_PARENT = 1,   /* parent[0] != -1 or parent[i] not in [0,i) */
    CONFU_REF_ST_BAD_OWNER = 2,    /* con_owner[k] not in [0,T) */
    CONFU_REF_ST_BAD_TOKEN = 3,    /* token id not in [0,V) */
    CONFU_REF_ST_DUP_SIBLING = 4,  /* two children of one node carry the same token (sibling_mode 1) */
    CONFU_REF_ST_NONFINITE = 5,    /* non-finite logit met */
    CONFU_REF_ST_DEGENERATE = 7,   /* residual had zero mass; fell back to the target row */
    CONFU_REF_ST_TOO_DEEP = 8      /* accepted path longer than the path buffer */
};

#define CONFU_REF_MAX_DEPTH 63     /* path holds CONFU_REF_MAX_DEPTH + 1 node ids */
#define CONFU_REF_ACCEPT_LAZY 0x100

typedef struct {
    int32_t B, Hq, Hkv, D, T, C, S;
    int32_t dtype;      /* CONFU_REF_* : element type of q, k_cache, v_cache, k_soft, v_soft */
    double  sm_scale;   /* 0 -> D^-1/2 */
} confu_ref_dims;

/*
 * Tree-masked attention of one layer (tree attention with one mask row per
 * draft node, Sec. 2 "tree of candidate tokens"; contemplate rows and
 * soft-prompt keys, Sec. 3.1 and Fig. 3).
 *
 * Rows 0..T-1 are tree nodes (node 0 the root), rows T..T+C-1 contemplate rows.
 * The cache pool of this layer is [n_slots][Hkv][D]; sequence b owns slots
 * seq_start[b] .. seq_start[b]+prefix_len[b]+R-1: first its prefix, then the
 * keys/values of the R query rows themselves.
 * Row r sees: every prefix slot; tree slot j iff j is r itself or an ancestor of
 * r (for a contemplate row: itself, its owner, the owner's ancestors); the S
 * soft-prompt entries iff r is a contemplate row.
 * out[b][r][h][:] = sum_j softmax_j(scale * q.k_j) v_j over that set, lse the
 * log of the softmax denominator (natural log, scaled scores).
 * out: [B][R][Hq][D] doubles; lse: [B][R][Hq] doubles (may be NULL).
 * status: [B] int32 (may be NULL).  Returns 0, or -1 on a bad argument.
 */
int confu_ref_tree_attention(const confu_ref_dims* dims,
                             const void* q, const void* k_cache, const void* v_cache,
                             const int64_t* seq_start, const int32_t* prefix_len,
                             const void* k_soft, const void* v_soft,
                             const int32_t* parent, const int32_t* con_owner,
                             double* out, double* lse, int32_t* status);

/* The same definition for a chosen list of (b, r, h) triples: sel is [n_sel][3],
 * out is [n_sel][D], lse is [n_sel]. */
int confu_ref_tree_attention_rows(const confu_ref_dims* dims,
                                  const void* q, const void* k_cache, const void* v_cache,
                                  const int64_t* seq_start, const int32_t* prefix_len,
                                  const void* k_soft, const void* v_soft,
                                  const int32_t* parent, const int32_t* con_owner,
                                  int32_t n_sel, const int32_t* sel,
                                  double* out, double* lse);

/*
 * Tree speculative-sampling acceptance (Sec. 2 steps 3-4: sequential accept /
 * reject, then a sample from the corrected distribution; tree variant of the
 * "Preliminaries" paragraph on token trees; choice of the future prediction of
 * the last accepted node, Sec. 3.1).
 *
 * target_logits / draft_logits: [B][T][V]; row i of the target is the
 * distribution of the token that follows node i; row i of the draft is the
 * distribution node i's children were drawn from.
 * tokens [B][T]; uniforms [B][T] doubles in [0,1): slot i>0 drives the test of
 * node i, slot 0 the final resample / bonus draw.
 * temperature 0 -> greedy.  sibling_mode 1: children drawn without replacement
 * (after a rejection the rejected token is removed from q and q renormalised);
 * 0: children i.i.d. (q unchanged).  A non-finite logit anywhere in the T rows
 * (target; draft too unless greedy) is an error -- unless CONFU_REF_ACCEPT_LAZY is
 * or-ed into sibling_mode: then only the rows the walk needs are looked at (both
 * rows of every visited node; greedy: the target row of every node whose children
 * are compared, and of the last node) and only they can raise that error.
 * Outputs per sequence: accept_len, path [CONFU_REF_MAX_DEPTH+1] (root first, -1
 * padded), next_token, future_row (in [T,T+C) or -1), counters [4] = {ratio
 * tests, rejections, ratio tests with |ratio-u| < 1e-5, resample draws within
 * 1e-5 of a CDF edge}, ratio_margin = min |ratio - u| over the tests made
 * (+inf if none), resample_margin = distance of u to the nearer edge of the
 * chosen token's normalised CDF cell, alt_token [2] = previous / next index of
 * non-zero weight around next_token (-1 if none).  Any output pointer other than
 * accept_len, path and next_token may be NULL.
 */
int confu_ref_tree_accept(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                          const void* target_logits, const void* draft_logits,
                          const int32_t* tokens, const int32_t* parent, const int32_t* con_owner,
                          const double* uniforms, double temperature, int32_t sibling_mode,
                          int32_t* accept_len, int32_t* path, int32_t* next_token,
                          int32_t* future_row, int32_t* counters,
                          double* ratio_margin, double* resample_margin, int32_t* alt_token,
                          int32_t* status);

/*
 * Acceptance by the sample-and-match rule, Sec. 2 steps 3-4 read literally: at the
 * current node (the root first) the target model's own next token x is drawn from
 * softmax(target_logits[node] / temperature) by inverse CDF in index order with
 * uniforms[b][node] (temperature 0: x = the lowest index of the largest logit); the
 * child of the node that carries x (lowest node index) is accepted and becomes the
 * current node; when no child carries x -- always so at a leaf -- the walk stops and
 * x itself is the next token (the replacement of the first rejected draft, or the
 * bonus token).  Only the target rows of the walked path are read: a non-finite
 * logit is an error only there.  No draft logits.
 * Outputs as for confu_ref_tree_accept, with counters [4] = {draws, accepted nodes,
 * draws within 1e-5 of a CDF edge, 0}, draw_margin = the smallest distance of a
 * uniform to an edge of its chosen CDF cell over all draws (+inf at temperature 0),
 * alt_token [2] = previous / next index of non-zero weight around the LAST draw.
 */
int confu_ref_tree_accept_match(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                                const void* target_logits, const int32_t* tokens,
                                const int32_t* parent, const int32_t* con_owner,
                                const double* uniforms, double temperature,
                                int32_t* accept_len, int32_t* path, int32_t* next_token,
                                int32_t* future_row, int32_t* counters, double* draw_margin,
                                int32_t* alt_token, int32_t* status);

/*
 * KV compaction of the accepted path ("the final accepted sequence becomes the
 * input for the next drafting step", Sec. 2 step 4).  For every layer and for K
 * and V: new[P_b + k] = old[P_b + path[b][k]], k = 1..accept_len[b], where "old"
 * is the cache before the call; slot P_b (the root) and the prefix stay as they
 * are; new_prefix_len[b] = P_b + accept_len[b] + 1.  Slots past the new prefix
 * are left with unspecified contents.  k_layers / v_layers: n_layers host
 * pointers to pools of row_bytes-sized slots.
 */
int confu_ref_kv_compact(int32_t B, int32_t n_layers, int64_t row_bytes,
                         void* const* k_layers, void* const* v_layers,
                         const int64_t* seq_start, const int32_t* prefix_len,
                         const int32_t* accept_len, const int32_t* path,
                         int32_t* new_prefix_len);

/*
 * Embedding of the contemplate token as a mixture of expert embeddings (Sec. 3.2,
 * "Dynamic Contemplate Tokens with MoE"): a linear layer maps the hidden state of
 * the most recently accepted token to one logit per expert (router_w
 * [n_expert][H_in], optional bias router_b [n_expert]), a softmax normalises them,
 * the k_expert experts with the largest scores are selected (the lower index on
 * equal scores) and the embedding is the sum of their embeddings (experts
 * [n_expert][H_out]) weighted by their gating scores -- the softmax values
 * themselves, or, with renormalize != 0, divided by their sum over the selection.
 * hidden [B][H_in]; out [B][H_out] doubles; optional: sel [B][k_expert] (largest
 * score first), gate [B][k_expert] (the weights used), gap [B] = score of the last
 * selected expert minus the largest score left out (+inf if none is left out).
 */
int confu_ref_con_embedding(int32_t B, int32_t H_in, int32_t H_out, int32_t n_expert, int32_t k_expert,
                            int32_t dtype, const void* hidden, const void* router_w, const void* router_b,
                            const void* experts, int32_t renormalize,
                            double* out, int32_t* sel, double* gate, double* gap);

/* number of OpenMP threads the oracle will use */
int confu_ref_num_threads(void);

/*
 * 8-bit floating point (E4M3) cache entries.  A cache that holds K and V as E4M3 bytes with one
 * fp32 scale per KV head stands for the values  decode(byte) * scale[head]  -- exactly: the
 * attention of such a cache is the definition above applied to those values (widened to double;
 * the product of a 4-bit significand and an fp32 scale is exact in double).  The paper has no cache
 * format; this is the 8-bit format serving engines use for KV caches.
 * decode: dst[i] = value of code src[i] (NaN for S.1111.111).
 * encode: dst[i] = nearest E4M3 code of src[i] / scale, the quotient taken in single precision,
 *         ties to the even mantissa, saturating at +-448; scale > 0.
 */
int confu_ref_e4m3_decode(const uint8_t* src, int64_t n, double* dst);
int confu_ref_e4m3_encode(const float* src, float scale, int64_t n, uint8_t* dst);

#ifdef __cplusplus
}
#endif
#endif
