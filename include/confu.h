/*
 * confu.h -- C ABI of the B200 (sm_100a) tree-verification library.
 *
 * The library implements the target model's verification step of ConFu-style
 * speculative decoding (ConFu, Sec. 2 "Preliminaries" steps 2-4 and the paragraph
 * on token trees; Sec. 3.1 "Capture Future with Contemplate Tokens", Fig. 3):
 *
 *   confu_tree_attention   tree-masked attention of the draft-tree rows and the
 *                          contemplate rows over prefix KV, soft-prompt KV and the
 *                          tree's own KV (one layer per call)
 *   confu_tree_accept      tree speculative-sampling acceptance over full-vocabulary
 *                          logits, residual resampling, accepted path, future row
 *   confu_kv_compact       keeps the accepted path's KV (all layers, one call)
 *
 * Conventions
 *   - every function returns an int: 0 = CONFU_OK, negative = an error detected on
 *     the host before anything was enqueued (see confu_status_string);
 *   - "device" pointers are CUDA device pointers of the context's device, "host"
 *     pointers are ordinary host memory; every device pointer must be 16-byte
 *     aligned; the caller owns every buffer it passes, for the whole time the
 *     enqueued work runs;
 *   - work is enqueued on the given stream (a cudaStream_t passed as void*); no call
 *     synchronises the host with the device and none allocates device memory; the
 *     context's device must be the current device of the calling thread;
 *   - data-dependent problems (a malformed tree, an out-of-range token, a
 *     non-finite logit, a bounded device-side wait that ran out) never trap: the
 *     kernels write a positive code into status[b] (int32, device, one per sequence).
 *     The library only ever writes non-zero codes there, so clear it before a step.
 *     A sequence with a non-zero status has unspecified outputs.
 *
 * Row and slot conventions
 *   T <= 64 tree rows (row 0 = root = the token emitted by the previous step), then
 *   C <= 64 contemplate rows; R = T + C <= 128.  parent[b][0] = -1 and 0 <= parent[b][i] < i.
 *   con_owner[b][k] in [0,T) is the tree node that contemplate row T+k sits behind.
 *   A layer's cache pool is [n_slots][Hkv][D]; sequence b owns slots
 *   seq_start[b] .. seq_start[b] + prefix_len[b] + R - 1: its prefix, then the K/V of
 *   its R query rows (written there by the caller before confu_tree_attention).
 *   Slots that belong to no sequence, or lie past a sequence's last row (pool padding, the
 *   unused tail of a page), are never interpreted: they may hold anything, NaN bit patterns
 *   included, and need not be initialised.
 */
#ifndef CONFU_H
#define CONFU_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct confu_ctx confu_ctx;

/* return codes (host side) */
enum {
    CONFU_OK = 0,
    CONFU_ERR_ARG = -1,          /* null pointer / negative size / bad enum */
    CONFU_ERR_SHAPE = -2,        /* Hq % Hkv != 0, D not in {64,128}, T < 1, ... */
    CONFU_ERR_ALIGN = -3,        /* a device pointer is not 16-byte aligned */
    CONFU_ERR_WORKSPACE = -4,    /* workspace missing or too small */
    CONFU_ERR_UNSUPPORTED = -5,  /* e.g. T > 64 or C > 64 */
    CONFU_ERR_CUDA = -6          /* a CUDA call failed: see confu_last_cuda_error */
};

/* per-sequence status codes written by the kernels (device side) */
enum {
    CONFU_ST_OK = 0,
    CONFU_ST_BAD_PARENT = 1,
    CONFU_ST_BAD_OWNER = 2,
    CONFU_ST_BAD_TOKEN = 3,
    CONFU_ST_DUP_SIBLING = 4,
    CONFU_ST_NONFINITE = 5,
    CONFU_ST_TIMEOUT = 6,        /* a bounded wait inside a kernel gave up */
    CONFU_ST_DEGENERATE = 7,     /* residual distribution had no mass; target row used instead */
    CONFU_ST_TOO_DEEP = 8,       /* accepted path longer than CONFU_MAX_DEPTH */
    CONFU_ST_BAD_PATH = 9,       /* confu_kv_compact: path is not 0 = path[0] < path[1] < ... < T, or accept_len out of range */
    CONFU_ST_BAD_PLAN = 10       /* confu_tree_attention: the plan was built for another attention path */
};

enum { CONFU_BF16 = 0, CONFU_F32 = 1, CONFU_FP8_E4M3 = 2 };   /* FP8: cache entries only, see confu_set_kv_scales */

#define CONFU_MAX_TREE  64      /* T: tree rows (one 64-bit ancestor word per row) */
#define CONFU_MAX_ROWS  128     /* R = T + C, with C <= 64: covers one contemplate row per node (R = 2T) */
#define CONFU_MAX_DEPTH 63      /* path buffers hold CONFU_MAX_DEPTH + 1 node ids */
#define CONFU_ACCEPT_LAZY 0x100 /* or-ed into sibling_mode: row statistics on demand (see confu_tree_accept) */

typedef struct {
    int32_t B;          /* sequences */
    int32_t Hq, Hkv;    /* query / KV heads, Hq % Hkv == 0 */
    int32_t D;          /* head dim: 64 or 128 */
    int32_t T, C;       /* tree rows (root included), contemplate rows */
    int32_t S;          /* soft-prompt KV entries, shared by all sequences (0 allowed) */
    int32_t kv_dtype;   /* CONFU_BF16 | CONFU_F32: type of q, caches, soft KV and out;
                           CONFU_FP8_E4M3: caches and soft KV are E4M3 bytes, q and out are bf16 */
    float   sm_scale;   /* 0 -> D^-1/2 */
} confu_dims;

/* ---- context ------------------------------------------------------------ */

/* Creates a context for a CUDA device (host state only: the SM count, the workspace and
 * paging settings, the last CUDA error).  confu_destroy frees it.  A context is not thread safe. */
int confu_create(confu_ctx** ctx, int device);
int confu_destroy(confu_ctx* ctx);

/* Device scratch the attention call needs for these dims (split-KV partial results,
 * the work plan, the ancestor masks); a pure function of dims and of the device's
 * SM count.  The caller allocates it and hands it over; it may be shared by all
 * layers of a step but not by calls that run concurrently. */
size_t confu_workspace_bytes(const confu_ctx* ctx, const confu_dims* dims);
int confu_set_workspace(confu_ctx* ctx, void* device_ptr, size_t bytes);

/*
 * Paged pools.  With a block table set, every layer's cache pool is read as pages of 128 slots:
 * slot s of sequence b (s = 0 is its first prefix token; the R query rows follow the prefix) lives
 * in page block_table[b][s / 128] at offset s % 128, i.e. at pool slot 128 * page + s % 128.
 * block_table: DEVICE int32 [B][max_pages], with at least ceil((prefix_len[b] + R) / 128) valid
 * page ids per sequence; read by every later call until it is cleared (NULL); seq_start is then
 * ignored and may be NULL, and n_slots must be a whole number of pages.  Page ids are the caller's: an id
 * past the pool reads as zeros in confu_tree_attention (the tile loads are bounds-checked by the hardware) but is an
 * out-of-bounds store in confu_kv_append and confu_kv_compact, which do not know the pool's size.  The paper has no cache
 * layout (Sec. 3.1 only says the K/V of accepted tokens are kept); pages of one key tile are what
 * serving engines use.
 */
int confu_set_paging(confu_ctx* ctx, const int32_t* block_table, int32_t max_pages);

/*
 * Options of a context (host state; they apply to the calls made after the setting).
 *   CONFU_OPT_ATTENTION_PATH  which kernel confu_tree_plan prepares for and confu_tree_attention
 *                             launches: CONFU_ATTENTION_AUTO (default: the fastest path that
 *                             supports the dims), _GENERIC (CUDA cores, every dtype and shape),
 *                             _TENSOR (tcgen05, one CTA per SM; bf16, D = 128, Hq/Hkv <= 4),
 *                             _TENSOR_PAIR (tcgen05 two-SM instructions, one CTA pair per two SMs;
 *                             as _TENSOR, and more than 32 query rows).  A path that does not
 *                             support the dims makes the calls return CONFU_ERR_UNSUPPORTED.  Set
 *                             it before confu_tree_plan: a plan only fits the path it was built
 *                             for (status CONFU_ST_BAD_PLAN otherwise).
 *   CONFU_OPT_WAIT_LIMIT_NS   wall-clock limit of every wait on a barrier inside the tensor-core
 *                             kernels (default 2 s; 1 us .. 10 s).  A wait that runs out makes the
 *                             kernel release what it holds and report CONFU_ST_TIMEOUT.
 */
enum { CONFU_OPT_ATTENTION_PATH = 1, CONFU_OPT_WAIT_LIMIT_NS = 2 };
enum { CONFU_ATTENTION_AUTO = 0, CONFU_ATTENTION_GENERIC = 1, CONFU_ATTENTION_TENSOR = 2, CONFU_ATTENTION_TENSOR_PAIR = 3 };
int confu_set_option(confu_ctx* ctx, int32_t option, int64_t value);

/*
 * The CONFU_ATTENTION_* path (never _AUTO) that confu_tree_plan and confu_tree_attention take for
 * these dims under the context's current options, or a negative CONFU_ERR_* code where they would
 * return it.  Host state only.
 */
int confu_attention_path(const confu_ctx* ctx, const confu_dims* dims);

/*
 * Self-test of the bounded device-side wait (no counterpart in the paper): one warp waits, through
 * the same routine the attention kernels use, on a barrier that nothing arrives at; after limit_ns
 * (1 us .. 1 s) of wall clock the wait gives up and the kernel writes CONFU_ST_TIMEOUT to status[0]
 * (device int32) and returns.  The context stays usable.
 */
int confu_selftest_bounded_wait(confu_ctx* ctx, int64_t limit_ns, int32_t* status, void* stream);

/*
 * 8-bit floating point caches (kv_dtype = CONFU_FP8_E4M3; the paper has no cache format: this is
 * the 8-bit KV cache of serving engines, a bandwidth and tensor-rate lever for the verification
 * forward of Sec. 3.1).  A cache entry is an E4M3 byte (OCP 8-bit floating point: 1-4-3, bias 7, no
 * infinities, largest magnitude 448) and stands for  code * scale[kv head] : k_scale, v_scale are
 * DEVICE fp32 arrays of Hkv entries, read by every later call of this context until they are set
 * again (set them per layer if the layers have scales of their own); the soft-prompt K/V use the
 * same scales.  With these dims
 *   - confu_tree_attention computes the attention of the values the cache stands for; q and out are
 *     bf16; inside, Q (per row) and the softmax weights are rounded to E4M3 for the tensor cores
 *     (kind::f8f6f4), accumulation is fp32 -- see the tolerance in the tests.  D = 128, Hq/Hkv <= 4,
 *     S <= 128; CONFU_ERR_UNSUPPORTED otherwise, or without scales;
 *   - confu_kv_append takes bf16 rows and stores  e4m3(row / scale)  (quotient in fp32, round to
 *     nearest even, saturating at 448);
 *   - confu_kv_compact moves bytes as for any other type.
 */
int confu_set_kv_scales(confu_ctx* ctx, const float* k_scale, const float* v_scale);

const char* confu_status_string(int code);      /* host return codes and device status codes */
const char* confu_last_cuda_error(const confu_ctx* ctx);

/* ---- tree attention (Sec. 2, token trees; Sec. 3.1 and Fig. 3) ----------- */

/* Bytes of a caller-held plan buffer for confu_tree_plan. */
size_t confu_plan_bytes(const confu_ctx* ctx, const confu_dims* dims);

/*
 * Builds what every layer of one step shares: the ancestor bitmask of each row
 * (a tree row sees itself and its ancestors; a contemplate row sees itself, its
 * owner and the owner's ancestors; only contemplate rows see the soft prompts)
 * and the balanced split-KV work list for this batch's prefix lengths.  Validates
 * the trees (status codes 1, 2).  All pointers device.  plan: confu_plan_bytes().
 */
int confu_tree_plan(confu_ctx* ctx, const confu_dims* dims,
                    const int64_t* seq_start, const int32_t* prefix_len,
                    const int32_t* parent,      /* [B][T] */
                    const int32_t* con_owner,   /* [B][C], may be NULL if C == 0 */
                    void* plan, int32_t* status, void* stream);

/*
 * One layer of tree-masked attention.
 *   out[b][r][h][:] = sum_j softmax_j(sm_scale * q[b][r][h] . k_j) v_j   over the keys row r sees:
 *   all prefix slots of sequence b, the tree slots its mask allows, and (contemplate
 *   rows only) the S soft-prompt entries.  KV head of query head h is h / (Hq/Hkv).
 * q, out: [B][R][Hq][D]; k_cache, v_cache: [n_slots][Hkv][D]; k_soft, v_soft:
 * [S][Hkv][D] (NULL if S == 0); lse: optional [B][R][Hq] fp32 natural-log softmax
 * denominators.  plan: a buffer filled by confu_tree_plan for these dims, lengths
 * and trees, or NULL to have the call build one in the workspace (then parent,
 * con_owner are read; otherwise they may be NULL).  Accumulation is fp32; bf16
 * inputs use the tensor-core path when D == 128 and Hq/Hkv <= 4; it takes the
 * query rows in groups of 64, so R > 64 streams the keys twice (the two groups walk
 * the same keys at the same time: the second read is served by L2).
 * Needs the workspace.  All pointers device.  Ordinary stream order holds: the kernels are
 * launched as programmatic dependents (their blocks may be scheduled while the kernel before them
 * drains) but wait for all earlier work of the stream before their first global memory access,
 * and whatever is enqueued after the call sees completed results.  A sequence with a malformed tree
 * (status 1 or 2) gets all-zero output rows and lse 0.  The call may be captured
 * into a CUDA graph (no allocation, no synchronisation; call it once outside the capture first).
 */
int confu_tree_attention(confu_ctx* ctx, const confu_dims* dims,
                         const void* q, const void* k_cache, const void* v_cache, int64_t n_slots,
                         const int64_t* seq_start, const int32_t* prefix_len,
                         const void* k_soft, const void* v_soft,
                         const int32_t* parent, const int32_t* con_owner,
                         const void* plan,
                         void* out, float* lse, int32_t* status, void* stream);

/* ---- acceptance (Sec. 2 steps 3-4; Sec. 3.1 "future prediction associated with the
 *      last accepted token") ------------------------------------------------ */

/* Device scratch for confu_tree_accept (row statistics). */
size_t confu_accept_workspace_bytes(int32_t B, int32_t T, int32_t V);

/*
 * target_logits, draft_logits: [B][T][V] (bf16 or fp32).  Row i of the target is
 * the distribution of the token after node i; row i of the draft is the one node
 * i's children were drawn from.  p = softmax(target / temperature), q likewise.
 * Walk from the root: test the children of the current node in increasing node
 * index with  u < p(x)/q(x)  (u = uniforms[b][child], x = tokens[b][child]); the
 * first success is accepted and becomes the current node; a failure replaces p by
 * norm(max(p - q, 0)) and, with sibling_mode 1 (children drawn without
 * replacement), removes x from q and renormalises (sibling_mode 0: q unchanged).
 * When no child is left the next token is drawn from the current p by inverse CDF
 * in index order with uniforms[b][0]; at a leaf it is drawn from the leaf's target
 * row.  temperature 0: greedy (accept a child iff its token is the argmax of its
 * parent's target row, lowest index on ties; deepest such path, lowest node index on
 * ties; next token = argmax of the last node's row; draft_logits, uniforms unused).
 * Outputs (device): accept_len [B] (accepted drafts, root excluded); path
 * [B][CONFU_MAX_DEPTH+1] node ids root first, -1 padded; next_token [B];
 * future_row [B] = row index in [T,T+C) of the contemplate row owned by the last
 * accepted node, else by its nearest ancestor that has one, else -1; counters
 * (optional) [B][4] = ratio tests made, rejections, ratio tests with |p(x)/q(x) - u| < 1e-5,
 * final draws (0 or 1) whose uniform lies within 1e-5 of an edge of the emitted token's cell
 * of the normalised CDF.  The last two count the decisions that rounding could turn: an
 * implementation in other arithmetic may legitimately differ there (greedy: always 0).
 * workspace: confu_accept_workspace_bytes().  All pointers device.
 * By default one streaming pass takes the softmax statistics of all T rows of both matrices
 * first, and a non-finite logit anywhere in them is an error (status 5).  With
 * sibling_mode | CONFU_ACCEPT_LAZY the statistics of a row are computed when the walk reaches its
 * node: only the rows of the walked path are read (two per visited node; greedy: the target row
 * of every node whose children are compared), a non-finite logit is an error only there, and the
 * workspace is not used (it may be NULL).  Decisions are the same up to rounding of the normalisers.
 */
int confu_tree_accept(confu_ctx* ctx, int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                      const void* target_logits, const void* draft_logits,
                      const int32_t* tokens, const int32_t* parent, const int32_t* con_owner,
                      const float* uniforms, float temperature, int32_t sibling_mode,
                      int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row,
                      int32_t* counters, void* workspace, size_t workspace_bytes,
                      int32_t* status, void* stream);

/*
 * confu_tree_accept without any allocation (the paper has no counterpart: this is a packaging
 * variant for hosts that cannot call cudaMalloc -- an engine whose pool owns the device, a plugin
 * that gets streams but no allocator, a loop that must not synchronise).  Same arguments, meaning,
 * outputs and error codes as confu_tree_accept, minus the context and the workspace: the row
 * statistics go to a fixed array inside the library image (2 MiB per device that loads the
 * library, held until the process exits).
 *   - limit: B * T <= confu_tree_accept_static_max_rows() (4096); beyond it CONFU_ERR_WORKSPACE;
 *   - the first call on a device looks the array's device address up (one runtime query, no
 *     allocation) with the current device; make that first call outside any stream capture;
 *   - all calls share the array and it keeps the last call's contents (nothing in it needs
 *     clearing: a call only reads what its own first kernel wrote); calls that overlap on the GPU
 *     race on it, so run them one after another (one stream, or ordered streams);
 *   - the call uses the current device; all pointers are device pointers of that device.
 */
size_t confu_tree_accept_static_max_rows(void);
int confu_tree_accept_static(int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                             const void* target_logits, const void* draft_logits,
                             const int32_t* tokens, const int32_t* parent, const int32_t* con_owner,
                             const float* uniforms, float temperature, int32_t sibling_mode,
                             int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row,
                             int32_t* counters, int32_t* status, void* stream);

/*
 * Acceptance by the sample-and-match rule (Sec. 2 steps 3-4 as the text states them: a draft
 * token is accepted if it matches the token sampled from the target model's distribution at its
 * position; the first mismatch is replaced by the target's own token).  Walk from the root: at the
 * current node draw x from softmax(target_logits[node] / temperature) by inverse CDF in index
 * order with uniforms[b][node] (temperature 0: x = lowest index of the largest logit); the child
 * that carries x (lowest node index) is accepted and becomes the current node; if none does --
 * always so at a leaf -- the walk ends and next_token = x.  Every emitted token is a sample of
 * the target model, so the output distribution is the target's.
 * Statistics are computed on demand: only the target rows of the walked path are read
 * ((accept_len + 1) * V logits per sequence) and a non-finite logit is an error (status 5) only
 * there.  No draft logits, no workspace.
 * Outputs as for confu_tree_accept; counters (optional) [B][4] = draws, accepted nodes,
 * draws within 1e-5 of an edge of the drawn token's cell of the normalised CDF, 0.  All pointers
 * device.
 */
int confu_tree_accept_match(confu_ctx* ctx, int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                            const void* target_logits, const int32_t* tokens, const int32_t* parent,
                            const int32_t* con_owner, const float* uniforms, float temperature,
                            int32_t* accept_len, int32_t* path, int32_t* next_token, int32_t* future_row,
                            int32_t* counters, int32_t* status, void* stream);

/* ---- KV compaction (Sec. 2 step 4: the accepted sequence is the next input) ---- */

/*
 * For every layer l < n_layers and for K and V, in place:
 *   cache[seq_start[b] + P_b + k] = old cache[seq_start[b] + P_b + path[b][k]],  k = 1..accept_len[b]
 * (P_b = prefix_len[b]; slot P_b, the root, and the prefix stay), and
 * new_prefix_len[b] = P_b + accept_len[b] + 1.  Slots past the new prefix keep
 * unspecified contents.  k_cache_layers / v_cache_layers: DEVICE arrays of
 * n_layers device pointers.  Uses dims->Hkv, D, kv_dtype, B, T.  All pointers device.
 * The path is checked on the device before anything moves: 0 <= accept_len[b] <=
 * CONFU_MAX_DEPTH and 0 = path[b][0] < path[b][1] < ... < path[b][accept_len[b]] < T (what
 * confu_tree_accept writes; node ids grow along a root path).  Otherwise status[b] =
 * CONFU_ST_BAD_PATH, nothing of sequence b is copied and new_prefix_len[b] = P_b + 1.
 */
int confu_kv_compact(confu_ctx* ctx, const confu_dims* dims, int32_t n_layers,
                     void* const* k_cache_layers, void* const* v_cache_layers,
                     const int64_t* seq_start, const int32_t* prefix_len,
                     const int32_t* accept_len, const int32_t* path,
                     int32_t* new_prefix_len, int32_t* status, void* stream);

/* ---- writing the step's own K/V into the cache (before confu_tree_attention) ---- */

/*
 * The verification forward computes K and V of the R query rows themselves (draft tree nodes and
 * contemplate tokens are processed in one pass, Sec. 3.1); this call places them behind the
 * prefix: cache[seq_start[b] + prefix_len[b] + r] = rows[b][r], for one layer.
 * k_rows, v_rows: [B][R][Hkv][D].  All pointers device.
 */
int confu_kv_append(confu_ctx* ctx, const confu_dims* dims, const void* k_rows, const void* v_rows,
                    void* k_cache, void* v_cache, const int64_t* seq_start, const int32_t* prefix_len,
                    void* stream);

/* ---- contemplate-token embedding (Sec. 3.2, "Dynamic Contemplate Tokens with MoE") ---- */

/*
 * The embedding of the contemplate token that the verification forward feeds to the target model,
 * as a mixture of n_expert learnable embeddings conditioned on the hidden state of the most
 * recently accepted token: a linear layer (router_w [n_expert][H_in], optional bias router_b
 * [n_expert]) maps hidden [B][H_in] to one logit per expert, a softmax normalises them, the
 * k_expert largest scores are selected (the lower index on equal scores) and
 *   out[b][:] = sum over the selection of  gate * experts[e][:]        (experts [n_expert][H_out])
 * with gate = the expert's softmax score, or, with renormalize != 0, that score divided by the sum
 * over the selection (the paper says "normalized gating scores" and does not say which; it gives
 * neither n_expert nor k_expert: both are arguments; limits n_expert <= 1024, k_expert <= 32).
 * All five tensors have the type `dtype` (CONFU_BF16 | CONFU_F32), rows contiguous; accumulation
 * is fp32.  Optional outputs: sel [B][k_expert] int32 (largest score first) and gate [B][k_expert]
 * fp32 (the weights used).  A sequence with a non-finite router logit (NaN or infinity in its
 * hidden state, or in the router) gets status[b] = CONFU_ST_NONFINITE (status: optional device
 * int32 [B]), an all-zero output row, sel = 0..k_expert-1 and gate = 0.  All pointers device,
 * 16-byte aligned.
 */
int confu_con_embedding(confu_ctx* ctx, int32_t B, int32_t H_in, int32_t H_out, int32_t n_expert, int32_t k_expert,
                        int32_t dtype, const void* hidden, const void* router_w, const void* router_b,
                        const void* experts, int32_t renormalize, void* out, int32_t* sel, float* gate,
                        int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CONFU_H */
