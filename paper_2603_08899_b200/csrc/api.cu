// C ABI of the library: argument checks, workspace carving, kernel launches.
#include <new>

#include "common.cuh"

using namespace confu;

struct confu_ctx : public confu::Ctx {};

namespace {

inline bool misaligned(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

int check_dims(const confu_dims* d)
{
    if (!d) return CONFU_ERR_ARG;
    if (d->B < 0 || d->Hq <= 0 || d->Hkv <= 0 || d->T <= 0 || d->C < 0 || d->S < 0) return CONFU_ERR_SHAPE;
    if (d->Hq % d->Hkv != 0) return CONFU_ERR_SHAPE;
    if (d->D != 64 && d->D != 128) return CONFU_ERR_SHAPE;
    if (d->kv_dtype != CONFU_BF16 && d->kv_dtype != CONFU_F32 && d->kv_dtype != CONFU_FP8_E4M3) return CONFU_ERR_ARG;
    if (d->kv_dtype == CONFU_FP8_E4M3 && (d->D != 128 || d->Hq / d->Hkv > 4 || d->S > 128)) return CONFU_ERR_UNSUPPORTED;
    if (d->T > CONFU_MAX_TREE || d->C > CONFU_MAX_TREE) return CONFU_ERR_UNSUPPORTED;
    if (!(d->sm_scale >= 0.f)) return CONFU_ERR_ARG;
    return CONFU_OK;
}

int cuda_fail(confu_ctx* ctx, cudaError_t e)
{
    if (ctx) ctx->last_error = e;
    return CONFU_ERR_CUDA;
}

// workspace carving: [plan built by the attention call itself][split-KV partial slots]
size_t ws_plan_offset() { return 0; }
size_t ws_partial_offset(const confu_dims* d) { return align_up(plan_bytes(d->B, d->Hkv), 256); }
size_t ws_total(const confu_ctx* ctx, const confu_dims* d)
{
    return ws_partial_offset(d) + (size_t)2 * ctx->sm_count * partial_slot_bytes();
}

}  // namespace

namespace confu {
cudaError_t launch_bounded_wait(unsigned long long limit_ns, int32_t* status, cudaStream_t st);
bool tc_attention_supported(const confu_dims& d);
bool pair_attention_supported(const confu_dims& d, int sm_count);
bool fp8_attention_supported(const confu_dims& d);
cudaError_t launch_attention_fp8(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                 const void* v_cache, int64_t n_slots, const SlotMap& map,
                                 const int32_t* prefix_len, const void* k_soft, const void* v_soft, const void* plan,
                                 void* partials, void* out, float* lse, int32_t* status, cudaStream_t st);
cudaError_t launch_append_fp8(int B, int R, int Hkv, int D, const void* k_rows, const void* v_rows, void* k_cache,
                              void* v_cache, const SlotMap& map, const int32_t* prefix_len, const float* k_scale,
                              const float* v_scale, cudaStream_t st);
cudaError_t launch_attention_pair(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                  const void* v_cache, int64_t n_slots, const SlotMap& map,
                                  const int32_t* prefix_len, const void* k_soft, const void* v_soft, const void* plan,
                                  void* partials, void* out, float* lse, int32_t* status, cudaStream_t st);
cudaError_t launch_attention_tc(const Ctx* ctx, const confu_dims& d, const void* q, const void* k_cache,
                                const void* v_cache, int64_t n_slots, const SlotMap& map,
                                const int32_t* prefix_len, const void* k_soft, const void* v_soft, const void* plan,
                                void* partials, void* out, float* lse, int32_t* status, cudaStream_t st);
}  // namespace confu

namespace {

// Which attention kernel serves these dims under the context's option: a CONFU_ATTENTION_* value
// (never _AUTO), or a negative error code when a forced path cannot take them.
int resolve_attention_path(const confu_ctx* ctx, const confu_dims& d)
{
    // (a share of the work is walked by one CTA, or CTA pair, per group of 64 query rows: at least two of them)
    const bool tc = tc_attention_supported(d) && ctx->sm_count >= 2, pair = pair_attention_supported(d, ctx->sm_count);
    if (d.kv_dtype == CONFU_FP8_E4M3) {         // one kernel serves E4M3 caches
        const bool ok = ctx->attention_path == CONFU_ATTENTION_AUTO || ctx->attention_path == CONFU_ATTENTION_TENSOR;
        return ok && fp8_attention_supported(d) && ctx->sm_count >= 2 ? (int)CONFU_ATTENTION_TENSOR : (int)CONFU_ERR_UNSUPPORTED;
    }
    switch (ctx->attention_path) {
        case CONFU_ATTENTION_GENERIC: return CONFU_ATTENTION_GENERIC;
        case CONFU_ATTENTION_TENSOR: return tc ? (int)CONFU_ATTENTION_TENSOR : (int)CONFU_ERR_UNSUPPORTED;
        case CONFU_ATTENTION_TENSOR_PAIR: return pair ? (int)CONFU_ATTENTION_TENSOR_PAIR : (int)CONFU_ERR_UNSUPPORTED;
        default: {
            // The two-SM kernel wins where a (sequence, kv head, row group) is split over many work units
            // (small batches: half as many, twice as long runs, half the partial results to merge); with
            // more such pairs than units the one-CTA kernel is the faster one.
            const int n_rg = (d.T + d.C + kGroupRows - 1) / kGroupRows;
            const bool few_pairs = (int64_t)d.B * d.Hkv * n_rg <= ctx->sm_count / 2;
            if (pair && few_pairs) return CONFU_ATTENTION_TENSOR_PAIR;
            return tc ? (int)CONFU_ATTENTION_TENSOR : (int)CONFU_ATTENTION_GENERIC;
        }
    }
}

}  // namespace

extern "C" {

int confu_create(confu_ctx** out, int device)
{
    if (!out) return CONFU_ERR_ARG;
    *out = nullptr;
    confu_ctx* c = new (std::nothrow) confu_ctx();
    if (!c) return CONFU_ERR_ARG;
    c->device = device;
    c->workspace = nullptr;
    c->workspace_bytes = 0;
    c->block_table = nullptr;
    c->max_pages = 0;
    c->last_error = cudaSuccess;
    c->k_scale = c->v_scale = nullptr;
    c->attention_path = CONFU_ATTENTION_AUTO;
    c->wait_ns = 2000000000ull;
    cudaError_t e = cudaSetDevice(device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e != cudaSuccess) {
        delete c;
        return CONFU_ERR_CUDA;
    }
    *out = c;
    return CONFU_OK;
}

int confu_destroy(confu_ctx* ctx)
{
    if (!ctx) return CONFU_ERR_ARG;
    delete ctx;
    return CONFU_OK;
}

size_t confu_workspace_bytes(const confu_ctx* ctx, const confu_dims* dims)
{
    if (!ctx || check_dims(dims) != CONFU_OK) return 0;
    return ws_total(ctx, dims);
}

int confu_set_workspace(confu_ctx* ctx, void* device_ptr, size_t bytes)
{
    if (!ctx) return CONFU_ERR_ARG;
    if (device_ptr && misaligned(device_ptr)) return CONFU_ERR_ALIGN;
    ctx->workspace = device_ptr;
    ctx->workspace_bytes = device_ptr ? bytes : 0;
    return CONFU_OK;
}

int confu_set_paging(confu_ctx* ctx, const int32_t* block_table, int32_t max_pages)
{
    if (!ctx) return CONFU_ERR_ARG;
    if (block_table && max_pages <= 0) return CONFU_ERR_ARG;
    ctx->block_table = block_table;
    ctx->max_pages = block_table ? max_pages : 0;
    return CONFU_OK;
}

int confu_set_kv_scales(confu_ctx* ctx, const float* k_scale, const float* v_scale)
{
    if (!ctx) return CONFU_ERR_ARG;
    if ((k_scale == nullptr) != (v_scale == nullptr)) return CONFU_ERR_ARG;
    ctx->k_scale = k_scale;
    ctx->v_scale = v_scale;
    return CONFU_OK;
}

int confu_set_option(confu_ctx* ctx, int32_t option, int64_t value)
{
    if (!ctx) return CONFU_ERR_ARG;
    switch (option) {
        case CONFU_OPT_ATTENTION_PATH:
            if (value < CONFU_ATTENTION_AUTO || value > CONFU_ATTENTION_TENSOR_PAIR) return CONFU_ERR_ARG;
            ctx->attention_path = (int)value;
            return CONFU_OK;
        case CONFU_OPT_WAIT_LIMIT_NS:
            if (value < 1000 || value > 10000000000ll) return CONFU_ERR_ARG;
            ctx->wait_ns = (unsigned long long)value;
            return CONFU_OK;
        default: return CONFU_ERR_ARG;
    }
}

int confu_attention_path(const confu_ctx* ctx, const confu_dims* dims)
{
    if (!ctx) return CONFU_ERR_ARG;
    const int rc = check_dims(dims);
    if (rc != CONFU_OK) return rc;
    return resolve_attention_path(ctx, *dims);
}

int confu_selftest_bounded_wait(confu_ctx* ctx, int64_t limit_ns, int32_t* status, void* stream)
{
    if (!ctx || !status) return CONFU_ERR_ARG;
    if (limit_ns < 1000 || limit_ns > 1000000000ll) return CONFU_ERR_ARG;     // the kernel ends within a second
    cudaError_t e = launch_bounded_wait((unsigned long long)limit_ns, status, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

const char* confu_status_string(int code)
{
    switch (code) {
        case CONFU_OK: return "ok";
        case CONFU_ERR_ARG: return "bad argument";
        case CONFU_ERR_SHAPE: return "unsupported or inconsistent shape";
        case CONFU_ERR_ALIGN: return "device pointer not 16-byte aligned";
        case CONFU_ERR_WORKSPACE: return "workspace missing or too small";
        case CONFU_ERR_UNSUPPORTED: return "configuration not supported";
        case CONFU_ERR_CUDA: return "CUDA call failed";
        case CONFU_ST_BAD_PARENT: return "malformed tree: parent index";
        case CONFU_ST_BAD_OWNER: return "malformed tree: contemplate owner";
        case CONFU_ST_BAD_TOKEN: return "token id out of range";
        case CONFU_ST_DUP_SIBLING: return "duplicate sibling tokens";
        case CONFU_ST_NONFINITE: return "non-finite logit";
        case CONFU_ST_TIMEOUT: return "bounded device wait expired";
        case CONFU_ST_DEGENERATE: return "residual distribution without mass";
        case CONFU_ST_TOO_DEEP: return "accepted path longer than CONFU_MAX_DEPTH";
        case CONFU_ST_BAD_PATH: return "accepted path is not an increasing chain of tree nodes from the root";
        case CONFU_ST_BAD_PLAN: return "plan was built for another attention path";
        default: return "unknown code";
    }
}

const char* confu_last_cuda_error(const confu_ctx* ctx)
{
    return cudaGetErrorString(ctx ? ctx->last_error : cudaSuccess);
}

size_t confu_plan_bytes(const confu_ctx* ctx, const confu_dims* dims)
{
    if (!ctx || check_dims(dims) != CONFU_OK) return 0;
    return plan_bytes(dims->B, dims->Hkv);
}

int confu_tree_plan(confu_ctx* ctx, const confu_dims* dims, const int64_t* seq_start, const int32_t* prefix_len,
                    const int32_t* parent, const int32_t* con_owner, void* plan, int32_t* status, void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    int rc = check_dims(dims);
    if (rc != CONFU_OK) return rc;
    if (!plan) return CONFU_ERR_ARG;
    if (dims->B > 0 && (!prefix_len || !parent || (dims->C > 0 && !con_owner))) return CONFU_ERR_ARG;
    if (misaligned(plan)) return CONFU_ERR_ALIGN;
    const int path = resolve_attention_path(ctx, *dims);
    if (path < 0) return path;
    cudaError_t e = launch_plan(ctx, *dims, seq_start, prefix_len, parent, con_owner, plan, status,
                                path == CONFU_ATTENTION_TENSOR_PAIR, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

int confu_tree_attention(confu_ctx* ctx, const confu_dims* dims, const void* q, const void* k_cache,
                         const void* v_cache, int64_t n_slots, const int64_t* seq_start, const int32_t* prefix_len,
                         const void* k_soft, const void* v_soft, const int32_t* parent, const int32_t* con_owner,
                         const void* plan, void* out, float* lse, int32_t* status, void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    int rc = check_dims(dims);
    if (rc != CONFU_OK) return rc;
    if (dims->B == 0) return CONFU_OK;
    if (!q || !k_cache || !v_cache || !prefix_len || !out || n_slots <= 0) return CONFU_ERR_ARG;
    if (!ctx->block_table && !seq_start) return CONFU_ERR_ARG;
    if (ctx->block_table && n_slots % kTileKeys != 0) return CONFU_ERR_SHAPE;      // a paged pool is whole pages
    const SlotMap map = {seq_start, ctx->block_table, ctx->max_pages};
    if (dims->S > 0 && (!k_soft || !v_soft)) return CONFU_ERR_ARG;
    if (!plan && (!parent || (dims->C > 0 && !con_owner))) return CONFU_ERR_ARG;
    if (misaligned(q) || misaligned(k_cache) || misaligned(v_cache) || misaligned(out) || misaligned(k_soft) ||
        misaligned(v_soft) || misaligned(plan))
        return CONFU_ERR_ALIGN;
    if (!ctx->workspace || ctx->workspace_bytes < ws_total(ctx, dims)) return CONFU_ERR_WORKSPACE;
    const int path = resolve_attention_path(ctx, *dims);
    if (path < 0) return path;
    if (dims->kv_dtype == CONFU_FP8_E4M3 && !ctx->k_scale) return CONFU_ERR_UNSUPPORTED;      // an E4M3 cache means nothing without its scales
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)ctx->workspace;
    const void* use_plan = plan;
    if (!plan) {
        void* own_plan = ws + ws_plan_offset();
        cudaError_t e = launch_plan(ctx, *dims, seq_start, prefix_len, parent, con_owner, own_plan, status,
                                    path == CONFU_ATTENTION_TENSOR_PAIR, st);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        use_plan = own_plan;
    }
    cudaError_t e;
    if (path == CONFU_ATTENTION_TENSOR_PAIR)
        e = launch_attention_pair(ctx, *dims, q, k_cache, v_cache, n_slots, map, prefix_len, k_soft, v_soft,
                                  use_plan, ws + ws_partial_offset(dims), out, lse, status, st);
    else if (path == CONFU_ATTENTION_TENSOR && dims->kv_dtype == CONFU_FP8_E4M3)
        e = launch_attention_fp8(ctx, *dims, q, k_cache, v_cache, n_slots, map, prefix_len, k_soft, v_soft,
                                 use_plan, ws + ws_partial_offset(dims), out, lse, status, st);
    else if (path == CONFU_ATTENTION_TENSOR)
        e = launch_attention_tc(ctx, *dims, q, k_cache, v_cache, n_slots, map, prefix_len, k_soft, v_soft,
                                use_plan, ws + ws_partial_offset(dims), out, lse, status, st);
    else
        e = launch_attention_generic(ctx, *dims, q, k_cache, v_cache, map, prefix_len, k_soft, v_soft, use_plan,
                                     out, lse, st);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

size_t confu_accept_workspace_bytes(int32_t B, int32_t T, int32_t V)
{
    if (B < 0 || T <= 0 || V <= 0) return 0;
    return accept_workspace_bytes(B, T, V);
}

int confu_tree_accept(confu_ctx* ctx, int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                      const void* target_logits, const void* draft_logits, const int32_t* tokens,
                      const int32_t* parent, const int32_t* con_owner, const float* uniforms, float temperature,
                      int32_t sibling_mode, int32_t* accept_len, int32_t* path, int32_t* next_token,
                      int32_t* future_row, int32_t* counters, void* workspace, size_t workspace_bytes,
                      int32_t* status, void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    if (B < 0 || T <= 0 || C < 0 || V <= 0) return CONFU_ERR_SHAPE;
    if (logit_dtype != CONFU_BF16 && logit_dtype != CONFU_F32) return CONFU_ERR_ARG;
    const bool lazy = (sibling_mode & CONFU_ACCEPT_LAZY) != 0;
    if ((sibling_mode & ~CONFU_ACCEPT_LAZY) != 0 && (sibling_mode & ~CONFU_ACCEPT_LAZY) != 1) return CONFU_ERR_ARG;
    if (!(temperature >= 0.f)) return CONFU_ERR_ARG;
    if (T > CONFU_MAX_TREE || C > CONFU_MAX_TREE || V > 262144) return CONFU_ERR_UNSUPPORTED;
    if (B == 0) return CONFU_OK;
    if (!target_logits || !tokens || !parent || !accept_len || !path || !next_token) return CONFU_ERR_ARG;
    if (C > 0 && !con_owner) return CONFU_ERR_ARG;
    if (temperature > 0.f && (!draft_logits || !uniforms)) return CONFU_ERR_ARG;
    if (misaligned(target_logits) || misaligned(draft_logits) || misaligned(workspace)) return CONFU_ERR_ALIGN;
    if (!lazy && (!workspace || workspace_bytes < accept_workspace_bytes(B, T, V))) return CONFU_ERR_WORKSPACE;
    cudaError_t e = launch_accept(ctx, B, T, C, V, logit_dtype, target_logits, draft_logits, tokens, parent, con_owner,
                                  uniforms, temperature, sibling_mode, accept_len, path, next_token, future_row,
                                  counters, workspace, status, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

int confu_tree_accept_match(confu_ctx* ctx, int32_t B, int32_t T, int32_t C, int32_t V, int32_t logit_dtype,
                            const void* target_logits, const int32_t* tokens, const int32_t* parent,
                            const int32_t* con_owner, const float* uniforms, float temperature, int32_t* accept_len,
                            int32_t* path, int32_t* next_token, int32_t* future_row, int32_t* counters, int32_t* status,
                            void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    if (B < 0 || T <= 0 || C < 0 || V <= 0) return CONFU_ERR_SHAPE;
    if (logit_dtype != CONFU_BF16 && logit_dtype != CONFU_F32) return CONFU_ERR_ARG;
    if (!(temperature >= 0.f)) return CONFU_ERR_ARG;
    if (T > CONFU_MAX_TREE || C > CONFU_MAX_TREE || V > 262144) return CONFU_ERR_UNSUPPORTED;
    if (B == 0) return CONFU_OK;
    if (!target_logits || !tokens || !parent || !accept_len || !path || !next_token) return CONFU_ERR_ARG;
    if (C > 0 && !con_owner) return CONFU_ERR_ARG;
    if (temperature > 0.f && !uniforms) return CONFU_ERR_ARG;
    if (misaligned(target_logits)) return CONFU_ERR_ALIGN;
    cudaError_t e = launch_accept_match(B, T, C, V, logit_dtype, target_logits, tokens, parent, con_owner, uniforms,
                                        temperature, accept_len, path, next_token, future_row, counters, status,
                                        (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

int confu_kv_compact(confu_ctx* ctx, const confu_dims* dims, int32_t n_layers, void* const* k_cache_layers,
                     void* const* v_cache_layers, const int64_t* seq_start, const int32_t* prefix_len,
                     const int32_t* accept_len, const int32_t* path, int32_t* new_prefix_len, int32_t* status,
                     void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    int rc = check_dims(dims);
    if (rc != CONFU_OK) return rc;
    if (n_layers < 0) return CONFU_ERR_ARG;
    if (dims->B == 0) return CONFU_OK;
    if (!prefix_len || !accept_len || !path) return CONFU_ERR_ARG;
    if (!ctx->block_table && !seq_start) return CONFU_ERR_ARG;
    const SlotMap map = {seq_start, ctx->block_table, ctx->max_pages};
    if (n_layers > 0 && (!k_cache_layers || !v_cache_layers)) return CONFU_ERR_ARG;
    const int64_t row_bytes = (int64_t)dims->Hkv * dims->D * (dims->kv_dtype == CONFU_BF16 ? 2 : dims->kv_dtype == CONFU_F32 ? 4 : 1);
    cudaError_t e = launch_compact(ctx, dims->B, dims->T, n_layers, row_bytes, k_cache_layers, v_cache_layers, map,
                                   prefix_len, accept_len, path, new_prefix_len, status, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

int confu_kv_append(confu_ctx* ctx, const confu_dims* dims, const void* k_rows, const void* v_rows, void* k_cache,
                    void* v_cache, const int64_t* seq_start, const int32_t* prefix_len, void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    int rc = check_dims(dims);
    if (rc != CONFU_OK) return rc;
    if (dims->B == 0) return CONFU_OK;
    if (!k_rows || !v_rows || !k_cache || !v_cache || !prefix_len) return CONFU_ERR_ARG;
    if (!ctx->block_table && !seq_start) return CONFU_ERR_ARG;
    const SlotMap map = {seq_start, ctx->block_table, ctx->max_pages};
    if (misaligned(k_rows) || misaligned(v_rows) || misaligned(k_cache) || misaligned(v_cache)) return CONFU_ERR_ALIGN;
    const int64_t row_bytes = (int64_t)dims->Hkv * dims->D * (dims->kv_dtype == CONFU_BF16 ? 2 : dims->kv_dtype == CONFU_F32 ? 4 : 1);
    if (dims->kv_dtype == CONFU_FP8_E4M3) {
        if (!ctx->k_scale) return CONFU_ERR_UNSUPPORTED;
        cudaError_t e8 = launch_append_fp8(dims->B, dims->T + dims->C, dims->Hkv, dims->D, k_rows, v_rows, k_cache, v_cache,
                                           map, prefix_len, ctx->k_scale, ctx->v_scale, (cudaStream_t)stream);
        return e8 == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e8);
    }
    cudaError_t e = launch_append(dims->B, dims->T + dims->C, row_bytes, k_rows, v_rows, k_cache, v_cache, map,
                                  prefix_len, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

int confu_con_embedding(confu_ctx* ctx, int32_t B, int32_t H_in, int32_t H_out, int32_t n_expert, int32_t k_expert,
                        int32_t dtype, const void* hidden, const void* router_w, const void* router_b,
                        const void* experts, int32_t renormalize, void* out, int32_t* sel, float* gate,
                        int32_t* status, void* stream)
{
    if (!ctx) return CONFU_ERR_ARG;
    if (B < 0 || H_in <= 0 || H_out <= 0 || n_expert <= 0 || k_expert <= 0 || k_expert > n_expert) return CONFU_ERR_SHAPE;
    if (dtype != CONFU_BF16 && dtype != CONFU_F32) return CONFU_ERR_ARG;
    if (n_expert > 1024 || k_expert > 32) return CONFU_ERR_UNSUPPORTED;
    if (B == 0) return CONFU_OK;
    if (!hidden || !router_w || !experts || !out) return CONFU_ERR_ARG;
    if (misaligned(hidden) || misaligned(router_w) || misaligned(experts) || misaligned(out)) return CONFU_ERR_ALIGN;
    cudaError_t e = launch_con_embedding(B, H_in, H_out, n_expert, k_expert, dtype, hidden, router_w, router_b, experts,
                                         renormalize != 0, out, sel, gate, status, (cudaStream_t)stream);
    return e == cudaSuccess ? CONFU_OK : cuda_fail(ctx, e);
}

}  // extern "C"
