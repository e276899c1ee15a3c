"""Thin ctypes binding of the C-ABI library (libconfu.so): argument marshalling only.

Every function here has the name of the C entry point it forwards to and does nothing but
turn torch CUDA tensors into pointers; every step of the path runs in the CUDA kernels.
There is no CPU fallback: if the library is missing, loading raises.
"""
import ctypes as C
import os

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libconfu.so")

MAX_TREE = 64
MAX_ROWS = 128
MAX_DEPTH = 63
ACCEPT_LAZY = 0x100          # or-ed into sibling_mode: row statistics on demand
BF16, F32, FP8_E4M3 = 0, 1, 2
OK = 0
OPT_ATTENTION_PATH, OPT_WAIT_LIMIT_NS = 1, 2
ATTENTION_AUTO, ATTENTION_GENERIC, ATTENTION_TENSOR, ATTENTION_TENSOR_PAIR = 0, 1, 2, 3
ST_TIMEOUT, ST_BAD_PATH, ST_BAD_PLAN = 6, 9, 10

EXPORTS = [
    "confu_create", "confu_destroy", "confu_workspace_bytes", "confu_set_workspace", "confu_status_string",
    "confu_last_cuda_error", "confu_plan_bytes", "confu_tree_plan", "confu_tree_attention",
    "confu_accept_workspace_bytes", "confu_tree_accept", "confu_kv_compact", "confu_kv_append",
    "confu_tree_accept_static_max_rows", "confu_tree_accept_static", "confu_set_paging",
    "confu_tree_accept_match", "confu_con_embedding", "confu_set_option", "confu_attention_path",
    "confu_selftest_bounded_wait", "confu_set_kv_scales",
]


class ConfuDims(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32), ("T", C.c_int32),
                ("C", C.c_int32), ("S", C.c_int32), ("kv_dtype", C.c_int32), ("sm_scale", C.c_float)]


_lib = None


def lib():
    """Load libconfu.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2603_08899_b200.build` "
                               "(the CUDA library is the only implementation)")
        L = C.CDLL(LIB_PATH)
        L.confu_workspace_bytes.restype = C.c_size_t
        L.confu_plan_bytes.restype = C.c_size_t
        L.confu_accept_workspace_bytes.restype = C.c_size_t
        L.confu_tree_accept_static_max_rows.restype = C.c_size_t
        L.confu_status_string.restype = C.c_char_p
        L.confu_last_cuda_error.restype = C.c_char_p
        for n in ("confu_create", "confu_destroy", "confu_set_workspace", "confu_tree_plan", "confu_tree_attention",
                  "confu_tree_accept", "confu_kv_compact", "confu_kv_append", "confu_tree_accept_static", "confu_set_paging",
                  "confu_tree_accept_match", "confu_con_embedding", "confu_set_option", "confu_attention_path", "confu_selftest_bounded_wait",
                  "confu_set_kv_scales"):
            getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


class ConfuError(RuntimeError):
    def __init__(self, fn, code, detail=""):
        self.code = code
        msg = lib().confu_status_string(code).decode()
        super().__init__(f"{fn}: {msg} ({code}) {detail}")


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    if isinstance(t, int):
        return C.c_void_p(t)
    assert t.is_cuda and t.is_contiguous(), "device, contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _stream(stream):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def _check(fn, rc, ctx=None):
    if rc != OK:
        detail = lib().confu_last_cuda_error(ctx).decode() if (ctx and rc == -6) else ""
        raise ConfuError(fn, rc, detail)


def dtype_code(dt):
    return {torch.bfloat16: BF16, torch.float32: F32, torch.uint8: FP8_E4M3, torch.float8_e4m3fn: FP8_E4M3}[dt]


def make_dims(B, Hq, Hkv, D, T, Cn, S, dtype, sm_scale=0.0):
    return ConfuDims(B, Hq, Hkv, D, T, Cn, S, dtype_code(dtype), float(sm_scale))


# --------------------------------------------------------------------------- entry points
def confu_create(device=0):
    h = C.c_void_p()
    _check("confu_create", lib().confu_create(C.byref(h), C.c_int(device)))
    return h


def confu_destroy(ctx):
    _check("confu_destroy", lib().confu_destroy(ctx))


def confu_workspace_bytes(ctx, dims):
    return int(lib().confu_workspace_bytes(ctx, C.byref(dims)))


def confu_set_workspace(ctx, tensor):
    nbytes = 0 if tensor is None else tensor.numel() * tensor.element_size()
    _check("confu_set_workspace", lib().confu_set_workspace(ctx, _ptr(tensor), C.c_size_t(nbytes)))


def confu_set_paging(ctx, block_table, max_pages=0):
    """block_table: int32 CUDA tensor [B, max_pages] (kept alive by the caller), or None for packed pools."""
    _check("confu_set_paging", lib().confu_set_paging(ctx, _ptr(block_table), C.c_int32(max_pages)))


def confu_set_kv_scales(ctx, k_scale, v_scale):
    """k_scale, v_scale: fp32 CUDA tensors [Hkv] (kept alive by the caller), or None, None."""
    _check("confu_set_kv_scales", lib().confu_set_kv_scales(ctx, _ptr(k_scale), _ptr(v_scale)))


def confu_set_option(ctx, option, value):
    _check("confu_set_option", lib().confu_set_option(ctx, C.c_int32(option), C.c_int64(value)))


def confu_attention_path(ctx, dims):
    """The ATTENTION_* path the library takes for these dims (never ATTENTION_AUTO); raises where the calls would fail."""
    rc = int(lib().confu_attention_path(ctx, C.byref(dims)))
    if rc < 0:
        _check("confu_attention_path", rc)
    return rc


def confu_selftest_bounded_wait(ctx, limit_ns, status, stream=None):
    _check("confu_selftest_bounded_wait",
           lib().confu_selftest_bounded_wait(ctx, C.c_int64(limit_ns), _ptr(status), _stream(stream)), ctx)


def confu_plan_bytes(ctx, dims):
    return int(lib().confu_plan_bytes(ctx, C.byref(dims)))


def confu_tree_plan(ctx, dims, seq_start, prefix_len, parent, con_owner, plan, status, stream=None):
    _check("confu_tree_plan",
           lib().confu_tree_plan(ctx, C.byref(dims), _ptr(seq_start), _ptr(prefix_len), _ptr(parent),
                                 _ptr(con_owner), _ptr(plan), _ptr(status), _stream(stream)), ctx)


def confu_tree_attention(ctx, dims, q, k_cache, v_cache, n_slots, seq_start, prefix_len, k_soft, v_soft, parent,
                         con_owner, plan, out, lse, status, stream=None):
    _check("confu_tree_attention",
           lib().confu_tree_attention(ctx, C.byref(dims), _ptr(q), _ptr(k_cache), _ptr(v_cache), C.c_int64(n_slots),
                                      _ptr(seq_start), _ptr(prefix_len), _ptr(k_soft), _ptr(v_soft), _ptr(parent),
                                      _ptr(con_owner), _ptr(plan), _ptr(out), _ptr(lse), _ptr(status),
                                      _stream(stream)), ctx)


def confu_accept_workspace_bytes(B, T, V):
    return int(lib().confu_accept_workspace_bytes(C.c_int32(B), C.c_int32(T), C.c_int32(V)))


def confu_tree_accept(ctx, B, T, Cn, V, logit_dtype, target_logits, draft_logits, tokens, parent, con_owner, uniforms,
                      temperature, sibling_mode, accept_len, path, next_token, future_row, counters, workspace,
                      status, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check("confu_tree_accept",
           lib().confu_tree_accept(ctx, C.c_int32(B), C.c_int32(T), C.c_int32(Cn), C.c_int32(V),
                                   C.c_int32(dtype_code(logit_dtype)), _ptr(target_logits), _ptr(draft_logits),
                                   _ptr(tokens), _ptr(parent), _ptr(con_owner), _ptr(uniforms),
                                   C.c_float(temperature), C.c_int32(sibling_mode), _ptr(accept_len), _ptr(path),
                                   _ptr(next_token), _ptr(future_row), _ptr(counters), _ptr(workspace),
                                   C.c_size_t(ws_bytes), _ptr(status), _stream(stream)), ctx)


def confu_tree_accept_match(ctx, B, T, Cn, V, logit_dtype, target_logits, tokens, parent, con_owner, uniforms,
                            temperature, accept_len, path, next_token, future_row, counters, status, stream=None):
    """Acceptance by the sample-and-match rule; reads only the target rows of the walked path."""
    _check("confu_tree_accept_match",
           lib().confu_tree_accept_match(ctx, C.c_int32(B), C.c_int32(T), C.c_int32(Cn), C.c_int32(V),
                                         C.c_int32(dtype_code(logit_dtype)), _ptr(target_logits), _ptr(tokens),
                                         _ptr(parent), _ptr(con_owner), _ptr(uniforms), C.c_float(temperature),
                                         _ptr(accept_len), _ptr(path), _ptr(next_token), _ptr(future_row),
                                         _ptr(counters), _ptr(status), _stream(stream)), ctx)


def confu_con_embedding(ctx, hidden, router_w, router_b, experts, k_expert, renormalize, out, sel=None, gate=None,
                        status=None, stream=None):
    """Contemplate-token embedding: router -> softmax -> top-k experts -> weighted sum of their embeddings."""
    B, H_in = hidden.shape
    n_expert, H_out = experts.shape
    _check("confu_con_embedding",
           lib().confu_con_embedding(ctx, C.c_int32(B), C.c_int32(H_in), C.c_int32(H_out), C.c_int32(n_expert),
                                     C.c_int32(k_expert), C.c_int32(dtype_code(hidden.dtype)), _ptr(hidden),
                                     _ptr(router_w), _ptr(router_b), _ptr(experts), C.c_int32(1 if renormalize else 0),
                                     _ptr(out), _ptr(sel), _ptr(gate), _ptr(status), _stream(stream)), ctx)


def confu_tree_accept_static_max_rows():
    return int(lib().confu_tree_accept_static_max_rows())


def confu_tree_accept_static(B, T, Cn, V, logit_dtype, target_logits, draft_logits, tokens, parent, con_owner,
                             uniforms, temperature, sibling_mode, accept_len, path, next_token, future_row, counters,
                             status, stream=None):
    """confu_tree_accept for callers that may not allocate: no context, no workspace (the library's
    fixed scratch is used; B * T is limited to confu_tree_accept_static_max_rows())."""
    _check("confu_tree_accept_static",
           lib().confu_tree_accept_static(C.c_int32(B), C.c_int32(T), C.c_int32(Cn), C.c_int32(V),
                                          C.c_int32(dtype_code(logit_dtype)), _ptr(target_logits),
                                          _ptr(draft_logits), _ptr(tokens), _ptr(parent), _ptr(con_owner),
                                          _ptr(uniforms), C.c_float(temperature), C.c_int32(sibling_mode),
                                          _ptr(accept_len), _ptr(path), _ptr(next_token), _ptr(future_row),
                                          _ptr(counters), _ptr(status), _stream(stream)))


def confu_kv_compact(ctx, dims, n_layers, k_layer_ptrs, v_layer_ptrs, seq_start, prefix_len, accept_len, path,
                     new_prefix_len, status, stream=None):
    """k_layer_ptrs / v_layer_ptrs: int64 CUDA tensors holding the per-layer pool addresses."""
    _check("confu_kv_compact",
           lib().confu_kv_compact(ctx, C.byref(dims), C.c_int32(n_layers), _ptr(k_layer_ptrs), _ptr(v_layer_ptrs),
                                  _ptr(seq_start), _ptr(prefix_len), _ptr(accept_len), _ptr(path),
                                  _ptr(new_prefix_len), _ptr(status), _stream(stream)), ctx)


def confu_kv_append(ctx, dims, k_rows, v_rows, k_cache, v_cache, seq_start, prefix_len, stream=None):
    _check("confu_kv_append",
           lib().confu_kv_append(ctx, C.byref(dims), _ptr(k_rows), _ptr(v_rows), _ptr(k_cache), _ptr(v_cache),
                                 _ptr(seq_start), _ptr(prefix_len), _stream(stream)), ctx)
