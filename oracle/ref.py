"""ctypes front end of the fp64 CPU oracle (oracle/confu_ref.c).

TEST INFRASTRUCTURE ONLY.  Imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg; the product package never imports it.

Every function takes CPU torch tensors (bf16 / fp32 / fp64 data, int32 / int64
indices) and returns CPU torch tensors in fp64 / int32.
"""
import ctypes as C
import os

import torch

from . import build as _build

MAX_DEPTH = 63
BF16, F32, F64 = 0, 1, 2

ST_OK, ST_BAD_PARENT, ST_BAD_OWNER, ST_BAD_TOKEN, ST_DUP_SIBLING, ST_NONFINITE = 0, 1, 2, 3, 4, 5
ST_DEGENERATE, ST_TOO_DEEP = 7, 8

_DT = {torch.bfloat16: BF16, torch.float32: F32, torch.float64: F64}


class _Dims(C.Structure):
    _fields_ = [("B", C.c_int32), ("Hq", C.c_int32), ("Hkv", C.c_int32), ("D", C.c_int32),
                ("T", C.c_int32), ("C", C.c_int32), ("S", C.c_int32), ("dtype", C.c_int32),
                ("sm_scale", C.c_double)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(_build.build())
        _lib.confu_ref_num_threads.restype = C.c_int
        for name in ("confu_ref_tree_attention", "confu_ref_tree_attention_rows",
                     "confu_ref_tree_accept", "confu_ref_tree_accept_match", "confu_ref_kv_compact",
                     "confu_ref_con_embedding", "confu_ref_e4m3_decode", "confu_ref_e4m3_encode"):
            getattr(_lib, name).restype = C.c_int
    return _lib


def num_threads() -> int:
    return int(lib().confu_ref_num_threads())


def _p(t):
    if t is None:
        return C.c_void_p(0)
    assert t.device.type == "cpu" and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _i32(t):
    return None if t is None else t.to(torch.int32).contiguous()


def _dims(q, k_cache, T, Cn, S, sm_scale):
    B, R, Hq, D = q.shape
    assert R == T + Cn
    Hkv = k_cache.shape[1]
    return _Dims(B, Hq, Hkv, D, T, Cn, S, _DT[q.dtype], float(sm_scale))


def tree_attention(q, k_cache, v_cache, seq_start, prefix_len, k_soft, v_soft, parent, con_owner,
                   sm_scale=0.0, want_lse=True):
    """Full-tensor attention of one layer.  Returns (out [B,R,Hq,D] f64, lse [B,R,Hq] f64, status [B])."""
    B, R, Hq, D = q.shape
    T = parent.shape[1]
    Cn = R - T
    S = 0 if k_soft is None else k_soft.shape[0]
    dm = _dims(q, k_cache, T, Cn, S, sm_scale)
    q, k_cache, v_cache = q.contiguous(), k_cache.contiguous(), v_cache.contiguous()
    assert k_cache.dtype == q.dtype and v_cache.dtype == q.dtype
    ks = None if k_soft is None else k_soft.contiguous()
    vs = None if v_soft is None else v_soft.contiguous()
    seq_start = seq_start.to(torch.int64).contiguous()
    prefix_len, parent, con_owner = _i32(prefix_len), _i32(parent), _i32(con_owner)
    out = torch.empty(B, R, Hq, D, dtype=torch.float64)
    lse = torch.empty(B, R, Hq, dtype=torch.float64) if want_lse else None
    status = torch.zeros(B, dtype=torch.int32)
    rc = lib().confu_ref_tree_attention(C.byref(dm), _p(q), _p(k_cache), _p(v_cache), _p(seq_start),
                                        _p(prefix_len), _p(ks), _p(vs), _p(parent), _p(con_owner),
                                        _p(out), _p(lse), _p(status))
    if rc != 0:
        raise ValueError("confu_ref_tree_attention: bad argument")
    return out, lse, status


def tree_attention_rows(q, k_cache, v_cache, seq_start, prefix_len, k_soft, v_soft, parent, con_owner,
                        sel, sm_scale=0.0):
    """Attention for chosen (b, r, h) triples.  sel: [n,3] ints.  Returns (out [n,D] f64, lse [n] f64)."""
    B, R, Hq, D = q.shape
    T = parent.shape[1]
    Cn = R - T
    S = 0 if k_soft is None else k_soft.shape[0]
    dm = _dims(q, k_cache, T, Cn, S, sm_scale)
    q, k_cache, v_cache = q.contiguous(), k_cache.contiguous(), v_cache.contiguous()
    ks = None if k_soft is None else k_soft.contiguous()
    vs = None if v_soft is None else v_soft.contiguous()
    seq_start = seq_start.to(torch.int64).contiguous()
    prefix_len, parent, con_owner = _i32(prefix_len), _i32(parent), _i32(con_owner)
    sel = _i32(torch.as_tensor(sel)).reshape(-1, 3).contiguous()
    n = sel.shape[0]
    out = torch.empty(n, D, dtype=torch.float64)
    lse = torch.empty(n, dtype=torch.float64)
    rc = lib().confu_ref_tree_attention_rows(C.byref(dm), _p(q), _p(k_cache), _p(v_cache), _p(seq_start),
                                             _p(prefix_len), _p(ks), _p(vs), _p(parent), _p(con_owner),
                                             C.c_int32(n), _p(sel), _p(out), _p(lse))
    if rc != 0:
        raise ValueError("confu_ref_tree_attention_rows: bad argument")
    return out, lse


def tree_accept(target_logits, draft_logits, tokens, parent, con_owner, uniforms, temperature=1.0,
                sibling_mode=1):
    """Acceptance walk.  Returns a dict of CPU tensors (see confu_ref.h for the fields)."""
    B, T, V = target_logits.shape
    Cn = 0 if con_owner is None else con_owner.shape[1]
    tl = target_logits.contiguous()
    dl = None if draft_logits is None else draft_logits.contiguous()
    if dl is not None:
        assert dl.dtype == tl.dtype
    tokens, parent, con_owner = _i32(tokens), _i32(parent), _i32(con_owner)
    uni = None if uniforms is None else uniforms.to(torch.float64).contiguous()
    o = {
        "accept_len": torch.zeros(B, dtype=torch.int32),
        "path": torch.full((B, MAX_DEPTH + 1), -1, dtype=torch.int32),
        "next_token": torch.zeros(B, dtype=torch.int32),
        "future_row": torch.zeros(B, dtype=torch.int32),
        "counters": torch.zeros(B, 4, dtype=torch.int32),
        "ratio_margin": torch.zeros(B, dtype=torch.float64),
        "resample_margin": torch.zeros(B, dtype=torch.float64),
        "alt_token": torch.zeros(B, 2, dtype=torch.int32),
        "status": torch.zeros(B, dtype=torch.int32),
    }
    rc = lib().confu_ref_tree_accept(C.c_int32(B), C.c_int32(T), C.c_int32(Cn), C.c_int32(V),
                                     C.c_int32(_DT[tl.dtype]), _p(tl), _p(dl), _p(tokens), _p(parent),
                                     _p(con_owner), _p(uni), C.c_double(temperature), C.c_int32(sibling_mode),
                                     _p(o["accept_len"]), _p(o["path"]), _p(o["next_token"]),
                                     _p(o["future_row"]), _p(o["counters"]), _p(o["ratio_margin"]),
                                     _p(o["resample_margin"]), _p(o["alt_token"]), _p(o["status"]))
    if rc != 0:
        raise ValueError("confu_ref_tree_accept: bad argument")
    return o


def tree_accept_match(target_logits, tokens, parent, con_owner, uniforms, temperature=1.0):
    """Acceptance by the sample-and-match rule.  Returns a dict of CPU tensors (see confu_ref.h)."""
    B, T, V = target_logits.shape
    Cn = 0 if con_owner is None else con_owner.shape[1]
    tl = target_logits.contiguous()
    tokens, parent, con_owner = _i32(tokens), _i32(parent), _i32(con_owner)
    uni = None if uniforms is None else uniforms.to(torch.float64).contiguous()
    o = {
        "accept_len": torch.zeros(B, dtype=torch.int32),
        "path": torch.full((B, MAX_DEPTH + 1), -1, dtype=torch.int32),
        "next_token": torch.zeros(B, dtype=torch.int32),
        "future_row": torch.zeros(B, dtype=torch.int32),
        "counters": torch.zeros(B, 4, dtype=torch.int32),
        "draw_margin": torch.zeros(B, dtype=torch.float64),
        "alt_token": torch.zeros(B, 2, dtype=torch.int32),
        "status": torch.zeros(B, dtype=torch.int32),
    }
    rc = lib().confu_ref_tree_accept_match(C.c_int32(B), C.c_int32(T), C.c_int32(Cn), C.c_int32(V),
                                           C.c_int32(_DT[tl.dtype]), _p(tl), _p(tokens), _p(parent),
                                           _p(con_owner), _p(uni), C.c_double(temperature),
                                           _p(o["accept_len"]), _p(o["path"]), _p(o["next_token"]),
                                           _p(o["future_row"]), _p(o["counters"]), _p(o["draw_margin"]),
                                           _p(o["alt_token"]), _p(o["status"]))
    if rc != 0:
        raise ValueError("confu_ref_tree_accept_match: bad argument")
    return o


def kv_compact(k_layers, v_layers, seq_start, prefix_len, accept_len, path):
    """In-place compaction of lists of per-layer CPU pools [n_slots, Hkv, D].  Returns new_prefix_len [B]."""
    L = len(k_layers)
    B = prefix_len.shape[0]
    row_bytes = k_layers[0][0].numel() * k_layers[0].element_size() if L else 1
    for t in list(k_layers) + list(v_layers):
        assert t.device.type == "cpu" and t.is_contiguous()
    kp = (C.c_void_p * L)(*[t.data_ptr() for t in k_layers])
    vp = (C.c_void_p * L)(*[t.data_ptr() for t in v_layers])
    seq_start = seq_start.to(torch.int64).contiguous()
    prefix_len, accept_len, path = _i32(prefix_len), _i32(accept_len), _i32(path)
    new_len = torch.zeros(B, dtype=torch.int32)
    rc = lib().confu_ref_kv_compact(C.c_int32(B), C.c_int32(L), C.c_int64(row_bytes), kp, vp,
                                    _p(seq_start), _p(prefix_len), _p(accept_len), _p(path), _p(new_len))
    if rc != 0:
        raise ValueError("confu_ref_kv_compact: bad argument")
    return new_len


def con_embedding(hidden, router_w, router_b, experts, k_expert, renormalize=False):
    """Mixture-of-experts embedding of the contemplate token.  Returns (out [B,H_out] fp64,
    sel [B,k] int32, gate [B,k] fp64, gap [B] fp64)."""
    B, H_in = hidden.shape
    n_expert, H_out = experts.shape
    dt = hidden.dtype
    assert router_w.dtype == dt and experts.dtype == dt and (router_b is None or router_b.dtype == dt)
    out = torch.zeros(B, H_out, dtype=torch.float64)
    sel = torch.zeros(B, k_expert, dtype=torch.int32)
    gate = torch.zeros(B, k_expert, dtype=torch.float64)
    gap = torch.zeros(B, dtype=torch.float64)
    rb = None if router_b is None else router_b.contiguous()
    rc = lib().confu_ref_con_embedding(C.c_int32(B), C.c_int32(H_in), C.c_int32(H_out), C.c_int32(n_expert),
                                       C.c_int32(k_expert), C.c_int32(_DT[dt]), _p(hidden.contiguous()),
                                       _p(router_w.contiguous()), _p(rb), _p(experts.contiguous()),
                                       C.c_int32(1 if renormalize else 0), _p(out), _p(sel), _p(gate), _p(gap))
    if rc != 0:
        raise ValueError("confu_ref_con_embedding: bad argument")
    return out, sel, gate, gap


def e4m3_decode(codes):
    """uint8 tensor of E4M3 codes -> fp64 values (same shape)."""
    c = codes.contiguous()
    assert c.dtype == torch.uint8 and c.device.type == "cpu"
    out = torch.empty(c.shape, dtype=torch.float64)
    if lib().confu_ref_e4m3_decode(_p(c), C.c_int64(c.numel()), _p(out)) != 0:
        raise ValueError("confu_ref_e4m3_decode: bad argument")
    return out


def e4m3_encode(x, scale):
    """fp32 tensor -> uint8 E4M3 codes of x / scale (one scale for the whole tensor)."""
    x = x.to(torch.float32).contiguous()
    out = torch.empty(x.shape, dtype=torch.uint8)
    if lib().confu_ref_e4m3_encode(_p(x), C.c_float(float(scale)), C.c_int64(x.numel()), _p(out)) != 0:
        raise ValueError("confu_ref_e4m3_encode: bad argument")
    return out


def quantize_cache(x, scale):
    """[n_slots, Hkv, D] bf16/fp32 rows -> E4M3 codes with one scale per KV head (scale: [Hkv] fp32)."""
    out = torch.empty(x.shape, dtype=torch.uint8)
    for g in range(x.shape[1]):
        out[:, g] = e4m3_encode(x[:, g].float(), float(scale[g]))
    return out


def dequantize_cache(codes, scale):
    """E4M3 codes [n, Hkv, D] and per-head scales [Hkv] -> the fp64 values the cache stands for."""
    v = e4m3_decode(codes)
    return v * scale.to(torch.float64).view(1, -1, 1)


def tree_attention_fp8(q, k_codes, v_codes, k_scale, v_scale, seq_start, prefix_len, ks_codes, vs_codes, parent,
                       con_owner, sm_scale=0.0):
    """Attention over an E4M3 cache: the definition applied to the values the cache stands for
    (bytes and scales widened exactly); q is widened exactly as well."""
    k = dequantize_cache(k_codes, k_scale)
    v = dequantize_cache(v_codes, v_scale)
    ks = None if ks_codes is None else dequantize_cache(ks_codes, k_scale)
    vs = None if vs_codes is None else dequantize_cache(vs_codes, v_scale)
    return tree_attention(q.to(torch.float64), k, v, seq_start, prefix_len, ks, vs, parent, con_owner, sm_scale=sm_scale)
