"""Shared helpers of the GPU parity tests: run the C-ABI path on seeded inputs, run the oracle on the
same inputs, compare.  The expected values always come from the oracle (CPU); nothing here feeds
a CUDA result back into an expectation."""
import math

import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs

# Parity bars.  bf16 path: max|err| <= 2e-2 and max|err| / max|ref| <= 1e-2 per (sequence, layer)
# tensor (outputs are rounded to bf16: half an ulp is 2^-9 of the element, the running sums are
# fp32).  fp32 path: 1e-4 and 1e-5.  lse is compared in absolute terms.
TOL = {torch.bfloat16: (2e-2, 1e-2, 5e-3), torch.float32: (1e-4, 1e-5, 1e-5)}
BORDERLINE = 1e-5


class Gpu:
    """A context plus a workspace sized for the given dims."""

    def __init__(self):
        self.ctx = cb.confu_create(0)
        self.ws = None

    def ensure_ws(self, dims):
        need = cb.confu_workspace_bytes(self.ctx, dims)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device="cuda")
            cb.confu_set_workspace(self.ctx, self.ws)

    def close(self):
        cb.confu_destroy(self.ctx)


def dims_of(cfg, sm_scale=0.0):
    return cb.make_dims(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.T, cfg.C, cfg.S, cfg.kv_dtype, sm_scale)


def gpu_attention(gpu, cfg, t, seq_start, prefix_len, parent, owner, n_slots, use_plan=False, sm_scale=0.0,
                  want_lse=True):
    """t: dict of CUDA tensors from inputs.layer_tensors.  Returns (out, lse, status) on the CPU."""
    dims = dims_of(cfg, sm_scale)
    gpu.ensure_ws(dims)
    dev = "cuda"
    ss, pl = seq_start.to(dev), prefix_len.to(dev)
    par, own = parent.to(dev), (owner.to(dev) if cfg.C else None)
    out = torch.full_like(t["q"], float("nan"))
    lse = torch.full((cfg.B, cfg.R, cfg.Hq), float("nan"), dtype=torch.float32, device=dev) if want_lse else None
    status = torch.zeros(max(cfg.B, 1), dtype=torch.int32, device=dev)
    plan = None
    if use_plan:
        plan = torch.empty(cb.confu_plan_bytes(gpu.ctx, dims), dtype=torch.uint8, device=dev)
        cb.confu_tree_plan(gpu.ctx, dims, ss, pl, par, own, plan, status)
        par_arg, own_arg = None, None
    else:
        par_arg, own_arg = par, own
    cb.confu_tree_attention(gpu.ctx, dims, t["q"], t["k_cache"], t["v_cache"], n_slots, ss, pl, t["k_soft"],
                            t["v_soft"], par_arg, own_arg, plan, out, lse, status)
    torch.cuda.synchronize()
    return out.cpu(), (lse.cpu() if want_lse else None), status.cpu()[:cfg.B]


def oracle_attention(cfg, t, seq_start, prefix_len, parent, owner, sm_scale=0.0):
    c = {k: (None if v is None else v.cpu()) for k, v in t.items()}
    return ref.tree_attention(c["q"], c["k_cache"], c["v_cache"], seq_start, prefix_len, c["k_soft"], c["v_soft"],
                              parent, owner, sm_scale=sm_scale)


def assert_attention_close(got, got_lse, want, want_lse, dtype, what=""):
    atol, rtol, ltol = TOL[dtype]
    B = want.shape[0]
    for b in range(B):
        g, w = got[b].double(), want[b]
        assert torch.isfinite(g).all(), f"{what}: non-finite output in sequence {b}"
        err = (g - w).abs().max().item()
        ref_max = w.abs().max().item()
        assert err <= atol, f"{what}: seq {b} max abs err {err:.3e} > {atol}"
        assert err <= rtol * ref_max, f"{what}: seq {b} max err {err:.3e} / max ref {ref_max:.3e} > {rtol}"
        if got_lse is not None:
            lerr = (got_lse[b].double() - want_lse[b]).abs().max().item()
            assert lerr <= ltol, f"{what}: seq {b} lse err {lerr:.3e} > {ltol}"


def setup_case(cfg, layer=0, device="cuda", tree_key_gain=1.0, pad_slots=0):
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen, pad_slots=pad_slots)
    t = inputs.layer_tensors(cfg, layer, n_slots, device=device, tree_key_gain=tree_key_gain, seq_start=seq_start,
                             prefix_len=plen)
    return parent, owner, plen, seq_start, n_slots, t


# ------------------------------------------------------------------------------- acceptance
def gpu_accept(gpu, cfg, tl, dl, tok, parent, owner, u, temperature, mode=1):
    dev = "cuda"
    B, T, V = tl.shape
    Cn = 0 if owner is None else owner.shape[1]
    o = {
        "accept_len": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "path": torch.full((B, cb.MAX_DEPTH + 1), -7, dtype=torch.int32, device=dev),
        "next_token": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "future_row": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "counters": torch.full((B, 4), -7, dtype=torch.int32, device=dev),
        "status": torch.zeros(B, dtype=torch.int32, device=dev),
    }
    ws = torch.empty(cb.confu_accept_workspace_bytes(B, T, V), dtype=torch.uint8, device=dev)
    cb.confu_tree_accept(gpu.ctx, B, T, Cn, V, tl.dtype, tl.to(dev), None if dl is None else dl.to(dev),
                         tok.to(dev), parent.to(dev), owner.to(dev) if Cn else None,
                         None if u is None else u.to(dev), temperature, mode, o["accept_len"], o["path"],
                         o["next_token"], o["future_row"], o["counters"], ws, o["status"])
    torch.cuda.synchronize()
    return {k: v.cpu() for k, v in o.items()}


def compare_accept(got, want, log=None):
    """Bit-exact comparison of accepted path, next token and future row, except where the oracle
    reports a borderline decision (|ratio - u| < 1e-5, or the final draw within 1e-5 of a CDF cell
    edge with the GPU picking the neighbouring cell): those sequences are counted, not compared
    further.  Returns (n_exact, n_borderline)."""
    B = want["accept_len"].shape[0]
    exact = border = 0
    for b in range(B):
        assert got["status"][b].item() == want["status"][b].item(), (b, got["status"][b], want["status"][b])
        same_path = (got["accept_len"][b] == want["accept_len"][b]) and torch.equal(got["path"][b], want["path"][b])
        if not same_path:
            assert want["ratio_margin"][b].item() < BORDERLINE, \
                f"seq {b}: path differs (gpu {got['path'][b][:8].tolist()} vs {want['path'][b][:8].tolist()}) " \
                f"with margin {want['ratio_margin'][b].item():.3e}"
            border += 1
            if log is not None:
                log.append(("ratio", b, want["ratio_margin"][b].item()))
            continue
        assert got["future_row"][b].item() == want["future_row"][b].item(), b
        if got["next_token"][b].item() != want["next_token"][b].item():
            ok = want["resample_margin"][b].item() < BORDERLINE and \
                got["next_token"][b].item() in want["alt_token"][b].tolist()
            assert ok, f"seq {b}: next token {got['next_token'][b].item()} vs {want['next_token'][b].item()} " \
                       f"(margin {want['resample_margin'][b].item():.3e})"
            border += 1
            if log is not None:
                log.append(("resample", b, want["resample_margin"][b].item()))
            continue
        assert got["counters"][b, :2].tolist() == want["counters"][b, :2].tolist(), b
        exact += 1
    return exact, border


def gpu_accept_match(gpu, cfg, tl, tok, parent, owner, u, temperature):
    dev = "cuda"
    B, T, V = tl.shape
    Cn = 0 if owner is None else owner.shape[1]
    o = {
        "accept_len": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "path": torch.full((B, cb.MAX_DEPTH + 1), -7, dtype=torch.int32, device=dev),
        "next_token": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "future_row": torch.full((B,), -7, dtype=torch.int32, device=dev),
        "counters": torch.full((B, 4), -7, dtype=torch.int32, device=dev),
        "status": torch.zeros(B, dtype=torch.int32, device=dev),
    }
    cb.confu_tree_accept_match(gpu.ctx, B, T, Cn, V, tl.dtype, tl.to(dev), tok.to(dev), parent.to(dev),
                               owner.to(dev) if Cn else None, None if u is None else u.to(dev), temperature,
                               o["accept_len"], o["path"], o["next_token"], o["future_row"], o["counters"], o["status"])
    torch.cuda.synchronize()
    return {k: v.cpu() for k, v in o.items()}


def compare_match(got, want, log=None):
    """Sample-and-match walk: everything bit-exact, except sequences in which some draw fell within
    BORDERLINE of an edge of its CDF cell (the oracle reports the smallest such distance): there a
    neighbouring token is an equally valid draw and the rest of the walk may differ; those sequences
    are counted, not compared further.  Returns (n_exact, n_borderline)."""
    B = want["accept_len"].shape[0]
    exact = border = 0
    for b in range(B):
        assert got["status"][b].item() == want["status"][b].item(), (b, got["status"][b], want["status"][b])
        same = all(torch.equal(got[k][b], want[k][b]) for k in ("accept_len", "path", "next_token", "future_row"))
        if not same:
            assert want["draw_margin"][b].item() < BORDERLINE, \
                f"seq {b}: gpu {got['path'][b][:8].tolist()} -> {got['next_token'][b].item()} vs " \
                f"{want['path'][b][:8].tolist()} -> {want['next_token'][b].item()}, margin {want['draw_margin'][b].item():.3e}"
            border += 1
            if log is not None:
                log.append((b, want["draw_margin"][b].item()))
            continue
        assert got["counters"][b, :2].tolist() == want["counters"][b, :2].tolist(), b
        exact += 1
    return exact, border
