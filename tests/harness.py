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


# Red zones: every buffer the library writes into is cut out of a larger allocation whose margins
# hold a known byte pattern; after the call the margins must still hold it.  (The stand-in for a
# memory checker: an out-of-bounds store next to an output shows up here instead of corrupting a
# neighbouring tensor silently.)
GUARD_BYTES = 4096
GUARD_BYTE = 0xA5


class Guarded:
    """A CUDA tensor with guard bands on both sides."""

    def __init__(self, shape, dtype, fill=None):
        n = 1
        for d in (shape if isinstance(shape, (tuple, list, torch.Size)) else (shape,)):
            n *= int(d)
        nbytes = n * torch.empty(0, dtype=dtype).element_size()
        self.raw = torch.full((nbytes + 2 * GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device="cuda")
        self.t = self.raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(shape)
        self.nbytes = nbytes
        if fill is not None:
            self.t.fill_(fill)

    def intact(self):
        lo = self.raw[:GUARD_BYTES]
        hi = self.raw[GUARD_BYTES + self.nbytes:]
        return bool((lo == GUARD_BYTE).all().item()) and bool((hi == GUARD_BYTE).all().item())


def guarded(registry, shape, dtype, fill=None):
    g = Guarded(shape, dtype, fill)
    registry.append(g)
    return g.t


def assert_guards(registry, what=""):
    for i, g in enumerate(registry):
        assert g.intact(), f"{what}: a store went outside buffer {i} (shape {tuple(g.t.shape)}, {g.t.dtype})"


class Gpu:
    """A context plus a workspace (with guard bands) sized for the given dims."""

    def __init__(self):
        self.ctx = cb.confu_create(0)
        self.ws = None
        self.ws_guard = None

    def ensure_ws(self, dims):
        need = cb.confu_workspace_bytes(self.ctx, dims)
        if self.ws is None or self.ws.numel() != need:
            self.ws_guard = Guarded((need,), torch.uint8)
            self.ws = self.ws_guard.t
            cb.confu_set_workspace(self.ctx, self.ws)

    def ws_intact(self):
        return self.ws_guard is None or self.ws_guard.intact()

    def set_path(self, path):
        cb.confu_set_option(self.ctx, cb.OPT_ATTENTION_PATH, path)

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
    reg = []
    out = guarded(reg, t["q"].shape, t["q"].dtype, float("nan"))
    lse = guarded(reg, (cfg.B, cfg.R, cfg.Hq), torch.float32, float("nan")) if want_lse else None
    status = guarded(reg, (max(cfg.B, 1),), torch.int32, 0)
    plan = None
    if use_plan:
        plan = guarded(reg, (cb.confu_plan_bytes(gpu.ctx, dims),), torch.uint8)
        cb.confu_tree_plan(gpu.ctx, dims, ss, pl, par, own, plan, status)
        par_arg, own_arg = None, None
    else:
        par_arg, own_arg = par, own
    cb.confu_tree_attention(gpu.ctx, dims, t["q"], t["k_cache"], t["v_cache"], n_slots, ss, pl, t["k_soft"],
                            t["v_soft"], par_arg, own_arg, plan, out, lse, status)
    torch.cuda.synchronize()
    assert_guards(reg, "confu_tree_attention")
    assert gpu.ws_intact(), "confu_tree_attention: a store went outside the workspace"
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
    reg = []
    o = {
        "accept_len": guarded(reg, (B,), torch.int32, -7),
        "path": guarded(reg, (B, cb.MAX_DEPTH + 1), torch.int32, -7),
        "next_token": guarded(reg, (B,), torch.int32, -7),
        "future_row": guarded(reg, (B,), torch.int32, -7),
        "counters": guarded(reg, (B, 4), torch.int32, -7),
        "status": guarded(reg, (B,), torch.int32, 0),
    }
    ws = guarded(reg, (cb.confu_accept_workspace_bytes(B, T, V),), torch.uint8)
    cb.confu_tree_accept(gpu.ctx, B, T, Cn, V, tl.dtype, tl.to(dev), None if dl is None else dl.to(dev),
                         tok.to(dev), parent.to(dev), owner.to(dev) if Cn else None,
                         None if u is None else u.to(dev), temperature, mode, o["accept_len"], o["path"],
                         o["next_token"], o["future_row"], o["counters"], ws, o["status"])
    torch.cuda.synchronize()
    assert_guards(reg, "confu_tree_accept")
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
        # the device's own count of borderline decisions: zero wherever the oracle saw every decision
        # at least twice the band away from its threshold, and equal to the oracle's count unless a
        # decision sits so close to the band's own edge that fp32 normalisers may move it across
        if want["ratio_margin"][b].item() > 2 * BORDERLINE:
            assert got["counters"][b, 2].item() == 0, b
        if want["resample_margin"][b].item() > 2 * BORDERLINE or want["resample_margin"][b].item() == math.inf:
            assert got["counters"][b, 3].item() == 0, b
        elif want["resample_margin"][b].item() < 0.5 * BORDERLINE:
            assert got["counters"][b, 3].item() == 1, b
        exact += 1
    return exact, border


def gpu_accept_match(gpu, cfg, tl, tok, parent, owner, u, temperature):
    dev = "cuda"
    B, T, V = tl.shape
    Cn = 0 if owner is None else owner.shape[1]
    reg = []
    o = {
        "accept_len": guarded(reg, (B,), torch.int32, -7),
        "path": guarded(reg, (B, cb.MAX_DEPTH + 1), torch.int32, -7),
        "next_token": guarded(reg, (B,), torch.int32, -7),
        "future_row": guarded(reg, (B,), torch.int32, -7),
        "counters": guarded(reg, (B, 4), torch.int32, -7),
        "status": guarded(reg, (B,), torch.int32, 0),
    }
    cb.confu_tree_accept_match(gpu.ctx, B, T, Cn, V, tl.dtype, tl.to(dev), tok.to(dev), parent.to(dev),
                               owner.to(dev) if Cn else None, None if u is None else u.to(dev), temperature,
                               o["accept_len"], o["path"], o["next_token"], o["future_row"], o["counters"], o["status"])
    torch.cuda.synchronize()
    assert_guards(reg, "confu_tree_accept_match")
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
        if want["draw_margin"][b].item() > 2 * BORDERLINE:
            assert got["counters"][b, 2:].tolist() == [0, 0], b
        exact += 1
    return exact, border
