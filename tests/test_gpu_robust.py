"""GPU behaviour at the edges of the boundary: cache slots nobody wrote, malformed inputs that must
come back as status codes (never a fault), the device's own count of borderline decisions, and the
bounded device-side wait.  Expected values come from the oracle or from hand-computed cases; every
bad input is made on the host and is within what the kernels check for themselves."""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs
from tests import harness as H
from tests.test_gpu_paged import PAGE, _page_layout

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


@pytest.fixture(scope="module")
def gpu():
    g = H.Gpu()
    yield g
    g.close()


def _cfg(**kw):
    base = dict(B=3, L=1, Hq=8, Hkv=2, D=128, T=20, C=6, S=4, V=32, prefix=(1, 700), tree="random",
                kv_dtype=torch.bfloat16, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent",
                temperatures=(1.0,), seed=71, max_depth=6, fanout=(1, 3))
    base.update(kw)
    return inputs.VerifyConfig("robust", **base)


def _poison(shape, dtype, seed):
    """Bit patterns a never-written cache slot might hold: NaN, both infinities, huge finite values."""
    g = torch.Generator().manual_seed(seed)
    pick = torch.randint(0, 4, shape, generator=g)
    vals = torch.tensor([float("nan"), float("inf"), float("-inf"), 3.0e38], dtype=torch.float32)
    return vals[pick].to(dtype)


# ------------------------------------------------------------------ slots nobody wrote
@pytest.mark.parametrize("name,cfg", [
    ("bf16_tensor_core", _cfg()),
    ("bf16_rows_100", _cfg(T=50, C=50, seed=72, max_depth=7, fanout=(1, 4))),
    ("bf16_single_tile_sequences", _cfg(prefix=(1, 90), seed=73)),
    ("fp32_generic", _cfg(kv_dtype=torch.float32, D=64, seed=74)),
])
def test_packed_pool_with_poisoned_gaps(gpu, name, cfg):
    """Sequences lie apart in the pool; every slot that belongs to no sequence holds NaN / Inf / 3e38.
    A key tile of a sequence reaches into those slots; the outputs must not notice."""
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    gap = 150                                             # more than one key tile between sequences
    sizes = plen.to(torch.int64) + cfg.R
    seq_start = torch.zeros(cfg.B, dtype=torch.int64)
    seq_start[1:] = torch.cumsum(sizes + gap, 0)[:-1]
    seq_start += 7                                        # and the first sequence does not start at slot 0
    n_slots = int(seq_start[-1] + sizes[-1]) + 200
    t = inputs.layer_tensors(cfg, 0, n_slots, device="cpu")
    owned = torch.zeros(n_slots, dtype=torch.bool)
    for b in range(cfg.B):
        owned[int(seq_start[b]):int(seq_start[b] + sizes[b])] = True
    for key, seed in (("k_cache", 1), ("v_cache", 2)):
        bad = _poison(t[key].shape, t[key].dtype, seed)
        t[key] = torch.where(owned[:, None, None], t[key], bad)
    want, want_lse, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"],
                                           t["v_soft"], parent, owner)
    td = {k: (None if v is None else v.cuda()) for k, v in t.items()}
    paths = [cb.ATTENTION_AUTO] + ([cb.ATTENTION_TENSOR] if cfg.kv_dtype == torch.bfloat16 else []) + \
        ([cb.ATTENTION_TENSOR_PAIR] if cfg.kv_dtype == torch.bfloat16 and cfg.R > 32 else [])
    try:
        for path in paths:
            gpu.set_path(path)
            for use_plan in (False, True):
                out, lse, st = H.gpu_attention(gpu, cfg, td, seq_start, plen, parent, owner, n_slots, use_plan=use_plan)
                assert st.tolist() == [0] * cfg.B
                H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, f"{name} path {path}")
    finally:
        gpu.set_path(cb.ATTENTION_AUTO)


@pytest.mark.parametrize("name,cfg", [
    ("bf16_tensor_core", _cfg(seed=75)),
    ("fp32_generic", _cfg(kv_dtype=torch.float32, D=64, seed=76)),
])
def test_paged_pool_with_poisoned_page_tails(name, cfg):
    """Pages come from an uninitialised pool: the tail of every sequence's last page, and the pages no
    sequence owns, hold NaN / Inf bit patterns."""
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
    table, n_pages, max_pages = _page_layout(cfg, plen, seed=cfg.seed)
    pools = {}
    for key, seed in (("k_cache", 3), ("v_cache", 4)):
        pool = _poison((n_pages * PAGE, cfg.Hkv, cfg.D), cfg.kv_dtype, seed).cuda()
        for b in range(cfg.B):
            n = int(plen[b]) + cfg.R
            for s0 in range(0, n, PAGE):
                m = min(PAGE, n - s0)
                page = int(table[b, s0 // PAGE])
                pool[page * PAGE:page * PAGE + m] = t[key][int(seq_start[b]) + s0:int(seq_start[b]) + s0 + m]
        pools[key] = pool
    gpu = H.Gpu()
    try:
        dims = H.dims_of(cfg)
        gpu.ensure_ws(dims)
        d_table = table.cuda()
        cb.confu_set_paging(gpu.ctx, d_table, max_pages)
        out = torch.full_like(t["q"], float("nan"))
        lse = torch.full((cfg.B, cfg.R, cfg.Hq), float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        cb.confu_tree_attention(gpu.ctx, dims, t["q"], pools["k_cache"], pools["v_cache"], n_pages * PAGE, None,
                                plen.cuda(), t["k_soft"], t["v_soft"], parent.cuda(), owner.cuda(), None, out, lse,
                                status)
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0] * cfg.B
        H.assert_attention_close(out.cpu(), lse.cpu(), want, want_lse, cfg.kv_dtype, name)
    finally:
        gpu.close()


# ------------------------------------------------------------------ malformed trees
@pytest.mark.parametrize("cfg", [_cfg(seed=77), _cfg(T=40, C=40, seed=78, max_depth=7, fanout=(1, 4)),
                                 _cfg(kv_dtype=torch.float32, seed=79)], ids=["bf16", "bf16_rows_80", "fp32"])
def test_a_malformed_tree_gives_zero_rows_on_every_path(gpu, cfg):
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    bad = parent.clone()
    bad[1, 7] = 9                                         # parent index not below the node's own
    want, want_lse, want_st = H.oracle_attention(cfg, t, seq_start, plen, bad, owner)
    paths = [cb.ATTENTION_AUTO] + ([cb.ATTENTION_TENSOR] if cfg.kv_dtype == torch.bfloat16 else []) + \
        ([cb.ATTENTION_TENSOR_PAIR] if cfg.kv_dtype == torch.bfloat16 and cfg.R > 32 else [])
    try:
        for path in paths:
            gpu.set_path(path)
            for use_plan in (False, True):
                out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, bad, owner, n_slots, use_plan=use_plan)
                assert st.tolist() == want_st.tolist() == [0, 1, 0]
                assert (out[1] == 0).all() and (lse[1] == 0).all()
                keep = [0, 2]
                H.assert_attention_close(out[keep], lse[keep], want[keep], want_lse[keep], cfg.kv_dtype, "bad tree")
    finally:
        gpu.set_path(cb.ATTENTION_AUTO)


# ------------------------------------------------------------------ compaction with a bad path
def test_compaction_refuses_a_corrupted_path(gpu):
    B, Hkv, D, L, R, T = 5, 2, 128, 2, 24, 20
    g = torch.Generator().manual_seed(5)
    plen = torch.tensor([17, 3, 200, 64, 9], dtype=torch.int32)
    sizes = plen.to(torch.int64) + R
    seq_start = torch.zeros(B, dtype=torch.int64)
    seq_start[1:] = torch.cumsum(sizes, 0)[:-1]
    n_slots = int(sizes.sum())
    k = [torch.randn(n_slots, Hkv, D, generator=g).to(torch.bfloat16) for _ in range(L)]
    v = [torch.randn(n_slots, Hkv, D, generator=g).to(torch.bfloat16) for _ in range(L)]
    good = [0, 2, 5, 11]
    rows = [good,                     # fine
            [0, 5, 2, 11],            # not increasing
            [0, 2, 5, T],             # a node id past the tree
            [1, 2, 5, 11],            # does not start at the root
            good]                     # fine, but accept_len says 70 (> CONFU_MAX_DEPTH)
    path = torch.full((B, cb.MAX_DEPTH + 1), -1, dtype=torch.int32)
    for i, r in enumerate(rows):
        path[i, :len(r)] = torch.tensor(r, dtype=torch.int32)
    alen = torch.tensor([3, 3, 3, 3, 70], dtype=torch.int32)
    kd, vd = [x.cuda() for x in k], [x.cuda() for x in v]
    kp = torch.tensor([x.data_ptr() for x in kd], dtype=torch.int64, device="cuda")
    vp = torch.tensor([x.data_ptr() for x in vd], dtype=torch.int64, device="cuda")
    reg = []
    new_len = H.guarded(reg, (B,), torch.int32, -7)
    status = H.guarded(reg, (B,), torch.int32, 0)
    dims = cb.make_dims(B, Hkv, Hkv, D, T, R - T, 0, torch.bfloat16)
    cb.confu_kv_compact(gpu.ctx, dims, L, kp, vp, seq_start.cuda(), plen.cuda(), alen.cuda(), path.cuda(), new_len,
                        status)
    torch.cuda.synchronize()
    H.assert_guards(reg, "confu_kv_compact")
    assert status.cpu().tolist() == [0, cb.ST_BAD_PATH, cb.ST_BAD_PATH, cb.ST_BAD_PATH, cb.ST_BAD_PATH]
    assert new_len.cpu().tolist() == [17 + 4, 3 + 1, 200 + 1, 64 + 1, 9 + 1]
    # sequence 0 was compacted as the oracle does it; the refused sequences are untouched, byte for byte
    alen_ok = torch.tensor([3, 0, 0, 0, 0], dtype=torch.int32)
    ref.kv_compact(k, v, seq_start, plen, alen_ok, path)
    for l in range(L):
        assert torch.equal(kd[l].cpu(), k[l]) and torch.equal(vd[l].cpu(), v[l])


# ------------------------------------------------------------------ borderline counters on the device
@pytest.mark.parametrize("case", json.load(open(os.path.join(GOLDEN, "accept_hand_cases.json")))["cases"],
                         ids=lambda c: c["name"])
def test_hand_computed_cases_and_their_borderline_counts(gpu, case):
    """The hand-computed walks through the CUDA path (fp32 logits): decisions, and the device's own
    count of ratio tests and draws inside the 1e-5 band.  The planted margins (3e-6, 4e-6, 2e-5 and an
    exact edge) are far from the band's own edge compared with fp32 rounding of the probabilities."""
    p = np.asarray(case["p"], dtype=np.float64)
    q = np.asarray(case["q"], dtype=np.float64)
    with np.errstate(divide="ignore"):
        tl = torch.from_numpy(np.where(p > 0, np.log(np.where(p > 0, p, 1.0)), -1e4)).float()[None]
        dl = torch.from_numpy(np.where(q > 0, np.log(np.where(q > 0, q, 1.0)), -1e4)).float()[None]
    tok, par = torch.tensor([case["tokens"]], dtype=torch.int32), torch.tensor([case["parent"]], dtype=torch.int32)
    own = torch.tensor([case["owner"]], dtype=torch.int32)
    u = torch.tensor([case["u"]], dtype=torch.float32)
    got = H.gpu_accept(gpu, None, tl, dl, tok, par, own, u, 1.0, case["mode"])
    assert got["status"].tolist() == [0]
    exact_edge = case["resample_margin"] == 0.0           # the draw sits on a cell edge: either neighbour is right
    n = len(case["path"])
    assert got["accept_len"].tolist() == [case["accept_len"]] and got["path"][0, :n].tolist() == case["path"]
    if exact_edge:
        assert got["next_token"].item() in [case["next_token"]] + case["alt"]
    else:
        assert got["next_token"].tolist() == [case["next_token"]]
    assert got["future_row"].tolist() == [case["future_row"]]
    assert got["counters"][0].tolist() == [case["tests"], case["rejections"]] + case["borderline"]


def test_match_rule_counts_borderline_draws(gpu):
    # the hand-computed walk of the sample-and-match rule with its first draw 2e-6 above the edge .6
    p = np.asarray([[.1, .2, .3, .4], [.25, .25, .25, .25], [.5, .5, 0, 0], [.25, .25, .25, .25]])
    with np.errstate(divide="ignore"):
        tl = torch.from_numpy(np.where(p > 0, np.log(np.where(p > 0, p, 1.0)), -1e4)).float()[None]
    parent = torch.tensor([[-1, 0, 0, 2]], dtype=torch.int32)
    tokens = torch.tensor([[1, 2, 3, 0]], dtype=torch.int32)
    owner = torch.tensor([[2, 0]], dtype=torch.int32)
    for u0, border in ((.65, 0), (.600002, 1)):
        u = torch.tensor([[u0, .99, .4, .8]], dtype=torch.float32)
        got = H.gpu_accept_match(gpu, None, tl, tokens, parent, owner, u, 1.0)
        assert got["path"][0, :4].tolist() == [0, 2, 3, -1] and got["next_token"].tolist() == [3]
        assert got["counters"][0].tolist() == [3, 2, border, 0]


# ------------------------------------------------------------------ contemplate-token MoE, non-finite input
@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_moe_nonfinite_hidden_state_is_a_status_not_an_address(gpu, dtype):
    B, H_in, H_out, n, k = 4, 256, 64, 8, 2
    g = torch.Generator().manual_seed(9)
    h = torch.randn(B, H_in, generator=g).to(dtype)
    w = (torch.randn(n, H_in, generator=g) / 16).to(dtype)
    e = torch.randn(n, H_out, generator=g).to(dtype)
    want, wsel, wgate, _ = ref.con_embedding(h, w, None, e, k, False)
    h[1, 5] = float("nan")
    h[3, 0] = float("inf")
    reg = []
    out = H.guarded(reg, (B, H_out), dtype, float("nan"))
    sel = H.guarded(reg, (B, k), torch.int32, -7)
    gate = H.guarded(reg, (B, k), torch.float32, float("nan"))
    status = H.guarded(reg, (B,), torch.int32, 0)
    cb.confu_con_embedding(gpu.ctx, h.cuda(), w.cuda(), None, e.cuda(), k, False, out, sel, gate, status)
    torch.cuda.synchronize()
    H.assert_guards(reg, "confu_con_embedding")
    assert status.cpu().tolist() == [0, 5, 0, 5]
    for b in (1, 3):
        assert (out[b] == 0).all() and sel[b].tolist() == [0, 1] and (gate[b] == 0).all()
    tol = 1e-2 if dtype == torch.bfloat16 else 1e-5
    for b in (0, 2):
        assert sel[b].cpu().tolist() == wsel[b].tolist()
        assert (out[b].cpu().double() - want[b]).abs().max().item() <= tol * want[b].abs().max().item()


# ------------------------------------------------------------------ bounded device-side wait
def test_bounded_wait_gives_up_and_the_context_stays_usable(gpu):
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    cb.confu_selftest_bounded_wait(gpu.ctx, 2_000_000, status)       # nothing arrives: gives up after 2 ms
    t1.record()
    torch.cuda.synchronize()
    assert status.item() == cb.ST_TIMEOUT
    assert 1.5 <= t0.elapsed_time(t1) <= 200.0
    assert cb.lib().confu_status_string(cb.ST_TIMEOUT) == b"bounded device wait expired"
    with pytest.raises(cb.ConfuError):
        cb.confu_selftest_bounded_wait(gpu.ctx, 5_000_000_000, status)          # over the one-second cap
    # the limit of the attention kernels' own waits is an option of the context; with a short limit
    # an ordinary call still completes (no wait of a healthy kernel takes 50 ms) and matches the oracle
    cb.confu_set_option(gpu.ctx, cb.OPT_WAIT_LIMIT_NS, 50_000_000)
    try:
        cfg = _cfg(seed=80)
        parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
        out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
        want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
        assert st.tolist() == [0] * cfg.B
        H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, "after the timeout")
    finally:
        cb.confu_set_option(gpu.ctx, cb.OPT_WAIT_LIMIT_NS, 2_000_000_000)


def test_attention_path_option(gpu):
    cfg = _cfg(T=30, C=10, seed=81)                       # more than 32 query rows: every path can take it
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
    try:
        for path in (cb.ATTENTION_GENERIC, cb.ATTENTION_TENSOR, cb.ATTENTION_TENSOR_PAIR, cb.ATTENTION_AUTO):
            gpu.set_path(path)
            out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
            H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, f"path {path}")
        # a plan only fits the path it was built for: the kernel refuses it with a status, nothing is computed
        dims = H.dims_of(cfg)
        gpu.set_path(cb.ATTENTION_TENSOR)
        plan = torch.empty(cb.confu_plan_bytes(gpu.ctx, dims), dtype=torch.uint8, device="cuda")
        status = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        cb.confu_tree_plan(gpu.ctx, dims, seq_start.cuda(), plen.cuda(), parent.cuda(), owner.cuda(), plan, status)
        gpu.set_path(cb.ATTENTION_TENSOR_PAIR)
        out = torch.zeros_like(t["q"])
        cb.confu_tree_attention(gpu.ctx, dims, t["q"], t["k_cache"], t["v_cache"], n_slots, seq_start.cuda(), plen.cuda(),
                                t["k_soft"], t["v_soft"], None, None, plan, out, None, status)
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [cb.ST_BAD_PLAN] * cfg.B
        # a forced tensor-core path refuses dims it cannot take
        gpu.set_path(cb.ATTENTION_TENSOR)
        cfg32 = _cfg(kv_dtype=torch.float32, seed=82)
        p2, o2, pl2, ss2, ns2, t2 = H.setup_case(cfg32)
        with pytest.raises(cb.ConfuError) as e:
            H.gpu_attention(gpu, cfg32, t2, ss2, pl2, p2, o2, ns2)
        assert e.value.code == -5
    finally:
        gpu.set_path(cb.ATTENTION_AUTO)
