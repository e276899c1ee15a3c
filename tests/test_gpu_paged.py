"""Paged cache pools (confu_set_paging): attention, append and compaction through a block table give
what the packed layout gives.  The oracle only knows the packed layout (the definition); the test
scatters the packed pool into randomly ordered pages of 128 slots for the GPU."""
import math

import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs
from tests import harness as H

pytestmark = pytest.mark.gpu
PAGE = 128


def _cfg(**kw):
    base = dict(B=3, L=1, Hq=8, Hkv=2, D=128, T=20, C=6, S=4, V=32, prefix=(1, 700), tree="random",
                kv_dtype=torch.bfloat16, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent",
                temperatures=(1.0,), seed=91, max_depth=6, fanout=(1, 3))
    base.update(kw)
    return inputs.VerifyConfig("paged", **base)


def _page_layout(cfg, plen, seed):
    """Random block table: [B, max_pages] page ids, pages of a sequence in no particular order."""
    g = torch.Generator().manual_seed(seed)
    need = [math.ceil((int(p) + cfg.R) / PAGE) for p in plen]
    n_pages = sum(need) + 3
    perm = torch.randperm(n_pages, generator=g).tolist()
    max_pages = max(need) + 1
    table = torch.zeros(cfg.B, max_pages, dtype=torch.int32)
    for b in range(cfg.B):
        for i in range(need[b]):
            table[b, i] = perm.pop()
    return table, n_pages, max_pages


def _scatter(packed, seq_start, plen, R, table, n_pages, upto_rows=True):
    """Copy each sequence's slots (prefix + R rows if upto_rows) from the packed pool into its pages."""
    pool = torch.zeros(n_pages * PAGE, *packed.shape[1:], dtype=packed.dtype, device=packed.device)
    for b in range(table.shape[0]):
        n = int(plen[b]) + (R if upto_rows else 0)
        for s0 in range(0, n, PAGE):
            m = min(PAGE, n - s0)
            page = int(table[b, s0 // PAGE])
            pool[page * PAGE:page * PAGE + m] = packed[int(seq_start[b]) + s0:int(seq_start[b]) + s0 + m]
    return pool


def _gather(pool, seq_start, lens, table, like):
    out = like.clone()
    for b in range(table.shape[0]):
        for s0 in range(0, int(lens[b]), PAGE):
            m = min(PAGE, int(lens[b]) - s0)
            page = int(table[b, s0 // PAGE])
            out[int(seq_start[b]) + s0:int(seq_start[b]) + s0 + m] = pool[page * PAGE:page * PAGE + m]
    return out


@pytest.mark.parametrize("name,cfg", [
    ("bf16_tensor_core", _cfg()),
    ("bf16_rows_100", _cfg(T=50, C=50, seed=92, max_depth=7, fanout=(1, 4))),
    ("fp32_generic", _cfg(kv_dtype=torch.float32, D=64, seed=93)),
])
def test_paged_attention_append_and_compaction_match_the_packed_layout(name, cfg):
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
    table, n_pages, max_pages = _page_layout(cfg, plen, seed=cfg.seed)
    # pools hold the prefixes only; the step's own rows arrive through confu_kv_append
    k_pool = _scatter(t["k_cache"], seq_start, plen, cfg.R, table, n_pages, upto_rows=False)
    v_pool = _scatter(t["v_cache"], seq_start, plen, cfg.R, table, n_pages, upto_rows=False)
    rows = torch.cat([torch.arange(int(seq_start[b]) + int(plen[b]), int(seq_start[b]) + int(plen[b]) + cfg.R)
                      for b in range(cfg.B)]).cuda()
    k_rows = t["k_cache"][rows].view(cfg.B, cfg.R, cfg.Hkv, cfg.D).contiguous()
    v_rows = t["v_cache"][rows].view(cfg.B, cfg.R, cfg.Hkv, cfg.D).contiguous()

    gpu = H.Gpu()
    try:
        dims = H.dims_of(cfg)
        gpu.ensure_ws(dims)
        d_table, d_plen = table.cuda(), plen.cuda()
        cb.confu_set_paging(gpu.ctx, d_table, max_pages)
        cb.confu_kv_append(gpu.ctx, dims, k_rows, v_rows, k_pool, v_pool, None, d_plen)
        out = torch.full_like(t["q"], float("nan"))
        lse = torch.full((cfg.B, cfg.R, cfg.Hq), float("nan"), dtype=torch.float32, device="cuda")
        status = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        cb.confu_tree_attention(gpu.ctx, dims, t["q"], k_pool, v_pool, n_pages * PAGE, None, d_plen, t["k_soft"],
                                t["v_soft"], parent.cuda(), owner.cuda(), None, out, lse, status)
        torch.cuda.synchronize()
        assert status.cpu().tolist() == [0] * cfg.B
        H.assert_attention_close(out.cpu(), lse.cpu(), want, want_lse, cfg.kv_dtype, name)

        # compaction of an arbitrary valid path per sequence, against the oracle on the packed pool
        accept_len = torch.zeros(cfg.B, dtype=torch.int32)
        path = torch.full((cfg.B, cb.MAX_DEPTH + 1), -1, dtype=torch.int32)
        for b in range(cfg.B):
            node, chain = cfg.T - 1 - b, []                  # root-to-node path of some deep node
            while node >= 0:
                chain.append(node)
                node = int(parent[b, node])
            chain.reverse()
            accept_len[b] = len(chain) - 1
            path[b, :len(chain)] = torch.tensor(chain, dtype=torch.int32)
        kh, vh = t["k_cache"].cpu().clone(), t["v_cache"].cpu().clone()
        new_len = ref.kv_compact([kh], [vh], seq_start, plen, accept_len, path)
        kp = torch.tensor([k_pool.data_ptr()], dtype=torch.int64, device="cuda")
        vp = torch.tensor([v_pool.data_ptr()], dtype=torch.int64, device="cuda")
        new_plen = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        cb.confu_kv_compact(gpu.ctx, dims, 1, kp, vp, None, d_plen, accept_len.cuda(), path.cuda(), new_plen, status)
        torch.cuda.synchronize()
        assert new_plen.cpu().tolist() == new_len.tolist()
        got_k = _gather(k_pool.cpu(), seq_start, new_len, table, kh)
        got_v = _gather(v_pool.cpu(), seq_start, new_len, table, vh)
        for b in range(cfg.B):
            lo, hi = int(seq_start[b]), int(seq_start[b]) + int(new_len[b])
            assert torch.equal(got_k[lo:hi], kh[lo:hi]) and torch.equal(got_v[lo:hi], vh[lo:hi])
        # back to packed pools: the same context serves the packed layout again
        cb.confu_set_paging(gpu.ctx, None)
        out2, lse2, _ = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
        H.assert_attention_close(out2, lse2, want, want_lse, cfg.kv_dtype, name + " packed again")
    finally:
        gpu.close()


def test_paged_pool_must_be_whole_pages():
    cfg = _cfg()
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    gpu = H.Gpu()
    try:
        dims = H.dims_of(cfg)
        gpu.ensure_ws(dims)
        table = torch.zeros(cfg.B, 8, dtype=torch.int32, device="cuda")
        cb.confu_set_paging(gpu.ctx, table, 8)
        with pytest.raises(cb.ConfuError) as e:
            cb.confu_tree_attention(gpu.ctx, dims, t["q"], t["k_cache"], t["v_cache"], 1000, None, plen.cuda(),
                                    t["k_soft"], t["v_soft"], parent.cuda(), owner.cuda(), None, t["q"], None, None)
        assert e.value.code == -2
    finally:
        gpu.close()
