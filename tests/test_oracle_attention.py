"""Pins of the oracle's tree attention against things other than itself.

Each test would fail for a plausible mistake in oracle/confu_ref.c: a wrong
ancestor walk, a contemplate row seeing too much or too little, soft prompts
leaking to tree rows, a transposed head mapping, a dropped scale, a wrong slot
offset.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_mask_example():
    parent = owner = None
    rows = {}
    for line in open(os.path.join(GOLDEN, "mask_example.txt")):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        head, vals = line.split(":")
        vals = [int(x) for x in vals.split()]
        if head.startswith("parent"):
            parent = vals
        elif head.startswith("owner"):
            owner = vals
        else:
            rows[int(head.split()[1])] = vals
    vis = np.array([rows[r] for r in range(len(rows))], dtype=bool)
    return np.array(parent, np.int32), np.array(owner, np.int32), vis


def _closure_visibility(parent, owner):
    """Tree-slot visibility by a different route than the oracle's parent walk:
    reflexive-transitive closure of the child->parent relation by boolean matrix powers."""
    T, C = len(parent), len(owner)
    R = T + C
    A = np.eye(T, dtype=bool)
    for i in range(1, T):
        A[i, parent[i]] = True
    reach = A.copy()
    for _ in range(T):
        reach = (reach.astype(np.int64) @ A.astype(np.int64)) > 0
    vis = np.zeros((R, R), dtype=bool)
    vis[:T, :T] = reach
    for k in range(C):
        vis[T + k, :T] = reach[owner[k]]
        vis[T + k, T + k] = True
    return vis


def _dense_attention(q, k_cache, v_cache, seq_start, prefix_len, k_soft, v_soft, vis_list, T, scale=None):
    """Brute force: materialise the whole score matrix, put -inf where the mask says no, normalise.
    vis_list[b] is the R x R tree-slot visibility of sequence b, supplied by the caller."""
    q, k_cache, v_cache = q.double().numpy(), k_cache.double().numpy(), v_cache.double().numpy()
    B, R, Hq, D = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    S = 0 if k_soft is None else k_soft.shape[0]
    scale = scale or 1.0 / math.sqrt(D)
    out = np.zeros((B, R, Hq, D))
    lse = np.zeros((B, R, Hq))
    for b in range(B):
        P, s0 = int(prefix_len[b]), int(seq_start[b])
        keys = k_cache[s0:s0 + P + R]
        vals = v_cache[s0:s0 + P + R]
        if S:
            keys = np.concatenate([k_soft.double().numpy(), keys], 0)
            vals = np.concatenate([v_soft.double().numpy(), vals], 0)
        mask = np.zeros((R, S + P + R), dtype=bool)
        mask[T:, :S] = True
        mask[:, S:S + P] = True
        mask[:, S + P:] = vis_list[b]
        for h in range(Hq):
            g = h // G
            sc = (q[b, :, h, :] @ keys[:, g, :].T) * scale
            sc = np.where(mask, sc, -np.inf)
            m = sc.max(axis=1, keepdims=True)
            w = np.exp(sc - m)
            den = w.sum(axis=1, keepdims=True)
            out[b, :, h, :] = (w / den) @ vals[:, g, :]
            lse[b, :, h] = (m + np.log(den))[:, 0]
    return out, lse


def _small_case(B=2, Hq=4, Hkv=2, D=16, T=8, C=2, S=2, P=(5, 16), tree="random", seed=11, dtype=torch.float64):
    cfg = inputs.VerifyConfig("t", B=B, L=1, Hq=Hq, Hkv=Hkv, D=D, T=T, C=C, S=S, V=16, prefix=P, tree=tree,
                              kv_dtype=dtype, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent",
                              temperatures=(1.0,), seed=seed, max_depth=4, fanout=(1, 3))
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen, pad_slots=3)
    t = inputs.layer_tensors(cfg, 0, n_slots)
    return cfg, parent, owner, plen, seq_start, t


def test_mask_golden_example():
    """All keys zero => output is the plain mean of the visible value rows; with a prefix of 0 and
    one-hot value rows the output *is* the visibility pattern, compared with the hand-derived one."""
    parent, owner, vis = _read_mask_example()
    T, C = len(parent), len(owner)
    R, D = T + C, 16
    S = 2
    q = torch.randn(1, R, 2, D, dtype=torch.float64)
    k = torch.zeros(R, 1, D, dtype=torch.float64)
    v = torch.zeros(R, 1, D, dtype=torch.float64)
    for j in range(R):
        v[j, 0, j] = 1.0                       # slot j marks coordinate j
    ks = torch.zeros(S, 1, D, dtype=torch.float64)
    vs = torch.zeros(S, 1, D, dtype=torch.float64)
    vs[0, 0, R] = 1.0
    vs[1, 0, R + 1] = 1.0
    out, lse, st = ref.tree_attention(q, k, v, torch.tensor([0]), torch.tensor([0]), ks, vs,
                                      torch.from_numpy(parent)[None], torch.from_numpy(owner)[None])
    assert st.tolist() == [0]
    for r in range(R):
        n_vis = vis[r].sum() + (S if r >= T else 0)
        want = np.zeros(D)
        want[:R] = vis[r] / n_vis
        if r >= T:
            want[R:R + S] = 1.0 / n_vis
        for h in range(2):
            np.testing.assert_allclose(out[0, r, h].numpy(), want, atol=1e-15)
            assert abs(lse[0, r, h].item() - math.log(n_vis)) < 1e-14


def test_closure_matches_golden():
    parent, owner, vis = _read_mask_example()
    assert (_closure_visibility(parent, owner) == vis).all()


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_brute_force_dense_mask(seed):
    cfg, parent, owner, plen, seq_start, t = _small_case(seed=seed)
    vis = [_closure_visibility(parent[b].numpy(), owner[b].numpy()) for b in range(cfg.B)]
    want, want_lse = _dense_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen,
                                      t["k_soft"], t["v_soft"], vis, cfg.T)
    out, lse, st = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen,
                                      t["k_soft"], t["v_soft"], parent, owner)
    assert st.tolist() == [0] * cfg.B
    np.testing.assert_allclose(out.numpy(), want, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(lse.numpy(), want_lse, rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_narrow_inputs_are_widened_exactly(dtype):
    cfg, parent, owner, plen, seq_start, t = _small_case(seed=21, dtype=dtype)
    wide = {k: (None if x is None else x.double()) for k, x in t.items()}
    a = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    b = ref.tree_attention(wide["q"], wide["k_cache"], wide["v_cache"], seq_start, plen, wide["k_soft"],
                           wide["v_soft"], parent, owner)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_chain_tree_is_causal_attention():
    """A chain-shaped tree with no contemplate rows and no soft prompts is causal attention of the
    last T positions over P+T keys: compared with the library's scaled_dot_product_attention."""
    cfg, parent, owner, plen, seq_start, t = _small_case(B=2, T=7, C=0, S=0, P=(3, 12), tree="chain", seed=5)
    out, _, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, None, None, parent, owner)
    G = cfg.Hq // cfg.Hkv
    for b in range(cfg.B):
        P, s0 = int(plen[b]), int(seq_start[b])
        n = P + cfg.T
        keys = t["k_cache"][s0:s0 + n].permute(1, 0, 2).repeat_interleave(G, 0)     # [Hq, n, D]
        vals = t["v_cache"][s0:s0 + n].permute(1, 0, 2).repeat_interleave(G, 0)
        # full causal problem over n positions; queries of the first P positions are dummies
        qfull = torch.zeros(cfg.Hq, n, cfg.D, dtype=torch.float64)
        qfull[:, P:, :] = t["q"][b].permute(1, 0, 2)
        want = torch.nn.functional.scaled_dot_product_attention(qfull, keys, vals, is_causal=True)[:, P:, :]
        np.testing.assert_allclose(out[b].permute(1, 0, 2).numpy(), want.numpy(), rtol=1e-11, atol=1e-12)


def test_star_tree_rows_see_prefix_root_self():
    cfg, parent, owner, plen, seq_start, t = _small_case(B=1, T=6, C=0, S=0, P=9, tree="star", seed=6)
    out, lse, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, None, None, parent, owner)
    G = cfg.Hq // cfg.Hkv
    P = 9
    for r in range(cfg.T):
        idx = list(range(P)) + sorted({P, P + r})
        for h in range(cfg.Hq):
            k = t["k_cache"][idx, h // G]
            v = t["v_cache"][idx, h // G]
            s = (k @ t["q"][0, r, h]) / math.sqrt(cfg.D)
            w = torch.softmax(s, 0)
            np.testing.assert_allclose(out[0, r, h].numpy(), (w @ v).numpy(), rtol=1e-12, atol=1e-13)
            assert abs(lse[0, r, h].item() - torch.logsumexp(s, 0).item()) < 1e-12


def test_single_query_decode_special_case():
    cfg, parent, owner, plen, seq_start, t = _small_case(B=2, T=1, C=0, S=0, P=(4, 20), seed=8)
    out, _, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, None, None, parent, owner)
    G = cfg.Hq // cfg.Hkv
    for b in range(2):
        s0, n = int(seq_start[b]), int(plen[b]) + 1
        for h in range(cfg.Hq):
            s = (t["k_cache"][s0:s0 + n, h // G] @ t["q"][b, 0, h]) / math.sqrt(cfg.D)
            want = torch.softmax(s, 0) @ t["v_cache"][s0:s0 + n, h // G]
            np.testing.assert_allclose(out[b, 0, h].numpy(), want.numpy(), rtol=1e-12, atol=1e-13)


def test_tree_rows_ignore_soft_prompts_and_contemplate_rows():
    """Only contemplate rows attend to the soft prompts; tree rows must come out bit-identical
    whatever the soft-prompt values are and whether contemplate rows exist at all."""
    cfg, parent, owner, plen, seq_start, t = _small_case(B=1, T=8, C=2, S=2, P=10, seed=9)
    a, la, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    b, lb, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"] * 7 + 1,
                                  t["v_soft"] * -3, parent, owner)
    assert torch.equal(a[:, :cfg.T], b[:, :cfg.T]) and torch.equal(la[:, :cfg.T], lb[:, :cfg.T])
    assert not torch.equal(a[:, cfg.T:], b[:, cfg.T:])
    # same tree without contemplate rows / soft prompts: the tree slots sit at the same cache offsets
    c, lc, _ = ref.tree_attention(t["q"][:, :cfg.T].contiguous(), t["k_cache"], t["v_cache"], seq_start, plen,
                                  None, None, parent, owner[:, :0])
    assert torch.equal(a[:, :cfg.T], c) and torch.equal(la[:, :cfg.T], lc)


def test_contemplate_row_equals_single_query_over_its_set():
    cfg, parent, owner, plen, seq_start, t = _small_case(B=1, T=8, C=2, S=2, P=10, seed=10)
    out, _, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    G = cfg.Hq // cfg.Hkv
    P = 10
    par = parent[0].tolist()
    for k in range(cfg.C):
        r = cfg.T + k
        branch = []
        a = int(owner[0, k])
        while a >= 0:
            branch.append(a)
            a = par[a]
        idx = list(range(P)) + [P + j for j in sorted(branch)] + [P + r]
        for h in range(cfg.Hq):
            g = h // G
            keys = torch.cat([t["k_soft"][:, g], t["k_cache"][idx, g]], 0)
            vals = torch.cat([t["v_soft"][:, g], t["v_cache"][idx, g]], 0)
            w = torch.softmax((keys @ t["q"][0, r, h]) / math.sqrt(cfg.D), 0)
            np.testing.assert_allclose(out[0, r, h].numpy(), (w @ vals).numpy(), rtol=1e-12, atol=1e-13)


def test_relabelling_nodes_permutes_outputs():
    """Another topological numbering of the same tree only permutes the rows."""
    cfg, parent, owner, plen, seq_start, t = _small_case(B=1, T=8, C=2, S=2, P=6, seed=14)
    par = parent[0].tolist()
    T, R, P = cfg.T, cfg.R, 6
    # new order: depth-first preorder (also topological)
    kids = {i: [j for j in range(T) if par[j] == i] for i in range(T)}
    order, stack = [], [0]
    while stack:
        u = stack.pop()
        order.append(u)
        stack.extend(reversed(kids[u]))
    assert sorted(order) == list(range(T)) and order != list(range(T))
    new_of = {old: new for new, old in enumerate(order)}
    parent2 = torch.tensor([[-1 if par[old] < 0 else new_of[par[old]] for old in order]], dtype=torch.int32)
    owner2 = torch.tensor([[new_of[int(o)] for o in owner[0]]], dtype=torch.int32)
    rows = order + list(range(T, R))                     # new row i holds old row rows[i]
    q2 = t["q"][:, rows].contiguous()
    k2, v2 = t["k_cache"].clone(), t["v_cache"].clone()
    k2[P:P + R] = t["k_cache"][[P + j for j in rows]]
    v2[P:P + R] = t["v_cache"][[P + j for j in rows]]
    a, la, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    b, lb, st = ref.tree_attention(q2, k2, v2, seq_start, plen, t["k_soft"], t["v_soft"], parent2, owner2)
    assert st.tolist() == [0]
    np.testing.assert_allclose(b.numpy(), a[:, rows].numpy(), rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lb.numpy(), la[:, rows].numpy(), rtol=1e-12, atol=1e-14)


def test_scale_override_and_default():
    cfg, parent, owner, plen, seq_start, t = _small_case(B=1, T=4, C=1, S=1, P=5, seed=15)
    vis = [_closure_visibility(parent[0].numpy(), owner[0].numpy())]
    want, _ = _dense_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], vis, cfg.T, scale=0.37)
    out, _, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner, sm_scale=0.37)
    np.testing.assert_allclose(out.numpy(), want, rtol=1e-12, atol=1e-13)


def test_selected_rows_equal_full_tensor():
    cfg, parent, owner, plen, seq_start, t = _small_case(seed=16)
    out, lse, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    sel = [(0, 0, 0), (1, 9, 3), (0, 5, 2), (1, 3, 1)]
    o2, l2 = ref.tree_attention_rows(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner, sel)
    for i, (b, r, h) in enumerate(sel):
        assert torch.equal(o2[i], out[b, r, h]) and l2[i] == lse[b, r, h]


def test_bad_tree_is_reported():
    cfg, parent, owner, plen, seq_start, t = _small_case(seed=17)
    bad = parent.clone()
    bad[1, 3] = 5                      # parent index not below the node
    _, _, st = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], bad, owner)
    assert st.tolist() == [ref.ST_OK, ref.ST_BAD_PARENT]
    bad_owner = owner.clone()
    bad_owner[0, 0] = cfg.T
    _, _, st = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, bad_owner)
    assert st.tolist() == [ref.ST_BAD_OWNER, ref.ST_OK]
