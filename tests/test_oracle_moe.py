"""Pins of the oracle's contemplate-token embedding (Sec. 3.2: router linear layer -> softmax ->
top-k experts -> sum of their embeddings weighted by the gating scores) against dense library
routines and closed forms."""
import math

import torch

from oracle import ref


def _case(B=5, H_in=48, H_out=24, n=12, seed=0, dtype=torch.float64, bias=True):
    g = torch.Generator().manual_seed(seed)
    h = torch.randn(B, H_in, generator=g, dtype=torch.float64).to(dtype)
    w = (torch.randn(n, H_in, generator=g, dtype=torch.float64) / math.sqrt(H_in) * 2).to(dtype)
    b = torch.randn(n, generator=g, dtype=torch.float64).to(dtype) if bias else None
    e = torch.randn(n, H_out, generator=g, dtype=torch.float64).to(dtype)
    return h, w, b, e


def _scores(h, w, b):
    lg = h.double() @ w.double().T
    if b is not None:
        lg = lg + b.double()
    return torch.softmax(lg, dim=1)


def test_all_experts_selected_is_the_dense_mixture():
    h, w, b, e = _case()
    out, sel, gate, gap = ref.con_embedding(h, w, b, e, k_expert=12)
    want = _scores(h, w, b) @ e.double()
    assert torch.allclose(out, want, rtol=1e-12, atol=1e-12)
    assert torch.isinf(gap).all() and torch.allclose(gate.sum(1), torch.ones(5, dtype=torch.float64))
    assert sorted(sel[0].tolist()) == list(range(12))


def test_top_k_against_torch_topk_and_gather():
    for seed, k, dtype, bias in ((1, 1, torch.float64, True), (2, 2, torch.float32, False), (3, 4, torch.bfloat16, True)):
        h, w, b, e = _case(seed=seed, dtype=dtype, bias=bias)
        out, sel, gate, gap = ref.con_embedding(h, w, b, e, k_expert=k)
        p = _scores(h, w, b)
        top = torch.topk(p, k, dim=1)
        assert torch.equal(sel.long(), top.indices)                  # largest first
        assert torch.allclose(gate, top.values, rtol=1e-12)
        want = torch.einsum("bk,bkd->bd", top.values, e.double()[top.indices])
        assert torch.allclose(out, want, rtol=1e-12, atol=1e-12)
        rest = p.clone().scatter_(1, top.indices, -1.0).max(1).values
        assert torch.allclose(gap, top.values[:, -1] - rest, rtol=1e-9, atol=1e-15)
        # renormalised weights: the same selection, weights summing to one
        out_r, sel_r, gate_r, _ = ref.con_embedding(h, w, b, e, k_expert=k, renormalize=True)
        assert torch.equal(sel_r, sel) and torch.allclose(gate_r.sum(1), torch.ones(5, dtype=torch.float64))
        assert torch.allclose(out_r, want / top.values.sum(1, keepdim=True), rtol=1e-12, atol=1e-12)


def test_one_hot_router_closed_form():
    n, c = 6, 3.0
    w = torch.eye(n, dtype=torch.float64) * c                       # H_in = n
    e = torch.arange(n * 4, dtype=torch.float64).reshape(n, 4)
    h = torch.eye(n, dtype=torch.float64)[[4, 1]]                   # hidden states e_4 and e_1
    out, sel, gate, gap = ref.con_embedding(h, w, None, e, k_expert=1)
    p_top = math.exp(c) / (math.exp(c) + n - 1)
    assert sel[:, 0].tolist() == [4, 1]
    assert torch.allclose(gate[:, 0], torch.full((2,), p_top, dtype=torch.float64), rtol=1e-14)
    assert torch.allclose(out, p_top * e[[4, 1]], rtol=1e-14)
    assert torch.allclose(gap, torch.full((2,), p_top - 1 / (math.exp(c) + n - 1), dtype=torch.float64), rtol=1e-12)


def test_equal_scores_take_the_lower_index_and_a_common_shift_changes_nothing():
    h, w, b, e = _case(n=8, seed=4)
    w[5] = w[2]; b[5] = b[2]                                        # experts 2 and 5 always score the same
    w[2] *= 0; w[5] *= 0; b[2] = b[5] = 50.0                        # ... and higher than everyone else
    out, sel, gate, gap = ref.con_embedding(h, w, b, e, k_expert=1)
    assert sel[:, 0].tolist() == [2] * 5 and gap.abs().max().item() == 0.0
    out2, sel2, _, _ = ref.con_embedding(h, w, b, e, k_expert=2)
    assert sel2.tolist() == [[2, 5]] * 5
    h, w, b, e = _case(seed=5)
    a = ref.con_embedding(h, w, b, e, k_expert=3)
    c = ref.con_embedding(h, w, b + 7.25, e, k_expert=3)            # softmax is shift invariant
    assert torch.equal(a[1], c[1]) and torch.allclose(a[0], c[0], rtol=1e-12, atol=1e-12)


def test_relabelling_the_experts_relabels_the_selection():
    h, w, b, e = _case(seed=6)
    perm = torch.randperm(12, generator=torch.Generator().manual_seed(1))
    a = ref.con_embedding(h, w, b, e, k_expert=3)
    c = ref.con_embedding(h, w[perm], b[perm], e[perm], k_expert=3)
    assert torch.equal(perm[c[1].long()], a[1].long()) and torch.allclose(a[0], c[0], rtol=1e-12, atol=1e-12)
