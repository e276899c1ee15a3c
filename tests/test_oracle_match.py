"""Pins of the oracle's sample-and-match acceptance (Sec. 2 steps 3-4 read literally) against things
other than itself: a hand-computed walk, the greedy walk it must reduce to at temperature 0, a
numpy walk built on cumsum / searchsorted, the closed forms "every emitted token follows the
target distribution" and "the root's draft is accepted with probability sum_x p(x) over its
children's tokens", and the rule that only rows on the walked path are read."""
from fractions import Fraction

import numpy as np
import pytest
import torch
from scipy import stats

from oracle import ref
from paper_2603_08899_b200 import inputs


def _logits_of(probs):
    p = np.asarray(probs, dtype=np.float64)
    with np.errstate(divide="ignore"):
        return torch.from_numpy(np.where(p > 0, np.log(np.where(p > 0, p, 1.0)), -1e4))


def test_hand_computed_walk():
    # node:   0 (root)   1 (tok 2, child of 0)   2 (tok 3, child of 0)   3 (tok 0, child of 2)
    # row 0: CDF edges .1 .3 .6 1.  -> u = .65 draws token 3 = node 2;  row 2: (.5 .5 0 0), u = .4 draws
    # token 0 = node 3;  row 3 (a leaf): uniform, u = .8 draws token 3, the bonus token.
    p = [[.1, .2, .3, .4], [.25, .25, .25, .25], [.5, .5, 0, 0], [.25, .25, .25, .25]]
    tl = _logits_of(p)[None]
    parent = torch.tensor([[-1, 0, 0, 2]])
    tokens = torch.tensor([[9 % 4, 2, 3, 0]])
    owner = torch.tensor([[2, 0]])                        # contemplate rows 4 (of node 2) and 5 (of the root)
    u = torch.tensor([[.65, .99, .4, .8]], dtype=torch.float64)
    o = ref.tree_accept_match(tl, tokens, parent, owner, u, temperature=1.0)
    assert o["status"].tolist() == [0]
    assert o["accept_len"].tolist() == [2] and o["path"][0, :4].tolist() == [0, 2, 3, -1]
    assert o["next_token"].tolist() == [3]
    assert o["future_row"].tolist() == [4]               # node 3 has none: nearest ancestor that has is node 2
    assert o["counters"][0, :2].tolist() == [3, 2]
    # how close the draws came to an edge of their cells: .65 in [.6, 1) -> .05; .4 in [0, .5) -> .1;
    # .8 in [.75, 1) -> .05.  Smallest .05, none inside the 1e-5 band; around the last drawn token 3 of
    # the uniform row: token 2 below, nothing above.
    assert o["draw_margin"].item() == pytest.approx(0.05, abs=1e-12)
    assert o["counters"][0, 2:].tolist() == [0, 0] and o["alt_token"][0].tolist() == [2, -1]
    # the first draw misses every child: nothing accepted, the drawn token itself is emitted
    u2 = torch.tensor([[.05, .99, .4, .8]], dtype=torch.float64)
    o2 = ref.tree_accept_match(tl, tokens, parent, owner, u2, temperature=1.0)
    assert o2["accept_len"].tolist() == [0] and o2["next_token"].tolist() == [0] and o2["future_row"].tolist() == [5]
    assert o2["draw_margin"].item() == pytest.approx(0.05, abs=1e-12) and o2["alt_token"][0].tolist() == [-1, 1]
    # a draw 2e-6 above the edge .6 of the root's row: still token 3 = node 2, counted as borderline
    u3 = torch.tensor([[.600002, .99, .4, .8]], dtype=torch.float64)
    o3 = ref.tree_accept_match(tl, tokens, parent, owner, u3, temperature=1.0)
    assert o3["path"][0, :3].tolist() == [0, 2, 3] and o3["counters"][0].tolist() == [3, 2, 1, 0]
    assert o3["draw_margin"].item() == pytest.approx(2e-6, abs=1e-12)


def test_draw_margin_against_exact_rationals():
    """A star tree with rational target rows: every draw of the walk redone in exact arithmetic; the
    reported margin is the smallest distance of a draw to an edge of its cell."""
    rng = np.random.default_rng(3)
    V = 10
    n_two_draws = 0
    for trial in range(50):
        rows = []
        for _ in range(4):
            w = rng.integers(0, 7, V)
            w[rng.integers(V)] += 1
            rows.append([Fraction(int(a), int(w.sum())) for a in w])
        kids = [int(t) for t in rng.choice(V, 3, replace=False)]
        us = [Fraction(int(rng.integers(0, 1 << 16)), 1 << 16) + Fraction(1, 1 << 20) for _ in range(4)]
        cur, margins = 0, []
        while True:
            c, x = Fraction(0), None
            for k in range(V):
                lo, c = c, c + rows[cur][k]
                if c > us[cur]:
                    x = k
                    break
            margins.append(min(us[cur] - lo, c - us[cur]))
            if cur == 0 and x in kids:
                cur = 1 + kids.index(x)
                continue
            break
        tl = _logits_of([[float(a) for a in r] for r in rows])[None]
        o = ref.tree_accept_match(tl, torch.tensor([[0] + kids]), torch.tensor([[-1, 0, 0, 0]]), None,
                                  torch.tensor([[float(u) for u in us]], dtype=torch.float64), temperature=1.0)
        assert o["accept_len"].item() == (1 if cur else 0) and o["next_token"].item() == x
        assert o["counters"][0, 0].item() == len(margins)
        assert o["draw_margin"].item() == pytest.approx(float(min(margins)), abs=1e-12)
        n_two_draws += len(margins) == 2
    assert n_two_draws >= 8


def _random_case(T=14, V=40, B=6, seed=11, dtype=torch.float32, sigma=2.0, tree="random"):
    cfg = inputs.VerifyConfig("m", B=B, L=1, Hq=2, Hkv=1, D=16, T=T, C=3, S=0, V=V, prefix=4, tree=tree,
                              kv_dtype=torch.float32, logit_dtype=dtype, sigma_logit=sigma, draft="noise",
                              temperatures=(1.0,), seed=seed, max_depth=5, fanout=(1, 3))
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, 1.0)      # distinct tokens among siblings
    u = inputs.uniforms(cfg)
    return cfg, parent, owner, tl, tok, u


def test_temperature_zero_is_the_greedy_walk():
    for seed in (11, 12, 13):
        cfg, parent, owner, tl, tok, u = _random_case(seed=seed, sigma=0.5)
        # make matches likely: every node's first child carries the target's argmax of the node's row
        for b in range(cfg.B):
            seen = set()
            for c in range(1, cfg.T):
                pa = parent[b, c].item()
                if pa not in seen:
                    seen.add(pa)
                    am = int(torch.argmax(tl[b, pa].double()).item())
                    sib = [j for j in range(1, cfg.T) if parent[b, j].item() == pa and j != c]
                    if all(tok[b, j].item() != am for j in sib):
                        tok[b, c] = am
        want = ref.tree_accept(tl, None, tok, parent, owner, None, temperature=0.0)
        got = ref.tree_accept_match(tl, tok, parent, owner, None, temperature=0.0)
        assert want["accept_len"].max().item() >= 2
        for k in ("accept_len", "path", "next_token", "future_row", "status"):
            assert torch.equal(got[k], want[k]), k


def _numpy_walk(tl, tok, parent, u, temperature):
    T, V = tl.shape
    cur, path = 0, [0]
    while True:
        z = tl[cur].astype(np.float64) / temperature
        w = np.exp(z - z.max())
        cdf = np.cumsum(w / w.sum())
        x = int(min(np.searchsorted(cdf, u[cur], side="right"), V - 1))
        hit = [c for c in range(cur + 1, T) if parent[c] == cur and tok[c] == x]
        if not hit:
            return path, x
        cur = hit[0]
        path.append(cur)


def test_numpy_cumsum_walk_agrees():
    n_long = 0
    for seed, temperature in ((21, 1.0), (22, 0.7), (23, 1.0), (24, 0.7), (25, 1.3)):
        cfg, parent, owner, tl, tok, u = _random_case(seed=seed, V=12, sigma=1.0, B=16)
        o = ref.tree_accept_match(tl, tok, parent, owner, u, temperature=temperature)
        for b in range(cfg.B):
            if o["draw_margin"][b].item() < 1e-9:
                continue
            path, x = _numpy_walk(tl[b].numpy(), tok[b].tolist(), parent[b].tolist(), u[b].double().numpy(), temperature)
            assert o["path"][b, :len(path)].tolist() == path and o["path"][b, len(path)].item() == -1
            assert o["accept_len"][b].item() == len(path) - 1 and o["next_token"][b].item() == x
            n_long += len(path) > 1
    assert n_long >= 10                                  # the comparison saw accepted drafts, not only misses


def test_emitted_token_follows_the_target_and_acceptance_rate_is_the_covered_mass():
    V, n = 10, 40000
    rng = np.random.default_rng(5)
    p = rng.dirichlet(np.ones(V))
    kids = [1, 4, 7]                                     # tokens of the root's three children (a star)
    tl = _logits_of(np.tile(p, (4, 1)))[None].repeat(n, 1, 1)
    parent = torch.tensor([[-1, 0, 0, 0]]).repeat(n, 1)
    tokens = torch.tensor([[0] + kids]).repeat(n, 1)
    u = torch.from_numpy(rng.random((n, 4)))
    o = ref.tree_accept_match(tl, tokens, parent, None, u, temperature=1.0)
    # first emitted token: the accepted child's token, else the next token
    first = torch.where(o["accept_len"] > 0, tokens.gather(1, o["path"][:, 1:2].clamp(min=0).long())[:, 0], o["next_token"])
    obs = np.bincount(first.numpy(), minlength=V)
    assert stats.chisquare(obs, p * n).pvalue > 1e-3
    rate = (o["accept_len"] > 0).double().mean().item()
    want = p[kids].sum()
    assert abs(rate - want) < 5 * np.sqrt(want * (1 - want) / n)
    # power: the same statistic rejects the draft's habit of emitting a fixed token
    assert stats.chisquare(np.bincount(np.full(n, kids[0]), minlength=V) + 1e-9, p * n).pvalue < 1e-6
    # temperature: tokens then follow p^(1/t) renormalised
    t = 0.5
    o = ref.tree_accept_match(tl, tokens, parent, None, u, temperature=t)
    first = torch.where(o["accept_len"] > 0, tokens.gather(1, o["path"][:, 1:2].clamp(min=0).long())[:, 0], o["next_token"])
    pt = p ** (1 / t) / (p ** (1 / t)).sum()
    assert stats.chisquare(np.bincount(first.numpy(), minlength=V), pt * n).pvalue > 1e-3
    assert stats.chisquare(np.bincount(first.numpy(), minlength=V), p * n).pvalue < 1e-6


def test_only_rows_on_the_walked_path_are_read():
    cfg, parent, owner, tl, tok, u = _random_case(seed=31, B=4)
    base = ref.tree_accept_match(tl, tok, parent, owner, u, temperature=1.0)
    for b in range(cfg.B):
        on_path = set(base["path"][b, :base["accept_len"][b].item() + 1].tolist())
        off = [i for i in range(cfg.T) if i not in on_path]
        bad = tl.clone()
        bad[b, off[0], 3] = float("inf")
        o = ref.tree_accept_match(bad, tok, parent, owner, u, temperature=1.0)
        assert o["status"][b].item() == 0 and torch.equal(o["path"], base["path"])
        last = base["path"][b, base["accept_len"][b].item()].item()
        bad = tl.clone()
        bad[b, last, 5] = float("nan")
        o = ref.tree_accept_match(bad, tok, parent, owner, u, temperature=1.0)
        assert o["status"][b].item() == ref.ST_NONFINITE and o["next_token"][b].item() == -1
        assert o["accept_len"][b].item() == 0


def test_tree_and_token_validation():
    cfg, parent, owner, tl, tok, u = _random_case(seed=32, B=3)
    p2 = parent.clone(); p2[1, 4] = 7
    t2 = tok.clone(); t2[2, 3] = cfg.V
    o = ref.tree_accept_match(tl, tok, p2, owner, u)
    assert o["status"].tolist()[1] == ref.ST_BAD_PARENT and o["status"].tolist()[0] == 0
    o = ref.tree_accept_match(tl, t2, parent, owner, u)
    assert o["status"].tolist()[2] == ref.ST_BAD_TOKEN
