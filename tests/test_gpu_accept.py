"""GPU parity of confu_tree_accept against the fp64 oracle: accepted path, next token and future
row bit-exact, except decisions the oracle marks as borderline (counted and reported)."""
import numpy as np
import pytest
import torch
from scipy import stats

from oracle import ref
from paper_2603_08899_b200 import inputs
from tests import harness as H
from tests.test_oracle_accept import PARENT10, V16, _chi2_pvalues, _emitted, _trials

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    g = H.Gpu()
    yield g
    g.close()


def _cfg(**kw):
    base = dict(B=8, L=1, Hq=4, Hkv=1, D=64, T=24, C=4, S=0, V=5000, prefix=4, tree="random",
                kv_dtype=torch.bfloat16, logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                temperatures=(1.0,), seed=51, max_depth=6, fanout=(1, 4))
    base.update(kw)
    return inputs.VerifyConfig("acc", **base)


def _run(gpu, cfg, temperature, mode=1):
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, temperature)
    u = inputs.uniforms(cfg)
    want = ref.tree_accept(tl, dl if temperature > 0 else None, tok, parent, owner, u if temperature > 0 else None,
                           temperature=temperature, sibling_mode=mode)
    got = H.gpu_accept(gpu, cfg, tl, dl if temperature > 0 else None, tok, parent, owner,
                       u if temperature > 0 else None, temperature, mode)
    return got, want


CASES = {
    "bf16_noise": _cfg(),
    "bf16_independent": _cfg(draft="independent", seed=52),
    "fp32_tiny_vocab_1000": _cfg(V=1000, logit_dtype=torch.float32, sigma_logit=2.0, draft="independent", seed=53),
    "ragged_vocab_not_multiple_of_8": _cfg(V=4999, seed=54),
    "odd_vocab_fp32": _cfg(V=1237, logit_dtype=torch.float32, seed=55),
    "vocab_llama": _cfg(B=3, V=128256, T=60, seed=56, max_depth=7),
    "vocab_qwen": _cfg(B=2, V=151936, T=60, seed=57, max_depth=7),
    "chain_12": _cfg(T=13, tree="chain", seed=58),
    "star": _cfg(T=30, tree="star", seed=59, draft="independent"),
    "single_node": _cfg(T=1, C=1, seed=60),
    "small_vocab_16": _cfg(V=16, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent", seed=61, B=32),
}


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("temperature", [1.0, 0.7])
def test_sampling_walk_matches_oracle(gpu, name, temperature):
    cfg = CASES[name]
    got, want = _run(gpu, cfg, temperature)
    log = []
    exact, border = H.compare_accept(got, want, log)
    assert exact + border == cfg.B
    assert border <= max(1, cfg.B // 8), log


@pytest.mark.parametrize("name", ["bf16_noise", "star", "small_vocab_16"])
def test_iid_sibling_mode_matches_oracle(gpu, name):
    cfg = CASES[name]
    got, want = _run(gpu, cfg, 1.0, mode=0)
    exact, border = H.compare_accept(got, want)
    assert exact >= cfg.B - 1


@pytest.mark.parametrize("name", ["bf16_noise", "vocab_qwen", "fp32_tiny_vocab_1000", "chain_12"])
def test_greedy_matches_oracle(gpu, name):
    cfg = CASES[name]
    got, want = _run(gpu, cfg, 0.0)
    for k in ("accept_len", "path", "next_token", "future_row", "status"):
        assert torch.equal(got[k], want[k]), k


def test_greedy_with_many_ties_and_matches(gpu):
    cfg = _cfg(V=6, T=14, B=16, seed=62, logit_dtype=torch.bfloat16)
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = torch.randint(0, cfg.V, (cfg.B, cfg.T), generator=torch.Generator().manual_seed(1), dtype=torch.int32)
    want = ref.tree_accept(tl, None, tok, parent, owner, None, temperature=0.0)
    got = H.gpu_accept(gpu, cfg, tl, None, tok, parent, owner, None, 0.0)
    for k in ("accept_len", "path", "next_token", "future_row"):
        assert torch.equal(got[k], want[k]), k
    assert want["accept_len"].max().item() >= 1


def test_identical_distributions_accept_to_a_leaf(gpu):
    cfg = CASES["bf16_noise"]
    parent, owner = inputs.trees(cfg)
    tl, _ = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, tl, 1.0)
    u = inputs.uniforms(cfg)
    want = ref.tree_accept(tl, tl.clone(), tok, parent, owner, u)
    got = H.gpu_accept(gpu, cfg, tl, tl.clone(), tok, parent, owner, u, 1.0)
    exact, border = H.compare_accept(got, want)
    assert exact >= cfg.B - 1
    assert (got["counters"][:, 1] == 0).all()


def test_input_errors_are_reported_per_sequence(gpu):
    cfg = CASES["bf16_noise"]
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, 1.0)
    u = inputs.uniforms(cfg)
    tok[1, 2] = cfg.V                      # bad token
    par = parent[2].tolist()
    i, j = next((i, j) for i in range(1, cfg.T) for j in range(i + 1, cfg.T) if par[i] == par[j])
    tok[2, j] = tok[2, i]                  # duplicate siblings
    tl[3, 4, 77] = float("inf")            # non-finite logit
    parent = parent.clone()
    parent[4, 3] = 3                       # bad parent
    owner = owner.clone()
    owner[5, 0] = cfg.T                    # bad owner
    want = ref.tree_accept(tl, dl, tok, parent, owner, u)
    got = H.gpu_accept(gpu, cfg, tl, dl, tok, parent, owner, u, 1.0)
    assert want["status"].tolist()[:6] == [0, 3, 4, 5, 1, 2]
    assert got["status"].tolist() == want["status"].tolist()
    for b in (1, 2, 3, 4, 5):
        assert got["accept_len"][b].item() == 0 and got["next_token"][b].item() == -1
        assert got["path"][b].tolist() == want["path"][b].tolist()
    exact, border = H.compare_accept({k: v[[0, 6, 7]] for k, v in got.items()},
                                     {k: v[[0, 6, 7]] for k, v in want.items()})
    assert exact + border == 3


@pytest.mark.parametrize("mode", [1, 0])
def test_emitted_tokens_follow_the_target_distribution_on_gpu(gpu, mode):
    """The same closed-form check the oracle passes, run on the CUDA path."""
    N = 40000
    tl, dl, tok, parent, u, (P0, P1) = _trials(N, mode, seed=199 + mode)
    cfg = _cfg(B=N, T=10, C=0, V=V16, logit_dtype=torch.float32)
    got = H.gpu_accept(gpu, cfg, tl.float(), dl.float(), tok, parent, None, u.float(), 1.0, mode)
    assert (got["status"] == 0).all()
    first, second = _emitted(got, tok)
    p_first, p_second = _chi2_pvalues(first, second, P0, P1)
    assert p_first > 1e-4 and p_second > 1e-4, (p_first, p_second)


# ---------------------------------------------------------------- statistics on demand
LAZY = 0x100


@pytest.mark.parametrize("name", ["bf16_noise", "bf16_independent", "ragged_vocab_not_multiple_of_8", "vocab_llama",
                                  "chain_12", "star", "single_node", "small_vocab_16"])
@pytest.mark.parametrize("temperature", [1.0, 0.7, 0.0])
def test_lazy_statistics_match_oracle(gpu, name, temperature):
    cfg = CASES[name]
    got, want = _run(gpu, cfg, temperature, mode=1 | LAZY)
    log = []
    exact, border = H.compare_accept(got, want, log)
    assert exact + border == cfg.B
    assert border <= max(1, cfg.B // 8), log


def test_lazy_statistics_need_no_workspace_and_read_only_the_walked_rows(gpu):
    from paper_2603_08899_b200 import binding as cb
    cfg = CASES["bf16_noise"]
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, 1.0)
    u = inputs.uniforms(cfg)
    base = H.gpu_accept(gpu, cfg, tl, dl, tok, parent, owner, u, 1.0, 1 | LAZY)
    bad_t, bad_d = tl.clone(), dl.clone()
    for b in range(cfg.B):
        on_path = set(base["path"][b, :base["accept_len"][b].item() + 1].tolist())
        off = [i for i in range(cfg.T) if i not in on_path]
        bad_t[b, off[0], 11] = float("nan")
        bad_d[b, off[-1], cfg.V - 1] = float("inf")
    dev = "cuda"
    o = {"accept_len": torch.zeros(cfg.B, dtype=torch.int32, device=dev),
         "path": torch.zeros((cfg.B, cb.MAX_DEPTH + 1), dtype=torch.int32, device=dev),
         "next_token": torch.zeros(cfg.B, dtype=torch.int32, device=dev),
         "status": torch.zeros(cfg.B, dtype=torch.int32, device=dev)}
    cb.confu_tree_accept(gpu.ctx, cfg.B, cfg.T, cfg.C, cfg.V, tl.dtype, bad_t.to(dev), bad_d.to(dev), tok.to(dev),
                         parent.to(dev), owner.to(dev), u.to(dev), 1.0, 1 | LAZY, o["accept_len"], o["path"],
                         o["next_token"], None, None, None, o["status"])          # no workspace
    torch.cuda.synchronize()
    assert o["status"].cpu().tolist() == [0] * cfg.B
    for k in ("accept_len", "path", "next_token"):
        assert torch.equal(o[k].cpu(), base[k]), k
    # the default mode sees them
    got = H.gpu_accept(gpu, cfg, bad_t, bad_d, tok, parent, owner, u, 1.0, 1)
    assert got["status"].tolist() == [5] * cfg.B
    # a bad logit on the path is an error in lazy mode too, and agrees with the oracle
    bad_d = dl.clone()
    last = base["path"][3, base["accept_len"][3].item()].item()
    bad_d[3, last, 17] = float("nan")
    got = H.gpu_accept(gpu, cfg, tl, bad_d, tok, parent, owner, u, 1.0, 1 | LAZY)
    want = ref.tree_accept(tl, bad_d, tok, parent, owner, u, temperature=1.0, sibling_mode=1 | LAZY)
    assert got["status"].tolist() == want["status"].tolist() and got["status"][3].item() == 5
    H.compare_accept(got, want)
