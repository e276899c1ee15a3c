"""GPU parity of confu_tree_accept_match (sample-and-match rule, statistics on demand) against the
fp64 oracle: path, next token, future row and counters bit-exact, except sequences where a draw
fell within 1e-5 of a CDF cell edge (counted and bounded)."""
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import inputs
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    g = H.Gpu()
    yield g
    g.close()


def _cfg(**kw):
    base = dict(B=8, L=1, Hq=4, Hkv=1, D=64, T=24, C=4, S=0, V=5000, prefix=4, tree="random",
                kv_dtype=torch.bfloat16, logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                temperatures=(1.0,), seed=81, max_depth=6, fanout=(1, 4))
    base.update(kw)
    return inputs.VerifyConfig("match", **base)


CASES = {
    "bf16_noise": _cfg(),
    "bf16_peaked": _cfg(sigma_logit=6.0, seed=82),
    "fp32_vocab_1000": _cfg(V=1000, logit_dtype=torch.float32, sigma_logit=4.0, seed=83),
    "ragged_vocab_not_multiple_of_8": _cfg(V=4999, seed=84),
    "odd_vocab_fp32": _cfg(V=1237, logit_dtype=torch.float32, seed=85),
    "vocab_llama": _cfg(B=4, V=128256, T=60, seed=86, max_depth=7, sigma_logit=5.0),
    "vocab_qwen": _cfg(B=2, V=151936, T=60, seed=87, max_depth=7, sigma_logit=5.0),
    "chain_12": _cfg(T=13, tree="chain", seed=88, sigma_logit=6.0),
    "star": _cfg(T=30, tree="star", seed=89),
    "single_node": _cfg(T=1, C=1, seed=90),
    "small_vocab_16": _cfg(V=16, logit_dtype=torch.float32, sigma_logit=1.0, seed=91, B=32),
}


def _inputs(cfg, temperature):
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, temperature)      # draft = target + noise: drafts often match
    u = inputs.uniforms(cfg)
    return parent, owner, tl, tok, u


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("temperature", [1.0, 0.7, 0.0])
def test_walk_matches_oracle(gpu, name, temperature):
    cfg = CASES[name]
    parent, owner, tl, tok, u = _inputs(cfg, temperature)
    want = ref.tree_accept_match(tl, tok, parent, owner, u if temperature > 0 else None, temperature=temperature)
    got = H.gpu_accept_match(gpu, cfg, tl, tok, parent, owner, u if temperature > 0 else None, temperature)
    log = []
    exact, border = H.compare_match(got, want, log)
    assert exact + border == cfg.B
    assert border <= max(1, cfg.B // 8), log
    assert got["status"].tolist() == [0] * cfg.B


def test_some_drafts_are_accepted_so_the_walk_is_exercised(gpu):
    cfg = CASES["bf16_peaked"]
    parent, owner, tl, tok, u = _inputs(cfg, 1.0)
    got = H.gpu_accept_match(gpu, cfg, tl, tok, parent, owner, u, 1.0)
    assert got["accept_len"].max().item() >= 2 and (got["accept_len"] == 0).any()
    assert (got["counters"][:, 0] == got["accept_len"] + 1).all()         # one draw per visited node


def test_only_rows_on_the_walked_path_are_read(gpu):
    cfg = CASES["bf16_noise"]
    parent, owner, tl, tok, u = _inputs(cfg, 1.0)
    base = H.gpu_accept_match(gpu, cfg, tl, tok, parent, owner, u, 1.0)
    bad = tl.clone()
    hit = []
    for b in range(cfg.B):
        on_path = set(base["path"][b, :base["accept_len"][b].item() + 1].tolist())
        off = [i for i in range(cfg.T) if i not in on_path]
        bad[b, off[0], 7] = float("inf")                         # never read: no error, same result
        bad[b, off[-1], cfg.V - 1] = float("nan")
    got = H.gpu_accept_match(gpu, cfg, bad, tok, parent, owner, u, 1.0)
    for k in base:
        assert torch.equal(got[k], base[k]), k
    bad = tl.clone()
    for b in (1, 5):
        last = base["path"][b, base["accept_len"][b].item()].item()
        bad[b, last, 4321] = float("nan") if b == 1 else float("-inf")
        hit.append(b)
    got = H.gpu_accept_match(gpu, cfg, bad, tok, parent, owner, u, 1.0)
    want = ref.tree_accept_match(bad, tok, parent, owner, u, temperature=1.0)
    assert got["status"].tolist() == want["status"].tolist()
    for b in range(cfg.B):
        assert got["status"][b].item() == (ref.ST_NONFINITE if b in hit else 0)
        if b in hit:
            assert got["accept_len"][b].item() == 0 and got["next_token"][b].item() == -1 and got["path"][b, 0].item() == 0


def test_malformed_trees_and_tokens_are_reported(gpu):
    cfg = CASES["bf16_noise"]
    parent, owner, tl, tok, u = _inputs(cfg, 1.0)
    p2 = parent.clone(); p2[2, 5] = 9
    t2 = tok.clone(); t2[3, 4] = cfg.V
    o2 = owner.clone(); o2[6, 1] = cfg.T
    for args in ((tl, tok, p2, owner), (tl, t2, parent, owner), (tl, tok, parent, o2)):
        got = H.gpu_accept_match(gpu, cfg, args[0], args[1], args[2], args[3], u, 1.0)
        want = ref.tree_accept_match(args[0], args[1], args[2], args[3], u, temperature=1.0)
        assert got["status"].tolist() == want["status"].tolist() and sum(got["status"].tolist()) > 0
        H.compare_match(got, want)


def test_host_side_argument_checks(gpu):
    from paper_2603_08899_b200 import binding as cb
    one = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(cb.ConfuError):
        cb.confu_tree_accept_match(gpu.ctx, 1, 65, 0, 100, torch.bfloat16, one, one, one, None, one, 1.0, one, one, one,
                                   None, None, None)
    with pytest.raises(cb.ConfuError):
        cb.confu_tree_accept_match(gpu.ctx, 1, 4, 0, 100, torch.bfloat16, one, one, one, None, None, 1.0, one, one, one,
                                   None, None, None)
