"""The whole verification step (L x attention + acceptance + compaction) through the C-ABI against the
oracle, on reduced copies of the five workloads, and at full size on sampled outputs."""
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs
from paper_2603_08899_b200.step import VerifyStep
from tests import harness as H

pytestmark = pytest.mark.gpu


def _build(cfg, layers, temperature):
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen)
    lt = [inputs.layer_tensors(cfg, l, n_slots, device="cuda") for l in range(layers)]
    tl, dl = inputs.logits(cfg, device="cuda")
    tok = inputs.draft_tokens(cfg, parent, dl, temperature)
    u = inputs.uniforms(cfg)
    return parent, owner, plen, seq_start, n_slots, lt, tl, dl, tok, u


def _run_step(cfg, layers, temperature):
    parent, owner, plen, seq_start, n_slots, lt, tl, dl, tok, u = _build(cfg, layers, temperature)
    host = [{k: (None if v is None else v.cpu().clone()) for k, v in t.items()} for t in lt]
    step = VerifyStep(cfg, n_slots)
    outs = [torch.empty_like(t["q"]) for t in lt]
    step.bind([t["q"] for t in lt], [t["k_cache"] for t in lt], [t["v_cache"] for t in lt],
              [t["k_soft"] for t in lt] if cfg.S else None, [t["v_soft"] for t in lt] if cfg.S else None, outs,
              seq_start.cuda(), plen.cuda(), parent.cuda(), owner.cuda() if cfg.C else None, tl, dl, tok.cuda(),
              u.cuda())
    step.run(temperature)
    torch.cuda.synchronize()
    got = {"accept_len": step.accept_len.cpu(), "path": step.path.cpu(), "next_token": step.next_token.cpu(),
           "future_row": step.future_row.cpu(), "counters": step.counters.cpu(), "status": step.status.cpu()}
    want = ref.tree_accept(tl.cpu(), dl.cpu() if temperature > 0 else None, tok, parent, owner,
                           u if temperature > 0 else None, temperature=temperature)
    exact, border = H.compare_accept(got, want)
    # attention, every layer
    for l in range(layers):
        w, _, _ = ref.tree_attention(host[l]["q"], host[l]["k_cache"], host[l]["v_cache"], seq_start, plen,
                                     host[l]["k_soft"], host[l]["v_soft"], parent, owner)
        H.assert_attention_close(outs[l].cpu(), None, w, None, cfg.kv_dtype, f"{cfg.name} layer {l}")
    # compaction: replay the GPU's accepted path on the host copies (byte-exact)
    kh = [h["k_cache"] for h in host]
    vh = [h["v_cache"] for h in host]
    new_len = ref.kv_compact(kh, vh, seq_start, plen, got["accept_len"], got["path"])
    assert step.new_prefix_len.cpu().tolist() == new_len.tolist()
    for l in range(layers):
        for b in range(cfg.B):
            lo, hi = int(seq_start[b]), int(seq_start[b]) + int(new_len[b])
            assert torch.equal(lt[l]["k_cache"][lo:hi].cpu(), kh[l][lo:hi])
            assert torch.equal(lt[l]["v_cache"][lo:hi].cpu(), vh[l][lo:hi])
    step.close()
    return exact, border, got


def test_tiny_config_full():
    cfg = inputs.CONFIGS["tiny"]
    for temp in cfg.temperatures:
        exact, border, _ = _run_step(cfg, cfg.L, temp)
        assert exact + border == 1


@pytest.mark.parametrize("name,prefix", [("llama3b", 700), ("llama8b", 900), ("qwen4b", 1100), ("llama8b_2t", 600)])
def test_llm_shaped_steps_reduced_prefix(name, prefix):
    """Real head counts, tree sizes and vocabularies; prefix and layer count cut so the oracle
    finishes in seconds; still several key tiles and a ragged tail."""
    base = inputs.CONFIGS[name]
    cfg = inputs.scaled(base, prefix=prefix, L=2)
    for temp in base.temperatures:
        exact, border, got = _run_step(cfg, 2, temp)
        assert exact + border == cfg.B


def test_batched_ragged_step_reduced():
    base = inputs.CONFIGS["batch32"]
    cfg = inputs.scaled(base, B=6, prefix=(1, 900), L=2)
    exact, border, got = _run_step(cfg, 2, 1.0)
    assert exact + border == cfg.B and border <= 1


@pytest.mark.parametrize("name", ["llama3b", "llama8b", "qwen4b", "batch32", "llama8b_2t", "llama8b_30", "batch32_2t"])
def test_full_size_attention_on_sampled_rows(name):
    """The full-size workload of the benchmark, one layer, in the launch configuration the
    benchmark times; the oracle recomputes a sample of output rows one by one."""
    cfg = inputs.CONFIGS[name]
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen)
    t = inputs.layer_tensors(cfg, 0, n_slots, device="cuda")
    step = VerifyStep(cfg, n_slots)
    out = torch.empty_like(t["q"])
    lse = torch.empty(cfg.B, cfg.R, cfg.Hq, dtype=torch.float32, device="cuda")
    tl = torch.zeros(1, device="cuda")
    step.bind([t["q"]], [t["k_cache"]], [t["v_cache"]], [t["k_soft"]], [t["v_soft"]], [out], seq_start.cuda(),
              plen.cuda(), parent.cuda(), owner.cuda(), tl, tl, tl, tl)
    step.run_attention([lse])
    torch.cuda.synchronize()
    assert (step.status == 0).all()
    g = torch.Generator().manual_seed(7)
    n_sel = 48
    sel = torch.stack([torch.randint(0, cfg.B, (n_sel,), generator=g), torch.randint(0, cfg.R, (n_sel,), generator=g),
                       torch.randint(0, cfg.Hq, (n_sel,), generator=g)], 1)
    # make sure first/last rows, contemplate rows and the longest / shortest sequences are in the sample
    b_long, b_short = int(plen.argmax()), int(plen.argmin())
    extra = torch.tensor([[b_long, 0, 0], [b_long, cfg.R - 1, cfg.Hq - 1], [b_short, cfg.T, 1],
                          [b_short, cfg.T - 1, cfg.Hq - 1]])
    sel = torch.cat([sel, extra]).to(torch.int32)
    host = {k: v.cpu() for k, v in t.items()}
    want, want_lse = ref.tree_attention_rows(host["q"], host["k_cache"], host["v_cache"], seq_start, plen,
                                             host["k_soft"], host["v_soft"], parent, owner, sel)
    out_c, lse_c = out.cpu(), lse.cpu()
    atol, rtol, ltol = H.TOL[cfg.kv_dtype]
    for i, (b, r, h) in enumerate(sel.tolist()):
        err = (out_c[b, r, h].double() - want[i]).abs().max().item()
        assert err <= atol and err <= rtol * want.abs().max().item(), (name, b, r, h, err)
        assert abs(lse_c[b, r, h].item() - want_lse[i].item()) <= ltol, (name, b, r, h)
    assert torch.isfinite(out_c.float()).all()
    step.close()


@pytest.mark.parametrize("name", ["llama8b", "batch32"])
def test_full_size_acceptance(name):
    """Full vocabulary, full batch: the oracle walks every sequence."""
    base = inputs.CONFIGS[name]
    cfg = inputs.scaled(base, B=min(base.B, 8))
    parent, owner = inputs.trees(cfg)
    tl, dl = inputs.logits(cfg)
    tok = inputs.draft_tokens(cfg, parent, dl, 1.0)
    u = inputs.uniforms(cfg)
    g = H.Gpu()
    got = H.gpu_accept(g, cfg, tl, dl, tok, parent, owner, u, 1.0)
    want = ref.tree_accept(tl, dl, tok, parent, owner, u, temperature=1.0)
    exact, border = H.compare_accept(got, want)
    assert exact + border == cfg.B and border <= 1
    g.close()


def test_two_chained_steps_through_compaction_and_append():
    """Step 1 (attention, acceptance, compaction), then a second step on the compacted cache: the new
    tree's K/V rows are placed behind the new prefix with confu_kv_append and attention runs with
    new_prefix_len as the prefix.  The oracle replays the same two steps on host copies."""
    cfg = inputs.scaled(inputs.CONFIGS["batch32"], B=4, prefix=(40, 500), L=2)
    parent, owner, plen, seq_start, n_slots, lt, tl, dl, tok, u = _build(cfg, cfg.L, 1.0)
    # leave room behind every sequence for the second step's rows: rebuild the layout with slack
    seq_start, n_slots = inputs.cache_layout(cfg, plen + 16)
    lt = [inputs.layer_tensors(cfg, l, n_slots, device="cuda") for l in range(cfg.L)]
    host = [{k: (None if v is None else v.cpu().clone()) for k, v in t.items()} for t in lt]
    step = VerifyStep(cfg, n_slots)
    outs = [torch.empty_like(t["q"]) for t in lt]
    step.bind([t["q"] for t in lt], [t["k_cache"] for t in lt], [t["v_cache"] for t in lt],
              [t["k_soft"] for t in lt], [t["v_soft"] for t in lt], outs, seq_start.cuda(), plen.cuda(),
              parent.cuda(), owner.cuda(), tl, dl, tok.cuda(), u.cuda())
    step.run(1.0)
    torch.cuda.synchronize()
    assert (step.status == 0).all()
    # ---- oracle: step 1 acceptance and compaction on the host copies
    want = ref.tree_accept(tl.cpu(), dl.cpu(), tok, parent, owner, u, temperature=1.0)
    got = {"accept_len": step.accept_len.cpu(), "path": step.path.cpu(), "next_token": step.next_token.cpu(),
           "future_row": step.future_row.cpu(), "counters": step.counters.cpu(), "status": step.status.cpu()}
    exact, border = H.compare_accept(got, want)
    kh, vh = [h["k_cache"] for h in host], [h["v_cache"] for h in host]
    # replay the GPU's accepted path (it equals the oracle's unless a borderline decision differed)
    new_len_host = ref.kv_compact(kh, vh, seq_start, plen, got["accept_len"], got["path"])
    assert step.new_prefix_len.cpu().tolist() == new_len_host.tolist()
    # ---- step 2: a fresh tree on the compacted cache
    cfg2 = inputs.scaled(cfg, seed=cfg.seed + 77)
    parent2, owner2 = inputs.trees(cfg2)
    g = torch.Generator().manual_seed(123)
    new_plen = step.new_prefix_len.clone()
    for l in range(cfg.L):
        q2 = torch.randn(cfg.B, cfg.R, cfg.Hq, cfg.D, generator=g).to(cfg.kv_dtype)
        k_rows = torch.randn(cfg.B, cfg.R, cfg.Hkv, cfg.D, generator=g).to(cfg.kv_dtype)
        v_rows = torch.randn(cfg.B, cfg.R, cfg.Hkv, cfg.D, generator=g).to(cfg.kv_dtype)
        cb.confu_kv_append(step.ctx, step.dims, k_rows.cuda(), v_rows.cuda(), lt[l]["k_cache"], lt[l]["v_cache"],
                           step.seq_start, new_plen)
        out2 = torch.empty_like(lt[l]["q"])
        lse2 = torch.empty(cfg.B, cfg.R, cfg.Hq, dtype=torch.float32, device="cuda")
        st2 = torch.zeros(cfg.B, dtype=torch.int32, device="cuda")
        cb.confu_tree_attention(step.ctx, step.dims, q2.cuda(), lt[l]["k_cache"], lt[l]["v_cache"], n_slots,
                                step.seq_start, new_plen, lt[l]["k_soft"], lt[l]["v_soft"], parent2.cuda(),
                                owner2.cuda(), None, out2, lse2, st2)
        torch.cuda.synchronize()
        assert (st2 == 0).all()
        # host: same append on the compacted host cache, then the oracle
        for b in range(cfg.B):
            lo = int(seq_start[b]) + int(new_len_host[b])
            kh[l][lo:lo + cfg.R] = k_rows[b]
            vh[l][lo:lo + cfg.R] = v_rows[b]
        w, wl, _ = ref.tree_attention(q2, kh[l], vh[l], seq_start, new_len_host, host[l]["k_soft"], host[l]["v_soft"],
                                      parent2, owner2)
        H.assert_attention_close(out2.cpu(), lse2.cpu(), w, wl, cfg.kv_dtype, f"second step layer {l}")
    step.close()


def test_captured_step_replays_to_the_same_results():
    """The step captured as CUDA graphs (what the benchmark times) writes the same bits as the
    launches issued one by one, also after the inputs behind the bound pointers have changed."""
    cfg = inputs.scaled(inputs.CONFIGS["llama8b"], B=3, L=2, prefix=(100, 700), V=4096)
    parent, owner, plen, seq_start, n_slots, lt, tl, dl, tok, u = _build(cfg, 2, 1.0)
    step = VerifyStep(cfg, n_slots)
    outs = [torch.empty_like(t["q"]) for t in lt]
    step.bind([t["q"] for t in lt], [t["k_cache"] for t in lt], [t["v_cache"] for t in lt],
              [t["k_soft"] for t in lt], [t["v_soft"] for t in lt], outs, seq_start.cuda(), plen.cuda(), parent.cuda(),
              owner.cuda(), tl, dl, tok.cuda(), u.cuda())
    keep = [(t["k_cache"].clone(), t["v_cache"].clone()) for t in lt]

    def restore():
        for t, (k, v) in zip(lt, keep):
            t["k_cache"].copy_(k)
            t["v_cache"].copy_(v)

    def snapshot():
        torch.cuda.synchronize()
        return [o.clone() for o in outs] + [step.accept_len.clone(), step.path.clone(), step.next_token.clone(),
                                            step.future_row.clone(), step.new_prefix_len.clone(), step.status.clone()] + \
               [t["k_cache"].clone() for t in lt]

    step.run(1.0)
    eager = snapshot()
    restore()
    step.capture(1.0)
    restore()                                   # (a capture does not run the kernels; this is for symmetry)
    for o in outs:
        o.zero_()
    step.accept_len.fill_(-1)
    step.replay()
    for a, b in zip(eager, snapshot()):
        assert torch.equal(a, b)
    # new queries behind the same pointers: replay follows, eager agrees
    restore()
    for t in lt:
        t["q"].copy_(torch.roll(t["q"], 1, dims=1))
    step.replay()
    replayed = snapshot()
    restore()
    step.run(1.0)
    for a, b in zip(snapshot(), replayed):
        assert torch.equal(a, b)
    assert not torch.equal(replayed[0], eager[0])
    # the whole step as a single graph (the launch the benchmark's headline times)
    restore()
    for o in outs:
        o.zero_()
    step.accept_len.fill_(-1)
    step.replay_step()
    for a, b in zip(snapshot(), replayed):
        assert torch.equal(a, b)
    step.close()
