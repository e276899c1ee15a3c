"""GPU parity of confu_tree_attention against the fp64 oracle, element by element."""
import pytest
import torch

from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    g = H.Gpu()
    yield g
    g.close()


def _cfg(name="c", **kw):
    base = dict(B=2, L=1, Hq=8, Hkv=2, D=128, T=12, C=3, S=4, V=32, prefix=(100, 300), tree="random",
                kv_dtype=torch.bfloat16, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent",
                temperatures=(1.0,), seed=31, max_depth=5, fanout=(1, 3))
    base.update(kw)
    return inputs.VerifyConfig(name, **base)


CASES = {
    "tiny_config": inputs.CONFIGS["tiny"],
    "fp32_d128_ragged": _cfg(kv_dtype=torch.float32, seed=32),
    "fp32_d64_g1": _cfg(kv_dtype=torch.float32, Hq=2, Hkv=2, D=64, seed=33),
    "bf16_d64": _cfg(D=64, seed=34),
    "bf16_g4_ragged_multi_tile": _cfg(B=3, prefix=(1, 700), seed=35),
    "bf16_g3": _cfg(Hq=6, Hkv=2, seed=36),
    "bf16_g8": _cfg(Hq=16, Hkv=2, seed=37),
    "bf16_full_rows": _cfg(B=2, T=60, C=4, S=16, prefix=(130, 520), max_depth=7, fanout=(1, 4), seed=38),
    "bf16_prefix_zero": _cfg(prefix=0, seed=39),
    "bf16_prefix_eight": _cfg(prefix=8, seed=40),
    "bf16_no_soft_no_contemplate": _cfg(C=0, S=0, seed=41),
    "bf16_single_row": _cfg(T=1, C=0, S=0, seed=42),
    "bf16_single_row_with_contemplate": _cfg(T=1, C=1, S=16, prefix=257, seed=43),
    "bf16_chain_depth12": _cfg(T=13, C=13, tree="chain", seed=44),
    "bf16_star": _cfg(T=20, C=2, tree="star", seed=45),
    "bf16_paper_sized_30_30": _cfg(B=1, T=30, C=30, S=16, prefix=1000, max_depth=7, fanout=(1, 4), seed=46),
    "bf16_exact_tile_multiple": _cfg(B=1, T=12, C=4, prefix=256 - 16, seed=47),
    "bf16_one_past_tile": _cfg(B=1, T=12, C=4, prefix=256 - 15, seed=48),
    # more than 64 query rows: one contemplate row per tree node (R = 2T), two groups of 64 rows
    "bf16_one_contemplate_per_node_60_60": _cfg(B=2, T=60, C=60, S=16, prefix=(130, 520), max_depth=7, fanout=(1, 4), seed=49),
    "bf16_rows_65": _cfg(T=33, C=32, S=16, prefix=(60, 200), max_depth=7, fanout=(1, 4), seed=50),
    "bf16_g3_rows_80": _cfg(Hq=6, Hkv=2, T=40, C=40, prefix=(1, 300), max_depth=7, fanout=(1, 4), seed=51),
    "bf16_rows_128_chain": _cfg(B=1, T=64, C=64, S=16, tree="chain", prefix=257, seed=52),
    "fp32_rows_100": _cfg(kv_dtype=torch.float32, T=50, C=50, prefix=(10, 150), max_depth=7, fanout=(1, 4), seed=53),
    "bf16_d64_rows_90": _cfg(D=64, T=45, C=45, prefix=(10, 150), max_depth=7, fanout=(1, 4), seed=54),
    # the largest soft-prompt block the tensor-core path takes (one whole key tile), and a ragged one
    "bf16_soft_128": _cfg(S=128, seed=55),
    "bf16_soft_100": _cfg(S=100, T=20, C=20, seed=56),
    # one pair of 131 key tiles: every CTA gets a single tile, the merge sees ~130 parts (more than one group of 32)
    "bf16_one_pair_130_parts": _cfg(B=1, Hq=4, Hkv=1, prefix=16500, seed=57),
    # more pairs than SMs: whole pairs per CTA, few splits
    "bf16_many_short_sequences": _cfg(B=170, Hq=4, Hkv=2, prefix=(1, 260), seed=58),
    # the same with two groups of 64 rows per pair (each share of the work is walked by two CTAs side by side),
    # and one long pair of two row groups spread over all CTAs
    "bf16_many_short_sequences_rows_80": _cfg(B=90, Hq=4, Hkv=2, T=40, C=40, prefix=(1, 260), max_depth=7, fanout=(1, 4), seed=59),
    "bf16_one_pair_rows_100_many_parts": _cfg(B=1, Hq=4, Hkv=1, T=50, C=50, prefix=12000, max_depth=7, fanout=(1, 4), seed=60),
}


def _takes_tensor_cores(cfg):
    return cfg.kv_dtype == torch.bfloat16 and cfg.D == 128 and cfg.Hq // cfg.Hkv <= 4 and cfg.S <= 128


@pytest.mark.parametrize("name", list(CASES))
@pytest.mark.parametrize("use_plan", [False, True])
@pytest.mark.parametrize("path", ["auto", "one_cta_per_sm", "cta_pairs"])
def test_attention_matches_oracle(gpu, name, use_plan, path):
    """path auto: the library's own choice (CUDA cores, one CTA per SM with tcgen05, or CTA pairs with
    the two-SM instructions, by dims and batch size); the two tensor-core kernels are also forced, each
    for every case it can take."""
    cfg = CASES[name]
    if path == "one_cta_per_sm" and not _takes_tensor_cores(cfg):
        pytest.skip("not a tensor-core case")
    if path == "cta_pairs" and not (_takes_tensor_cores(cfg) and cfg.R > 32):
        pytest.skip("the two-SM kernel takes more than 32 query rows")
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    gpu.set_path({"auto": cb.ATTENTION_AUTO, "one_cta_per_sm": cb.ATTENTION_TENSOR, "cta_pairs": cb.ATTENTION_TENSOR_PAIR}[path])
    try:
        out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots, use_plan=use_plan)
    finally:
        gpu.set_path(cb.ATTENTION_AUTO)
    want, want_lse, want_st = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
    assert st.tolist() == want_st.tolist() == [0] * cfg.B
    H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, name)


@pytest.mark.parametrize("name", ["bf16_full_rows", "bf16_g3", "bf16_paper_sized_30_30", "fp32_d128_ragged",
                                  "bf16_one_contemplate_per_node_60_60", "bf16_g3_rows_80", "fp32_rows_100"])
def test_mask_sensitivity_with_boosted_tree_keys(gpu, name):
    """With the tree slots' keys scaled up the tree columns dominate the softmax, so a wrong
    ancestor bit moves the output far beyond tolerance even behind a long prefix."""
    cfg = CASES[name]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg, tree_key_gain=4.0)
    out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
    want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner)
    H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, name)
    # power of this case: the oracle with a *different* tree (all nodes children of the root) is far away
    star = torch.zeros_like(parent)
    star[:, 0] = -1
    other, _, _ = H.oracle_attention(cfg, t, seq_start, plen, star, owner)
    assert (other - want).abs().max().item() > 0.2


def test_tree_rows_do_not_depend_on_soft_prompts_or_contemplate_rows(gpu):
    cfg = CASES["bf16_full_rows"]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    a, la, _ = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
    t2 = dict(t)
    t2["k_soft"] = (t["k_soft"].float() * 3 + 1).to(t["k_soft"].dtype)
    t2["v_soft"] = (t["v_soft"].float() * -2).to(t["v_soft"].dtype)
    b, lb, _ = H.gpu_attention(gpu, cfg, t2, seq_start, plen, parent, owner, n_slots)
    assert torch.equal(a[:, :cfg.T], b[:, :cfg.T]) and torch.equal(la[:, :cfg.T], lb[:, :cfg.T])
    assert not torch.equal(a[:, cfg.T:], b[:, cfg.T:])


@pytest.mark.parametrize("name", ["bf16_g4_ragged_multi_tile", "bf16_full_rows", "bf16_one_pair_130_parts"])
def test_run_to_run_determinism(gpu, name):
    cfg = CASES[name]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    a, la, _ = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
    for _ in range(3):
        b, lb, _ = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots)
        assert torch.equal(a, b) and torch.equal(la, lb)


def test_scale_override(gpu):
    cfg = CASES["bf16_g4_ragged_multi_tile"]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    out, lse, _ = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, owner, n_slots, sm_scale=0.05)
    want, want_lse, _ = H.oracle_attention(cfg, t, seq_start, plen, parent, owner, sm_scale=0.05)
    H.assert_attention_close(out, lse, want, want_lse, cfg.kv_dtype, "scale")


def test_malformed_tree_sets_status_and_leaves_others_intact(gpu):
    cfg = CASES["bf16_g4_ragged_multi_tile"]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    bad = parent.clone()
    bad[1, 5] = 9
    out, lse, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, bad, owner, n_slots)
    want, want_lse, want_st = H.oracle_attention(cfg, t, seq_start, plen, bad, owner)
    assert st.tolist() == want_st.tolist() == [0, 1, 0]
    keep = [0, 2]
    H.assert_attention_close(out[keep], lse[keep], want[keep], want_lse[keep], cfg.kv_dtype, "bad tree")
    bad_owner = owner.clone()
    bad_owner[0, 1] = -3
    _, _, st = H.gpu_attention(gpu, cfg, t, seq_start, plen, parent, bad_owner, n_slots)
    assert st.tolist() == [2, 0, 0]


def test_host_side_argument_errors(gpu):
    from paper_2603_08899_b200 import binding as cb
    cfg = CASES["bf16_g4_ragged_multi_tile"]
    parent, owner, plen, seq_start, n_slots, t = H.setup_case(cfg)
    with pytest.raises(cb.ConfuError) as e:
        H.gpu_attention(gpu, inputs.scaled(cfg, D=96), t, seq_start, plen, parent, owner, n_slots)
    assert e.value.code == -2
    dims = H.dims_of(inputs.scaled(cfg, T=65, C=3))
    assert cb.lib().confu_workspace_bytes(gpu.ctx, __import__("ctypes").byref(dims)) == 0      # T > 64 unsupported
    dims = H.dims_of(inputs.scaled(cfg, T=64, C=64))
    assert cb.lib().confu_workspace_bytes(gpu.ctx, __import__("ctypes").byref(dims)) > 0       # R = 128 is the limit
    # unaligned q pointer
    dims = H.dims_of(cfg)
    gpu.ensure_ws(dims)
    q_off = t["q"].view(-1)[1:]
    import ctypes as C
    rc = cb.lib().confu_tree_attention(gpu.ctx, C.byref(dims), C.c_void_p(q_off.data_ptr()), cb._ptr(t["k_cache"]),
                                       cb._ptr(t["v_cache"]), C.c_int64(n_slots), cb._ptr(seq_start.cuda()),
                                       cb._ptr(plen.cuda()), cb._ptr(t["k_soft"]), cb._ptr(t["v_soft"]),
                                       cb._ptr(parent.cuda()), cb._ptr(owner.cuda()), None, cb._ptr(t["q"]), None, None,
                                       None)
    assert rc == -3


def test_empty_batch_is_a_no_op(gpu):
    from paper_2603_08899_b200 import binding as cb
    import ctypes as C
    dims = cb.make_dims(0, 8, 2, 128, 12, 3, 4, torch.bfloat16)
    rc = cb.lib().confu_tree_attention(gpu.ctx, C.byref(dims), None, None, None, C.c_int64(0), None, None, None, None,
                                       None, None, None, None, None, None, None)
    assert rc == 0
