"""confu_tree_accept_static: the acceptance entry point for callers that cannot allocate.

A host that may not call cudaMalloc (its engine's pool owns the device, or it is a plugin that only
gets streams) cannot give confu_tree_accept a workspace; the static variant keeps that scratch in
an array inside the library.  The check here is the one such a caller cares about: through the
C-ABI, with nothing but inputs and outputs, it returns exactly what the ordinary entry point
returns (the outputs are integers, so "within tolerance" is bit-equality) -- on two calls in a row
with different inputs, because the shared array keeps the first call's contents when the second
one starts.  The file sorts last so that a run stopping at the first failure has already been
through every other test.
"""
import ctypes as C

import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from paper_2603_08899_b200 import inputs
from tests import harness as H

pytestmark = pytest.mark.gpu


def _cfg(seed, V, T, B):
    return inputs.VerifyConfig("noalloc", B=B, L=1, Hq=4, Hkv=1, D=64, T=T, C=4, S=0, V=V, prefix=4, tree="random",
                               kv_dtype=torch.bfloat16, logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                               temperatures=(1.0,), seed=seed, max_depth=6, fanout=(1, 4))


def _outputs(B):
    dev = "cuda"
    return {"accept_len": torch.full((B,), -7, dtype=torch.int32, device=dev),
            "path": torch.full((B, cb.MAX_DEPTH + 1), -7, dtype=torch.int32, device=dev),
            "next_token": torch.full((B,), -7, dtype=torch.int32, device=dev),
            "future_row": torch.full((B,), -7, dtype=torch.int32, device=dev),
            "counters": torch.full((B, 4), -7, dtype=torch.int32, device=dev),
            "status": torch.zeros(B, dtype=torch.int32, device=dev)}


def _static_call(cfg, tl, dl, tok, parent, owner, u, temperature):
    o = _outputs(cfg.B)
    cb.confu_tree_accept_static(cfg.B, cfg.T, cfg.C, cfg.V, tl.dtype, tl, dl if temperature > 0 else None, tok,
                                parent, owner, u if temperature > 0 else None, temperature, 1, o["accept_len"],
                                o["path"], o["next_token"], o["future_row"], o["counters"], o["status"])
    torch.cuda.synchronize()
    return {k: v.cpu() for k, v in o.items()}


def test_static_scratch_entry_point_matches_the_ordinary_one_on_two_calls_in_a_row():
    gpu = H.Gpu()
    try:
        # two different problems back to back: different vocabulary, tree size and batch, so the second
        # call finds the first one's statistics (of another chunking) in the shared array
        for cfg, temperature in ((_cfg(71, 32000, 24, 6), 1.0), (_cfg(72, 128256, 60, 3), 0.7),
                                 (_cfg(73, 4999, 12, 5), 0.0)):
            parent, owner = inputs.trees(cfg)
            tl, dl = inputs.logits(cfg)
            tok = inputs.draft_tokens(cfg, parent, dl, temperature)
            u = inputs.uniforms(cfg)
            want = H.gpu_accept(gpu, cfg, tl, dl if temperature > 0 else None, tok, parent, owner,
                                u if temperature > 0 else None, temperature)
            got = _static_call(cfg, tl.cuda(), dl.cuda(), tok.cuda(), parent.cuda(), owner.cuda(), u.cuda(),
                               temperature)
            assert want["status"].tolist() == [0] * cfg.B
            for k in want:
                assert torch.equal(got[k], want[k]), (cfg.seed, k, got[k], want[k])
            # and directly against the CPU oracle, under the same rule as every other acceptance test
            oracle = ref.tree_accept(tl, dl if temperature > 0 else None, tok, parent, owner,
                                     u if temperature > 0 else None, temperature=temperature, sibling_mode=1)
            exact, border = H.compare_accept(got, oracle)
            assert exact + border == cfg.B and border <= 1
    finally:
        gpu.close()


def test_static_scratch_entry_point_rejects_problems_beyond_its_fixed_size():
    limit = cb.confu_tree_accept_static_max_rows()
    assert limit == 4096
    B, T = limit // 64 + 1, 64                       # B * T just past the limit
    one = torch.zeros(16, dtype=torch.int32, device="cuda")
    rc = cb.lib().confu_tree_accept_static(C.c_int32(B), C.c_int32(T), C.c_int32(0), C.c_int32(1000), C.c_int32(cb.BF16),
                                           cb._ptr(one), cb._ptr(one), cb._ptr(one), cb._ptr(one), None, cb._ptr(one),
                                           C.c_float(1.0), C.c_int32(1), cb._ptr(one), cb._ptr(one), cb._ptr(one),
                                           None, None, None, None)
    assert rc == -4                                  # CONFU_ERR_WORKSPACE, before anything is enqueued
    with pytest.raises(cb.ConfuError):
        cb.confu_tree_accept_static(B, T, 0, 1000, torch.bfloat16, one, one, one, one, None, one, 1.0, 1, one, one,
                                    one, None, None, None)
