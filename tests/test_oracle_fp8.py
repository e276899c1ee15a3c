"""Pins of the oracle's E4M3 conversion against things other than itself: hand-written values of the
format, the library's conversion (torch.float8_e4m3fn) on all 256 codes and on random values, ties,
saturation, subnormals; and that the attention of an E4M3 cache is the attention of the values
the cache stands for."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import inputs


def test_decode_hand_written_values():
    # code: S EEEE MMM.  0x38 = 0 0111 000 = 1.0; 0x40 = 2.0; 0x3c = 1.5; 0x7e = 448 (largest); 0x08 = 2^-6
    # (smallest normal); 0x01 = 2^-9 (smallest subnormal); 0x07 = 7 * 2^-9; 0xb8 = -1.0; 0x00 / 0x80 = +-0
    codes = torch.tensor([0x38, 0x40, 0x3c, 0x7e, 0x08, 0x01, 0x07, 0xb8, 0x00, 0x80, 0x30, 0x77], dtype=torch.uint8)
    want = [1.0, 2.0, 1.5, 448.0, 2.0 ** -6, 2.0 ** -9, 7 * 2.0 ** -9, -1.0, 0.0, -0.0, 0.5, 240.0]
    got = ref.e4m3_decode(codes).tolist()
    assert got == want
    assert np.signbit(got[9]) and not np.signbit(got[8])
    nan = ref.e4m3_decode(torch.tensor([0x7f, 0xff], dtype=torch.uint8))
    assert torch.isnan(nan).all()


def test_decode_agrees_with_the_library_on_every_code():
    codes = torch.arange(256, dtype=torch.uint8)
    lib = codes.view(torch.float8_e4m3fn).to(torch.float64)
    got = ref.e4m3_decode(codes)
    finite = ~torch.isnan(lib)
    assert finite.sum().item() == 254
    assert torch.equal(got[finite], lib[finite]) and torch.isnan(got[~finite]).all()


def test_encode_ties_saturation_and_subnormals():
    # between 1.0 (mantissa 000) and 1.125 (001): 1.0625 is a tie -> even mantissa = 1.0; between 1.125 and
    # 1.25 (010): 1.1875 -> 1.25.  17 lies between 16 (0x58) and 18 (0x59): tie -> 16.  Beyond 448 saturates.
    x = torch.tensor([1.0625, 1.1875, 17.0, 19.0, 448.0, 449.0, 1e9, -1e9, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -11, 0.0])
    want = [0x38, 0x3a, 0x58, 0x5a, 0x7e, 0x7e, 0x7e, 0xfe, 0x00, 0x02, 0x00, 0x00]
    #        1.0   1.25  16    20 (tie 19 between 18 and 20 -> even mantissa 010 = 20)   2^-10: tie between 0 and 2^-9 -> 0;
    #        3*2^-10: tie between 2^-9 (001) and 2^-8 (010) -> 2^-8; 2^-11 -> 0
    assert ref.e4m3_encode(x, 1.0).tolist() == want
    assert ref.e4m3_encode(torch.tensor([float("nan")]), 1.0).tolist() == [0x7f]
    # the scale divides first, in single precision
    assert ref.e4m3_encode(torch.tensor([3.0, 0.75]), 0.5).tolist() == [0x4c, 0x3c]       # 6.0, 1.5


def test_encode_agrees_with_the_library_on_random_values():
    g = torch.Generator().manual_seed(3)
    x = torch.cat([torch.randn(20000, generator=g) * 3, torch.randn(20000, generator=g) * 100,
                   torch.randn(5000, generator=g) * 0.01]).clamp(-448, 448)
    got = ref.e4m3_encode(x, 1.0)
    lib = x.to(torch.float8_e4m3fn).view(torch.uint8)
    same = got == lib
    # the only codes that may differ are the two zeros
    assert bool(((got & 0x7f) == (lib & 0x7f))[~same].all()) and bool(((got & 0x7f) == 0)[~same].all())
    # round trip: decode(encode(x)) is the nearest representable value
    back = ref.e4m3_decode(got)
    grid = ref.e4m3_decode(torch.arange(0x7f, dtype=torch.uint8))
    nearest = (x.abs().double()[:, None] - grid[None, :]).abs().min(1).values
    assert torch.allclose((back.abs() - x.abs().double()).abs(), nearest, rtol=0, atol=0)


def test_fp8_cache_attention_is_the_attention_of_the_dequantised_values():
    cfg = inputs.VerifyConfig("f8", B=2, L=1, Hq=4, Hkv=2, D=16, T=6, C=2, S=2, V=16, prefix=(3, 20), tree="random",
                              kv_dtype=torch.bfloat16, logit_dtype=torch.float32, sigma_logit=1.0, draft="independent",
                              temperatures=(1.0,), seed=5, max_depth=4, fanout=(1, 2))
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen)
    t = inputs.layer_tensors(cfg, 0, n_slots)
    k_scale, v_scale = inputs.fp8_scales(cfg, 0)
    k8, v8 = ref.quantize_cache(t["k_cache"], k_scale), ref.quantize_cache(t["v_cache"], v_scale)
    ks8, vs8 = ref.quantize_cache(t["k_soft"], k_scale), ref.quantize_cache(t["v_soft"], v_scale)
    out, lse, st = ref.tree_attention_fp8(t["q"], k8, v8, k_scale, v_scale, seq_start, plen, ks8, vs8, parent, owner)
    # the same through the library's conversion of the codes, and the fp64 attention oracle
    deq = lambda c, s: c.view(torch.float8_e4m3fn).to(torch.float64) * s.double().view(1, -1, 1)
    want, want_lse, _ = ref.tree_attention(t["q"].double(), deq(k8, k_scale), deq(v8, v_scale), seq_start, plen,
                                           deq(ks8, k_scale), deq(vs8, v_scale), parent, owner)
    assert torch.equal(out, want) and torch.equal(lse, want_lse)
    # and it is close to, but not the same as, the attention of the unquantised cache
    full, _, _ = ref.tree_attention(t["q"], t["k_cache"], t["v_cache"], seq_start, plen, t["k_soft"], t["v_soft"], parent, owner)
    err = (out - full).abs().max().item()
    assert 1e-4 < err < 0.2
