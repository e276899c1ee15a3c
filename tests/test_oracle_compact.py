"""Pins of the oracle's KV compaction: the definition written out with plain tensor indexing."""
import torch

from oracle import ref


def _pools(L=3, n_slots=40, Hkv=2, D=8, seed=0):
    g = torch.Generator().manual_seed(seed)
    k = [torch.randn(n_slots, Hkv, D, generator=g).to(torch.bfloat16) for _ in range(L)]
    v = [torch.randn(n_slots, Hkv, D, generator=g).to(torch.bfloat16) for _ in range(L)]
    return k, v


def _path(nodes):
    p = torch.full((1, ref.MAX_DEPTH + 1), -1, dtype=torch.int32)
    p[0, :len(nodes)] = torch.tensor(nodes, dtype=torch.int32)
    return p


def test_gather_definition_and_untouched_prefix():
    k, v = _pools()
    k0 = [t.clone() for t in k]
    v0 = [t.clone() for t in v]
    seq_start = torch.tensor([3, 20])
    plen = torch.tensor([5, 7], dtype=torch.int32)
    path = torch.cat([_path([0, 1, 4, 6]), _path([0, 3])])
    alen = torch.tensor([3, 1], dtype=torch.int32)
    new_len = ref.kv_compact(k, v, seq_start, plen, alen, path)
    assert new_len.tolist() == [9, 9]
    for pools, olds in ((k, k0), (v, v0)):
        for t, o in zip(pools, olds):
            for b in range(2):
                s0, P, a = int(seq_start[b]), int(plen[b]), int(alen[b])
                assert torch.equal(t[s0:s0 + P + 1], o[s0:s0 + P + 1])          # prefix and root untouched
                for kk in range(1, a + 1):
                    assert torch.equal(t[s0 + P + kk], o[s0 + P + int(path[b, kk])])
            assert torch.equal(t[:3], o[:3]) and torch.equal(t[15:20], o[15:20])   # slots of nobody


def test_in_place_hazard_path_0_2_5():
    """Slot 2 is the destination of step 2 and the source of step 1: sources are the OLD cache."""
    k, v = _pools(L=1, n_slots=12)
    k0 = k[0].clone()
    ref.kv_compact(k, v, torch.tensor([0]), torch.tensor([4], dtype=torch.int32),
                   torch.tensor([2], dtype=torch.int32), _path([0, 2, 5]))
    assert torch.equal(k[0][4 + 1], k0[4 + 2]) and torch.equal(k[0][4 + 2], k0[4 + 5])


def test_accept_len_zero_is_a_no_op():
    k, v = _pools(L=2)
    k0 = [t.clone() for t in k]
    new_len = ref.kv_compact(k, v, torch.tensor([0]), torch.tensor([6], dtype=torch.int32),
                             torch.tensor([0], dtype=torch.int32), _path([0]))
    assert new_len.tolist() == [7]
    assert all(torch.equal(a, b) for a, b in zip(k, k0))
