"""GPU parity of confu_kv_compact against the oracle's definition: byte-exact."""
import pytest
import torch

from oracle import ref
from paper_2603_08899_b200 import binding as cb
from tests import harness as H

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    g = H.Gpu()
    yield g
    g.close()


def _paths(rows):
    p = torch.full((len(rows), cb.MAX_DEPTH + 1), -1, dtype=torch.int32)
    for i, r in enumerate(rows):
        p[i, :len(r)] = torch.tensor(r, dtype=torch.int32)
    return p


def _run(gpu, dtype, Hkv, D, L, paths, plen_list, R=64, seed=0):
    B = len(paths)
    g = torch.Generator().manual_seed(seed)
    plen = torch.tensor(plen_list, dtype=torch.int32)
    sizes = plen.to(torch.int64) + R
    seq_start = torch.zeros(B, dtype=torch.int64)
    seq_start[1:] = torch.cumsum(sizes, 0)[:-1]
    n_slots = int(sizes.sum()) + 5
    k = [torch.randn(n_slots, Hkv, D, generator=g).to(dtype) for _ in range(L)]
    v = [torch.randn(n_slots, Hkv, D, generator=g).to(dtype) for _ in range(L)]
    path = _paths(paths)
    alen = torch.tensor([len(p) - 1 for p in paths], dtype=torch.int32)
    kd = [t.cuda() for t in k]
    vd = [t.cuda() for t in v]
    kp = torch.tensor([t.data_ptr() for t in kd], dtype=torch.int64, device="cuda")
    vp = torch.tensor([t.data_ptr() for t in vd], dtype=torch.int64, device="cuda")
    new_len = torch.zeros(B, dtype=torch.int32, device="cuda")
    dims = cb.make_dims(B, Hkv, Hkv, D, R, 0, 0, dtype)          # T = 64: node ids up to 63 are valid
    cb.confu_kv_compact(gpu.ctx, dims, L, kp, vp, seq_start.cuda(), plen.cuda(), alen.cuda(), path.cuda(), new_len,
                        None)
    torch.cuda.synchronize()
    want_len = ref.kv_compact(k, v, seq_start, plen, alen, path)
    assert new_len.cpu().tolist() == want_len.tolist()
    for b in range(B):
        lo, hi = int(seq_start[b]), int(seq_start[b]) + int(want_len[b])
        for l in range(L):
            assert torch.equal(kd[l].cpu()[lo:hi], k[l][lo:hi]), (b, l)
            assert torch.equal(vd[l].cpu()[lo:hi], v[l][lo:hi]), (b, l)
    # nothing outside the sequences' own slots may change
    for l in range(L):
        assert torch.equal(kd[l].cpu()[n_slots - 5:], k[l][n_slots - 5:])


def test_llm_shaped_rows_bf16(gpu):
    _run(gpu, torch.bfloat16, 8, 128, 3, [[0, 2, 5], [0], [0, 1, 2, 3, 4, 5, 6, 7], [0, 3, 9, 20, 41, 59]],
         [17, 1, 300, 64])


def test_in_place_hazard_and_long_chain(gpu):
    chain = list(range(0, 64))
    skip = [0] + list(range(2, 64, 2))
    _run(gpu, torch.bfloat16, 2, 64, 2, [[0, 2, 5], chain, skip, [0, 63]], [4, 0, 9, 100], seed=1)


def test_fp32_rows_and_no_layers(gpu):
    _run(gpu, torch.float32, 2, 64, 1, [[0, 1, 3], [0, 5]], [3, 8], seed=2)
    _run(gpu, torch.float32, 2, 64, 0, [[0, 1, 3], [0, 5]], [3, 8], seed=3)
