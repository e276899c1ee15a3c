"""Host logic of the benchmark that needs no GPU: the byte / flop model, the per-rank sharding and the
max-over-ranks timing of a multi-rank run (two gloo ranks on the CPU)."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2603_08899_b200 import inputs  # noqa: E402


def test_attention_byte_and_flop_model_small_case():
    cfg = inputs.scaled(inputs.CONFIGS["llama8b"], B=2, prefix=(10, 20))
    plen = torch.tensor([10, 20], dtype=torch.int32)
    row = cfg.Hkv * cfg.D * 2
    kv = 2 * row * (10 + 64 + 20 + 64)
    soft = 2 * row * 16
    qo = 2 * 2 * 64 * cfg.Hq * cfg.D * 2
    assert bench.attention_bytes_per_layer(cfg, plen) == kv + soft + qo
    assert bench.attention_flops_per_layer(cfg, plen) == 4 * 64 * cfg.Hq * cfg.D * (10 + 20 + 2 * (64 + 16))
    # 4096 bytes of K+V per slot per layer for the three model shapes
    assert 2 * row == 4096


def test_step_bytes_counts_every_layer_both_logit_matrices_and_the_moved_rows():
    cfg = inputs.CONFIGS["llama8b"]
    plen = inputs.prefix_lens(cfg)
    a = bench.attention_bytes_per_layer(cfg, plen)
    got = bench.step_bytes(cfg, plen, accept_len_mean=3.0)
    logits = 2 * cfg.T * cfg.V * 2
    moved = 2 * 2 * 3 * 2048 * cfg.L          # K and V, read and written, 3 rows of 2048 B
    assert got == cfg.L * a + logits + moved


def test_rank_config_gives_every_rank_its_own_batch_of_the_same_shape():
    cfg = inputs.scaled(inputs.CONFIGS["batch32"], B=4)
    c0, c1 = bench.rank_config(cfg, 0), bench.rank_config(cfg, 1)
    assert c0 is cfg and c1.seed != c0.seed
    assert (c1.B, c1.L, c1.T, c1.C, c1.V) == (c0.B, c0.L, c0.T, c0.C, c0.V)
    assert not torch.equal(inputs.prefix_lens(c0), inputs.prefix_lens(c1))
    assert not torch.equal(inputs.trees(c0)[0], inputs.trees(c1)[0])


def test_profile_traffic_is_dropped_when_the_kernel_source_changed(tmp_path, monkeypatch):
    monkeypatch.setattr(bench, "ROOT", str(tmp_path))
    os.makedirs(tmp_path / "profiles")
    os.makedirs(tmp_path / "paper_2603_08899_b200" / "csrc")
    for name in bench.KERNEL_SOURCES["attention_tc_kernel"]:
        (tmp_path / "paper_2603_08899_b200" / "csrc" / name).write_text("// h1\n")
    (tmp_path / "paper_2603_08899_b200" / "csrc" / "attn_tc.cu").write_text("// v1\n")
    sha = bench.kernel_source_hash("attention_tc_kernel")
    (tmp_path / "profiles" / "attention_tc_kernel_batch32_L1.md").write_text(
        f"x\ntraffic_bytes_per_launch: 123\nkernel_source_sha256_16: {sha}\n")
    assert bench.profile_traffic("attention_tc_kernel", "batch32") == 123
    (tmp_path / "paper_2603_08899_b200" / "csrc" / "attn_tc.cu").write_text("// v2\n")
    assert bench.profile_traffic("attention_tc_kernel", "batch32") is None
    (tmp_path / "paper_2603_08899_b200" / "csrc" / "attn_tc.cu").write_text("// v1\n")
    assert bench.profile_traffic("attention_tc_kernel", "batch32") == 123
    (tmp_path / "paper_2603_08899_b200" / "csrc" / "attn_tc.cuh").write_text("// h2\n")     # the kernel's header counts too
    assert bench.profile_traffic("attention_tc_kernel", "batch32") is None
    assert bench.profile_traffic("attention_tc_kernel", "llama8b") is None


def _rank_main(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        total = bench.max_over_ranks(my_ms, dist, "cpu")
        value = bench.aggregate_value(world, 4, total)
        cfg = bench.rank_config(inputs.scaled(inputs.CONFIGS["batch32"], B=2), rank)
        out.put((rank, total, value, cfg.seed))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_ranks_time_and_the_aggregate():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]
    assert all(abs(r[2] - 2 * 4 / 0.015) < 1e-9 for r in res)
    assert res[0][3] != res[1][3]
