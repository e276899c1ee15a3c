#!/usr/bin/env python
"""Benchmark of the tree-verification step (L x tree attention + acceptance + KV compaction).

    python bench.py --gpus 1 --steps 20 --warmup 3                # this library, on the GPU
    python bench.py --impl reference --steps 2 --warmup 1         # the fp64 CPU oracle on the host cores
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...

Prints ONE JSON line.  Workload: seeded synthetic inputs shaped like a batched Llama-3.1-8B
verification step (32 sequences, ragged prefixes, 60-node trees + 4 contemplate rows).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2603_08899_b200 import inputs  # noqa: E402

ATTENTION_PATH = 0          # --attention-path
METRIC = "verify_steps_per_sec"
UNIT = "steps/s"


# ----------------------------------------------------------------------------- byte / flop model
def attention_bytes_per_layer(cfg, plen):
    """Algorithmic HBM bytes of one attention launch: every K and V row of every sequence read once
    (prefix + the R rows' own slots), the soft-prompt K/V once, Q read and O written once."""
    es = {torch.bfloat16: 2, torch.float32: 4, torch.float8_e4m3fn: 1}[cfg.kv_dtype]      # cache entries
    qs = 2 if cfg.kv_dtype == torch.float8_e4m3fn else es                                   # q and out (bf16 over an E4M3 cache)
    row = cfg.Hkv * cfg.D * es
    kv = 2 * row * int((plen.to(torch.int64) + cfg.R).sum())
    soft = 2 * row * cfg.S
    qo = 2 * cfg.B * cfg.R * cfg.Hq * cfg.D * qs
    return kv + soft + qo


def attention_flops_per_layer(cfg, plen):
    keys = int((plen.to(torch.int64) + cfg.R + cfg.S).sum())
    return 4 * cfg.R * cfg.Hq * cfg.D * keys


def step_bytes(cfg, plen, accept_len_mean):
    es = 2 if cfg.logit_dtype == torch.bfloat16 else 4
    logits = 2 * cfg.B * cfg.T * cfg.V * es
    row = cfg.Hkv * cfg.D * {torch.bfloat16: 2, torch.float32: 4, torch.float8_e4m3fn: 1}[cfg.kv_dtype]
    compact = int(2 * 2 * accept_len_mean * row * cfg.L * cfg.B)
    return cfg.L * attention_bytes_per_layer(cfg, plen) + logits + compact


def key_tiles_per_layer(cfg, plen):
    """128-key tiles one attention launch walks on the tensor-core path: per (sequence, KV head, group of
    64 query rows) the key tiles of prefix + R slots, plus one tile for the soft prompts."""
    n_rg = (cfg.R + 63) // 64
    per_seq = sum((int(p) + cfg.R + 127) // 128 + (1 if cfg.S else 0) for p in plen)
    return per_seq * cfg.Hkv * n_rg


def attention_lens(cfg, plen, launch_s, clocks, peaks, sm_count):
    """One attention launch against both ceilings.  `bound` is the ceiling that binds at the measured
    peaks (the larger of bytes / copy bandwidth and FLOPs / sustained bf16 matmul rate)."""
    a_bytes = attention_bytes_per_layer(cfg, plen)
    a_flops = attention_flops_per_layer(cfg, plen)
    # tensor ceiling of the type the products run in: E4M3 products at twice the measured bf16 rate (nominal ratio)
    tc_peak = peaks["bf16_tflops"] * (2.0 if cfg.kv_dtype == torch.float8_e4m3fn else 1.0)
    t_hbm, t_tc = a_bytes / (peaks["hbm_gbs"] * 1e9), a_flops / (tc_peak * 1e12)
    gbs, tf = a_bytes / launch_s / 1e9, a_flops / launch_s / 1e12
    mhz = clocks["sm_mhz"] if clocks and clocks.get("sm_mhz") else None
    tiles = key_tiles_per_layer(cfg, plen)
    return {"bound": "tensor" if t_tc > t_hbm else "hbm", "launch_us": launch_s * 1e6,
            "floor_us": {"hbm": t_hbm * 1e6, "tensor": t_tc * 1e6},
            "bytes_per_launch": a_bytes, "flops_per_launch": a_flops, "key_tiles_per_launch": tiles,
            "hbm_gbs": gbs, "frac_of_measured_hbm": gbs / peaks["hbm_gbs"], "frac_of_nominal_8TBs": gbs / 8000.0,
            "tensor_tflops": tf, "tensor_peak_tflops": tc_peak, "frac_of_measured_bf16_sustained": tf / tc_peak,
            # clock-independent figures: time x median SM clock under load
            "mcycles_per_launch": None if mhz is None else launch_s * mhz,
            "cycles_per_key_tile_per_sm": None if mhz is None else launch_s * mhz * 1e6 * sm_count / max(tiles, 1)}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1400.0, "source": "fallback"}


KERNEL_SOURCES = {"attention_fp8_kernel": ("attn_fp8.cu", "tc_walk.cuh", "tc_ptx.cuh", "attn_tc.cuh"),
                  "attention_pair_kernel": ("attn_tc2.cu", "tc_walk.cuh", "tc_ptx.cuh", "attn_tc.cuh"),
                  "attention_tc_kernel": ("attn_tc.cu", "tc_walk.cuh", "tc_ptx.cuh", "attn_tc.cuh"),
                  "attention_generic_kernel": ("attn_generic.cu",)}


def kernel_source_hash(kernel):
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES[kernel]:
        h.update(open(os.path.join(ROOT, "paper_2603_08899_b200", "csrc", name), "rb").read())
    return h.hexdigest()[:16]


def profile_traffic(kernel, workload):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel from the
    committed ncu summary of this workload; None when there is no summary or when the kernel's source has
    changed since the counters were taken (the summary records the source's hash)."""
    p = os.path.join(ROOT, "profiles", f"{kernel}_{workload}_L1.md")
    if not os.path.exists(p):
        return None
    traffic = sha = None
    for line in open(p):
        if line.startswith("traffic_bytes_per_launch:"):
            traffic = int(line.split(":")[1])
        if line.startswith("kernel_source_sha256_16:"):
            sha = line.split(":")[1].strip()
    if traffic is None or sha != kernel_source_hash(kernel):
        return None
    return traffic


def rank_config(cfg, rank):
    """Weak scaling by sequence: every rank verifies its own seeded batch of the same shape."""
    return inputs.scaled(cfg, seed=cfg.seed + 1000 * rank) if rank else cfg


def max_over_ranks(ms, dist, device):
    """Timing of a multi-rank run: the slowest rank's device time (no other collective is on the path)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(world, steps, total_ms):
    """Whole-job throughput: steps of all ranks over the slowest rank's time."""
    return world * steps / (total_ms * 1e-3)


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.Q}",
                                       "--format=csv,noheader,nounits", "-lms", "20"], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_prepare(cfg, target_visits=1e9, max_seqs=32):
    """Inputs of the bounded oracle sample (generation is not timed).  The number of sampled attention
    rows is set so that the sample visits at most about `target_visits` (row, key) pairs (capped at
    every output row of one layer of the sampled sequences): 10-20 s of work on 16 cores by default."""
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    nseq = min(cfg.B, max_seqs)
    sub = inputs.scaled(cfg, B=nseq)
    sp = {"cfg": cfg, "nseq": nseq, "plen_all": plen, "parent": parent[:nseq].contiguous(),
          "owner": owner[:nseq].contiguous(), "plen": plen[:nseq].contiguous()}
    sp["seq_start"], n_slots = inputs.cache_layout(sub, sp["plen"])
    sp["t"] = inputs.layer_tensors(sub, 0, n_slots)
    rows_per_seq = max(8, min(cfg.R * cfg.Hq, int(target_visits / max(1, int(sp["plen"].sum()) + nseq * cfg.R))))
    g = torch.Generator().manual_seed(11)
    sp["sel"] = [(b, int(torch.randint(0, cfg.R, (1,), generator=g)), int(torch.randint(0, cfg.Hq, (1,), generator=g)))
                 for b in range(nseq) for _ in range(rows_per_seq)]
    sp["tl"], sp["dl"] = inputs.logits(sub)
    sp["tok"] = inputs.draft_tokens(sub, sp["parent"], sp["dl"], 1.0)
    sp["u"] = inputs.uniforms(sub)
    return sp


def oracle_sample(sp):
    """Times the fp64 oracle, as it stands, on a bounded sample of the workload and scales the result
    to one whole step.  Sample: (row, head) outputs of layer 0 of the sampled sequences
    (attention cost is proportional to the visible keys, which the scaling uses), the acceptance walk
    of those sequences at full vocabulary, and the compaction of one layer."""
    from oracle import ref
    cfg, nseq, t = sp["cfg"], sp["nseq"], sp["t"]
    t0 = time.perf_counter()
    ref.tree_attention_rows(t["q"], t["k_cache"], t["v_cache"], sp["seq_start"], sp["plen"], t["k_soft"], t["v_soft"],
                            sp["parent"], sp["owner"], sp["sel"])
    t_attn = time.perf_counter() - t0
    keys_sampled = sum(int(sp["plen"][b]) + cfg.R + (cfg.S if r >= cfg.T else 0) for b, r, _ in sp["sel"])
    keys_step = cfg.L * cfg.Hq * sum((int(p) + cfg.R) * cfg.R + cfg.S * cfg.C for p in sp["plen_all"])
    t0 = time.perf_counter()
    o = ref.tree_accept(sp["tl"], sp["dl"], sp["tok"], sp["parent"], sp["owner"], sp["u"], temperature=1.0)
    t_acc = time.perf_counter() - t0
    kc, vc = t["k_cache"].clone(), t["v_cache"].clone()
    t0 = time.perf_counter()
    ref.kv_compact([kc], [vc], sp["seq_start"], sp["plen"], o["accept_len"], o["path"])
    t_cmp = time.perf_counter() - t0
    est = t_attn * keys_step / keys_sampled + (t_acc + t_cmp * cfg.L) * cfg.B / nseq
    return {"step_seconds_estimate": est, "sample_seconds": t_attn + t_acc + t_cmp, "cores": ref.num_threads(),
            "sample": f"{len(sp['sel'])} attention output rows of layer 0 over {nseq} sequences ({keys_sampled} key "
                      f"visits of {keys_step} per step), acceptance of {nseq} sequences at full vocabulary, "
                      f"compaction of 1 layer; scaled linearly to {cfg.L} layers x {cfg.B} sequences"}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sp = oracle_prepare(cfg, target_visits=args.reference_visits, max_seqs=args.reference_seqs)
    for i in range(args.warmup):
        oracle_sample(sp)
    t0 = time.perf_counter()
    res = [oracle_sample(sp) for i in range(args.steps)]
    wall = time.perf_counter() - t0
    est = statistics.mean(r["step_seconds_estimate"] for r in res)
    value = 1.0 / est
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": est * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "layers": cfg.L, "heads": f"{cfg.Hq}q/{cfg.Hkv}kv", "head_dim": cfg.D,
                       "tree_rows": cfg.T, "contemplate_rows": cfg.C, "soft_prompt": cfg.S, "vocab": cfg.V,
                       "prefix": "ragged U[512,16384]" if isinstance(cfg.prefix, tuple) else cfg.prefix,
                       "temperature": 1.0, "note": "oracle timed on a bounded sample, scaled to a whole step",
                       "sample_wall_seconds": wall},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": res[0]["cores"], "kind": "oracle",
                             "sample": res[0]["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- GPU leg
def build_workload(cfg, device, rank, temperature=1.0):
    from paper_2603_08899_b200.step import VerifyStep
    cfg = rank_config(cfg, rank)
    parent, owner = inputs.trees(cfg)
    plen = inputs.prefix_lens(cfg)
    seq_start, n_slots = inputs.cache_layout(cfg, plen)
    q, k, v, ks, vs, out, scales = [], [], [], [], [], [], []
    for l in range(cfg.L):
        t = inputs.layer_tensors(cfg, l, n_slots, device=device)
        q.append(t["q"]); k.append(t["k_cache"]); v.append(t["v_cache"]); ks.append(t["k_soft"]); vs.append(t["v_soft"])
        out.append(torch.empty_like(t["q"]))
        if "k_scale" in t:
            scales.append((t["k_scale"], t["v_scale"]))
    tl, dl = inputs.logits(cfg, device=device)
    tok = inputs.draft_tokens(cfg, parent, dl, temperature)
    u = inputs.uniforms(cfg)
    step = VerifyStep(cfg, n_slots, device=device)
    if ATTENTION_PATH:
        from paper_2603_08899_b200 import binding as cb
        cb.confu_set_option(step.ctx, cb.OPT_ATTENTION_PATH, ATTENTION_PATH)
    step.bind(q, k, v, ks if cfg.S else None, vs if cfg.S else None, out, seq_start.to(device), plen.to(device),
              parent.to(device), owner.to(device) if cfg.C else None, tl, dl, tok.to(device), u.to(device),
              kv_scales=scales or None)
    host = {"parent": parent, "owner": owner, "plen": plen, "seq_start": seq_start, "tok": tok, "u": u}
    return cfg, step, host


def spot_check(cfg, step, host):
    """Before timing: the acceptance outputs of the first sequences against the oracle (cheap)."""
    from oracle import ref
    n = min(cfg.B, 2)
    o = ref.tree_accept(step.tl[:n].cpu(), step.dl[:n].cpu(), host["tok"][:n], host["parent"][:n], host["owner"][:n],
                        host["u"][:n], temperature=1.0)
    ok = True
    for b in range(n):
        same = step.accept_len[b].item() == o["accept_len"][b].item() and \
            step.next_token[b].item() == o["next_token"][b].item()
        ok &= bool(same or o["ratio_margin"][b].item() < 1e-5 or o["resample_margin"][b].item() < 1e-5)
    return ok


def time_other_workload(name, temperature, device, gpu_index, peaks, min_seconds=1.0):
    """One more workload of the table, timed as replays of its captured step (one graph launch per step)
    for at least min_seconds (so that the clock sampler sees the load), its KV freed afterwards.  Returns the record that goes
    under config.workloads[name]."""
    from paper_2603_08899_b200 import step as step_mod
    cfg, step, host = build_workload(inputs.CONFIGS[name], device, 0, temperature)
    plen = host["plen"]
    for _ in range(3):
        step.status.zero_()
        step.run(temperature)
    torch.cuda.synchronize()
    status_ok = bool((step.status == 0).all().item())
    step.capture(temperature)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        step.replay()
    e1.record()
    torch.cuda.synchronize()
    n = int(min(20000, max(20, min_seconds * 1e3 / max(e0.elapsed_time(e1) / 5, 1e-3))))
    # the parts of a step from replays as four graphs (a tenth as many), the step itself as one graph per step
    n_parts = max(20, n // 10)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(n_parts)]
    for i in range(n_parts):
        step.replay(ev[i])
    torch.cuda.synchronize()
    ms_attn = statistics.mean(ev[i][1].elapsed_time(ev[i][2]) for i in range(n_parts))
    ms_acc = statistics.mean(ev[i][2].elapsed_time(ev[i][3]) for i in range(n_parts))
    ev_step = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    sampler = ClockSampler(gpu_index)
    torch.cuda.synchronize()
    for i in range(n):
        ev_step[i].record()
        step.replay_step()
    ev_step[n].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = [ev_step[i].elapsed_time(ev_step[i + 1]) for i in range(n)]
    total_ms = ev_step[0].elapsed_time(ev_step[n])
    alen = step.accept_len.float().mean().item()
    sbytes = step_bytes(cfg, plen, alen) if temperature > 0 else \
        step_bytes(cfg, plen, alen) - cfg.B * cfg.T * cfg.V * step.tl.element_size()       # greedy reads the target matrix only
    rec = {"temperature": temperature, "steps": n, "ms_per_step": total_ms / n, "ms_per_step_median": statistics.median(ms),
           "ms_per_step_min": min(ms), "steps_per_sec": n / (total_ms * 1e-3),
           "parts_ms": {"attention": ms_attn, "accept": ms_acc},
           "attention": attention_lens(cfg, plen, ms_attn * 1e-3 / cfg.L, clocks, peaks, step_mod.sm_count(step)),
           "step_bytes": sbytes, "step_frac_of_measured_hbm": sbytes / (total_ms / n * 1e-3) / 1e9 / peaks["hbm_gbs"],
           "mcycles_per_step": None if not clocks.get("sm_mhz") else total_ms / n * 1e-3 * clocks["sm_mhz"],
           "mean_accept_len": alen, "status_ok": status_ok, "clocks": clocks}
    step.close()
    del step, host
    torch.cuda.empty_cache()
    return rec


def oracle_one_thread(names):
    """The oracle on ONE host thread (its OpenMP loops cut to a single thread), per workload, by the
    same bounded-sample method as the reference arm: a child process of this script."""
    out = {}
    for name in names:
        env = dict(os.environ, OMP_NUM_THREADS="1")
        for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
            env.pop(k, None)
        try:
            r = subprocess.run([sys.executable, os.path.abspath(__file__), "--impl", "reference", "--config", name,
                                "--steps", "1", "--warmup", "0", "--reference-visits", "2e7", "--reference-seqs", "1"],
                               env=env, capture_output=True, text=True, timeout=240)
            d = json.loads(r.stdout.strip().splitlines()[-1])
            out[name] = {"value": d["value"], "unit": UNIT, "cores": d["cpu_baseline"]["cores"],
                         "sample": d["cpu_baseline"]["sample"]}
        except Exception as e:                                              # reported, never fatal for the GPU line
            out[name] = {"error": repr(e)[:200]}
    return out


def run_ours(args, cfg):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; this library has no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(device))
    from paper_2603_08899_b200 import binding as cb
    from paper_2603_08899_b200 import step as step_mod

    cfg, step, host = build_workload(cfg, device, rank)
    plen = host["plen"]

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    for _ in range(args.warmup):
        step.status.zero_()
        step.run(1.0)
    torch.cuda.synchronize()
    checked = spot_check(cfg, step, host) if rank == 0 else True
    status_ok = bool((step.status == 0).all().item())
    # The timed steps replay the step's launches from a CUDA graph captured here (the same kernels with
    # the same arguments; the host then issues one graph launch per step instead of 2 L + 4 kernels).
    use_graph = not args.no_graph
    if use_graph:
        step.capture(1.0)
        for _ in range(2):
            step.replay_step()
        torch.cuda.synchronize()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
    ev_step = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    t_begin = torch.cuda.Event(enable_timing=True)
    t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for i in range(args.steps):
        if use_graph:
            ev_step[i].record()
            step.replay_step()              # the whole step: one graph launch
            continue
        ev[i][0].record()
        step.run_plan()
        ev[i][1].record()
        step.run_layers()
        ev[i][2].record()
        step.run_accept(1.0)
        ev[i][3].record()
        step.run_compact()
        ev[i][4].record()
    ev_step[args.steps].record()
    t_end.record()
    barrier()
    clocks = sampler.stop() if sampler else None
    if use_graph:
        # the parts of a step (plan | attention | acceptance | compaction), timed apart from the headline:
        # the same steps once more as four graphs with events between them
        for i in range(args.steps):
            step.replay(ev[i])
        torch.cuda.synchronize()
    total_ms = max_over_ranks(t_begin.elapsed_time(t_end), dist, device)
    ms_step = total_ms / args.steps
    part = lambda a, b: statistics.mean(ev[i][a].elapsed_time(ev[i][b]) for i in range(args.steps))  # noqa: E731
    ms_plan, ms_attn, ms_acc, ms_cmp = part(0, 1), part(1, 2), part(2, 3), part(3, 4)
    ms_each = [ev_step[i].elapsed_time(ev_step[i + 1]) for i in range(args.steps)] if use_graph else \
        [ev[i][0].elapsed_time(ev[i][4]) for i in range(args.steps)]
    alen = step.accept_len.float().mean().item()

    def time_accept_variants():
        """Outside the timed step: the acceptance variants that read only the walked path's rows.
        ms per call, and the logit bytes each one actually reads (from its own accepted lengths)."""
        out = {}
        for name in ("lazy", "match"):
            def call():
                if name == "lazy":
                    step.run_accept(1.0, 1 | cb.ACCEPT_LAZY)
                else:
                    cb.confu_tree_accept_match(step.ctx, cfg.B, cfg.T, cfg.C, cfg.V, cfg.logit_dtype, step.tl, step.tokens,
                                               step.parent, step.con_owner, step.uniforms, 1.0, step.accept_len, step.path,
                                               step.next_token, step.future_row, step.counters, step.status)
            call()
            torch.cuda.synchronize()
            e = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
            for i in range(5):
                e[i].record()
                call()
            e[5].record()
            torch.cuda.synchronize()
            rows = (step.accept_len.long() + 1).sum().item() * (2 if name == "lazy" else 1)
            out[name] = {"ms": e[0].elapsed_time(e[5]) / 5, "logit_bytes_read": rows * cfg.V * step.tl.element_size(),
                         "mean_accept_len": step.accept_len.float().mean().item()}
        step.run_accept(1.0)                      # leave the default rule's results in place
        torch.cuda.synchronize()
        return out

    accept_variants = time_accept_variants() if rank == 0 else None

    def measure_e2e():
        # ---- end to end: this step's inputs come from pinned host memory, results go back ----
        h = {"q": [t.cpu().pin_memory() for t in step.q],
             "krows": [], "vrows": [],
             "tl": step.tl.cpu().pin_memory(), "dl": step.dl.cpu().pin_memory(),
             "tok": host["tok"].pin_memory(), "u": host["u"].pin_memory(), "parent": host["parent"].pin_memory(),
             "owner": host["owner"].pin_memory()}
        R = cfg.R
        idx = torch.cat([torch.arange(int(host["seq_start"][b]) + int(plen[b]), int(host["seq_start"][b]) + int(plen[b]) + R)
                         for b in range(cfg.B)]).to(device)
        for l in range(cfg.L):
            h["krows"].append(step.k[l][idx].view(cfg.B, R, cfg.Hkv, cfg.D).cpu().pin_memory())
            h["vrows"].append(step.v[l][idx].view(cfg.B, R, cfg.Hkv, cfg.D).cpu().pin_memory())
        d_krows = [torch.empty_like(t, device=device) for t in h["krows"]]     # per layer: copies run ahead of compute
        d_vrows = [torch.empty_like(t, device=device) for t in h["vrows"]]
        res_host = {k: torch.empty_like(getattr(step, k), device="cpu").pin_memory()
                    for k in ("accept_len", "path", "next_token", "future_row", "new_prefix_len", "status")}
        h2d = sum(t.numel() * t.element_size() for t in h["q"] + h["krows"] + h["vrows"]) + \
            sum(h[k].numel() * h[k].element_size() for k in ("tl", "dl", "tok", "u", "parent", "owner"))
        d2h = sum(t.numel() * t.element_size() for t in res_host.values())

        # All inputs of a step travel on one copy stream in the order the step uses them (tree arrays, then
        # layer by layer Q and the rows' K/V, the logits last), each followed by an event the compute stream
        # waits for; the copies of the next step start when this step's last kernel has been enqueued and
        # finished (its inputs must not be overwritten under it).
        copy_stream = torch.cuda.Stream()
        ev_tree = torch.cuda.Event()
        ev_layer = [torch.cuda.Event() for _ in range(cfg.L)]
        ev_logits, ev_done = torch.cuda.Event(), torch.cuda.Event()
        ev_done.record()

        def e2e_step():
            main = torch.cuda.current_stream()
            copy_stream.wait_event(ev_done)
            with torch.cuda.stream(copy_stream):
                step.parent.copy_(h["parent"], non_blocking=True)
                if cfg.C:
                    step.con_owner.copy_(h["owner"], non_blocking=True)
                ev_tree.record(copy_stream)
                for l in range(cfg.L):
                    step.q[l].copy_(h["q"][l], non_blocking=True)
                    d_krows[l].copy_(h["krows"][l], non_blocking=True)
                    d_vrows[l].copy_(h["vrows"][l], non_blocking=True)
                    ev_layer[l].record(copy_stream)
                step.tl.copy_(h["tl"], non_blocking=True)
                step.dl.copy_(h["dl"], non_blocking=True)
                step.tokens.copy_(h["tok"], non_blocking=True)
                step.uniforms.copy_(h["u"], non_blocking=True)
                ev_logits.record(copy_stream)
            main.wait_event(ev_tree)
            cb.confu_tree_plan(step.ctx, step.dims, step.seq_start, step.prefix_len, step.parent, step.con_owner,
                               step.plan, step.status)
            for l in range(cfg.L):
                main.wait_event(ev_layer[l])
                cb.confu_kv_append(step.ctx, step.dims, d_krows[l], d_vrows[l], step.k[l], step.v[l], step.seq_start,
                                   step.prefix_len)
                cb.confu_tree_attention(step.ctx, step.dims, step.q[l], step.k[l], step.v[l], step.n_slots,
                                        step.seq_start, step.prefix_len, step.ks[l] if step.ks else None,
                                        step.vs[l] if step.vs else None, None, None, step.plan, step.out[l], None,
                                        step.status)
            main.wait_event(ev_logits)
            step.run_accept(1.0)
            step.run_compact()
            ev_done.record(main)
            for k, t in res_host.items():
                t.copy_(getattr(step, k), non_blocking=True)

        n_e2e = max(2, min(args.steps, 5))
        e2e_step()
        torch.cuda.synchronize()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(n_e2e):
            e2e_step()
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1), dist, device)
        e2e_value = aggregate_value(world, n_e2e, e2e_ms)

        return e2e_value, e2e_ms / n_e2e, n_e2e, h2d, d2h

    e2e = None if args.no_e2e else measure_e2e()

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peaks = measured_peaks()
    sm_count = step_mod.sm_count(step)
    kname = step.attention_kernel_name()
    lens = attention_lens(cfg, plen, ms_attn * 1e-3 / cfg.L, clocks, peaks, sm_count)
    # the other workloads of the table (batch 1 shapes of the three model families, and one contemplate
    # row per node), each with its own clock record; one GPU only, after the main workload's memory is gone
    others = None
    if world == 1 and not args.no_other_workloads and args.config == "batch32":
        launches_main = args.steps * step.launches_per_step()
        step.close()
        for name in ("q", "k", "v", "ks", "vs", "out", "tl", "dl", "graphs", "graph_step"):
            setattr(step, name, None)
        torch.cuda.empty_cache()
        others = {}
        for name, temperature in (("llama3b", 1.0), ("llama8b", 1.0), ("llama8b", 0.7), ("qwen4b", 1.0), ("qwen4b", 0.0),
                                  ("llama8b_30", 1.0), ("llama8b_2t", 1.0), ("batch32_2t", 1.0), ("batch32_fp8", 1.0)):
            key = name if temperature == 1.0 else name + ("_greedy" if temperature == 0 else f"_t{temperature:g}")
            others[key] = time_other_workload(name, temperature, device, local, peaks)
    else:
        launches_main = args.steps * step.launches_per_step()
    sbytes = step_bytes(cfg, plen, alen)
    cpu = oracle_sample(oracle_prepare(cfg)) if not args.no_cpu_baseline else None
    cpu_1t = oracle_one_thread(("tiny", "llama3b")) if not args.no_cpu_baseline else None
    tensor_bound = lens["bound"] == "tensor"
    line = {
        "metric": METRIC, "value": aggregate_value(world, args.steps, total_ms), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "ms_per_step_median": statistics.median(ms_each),
        "ms_per_step_min": min(ms_each), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "layers": cfg.L, "heads": f"{cfg.Hq}q/{cfg.Hkv}kv", "head_dim": cfg.D,
                   "tree_rows": cfg.T, "contemplate_rows": cfg.C, "soft_prompt": cfg.S, "vocab": cfg.V,
                   "prefix": "ragged U[512,16384]" if isinstance(cfg.prefix, tuple) else cfg.prefix,
                   "sum_prefix": int(plen.sum()), "temperature": 1.0,
                   "l2": "inputs larger than L2 (every layer has its own KV; no flush needed)",
                   "parallelism": f"replicas x{world}, sequences sharded, no collective",
                   "parts_ms": {"plan": ms_plan, "attention": ms_attn, "accept": ms_acc, "compact": ms_cmp},
                   "launch": "1 CUDA graph per step; parts_ms from the same steps replayed as 4 graphs (plan | L attention layers | acceptance | compaction) after the timed region" if use_graph
                             else "kernel launches from the host, one by one",
                   "accept_rule": "ratio test, statistics of all rows (timed); variants timed apart: " \
                                  "lazy = same rule, rows on demand; match = sample-and-match, rows on demand",
                   "accept_variants": accept_variants,
                   "step_bytes": sbytes, "step_gbs": sbytes / (ms_step * 1e-3) / 1e9,
                   "step_frac_of_hbm_roofline": sbytes / (ms_step * 1e-3) / 1e9 / peaks["hbm_gbs"],
                   "mcycles_per_step": None if not (clocks and clocks.get("sm_mhz")) else ms_step * 1e-3 * clocks["sm_mhz"],
                   "mean_accept_len": alen, "status_ok": status_ok, "spot_check_vs_oracle": checked,
                   "workloads": others},
        # The dominant kernel (one attention launch = kernel + merge of the split partials) against the
        # ceiling that binds at the measured peaks; the other ceiling's figures stand beside it.
        "roofline": {"bound": lens["bound"], "kernel": kname,
                     "achieved": lens["tensor_tflops"] if tensor_bound else lens["hbm_gbs"],
                     "peak": peaks["bf16_tflops"] if tensor_bound else peaks["hbm_gbs"],
                     "unit": "TFLOP/s" if tensor_bound else "GB/s",
                     "frac": lens["frac_of_measured_bf16_sustained"] if tensor_bound else lens["frac_of_measured_hbm"],
                     "traffic": profile_traffic(kname, inputs.CONFIGS[args.config].name),
                     "peak_source": peaks["source"] + (" (sustained bf16 matmul rate: the kernel is timed inside a long step)"
                                                       if tensor_bound else " (copy bandwidth)"),
                     "hbm": {"achieved": lens["hbm_gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": lens["frac_of_measured_hbm"], "frac_of_nominal_8TBs": lens["frac_of_nominal_8TBs"]},
                     "tensor": {"achieved": lens["tensor_tflops"], "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                "frac": lens["frac_of_measured_bf16_sustained"]},
                     "floor_us": lens["floor_us"], "launch_ms": lens["launch_us"] * 1e-3,
                     "bytes_per_launch": lens["bytes_per_launch"], "flops_per_launch": lens["flops_per_launch"],
                     "key_tiles_per_launch": lens["key_tiles_per_launch"],
                     "cycles_per_key_tile_per_sm": lens["cycles_per_key_tile_per_sm"]},
        "e2e": None if e2e is None else {
            "value": e2e[0], "unit": UNIT, "h2d_bytes_per_step": e2e[3], "d2h_bytes_per_step": e2e[4],
            "ms_per_step": e2e[1], "steps": e2e[2],
            "note": "per step: Q, the R rows' K/V (all layers), both logit matrices, tree arrays and uniforms "
                    "copied from pinned host memory on a copy stream that runs ahead of the compute stream (an event per layer); "
                    "results copied back; the prefix KV cache is resident state"},
        "gpu_launches": launches_main,
        "clocks": clocks,
    }
    if cpu is not None:
        line["cpu_baseline"] = {"value": 1.0 / cpu["step_seconds_estimate"], "unit": UNIT, "cores": cpu["cores"],
                                "kind": "oracle", "sample": cpu["sample"], "sample_seconds": cpu["sample_seconds"],
                                "one_thread": cpu_1t}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="batch32", choices=list(inputs.CONFIGS))
    ap.add_argument("--no-graph", action="store_true", help="time kernel launches issued one by one from the host")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-other-workloads", action="store_true", help="time the chosen workload only")
    ap.add_argument("--attention-path", type=int, default=0,
                    help="CONFU_ATTENTION_* for A/B runs: 0 the library's choice, 2 one CTA per SM, 3 CTA pairs")
    ap.add_argument("--reference-visits", type=float, default=1.2e8,
                    help="--impl reference: (row, key) pairs one timed sample of the oracle's attention visits")
    ap.add_argument("--reference-seqs", type=int, default=8, help="--impl reference: sequences in one sample")
    ap.add_argument("--layers", type=int, default=0, help="cut the layer count (profiling runs; named in config.workload)")
    ap.add_argument("--batch", type=int, default=0, help="cut the batch (profiling runs; named in config.workload)")
    args = ap.parse_args()
    global ATTENTION_PATH
    ATTENTION_PATH = args.attention_path
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = inputs.CONFIGS[args.config]
    cut = {k: v for k, v in (("L", args.layers), ("B", args.batch)) if v > 0}
    if cut:
        cfg = inputs.scaled(cfg, name=cfg.name + "[" + ",".join(f"{k}={v}" for k, v in cut.items()) + "]", **cut)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
