"""Seeded synthetic inputs for the tree-verification step.

This module only *draws inputs*: shapes, trees, random tensors, draft tokens.
It contains none of the method's arithmetic (no attention, no acceptance, no
compaction) and is the one module the CUDA tests, the CPU oracle tests and the
benchmark all share.

The five workloads stand in for verification steps of Llama-3.2-3B,
Llama-3.1-8B and Qwen3-4B decoding (only the public shape parameters of those
models are used; there are no weights, prompts or benchmark items here).
"""
from dataclasses import dataclass, field
from typing import Tuple, Union

import numpy as np
import torch


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int                      # sequences
    L: int                      # attention layers
    Hq: int
    Hkv: int
    D: int
    T: int                      # tree rows, root included
    C: int                      # contemplate rows
    S: int                      # soft-prompt KV entries (shared by all sequences)
    V: int                      # vocabulary
    prefix: Union[int, Tuple[int, int]]   # fixed length, or (lo, hi) inclusive for a ragged batch
    tree: str                   # "chain" | "random"
    kv_dtype: torch.dtype
    logit_dtype: torch.dtype
    sigma_logit: float          # std of the target logits
    draft: str                  # "independent" | "noise" (draft = target + N(0,1))
    temperatures: Tuple[float, ...]
    seed: int
    max_depth: int = 7
    fanout: Tuple[int, int] = (1, 4)
    fixed_owners: Tuple[int, ...] = field(default=())

    @property
    def R(self) -> int:
        return self.T + self.C


CONFIGS = {
    "tiny": VerifyConfig("tiny", B=1, L=1, Hq=4, Hkv=2, D=64, T=8, C=2, S=2, V=1000, prefix=256,
                         tree="chain", kv_dtype=torch.float32, logit_dtype=torch.float32,
                         sigma_logit=2.0, draft="independent", temperatures=(1.0, 0.0), seed=1,
                         fixed_owners=(3, 7)),
    "llama3b": VerifyConfig("llama3b", B=1, L=28, Hq=24, Hkv=8, D=128, T=60, C=4, S=16, V=128256,
                            prefix=2048, tree="random", kv_dtype=torch.bfloat16,
                            logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="independent",
                            temperatures=(1.0,), seed=2),
    "llama8b": VerifyConfig("llama8b", B=1, L=32, Hq=32, Hkv=8, D=128, T=60, C=4, S=16, V=128256,
                            prefix=4096, tree="random", kv_dtype=torch.bfloat16,
                            logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                            temperatures=(1.0,), seed=3),
    "qwen4b": VerifyConfig("qwen4b", B=1, L=36, Hq=32, Hkv=8, D=128, T=60, C=4, S=16, V=151936,
                           prefix=8192, tree="random", kv_dtype=torch.bfloat16,
                           logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                           temperatures=(1.0, 0.0), seed=4),
    "batch32": VerifyConfig("batch32", B=32, L=32, Hq=32, Hkv=8, D=128, T=60, C=4, S=16, V=128256,
                            prefix=(512, 16384), tree="random", kv_dtype=torch.bfloat16,
                            logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                            temperatures=(1.0,), seed=5),
    # one contemplate row per draft node (the verification forward of Sec. 3.1 processes 2T rows)
    "llama8b_2t": VerifyConfig("llama8b_2t", B=1, L=32, Hq=32, Hkv=8, D=128, T=60, C=60, S=16, V=128256,
                               prefix=4096, tree="random", kv_dtype=torch.bfloat16,
                               logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                               temperatures=(1.0,), seed=6),
    # the size Sec. 3.1 calls typical: a draft tree of 30 nodes, one contemplate row each
    "llama8b_30": VerifyConfig("llama8b_30", B=1, L=32, Hq=32, Hkv=8, D=128, T=30, C=30, S=16, V=128256,
                               prefix=4096, tree="random", kv_dtype=torch.bfloat16,
                               logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                               temperatures=(1.0,), seed=8),
    # the batched workload over an 8-bit floating point (E4M3) cache with one scale per KV head
    "batch32_fp8": VerifyConfig("batch32_fp8", B=32, L=32, Hq=32, Hkv=8, D=128, T=60, C=4, S=16, V=128256,
                                prefix=(512, 16384), tree="random", kv_dtype=torch.float8_e4m3fn,
                                logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                                temperatures=(1.0,), seed=5),
    "batch32_2t": VerifyConfig("batch32_2t", B=32, L=32, Hq=32, Hkv=8, D=128, T=60, C=60, S=16, V=128256,
                               prefix=(512, 16384), tree="random", kv_dtype=torch.bfloat16,
                               logit_dtype=torch.bfloat16, sigma_logit=3.0, draft="noise",
                               temperatures=(1.0,), seed=7),
}


def scaled(cfg: VerifyConfig, **kw) -> VerifyConfig:
    """A copy of cfg with some fields replaced (smaller test-sized variants)."""
    d = {f: getattr(cfg, f) for f in cfg.__dataclass_fields__}
    d.update(kw)
    return VerifyConfig(**d)


def _rng(cfg: VerifyConfig, stream: int) -> np.random.Generator:
    return np.random.default_rng([cfg.seed, stream])


def _gen(cfg: VerifyConfig, stream: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 1_000_003 + stream)
    return g


# ---------------------------------------------------------------- trees
def random_tree(rng: np.random.Generator, T: int, max_depth: int = 7, fanout=(1, 4)) -> np.ndarray:
    """Breadth-first random tree: each expanded node below max_depth gets U{fanout} children
    (cut to the nodes still missing); nodes are numbered in BFS order, so parent[i] < i.
    Redrawn if the frontier dies out before T nodes exist."""
    while True:
        parent = [-1]
        depth = [0]
        frontier = [0]
        while frontier and len(parent) < T:
            nxt = []
            for u in frontier:
                if len(parent) >= T:
                    break
                if depth[u] >= max_depth:
                    continue
                f = int(rng.integers(fanout[0], fanout[1] + 1))
                f = min(f, T - len(parent))
                for _ in range(f):
                    parent.append(u)
                    depth.append(depth[u] + 1)
                    nxt.append(len(parent) - 1)
            frontier = nxt
        if len(parent) == T:
            return np.asarray(parent, dtype=np.int32)


def chain_tree(T: int) -> np.ndarray:
    return np.arange(-1, T - 1, dtype=np.int32)


def star_tree(T: int) -> np.ndarray:
    p = np.zeros(T, dtype=np.int32)
    p[0] = -1
    return p


def trees(cfg: VerifyConfig):
    """parent [B,T] int32 and con_owner [B,C] int32 (distinct owners, increasing)."""
    rng = _rng(cfg, 1)
    parent = np.zeros((cfg.B, cfg.T), dtype=np.int32)
    owner = np.zeros((cfg.B, cfg.C), dtype=np.int32)
    for b in range(cfg.B):
        if cfg.tree == "chain":
            parent[b] = chain_tree(cfg.T)
        elif cfg.tree == "star":
            parent[b] = star_tree(cfg.T)
        else:
            parent[b] = random_tree(rng, cfg.T, cfg.max_depth, cfg.fanout)
        if cfg.fixed_owners:
            owner[b] = np.asarray(cfg.fixed_owners, dtype=np.int32)
        elif cfg.C:
            owner[b] = np.sort(rng.choice(cfg.T, size=cfg.C, replace=False)).astype(np.int32)
    return torch.from_numpy(parent), torch.from_numpy(owner)


def prefix_lens(cfg: VerifyConfig) -> torch.Tensor:
    if isinstance(cfg.prefix, tuple):
        rng = _rng(cfg, 2)
        p = rng.integers(cfg.prefix[0], cfg.prefix[1] + 1, size=cfg.B)
    else:
        p = np.full(cfg.B, cfg.prefix)
    return torch.from_numpy(p.astype(np.int32))


def cache_layout(cfg: VerifyConfig, prefix_len: torch.Tensor, pad_slots: int = 0):
    """Packed pool: sequence b owns slots seq_start[b] .. +prefix_len[b]+R-1.  Returns (seq_start, n_slots)."""
    sizes = prefix_len.to(torch.int64) + cfg.R
    seq_start = torch.zeros(cfg.B, dtype=torch.int64)
    if cfg.B > 1:
        seq_start[1:] = torch.cumsum(sizes, 0)[:-1]
    return seq_start, int(sizes.sum().item()) + pad_slots


# ---------------------------------------------------------------- tensors
def _randn(shape, gen, device, dtype, std=1.0):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32)
    if std != 1.0:
        x = x * std
    return x.to(dtype)


def layer_tensors(cfg: VerifyConfig, layer: int, n_slots: int, device="cpu", tree_key_gain: float = 1.0,
                  seq_start=None, prefix_len=None):
    """Q, this layer's K/V pool and the soft-prompt K/V, all ~N(0,1) in cfg.kv_dtype.
    tree_key_gain > 1 scales the keys of the tree slots so that tree columns dominate the softmax
    (makes mask mistakes visible at long prefixes)."""
    g = _gen(cfg, 100 + layer, device)
    fp8 = cfg.kv_dtype == torch.float8_e4m3fn
    dt = torch.bfloat16 if fp8 else cfg.kv_dtype
    q = _randn((cfg.B, cfg.R, cfg.Hq, cfg.D), g, device, dt)
    k = _randn((n_slots, cfg.Hkv, cfg.D), g, device, dt)
    v = _randn((n_slots, cfg.Hkv, cfg.D), g, device, dt)
    ks = _randn((cfg.S, cfg.Hkv, cfg.D), g, device, dt) if cfg.S else None
    vs = _randn((cfg.S, cfg.Hkv, cfg.D), g, device, dt) if cfg.S else None
    if fp8:
        # E4M3 cache entries (bytes) with one scale per KV head; q stays bf16.  (The library's cast is
        # input preparation here: the synthetic cache just has to hold valid codes.)
        k_scale, v_scale = fp8_scales(cfg, layer)
        to8 = lambda x, s: (x.float() / s.to(x.device).view(1, -1, 1)).clamp(-448, 448).to(torch.float8_e4m3fn).view(torch.uint8)
        out = {"q": q, "k_cache": to8(k, k_scale), "v_cache": to8(v, v_scale),
               "k_soft": to8(ks, k_scale) if cfg.S else None, "v_soft": to8(vs, v_scale) if cfg.S else None,
               "k_scale": k_scale.to(device), "v_scale": v_scale.to(device)}
        return out
    if tree_key_gain != 1.0:
        for b in range(cfg.B):
            lo = int(seq_start[b]) + int(prefix_len[b])
            k[lo:lo + cfg.R] = (k[lo:lo + cfg.R].float() * tree_key_gain).to(dt)
    return {"q": q, "k_cache": k, "v_cache": v, "k_soft": ks, "v_soft": vs}


def fp8_scales(cfg: VerifyConfig, layer: int):
    """Per-KV-head fp32 scales of an E4M3 cache: the N(0,1) entries are mapped so that about 6 standard
    deviations reach the format's largest value (448), jittered per head and layer."""
    rng = _rng(cfg, 300 + layer)
    k = (6.0 / 448.0) * (1.0 + 0.2 * rng.random(cfg.Hkv))
    v = (6.0 / 448.0) * (1.0 + 0.2 * rng.random(cfg.Hkv))
    return torch.from_numpy(k.astype(np.float32)), torch.from_numpy(v.astype(np.float32))


def logits(cfg: VerifyConfig, device="cpu"):
    """target, draft logits [B,T,V] in cfg.logit_dtype."""
    g = _gen(cfg, 7, device)
    shape = (cfg.B, cfg.T, cfg.V)
    target = torch.empty(shape, device=device, dtype=cfg.logit_dtype)
    draft = torch.empty(shape, device=device, dtype=cfg.logit_dtype)
    for b in range(cfg.B):          # per sequence, to bound the fp32 temporaries
        t32 = torch.randn((cfg.T, cfg.V), generator=g, device=device, dtype=torch.float32) * cfg.sigma_logit
        if cfg.draft == "noise":
            d32 = t32 + torch.randn((cfg.T, cfg.V), generator=g, device=device, dtype=torch.float32)
        else:
            d32 = torch.randn((cfg.T, cfg.V), generator=g, device=device, dtype=torch.float32) * cfg.sigma_logit
        target[b] = t32.to(cfg.logit_dtype)
        draft[b] = d32.to(cfg.logit_dtype)
    return target, draft


def draft_tokens(cfg: VerifyConfig, parent: torch.Tensor, draft_logits: torch.Tensor, temperature: float):
    """Token of every node: the children of node u are drawn from the draft row of u without
    replacement (top-f of logits/temperature + Gumbel noise); greedy run: the f largest draft logits."""
    device = draft_logits.device
    g = _gen(cfg, 8, device)
    B, T = parent.shape
    tok = torch.zeros((B, T), dtype=torch.int32)
    root = torch.randint(0, cfg.V, (B,), generator=_gen(cfg, 9, "cpu"))
    par = parent.numpy()
    for b in range(B):
        tok[b, 0] = int(root[b])
        kids = {}
        for i in range(1, T):
            kids.setdefault(int(par[b, i]), []).append(i)
        for u, ch in kids.items():
            row = draft_logits[b, u].float()
            if temperature > 0:
                uu = torch.rand(row.shape, generator=g, device=device, dtype=torch.float32)
                gumbel = -torch.log((-torch.log(uu.clamp_min(1e-20))).clamp_min(1e-20))
                row = row / temperature + gumbel
            top = torch.topk(row, len(ch)).indices.cpu()
            for c, t in zip(ch, top.tolist()):
                tok[b, c] = t
    return tok


def uniforms(cfg: VerifyConfig) -> torch.Tensor:
    """[B,T] fp32 in [0,1): slot i>0 drives the accept test of node i, slot 0 the final draw."""
    g = _gen(cfg, 10, "cpu")
    return torch.rand((cfg.B, cfg.T), generator=g, dtype=torch.float32)
