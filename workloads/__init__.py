"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds input generation only (logits, uniforms, tree tables, bf16
rounding).  None of the method's arithmetic lives here: it serves the CUDA
library's tests and benchmark and the CPU oracle alike, and imports neither.

The five configurations stand in for the paper's Llama-2 (V = 32000) and
Llama-3 (V = 128256) sized vocabularies and its 3/7/15/31-node binary token
trees (Section 5 and Appendix E of arXiv 2411.05289); the paper's datasets and
model weights are not used.

Recipe (per row): target logits = Zipf-shaped log-prior over a seeded
permutation of the ids, -s * ln(1 + rank), plus N(0, 1) noise (config 1: plain
N(0, 2^2)); draft logits = target + N(0, sigma^2); rounded to the storage type
(bf16 round-to-nearest-even where the config says bf16).  Uniforms are
(u32 >> 8) * 2^-24 in [0, 1), five per (sequence, node).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional

import numpy as np


@dataclass(frozen=True)
class Config:
    name: str
    batch: int
    nodes: int
    vocab: int
    dtype: str              # "fp32" | "bf16"
    zipf_s: Optional[float]  # None: target ~ N(0, target_sd^2) without a prior
    target_sd: float
    sigma: float            # draft-target noise
    temperature: float
    adversarial: float = 0.0  # fraction of rows replaced by adversarial kinds
    seed: int = 0

    @property
    def levels(self) -> int:
        return (self.nodes + 1).bit_length() - 1

    @property
    def rows(self) -> int:
        return self.batch * self.nodes


CONFIGS = {
    # tiny single-level verify: 1000 independent instances of a 3-node tree
    "c1": Config("c1", 1000, 3, 1000, "fp32", None, 2.0, 1.0, 1.0, seed=1000),
    # Llama-2-sized vocabulary, 7-node tree
    "c2": Config("c2", 64, 7, 32000, "bf16", 1.1, 1.0, 1.5, 1.0, seed=2000),
    # deeper tree, temperature x noise sweep (variants c3_T0.6_s0.5 ... built by variants())
    "c3": Config("c3", 256, 15, 32000, "bf16", 1.1, 1.0, 1.5, 1.0, seed=3000),
    # Llama-3-sized vocabulary, 31-node tree: headline throughput configuration
    "c4": Config("c4", 256, 31, 128256, "bf16", 1.2, 1.0, 1.0, 1.0, seed=4000),
    # stress: larger vocabulary and batch, 10 % adversarial rows
    "c5": Config("c5", 1024, 31, 152064, "bf16", 1.2, 1.0, 1.0, 1.0, adversarial=0.10, seed=5000),
}


def variants(name: str):
    """Config 3 is a sweep over temperature x draft-target noise; the others have one variant."""
    c = CONFIGS[name]
    if name != "c3":
        return [c]
    out = []
    for i, (T, s) in enumerate([(0.6, 0.5), (0.6, 1.5), (1.0, 0.5), (1.0, 1.5)]):
        out.append(replace(c, name="c3_T%g_s%g" % (T, s), temperature=T, sigma=s, seed=c.seed + i))
    return out


def all_configs():
    """Every configuration by name, config 3's four variants included (and its base, c3)."""
    out = dict(CONFIGS)
    for v in variants("c3"):
        out[v.name] = v
    return out


def lookup(name: str) -> Config:
    return all_configs()[name]


# ---- bf16 <-> fp32 on the host (numpy has no bf16) ------------------------------------------------

def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16, returned as uint16 bit patterns."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rnd = ((b >> 16) & 1) + np.uint32(0x7FFF)
    return ((b + rnd) >> 16).astype(np.uint16)


def bf16_bits_to_f32(h: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def round_to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """fp32 array holding exactly the values the storage type can represent."""
    if dtype == "bf16":
        return bf16_bits_to_f32(f32_to_bf16_bits(x))
    return np.ascontiguousarray(x, dtype=np.float32)


# ---- adversarial row kinds (config 5) ------------------------------------------------------------
ADV_KINDS = ("same", "one_hot_hard", "one_hot_soft", "disjoint", "near_uniform", "ties")


def _adversarial_kind(cfg: Config, b: int, n: int) -> int:
    """-1 for an ordinary row, else an index into ADV_KINDS; a pure function of (seed, b, n)."""
    if cfg.adversarial <= 0:
        return -1
    h = (cfg.seed * 1000003 + b * 7919 + n * 104729 + 12345) * 2654435761 % (1 << 32)
    u = h / float(1 << 32)
    if u >= cfg.adversarial:
        return -1
    return int(u / cfg.adversarial * len(ADV_KINDS)) % len(ADV_KINDS)


def _apply_adversarial(kind: int, lp: np.ndarray, lq: np.ndarray, rng) -> None:
    V = lp.shape[0]
    name = ADV_KINDS[kind]
    if name == "same":
        lq[:] = lp
    elif name == "one_hot_hard":
        j = int(rng.integers(V)); lq[:] = -np.inf; lq[j] = 0.0
    elif name == "one_hot_soft":
        j = int(rng.integers(V)); lq[:] = -60.0; lq[j] = 0.0
    elif name == "disjoint":
        tp = np.argpartition(-lp, 64)[:64]
        tq = np.argpartition(-lq, 64)[:64]
        lq[tp] = -np.inf
        lp[tq] = -np.inf
    elif name == "near_uniform":
        lq[:] = rng.normal(0.0, 0.01, V)
    elif name == "ties":
        lp[:] = np.round(lp * 2.0) / 2.0
        lq[:] = np.round(lq * 2.0) / 2.0


# ---- host generator (numpy, PCG64) ---------------------------------------------------------------

def _prior(cfg: Config) -> Optional[np.ndarray]:
    if cfg.zipf_s is None:
        return None
    rng = np.random.Generator(np.random.PCG64([cfg.seed, 0xABCDEF]))
    rank = rng.permutation(cfg.vocab)
    return (-cfg.zipf_s * np.log1p(rank)).astype(np.float32)


def host_sequence(cfg: Config, b: int, prior: Optional[np.ndarray] = None):
    """Logits of sequence b: (target, draft), each fp32 [nodes][vocab] holding storage-rounded
    values.  Any sequence can be produced on its own (seeded by (config seed, b))."""
    if prior is None:
        prior = _prior(cfg)
    rng = np.random.Generator(np.random.PCG64([cfg.seed, 1, b]))
    N, V = cfg.nodes, cfg.vocab
    lp = rng.normal(0.0, cfg.target_sd, (N, V)).astype(np.float32)
    if prior is not None:
        lp += prior[None, :]
    lq = lp + rng.normal(0.0, cfg.sigma, (N, V)).astype(np.float32)
    for n in range(N):
        kind = _adversarial_kind(cfg, b, n)
        if kind >= 0:
            _apply_adversarial(kind, lp[n], lq[n], rng)
    return round_to_storage(lp, cfg.dtype), round_to_storage(lq, cfg.dtype)


def host_logits(cfg: Config, seqs=None):
    """(target, draft) fp32 [len(seqs)][nodes][vocab] for the given sequence ids (default: all)."""
    seqs = range(cfg.batch) if seqs is None else seqs
    prior = _prior(cfg)
    tp, tq = [], []
    for b in seqs:
        lp, lq = host_sequence(cfg, b, prior)
        tp.append(lp); tq.append(lq)
    return np.stack(tp), np.stack(tq)


def host_uniforms(cfg: Config, seqs=None) -> np.ndarray:
    """fp32 [len(seqs)][nodes][5] = (u_d1, u_d2, r1, r2, u_res), (u32 >> 8) * 2^-24."""
    seqs = range(cfg.batch) if seqs is None else seqs
    out = np.empty((len(seqs), cfg.nodes, 5), np.float32)
    for i, b in enumerate(seqs):
        rng = np.random.Generator(np.random.PCG64([cfg.seed, 2, b]))
        out[i] = (rng.integers(0, 1 << 24, (cfg.nodes, 5)).astype(np.float32)) * np.float32(2.0 ** -24)
    return out


# ---- tree tables ----------------------------------------------------------------------------------

def heap_children(nodes: int) -> np.ndarray:
    """int32 [nodes][2]: children of n are 2n+1, 2n+2; -1 beyond the last node."""
    ch = np.full((nodes, 2), -1, np.int32)
    for n in range(nodes):
        for i in range(2):
            c = 2 * n + 1 + i
            if c < nodes:
                ch[n, i] = c
    return ch


def paper_node_kind(nodes: int) -> np.ndarray:
    """uint8 [nodes]: internal nodes verify (0); the last level's nodes are leaves (1) that only
    draw the bonus token from p -- the paper's count of a 2^d - 1 node tree."""
    kind = np.zeros(nodes, np.uint8)
    kind[nodes // 2:] = 1
    return kind


# ---- device generator (torch; same recipe, its own random stream) ---------------------------------

def device_logits(cfg: Config, device="cuda", batch: Optional[int] = None):
    """(target, draft) torch tensors [batch][nodes][vocab] of the storage dtype, generated on the
    device in per-sequence chunks.  Same distributions as the host generator, different stream;
    parity tests copy the rows they check back to the host, so both sides see identical values."""
    import torch

    B = cfg.batch if batch is None else batch
    N, V = cfg.nodes, cfg.vocab
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed)
    prior = None
    if cfg.zipf_s is not None:
        rank = torch.randperm(V, generator=gen, device=device).to(torch.float32)
        prior = -cfg.zipf_s * torch.log1p(rank)
    tp = torch.empty((B, N, V), dtype=dt, device=device)
    tq = torch.empty((B, N, V), dtype=dt, device=device)
    chunk = max(1, min(B, (1 << 26) // (N * V) + 1))
    for b0 in range(0, B, chunk):
        b1 = min(B, b0 + chunk)
        lp = torch.randn((b1 - b0, N, V), generator=gen, device=device) * cfg.target_sd
        if prior is not None:
            lp += prior
        lq = lp + torch.randn((b1 - b0, N, V), generator=gen, device=device) * cfg.sigma
        if cfg.adversarial > 0:
            cpu_rng = np.random.Generator(np.random.PCG64([cfg.seed, 3, b0]))
            for b in range(b0, b1):
                for n in range(N):
                    kind = _adversarial_kind(cfg, b, n)
                    if kind < 0:
                        continue
                    _apply_adversarial_torch(ADV_KINDS[kind], lp[b - b0, n], lq[b - b0, n], cpu_rng, gen)
        tp[b0:b1] = lp.to(dt)
        tq[b0:b1] = lq.to(dt)
    return tp, tq


def _apply_adversarial_torch(name, lp, lq, cpu_rng, gen):
    import torch

    V = lp.shape[0]
    if name == "same":
        lq.copy_(lp)
    elif name == "one_hot_hard":
        j = int(cpu_rng.integers(V)); lq.fill_(-math.inf); lq[j] = 0.0
    elif name == "one_hot_soft":
        j = int(cpu_rng.integers(V)); lq.fill_(-60.0); lq[j] = 0.0
    elif name == "disjoint":
        tp = torch.topk(lp, 64).indices
        tq = torch.topk(lq, 64).indices
        lq[tp] = -math.inf
        lp[tq] = -math.inf
    elif name == "near_uniform":
        lq.copy_(torch.randn(V, generator=gen, device=lp.device) * 0.01)
    elif name == "ties":
        lp.copy_(torch.round(lp * 2.0) / 2.0)
        lq.copy_(torch.round(lq * 2.0) / 2.0)


def device_uniforms(cfg: Config, device="cuda", batch: Optional[int] = None):
    import torch

    B = cfg.batch if batch is None else batch
    gen = torch.Generator(device=device)
    gen.manual_seed(cfg.seed + 7)
    bits = torch.randint(0, 1 << 24, (B, cfg.nodes, 5), generator=gen, device=device)
    return bits.to(torch.float32) * (2.0 ** -24)


def to_device(x: np.ndarray, dtype: str, device="cuda"):
    """Host fp32 array of storage-rounded values -> torch tensor of the storage dtype."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(x)).to(device)
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def to_host_f32(t) -> np.ndarray:
    """Device tensor of the storage dtype -> host fp32 array with the same values."""
    return t.detach().to("cpu", copy=True).float().numpy()
