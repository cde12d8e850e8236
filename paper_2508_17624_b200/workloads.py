"""Seeded synthetic workloads for the adapter-aware MoE layer.

This module only *draws inputs*: configuration records, bf16 weight bits, token activations,
adapter-id arrays and the sets of experts each adapter re-tunes.  It contains none of the method's
arithmetic (no gating, no rerouting, no FFN), so both the CPU oracle's tests and the CUDA path's
tests can consume the same bits without sharing any computation.

The shapes follow the paper's setting: a DeepSeek-V2-Lite-shaped MoE layer (64 routed experts,
top-6, hidden 2048, expert intermediate 1408, 2 shared experts; Section 3.1 names that model) and
ESFT adapters that re-tune roughly 5-15 % of the experts of a layer (Section 2.2, Table 1).  The real
model, adapters and prompt sets are not available, so weights are N(0, 0.02), activations N(0, 1),
and tuned expert sets are seeded uniform samples.

Weight tensors are slices of one seeded "noise bank" (2^25 bf16 N(0,1) draws scaled on use): tensor
(layer, kind, expert) starts at a hashed offset in the bank and wraps around.  Distinct tensors are
distinct shifted windows, which keeps generation at memcpy speed for the 95 GiB pool of the stacked
configuration while a wrongly chosen expert still produces a visibly different result.
"""
from __future__ import annotations

import dataclasses
import hashlib
from typing import Dict, List, Optional, Tuple

import numpy as np

BANK_LOG2 = 25
W_STD = 0.02


@dataclasses.dataclass(frozen=True)
class MoEConfig:
    name: str
    hidden: int            # H
    inter: int             # I
    num_experts: int       # M routed experts of the base model
    num_shared: int        # S
    top_k: int             # k
    max_adapters: int      # N
    e_max: int             # E_max, slots reserved per adapter
    num_layers: int        # L
    n_tokens: int          # B per layer call
    seed: int

    @property
    def num_slots(self) -> int:  # P = M + N * E_max (first dimension of the virtual weight tensor)
        return self.num_experts + self.max_adapters * self.e_max


# The five workload configurations (index 0 = tiny correctness case, 1 = decode, 2 = prefill,
# 3 = 26 stacked layers, 4 = reroute-only microbenchmark).
CONFIGS: Dict[str, MoEConfig] = {
    "c0": MoEConfig("c0", 256, 128, 16, 1, 2, 2, 3, 1, 64, 0),
    "c1": MoEConfig("c1", 2048, 1408, 64, 2, 6, 4, 8, 1, 256, 1),
    "c2": MoEConfig("c2", 2048, 1408, 64, 2, 6, 20, 16, 1, 8192, 2),
    "c3": MoEConfig("c3", 2048, 1408, 64, 2, 6, 20, 10, 26, 1024, 3),
    "c4": MoEConfig("c4", 2048, 1408, 64, 0, 6, 20, 32, 1, 65536, 4),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even float32 -> bf16, returned as uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, *stream: int) -> np.random.Generator:
    key = hashlib.sha256(repr((seed,) + tuple(stream)).encode()).digest()
    return np.random.Generator(np.random.Philox(key=int.from_bytes(key[:8], "little")))


def _h64(*parts: int) -> int:
    return int.from_bytes(hashlib.sha256(repr(parts).encode()).digest()[:8], "little")


class NoiseBank:
    """2^25 seeded N(0, W_STD) draws, already rounded to bf16."""

    def __init__(self, seed: int):
        g = _rng(seed, 0xBA4C)
        n = 1 << BANK_LOG2
        self.bits = f32_to_bf16_bits(g.standard_normal(n, dtype=np.float32) * np.float32(W_STD))
        self.seed = seed

    def window(self, n: int, *key: int) -> np.ndarray:
        size = self.bits.shape[0]
        off = _h64(self.seed, *key) % size
        out = np.empty(n, dtype=np.uint16)
        pos = 0
        while pos < n:
            take = min(n - pos, size - off)
            out[pos:pos + take] = self.bits[off:off + take]
            pos += take
            off = 0
        return out


KIND_GATE, KIND_UP, KIND_DOWN, KIND_ROUTER = 1, 2, 3, 4
SHARED_BASE = 1 << 20      # expert key offset for shared experts
ADAPTER_BASE = 1 << 24     # expert key offset for adapter copies


@dataclasses.dataclass
class ExpertWeights:
    """bf16 bit patterns; w_gate, w_up: [n, I, H]; w_down: [n, H, I] (row-major, K contiguous)."""
    w_gate: np.ndarray
    w_up: np.ndarray
    w_down: np.ndarray

    @property
    def n(self) -> int:
        return self.w_gate.shape[0]


def _experts(bank: NoiseBank, cfg: MoEConfig, layer: int, keys: List[int]) -> ExpertWeights:
    n, I, H = len(keys), cfg.inter, cfg.hidden
    g = np.empty((n, I, H), np.uint16)
    u = np.empty((n, I, H), np.uint16)
    d = np.empty((n, H, I), np.uint16)
    for r, key in enumerate(keys):
        g[r] = bank.window(I * H, layer, KIND_GATE, key).reshape(I, H)
        u[r] = bank.window(I * H, layer, KIND_UP, key).reshape(I, H)
        d[r] = bank.window(I * H, layer, KIND_DOWN, key).reshape(H, I)
    return ExpertWeights(g, u, d)


@dataclasses.dataclass
class BaseLayer:
    router_w: np.ndarray        # [M, H] bf16 bits
    routed: ExpertWeights       # n = M
    shared: ExpertWeights       # n = S


def gen_base_layer(cfg: MoEConfig, layer: int, bank: Optional[NoiseBank] = None,
                   router_std: float = 1.0) -> BaseLayer:
    """Base-model weights of one MoE layer.  `router_std` scales the router rows (in units of W_STD)."""
    bank = bank or NoiseBank(cfg.seed)
    rw = bank.window(cfg.num_experts * cfg.hidden, layer, KIND_ROUTER, 0)
    if router_std != 1.0:
        rw = f32_to_bf16_bits(bf16_bits_to_f32(rw) * np.float32(router_std))
    routed = _experts(bank, cfg, layer, list(range(cfg.num_experts)))
    shared = _experts(bank, cfg, layer, [SHARED_BASE + r for r in range(cfg.num_shared)])
    return BaseLayer(rw.reshape(cfg.num_experts, cfg.hidden), routed, shared)


def tuned_counts(cfg: MoEConfig) -> np.ndarray:
    """e_i^(l): number of experts adapter i re-tunes in layer l, shape [N, L]."""
    N, L = cfg.max_adapters, cfg.num_layers
    g = _rng(cfg.seed, 0xE)
    if cfg.name == "c0":
        return np.full((N, L), 3, np.int32)
    if cfg.name == "c1":
        return np.full((N, L), 8, np.int32)
    if cfg.name == "c2":
        return g.integers(4, 17, size=(N, L)).astype(np.int32)
    if cfg.name == "c3":
        return g.integers(7, 10, size=(N, L)).astype(np.int32)
    raise ValueError("tuned_counts: give explicit counts for " + cfg.name)


def tuned_sets(cfg: MoEConfig, counts: Optional[np.ndarray] = None) -> List[List[np.ndarray]]:
    """tuned[i][l] = strictly ascending int32 array of the base experts adapter i re-tunes in layer l."""
    if cfg.name == "c0" and counts is None:
        fixed = [np.array([1, 5, 9], np.int32), np.array([5, 6, 14], np.int32)]
        return [[fixed[i].copy() for _ in range(cfg.num_layers)] for i in range(cfg.max_adapters)]
    counts = tuned_counts(cfg) if counts is None else np.asarray(counts, np.int32)
    out = []
    for i in range(cfg.max_adapters):
        per_layer = []
        for l in range(cfg.num_layers):
            g = _rng(cfg.seed, 0x5E7, i, l)
            ids = np.sort(g.choice(cfg.num_experts, size=int(counts[i, l]), replace=False))
            per_layer.append(ids.astype(np.int32))
        out.append(per_layer)
    return out


def gen_adapter_layer(cfg: MoEConfig, adapter: int, layer: int, expert_ids: np.ndarray,
                      bank: Optional[NoiseBank] = None) -> ExpertWeights:
    """Independent draws for adapter `adapter`'s copies of `expert_ids` in `layer` (same order)."""
    bank = bank or NoiseBank(cfg.seed)
    keys = [ADAPTER_BASE + adapter * 4096 + int(j) for j in expert_ids]
    return _experts(bank, cfg, layer, keys)


def gen_tokens(cfg: MoEConfig, layer: int = 0, n_tokens: Optional[int] = None) -> np.ndarray:
    """x[B, H] ~ N(0,1) rounded to bf16 (bit patterns)."""
    B = cfg.n_tokens if n_tokens is None else n_tokens
    g = _rng(cfg.seed, 0x70, layer)
    return f32_to_bf16_bits(g.standard_normal((B, cfg.hidden), dtype=np.float32))


def gen_adapter_ids(cfg: MoEConfig, n_tokens: Optional[int] = None, mode: Optional[str] = None) -> np.ndarray:
    """Per-token adapter id (AID), -1 = base model.

    modes: "uniform" per token over {-1, 0..N-1}; "requests" = runs of 256 consecutive tokens that
    share one uniformly drawn id; "zipf" = rank-r adapter with probability ~ 1/r, no base tokens.
    """
    B = cfg.n_tokens if n_tokens is None else n_tokens
    N = cfg.max_adapters
    mode = mode or {"c2": "requests", "c3": "zipf"}.get(cfg.name, "uniform")
    g = _rng(cfg.seed, 0xA1D)
    if mode == "uniform":
        return g.integers(-1, N, size=B).astype(np.int32)
    if mode == "requests":
        n_req = (B + 255) // 256
        return np.repeat(g.integers(-1, N, size=n_req), 256)[:B].astype(np.int32)
    if mode == "zipf":
        p = 1.0 / np.arange(1, N + 1)
        return g.choice(N, size=B, p=p / p.sum()).astype(np.int32)
    if mode == "base":
        return np.full(B, -1, np.int32)
    raise ValueError(mode)


def gen_logits(cfg: MoEConfig, n_tokens: Optional[int] = None) -> np.ndarray:
    """Router logits ~ N(0,1) as float32 [B, M] (reroute-only microbenchmark input)."""
    B = cfg.n_tokens if n_tokens is None else n_tokens
    g = _rng(cfg.seed, 0x106)
    return g.standard_normal((B, cfg.num_experts), dtype=np.float32)


def with_(cfg: MoEConfig, **kw) -> MoEConfig:
    return dataclasses.replace(cfg, **kw)
