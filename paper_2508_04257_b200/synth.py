"""Seeded synthetic inputs shaped like the paper's LLaMA-class workloads.

This module only draws numbers: it contains none of the method's arithmetic (no quantization, no top-k,
no attention) and is the one module that both the tests of the CPU oracle and the drivers of the CUDA
library import.  Real model activations and the text corpora the paper evaluates on are not available
offline, so the tensors below stand in for them: shapes follow the paper's model table (Appendix D) and
efficiency table (Appendix F); the value structure follows Section 3 (sink tokens carry extreme values on a
few fixed hidden channels, have small-norm K and V, and keys that align with the queries) and Section 4.1
(keys have channel-wise outliers, values do not).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Tuple

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    hidden: int
    bits: int
    group: int
    seq: int              # prefill length S
    topk: int
    pfn_n: int
    channels: Tuple[int, ...]
    layers: int = 1
    outlier: float = 1000.0      # magnitude planted on the outlier channels of sink tokens
    sink_kv_scale: float = 0.02  # K/V rows of sink tokens are scaled by this
    k_outlier_channels: int = 0  # per-head key channels multiplied by k_outlier_gain and offset
    k_outlier_gain: float = 20.0
    clustered: bool = False      # sink tokens in runs of consecutive positions
    seed: int = 0x5EED0000

    @property
    def max_seq(self) -> int:
        # room for one more group of appended tokens
        return (self.seq // self.group + 1) * self.group

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


WORKLOADS: Dict[str, Workload] = {
    # 1 tiny
    "tiny": Workload("tiny", 1, 8, 8, 64, 512, 4, 32, 256, 2, 1, (37, 190, 411), outlier=500.0, sink_kv_scale=0.05,
                     seed=0x5EED0001),
    # 2 LLaMA2-7B-shaped single layer (outlier channels of LLaMA2-7B, Appendix D)
    "llama2_7b_layer": Workload("llama2_7b_layer", 8, 32, 32, 128, 4096, 2, 128, 4096, 8, 1, (2533, 1415),
                                seed=0x5EED0002),
    # 3 LLaMA3-8B-shaped GQA layer (outlier channels of LLaMA3-8B)
    "llama3_8b_gqa": Workload("llama3_8b_gqa", 4, 32, 8, 128, 4096, 2, 128, 32768, 33, 1, (788, 1384, 4062),
                              k_outlier_channels=4, seed=0x5EED0003),
    # 4 full 32-layer decode step, LLaMA2-7B shapes, 3 bit and 4 bit
    "decode32_3bit": Workload("decode32_3bit", 64, 32, 32, 128, 4096, 3, 64, 8192, 16, 1, (2533, 1415), layers=32,
                              seed=0x5EED0004),
    "decode32_4bit": Workload("decode32_4bit", 64, 32, 32, 128, 4096, 4, 64, 8192, 16, 1, (2533, 1415), layers=32,
                              seed=0x5EED0004),
    # 5 long-context GQA with 1 % clustered sinks
    "long_gqa": Workload("long_gqa", 1, 32, 8, 128, 4096, 2, 128, 131072, 1311, 1, (788, 1384, 4062), clustered=True,
                         seed=0x5EED0005),
}


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed) & 0x7FFFFFFFFFFFFFFF)
    return g


def _randn_half(shape, gen: torch.Generator, device, chunk_rows: int = 1 << 14) -> torch.Tensor:
    """N(0,1) in fp16, drawn in fp32 slabs along the first axis to bound the fp32 footprint."""
    out = torch.empty(shape, dtype=torch.float16, device=device)
    flat = out.view(-1, shape[-1]) if len(shape) > 1 else out.view(-1, 1)
    n = flat.shape[0]
    for i in range(0, n, chunk_rows):
        j = min(n, i + chunk_rows)
        flat[i:j] = torch.randn((j - i, flat.shape[1]), generator=gen, device=device, dtype=torch.float32).to(torch.float16)
    return out


def sink_positions(wl: Workload) -> np.ndarray:
    """Planted sink tokens per sequence, int64 [B, min(topk, S)] ascending; token 0 is always one of them."""
    rng = np.random.default_rng(wl.seed ^ 0xA11CE)
    out = np.zeros((wl.batch, max(min(wl.topk, wl.seq), 0)), np.int64)
    for b in range(wl.batch):
        k = min(wl.topk, wl.seq)
        if k <= 0:
            continue
        chosen = {0}
        if wl.clustered:
            # runs of 8..32 consecutive tokens ("delimiter-like"); the first run straddles a group boundary
            start = wl.group * 5 - 3
            while len(chosen) < k:
                run = int(rng.integers(8, 33))
                for p in range(start, min(start + run, wl.seq)):
                    if len(chosen) < k:
                        chosen.add(p)
                start = int(rng.integers(1, max(2, wl.seq - 40)))
        else:
            while len(chosen) < min(k, wl.seq):
                chosen.add(int(rng.integers(1, wl.seq)))
        out[b] = np.sort(np.fromiter(chosen, np.int64, len(chosen)))[:k]
    return out


def make_hidden(wl: Workload, device="cpu") -> torch.Tensor:
    """Hidden state at the emergence layer, fp16 [B, S, d]: N(0,1) with +-outlier on the listed channels at sinks."""
    g = _gen(device, wl.seed + 11)
    H = _randn_half((wl.batch, wl.seq, wl.hidden), g, device)
    pos = sink_positions(wl)
    rng = np.random.default_rng(wl.seed ^ 0xBEEF)
    for b in range(wl.batch):
        for p in pos[b]:
            for c in wl.channels:
                sign = 1.0 if rng.integers(0, 2) else -1.0
                # distinct magnitudes, well inside the fp16 range
                mag = wl.outlier * (1.0 + 0.25 * float(rng.random()))
                H[b, int(p), int(c)] = sign * mag
    return H


def make_kv(wl: Workload, layer: int = 0, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """K, V fp16 [B, Hkv, S, D].  Sink rows are shrunk; optional per-head key channels get a gain and an offset."""
    g = _gen(device, wl.seed + 101 + 7 * layer)
    K = _randn_half((wl.batch, wl.n_kv_heads, wl.seq, wl.head_dim), g, device)
    V = _randn_half((wl.batch, wl.n_kv_heads, wl.seq, wl.head_dim), g, device)
    if wl.k_outlier_channels:
        rng = np.random.default_rng(wl.seed ^ (0xC0FFEE + layer))
        for h in range(wl.n_kv_heads):
            chans = rng.choice(wl.head_dim, wl.k_outlier_channels, replace=False)
            for c in chans:
                off = float(rng.choice([-1.0, 1.0])) * float(rng.uniform(4.0, 12.0))
                K[:, h, :, int(c)] = (K[:, h, :, int(c)].float() * wl.k_outlier_gain + off).to(torch.float16)
    pos = sink_positions(wl)
    for b in range(wl.batch):
        idx = torch.as_tensor(pos[b], device=device, dtype=torch.long)
        if idx.numel():
            K[b, :, idx, :] = (K[b, :, idx, :].float() * wl.sink_kv_scale).to(torch.float16)
            V[b, :, idx, :] = (V[b, :, idx, :].float() * wl.sink_kv_scale).to(torch.float16)
    return K, V


def make_new_token(wl: Workload, layer: int = 0, step: int = 0, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """One decode-time token per sequence: k, v fp16 [B, Hkv, 1, D]."""
    g = _gen(device, wl.seed + 100003 + 31 * layer + 1009 * step)
    k = _randn_half((wl.batch, wl.n_kv_heads, 1, wl.head_dim), g, device)
    v = _randn_half((wl.batch, wl.n_kv_heads, 1, wl.head_dim), g, device)
    return k, v


def make_query(wl: Workload, K: torch.Tensor, layer: int = 0, step: int = 0) -> torch.Tensor:
    """Decode query fp16 [B, Hq, D]: N(0,1); on every other head pulled toward the first sink key of its KV head."""
    device = K.device
    g = _gen(device, wl.seed + 200003 + 31 * layer + 1009 * step)
    q = torch.randn((wl.batch, wl.n_q_heads, wl.head_dim), generator=g, device=device, dtype=torch.float32)
    rep = wl.n_q_heads // wl.n_kv_heads
    pos = sink_positions(wl)
    if pos.shape[1]:
        for b in range(wl.batch):
            p = int(pos[b][min(1, pos.shape[1] - 1)])
            ks = K[b, :, p, :].float()                      # [Hkv, D]
            ks = ks / ks.norm(dim=-1, keepdim=True).clamp_min(1e-6)
            pull = ks.repeat_interleave(rep, dim=0) * 4.0   # [Hq, D]
            pull[1::2] = 0.0
            q[b] += pull
    return q.to(torch.float16)


# ---- pure-integer generator for committed golden files (independent of the torch build) ----
def _splitmix64(x: np.ndarray) -> np.ndarray:
    x = (x + np.uint64(0x9E3779B97F4A7C15)).astype(np.uint64)
    z = x
    z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
    z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
    return z ^ (z >> np.uint64(31))


def hash_half(shape, seed: int, spread: int = 6) -> np.ndarray:
    """Bell-shaped fp16 values from integer hashing only: (sum of four bytes - 510) / 2^spread, exact in fp16."""
    n = int(np.prod(shape))
    with np.errstate(over="ignore"):
        z = _splitmix64(np.arange(n, dtype=np.uint64) + np.uint64(seed) * np.uint64(0x100000001B3))
    s = ((z & np.uint64(0xFF)) + ((z >> np.uint64(8)) & np.uint64(0xFF)) + ((z >> np.uint64(16)) & np.uint64(0xFF))
         + ((z >> np.uint64(24)) & np.uint64(0xFF))).astype(np.int64) - 510
    return (s.astype(np.float32) / np.float32(1 << spread)).astype(np.float16).reshape(shape)
