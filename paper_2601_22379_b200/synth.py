"""Seeded synthetic long-context decode workloads.

This module only draws inputs.  It holds none of the method's arithmetic and
imports neither the CUDA binding nor the CPU oracle, so that both can be fed
the same bits from one place.

The five workloads mirror the configurations the benchmark is quoted on:
N(0,1) keys and values, optional outlier key channels (x8), "needle" blocks
whose keys are shifted toward the unit's query direction by 3 sigma, an
optional random-walk drift of the per-block key mean, and ragged per-sequence
context lengths.  They stand in for the long-document corpora and retrieval
suites the paper evaluates on, none of which is reproduced here.

Structure (lengths, needle positions, outlier channels, query directions) is
always drawn from CPU generators, so it does not depend on the device; the
bulk K/V values come from a generator on the requested device, so CPU- and
GPU-generated caches differ in values but not in distribution.  Whoever
compares two implementations must hand both the same tensors.
"""
from __future__ import annotations

import dataclasses
import math
from dataclasses import dataclass

import numpy as np
import torch

MASTER_SEED = 2601


@dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # position in the configuration list (seed offset)
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    block_size: int
    top_k: int
    context: int               # tokens prefilled per sequence (upper end when ragged)
    context_min: int = 0       # > 0: lengths uniform in [context_min, context]
    kv_dtype: str = "bf16"     # "bf16" or "f32"; queries use the same type
    n_sink: int = 1
    n_local: int = 4
    n_needles: int = 0
    n_outlier_channels: int = 0
    outlier_scale: float = 8.0
    drift_step: float = 0.0
    n_steps: int = 1           # decode steps, each appending one token per sequence
    needle_shift: float = 3.0

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def seed(self) -> int:
        return MASTER_SEED + self.index

    @property
    def max_context(self) -> int:
        return self.context + self.n_steps

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.kv_dtype == "bf16" else torch.float32

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


CONFIGS = [
    Workload("tiny_ref", 0, batch=1, n_q_heads=1, n_kv_heads=1, head_dim=64, block_size=64, top_k=8,
             context=4096, kv_dtype="f32", n_needles=2, n_steps=16),
    Workload("gqa_32k", 1, batch=8, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=16,
             context=32768, n_needles=8, n_outlier_channels=4, n_steps=1),
    Workload("long_128k", 2, batch=4, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=32,
             context=131072, n_needles=8, n_outlier_channels=4, n_steps=64),
    Workload("very_long_1m", 3, batch=1, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=128, top_k=32,
             context=1048576, n_needles=16, drift_step=0.05, n_steps=1),
    Workload("ragged_serving", 4, batch=64, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=16,
             context=65536, context_min=4096, n_outlier_channels=4, n_steps=256),
]
BY_NAME = {w.name: w for w in CONFIGS}


def _cpu_gen(w: Workload, tag: int, *extra: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    s = (w.seed * 1_000_003 + tag * 10_007) & 0x7FFFFFFF
    for e in extra:
        s = (s * 31 + int(e) + 17) & 0x7FFFFFFF
    g.manual_seed(s)
    return g


def _dev_gen(w: Workload, device, tag: int, *extra: int) -> torch.Generator:
    g = torch.Generator(device=device)
    s = (w.seed * 1_000_003 + tag * 10_007) & 0x7FFFFFFF
    for e in extra:
        s = (s * 31 + int(e) + 17) & 0x7FFFFFFF
    g.manual_seed(s)
    return g


def seq_lens(w: Workload) -> np.ndarray:
    """Prefilled context length of every sequence, int32 [batch]."""
    if w.context_min <= 0:
        return np.full(w.batch, w.context, dtype=np.int32)
    g = _cpu_gen(w, 1)
    return torch.randint(w.context_min, w.context + 1, (w.batch,), generator=g).numpy().astype(np.int32)


def query_directions(w: Workload) -> torch.Tensor:
    """q0 ~ N(0, I_d) per (sequence, KV head): the direction needles are planted along.  fp32 CPU."""
    return torch.randn(w.batch, w.n_kv_heads, w.head_dim, generator=_cpu_gen(w, 2))


def outlier_channels(w: Workload) -> np.ndarray:
    """Indices of the key channels scaled by `outlier_scale`, int64 [H_kv, n_outlier_channels]."""
    g = _cpu_gen(w, 3)
    rows = [torch.randperm(w.head_dim, generator=g)[:w.n_outlier_channels].numpy() for _ in range(w.n_kv_heads)]
    return np.stack(rows) if w.n_outlier_channels else np.zeros((w.n_kv_heads, 0), dtype=np.int64)


def needle_blocks(w: Workload) -> np.ndarray:
    """Needle block indices, int64 [batch, H_kv, n_needles], among the blocks that are not forced."""
    lens = seq_lens(w)
    out = np.zeros((w.batch, w.n_kv_heads, w.n_needles), dtype=np.int64)
    g = _cpu_gen(w, 4)
    for b in range(w.batch):
        nblk = -(-int(lens[b]) // w.block_size)
        lo, hi = w.n_sink, nblk - w.n_local - 1      # -1: the block the decode steps append into stays free of needles
        for h in range(w.n_kv_heads):
            if w.n_needles:
                if hi - lo < w.n_needles:
                    raise ValueError("context too short for the requested needles")
                out[b, h] = np.sort(lo + torch.randperm(hi - lo, generator=g)[:w.n_needles].numpy())
    return out


def gamma(w: Workload) -> torch.Tensor:
    """RMSNorm scale, fp32 [H_q, d]: 0.1 * (1 + 0.1 g), so both branches have comparable magnitude."""
    g = torch.randn(w.n_q_heads, w.head_dim, generator=_cpu_gen(w, 5))
    return (0.1 * (1.0 + 0.1 * g)).float()


def prefill_kv(w: Workload, b: int, device="cpu"):
    """The prefilled K and V of sequence b: two tensors [H_kv, L_b, d] in the workload's dtype."""
    L = int(seq_lens(w)[b])
    B, d, H = w.block_size, w.head_dim, w.n_kv_heads
    g = _dev_gen(w, device, 6, b)
    K = torch.randn(H, L, d, generator=g, device=device, dtype=torch.float32)
    V = torch.randn(H, L, d, generator=g, device=device, dtype=torch.float32)
    if w.n_outlier_channels:
        ch = torch.as_tensor(outlier_channels(w), device=device)
        for h in range(H):
            K[h, :, ch[h]] *= w.outlier_scale
    if w.drift_step > 0:
        nblk = -(-L // B)
        steps = w.drift_step * torch.randn(H, nblk, d, generator=g, device=device, dtype=torch.float32)
        steps[:, 0] = 0
        mu = torch.cumsum(steps, dim=1)
        K += torch.repeat_interleave(mu, B, dim=1)[:, :L]
    if w.n_needles:
        q0 = query_directions(w)[b].to(device)
        unit = q0 / q0.norm(dim=-1, keepdim=True)
        nb = needle_blocks(w)[b]
        for h in range(H):
            for blk in nb[h]:
                K[h, int(blk) * B:(int(blk) + 1) * B] += w.needle_shift * unit[h]
    return K.to(w.torch_dtype), V.to(w.torch_dtype)


def step_queries(w: Workload, step: int, device="cpu") -> torch.Tensor:
    """Queries of decode step `step`: [batch, H_q, d]; q = (q0 + 0.5 g) / sqrt(1.25), g fresh per head and step."""
    q0 = query_directions(w)
    g = torch.randn(w.batch, w.n_q_heads, w.head_dim, generator=_cpu_gen(w, 7, step))
    q = (q0.repeat_interleave(w.group, dim=1) + 0.5 * g) / math.sqrt(1.25)
    return q.to(w.torch_dtype).to(device)


def step_kv(w: Workload, step: int, device="cpu"):
    """The token each sequence appends at decode step `step`: k, v [batch, H_kv, 1, d] (base distribution)."""
    g = _cpu_gen(w, 8, step)
    k = torch.randn(w.batch, w.n_kv_heads, 1, w.head_dim, generator=g)
    v = torch.randn(w.batch, w.n_kv_heads, 1, w.head_dim, generator=g)
    if w.n_outlier_channels:
        ch = outlier_channels(w)
        for h in range(w.n_kv_heads):
            k[:, h, :, ch[h]] *= w.outlier_scale
    return k.to(w.torch_dtype).to(device), v.to(w.torch_dtype).to(device)


def algorithmic_bytes_per_step(w: Workload, lens=None, n_windows: int = 1, stat_bytes: int = 4) -> dict:
    """Bytes one decode step must move, per the method's own accounting.

    Block statistics of every block + K and V of the selected blocks + the
    global RLA state, summed over units; next to the dense-decode KV footprint.
    With strided selection windows every block carries `n_windows` statistics records; `stat_bytes` is the size of
    one statistics element (4: fp32, 2: the bfloat16 option).
    """
    lens = seq_lens(w) if lens is None else np.asarray(lens)
    e = 2 if w.kv_dtype == "bf16" else 4
    d, B, H = w.head_dim, w.block_size, w.n_kv_heads
    stats = sel = state = dense = 0
    for L in lens:
        nblk = -(-int(L) // B)
        stats += H * nblk * n_windows * 2 * d * stat_bytes
        sel += H * min(w.top_k, nblk) * B * d * 2 * e
        state += H * d * d * 4
        dense += H * int(L) * d * 2 * e
    return dict(stats=stats, selected_kv=sel, state=state, total=stats + sel + state, dense_kv=dense)
