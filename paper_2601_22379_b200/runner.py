"""Drives the library on a synthetic workload: prefill a cache, then append + decode step by step.

Used by the benchmark, the smoke test and the GPU parity tests.  Everything numerical happens inside
libspla.so; this file only moves seeded inputs into place.
"""
from __future__ import annotations

import torch

from . import binding, synth


def config_for(w: synth.Workload, *, flags: int = 0, n_sink=None, n_local=None, extra_context: int = 0,
               window=None):
    return binding.make_config(
        batch=w.batch, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
        block_size=w.block_size, top_k=w.top_k, max_context=w.max_context + extra_context,
        n_sink_blocks=w.n_sink if n_sink is None else n_sink,
        n_local_blocks=w.n_local if n_local is None else n_local,
        kv_dtype=w.kv_dtype, flags=flags, window_size=window[0] if window else 0,
        window_stride=window[1] if window else 0)


def generate_prefill(w: synth.Workload, device):
    """All sequences' prefilled K, V padded to the longest: [batch, H_kv, Lmax, d], plus lengths (int32 device)."""
    lens = synth.seq_lens(w)
    Lmax = int(lens.max())
    K = torch.zeros(w.batch, w.n_kv_heads, Lmax, w.head_dim, dtype=w.torch_dtype, device=device)
    V = torch.zeros_like(K)
    for b in range(w.batch):
        kb, vb = synth.prefill_kv(w, b, device)
        K[b, :, :kb.shape[1]] = kb
        V[b, :, :vb.shape[1]] = vb
        del kb, vb
    return K, V, torch.as_tensor(lens, dtype=torch.int32, device=device)


def build_cache(w: synth.Workload, device="cuda:0", *, flags: int = 0, n_sink=None, n_local=None, chunk: int = 0,
                prefill=None, window=None):
    """Creates a cache for `w` and appends the whole prefilled context (optionally in `chunk`-token calls).

    `window` = (C, s) turns on strided selection windows.  Returns (cache, K, V, lens) with K, V the generated inputs (kept so that a checker can hand the same bits
    to another implementation).
    """
    cache = binding.SplaCache(config_for(w, flags=flags, n_sink=n_sink, n_local=n_local, window=window), device)
    K, V, lens = prefill if prefill is not None else generate_prefill(w, device)
    Lmax = K.shape[2]
    ragged = bool((lens != Lmax).any().item())
    if chunk <= 0 or chunk >= Lmax:
        cache.append_tokens(K, V, lens if ragged else None)
    else:
        for c0 in range(0, Lmax, chunk):
            c1 = min(Lmax, c0 + chunk)
            n_new = (lens - c0).clamp_(0, c1 - c0).to(torch.int32)
            cache.append_tokens(K[:, :, c0:c1].contiguous(), V[:, :, c0:c1].contiguous(), n_new if ragged else None)
    return cache, K, V, lens
