"""Seeded random configurations of the whole path (shapes, lengths, forced blocks, windows, flags) against the oracle:
a net under the hand-picked cases of the other files.  Every case is small enough for the oracle to check several
units in well under a second."""
import os
import random

import pytest
import torch

from paper_2601_22379_b200 import binding, runner, synth
from tests import parity
from tests.test_gpu_parity import DEV, _check_units

pytestmark = pytest.mark.gpu


def _draw(case: int):
    rnd = random.Random(22379 * 1000 + case + int(os.environ.get("SPLA_FUZZ_OFFSET", "0")))   # other offsets: more cases by hand
    d = rnd.choice([64, 128])
    B = rnd.choice([16, 32, 64, 128])
    hkv = rnd.choice([1, 2, 3])
    G = rnd.choice([1, 2, 3, 4, 4, 4, 5, 6, 7, 8, 16])
    top_k = rnd.choice([4, 8, 16, 32, 48, 64])
    n_sink = rnd.choice([0, 1, 2])
    n_local = rnd.choice([0, 1, 4])
    while n_sink + n_local > top_k:
        n_local -= 1
    nblk = rnd.choice([1, 2, 3, top_k - 1, top_k, top_k + 1, 40, 200, 700, 1500, 3000])
    nblk = max(1, nblk)
    ctx = max(1, nblk * B - rnd.randrange(B))
    if ctx * d * hkv > 40_000_000:                      # keep the oracle quick
        ctx = 40_000_000 // (d * hkv)
    batch = rnd.choice([1, 2, 3])
    ragged = batch > 1 and rnd.random() < 0.5
    dt = rnd.choice(["bf16", "bf16", "bf16", "f32"])
    flags = 0
    if rnd.random() < 0.4:
        flags |= binding.SPLA_STATS_BF16
    if rnd.random() < 0.2:
        flags |= binding.SPLA_FIRST_ORDER
    if rnd.random() < 0.2:
        flags |= binding.SPLA_GENERAL_KERNELS
    window = None
    if rnd.random() < 0.35 and B >= 32:
        C = rnd.choice([B // 2, B // 4, B])
        s = rnd.choice([C, C // 2])
        if (B - C) // s + 1 <= 8:
            window = (C, s)
    n_steps = rnd.choice([0, 1, 3, 20])
    w = synth.BY_NAME["gqa_32k"].scaled(batch=batch, n_q_heads=G * hkv, n_kv_heads=hkv, head_dim=d, block_size=B,
                                       top_k=top_k, context=ctx, context_min=max(1, ctx // 3) if ragged else 0,
                                       kv_dtype=dt, n_sink=n_sink, n_local=n_local, n_steps=max(n_steps, 1),
                                       n_needles=0 if ragged else min(3, max(0, ctx // B - n_sink - n_local - 1)),
                                       n_outlier_channels=rnd.choice([0, 2]))
    return w, flags, window, n_steps, rnd


@pytest.mark.parametrize("case", range(160))
def test_random_configuration_matches_oracle(case):
    w, flags, window, n_steps, rnd = _draw(case)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags, window=window, chunk=rnd.choice([0, 0, 37, 300]))
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    units = [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]
    rnd.shuffle(units)
    units = units[:3]
    order = 1 if flags & binding.SPLA_FIRST_ORDER else 2
    stats_bf16 = bool(flags & binding.SPLA_STATS_BF16)
    tie_band = parity.TIE_BAND_STATS_BF16 if stats_bf16 else parity.TIE_BAND
    extra = {u: (torch.zeros(0, w.head_dim, dtype=w.torch_dtype, device=DEV),) * 2 for u in units}
    one_call = n_steps > 0 and rnd.random() < 0.5         # the last append and the decode as one call
    q = synth.step_queries(w, 0, DEV)
    cfg = cache.cfg
    res_gpu = None
    for step in range(n_steps):                          # decode-step appends through the fused kernel
        k1, v1 = synth.step_kv(w, step, DEV)
        for (b, h) in units:
            extra[(b, h)] = (torch.cat([extra[(b, h)][0], k1[b, h]]), torch.cat([extra[(b, h)][1], v1[b, h]]))
        if one_call and step == n_steps - 1:
            sel = cache.new_sel_buffer()
            osp = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=DEV)
            orla = torch.empty_like(osp)
            out = cache.append_decode(k1, v1, q, gamma, sel_idx=sel, dbg_o_sparse=osp, dbg_o_rla=orla)
            torch.cuda.synchronize()
            res_gpu = (out.cpu().numpy(), osp.cpu().numpy(), orla.cpu().numpy(), sel.cpu().numpy())
        else:
            cache.append_tokens(k1, v1)
    if res_gpu is None:
        _check_units(w, cache, q, gamma, K, V, lens_h, units, w.n_sink, w.n_local, extra=extra, order=order, window=window)
    else:
        out, osp, orla, sel = res_gpu
        for (b, h) in units:
            Ku = torch.cat([K[b, h, :int(lens_h[b])], extra[(b, h)][0]])
            Vu = torch.cat([V[b, h, :int(lens_h[b])], extra[(b, h)][1]])

            def run(override=None):
                return parity.oracle_unit(w, q[b], Ku, Vu, gamma, h, n_sink=w.n_sink, n_local=w.n_local,
                                          override=override, order=order, window=window, stats_bf16=stats_bf16)
            parity.compare_unit(w, run(), out[b], osp[b], orla[b], sel[b, h], h, n_sink=w.n_sink, n_local=w.n_local,
                                rerun=run, tie_band=tie_band)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
