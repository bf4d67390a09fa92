"""The prefill- / training-shaped forward (spla_prefill) against the oracle's prefill_unit: the output of every query
position of a chunk equals what a decode step at that position gives (Section 2, opening; Section 3.3)."""
import numpy as np
import pytest
import torch

from oracle import spla_oracle as O
from paper_2601_22379_b200 import binding, runner, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _chunk(w, T, seed):
    """T new tokens per sequence and their queries, from the workload's step generators: k, v [batch, H_kv, T, d],
    q [batch, T, H_q, d]."""
    ks, vs, qs = [], [], []
    for i in range(T):
        k1, v1 = synth.step_kv(w, seed + i, DEV)
        ks.append(k1)
        vs.append(v1)
        qs.append(synth.step_queries(w, seed + i, DEV))
    return torch.cat(ks, dim=2).contiguous(), torch.cat(vs, dim=2).contiguous(), torch.stack(qs, dim=1).contiguous()


def _check_positions(w, K_all, V_all, q, gamma, out, sel, L0, positions, units, flags=0, tie_band=parity.TIE_BAND):
    """out [batch, T, H_q, d], sel [batch, T, H_kv, k]; K_all, V_all [batch, H_kv, L0 + T, d]."""
    G = w.group
    order = 1 if flags & binding.SPLA_FIRST_ORDER else 2
    use_rla = not (flags & binding.SPLA_NO_RLA)
    stats_bf16 = bool(flags & binding.SPLA_STATS_BF16)
    n_same = 0
    for (b, h) in units:
        for i in positions:
            n_tok = L0 + i + 1

            def run(override=None):
                return parity.oracle_unit(w, q[b, i], K_all[b, h, :n_tok], V_all[b, h, :n_tok], gamma, h, n_sink=w.n_sink,
                                          n_local=w.n_local, override=override, order=order, use_rla=use_rla,
                                          stats_bf16=stats_bf16)
            res = run()
            same = parity.check_selection(sel[b, i, h], res, w.top_k, w.n_sink, w.n_local, tie_band)
            if not same:
                res = run([int(x) for x in sel[b, i, h] if x >= 0])
            n_same += same
            parity.check_outputs(f"out[b={b},h={h},pos={i}]", out[b, i, h * G:(h + 1) * G], res["out"], w.kv_dtype)
    return n_same


CASES = [
    # name, overrides, L0 (tokens cached before the chunk), T, flags
    ("gqa_32k", dict(batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, block_size=16, top_k=4, n_sink=1, n_local=1), 16 * 5 + 3, 37, 0),
    ("gqa_32k", dict(batch=1, n_q_heads=4, n_kv_heads=1, head_dim=64, block_size=32, top_k=8), 0, 70, 0),
    ("tiny_ref", dict(batch=1, block_size=16, top_k=4, n_sink=1, n_local=1), 16 * 7 + 9, 40, 0),
    ("gqa_32k", dict(batch=1, n_q_heads=10, n_kv_heads=2, head_dim=128, block_size=16, top_k=6, n_sink=1, n_local=2), 50, 33, binding.SPLA_STATS_BF16),
    ("gqa_32k", dict(batch=1, n_q_heads=3, n_kv_heads=1, head_dim=64, block_size=16, top_k=4, n_sink=0, n_local=0), 16 * 6, 20, binding.SPLA_FIRST_ORDER),
    ("gqa_32k", dict(batch=1, n_q_heads=2, n_kv_heads=2, head_dim=128, block_size=64, top_k=4, n_sink=1, n_local=1), 64 * 9 + 60, 12, binding.SPLA_NO_RLA),
]


@pytest.mark.parametrize("name,over,L0,T,flags", CASES)
def test_prefill_matches_the_oracle_at_every_position(name, over, L0, T, flags):
    w = synth.BY_NAME[name].scaled(**dict(over, context=max(L0, 1), n_needles=0, n_steps=T + 1))
    cfg = runner.config_for(w, flags=flags)
    cache = binding.SplaCache(cfg, DEV)
    K0, V0, _ = runner.generate_prefill(w, DEV)
    if L0 > 0:
        cache.append_tokens(K0[:, :, :L0].contiguous(), V0[:, :, :L0].contiguous())
    kc, vc, q = _chunk(w, T, 100)
    gamma = synth.gamma(w).to(DEV)
    sel = torch.full((w.batch, T, w.n_kv_heads, w.top_k), -9, dtype=torch.int32, device=DEV)
    out = cache.prefill(kc, vc, q, gamma, sel_idx=sel)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert cache.bufs.seq_lens.cpu().tolist() == [L0 + T] * w.batch
    K_all = torch.cat([K0[:, :, :L0], kc], dim=2)
    V_all = torch.cat([V0[:, :, :L0], vc], dim=2)
    units = [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]
    tie = parity.TIE_BAND_STATS_BF16 if flags & binding.SPLA_STATS_BF16 else parity.TIE_BAND
    n_same = _check_positions(w, K_all, V_all, q, gamma, out.cpu().numpy(), sel.cpu().numpy(), L0, range(T), units, flags, tie)
    assert n_same >= 0.9 * len(units) * T
    # the oracle's own prefill form says the same (one unit)
    if not flags:
        G = w.group
        ref, sels = O.prefill_unit(q[0, :, :G].double().cpu().numpy(), K_all[0, 0].double().cpu().numpy(),
                                   V_all[0, 0].double().cpu().numpy(), gamma[:G].double().cpu().numpy(), L0,
                                   block_size=w.block_size, top_k=w.top_k, n_sink=w.n_sink, n_local=w.n_local)
        same = [np.array_equal(sels[i], sel[0, i, 0].cpu().numpy()) for i in range(T)]
        got = out[0, :, :G].cpu().numpy()
        for i in range(T):
            if same[i]:
                parity.check_outputs(f"prefill_unit pos {i}", got[i], ref[i], w.kv_dtype)
    # afterwards the cache is what a plain append of the chunk leaves: statistics bit for bit, the state to rounding
    plain = binding.SplaCache(cfg, DEV)
    plain.append_tokens(K_all.contiguous(), V_all.contiguous())
    torch.cuda.synchronize()
    nblk = -(-(L0 + T) // w.block_size)
    assert torch.equal(plain.bufs.stats[:, :, :nblk], cache.bufs.stats[:, :, :nblk])
    assert torch.equal(plain.bufs.k_cache.reshape(w.batch, w.n_kv_heads, -1, w.head_dim)[:, :, :L0 + T],
                       cache.bufs.k_cache.reshape(w.batch, w.n_kv_heads, -1, w.head_dim)[:, :, :L0 + T])
    if not flags & binding.SPLA_NO_RLA:
        assert parity.rel_l2(cache.bufs.rla_state.cpu().numpy(), plain.bufs.rla_state.cpu().numpy()) < 2 * parity.STATE_TOL_TENSOR


def test_prefill_equals_token_by_token_steps_and_does_not_depend_on_the_workspace_size():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, n_q_heads=8, n_kv_heads=2, block_size=32, top_k=6, context=32 * 11 + 7,
                                       n_needles=2, n_steps=64)
    T = 45
    gamma = synth.gamma(w).to(DEV)
    a, K, V, lens = runner.build_cache(w, DEV, flags=binding.SPLA_GENERAL_KERNELS)
    b, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    c, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    kc, vc, q = _chunk(w, T, 7)
    steps = []
    sel_steps = []
    for i in range(T):                                        # the definition: one token at a time
        s = a.new_sel_buffer()
        steps.append(a.append_decode(kc[:, :, i:i + 1].contiguous(), vc[:, :, i:i + 1].contiguous(), q[:, i].contiguous(),
                                     gamma, sel_idx=s).clone())
        sel_steps.append(s)
    sel_b = torch.empty(w.batch, T, w.n_kv_heads, w.top_k, dtype=torch.int32, device=DEV)
    out_b = b.prefill(kc, vc, q, gamma, sel_idx=sel_b)
    out_c = c.prefill(kc, vc, q, gamma, workspace_bytes=1)    # the minimum: one position per launch
    torch.cuda.synchronize()
    assert a.sync_status() == 0 and b.sync_status() == 0 and c.sync_status() == 0
    assert torch.equal(out_b, out_c)
    assert torch.equal(sel_b, torch.stack(sel_steps, dim=1))
    np.testing.assert_allclose(out_b.cpu().numpy(), torch.stack(steps, dim=1).cpu().numpy(), rtol=2e-4, atol=2e-5)
    assert torch.equal(a.bufs.stats, b.bufs.stats) and torch.equal(a.bufs.seq_lens, b.bufs.seq_lens)


def test_prefill_of_a_4k_token_chunk_at_head_dim_128():
    """One chunk of 4096 tokens on top of 2000 cached ones, d = 128, blocks of 64, bf16: sampled positions of two units
    against the oracle (every position needs its own O(L d) oracle pass)."""
    w = synth.BY_NAME["long_128k"].scaled(batch=1, context=2000, n_needles=3, n_steps=4097)
    T, L0 = 4096, 2000
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    gen = torch.Generator(device=DEV).manual_seed(4096)
    kc = torch.randn(w.batch, w.n_kv_heads, T, w.head_dim, device=DEV, generator=gen).to(torch.bfloat16)
    vc = torch.randn(w.batch, w.n_kv_heads, T, w.head_dim, device=DEV, generator=gen).to(torch.bfloat16)
    q = torch.randn(w.batch, T, w.n_q_heads, w.head_dim, device=DEV, generator=gen).to(torch.bfloat16)
    sel = torch.empty(w.batch, T, w.n_kv_heads, w.top_k, dtype=torch.int32, device=DEV)
    out = cache.prefill(kc, vc, q, gamma, sel_idx=sel)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0 and cache.bufs.seq_lens.cpu().tolist() == [L0 + T]
    K_all, V_all = torch.cat([K, kc], dim=2), torch.cat([V, vc], dim=2)
    rng = np.random.default_rng(3)
    positions = sorted(set([0, 1, 47, 48, 63, 64, T - 1]) | set(int(x) for x in rng.integers(0, T, 14)))
    _check_positions(w, K_all, V_all, q, gamma, out.cpu().numpy(), sel.cpu().numpy(), L0, positions, [(0, 0), (0, 5)])


def test_prefill_argument_checks():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=200, n_steps=8, n_needles=0)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    kc, vc, q = _chunk(w, 9, 0)
    with pytest.raises(binding.SplaError) as e:
        cache.prefill(kc, vc, q, gamma)                       # 200 + 9 > capacity 208
    assert e.value.status == binding.SPLA_ERR_CAPACITY
    win = binding.SplaCache(runner.config_for(w, window=(32, 16)), DEV)
    with pytest.raises(binding.SplaError) as e:
        win.prefill(kc[:, :, :4].contiguous(), vc[:, :, :4].contiguous(), q[:, :4].contiguous(), gamma)
    assert e.value.status == binding.SPLA_ERR_UNSUPPORTED
