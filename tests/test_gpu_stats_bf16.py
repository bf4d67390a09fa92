"""GPU parity of the 16-bit statistics option (SPLA_STATS_BF16): the block (or window) means and variances of the
Taylor score (Section 3.1) are computed in fp32, rounded once to bfloat16 when stored, and the score reads the rounded
values.  The oracle rounds its float64 statistics the same way."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import spla_oracle as O
from paper_2601_22379_b200 import binding, runner, synth
from tests import parity
from tests.test_gpu_parity import DEV, _all_units, _check_units, _decode_all, _stepped_full

pytestmark = pytest.mark.gpu
F16 = binding.SPLA_STATS_BF16
WIN = (32, 16)


def _ulp_bf16(x):
    """Spacing of bfloat16 at |x| (normal range): 2^(floor(log2 |x|) - 7)."""
    ax = np.maximum(np.abs(x), 1e-30)
    return 2.0 ** (np.floor(np.log2(ax)) - 7)


def _stats_match_rounded_oracle(st, mean, var, live=None):
    """Stored records equal the rounded oracle statistics, except where the fp32 and the float64 value straddle a
    rounding boundary (one unit in the last place, rare)."""
    got_m, got_v = st[..., 0, :].astype(np.float64), st[..., 1, :].astype(np.float64)
    if live is not None:
        got_m, got_v, mean, var = got_m[live], got_v[live], mean[live], var[live]
    for got, want in ((got_m, O.round_bf16(mean)), (got_v, O.round_bf16(var))):
        diff = np.abs(got - want)
        assert np.all(diff <= _ulp_bf16(want) * 1.0001), "a stored statistic is more than one bfloat16 step away"
        assert np.mean(diff > 0) < 2e-3, f"{np.mean(diff > 0):.2e} of the statistics differ from the rounded oracle"


@pytest.mark.parametrize("name,ctx,window", [
    ("tiny_ref", 64 * 9 + 17, None),
    ("gqa_32k", 64 * 11 + 5, None),
    ("gqa_32k", 64 * 11 + 37, WIN),
    ("very_long_1m", 128 * 9 + 100, WIN),
])
def test_bf16_statistics_on_every_append_path(name, ctx, window):
    w = synth.BY_NAME[name].scaled(batch=2, context=ctx, n_needles=0)
    bulk, K, V, lens = runner.build_cache(w, DEV, flags=F16, window=window)
    chunked, _, _, _ = runner.build_cache(w, DEV, flags=F16, window=window, chunk=100, prefill=(K, V, lens))
    small, _, _, _ = runner.build_cache(w, DEV, flags=F16, window=window, chunk=19, prefill=(K, V, lens))   # fused kernel
    plain, _, _, _ = runner.build_cache(w, DEV, window=window, prefill=(K, V, lens))
    torch.cuda.synchronize()
    assert bulk.bufs.stats.dtype == torch.bfloat16 and bulk.sizes.stats * 2 == plain.sizes.stats
    nblk = -(-ctx // w.block_size)
    for b in range(w.batch):
        for h in (0, w.n_kv_heads - 1):
            Kd = K[b, h].double().cpu().numpy()
            st = bulk.bufs.stats[b, h, :nblk].float().cpu().numpy()
            if window is None:
                mean, var, _ = O.block_statistics(Kd, w.block_size)
                _stats_match_rounded_oracle(st, mean, var)
            else:
                mean, var, n = O.window_statistics(Kd, w.block_size, *window)
                _stats_match_rounded_oracle(st, mean, var, live=n > 0)
    # the records are the fp32 ones rounded: bit for bit
    live = slice(None)
    if window is not None:
        n = O.window_statistics(K[0, 0].double().cpu().numpy(), w.block_size, *window)[2]
        live = torch.as_tensor(n > 0, device=DEV)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            want = plain.bufs.stats[b, h, :nblk][live].to(torch.bfloat16)
            for c in (bulk, chunked, small):
                assert torch.equal(c.bufs.stats[b, h, :nblk][live], want)
    # everything else the append maintains is untouched by the option
    assert torch.equal(bulk.bufs.tok_lse[:, :, :ctx], plain.bufs.tok_lse[:, :, :ctx])
    assert torch.equal(bulk.bufs.rla_state, plain.bufs.rla_state)
    assert torch.equal(bulk.bufs.k_cache.reshape(2, w.n_kv_heads, -1, w.head_dim)[:, :, :ctx], K)


SMALL = [
    ("tiny_ref", dict(context=64 * 20 + 13)),
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31)),
    ("long_128k", dict(batch=1, context=64 * 150 + 1, n_steps=2)),
    ("very_long_1m", dict(context=128 * 140 + 77, n_needles=4)),
    ("ragged_serving", dict(batch=6, context=6000, context_min=300, n_steps=2)),
]


@pytest.mark.parametrize("name,over", SMALL)
@pytest.mark.parametrize("flags", [F16, F16 | binding.SPLA_GENERAL_KERNELS])
@pytest.mark.parametrize("window", [None, WIN])
def test_bf16_statistics_decode_matches_oracle_small(name, over, flags, window):
    w = synth.BY_NAME[name].scaled(**over)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags, window=window)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    n_exact = _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, window=window)
    assert n_exact >= 0.9 * w.batch * w.n_kv_heads


def test_bf16_statistics_cluster_and_general_kernels_select_the_same_blocks():
    w = synth.BY_NAME["long_128k"].scaled(batch=1, context=64 * 300 + 7, n_steps=1)
    a, K, V, lens = runner.build_cache(w, DEV, flags=F16)
    b, _, _, _ = runner.build_cache(w, DEV, flags=F16 | binding.SPLA_GENERAL_KERNELS, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    ra, rb = _decode_all(a, w, q, gamma), _decode_all(b, w, q, gamma)
    assert np.mean(ra[3] == rb[3]) > 0.98                 # different summation orders: ties at most


def test_bf16_statistics_first_order_flag():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 40 + 9)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=F16 | binding.SPLA_FIRST_ORDER)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, order=1)


@pytest.mark.parametrize("window", [None, WIN])
def test_bf16_statistics_one_call_step_equals_separate_calls(window):
    """append + decode in one call (the score kernel streams 16-bit records while the append runs) against the two
    separate calls, bit for bit, across a block boundary."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 40 + 60, n_steps=8)
    a, K, V, lens = runner.build_cache(w, DEV, flags=F16, window=window)
    b, _, _, _ = runner.build_cache(w, DEV, flags=F16, window=window, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        q = synth.step_queries(w, step, DEV)
        sa, sb = a.new_sel_buffer(), b.new_sel_buffer()
        a.append_tokens(k1, v1)
        oa = a.decode(q, gamma, sel_idx=sa)
        ob = b.append_decode(k1, v1, q, gamma, sel_idx=sb)
        torch.cuda.synchronize()
        assert a.sync_status() == 0 and b.sync_status() == 0
        assert torch.equal(sa, sb) and torch.equal(oa, ob)
    assert torch.equal(a.bufs.stats, b.bufs.stats)


def test_bf16_statistics_long_128k_full_size_sampled_units():
    """The benchmark's configuration at full size with 16-bit statistics, three sampled units, append + decode."""
    _stepped_full(synth.CONFIGS[2].scaled(n_steps=3), n_units=3, check_steps={0, 2}, flags=F16)


@pytest.mark.parametrize("hq", [40, 64])
def test_bf16_statistics_long_128k_full_size_groups_of_five_and_eight(hq):
    """Groups of five (the paper's model) and eight heads at the full 128K context: the tensor-core score path with two
    column tiles, inside the fused decode kernel."""
    _stepped_full(synth.CONFIGS[2].scaled(n_q_heads=hq, n_steps=2), n_units=2, check_steps={0, 1}, flags=F16)


def test_bf16_statistics_windows_long_128k_full_size_sampled_units():
    _stepped_full(synth.CONFIGS[2].scaled(n_steps=2), n_units=2, check_steps={1}, window=WIN, flags=F16)


def test_noalloc_entry_rejects_bf16_statistics():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 8, n_needles=0)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=F16)
    q = synth.step_queries(w, 0, DEV)
    cfg = cache.cfg
    rc = binding.load().spla_select_blocks_noalloc(
        ctypes.byref(cfg), cache.bufs.stats.data_ptr(), cache.bufs.seq_lens.data_ptr(), q.data_ptr(),
        cache.new_sel_buffer().data_ptr(), None, None, None)          # rejected on the host: nothing is launched
    assert rc == binding.SPLA_ERR_UNSUPPORTED


@pytest.mark.parametrize("hq,hkv", [(1, 1), (2, 1), (3, 1), (5, 1), (8, 1), (16, 1), (6, 2)])
def test_bf16_statistics_group_sizes(hq, hkv):
    """Groups of 1-4 heads take the tensor-core score path (unused B columns are zero), 5-8 the FMA path of the
    cluster kernel, 16 the general kernel."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, n_q_heads=hq, n_kv_heads=hkv, context=64 * 40 + 3, n_needles=3)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=F16)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local)


@pytest.mark.parametrize("B,d,dt", [(16, 64, "bf16"), (32, 128, "f32"), (128, 64, "f32"), (128, 128, "bf16"), (64, 64, "bf16")])
@pytest.mark.parametrize("window", [None, "half"])
def test_bf16_statistics_block_sizes_head_dims_dtypes(B, d, dt, window):
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, n_q_heads=4, n_kv_heads=2, head_dim=d, block_size=B, kv_dtype=dt,
                                       context=B * 33 + B // 2, n_needles=2, top_k=8, n_outlier_channels=2)
    win = (B // 2, B // 4) if window else None
    cache, K, V, lens = runner.build_cache(w, DEV, flags=F16, window=win)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, window=win)


def test_bf16_statistics_steps_across_block_boundaries_every_unit():
    """Append one token then decode, 70 steps (more than a block), every unit checked at every eighth step: the
    one-call step with the early-starting tensor-core score kernel."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 30 + 40, n_steps=70)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=F16)
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    extra = {u: (torch.zeros(0, w.head_dim, dtype=w.torch_dtype, device=DEV),) * 2 for u in _all_units(w)}
    cfg = cache.cfg
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        q = synth.step_queries(w, step, DEV)
        for (b, h) in extra:
            extra[(b, h)] = (torch.cat([extra[(b, h)][0], k1[b, h]]), torch.cat([extra[(b, h)][1], v1[b, h]]))
        sel = cache.new_sel_buffer()
        osp = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=DEV)
        orla = torch.empty_like(osp)
        out = cache.append_decode(k1, v1, q, gamma, sel_idx=sel, dbg_o_sparse=osp, dbg_o_rla=orla)
        torch.cuda.synchronize()
        assert cache.sync_status() == 0
        if step % 8 and step != w.n_steps - 1:
            continue
        for (b, h) in _all_units(w):
            Ku = torch.cat([K[b, h, :int(lens_h[b])], extra[(b, h)][0]])
            Vu = torch.cat([V[b, h, :int(lens_h[b])], extra[(b, h)][1]])

            def run(override=None):
                return parity.oracle_unit(w, q[b], Ku, Vu, gamma, h, n_sink=w.n_sink, n_local=w.n_local,
                                          override=override, stats_bf16=True)
            parity.compare_unit(w, run(), out[b].cpu().numpy(), osp[b].cpu().numpy(), orla[b].cpu().numpy(),
                                sel[b, h].cpu().numpy(), h, n_sink=w.n_sink, n_local=w.n_local, rerun=run,
                                tie_band=parity.TIE_BAND_STATS_BF16)
