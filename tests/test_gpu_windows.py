"""GPU parity of the strided-window selection (Section 3.1, "Strided Block Selection": Taylor statistics on windows of
C tokens every s tokens, max-pooled per block) against the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import spla_oracle as O
from paper_2601_22379_b200 import binding, runner, synth
from tests import parity
from tests.test_gpu_parity import DEV, _all_units, _check_units, _decode_all, _stepped_full

pytestmark = pytest.mark.gpu
WIN = (32, 16)            # the paper's C and s


def _window_stats_close(cache, K, lens, w, window):
    for b in range(w.batch):
        for h in (0, w.n_kv_heads - 1):
            L = int(lens[b])
            nblk = -(-L // w.block_size)
            mean, var, n = O.window_statistics(K[b, h, :L].double().cpu().numpy(), w.block_size, *window)
            st = cache.bufs.stats[b, h, :nblk].cpu().numpy()          # [nblk, NW, 2, d]
            live = n > 0
            assert parity.rel_l2(st[:, :, 0][live], mean[live]) < 2e-6
            assert parity.rel_l2(st[:, :, 1][live], var[live]) < 2e-6


@pytest.mark.parametrize("name,over,window", [
    ("gqa_32k", dict(batch=2, context=64 * 11 + 37, n_needles=0), WIN),
    ("very_long_1m", dict(context=128 * 9 + 100, n_needles=0), WIN),           # B = 128: seven windows per block
    ("tiny_ref", dict(batch=2, context=64 * 9 + 5, n_needles=0), (16, 16)),    # fp32, disjoint windows
])
def test_window_statistics_match_oracle_on_every_append_path(name, over, window):
    w = synth.BY_NAME[name].scaled(**over)
    bulk, K, V, lens = runner.build_cache(w, DEV, window=window)
    chunked, _, _, _ = runner.build_cache(w, DEV, window=window, chunk=77, prefill=(K, V, lens))
    small, _, _, _ = runner.build_cache(w, DEV, window=window, chunk=19, prefill=(K, V, lens))      # the fused kernel
    torch.cuda.synchronize()
    assert bulk.cfg.n_windows == (w.block_size - window[0]) // window[1] + 1
    lens_h = lens.cpu().numpy()
    _window_stats_close(bulk, K, lens_h, w, window)
    nblk = -(-int(lens_h.max()) // w.block_size)
    # the statistics do not depend on how the tokens were split across calls; compare what is defined: windows
    # that hold at least one token
    n = O.window_statistics(K[0, 0, :int(lens_h[0])].double().cpu().numpy(), w.block_size, *window)[2]
    live = torch.as_tensor(n > 0, device=DEV)
    for other in (chunked, small):
        a, b = bulk.bufs.stats[0, 0, :nblk][live], other.bufs.stats[0, 0, :nblk][live]
        assert torch.equal(a, b)


SMALL = [
    ("tiny_ref", dict(context=64 * 20 + 13)),
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31)),
    ("long_128k", dict(batch=1, context=64 * 150 + 1, n_steps=2)),
    ("very_long_1m", dict(context=128 * 140 + 77, n_needles=4)),
    ("ragged_serving", dict(batch=6, context=6000, context_min=300, n_steps=2)),
]


@pytest.mark.parametrize("name,over", SMALL)
@pytest.mark.parametrize("flags", [0, binding.SPLA_GENERAL_KERNELS])
def test_window_decode_matches_oracle_small(name, over, flags):
    w = synth.BY_NAME[name].scaled(**over)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags, window=WIN)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    n_exact = _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, window=WIN)
    assert n_exact >= 0.9 * w.batch * w.n_kv_heads


@pytest.mark.parametrize("last", [1, 15, 16, 17, 33, 48, 63])
def test_window_partial_last_block_counts(last):
    """The open block holds `last` tokens: windows with fewer than C tokens, and windows with none."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 24 + last, n_needles=2)
    cache, K, V, lens = runner.build_cache(w, DEV, window=WIN, n_sink=0, n_local=0)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), 0, 0, window=WIN)


def test_window_first_order_flag():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 40 + 9)
    cache, K, V, lens = runner.build_cache(w, DEV, window=WIN, flags=binding.SPLA_FIRST_ORDER)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, window=WIN, order=1)


def test_window_steps_with_append_small():
    """Append one token then decode with windows, across a block boundary; every unit, every step."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 40 + 61, n_steps=6)
    cache, K, V, lens = runner.build_cache(w, DEV, window=WIN)
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    extra = {u: (torch.zeros(0, w.head_dim, dtype=w.torch_dtype, device=DEV),) * 2 for u in _all_units(w)}
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        cache.append_tokens(k1, v1)
        for (b, h) in extra:
            extra[(b, h)] = (torch.cat([extra[(b, h)][0], k1[b, h]]), torch.cat([extra[(b, h)][1], v1[b, h]]))
        q = synth.step_queries(w, step, DEV)
        _check_units(w, cache, q, gamma, K, V, lens_h, _all_units(w), w.n_sink, w.n_local, extra=extra, window=WIN)


def test_window_equal_to_block_is_block_mode_bit_for_bit():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 30 + 21)
    a, K, V, lens = runner.build_cache(w, DEV)
    b, _, _, _ = runner.build_cache(w, DEV, window=(64, 64), prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    ra, rb = _decode_all(a, w, q, gamma), _decode_all(b, w, q, gamma)
    assert np.array_equal(ra[3], rb[3]) and np.array_equal(ra[0], rb[0])
    assert torch.equal(a.bufs.stats, b.bufs.stats.reshape(a.bufs.stats.shape))


def test_window_long_128k_full_size_sampled_units():
    """The benchmark's window configuration at full size: 128K context, C = 32, s = 16, three sampled units."""
    _stepped_full(synth.CONFIGS[2].scaled(n_steps=3), n_units=3, check_steps={0, 2}, window=WIN)


def test_noalloc_entry_rejects_windows():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 8, n_needles=0)
    cache, K, V, lens = runner.build_cache(w, DEV, window=WIN)
    q = synth.step_queries(w, 0, DEV)
    rc = binding.select_blocks_noalloc(cache.cfg, cache.bufs.stats, cache.bufs.seq_lens, q, cache.new_sel_buffer())
    assert rc == binding.SPLA_ERR_UNSUPPORTED
