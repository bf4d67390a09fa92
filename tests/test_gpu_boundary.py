"""Device-side error reporting of the library: conditions only a kernel can see are reported through the status word
that spla_sync_status returns, never through a fault, a trap or a hang."""
import numpy as np
import pytest
import torch

from paper_2601_22379_b200 import binding, runner, synth
from tests import parity
from tests.test_gpu_parity import DEV, _all_units, _check_units, _decode_all

pytestmark = pytest.mark.gpu


def _small(name="gqa_32k", **over):
    kw = dict(batch=2, context=64 * 40 + 9, n_needles=2)
    kw.update(over)
    return synth.BY_NAME[name].scaled(**kw)


@pytest.mark.parametrize("flags", [0, binding.SPLA_GENERAL_KERNELS])
def test_a_wait_that_runs_out_is_reported_as_timeout_and_the_context_stays_usable(flags):
    """The copy barriers of the decode kernels are told to expect 16 bytes more than will ever arrive and to give up
    after a few thousand polls: every wait runs out, the kernels skip their arithmetic, return, and latch
    SPLA_ERR_TIMEOUT.  With the hook cleared the same cache decodes correctly again."""
    w = _small()
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    good = cache.decode(q, gamma).clone()
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    cache.debug_wait_hook(4000, 16)
    cache.decode(q, gamma)
    torch.cuda.synchronize()                                   # returns: nothing hangs
    assert cache.sync_status() == binding.SPLA_ERR_TIMEOUT
    assert cache.sync_status() == 0                            # reading clears it
    cache.debug_wait_hook(0, 0)
    again = cache.decode(q, gamma)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert torch.equal(again, good)
    assert binding.load().spla_status_string(binding.SPLA_ERR_TIMEOUT) != binding.load().spla_status_string(binding.SPLA_ERR_CUDA)
    with pytest.raises(binding.SplaError):
        cache.debug_wait_hook(10, 7)                           # not a multiple of 16


@pytest.mark.parametrize("flags", [0, binding.SPLA_GENERAL_KERNELS])
def test_invalid_entries_of_a_given_selection_are_dropped_and_reported(flags):
    """spla_decode_selected does not trust its index list: a hole, an index past the last block and a duplicate are
    dropped, the rest is attended to, SPLA_ERR_BOUNDS is latched, and the outputs are those of the surviving set."""
    w = _small(top_k=8)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    nblk = -(-w.context // w.block_size)
    bad = np.full((w.batch, w.n_kv_heads, w.top_k), -1, dtype=np.int32)
    bad[:, :, :7] = [0, -1, 5, nblk + 3, 5, 2 ** 30, nblk - 1]          # hole, past the end, duplicate, far outside
    clean = np.full_like(bad, -1)
    clean[:, :, :3] = [0, 5, nblk - 1]
    osp = torch.empty(w.batch, w.n_q_heads, w.head_dim, device=DEV)
    out_bad = cache.decode_selected(q, gamma, torch.as_tensor(bad, device=DEV), dbg_o_sparse=osp).clone()
    torch.cuda.synchronize()
    assert cache.sync_status() == binding.SPLA_ERR_BOUNDS
    assert torch.isfinite(out_bad).all() and torch.isfinite(osp).all()
    out_clean = cache.decode_selected(q, gamma, torch.as_tensor(clean, device=DEV))
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert torch.equal(out_bad, out_clean)
    # a list of padding only: nothing selected, nothing reported, finite output
    none = torch.full((w.batch, w.n_kv_heads, w.top_k), -1, dtype=torch.int32, device=DEV)
    out_none = cache.decode_selected(q, gamma, none)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0 and torch.isfinite(out_none).all()


@pytest.mark.parametrize("flags", [0, binding.SPLA_GENERAL_KERNELS])
def test_a_corrupt_length_is_clamped_and_reported(flags):
    """seq_lens belongs to the caller.  A value above max_context (or below zero) is clamped by every decode kernel
    and reported; nothing is read outside the buffers, and the other sequence decodes as before."""
    w = _small()
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    good = cache.decode(q, gamma).clone()
    torch.cuda.synchronize()
    keep = cache.bufs.seq_lens.clone()
    for poison in (cache.cfg.max_context + 1000, -5):
        cache.bufs.seq_lens[1] = poison
        sel = cache.new_sel_buffer()
        out = cache.decode(q, gamma, sel_idx=sel)
        torch.cuda.synchronize()
        assert cache.sync_status() == binding.SPLA_ERR_BOUNDS
        s = sel.cpu().numpy()
        assert ((s >= -1) & (s < cache.max_blocks)).all()
        assert torch.equal(out[0], good[0])
    cache.bufs.seq_lens.copy_(keep)
    out = cache.decode(q, gamma)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0 and torch.equal(out, good)


@pytest.mark.parametrize("name,over,flags,window", [
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31), 0, None),
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31), binding.SPLA_GENERAL_KERNELS, None),
    ("gqa_32k", dict(batch=1, context=64 * 30 + 5), binding.SPLA_STATS_BF16, (32, 16)),
    ("tiny_ref", dict(context=64 * 20 + 13), 0, None),
    ("ragged_serving", dict(batch=6, context=6000, context_min=300, n_steps=2), 0, None),
    ("very_long_1m", dict(context=128 * 140 + 77, n_needles=4), 0, None),
])
def test_checked_mode_finds_nothing_and_changes_nothing(name, over, flags, window):
    """SPLA_DEBUG_BOUNDS (the stand-in for a memory checker): every kernel checks the indices it derives before it
    uses them.  On correct inputs no check fires on any path (bulk append, decode-step appends, score, select, attend),
    the results equal those of the unchecked build bit for bit, and they match the oracle."""
    w = synth.BY_NAME[name].scaled(**dict(over, n_steps=2))
    plain, K, V, lens = runner.build_cache(w, DEV, flags=flags, window=window)
    chk, _, _, _ = runner.build_cache(w, DEV, flags=flags | binding.SPLA_DEBUG_BOUNDS, window=window, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    for step in range(2):
        k1, v1 = synth.step_kv(w, step, DEV)
        q = synth.step_queries(w, step, DEV)
        a = plain.append_decode(k1, v1, q, gamma).clone()
        b = chk.append_decode(k1, v1, q, gamma).clone()
        torch.cuda.synchronize()
        assert plain.sync_status() == 0 and chk.sync_status() == 0
        assert torch.equal(a, b)
    assert torch.equal(plain.bufs.stats, chk.bufs.stats) and torch.equal(plain.bufs.rla_state, chk.bufs.rla_state)
    lens_h = lens.cpu().numpy()
    extra = {}
    for (b_, h) in _all_units(w):
        ks = [synth.step_kv(w, s, DEV) for s in range(2)]
        extra[(b_, h)] = (torch.cat([k[0][b_, h] for k in ks]), torch.cat([k[1][b_, h] for k in ks]))
    _check_units(w, chk, synth.step_queries(w, 1, DEV), gamma, K, V, lens_h, _all_units(w)[:4], w.n_sink, w.n_local,
                 extra=extra, window=window)


def test_near_complete_selection_keeps_the_strict_tolerance():
    """All blocks but one or two selected: o_bar - o_tilde (Section 3.2, Eq. rla-impl-3) is a small difference of two
    large sums and the RMSNorm rescales it, so the rounding of the selected linear term reaches the output amplified
    by |o_bar| / |o_rla|.  The linear branch carries its operands with 17 to 24 bits for this reason; the outputs must
    stay inside the ordinary tolerances with nothing widened."""
    worst = 0.0
    for (nblk, top_k, hq, hkv, d, B) in [(17, 16, 8, 2, 128, 64), (17, 16, 4, 1, 64, 64), (33, 32, 10, 2, 128, 32),
                                         (65, 64, 8, 2, 128, 16), (18, 16, 6, 1, 128, 64), (9, 8, 16, 2, 64, 128)]:
        for outl in (0, 2):
            w = synth.BY_NAME["gqa_32k"].scaled(batch=2, n_q_heads=hq, n_kv_heads=hkv, head_dim=d, block_size=B, top_k=top_k,
                                               context=nblk * B - 3, n_needles=0, n_outlier_channels=outl, n_sink=1, n_local=1)
            cache, K, V, lens = runner.build_cache(w, DEV)
            gamma = synth.gamma(w).to(DEV)
            q = synth.step_queries(w, 0, DEV)
            out, osp, orla, sel = _decode_all(cache, w, q, gamma)
            for (b, h) in _all_units(w):
                def run(override=None):
                    return parity.oracle_unit(w, q[b], K[b, h], V[b, h], gamma, h, n_sink=1, n_local=1, override=override)
                res = run()
                parity.compare_unit(w, res, out[b], osp[b], orla[b], sel[b, h], h, n_sink=1, n_local=1, rerun=run)
                worst = max(worst, np.linalg.norm(res["o_bar"]) / max(np.linalg.norm(res["o_rla"]), 1e-30))
    assert worst > 3.0                                        # the cases do cancel


@pytest.mark.parametrize("flags,window", [(0, None), (binding.SPLA_STATS_BF16, None), (binding.SPLA_STATS_BF16, (32, 16)),
                                          (0, (32, 16)), (binding.SPLA_GENERAL_KERNELS, None)])
def test_what_lies_beyond_the_end_of_a_sequence_never_reaches_the_results(flags, window):
    """The caches are caller memory and are never cleared: past the last token of a sequence they hold whatever was
    there before.  Here that is NaN everywhere (a large NaN-filled tensor is freed just before the caches are
    allocated, so that they reuse its memory).  Steps across a block boundary - the new block then holds one valid
    token and 63 rows of NaN - must give finite outputs, the same from the one-call step as from separate calls."""
    junk = torch.full((3 << 30,), float("nan"), dtype=torch.bfloat16, device=DEV)
    del junk
    torch.cuda.synchronize()
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 40 + 60, n_steps=8)
    a, K, V, lens = runner.build_cache(w, DEV, flags=flags, window=window)
    b, _, _, _ = runner.build_cache(w, DEV, flags=flags, window=window, prefill=(K, V, lens))
    assert torch.isnan(a.bufs.k_cache.float()).any()          # the poison is where the test wants it
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
        assert torch.isfinite(oa).all() and torch.isfinite(ob).all(), f"step {step}"
        assert torch.equal(sa, sb) and torch.equal(oa, ob), f"step {step}"
