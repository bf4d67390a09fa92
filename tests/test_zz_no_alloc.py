"""The allocation-free selection entry point against the regular decode path (collected last on purpose).

Callers that cannot allocate device memory (a frozen memory pool, a plug-in without an allocator, a loop where
cudaMalloc is forbidden) use spla_select_blocks_noalloc, whose scratch is a fixed array inside the library.
It must pick exactly the blocks spla_decode picks, call after call, even though the array still holds the
previous call's data.
"""
import numpy as np
import pytest
import torch

from paper_2601_22379_b200 import binding, runner, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_noalloc_selection_matches_decode_on_two_calls_in_a_row():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=3, context=64 * 90 + 37, n_needles=4)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    cfg = cache.cfg
    sel_new = cache.new_sel_buffer()
    scores_new = torch.empty(w.batch, w.n_kv_heads, cache.max_blocks, dtype=torch.float32, device=DEV)
    for call, step in enumerate((0, 1)):                      # two calls in a row, different queries
        q = synth.step_queries(w, step, DEV)
        sel_ref = cache.new_sel_buffer()
        cache.decode(q, gamma, sel_idx=sel_ref)
        scores_ref = cache.scores()
        sel_new.fill_(-7)
        free_before = torch.cuda.mem_get_info()[0]
        rc = binding.select_blocks_noalloc(cfg, cache.bufs.stats, cache.bufs.seq_lens, q, sel_new, scores_new)
        torch.cuda.synchronize()
        assert rc == binding.SPLA_OK, rc
        if call == 1:                                         # (the first call may load the library's device image)
            assert torch.cuda.mem_get_info()[0] == free_before   # nothing was allocated on the device
        assert torch.equal(sel_new, sel_ref), f"call {call}: selections differ"
        nblk = -(-w.context // w.block_size)
        np.testing.assert_allclose(scores_new[:, :, :nblk].cpu().numpy(), scores_ref[:, :, :nblk].cpu().numpy(),
                                   rtol=2e-5)
        assert torch.all(scores_new[:, :, nblk:] == 0)
    # after a shorter problem the longer one is still right: stale tails of the shared array are not read
    w2 = w.scaled(batch=1, context=64 * 7 + 3, n_needles=0)
    c2, _, _, _ = runner.build_cache(w2, DEV)
    q2 = synth.step_queries(w2, 0, DEV)
    ref2, new2 = c2.new_sel_buffer(), c2.new_sel_buffer()
    c2.decode(q2, synth.gamma(w2).to(DEV), sel_idx=ref2)
    assert binding.select_blocks_noalloc(c2.cfg, c2.bufs.stats, c2.bufs.seq_lens, q2, new2) == binding.SPLA_OK
    torch.cuda.synchronize()
    assert torch.equal(new2, ref2)


def test_noalloc_rejects_what_does_not_fit_its_fixed_scratch():
    big = binding.make_config(batch=64, n_q_heads=32, n_kv_heads=8, head_dim=128, block_size=64, top_k=16,
                              max_context=65536)
    dummy = torch.zeros(64, dtype=torch.float32, device=DEV)
    idx = torch.zeros(64, dtype=torch.int32, device=DEV)
    rc = binding.load().spla_select_blocks_noalloc(big, dummy.data_ptr(), idx.data_ptr(), dummy.data_ptr(),
                                                   idx.data_ptr(), None, None, None)
    assert rc == binding.SPLA_ERR_UNSUPPORTED
    assert binding.load().spla_select_blocks_noalloc(big, None, None, None, None, None, None, None) == binding.SPLA_ERR_INVALID_ARG


def test_noalloc_clamps_a_length_beyond_the_capacity_and_says_so():
    """seq_lens is the caller's buffer: a stale value above max_context must neither overrun the fixed scratch nor
    the kernel's shared arrays.  It is clamped to the capacity and reported through status_out."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 20, n_needles=0)
    cache, K, V, lens = runner.build_cache(w, DEV)
    q = synth.step_queries(w, 0, DEV)
    sel = cache.new_sel_buffer()
    status = torch.full((1,), 77, dtype=torch.int32, device=DEV)
    assert binding.select_blocks_noalloc(cache.cfg, cache.bufs.stats, cache.bufs.seq_lens, q, sel, None, status) == binding.SPLA_OK
    torch.cuda.synchronize()
    assert status.item() == 0
    bad = cache.bufs.seq_lens.clone()
    bad[1] = cache.cfg.max_context + 12345
    sel.fill_(-7)
    assert binding.select_blocks_noalloc(cache.cfg, cache.bufs.stats, bad, q, sel, None, status) == binding.SPLA_OK
    torch.cuda.synchronize()
    assert status.item() == binding.SPLA_ERR_BOUNDS
    s = sel.cpu().numpy()
    assert ((s >= -1) & (s < cache.max_blocks)).all()                 # a clean selection inside the cache for every unit
    ref = cache.new_sel_buffer()
    cache.select(q, ref)
    assert torch.equal(sel[0], ref[0])                                # the untouched sequence selects as before
