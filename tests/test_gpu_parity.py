"""GPU parity: the CUDA library, called through its C ABI, against the float64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import spla_oracle as O
from paper_2601_22379_b200 import binding, runner, synth
from tests import parity

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _decode_all(cache, w, q, gamma):
    cfg = cache.cfg
    sel = cache.new_sel_buffer()
    osp = torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=DEV)
    orla = torch.empty_like(osp)
    out = cache.decode(q, gamma, sel_idx=sel, dbg_o_sparse=osp, dbg_o_rla=orla)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    return out.cpu().numpy(), osp.cpu().numpy(), orla.cpu().numpy(), sel.cpu().numpy()


def _check_units(w, cache, q, gamma, K, V, lens, units, n_sink, n_local, extra=None, order=2, use_rla=True,
                 window=None):
    stats_bf16 = bool(cache.cfg.flags & binding.SPLA_STATS_BF16)
    tie_band = parity.TIE_BAND_STATS_BF16 if stats_bf16 else parity.TIE_BAND
    """extra: optional dict (b,h) -> (K_tail, V_tail) of appended tokens."""
    out, osp, orla, sel = _decode_all(cache, w, q, gamma)
    n_exact = 0
    for (b, h) in units:
        L = int(lens[b])
        Ku, Vu = K[b, h, :L], V[b, h, :L]
        if extra is not None:
            Ku = torch.cat([Ku, extra[(b, h)][0]], dim=0)
            Vu = torch.cat([Vu, extra[(b, h)][1]], dim=0)

        def run(override=None):
            return parity.oracle_unit(w, q[b], Ku, Vu, gamma, h, n_sink=n_sink, n_local=n_local, override=override,
                                      order=order, use_rla=use_rla, window=window, stats_bf16=stats_bf16)
        res = run()
        n_exact += parity.compare_unit(w, res, out[b], osp[b], orla[b], sel[b, h], h, n_sink=n_sink, n_local=n_local,
                                       rerun=run, tie_band=tie_band)
    return n_exact


def _all_units(w):
    return [(b, h) for b in range(w.batch) for h in range(w.n_kv_heads)]


# ---------------------------------------------------------------------------------------------------------
# append: statistics, state, per-token lse, lengths
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,ctx", [("tiny_ref", 64 * 9 + 17), ("gqa_32k", 64 * 11 + 5)])
def test_append_statistics_and_state_match_oracle(name, ctx):
    w = synth.BY_NAME[name].scaled(batch=2, context=ctx, n_needles=0)
    cache, K, V, lens = runner.build_cache(w, DEV)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert cache.bufs.seq_lens.cpu().tolist() == [ctx, ctx]
    nblk = -(-ctx // w.block_size)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            Kd, Vd = K[b, h].double().cpu().numpy(), V[b, h].double().cpu().numpy()
            mean, var, n = O.block_statistics(Kd, w.block_size)
            st = cache.bufs.stats[b, h, :nblk].cpu().numpy()
            assert parity.rel_l2(st[:, 0], mean) < 2e-6 and parity.rel_l2(st[:, 1], var) < 2e-6
            S = cache.bufs.rla_state[b, h].cpu().numpy()
            tensor_path = w.kv_dtype == "bf16" and w.head_dim == 128 and ctx >= 256
            assert parity.rel_l2(S, O.rla_global_state(Kd, Vd)) < (parity.STATE_TOL_TENSOR if tensor_path else parity.STATE_TOL_FMA)
            lse = cache.bufs.tok_lse[b, h, :ctx].cpu().numpy()
            ref = np.log(np.sum(np.exp(Kd - Kd.max(axis=1, keepdims=True)), axis=1)) + Kd.max(axis=1)
            assert np.max(np.abs(lse - ref)) < 2e-5
            kc = cache.bufs.k_cache[b, h].reshape(-1, w.head_dim)[:ctx]
            assert torch.equal(kc, K[b, h]) and torch.equal(cache.bufs.v_cache[b, h].reshape(-1, w.head_dim)[:ctx], V[b, h])
    # chunked and token-by-token appends give the same statistics bit for bit, and the same state to rounding
    cache2, _, _, _ = runner.build_cache(w, DEV, chunk=100, prefill=(K, V, lens))
    torch.cuda.synchronize()
    assert torch.equal(cache2.bufs.stats[:, :, :nblk], cache.bufs.stats[:, :, :nblk])
    assert torch.equal(cache2.bufs.tok_lse[:, :, :ctx], cache.bufs.tok_lse[:, :, :ctx])
    assert parity.rel_l2(cache2.bufs.rla_state.cpu().numpy(), cache.bufs.rla_state.cpu().numpy()) < parity.STATE_TOL_TENSOR
    # ... and so does the fused decode-step kernel (one, three and seventeen tokens per call)
    cache3 = binding.SplaCache(runner.config_for(w), DEV)
    pos, sizes = 0, [1, 3, 17, 1, 1, 32, 5]
    i = 0
    while pos < ctx:
        m = min(sizes[i % len(sizes)], ctx - pos)
        cache3.append_tokens(K[:, :, pos:pos + m].contiguous(), V[:, :, pos:pos + m].contiguous())
        pos += m
        i += 1
    torch.cuda.synchronize()
    assert cache3.sync_status() == 0 and cache3.bufs.seq_lens.cpu().tolist() == [ctx, ctx]
    assert torch.equal(cache3.bufs.stats[:, :, :nblk], cache.bufs.stats[:, :, :nblk])
    assert torch.equal(cache3.bufs.tok_lse[:, :, :ctx], cache.bufs.tok_lse[:, :, :ctx])
    assert torch.equal(cache3.bufs.k_cache.reshape(2, w.n_kv_heads, -1, w.head_dim)[:, :, :ctx], K)
    assert parity.rel_l2(cache3.bufs.rla_state.cpu().numpy(), cache.bufs.rla_state.cpu().numpy()) < parity.STATE_TOL_TENSOR


def test_ragged_append_with_device_lengths():
    w = synth.BY_NAME["ragged_serving"].scaled(batch=5, context=1500, context_min=1, n_steps=4)
    cache, K, V, lens = runner.build_cache(w, DEV, chunk=333)
    torch.cuda.synchronize()
    assert torch.equal(cache.bufs.seq_lens, lens)
    for b in range(w.batch):
        L = int(lens[b])
        nblk = -(-L // w.block_size)
        mean, var, _ = O.block_statistics(K[b, 3, :L].double().cpu().numpy(), w.block_size)
        st = cache.bufs.stats[b, 3, :nblk].cpu().numpy()
        assert parity.rel_l2(st[:, 0], mean) < 2e-6 and parity.rel_l2(st[:, 1], var) < 2e-6


# ---------------------------------------------------------------------------------------------------------
# decode on scaled-down versions of the five configurations: every unit, ragged tails, forced-block variants
# ---------------------------------------------------------------------------------------------------------
SMALL = [
    ("tiny_ref", dict(context=64 * 20 + 13)),
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31)),
    ("long_128k", dict(batch=1, context=64 * 150 + 1, n_steps=2)),
    ("very_long_1m", dict(context=128 * 140 + 77, n_needles=4)),
    ("ragged_serving", dict(batch=6, context=6000, context_min=300, n_steps=2)),
]


@pytest.mark.parametrize("name,over", SMALL)
@pytest.mark.parametrize("forced,flags", [((1, 4), 0), ((0, 0), 0), ((1, 1), 0), ((1, 4), binding.SPLA_GENERAL_KERNELS)])
def test_decode_matches_oracle_small(name, over, forced, flags):
    """Default (cluster / tensor-core) kernels with three forced-block settings, and the general kernels."""
    w = synth.BY_NAME[name].scaled(**over)
    n_sink, n_local = forced
    cache, K, V, lens = runner.build_cache(w, DEV, n_sink=n_sink, n_local=n_local, flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    lens_h = lens.cpu().numpy()
    n_exact = _check_units(w, cache, q, gamma, K, V, lens_h, _all_units(w), n_sink, n_local)
    assert n_exact >= 0.9 * w.batch * w.n_kv_heads        # tie-band swaps are rare


def test_decode_steps_with_append_small():
    """Append one token then decode, across a block boundary; every unit checked at every step."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 40 + 62, n_steps=5)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    extra = {u: (torch.zeros(0, w.head_dim, dtype=w.torch_dtype, device=DEV),) * 2 for u in _all_units(w)}
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        cache.append_tokens(k1, v1)
        for (b, h) in extra:
            extra[(b, h)] = (torch.cat([extra[(b, h)][0], k1[b, h]]), torch.cat([extra[(b, h)][1], v1[b, h]]))
        q = synth.step_queries(w, step, DEV)
        _check_units(w, cache, q, gamma, K, V, lens_h, _all_units(w), w.n_sink, w.n_local, extra=extra)
    assert cache.bufs.seq_lens.cpu().tolist() == [w.context + w.n_steps] * w.batch


# ---------------------------------------------------------------------------------------------------------
# the five configurations at full size, in the launch configuration the benchmark times; sampled units
# ---------------------------------------------------------------------------------------------------------
def _sample_units(w, n, seed=0):
    rng = np.random.default_rng(seed)
    allu = _all_units(w)
    idx = rng.permutation(len(allu))[:n]
    return [allu[i] for i in idx]


def _check_all_selections(w, cache, q, K, V, lens_h, window=None):
    """Steps a1-a2 for EVERY unit at full size: the library's index set against the oracle's score-only path
    (block statistics -> grouped BlockScore -> Select; Section 3.1 Eq. taylor-2nd, Section 2.2, Section 2.1), which
    needs no attention and is therefore cheap enough to run on all units."""
    assert window is None
    sel = cache.select(q)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    sel = sel.cpu().numpy()
    G = w.group
    scale = 1.0 / np.sqrt(w.head_dim)
    n_same = 0
    for b in range(w.batch):
        L = int(lens_h[b])
        for h in range(w.n_kv_heads):
            mean, var, n = O.block_statistics(K[b, h, :L].double().cpu().numpy(), w.block_size)
            qh = q[b, h * G:(h + 1) * G].double().cpu().numpy() * scale
            _, _, score = O.block_scores(qh, mean, var, n)
            ref = {"sel": O.select_blocks(score, w.top_k, w.n_sink, w.n_local), "score": score}
            n_same += parity.check_selection(sel[b, h], ref, w.top_k, w.n_sink, w.n_local)
    assert n_same >= 0.9 * w.batch * w.n_kv_heads          # tie-band swaps are rare
    return n_same


def test_config1_tiny_ref_full_16_steps():
    w = synth.CONFIGS[0]
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    extra = {(0, 0): (torch.zeros(0, w.head_dim, device=DEV), torch.zeros(0, w.head_dim, device=DEV))}
    needles = set(synth.needle_blocks(w)[0, 0].tolist())
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        cache.append_tokens(k1, v1)
        extra[(0, 0)] = (torch.cat([extra[(0, 0)][0], k1[0, 0]]), torch.cat([extra[(0, 0)][1], v1[0, 0]]))
        q = synth.step_queries(w, step, DEV)
        _check_units(w, cache, q, gamma, K, V, lens_h, [(0, 0)], w.n_sink, w.n_local, extra=extra)
        sel = cache.new_sel_buffer()
        cache.decode(q, gamma, sel_idx=sel)
        assert needles <= set(sel.cpu().numpy()[0, 0].tolist())


def test_config2_gqa_32k_full_three_query_seeds():
    w = synth.CONFIGS[1]
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    lens_h = lens.cpu().numpy()
    nb = synth.needle_blocks(w)
    for seed in range(3):
        q = synth.step_queries(w, seed, DEV)
        units = _sample_units(w, 4, seed)
        _check_units(w, cache, q, gamma, K, V, lens_h, units, w.n_sink, w.n_local)
        sel = cache.new_sel_buffer()
        cache.decode(q, gamma, sel_idx=sel)
        sel = sel.cpu().numpy()
        for b in range(w.batch):
            for h in range(w.n_kv_heads):
                assert set(nb[b, h].tolist()) <= set(sel[b, h].tolist())


def _stepped_full(w, n_units, check_steps, window=None, flags=0, all_selections=False):
    cache, K, V, lens = runner.build_cache(w, DEV, window=window, flags=flags)
    stats_bf16 = bool(flags & binding.SPLA_STATS_BF16)
    tie_band = parity.TIE_BAND_STATS_BF16 if stats_bf16 else parity.TIE_BAND
    gamma = synth.gamma(w).to(DEV)
    gam = gamma.double().cpu().numpy()
    lens_h = lens.cpu().numpy()
    if all_selections:                                     # every unit's index set on the prefilled cache
        _check_all_selections(w, cache, synth.step_queries(w, 0, DEV), K, V, lens_h)
    units = _sample_units(w, n_units, 1)
    G = w.group
    orc = {}
    for (b, h) in units:
        L = int(lens_h[b])
        orc[(b, h)] = O.UnitCache.from_prefill(K[b, h, :L].double().cpu().numpy(), V[b, h, :L].double().cpu().numpy(),
                                               w.block_size, window=window)
    del K, V
    for step in range(w.n_steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        cache.append_tokens(k1, v1)
        for (b, h), oc in orc.items():
            oc.append(k1[b, h].double().cpu().numpy(), v1[b, h].double().cpu().numpy())
        if step not in check_steps:
            continue
        q = synth.step_queries(w, step, DEV)
        out, osp, orla, sel = _decode_all(cache, w, q, gamma)
        qh = q.double().cpu().numpy()
        for (b, h), oc in orc.items():
            def run(override=None):
                return oc.decode(qh[b, h * G:(h + 1) * G], gam[h * G:(h + 1) * G], top_k=w.top_k, n_sink=w.n_sink,
                                 n_local=w.n_local, override_selection=override, stats_bf16=stats_bf16)
            parity.compare_unit(w, run(), out[b], osp[b], orla[b], sel[b, h], h, n_sink=w.n_sink, n_local=w.n_local,
                                rerun=run, tie_band=tie_band)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert torch.equal(cache.bufs.seq_lens.cpu(), torch.as_tensor(lens_h) + w.n_steps)


def test_config3_long_128k_full_64_steps():
    _stepped_full(synth.CONFIGS[2], n_units=3, check_steps={0, 1, 31, 62, 63}, all_selections=True)


def test_long_128k_full_size_with_the_group_size_of_the_papers_model():
    """40 query heads over 8 KV heads (G = 5, Table 1 of the paper) at the full 128K context: all selections, and
    sampled units' outputs over a few steps."""
    w = synth.CONFIGS[2].scaled(n_q_heads=40, n_steps=6)
    _stepped_full(w, n_units=2, check_steps={0, 5}, all_selections=True)


@pytest.mark.parametrize("hq,flags", [(64, 0), (40, 0), (64, binding.SPLA_STATS_BF16), (24, 0)])
def test_more_heads_per_group_than_ctas_per_unit(hq, flags):
    """64 units share the device, so a unit gets a cluster of four CTAs or fewer; with groups of up to eight heads a CTA
    then merges two heads (and computes o_bar of both), and the partial results of a head arrive in the second row of
    its receive area."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=8, n_q_heads=hq, n_kv_heads=8, context=64 * 44 + 9, n_needles=3)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _sample_units(w, 6, 3), w.n_sink, w.n_local)


def test_sequences_of_more_than_8192_blocks_on_the_cluster_kernels():
    """More blocks than the selection's per-thread bit masks cover (128 x 64): the cluster kernels then select with the
    histogram method over the whole key table.  One sequence, two KV heads, 9000 blocks of 64 tokens: index sets of both
    units, outputs of one."""
    w = synth.BY_NAME["long_128k"].scaled(batch=1, n_q_heads=4, n_kv_heads=2, context=64 * 9000 + 17, n_needles=6)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_all_selections(w, cache, q, K, V, lens.cpu().numpy())
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), [(0, 1)], w.n_sink, w.n_local)


def test_config4_very_long_1m_full():
    w = synth.CONFIGS[3]
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _sample_units(w, 2, 4), w.n_sink, w.n_local)
    _check_all_selections(w, cache, q, K, V, lens.cpu().numpy())


def test_config5_ragged_serving_full_256_steps():
    _stepped_full(synth.CONFIGS[4], n_units=4, check_steps={0, 63, 64, 255}, all_selections=True)


# ---------------------------------------------------------------------------------------------------------
# edge and degenerate cases
# ---------------------------------------------------------------------------------------------------------
def test_fewer_blocks_than_top_k_is_dense_attention():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 5 + 9, n_needles=0, top_k=16)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    out, osp, orla, sel = _decode_all(cache, w, q, gamma)
    assert sel[0, 0].tolist() == [0, 1, 2, 3, 4, 5] + [-1] * 10
    G = w.group
    for h in range(w.n_kv_heads):
        dense = torch.nn.functional.scaled_dot_product_attention(
            q[0, h * G:(h + 1) * G].double()[None], K[0, h].double()[None], V[0, h].double()[None])[0].cpu().numpy()
        parity.check_outputs("o_sparse", osp[0, h * G:(h + 1) * G], dense, "bf16")
        obar = parity.oracle_unit(w, q[0], K[0, h], V[0, h], gamma, h, n_sink=1, n_local=4)["o_bar"]
        # everything selected: the residual is rounding noise relative to the global term
        assert np.abs(orla[0, h * G:(h + 1) * G]).max() < 5e-3 * np.abs(obar).max()


def test_empty_and_one_token_sequences():
    w = synth.BY_NAME["ragged_serving"].scaled(batch=3, context=200, context_min=200, n_steps=2)
    cache = binding.SplaCache(runner.config_for(w), DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    out, osp, orla, sel = _decode_all(cache, w, q, gamma)
    assert np.all(out == 0) and np.all(sel == -1)
    # sequence 0 stays empty, 1 gets one token, 2 gets 130 tokens
    K, V, _ = runner.generate_prefill(w, DEV)
    n_new = torch.tensor([0, 1, 130], dtype=torch.int32, device=DEV)
    cache.append_tokens(K, V, n_new)
    out, osp, orla, sel = _decode_all(cache, w, q, gamma)
    assert np.all(out[0] == 0) and np.all(sel[0] == -1)
    assert np.all(sel[1, :, 0] == 0) and np.all(sel[1, :, 1:] == -1)
    # one token: softmax over a single token returns its value; the residual branch vanishes
    np.testing.assert_allclose(osp[1].reshape(8, 4, -1), np.repeat(V[1, :, :1].float().cpu().numpy(), 4, axis=1), atol=1e-6)
    lens = np.array([0, 1, 130])
    _check_units(w, cache, q, gamma, K, V, lens, [(2, h) for h in range(8)], w.n_sink, w.n_local)


@pytest.mark.parametrize("hq,hkv", [(1, 1), (2, 1), (5, 1), (8, 1), (16, 1), (6, 2)])
def test_group_sizes(hq, hkv):
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, n_q_heads=hq, n_kv_heads=hkv, context=64 * 40 + 3, n_needles=3)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local)


@pytest.mark.parametrize("B,d,dt", [(16, 64, "bf16"), (32, 128, "f32"), (128, 64, "f32"), (128, 128, "bf16"), (64, 64, "bf16")])
def test_block_sizes_head_dims_dtypes(B, d, dt):
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, n_q_heads=4, n_kv_heads=2, head_dim=d, block_size=B, kv_dtype=dt,
                                       context=B * 33 + B // 2, n_needles=2, top_k=8, n_outlier_channels=2)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local)


def test_first_order_and_no_rla_flags():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 60 + 20, n_needles=3)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    cache, K, V, lens = runner.build_cache(w, DEV, flags=binding.SPLA_FIRST_ORDER)
    _check_units(w, cache, q, gamma, K, V, lens.cpu().numpy(), _all_units(w), w.n_sink, w.n_local, order=1)
    cache2, _, _, _ = runner.build_cache(w, DEV, flags=binding.SPLA_NO_RLA, prefill=(K, V, lens))
    out, osp, orla, sel = _decode_all(cache2, w, q, gamma)
    assert np.array_equal(out, osp)
    for h in range(w.n_kv_heads):
        res = parity.oracle_unit(w, q[0], K[0, h], V[0, h], gamma, h, n_sink=w.n_sink, n_local=w.n_local, use_rla=False)
        if parity.check_selection(sel[0, h], res, w.top_k, w.n_sink, w.n_local):
            parity.check_outputs("out", out[0, h * 4:(h + 1) * 4], res["out"], "bf16")


def test_decode_selected_uses_the_given_blocks():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 30 + 7, n_needles=0, top_k=6)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    rng = np.random.default_rng(5)
    sel = np.full((w.batch, w.n_kv_heads, w.top_k), -1, dtype=np.int32)
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            n = int(rng.integers(1, w.top_k + 1))
            sel[b, h, :n] = np.sort(rng.permutation(31)[:n])
    osp = torch.empty(w.batch, w.n_q_heads, w.head_dim, device=DEV)
    orla = torch.empty_like(osp)
    out = cache.decode_selected(q, gamma, torch.as_tensor(sel, device=DEV), dbg_o_sparse=osp, dbg_o_rla=orla)
    out, osp, orla = out.cpu().numpy(), osp.cpu().numpy(), orla.cpu().numpy()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            res = parity.oracle_unit(w, q[b], K[b, h], V[b, h], gamma, h, n_sink=1, n_local=4,
                                     override=[int(i) for i in sel[b, h] if i >= 0])
            sl = slice(h * 4, (h + 1) * 4)
            parity.check_outputs("o_sparse", osp[b, sl], res["o_sparse"], "bf16")
            parity.check_outputs("o_rla", orla[b, sl], res["o_rla"], "bf16")
            parity.check_outputs("out", out[b, sl], res["out"], "bf16")


def test_graph_replay_of_append_and_decode_matches_eager_calls():
    """The benchmark replays steps from a CUDA graph (with programmatic dependent launch between the kernels):
    the replayed steps must give what the same calls give one by one."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 200 + 30, n_steps=40)
    gamma = synth.gamma(w).to(DEV)
    steps = [(synth.step_kv(w, s, DEV), synth.step_queries(w, s, DEV)) for s in range(6)]
    eager, K, V, lens = runner.build_cache(w, DEV)
    ref = []
    for (k1, v1), q in steps:
        eager.append_tokens(k1, v1)
        ref.append(eager.decode(q, gamma).clone())
    cache, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    cache.set_length_bound(w.max_context - 8)               # replays append without the host seeing it
    outs = [torch.empty_like(ref[0]) for _ in steps]
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        cache.decode(steps[0][1], gamma, out=outs[0])        # load the kernels before capturing
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            for i, ((k1, v1), q) in enumerate(steps):
                cache.append_tokens(k1, v1)
                cache.decode(q, gamma, out=outs[i])
        graph.replay()
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert torch.equal(cache.bufs.seq_lens, eager.bufs.seq_lens)
    for a, b in zip(outs, ref):
        np.testing.assert_allclose(a.cpu().numpy(), b.cpu().numpy(), rtol=1e-5, atol=1e-6)


def test_select_then_decode_selected_equals_decode():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 50 + 9, n_needles=3)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    sel_a = cache.new_sel_buffer()
    out_a = cache.decode(q, gamma, sel_idx=sel_a).clone()
    sel_b = cache.select(q)
    out_b = cache.decode_selected(q, gamma, sel_b)
    torch.cuda.synchronize()
    assert torch.equal(sel_a, sel_b)
    # the two routes may split a unit's blocks over a different number of CTAs: the softmax weights are then rounded to
    # bf16 against other running maxima, so the outputs agree to bf16 accuracy (1e-4 .. 1e-3), not to fp32 accuracy
    a, b = out_a.cpu().numpy(), out_b.cpu().numpy()
    assert parity.rel_l2(b, a) < 1e-3 and parity.max_abs(b, a) < 2e-3


def test_scores_are_normalised_and_match_oracle():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 100 + 40, n_needles=4)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    cache.decode(q, gamma)
    sc = cache.scores().cpu().numpy()
    nblk = 101
    for h in range(w.n_kv_heads):
        res = parity.oracle_unit(w, q[0], K[0, h], V[0, h], gamma, h, n_sink=1, n_local=4)
        np.testing.assert_allclose(sc[0, h, :nblk], res["score"], rtol=2e-5)
        assert abs(sc[0, h, :nblk].sum() - w.group) < 1e-4


def test_capacity_overflow_is_reported_not_faulted():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=256, n_needles=0, n_steps=3)
    cache, K, V, lens = runner.build_cache(w, DEV)
    k1, v1 = synth.step_kv(w, 0, DEV)
    for _ in range(3):
        cache.append_tokens(k1, v1)
    with pytest.raises(binding.SplaError) as e:          # host-side bound: 256 + 3 is full
        cache.append_tokens(k1, v1)
    assert e.value.status == binding.SPLA_ERR_CAPACITY
    # device-side: lie to the host bound, the kernel skips the overflowing sequences and latches the status
    cache.set_length_bound(0)
    before = cache.bufs.rla_state.clone()
    cache.append_tokens(k1, v1)
    torch.cuda.synchronize()
    assert cache.sync_status() == binding.SPLA_ERR_CAPACITY
    assert cache.sync_status() == 0
    assert cache.bufs.seq_lens.cpu().tolist() == [259, 259] and torch.equal(before, cache.bufs.rla_state)


# ---------------------------------------------------------------------------------------------------------
# bulk state update on the tensor cores (bf16 cache, d = 128, appends of at least 256 tokens)
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("name,over,chunk", [
    ("gqa_32k", dict(batch=2, context=64 * 40 + 37, n_needles=0), 0),                    # 16 splits, ragged last tile
    ("ragged_serving", dict(batch=9, context=5000, context_min=1, n_steps=4), 0),        # device lengths, 2 splits
    ("ragged_serving", dict(batch=24, context=1200, context_min=200, n_steps=4), 0),     # one split: adds to S_bar itself
    ("long_128k", dict(batch=1, context=64 * 300 + 1, n_needles=0), 4096 + 333),         # several tensor-core appends in a row
    ("very_long_1m", dict(context=128 * 100 + 77, n_needles=0), 0),                      # B = 128
])
def test_tensor_core_state_update_matches_oracle_and_fma_kernel(name, over, chunk):
    w = synth.BY_NAME[name].scaled(**over)
    cache, K, V, lens = runner.build_cache(w, DEV, chunk=chunk)
    fma, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens), flags=binding.SPLA_GENERAL_KERNELS, chunk=chunk)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0 and fma.sync_status() == 0
    assert torch.equal(cache.bufs.seq_lens, lens)
    lens_h = lens.cpu().numpy()
    for b in range(w.batch):
        L = int(lens_h[b])
        for h in (0, w.n_kv_heads - 1):
            S = O.rla_global_state(K[b, h, :L].double().cpu().numpy(), V[b, h, :L].double().cpu().numpy())
            got = cache.bufs.rla_state[b, h].cpu().numpy()
            if L == 0:
                assert not got.any()
                continue
            tol = parity.STATE_TOL_TENSOR if L >= 64 else 1e-5      # a handful of tokens: few terms, same per-term error
            assert parity.rel_l2(got, S) < tol, (b, h, L)
            assert parity.rel_l2(got, fma.bufs.rla_state[b, h].cpu().numpy()) < 2 * parity.STATE_TOL_TENSOR
    # same inputs, same launch configuration: the update is reproducible bit for bit (partials are added in split order)
    again, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens), chunk=chunk)
    torch.cuda.synchronize()
    assert torch.equal(again.bufs.rla_state, cache.bufs.rla_state)


def test_decode_into_pinned_host_memory_equals_decode_into_device_memory():
    """`out` may be page-locked host memory (what the benchmark's end-to-end leg passes): same bits as a device buffer."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 30 + 9)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    dev_out = cache.decode(q, gamma)
    host_out = torch.empty(w.batch, w.n_q_heads, w.head_dim, dtype=torch.float32).pin_memory()
    cache.decode(q, gamma, out=host_out)
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    assert torch.equal(host_out, dev_out.cpu())


@pytest.mark.parametrize("ctx,top_k,flags", [
    (64 * 700 + 10, 16, 0),                                # cluster kernel, few candidates: ranked by counting
    (64 * 2500, 64, 0),                                    # 16 CTAs x 64 candidates, all equal: the histogram path
    (64 * 700 + 10, 16, binding.SPLA_STATS_BF16),          # tensor-core score path
    (64 * 300, 16, binding.SPLA_GENERAL_KERNELS),
])
def test_equal_scores_select_the_lowest_block_indices(ctx, top_k, flags):
    """Every block holds the same keys, so all full blocks score exactly the same: the selection is decided by the
    tie rule alone (score descending, then block index ascending) after the forced sink and local blocks."""
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=ctx, n_needles=0, top_k=top_k)
    K, V, lens = runner.generate_prefill(w, DEV)
    K = K[:, :, :w.block_size].repeat(1, 1, -(-ctx // w.block_size), 1)[:, :, :ctx].contiguous()
    cache, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens), flags=flags)
    gamma = synth.gamma(w).to(DEV)
    q = synth.step_queries(w, 0, DEV)
    out, osp, orla, sel = _decode_all(cache, w, q, gamma)
    nblk = -(-ctx // w.block_size)
    n_free = top_k - w.n_sink - w.n_local
    want = sorted(set(range(w.n_sink)) | set(range(nblk - w.n_local, nblk)) | set(range(w.n_sink, w.n_sink + n_free)))
    for h in range(w.n_kv_heads):
        assert sel[0, h].tolist() == want
    res = parity.oracle_unit(w, q[0], K[0, 0], V[0, 0], gamma, 0, n_sink=w.n_sink, n_local=w.n_local,
                             stats_bf16=bool(flags & binding.SPLA_STATS_BF16))
    assert res["sel"].tolist() == want
    parity.check_outputs("out", out[0, :w.group], res["out"], w.kv_dtype)
