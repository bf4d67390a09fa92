"""The one-call step (`spla_append_decode`: the score kernel streams the older blocks' statistics while the step's
append is still running) against the two separate calls it stands for: same cache contents, statistics, state,
selection and outputs, bit for bit; and against the float64 oracle."""
import pytest
import torch

from paper_2601_22379_b200 import binding, runner, synth
from tests import parity
from tests.test_gpu_parity import DEV, _all_units

pytestmark = pytest.mark.gpu


def _same_cache(a, b):
    for name in ("stats", "rla_state", "seq_lens"):
        assert torch.equal(getattr(a.bufs, name), getattr(b.bufs, name)), name


@pytest.mark.parametrize("name,over,window,steps", [
    ("long_128k", dict(batch=2, context=64 * 40 + 61), None, 6),            # crosses a block boundary
    ("gqa_32k", dict(batch=2, context=64 * 70 + 31, n_steps=4), None, 4),
    ("very_long_1m", dict(context=128 * 140 + 126, n_needles=4, n_steps=4), None, 4),   # B = 128, 16 CTAs per unit
    ("ragged_serving", dict(batch=6, context=6000, context_min=300, n_steps=5), None, 5),
    ("long_128k", dict(batch=1, context=64 * 30 + 63), (32, 16), 4),         # strided windows
    ("gqa_32k", dict(batch=1, context=64 * 3 + 2, n_needles=0, n_steps=3), None, 3),    # a cluster of one CTA
    ("gqa_32k", dict(batch=1, context=5, n_needles=0, n_steps=3), None, 3),             # shorter than a block
])
def test_one_call_step_equals_append_then_decode(name, over, window, steps):
    w = synth.BY_NAME[name].scaled(**over)
    a, K, V, lens = runner.build_cache(w, DEV, window=window)
    b, _, _, _ = runner.build_cache(w, DEV, window=window, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    for step in range(steps):
        k1, v1 = synth.step_kv(w, step, DEV)
        q = synth.step_queries(w, step, DEV)
        sa, sb = a.new_sel_buffer(), b.new_sel_buffer()
        a.append_tokens(k1, v1)
        oa = a.decode(q, gamma, sel_idx=sa)
        ob = b.append_decode(k1, v1, q, gamma, sel_idx=sb)
        torch.cuda.synchronize()
        assert a.sync_status() == 0 and b.sync_status() == 0
        assert torch.equal(sa, sb), step
        assert torch.equal(oa, ob), step
        _same_cache(a, b)
    ka = a.bufs.k_cache.reshape(w.batch, w.n_kv_heads, -1, w.head_dim)
    kb = b.bufs.k_cache.reshape(w.batch, w.n_kv_heads, -1, w.head_dim)
    for bi in range(w.batch):
        Lb = int(lens[bi]) + steps
        assert torch.equal(ka[bi, :, :Lb], kb[bi, :, :Lb])
        assert torch.equal(a.bufs.tok_lse[bi, :, :Lb], b.bufs.tok_lse[bi, :, :Lb])


def test_one_call_step_with_device_counts_and_several_tokens():
    """n_new on the device (some sequences add nothing), three tokens per call."""
    w = synth.BY_NAME["ragged_serving"].scaled(batch=4, context=3000, context_min=500, n_steps=4)
    a, K, V, lens = runner.build_cache(w, DEV)
    b, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    n_new = torch.tensor([3, 0, 1, 2], dtype=torch.int32, device=DEV)
    for step in range(3):
        ks = [synth.step_kv(w, 3 * step + j, DEV) for j in range(3)]
        k3 = torch.cat([k for k, _ in ks], dim=2).contiguous()
        v3 = torch.cat([v for _, v in ks], dim=2).contiguous()
        q = synth.step_queries(w, step, DEV)
        a.append_tokens(k3, v3, n_new)
        oa = a.decode(q, gamma)
        ob = b.append_decode(k3, v3, q, gamma, n_new=n_new)
        torch.cuda.synchronize()
        assert torch.equal(oa, ob)
        _same_cache(a, b)
    assert torch.equal(a.bufs.seq_lens, lens + 3 * n_new)


def test_one_call_step_in_a_replayed_graph_matches_oracle():
    """Eight steps captured once and replayed (the launch configuration the benchmark times), then the oracle."""
    w = synth.BY_NAME["long_128k"].scaled(batch=2, context=64 * 40 + 60, n_steps=8)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    kvs = [synth.step_kv(w, s, DEV) for s in range(8)]
    qs = [synth.step_queries(w, s, DEV) for s in range(8)]
    cfg = cache.cfg
    outs = [torch.empty(cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=DEV) for _ in range(8)]
    sels = [cache.new_sel_buffer() for _ in range(8)]
    osp, orla = torch.empty_like(outs[0]), torch.empty_like(outs[0])
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for s in range(8):
                cache.append_decode(*kvs[s], qs[s], gamma, out=outs[s], sel_idx=sels[s],
                                    dbg_o_sparse=osp if s == 7 else None, dbg_o_rla=orla if s == 7 else None)
        g.replay()
    torch.cuda.synchronize()
    assert cache.sync_status() == 0
    lens_h = lens.cpu().numpy()
    for (b, h) in _all_units(w):
        L = int(lens_h[b])
        Ku = torch.cat([K[b, h, :L]] + [kvs[s][0][b, h] for s in range(8)])
        Vu = torch.cat([V[b, h, :L]] + [kvs[s][1][b, h] for s in range(8)])

        def run(override=None):
            return parity.oracle_unit(w, qs[7][b], Ku, Vu, gamma, h, n_sink=w.n_sink, n_local=w.n_local, override=override)
        parity.compare_unit(w, run(), outs[7][b].cpu().numpy(), osp[b].cpu().numpy(), orla[b].cpu().numpy(),
                            sels[7][b, h].cpu().numpy(), h, n_sink=w.n_sink, n_local=w.n_local, rerun=run)


def test_one_call_step_for_fp32_caches_and_long_appends():
    w = synth.BY_NAME["tiny_ref"].scaled(batch=2, context=64 * 9 + 5, n_needles=0)       # fp32: general kernels
    a, K, V, lens = runner.build_cache(w, DEV)
    b, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    k1, v1 = synth.step_kv(w, 0, DEV)
    q = synth.step_queries(w, 0, DEV)
    a.append_tokens(k1, v1)
    assert torch.equal(a.decode(q, gamma), b.append_decode(k1, v1, q, gamma))
    _same_cache(a, b)


def test_one_call_step_capacity_is_checked_on_the_host():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=64 * 4, n_needles=0, n_steps=1)
    cache, K, V, lens = runner.build_cache(w, DEV)
    gamma = synth.gamma(w).to(DEV)
    k1, v1 = synth.step_kv(w, 0, DEV)
    q = synth.step_queries(w, 0, DEV)
    cache.append_decode(k1, v1, q, gamma)                       # fills the cache to its capacity (context + n_steps)
    with pytest.raises(binding.SplaError) as e:
        cache.append_decode(k1, v1, q, gamma)
    assert e.value.status == binding.SPLA_ERR_CAPACITY


def test_many_one_call_steps_on_one_cache_in_one_graph():
    """150 steps on the same cache captured in one graph (every score kernel starts while the append in front of it
    is running, across two block boundaries), against the same steps made as separate calls: bit for bit."""
    n = 150
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=64 * 20 + 50, n_needles=0, n_steps=n)
    a, K, V, lens = runner.build_cache(w, DEV)
    b, _, _, _ = runner.build_cache(w, DEV, prefill=(K, V, lens))
    gamma = synth.gamma(w).to(DEV)
    kvs = [synth.step_kv(w, s, DEV) for s in range(8)]
    qs = [synth.step_queries(w, s, DEV) for s in range(8)]
    cfg = a.cfg
    outs_a = torch.empty(n, cfg.batch, cfg.n_q_heads, cfg.head_dim, dtype=torch.float32, device=DEV)
    outs_b = torch.empty_like(outs_a)
    sel_a = torch.empty(n, cfg.batch, cfg.n_kv_heads, cfg.top_k, dtype=torch.int32, device=DEV)
    sel_b = torch.empty_like(sel_a)
    for s in range(n):
        a.append_tokens(*kvs[s % 8])
        a.decode(qs[s % 8], gamma, out=outs_a[s], sel_idx=sel_a[s])
    g = torch.cuda.CUDAGraph()
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        with torch.cuda.graph(g, stream=st):
            for s in range(n):
                b.append_decode(*kvs[s % 8], qs[s % 8], gamma, out=outs_b[s], sel_idx=sel_b[s])
        g.replay()
    torch.cuda.synchronize()
    assert a.sync_status() == 0 and b.sync_status() == 0
    assert torch.equal(sel_a, sel_b)
    assert torch.equal(outs_a, outs_b)
    _same_cache(a, b)
