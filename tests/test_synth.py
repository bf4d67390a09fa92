"""The synthetic workloads: shapes, determinism, structure, and (via the oracle) that needles are retrievable."""
import numpy as np
import torch

from oracle import spla_oracle as O
from paper_2601_22379_b200 import synth


def test_five_configurations_match_the_benchmark_table():
    w = synth.CONFIGS
    assert [c.name for c in w] == ["tiny_ref", "gqa_32k", "long_128k", "very_long_1m", "ragged_serving"]
    assert (w[0].head_dim, w[0].context, w[0].block_size, w[0].top_k, w[0].kv_dtype) == (64, 4096, 64, 8, "f32")
    assert (w[2].batch, w[2].group, w[2].context // w[2].block_size, w[2].top_k, w[2].n_steps) == (4, 4, 2048, 32, 64)
    assert (w[3].context // w[3].block_size, w[3].block_size) == (8192, 128)
    lens = synth.seq_lens(w[4])
    assert lens.shape == (64,) and lens.min() >= 4096 and lens.max() <= 65536 and len(set(lens.tolist())) > 32
    by = synth.algorithmic_bytes_per_step(w[2])
    assert by["stats"] == 32 * 2048 * 1024 and by["selected_kv"] == 32 * 32 * 64 * 128 * 4 and by["state"] == 32 * 65536


def test_generation_is_deterministic_and_typed():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=2, context=1024)
    K1, V1 = synth.prefill_kv(w, 1)
    K2, V2 = synth.prefill_kv(w, 1)
    assert K1.dtype == torch.bfloat16 and K1.shape == (8, 1024, 128)
    assert torch.equal(K1, K2) and torch.equal(V1, V2)
    K0, _ = synth.prefill_kv(w, 0)
    assert not torch.equal(K0, K1)
    q = synth.step_queries(w, 0)
    assert q.shape == (2, 32, 128) and q.dtype == torch.bfloat16
    assert not torch.equal(q, synth.step_queries(w, 1))
    k, v = synth.step_kv(w, 3)
    assert k.shape == (2, 8, 1, 128)


def test_outlier_channels_and_drift():
    w = synth.BY_NAME["gqa_32k"].scaled(batch=1, context=4096, n_needles=0)
    K, _ = synth.prefill_kv(w, 0)
    ch = synth.outlier_channels(w)
    std = K.float().std(dim=1)
    for h in range(w.n_kv_heads):
        mask = np.zeros(128, bool)
        mask[ch[h]] = True
        assert np.all(std[h].numpy()[mask] > 6) and np.all(std[h].numpy()[~mask] < 1.3)
    w4 = synth.BY_NAME["very_long_1m"].scaled(context=128 * 256, n_needles=0)
    K4, _ = synth.prefill_kv(w4, 0)
    means = K4.float().reshape(8, 256, 128, 128).mean(dim=2)
    walk = (means[:, -1] - means[:, 0]).std()
    assert 0.4 < walk < 1.3                      # 0.05 * sqrt(255) = 0.8


def test_p10_planted_needles_are_selected_by_the_oracle():
    for name, ctx in (("tiny_ref", 4096), ("gqa_32k", 8192)):
        w = synth.BY_NAME[name].scaled(batch=1, context=ctx)
        K, V = synth.prefill_kv(w, 0)
        q = synth.step_queries(w, 0).double().numpy()
        g = synth.gamma(w).double().numpy()
        nb = synth.needle_blocks(w)
        G = w.group
        for h in range(min(w.n_kv_heads, 3)):
            r = O.decode_unit(q[0, h * G:(h + 1) * G], K[h].double().numpy(), V[h].double().numpy(), g[h * G:(h + 1) * G],
                              block_size=w.block_size, top_k=w.top_k, n_sink=w.n_sink, n_local=w.n_local)
            assert set(nb[0, h].tolist()) <= set(r["sel"].tolist()), (name, h)


def test_benchmark_configurations_use_the_papers_sparsity_specifications():
    """Golden: the hyper-parameters the paper states (tests/golden/sparsity_specifications.txt)."""
    import pathlib
    from oracle import spla_oracle as O
    spec = {}
    for line in (pathlib.Path(__file__).parent / "golden" / "sparsity_specifications.txt").read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            k, v = line.split("=")
            spec[k.strip()] = int(v)
    long_128k, very_long = synth.BY_NAME["long_128k"], synth.BY_NAME["very_long_1m"]
    assert long_128k.top_k == very_long.top_k == spec["top_k"]
    assert long_128k.block_size == spec["block_size_gpu"] and very_long.block_size == spec["block_size_tpu"]
    for w in synth.CONFIGS:
        assert (w.n_sink, w.n_local) == (spec["n_sink_blocks"], spec["n_local_blocks"])
    C, s = spec["window_size"], spec["window_stride"]
    assert O.window_starts(spec["block_size_gpu"], C, s) == [0, 16, 32]
    assert O.window_starts(spec["block_size_tpu"], C, s) == [0, 16, 32, 48, 64, 80, 96]
