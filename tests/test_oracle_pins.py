"""Pins of the float64 oracle to what the paper and the mathematics fix.

Each test compares the oracle with something that is NOT the oracle: a brute
force sum, an explicit token-by-token recurrence, a library routine, a closed
form or an invariant.  A plausible slip anywhere in the oracle (dropped 1/2,
1/(n-1) variance, transposed state, wrong normaliser, missing partial-block
weight ...) fails at least one of them.
"""
import itertools
import zlib

import numpy as np
import pytest
import scipy.special
import torch

from oracle import spla_oracle as O

RNG = np.random.default_rng(22379)


@pytest.fixture(autouse=True)
def _reseed(request):
    """Every test draws from its own stream, so results do not depend on which tests ran before."""
    global RNG
    RNG = np.random.default_rng(zlib.crc32(request.node.name.encode()))


# ---------------------------------------------------------------------------
# P1  Taylor order (Section 3.1, Eq. taylor-2nd / taylor-1st) vs brute-force block mass
# ---------------------------------------------------------------------------
def _brute_mass(q, keys):
    return float(np.sum(np.exp(keys @ q)))


def _taylor_errors(q, kbar, delta, eps_list, order, mode):
    errs = []
    for eps in eps_list:
        keys = kbar + eps * delta
        B = keys.shape[0]
        mean, var, n = O.block_statistics(keys, B)
        cov = O.block_covariance_full(keys, B) if mode == "full" else None
        ell = O.taylor_log_mass(q, mean, var, n, order=order, full_cov=cov)
        errs.append(abs(np.exp(ell[0]) - _brute_mass(q, keys)) / _brute_mass(q, keys))
    return np.array(errs)


def _ratios(errs):
    return errs[:-1] / errs[1:]


def test_p1_full_covariance_second_order_error_is_cubic():
    d, B = 6, 12
    q, kbar = RNG.standard_normal(d), RNG.standard_normal(d)
    delta = RNG.standard_normal((B, d))
    delta -= delta.mean(axis=0)
    r = _ratios(_taylor_errors(q, kbar, delta, [0.2, 0.1, 0.05, 0.025, 0.0125], 2, "full"))
    assert np.all(r > 6.5) and np.all(r < 10.5), r       # O(eps^3): halving divides the error by 8


def test_p1_first_order_error_is_quadratic():
    d, B = 6, 12
    q, kbar = RNG.standard_normal(d), RNG.standard_normal(d)
    delta = RNG.standard_normal((B, d))
    delta -= delta.mean(axis=0)
    r = _ratios(_taylor_errors(q, kbar, delta, [0.1, 0.05, 0.025, 0.0125], 1, "full"))
    assert np.all(r > 3.5) and np.all(r < 4.6), r


def _axis_aligned_deviations(d, pattern):
    """Deviations whose empirical covariance is exactly diagonal: a disjoint token group per
    coordinate, each token moving along its group's coordinate only, each group summing to 0."""
    rows = []
    for c in range(d):
        for a in pattern:
            v = np.zeros(d)
            v[c] = a * (1.0 + 0.3 * c)
            rows.append(v)
    return np.array(rows)


@pytest.mark.parametrize("pattern,lo,hi", [((1.0, -1.0), 13.0, 19.0),          # symmetric: O(eps^4)
                                           ((2.0, -1.0, -1.0), 6.5, 10.5)])    # skewed: O(eps^3)
def test_p1_diagonal_mode_exact_order_when_covariance_is_diagonal(pattern, lo, hi):
    d = 5
    q, kbar = RNG.standard_normal(d), RNG.standard_normal(d)
    delta = _axis_aligned_deviations(d, pattern)
    cov = O.block_covariance_full(kbar + 0.1 * delta, delta.shape[0])[0]
    assert np.abs(cov - np.diag(np.diag(cov))).max() < 1e-15
    r = _ratios(_taylor_errors(q, kbar, delta, [0.2, 0.1, 0.05, 0.025], 2, "diag"))
    assert np.all(r > lo) and np.all(r < hi), r


def test_p1_diagonal_approximation_differs_from_full_at_second_order():
    d, B = 6, 12
    q, kbar = RNG.standard_normal(d), RNG.standard_normal(d)
    delta = RNG.standard_normal((B, d))
    delta -= delta.mean(axis=0)
    r = _ratios(_taylor_errors(q, kbar, delta, [0.04, 0.02, 0.01, 0.005], 2, "diag"))
    assert np.all(r > 3.3) and np.all(r < 4.7), r        # the diagonal shortcut is an approximation


def test_p1_sample_variance_would_fail():
    """The population (1/n) variance is what makes the estimate third-order accurate."""
    d = 4
    q, kbar = RNG.standard_normal(d), RNG.standard_normal(d)
    delta = _axis_aligned_deviations(d, (2.0, -1.0, -1.0))
    n = delta.shape[0]
    errs = []
    for eps in [0.1, 0.05, 0.025]:
        keys = kbar + eps * delta
        mean, var, cnt = O.block_statistics(keys, n)
        wrong = O.taylor_log_mass(q, mean, var * n / (n - 1), cnt)
        errs.append(abs(np.exp(wrong[0]) - _brute_mass(q, keys)))
    r = _ratios(np.array(errs))
    assert np.all(r < 4.6), r


# ---------------------------------------------------------------------------
# P5  zero variance => the Taylor mass is the exact mass, partial last block included
# ---------------------------------------------------------------------------
def test_p5_zero_variance_blocks_are_exact():
    d, B, L = 8, 16, 16 * 5 + 7
    nblk = -(-L // B)
    centers = RNG.standard_normal((nblk, d))
    K = np.repeat(centers, B, axis=0)[:L]
    q = RNG.standard_normal(d) * 0.7
    mean, var, n = O.block_statistics(K, B)
    assert np.all(var < 1e-28) and n[-1] == 7
    for order in (1, 2):
        ell = O.taylor_log_mass(q, mean, var, n, order=order)
        exact = np.array([np.sum(np.exp(K[i * B:i * B + n[i]] @ q)) for i in range(nblk)])
        np.testing.assert_allclose(np.exp(ell), exact, rtol=1e-12)


# ---------------------------------------------------------------------------
# P6  Gaussian keys: Taylor2 / closed form = (1 + x) / e^x with x = 1/2 sum q^2 sigma^2
# ---------------------------------------------------------------------------
def test_p6_gaussian_closed_form_ratio():
    d, B = 16, 200_000
    rng = np.random.default_rng(6)
    mu, sig = rng.standard_normal(d), 0.5 + rng.random(d)
    q = rng.standard_normal(d) * 0.25
    K = mu + sig * rng.standard_normal((B, d))
    mean, var, n = O.block_statistics(K, B)
    ell2 = O.taylor_log_mass(q, mean, var, n, order=2)[0] - np.log(B)
    x = 0.5 * np.sum(q * q * sig * sig)
    closed = q @ mu + x
    assert abs((ell2 - closed) - (np.log1p(x) - x)) < 0.03
    brute = np.log(np.mean(np.exp(K @ q)))
    assert abs(brute - closed) < 0.03


# ---------------------------------------------------------------------------
# P4  normalisation of the grouped BlockScore
# ---------------------------------------------------------------------------
def test_p4_block_probabilities_sum_to_one_and_scores_to_G():
    d, B, L, G = 16, 8, 8 * 37 + 3, 4
    K = RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d)) * 0.4
    mean, var, n = O.block_statistics(K, B)
    ell, p, score = O.block_scores(q, mean, var, n)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, atol=1e-14)
    np.testing.assert_allclose(score.sum(), G, atol=1e-13)
    assert np.all(score > 0) and np.all(score <= G)
    # G = 1: ranking by score is ranking by the log mass
    ell1, _, score1 = O.block_scores(q[:1], mean, var, n)
    assert np.array_equal(np.argsort(-score1, kind="stable"), np.argsort(-ell1[0], kind="stable"))
    # and p is the textbook softmax of ell
    np.testing.assert_allclose(p, scipy.special.softmax(ell, axis=1), atol=1e-15)


def test_block_score_matches_exact_mass_share_for_tight_blocks():
    """With nearly constant blocks the normalised score is the exact attention mass share (Eq. block-score-expand)."""
    d, B, nblk = 8, 16, 10
    centers = RNG.standard_normal((nblk, d))
    K = np.repeat(centers, B, axis=0) + 1e-4 * RNG.standard_normal((nblk * B, d))
    q = RNG.standard_normal((1, d))
    mean, var, n = O.block_statistics(K, B)
    _, p, _ = O.block_scores(q, mean, var, n)
    w = np.exp(K @ q[0])
    share = w.reshape(nblk, B).sum(axis=1) / w.sum()
    np.testing.assert_allclose(p[0], share, rtol=1e-7)   # what remains: off-diagonal covariance, O(eps^2)


# ---------------------------------------------------------------------------
# Select: forced blocks + top-k, against brute force over all subsets
# ---------------------------------------------------------------------------
def test_select_blocks_brute_force():
    rng = np.random.default_rng(3)
    for trial in range(40):
        nblk = int(rng.integers(1, 10))
        k = int(rng.integers(1, 7))
        n_sink = int(rng.integers(0, 2))
        n_local = int(rng.integers(0, 3))
        if n_sink + n_local > k:
            continue
        score = np.round(rng.random(nblk), 1)            # coarse values => ties occur
        sel = O.select_blocks(score, k, n_sink, n_local)
        chosen = [int(i) for i in sel if i >= 0]
        forced = set(range(min(n_sink, nblk))) | set(range(max(nblk - n_local, 0), nblk))
        k_eff = min(k, nblk)
        assert len(chosen) == k_eff and chosen == sorted(set(chosen)) and forced <= set(chosen)
        assert list(sel[k_eff:]) == [-1] * (k - k_eff)
        free = [i for i in range(nblk) if i not in forced]
        n_free = k_eff - len(forced)
        # brute force: the lexicographically best subset under (score desc, index asc)
        best = max(itertools.combinations(free, n_free),
                   key=lambda S: sorted(((score[i], -i) for i in S), reverse=True)) if n_free else ()
        assert set(chosen) - forced == set(best)


# ---------------------------------------------------------------------------
# P2  subtraction identity vs the naive recurrence with the indicator (Eq. rla-naive)
# ---------------------------------------------------------------------------
def _softmax_rows(x):
    return scipy.special.softmax(x, axis=-1)


def test_selected_tokens_against_a_hand_written_list():
    """Blocks 1 and 3 of a 14-token context in blocks of 4: block 1 holds tokens 4..7, block 3 is the partial
    last block with tokens 12 and 13; the -1 padding names nothing (Section 2.1, Eq. dense: the tokens of the
    blocks in the index set)."""
    np.testing.assert_array_equal(O.selected_tokens(np.array([1, 3, -1]), 14, 4), [4, 5, 6, 7, 12, 13])
    np.testing.assert_array_equal(O.selected_tokens(np.array([0, -1, -1]), 3, 4), [0, 1, 2])
    np.testing.assert_array_equal(O.selected_tokens(np.array([-1, -1]), 9, 4), [])
    np.testing.assert_array_equal(O.selected_tokens(np.array([0, 2]), 12, 4), [0, 1, 2, 3, 8, 9, 10, 11])


def test_p2_subtraction_equals_explicit_sum_over_unselected_blocks():
    d, B, L, G = 12, 8, 8 * 9 + 5, 3
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d))
    sel = np.array([0, 3, 4, 9, -1])                     # includes the partial last block
    toks = O.selected_tokens(sel, L, B)
    S_bar = O.rla_global_state(K, V)
    _, _, o_rla = O.rla_by_subtraction(q, S_bar, K, V, toks)
    # naive recurrence: S_t = S_{t-1} + I_t phi(k_t)^T v_t over unselected tokens, o = phi(q) S
    S = np.zeros((d, d))
    selected = set(int(t) for t in toks)
    for t in range(L):
        if t not in selected:
            S += np.outer(_softmax_rows(K[t]), V[t])
    naive = _softmax_rows(q) @ S
    np.testing.assert_allclose(o_rla, naive, rtol=1e-12, atol=1e-14)
    # a transposed state would not survive this
    assert np.abs(_softmax_rows(q) @ S.T - naive).max() > 1e-3


def test_p2_state_layout_rows_are_key_features():
    d = 5
    k, v = RNG.standard_normal((1, d)), RNG.standard_normal((1, d))
    S = O.rla_global_state(k, v)
    np.testing.assert_allclose(S, np.outer(_softmax_rows(k[0]), v[0]), rtol=1e-14)


# ---------------------------------------------------------------------------
# P3  full selection reduces to dense softmax attention, residual branch vanishes
# ---------------------------------------------------------------------------
def test_p3_full_selection_is_dense_attention():
    d, B, L, G = 16, 8, 8 * 6 + 3, 4
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d))
    gamma = 1.0 + 0.1 * RNG.standard_normal((G, d))
    r = O.decode_unit(q, K, V, gamma, block_size=B, top_k=16, n_sink=1, n_local=2)
    nblk = -(-L // B)
    assert list(r["sel"][:nblk]) == list(range(nblk)) and np.all(r["sel"][nblk:] == -1)
    dense = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None]).numpy()[0]
    np.testing.assert_allclose(r["o_sparse"], dense, rtol=1e-12, atol=1e-14)
    assert np.sqrt(np.mean(r["o_rla"] ** 2)) < 1e-12
    np.testing.assert_allclose(r["out"], dense, atol=1e-8)


def test_partial_selection_is_softmax_over_selected_tokens_only():
    d, B, L = 8, 4, 40
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((2, d))
    toks = O.selected_tokens(np.array([1, 7]), L, B)
    got = O.sparse_attention(q, K, V, toks)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(K[toks])[None], torch.from_numpy(V[toks])[None],
        scale=1.0).numpy()[0]
    np.testing.assert_allclose(got, ref, rtol=1e-12)


def test_default_scale_is_inverse_sqrt_d_and_applies_to_score_and_attention():
    d, B, L = 16, 8, 64
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((1, d))
    g = np.ones((1, d))
    a = O.decode_unit(q, K, V, g, block_size=B, top_k=3)
    b = O.decode_unit(q * 2.0, K, V, g, block_size=B, top_k=3, sm_scale=0.5 / np.sqrt(d))
    np.testing.assert_allclose(a["ell"], b["ell"], rtol=1e-13)
    np.testing.assert_allclose(a["o_sparse"], b["o_sparse"], rtol=1e-12)
    mean, var, n = O.block_statistics(K, B)
    want = np.log(n) + mean @ (q[0] / 4) + np.log1p(0.5 * var @ (q[0] / 4) ** 2)
    np.testing.assert_allclose(a["ell"][0], want, rtol=1e-13)


# ---------------------------------------------------------------------------
# P7  feature map and RMSNorm against library routines and their invariances
# ---------------------------------------------------------------------------
def test_p7_phi_and_rmsnorm_special_cases():
    x = RNG.standard_normal((7, 32)) * 3
    np.testing.assert_allclose(O.phi(x), scipy.special.softmax(x, axis=-1), rtol=1e-13)
    np.testing.assert_allclose(O.phi(x, 0.5), scipy.special.softmax(0.5 * x, axis=-1), rtol=1e-13)
    np.testing.assert_allclose(O.phi(x).sum(axis=-1), 1.0, atol=1e-14)
    np.testing.assert_allclose(O.phi(x + 11.0), O.phi(x), rtol=1e-12)
    gamma = RNG.standard_normal(32)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (32,), torch.from_numpy(gamma), eps=1e-6).numpy()
    np.testing.assert_allclose(O.rms_norm(x, gamma, 1e-6), ref, rtol=1e-13)
    np.testing.assert_allclose(O.rms_norm(5.0 * x, gamma, 0.0), O.rms_norm(x, gamma, 0.0), rtol=1e-13)


def test_merge_is_sparse_plus_rmsnorm_of_residual():
    d, B, L, G = 16, 8, 96, 2
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d))
    gamma = RNG.standard_normal((G, d))
    r = O.decode_unit(q, K, V, gamma, block_size=B, top_k=4, n_sink=1, n_local=1, rms_eps=1e-5)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(r["o_rla"]), (d,), eps=1e-5).numpy() * gamma
    np.testing.assert_allclose(r["out"], r["o_sparse"] + ref, rtol=1e-12)
    np.testing.assert_allclose(r["o_rla"], r["o_bar"] - r["o_tilde"], rtol=0, atol=0)
    off = O.decode_unit(q, K, V, gamma, block_size=B, top_k=4, n_sink=1, n_local=1, use_rla=False)
    np.testing.assert_allclose(off["out"], off["o_sparse"], rtol=0, atol=0)


# ---------------------------------------------------------------------------
# P8  symmetries
# ---------------------------------------------------------------------------
def test_p8_permutation_within_blocks_and_duplicate_heads():
    d, B, L, G = 16, 8, 8 * 12, 2
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d))
    gamma = np.ones((G, d))
    cfg = dict(block_size=B, top_k=4, n_sink=1, n_local=1)
    base = O.decode_unit(q, K, V, gamma, **cfg)
    perm = np.concatenate([i * B + RNG.permutation(B) for i in range(L // B)])
    shuf = O.decode_unit(q, K[perm], V[perm], gamma, **cfg)
    assert np.array_equal(base["sel"], shuf["sel"])
    np.testing.assert_allclose(shuf["out"], base["out"], rtol=1e-11, atol=1e-13)
    # G identical query heads select what a single head selects
    one = O.decode_unit(q[:1], K, V, gamma[:1], **cfg)
    rep = O.decode_unit(np.repeat(q[:1], 3, axis=0), K, V, np.ones((3, d)), **cfg)
    assert np.array_equal(one["sel"], rep["sel"])
    np.testing.assert_allclose(rep["out"][2], one["out"][0], rtol=1e-13)


def test_p8_batch_layout_maps_query_head_to_kv_head():
    d, B, L = 8, 4, 32
    Hq, Hkv = 4, 2
    K, V = RNG.standard_normal((1, Hkv, L, d)), RNG.standard_normal((1, Hkv, L, d))
    q = RNG.standard_normal((1, Hq, d))
    gamma = RNG.standard_normal((Hq, d))
    out, units = O.decode(q, K, V, gamma, [L], n_kv_heads=Hkv, block_size=B, top_k=3)
    for m in range(Hq):
        h = m // 2
        solo = O.decode_unit(q[0, m:m + 1], K[0, h], V[0, h], gamma[m:m + 1], block_size=B, top_k=3,
                             override_selection=units[(0, h)]["sel"])
        np.testing.assert_allclose(out[0, m], solo["out"][0], rtol=1e-13)


# ---------------------------------------------------------------------------
# P9  incremental form == definitional form
# ---------------------------------------------------------------------------
def test_p9_incremental_cache_equals_from_scratch():
    d, B, L, G = 16, 8, 8 * 7 + 5, 2
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d))
    gamma = np.ones((G, d))
    cache = O.UnitCache(d, B)
    cache.append(K[:20], V[:20])
    for t in range(20, L):
        cache.append(K[t], V[t])
    mean, var, n = O.block_statistics(K, B)
    cm, cv, cn = cache.stats()
    np.testing.assert_allclose(cm, mean, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(cv, var, rtol=1e-11, atol=1e-14)
    assert np.array_equal(cn, n) and cache.L == L
    np.testing.assert_allclose(cache.S_bar, O.rla_global_state(K, V), rtol=1e-12, atol=1e-15)
    cfg = dict(top_k=4, n_sink=1, n_local=2)
    a = cache.decode(q, gamma, **cfg)
    b = O.decode_unit(q, K, V, gamma, block_size=B, **cfg)
    assert np.array_equal(a["sel"], b["sel"])
    np.testing.assert_allclose(a["out"], b["out"], rtol=1e-10, atol=1e-12)
    pre = O.UnitCache.from_prefill(K, V, B)
    np.testing.assert_allclose(pre.decode(q, gamma, **cfg)["out"], b["out"], rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------------------
# Strided windows (Section 3.1, "Strided Block Selection"): statistics on windows of C tokens
# every s tokens, max-pooled per block
# ---------------------------------------------------------------------------
def test_window_layout_and_counts_small_table():
    # B = 8, C = 4, s = 2: windows start at 0, 2, 4 inside a block.  13 tokens = one full block and one of 5:
    # its windows [0,4), [2,6), [4,8) hold 4, 3 and 1 tokens (counted by hand).
    assert O.window_starts(8, 4, 2) == [0, 2, 4]
    assert O.window_starts(64, 32, 16) == [0, 16, 32]
    assert len(O.window_starts(128, 32, 16)) == 7
    K = RNG.standard_normal((13, 3))
    mean, var, n = O.window_statistics(K, 8, 4, 2)
    assert n.tolist() == [[4, 4, 4], [4, 3, 1]]
    np.testing.assert_allclose(mean[1, 1], K[10:13].mean(axis=0), rtol=1e-14)
    np.testing.assert_allclose(var[0, 2], K[4:8].var(axis=0), rtol=1e-13)     # numpy's population variance
    np.testing.assert_allclose(var[1, 2], 0.0, atol=0)                        # one token: no spread


def test_window_equal_to_block_reduces_to_block_mode():
    d, B, L = 8, 16, 16 * 5 + 7
    K, V = RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    q, g = RNG.standard_normal((3, d)), 0.1 * RNG.standard_normal((3, d))
    a = O.decode_unit(q, K, V, g, block_size=B, top_k=3, n_sink=1, n_local=1)
    b = O.decode_unit(q, K, V, g, block_size=B, top_k=3, n_sink=1, n_local=1, window=(B, B))
    np.testing.assert_array_equal(a["sel"], b["sel"])
    np.testing.assert_allclose(a["score"], b["score"], rtol=1e-14)
    np.testing.assert_allclose(a["out"], b["out"], rtol=1e-14)


def test_window_constant_blocks_give_exact_largest_window_mass():
    # every key of a block equal: each window's Taylor mass is exact, n_w exp(q k); the pooled value is the one
    # of the fullest window, min(C, n_i) exp(q k_i), at both orders, partial last block included
    d, B, C, s, L = 5, 16, 8, 4, 16 * 3 + 6
    centres = RNG.standard_normal((4, d))
    K = np.repeat(centres, B, axis=0)[:L]
    q = RNG.standard_normal((1, d))
    wm, wv, wn = O.window_statistics(K, B, C, s)
    for order in (1, 2):
        _, ell, p, score = O.pooled_block_scores(q, wm, wv, wn, order=order)
        exact = np.log(np.minimum(C, [16, 16, 16, 6])) + centres @ q[0]
        np.testing.assert_allclose(ell[0], exact, rtol=1e-13)
        share = np.exp(exact - scipy.special.logsumexp(exact))
        np.testing.assert_allclose(score, share, rtol=1e-12)


def test_window_first_order_pooled_mass_never_exceeds_exact_block_mass():
    # Jensen: n_w exp(q mean_w) <= sum over the window of exp(q k_t) <= the block's exact mass
    d, B, C, s, L = 6, 32, 8, 4, 32 * 6 + 11
    K = 1.5 * RNG.standard_normal((L, d))
    q = RNG.standard_normal((2, d))
    wm, wv, wn = O.window_statistics(K, B, C, s)
    ell_w, ell, _, _ = O.pooled_block_scores(q, wm, wv, wn, order=1)
    for m in range(2):
        for i in range(ell.shape[1]):
            exact = np.log(np.sum(np.exp(K[i * B:(i + 1) * B] @ q[m])))
            assert ell[m, i] <= exact + 1e-12
            assert ell[m, i] == ell_w[m, i].max()


def test_window_pooling_finds_a_needle_that_fills_half_a_block():
    # 32 of a block's 64 keys (one whole window) are shifted toward q: the window that holds exactly them sees the
    # full shift, the block mean only half of it, so pooling ranks the block first where the block mean does not
    d, B = 16, 64
    K = 0.3 * RNG.standard_normal((B * 8, d))
    V = RNG.standard_normal((B * 8, d))
    q = RNG.standard_normal((1, d))
    u = q[0] / np.linalg.norm(q[0])
    K[3 * B + 16:3 * B + 48] += 2.0 * u          # half-block needle in block 3, window [16, 48)
    K[5 * B:6 * B] += 1.3 * u                    # whole-block decoy in block 5
    g = np.ones((1, d))
    blk = O.decode_unit(q, K, V, g, block_size=B, top_k=1, sm_scale=1.0)
    win = O.decode_unit(q, K, V, g, block_size=B, top_k=1, sm_scale=1.0, window=(32, 16))
    assert blk["sel"][0] == 5 and win["sel"][0] == 3
    assert int(np.argmax(win["ell_w"][0, 3])) == 1


def test_window_scores_normalise_and_incremental_equals_definitional():
    d, B, C, s = 8, 32, 16, 8
    L0, L1 = 32 * 3 + 5, 32 * 5 + 19
    K, V = RNG.standard_normal((L1, d)), RNG.standard_normal((L1, d))
    q, g = RNG.standard_normal((4, d)), 0.1 * RNG.standard_normal((4, d))
    ref = O.decode_unit(q, K, V, g, block_size=B, top_k=3, n_sink=1, n_local=1, window=(C, s))
    np.testing.assert_allclose(ref["p"].sum(axis=1), 1.0, rtol=1e-14)
    np.testing.assert_allclose(ref["score"].sum(), 4.0, rtol=1e-13)
    c = O.UnitCache.from_prefill(K[:L0], V[:L0], B, window=(C, s))
    for t in range(L0, L1):
        c.append(K[t], V[t])
    inc = c.decode(q, g, top_k=3, n_sink=1, n_local=1)
    np.testing.assert_array_equal(inc["n"], ref["n"])
    np.testing.assert_allclose(inc["mean"], ref["mean"], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(inc["var"], ref["var"], rtol=1e-10, atol=1e-13)
    np.testing.assert_allclose(inc["out"], ref["out"], rtol=1e-10, atol=1e-12)
    # tokens permuted inside one stride segment leave every window untouched
    Kp = K.copy()
    Kp[8:16] = K[8:16][::-1]
    wm, wv, _ = O.window_statistics(Kp, B, C, s)
    np.testing.assert_allclose(wm, ref["mean"], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(wv, ref["var"], rtol=1e-11, atol=1e-14)


# ---------------------------------------------------------------------------
# Q  16-bit statistics (a reading: the paper leaves the precision of the block summaries open)
# ---------------------------------------------------------------------------
def test_bf16_rounding_matches_the_library_cast_and_ties_go_to_even():
    x = np.concatenate([RNG.standard_normal(20000) * np.exp(RNG.uniform(-20, 20, 20000)), [0.0, -0.0, 1.0, -1.0, 3.0e38]])
    want = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), want)
    # bfloat16 has 8 significant bits: the spacing in [1, 2) is 2^-7, so 1 + 2^-8 is a tie
    u = 2.0 ** -7
    assert O.round_bf16(1 + u / 2) == 1.0                 # tie -> even mantissa (1.0)
    assert O.round_bf16(1 + 3 * u / 2) == 1 + 2 * u       # tie -> even mantissa (1 + 2u)
    assert O.round_bf16(1 + u / 2 + 1e-6) == 1 + u        # just above the tie (by more than a float32 step)
    assert O.round_bf16(-(1 + 3 * u / 2)) == -(1 + 2 * u)
    assert np.max(np.abs(O.round_bf16(x[:20000]) - x[:20000]) / np.abs(x[:20000])) <= 2.0 ** -8 * (1 + 1e-6)


def test_bf16_statistics_change_the_log_mass_by_at_most_the_rounding_bound():
    """|ell_16 - ell| <= 2^-8 (sum_c |q_c||mean_c| + 1/2 sum_c q_c^2 var_c): every statistic moves by at most half a
    unit in the last place, i.e. 2^-8 relative (8 significant bits), and log(1 + x) is 1-Lipschitz for x >= 0."""
    d, B, G, L = 32, 16, 4, 16 * 37 + 5
    K = RNG.standard_normal((L, d)) * np.exp(RNG.uniform(-1, 1, d))
    V = RNG.standard_normal((L, d))
    q = RNG.standard_normal((G, d)) * 3
    gamma = np.ones((G, d))
    cfg = dict(block_size=B, top_k=6, n_sink=1, n_local=1)
    a = O.decode_unit(q, K, V, gamma, **cfg)
    b = O.decode_unit(q, K, V, gamma, stats_bf16=True, **cfg)
    q_hat = q / np.sqrt(d)
    bound = 2.0 ** -8 * (1 + 1e-6) * (np.abs(q_hat) @ np.abs(a["mean"]).T + 0.5 * (q_hat ** 2) @ a["var"].T)
    diff = np.abs(b["ell"] - a["ell"])
    assert np.all(diff <= bound + 1e-15)
    assert np.max(diff) > 1e-6                                   # and the option is not a no-op
    assert np.array_equal(b["mean"], O.round_bf16(a["mean"])) and np.array_equal(b["var"], O.round_bf16(a["var"]))
    # the rest of the path is untouched by the option: same selection -> same outputs
    c = O.decode_unit(q, K, V, gamma, stats_bf16=True, override_selection=a["sel"], **cfg)
    assert np.array_equal(c["out"], a["out"])


def test_bf16_statistics_are_exact_when_the_statistics_are_representable():
    """Blocks of identical keys with bfloat16-representable entries: mean = key, variance = 0, nothing is rounded,
    so the option must not change a single bit; same for windows."""
    d, B, G = 16, 8, 2
    nblk = 9
    base = O.round_bf16(RNG.standard_normal((nblk, d)))
    K = np.repeat(base, B, axis=0)[: nblk * B - 3]
    V = RNG.standard_normal(K.shape)
    q = RNG.standard_normal((G, d))
    gamma = np.ones((G, d))
    for window in (None, (4, 2)):
        cfg = dict(block_size=B, top_k=4, n_sink=1, n_local=1, window=window)
        a = O.decode_unit(q, K, V, gamma, **cfg)
        b = O.decode_unit(q, K, V, gamma, stats_bf16=True, **cfg)
        assert np.array_equal(a["score"], b["score"]) and np.array_equal(a["out"], b["out"])


def test_bf16_statistics_incremental_cache_equals_definitional_form():
    d, B, G = 16, 8, 2
    K = RNG.standard_normal((8 * 11 + 3, d))
    V = RNG.standard_normal(K.shape)
    q = RNG.standard_normal((G, d))
    gamma = RNG.uniform(0.5, 1.5, (G, d))
    for window in (None, (4, 4)):
        cache = O.UnitCache.from_prefill(K[:40], V[:40], B, window=window)
        cache.append(K[40:], V[40:])
        cfg = dict(top_k=5, n_sink=1, n_local=1, stats_bf16=True)
        a = cache.decode(q, gamma, **cfg)
        b = O.decode_unit(q, K, V, gamma, block_size=B, window=window, **cfg)
        assert np.array_equal(a["sel"], b["sel"])
        np.testing.assert_allclose(a["score"], b["score"], rtol=1e-2, atol=0)   # rounding may flip where Welford and two-pass differ in the last bit
        np.testing.assert_allclose(a["out"], b["out"], rtol=1e-9, atol=1e-12)


# ---------------------------------------------------------------------------
# F  prefill-shaped forward (a reading: the paper only says that the decode formulation carries over)
# ---------------------------------------------------------------------------
def test_prefill_forward_is_causal_and_ends_in_the_decode_step():
    d, B, G, L0, T = 16, 8, 2, 8 * 5 + 3, 21
    K = RNG.standard_normal((L0 + T, d))
    V = RNG.standard_normal((L0 + T, d))
    q = RNG.standard_normal((T, G, d))
    gamma = RNG.uniform(0.5, 1.5, (G, d))
    cfg = dict(block_size=B, top_k=4, n_sink=1, n_local=1)
    out, sels = O.prefill_unit(q, K, V, gamma, L0, **cfg)
    # the last position is the decode step on the whole cache
    np.testing.assert_array_equal(out[-1], O.decode_unit(q[-1], K, V, gamma, **cfg)["out"])
    # causality: what comes after position p cannot change the outputs up to p
    p = 9
    K2, V2 = K.copy(), V.copy()
    K2[L0 + p + 1:] += 5.0
    V2[L0 + p + 1:] -= 3.0
    out2, _ = O.prefill_unit(q, K2, V2, gamma, L0, **cfg)
    np.testing.assert_array_equal(out2[:p + 1], out[:p + 1])
    assert np.abs(out2[p + 1:] - out[p + 1:]).max() > 1e-3
    # every position keeps its own (partial) block and the sink block
    for i, sel in enumerate(sels):
        nblk = -(-(L0 + i + 1) // B)
        assert 0 in sel and nblk - 1 in sel and sel.max() == nblk - 1


def test_prefill_forward_with_full_selection_is_causal_dense_attention():
    d, B, G, L0, T = 16, 8, 3, 8 * 2, 13
    K = RNG.standard_normal((L0 + T, d))
    V = RNG.standard_normal((L0 + T, d))
    q = RNG.standard_normal((T, G, d))
    gamma = np.ones((G, d))
    out, _ = O.prefill_unit(q, K, V, gamma, L0, block_size=B, top_k=64)
    # library routine: causal attention of T queries placed at the end of L0 + T keys (boolean mask, float64)
    qt = torch.from_numpy(q).permute(1, 0, 2)                       # [G, T, d]
    mask = torch.arange(L0 + T)[None, :] <= (L0 + torch.arange(T))[:, None]
    want = torch.nn.functional.scaled_dot_product_attention(qt, torch.from_numpy(K)[None].expand(G, -1, -1),
                                                            torch.from_numpy(V)[None].expand(G, -1, -1), attn_mask=mask)
    np.testing.assert_allclose(out, want.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
