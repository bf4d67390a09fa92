"""Float64 CPU oracle for SPLA decode-step attention (arXiv 2601.22379).

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain restatement of what
the paper defines; it exists to check the CUDA library and to be timed as a
CPU baseline.  Nothing in the product path may import it, and it imports
nothing from the product: it shares no code, table or helper with the CUDA
kernels.  Every function is numpy float64 and follows the paper's steps in the
paper's order, without blocking, fusion or reordering.

Notation (paper, Section 2 "Notation"): block size B, GQA group size G, number
of selected blocks k, head dimension d, sequence length N (here L, the number
of cached tokens of one sequence).  One *unit* is one (sequence, KV head)
pair; its G query heads share one selected index set (Section 2.2, "Grouped
Sparsity").

Readings adopted where the paper is silent (each is listed in the design
notes of the repository):
  * the paper writes exp(q k^T) with no 1/sqrt(d); here q_hat = sm_scale * q
    is what enters the block score and the exact attention;
  * the feature map is phi(x) = softmax(phi_scale * x) over the d features
    (Section 3.2, "Numerical Stability"), applied to the *unscaled* q and k;
  * Cov(k) is the population (1/n) covariance of the keys of a block, kept
    as its diagonal (Section 3.1, after the Taylor equations);
  * a partial last block of n_i < B tokens has weight n_i instead of B;
  * BlockScore normalises per query head over all blocks, then sums over
    the G heads of the group (Section 2.2, grouped BlockScore equation);
  * the sink and local blocks the experiments force (Section 4, "Sparsity
    Specifications") count inside the top-k budget;
  * strided selection (Section 3.1, "Strided Block Selection"): windows of C
    tokens every s tokens, only those lying entirely inside one block
    (starts 0, s, 2s, ... while start + C <= B); a window of a partial last
    block counts the tokens it actually holds; a block's log mass is the
    maximum of its windows' Taylor log masses, and the per-head
    normalisation over blocks comes after this pooling;
  * ties are broken by (score descending, block index ascending);
  * training / prefilling (said only to carry over from decoding): the query
    at position t sees the cache a decode step at t would see (prefill_unit);
  * 16-bit statistics (an option; the paper does not say in which precision
    the block summaries are kept): mean and variance are computed in full
    precision, rounded once to bfloat16 (round to nearest, ties to even)
    and the Taylor score uses the rounded values; ln n_i stays exact;
  * RLA has no normaliser; RMS(.) is RMSNorm with a learnable scale gamma.

Parity unpinned: the paper prints no worked numeric example, so the *final
merged output under partial selection* and the conventions above (sm_scale,
phi_scale, epsilon, gamma's shape, tie-break, forced blocks inside the budget)
are pinned only through the composition of the identities the tests check
(Taylor order, subtraction identity, full selection = dense attention,
normalisation, zero-variance exactness, textbook softmax / RMSNorm).
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ---------------------------------------------------------------------------
# Elementary pieces
# ---------------------------------------------------------------------------
def round_bf16(x):
    """The bfloat16 value nearest to x (ties to even), returned as float64.

    bfloat16 keeps the sign, the 8 exponent bits and the upper 7 fraction bits
    of a float32: round the float32 nearest to x to a multiple of 2^16 in its
    bit pattern.  Finite inputs of normal float32 range are expected.
    """
    bits = np.asarray(x, dtype=F64).astype(np.float32).view(np.uint32).astype(np.uint64)
    keep_odd = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + keep_odd) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).astype(F64)


def phi(x, phi_scale: float = 1.0):
    """Feature map of the linear branch: softmax over the feature dimension.

    Section 3.2, "Parameterization" (phi(x) ~ exp(x)) with the normalisation
    of "Numerical Stability" (phi(x) = softmax(x)).  Works on [..., d].
    """
    z = phi_scale * np.asarray(x, dtype=F64)
    z = z - np.max(z, axis=-1, keepdims=True)
    e = np.exp(z)
    return e / np.sum(e, axis=-1, keepdims=True)


def rms_norm(x, gamma, eps: float):
    """RMS(.) of the merge equation (Section 3.3): x * gamma / sqrt(mean(x^2)+eps)."""
    x = np.asarray(x, dtype=F64)
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * np.asarray(gamma, dtype=F64) / np.sqrt(ms + eps)


def block_lengths(L: int, B: int):
    """Number of blocks and tokens per block: n_i = B except a partial last block."""
    nblk = (L + B - 1) // B
    n = np.full(nblk, B, dtype=np.int64)
    if nblk > 0 and L % B:
        n[-1] = L % B
    return nblk, n


def block_statistics(K, B: int):
    """Per-block key mean and diagonal population variance.

    These are the first- and second-order statistics the Taylor estimate uses
    (Section 3.1, Eq. taylor-2nd; diagonal approximation stated right after).
    K: [L, d].  Returns mean [nblk, d], var [nblk, d], n [nblk].
    """
    K = np.asarray(K, dtype=F64)
    L, d = K.shape
    nblk, n = block_lengths(L, B)
    mean = np.zeros((nblk, d), dtype=F64)
    var = np.zeros((nblk, d), dtype=F64)
    for i in range(nblk):
        kb = K[i * B:i * B + n[i]]
        mean[i] = kb.sum(axis=0) / n[i]
        dev = kb - mean[i]
        var[i] = (dev * dev).sum(axis=0) / n[i]
    return mean, var, n


def block_covariance_full(K, B: int):
    """Full d x d population covariance per block (test mode for the Taylor pin only)."""
    K = np.asarray(K, dtype=F64)
    L, d = K.shape
    nblk, n = block_lengths(L, B)
    cov = np.zeros((nblk, d, d), dtype=F64)
    for i in range(nblk):
        kb = K[i * B:i * B + n[i]]
        dev = kb - kb.sum(axis=0) / n[i]
        cov[i] = dev.T @ dev / n[i]
    return cov


def window_starts(B: int, C: int, s: int):
    """In-block start offsets of the strided windows that lie entirely inside a block."""
    if not (0 < C <= B and s > 0):
        raise ValueError("need 0 < C <= B and s > 0")
    return list(range(0, B - C + 1, s))


def window_statistics(K, B: int, C: int, s: int):
    """Key mean and diagonal population variance of every strided window of every block
    (Section 3.1, "Strided Block Selection": the Taylor statistics on sliding windows).

    K: [L, d].  Returns mean [nblk, NW, d], var [nblk, NW, d], n [nblk, NW]; a window of
    the partial last block holds n < C tokens, possibly none (then mean = var = 0).
    """
    K = np.asarray(K, dtype=F64)
    L, d = K.shape
    nblk, nb = block_lengths(L, B)
    starts = window_starts(B, C, s)
    NW = len(starts)
    mean = np.zeros((nblk, NW, d), dtype=F64)
    var = np.zeros((nblk, NW, d), dtype=F64)
    n = np.zeros((nblk, NW), dtype=np.int64)
    for i in range(nblk):
        for w, t0 in enumerate(starts):
            cnt = int(min(C, nb[i] - t0))
            if cnt <= 0:
                continue
            kw = K[i * B + t0:i * B + t0 + cnt]
            n[i, w] = cnt
            mean[i, w] = kw.sum(axis=0) / cnt
            dev = kw - mean[i, w]
            var[i, w] = (dev * dev).sum(axis=0) / cnt
    return mean, var, n


# ---------------------------------------------------------------------------
# Step 1: block score (Section 3.1)
# ---------------------------------------------------------------------------
def taylor_log_mass(q_hat, mean, var, n, order: int = 2, full_cov=None):
    """Log of the estimated un-normalised probability mass of every block.

    Block mass = n_i * E_j[exp(q k_j)] (Eq. block-score-expand), and the
    expectation is estimated as exp(q k_bar) (1 + 1/2 q^T Cov q) at second
    order (Eq. taylor-2nd) or exp(q k_bar) at first order (Eq. taylor-1st).
    q_hat: [d] (already scaled).  Returns ell [nblk] with
    ell_i = ln n_i + q_hat.mean_i + ln(1 + 1/2 quad_i).
    """
    q_hat = np.asarray(q_hat, dtype=F64)
    lin = np.asarray(mean, dtype=F64) @ q_hat
    ell = np.log(np.asarray(n, dtype=F64)) + lin
    if order == 2:
        if full_cov is not None:
            quad = np.einsum("c,icd,d->i", q_hat, np.asarray(full_cov, dtype=F64), q_hat)
        else:
            quad = np.asarray(var, dtype=F64) @ (q_hat * q_hat)
        ell = ell + np.log1p(0.5 * quad)
    elif order != 1:
        raise ValueError("order must be 1 or 2")
    return ell


def block_scores(q_hat_group, mean, var, n, order: int = 2):
    """GQA-aggregated BlockScore (Section 2.2, grouped BlockScore equation).

    For every query head m: p^m_i = mass^m_i / Z^m with Z^m the sum of the
    block masses (Eq. block-score-expand-z); score_i = sum_m p^m_i.
    Returns ell [G, nblk], p [G, nblk], score [nblk].
    """
    q_hat_group = np.asarray(q_hat_group, dtype=F64)
    G = q_hat_group.shape[0]
    nblk = len(n)
    ell = np.zeros((G, nblk), dtype=F64)
    p = np.zeros((G, nblk), dtype=F64)
    for m in range(G):
        ell[m] = taylor_log_mass(q_hat_group[m], mean, var, n, order=order)
        top = np.max(ell[m])
        w = np.exp(ell[m] - top)
        p[m] = w / np.sum(w)
    return ell, p, p.sum(axis=0)


def pooled_block_scores(q_hat_group, wmean, wvar, wn, order: int = 2):
    """BlockScore with strided windows: Taylor log mass per window, max-pooled over the
    windows of a block, then normalised per head over the blocks and summed over the group
    (Section 3.1, "Strided Block Selection"; Section 2.2 for the normalisation).

    wmean, wvar [nblk, NW, d], wn [nblk, NW].  Returns ell_w [G, nblk, NW] (-inf for empty
    windows), ell [G, nblk], p [G, nblk], score [nblk].
    """
    q_hat_group = np.asarray(q_hat_group, dtype=F64)
    G = q_hat_group.shape[0]
    nblk, NW = np.asarray(wn).shape
    ell_w = np.full((G, nblk, NW), -np.inf, dtype=F64)
    ell = np.zeros((G, nblk), dtype=F64)
    p = np.zeros((G, nblk), dtype=F64)
    for m in range(G):
        for w in range(NW):
            live = np.asarray(wn)[:, w] > 0
            if live.any():
                ell_w[m, live, w] = taylor_log_mass(q_hat_group[m], wmean[live, w], wvar[live, w], wn[live, w], order=order)
        ell[m] = ell_w[m].max(axis=1)
        top = np.max(ell[m])
        e = np.exp(ell[m] - top)
        p[m] = e / np.sum(e)
    return ell_w, ell, p, p.sum(axis=0)


# ---------------------------------------------------------------------------
# Step 2: Select = forced blocks + TopK (Section 2.1, Eq. sparse-attn; Section 4)
# ---------------------------------------------------------------------------
def forced_blocks(nblk: int, n_sink: int, n_local: int):
    """Initial (sink) blocks and most recent (local) blocks, clipped and de-duplicated."""
    forced = set(range(min(n_sink, nblk)))
    forced |= set(range(max(nblk - n_local, 0), nblk))
    return sorted(forced)


def select_blocks(score, top_k: int, n_sink: int = 0, n_local: int = 0):
    """Index set I: forced blocks plus the highest-scoring others, k_eff = min(k, nblk) in total.

    Returns an int64 array of length top_k: the selected block indices in
    ascending order, padded with -1.  Free blocks are ranked by (score
    descending, index ascending).
    """
    score = np.asarray(score, dtype=F64)
    nblk = score.shape[0]
    forced = forced_blocks(nblk, n_sink, n_local)
    if len(forced) > top_k:
        raise ValueError("n_sink + n_local exceeds top_k")
    k_eff = min(top_k, nblk)
    free = [i for i in range(nblk) if i not in set(forced)]
    free.sort(key=lambda i: (-score[i], i))
    chosen = sorted(forced + free[:k_eff - len(forced)])
    out = np.full(top_k, -1, dtype=np.int64)
    out[:len(chosen)] = chosen
    return out


def selected_tokens(sel, L: int, B: int):
    """Token positions covered by the selected blocks (valid tokens only)."""
    toks = []
    for i in sel:
        if i >= 0:
            toks.extend(range(int(i) * B, min((int(i) + 1) * B, L)))
    return np.asarray(toks, dtype=np.int64)


# ---------------------------------------------------------------------------
# Step 3: exact attention over the selected blocks (Eq. dense / Eq. gqa-sparse)
# ---------------------------------------------------------------------------
def sparse_attention(q_hat_group, K, V, toks):
    """o^sparse [G, d]: softmax attention restricted to the tokens `toks`, row-wise per head."""
    q_hat_group = np.asarray(q_hat_group, dtype=F64)
    Ks = np.asarray(K, dtype=F64)[toks]
    Vs = np.asarray(V, dtype=F64)[toks]
    s = q_hat_group @ Ks.T                      # [G, |T|]
    s = s - np.max(s, axis=1, keepdims=True)
    w = np.exp(s)
    w = w / np.sum(w, axis=1, keepdims=True)
    return w @ Vs


# ---------------------------------------------------------------------------
# Step 4: residual linear attention by subtraction (Section 3.2, Eq. rla-impl-1..3)
# ---------------------------------------------------------------------------
def rla_global_state(K, V, phi_scale: float = 1.0):
    """S_bar = sum_t phi(k_t)^T v_t over ALL cached tokens; [d, d], row = key feature, column = value dim."""
    return phi(K, phi_scale).T @ np.asarray(V, dtype=F64)


def rla_by_subtraction(q_group, S_bar, K, V, toks, phi_scale: float = 1.0):
    """o_bar = phi(q) S_bar, o_tilde = phi(q) S_tilde with S_tilde over the selected tokens only.

    Returns (o_bar, o_tilde, o_rla = o_bar - o_tilde), each [G, d].  phi acts
    on the raw (unscaled) q.
    """
    f = phi(q_group, phi_scale)                                  # [G, d]
    o_bar = f @ np.asarray(S_bar, dtype=F64)
    S_tilde = phi(np.asarray(K, dtype=F64)[toks], phi_scale).T @ np.asarray(V, dtype=F64)[toks]
    o_tilde = f @ S_tilde
    return o_bar, o_tilde, o_bar - o_tilde


# ---------------------------------------------------------------------------
# One unit, all steps (definitional form: everything from the raw K, V)
# ---------------------------------------------------------------------------
def decode_unit(q_group, K, V, gamma_group, *, block_size, top_k, n_sink=0, n_local=0,
                sm_scale=None, phi_scale=1.0, rms_eps=1e-6, order=2, use_rla=True,
                override_selection=None, S_bar=None, stats=None, window=None, stats_bf16=False):
    """SPLA decode output for one (sequence, KV head) unit.

    q_group [G, d] raw queries of the group, K, V [L, d] the whole cache of
    the unit (the current token included: the query at position N attends to
    all N cached tokens), gamma_group [G, d] RMSNorm scales.
    `override_selection` replaces steps 1-2 by a given index set (used when a
    correct implementation picked a different set inside the tie tolerance).
    `S_bar` / `stats` may be passed in pre-computed (incremental form).
    `window` = (C, s) switches the score to strided windows with max-pooling;
    `stats` then holds window statistics.
    `stats_bf16` rounds the means and variances to bfloat16 before the score.
    Returns a dict with every intermediate the tests compare.
    """
    q_group = np.asarray(q_group, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    L, d = K.shape
    B = block_size
    if sm_scale is None:
        sm_scale = 1.0 / np.sqrt(d)
    q_hat = sm_scale * q_group

    ell_w = None
    if window is None:
        mean, var, n = block_statistics(K, B) if stats is None else stats
    else:
        mean, var, n = window_statistics(K, B, window[0], window[1]) if stats is None else stats
    if stats_bf16:
        mean, var = round_bf16(mean), round_bf16(var)
    if window is None:
        ell, p, score = block_scores(q_hat, mean, var, n, order=order)
    else:
        ell_w, ell, p, score = pooled_block_scores(q_hat, mean, var, n, order=order)
    if override_selection is None:
        sel = select_blocks(score, top_k, n_sink, n_local)
    else:
        sel = np.full(top_k, -1, dtype=np.int64)
        ov = np.sort(np.asarray([i for i in override_selection if i >= 0], dtype=np.int64))
        sel[:len(ov)] = ov
    toks = selected_tokens(sel, L, B)

    o_sparse = sparse_attention(q_hat, K, V, toks)
    if use_rla:
        if S_bar is None:
            S_bar = rla_global_state(K, V, phi_scale)
        o_bar, o_tilde, o_rla = rla_by_subtraction(q_group, S_bar, K, V, toks, phi_scale)
        out = o_sparse + rms_norm(o_rla, gamma_group, rms_eps)
    else:
        o_bar = o_tilde = o_rla = np.zeros_like(o_sparse)
        out = o_sparse.copy()
    return dict(ell=ell, p=p, score=score, sel=sel, o_sparse=o_sparse, o_bar=o_bar,
                o_tilde=o_tilde, o_rla=o_rla, out=out, mean=mean, var=var, n=n, ell_w=ell_w)


def decode(q, K, V, gamma, seq_lens, *, n_kv_heads, **cfg):
    """Batch form: q [batch, H_q, d], K, V [batch, H_kv, Lmax, d], gamma [H_q, d], seq_lens [batch].

    Query head m uses KV head m // G.  Returns out [batch, H_q, d] and the
    per-unit result dicts keyed by (b, h).
    """
    q = np.asarray(q, dtype=F64)
    batch, Hq, d = q.shape
    G = Hq // n_kv_heads
    out = np.zeros((batch, Hq, d), dtype=F64)
    units = {}
    for b in range(batch):
        L = int(seq_lens[b])
        for h in range(n_kv_heads):
            r = decode_unit(q[b, h * G:(h + 1) * G], K[b, h, :L], V[b, h, :L],
                            np.asarray(gamma, dtype=F64)[h * G:(h + 1) * G], **cfg)
            out[b, h * G:(h + 1) * G] = r["out"]
            units[(b, h)] = r
    return out, units


def prefill_unit(q_positions, K, V, gamma_group, first_position: int, **cfg):
    """Prefill / training-shaped forward of one unit: the output at every query position of a chunk.

    The paper describes the method on the decoding workload and notes that it carries over to training and
    prefilling (Section 2, opening paragraph).  The reading taken here is the causal one: the query at absolute
    position t sees exactly the cache a decode step at that position would see, tokens 0..t, with the block
    statistics, the selection and the recurrent state of that prefix.  q_positions [T, G, d] holds the queries of
    positions first_position .. first_position + T - 1; K, V [L, d] with L >= first_position + T.
    Returns out [T, G, d] and the list of selected index arrays.  No GPU counterpart exists yet: this is the
    reference the next kernel row will be checked against.
    """
    q_positions = np.asarray(q_positions, dtype=F64)
    T = q_positions.shape[0]
    outs, sels = [], []
    for i in range(T):
        n_tok = first_position + i + 1
        r = decode_unit(q_positions[i], K[:n_tok], V[:n_tok], gamma_group, **cfg)
        outs.append(r["out"])
        sels.append(r["sel"])
    return np.stack(outs), sels


# ---------------------------------------------------------------------------
# Incremental form: what a serving cache maintains between decode steps
# ---------------------------------------------------------------------------
class UnitCache:
    """One unit's cache kept the way the method prescribes for inference.

    `append` stores k_t, v_t, updates the open block's running mean and sum of
    squared deviations, and adds phi(k_t)^T v_t to the global state (Eq.
    rla-impl-1); `decode` then touches only the block statistics, the selected
    blocks and S_bar (Section 3.3, "Kernel Design").  Must agree with the
    definitional form.
    """

    def __init__(self, d: int, block_size: int, phi_scale: float = 1.0, window=None):
        self.d, self.B, self.phi_scale = d, block_size, phi_scale
        self.window = window                      # (C, s) or None: strided windows kept beside the blocks
        self.starts = window_starts(block_size, window[0], window[1]) if window else []
        NW = len(self.starts)
        self.wmean = np.zeros((0, NW, d), dtype=F64)
        self.wm2 = np.zeros((0, NW, d), dtype=F64)
        self.wn = np.zeros((0, NW), dtype=np.int64)
        self.K = np.zeros((0, d), dtype=F64)
        self.V = np.zeros((0, d), dtype=F64)
        self.mean = np.zeros((0, d), dtype=F64)
        self.m2 = np.zeros((0, d), dtype=F64)     # sum of squared deviations per block
        self.n = np.zeros(0, dtype=np.int64)
        self.S_bar = np.zeros((d, d), dtype=F64)
        self._chunks_k, self._chunks_v = [], []

    @classmethod
    def from_prefill(cls, K, V, block_size: int, phi_scale: float = 1.0, window=None):
        """Cache holding an existing context: statistics and S_bar from their definitions."""
        K = np.asarray(K, dtype=F64)
        V = np.asarray(V, dtype=F64)
        c = cls(K.shape[1], block_size, phi_scale, window)
        c.K, c.V = K, V
        c.mean, var, c.n = block_statistics(K, block_size)
        c.m2 = var * c.n[:, None]
        if window:
            c.wmean, wvar, c.wn = window_statistics(K, block_size, window[0], window[1])
            c.wm2 = wvar * c.wn[:, :, None]
        c.S_bar = rla_global_state(K, V, phi_scale)
        return c

    @property
    def L(self):
        return int(self.n.sum())

    def append(self, k_new, v_new):
        k_new = np.atleast_2d(np.asarray(k_new, dtype=F64))
        v_new = np.atleast_2d(np.asarray(v_new, dtype=F64))
        for k_t, v_t in zip(k_new, v_new):
            if len(self.n) == 0 or self.n[-1] == self.B:
                self.mean = np.vstack([self.mean, np.zeros((1, self.d))])
                self.m2 = np.vstack([self.m2, np.zeros((1, self.d))])
                self.n = np.append(self.n, 0)
                if self.window:
                    NW = len(self.starts)
                    self.wmean = np.concatenate([self.wmean, np.zeros((1, NW, self.d))])
                    self.wm2 = np.concatenate([self.wm2, np.zeros((1, NW, self.d))])
                    self.wn = np.concatenate([self.wn, np.zeros((1, NW), dtype=np.int64)])
            t_in = int(self.n[-1])                # position of the new token inside its block
            for w, t0 in enumerate(self.starts):
                if t0 <= t_in < t0 + self.window[0]:
                    self.wn[-1, w] += 1
                    dw = k_t - self.wmean[-1, w]
                    self.wmean[-1, w] += dw / self.wn[-1, w]
                    self.wm2[-1, w] += dw * (k_t - self.wmean[-1, w])
            self.n[-1] += 1
            delta = k_t - self.mean[-1]
            self.mean[-1] += delta / self.n[-1]
            self.m2[-1] += delta * (k_t - self.mean[-1])
            self.S_bar += np.outer(phi(k_t, self.phi_scale), v_t)
        self._chunks_k.append(k_new)
        self._chunks_v.append(v_new)

    def _materialise(self):
        if self._chunks_k:
            self.K = np.vstack([self.K] + self._chunks_k)
            self.V = np.vstack([self.V] + self._chunks_v)
            self._chunks_k, self._chunks_v = [], []

    def stats(self):
        if self.window:
            return self.wmean, self.wm2 / np.maximum(self.wn, 1)[:, :, None], self.wn
        return self.mean, self.m2 / self.n[:, None], self.n

    def decode(self, q_group, gamma_group, **cfg):
        self._materialise()
        return decode_unit(q_group, self.K, self.V, gamma_group, block_size=self.B,
                           phi_scale=self.phi_scale, S_bar=self.S_bar, stats=self.stats(),
                           window=self.window, **cfg)
