/*
 * spla.h — C ABI of the SPLA decode-step attention library for NVIDIA B200 (sm_100a).
 *
 * SPLA = block Sparse Plus Linear Attention (arXiv 2601.22379).  For every
 * (sequence, KV head) "unit" one decode step
 *   1. scores every KV block with the second-order Taylor estimate of its
 *      attention mass, from the block's key mean and diagonal covariance
 *      (Section 3.1, Eq. block-score-expand, Eq. taylor-2nd), summed over the
 *      G query heads of the GQA group after per-head normalisation
 *      (Section 2.2, grouped BlockScore equation);
 *   2. selects top_k blocks: forced sink/local blocks plus the best others
 *      (Section 2.1, Eq. sparse-attn; Section 4 "Sparsity Specifications");
 *   3. runs exact softmax attention over the selected blocks only
 *      (Section 2.2, Eq. gqa-sparse);
 *   4. adds residual linear attention over the unselected blocks by
 *      subtraction: o_rla = phi(q) S_bar - phi(q) S_tilde, S_bar the global
 *      recurrent state, S_tilde rebuilt from the selected K/V already on chip
 *      (Section 3.2, Eq. rla-impl-1..3), phi = softmax over features;
 *   5. merges: out = o_sparse + RMSNorm(o_rla) (Section 3.3).
 *
 * General rules
 *   - All device buffers are owned by the caller.  The library allocates no
 *     device memory, frees none, and never synchronises the device except in
 *     spla_sync_status.  Every call enqueues its work on the given stream
 *     (a cudaStream_t passed as void*; NULL = the legacy default stream) and
 *     returns; results are ready when that stream reaches them.
 *   - Pointers marked DEVICE must be device memory of the current device,
 *     16-byte aligned (k_cache, v_cache, stats, rla_state, tok_lse and the
 *     workspace: 256-byte aligned).  Pointers marked HOST are ordinary host
 *     memory and are read before the call returns.
 *   - Every function returns SPLA_OK (0) or a negative spla_status_t.
 *     Argument errors are detected on the host before anything is launched.
 *     A condition only the device can see (a sequence that would exceed
 *     max_context, a length or block index outside the cache, a copy that
 *     did not arrive within the wait limit) skips the offending work without
 *     faulting and latches a status word that spla_sync_status reports.
 *   - Query head m belongs to KV head m / G, G = n_q_heads / n_kv_heads.
 *   - Order per decode step: spla_append_tokens(k_t, v_t) then
 *     spla_decode(q_t): the query attends to every cached token, its own
 *     position included (Section 2, problem statement), and S_bar_t includes
 *     token t (Eq. rla-impl-1).
 */
#ifndef SPLA_H_
#define SPLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SPLA_OK = 0,
  SPLA_ERR_INVALID_ARG = -1,  /* NULL pointer, bad shape, misaligned buffer, workspace too small */
  SPLA_ERR_CAPACITY = -2,     /* an append would exceed max_context (host- or device-detected) */
  SPLA_ERR_CUDA = -3,         /* a CUDA runtime call or launch failed; see spla_last_cuda_error */
  SPLA_ERR_UNSUPPORTED = -4,  /* valid request outside what the kernels are built for */
  SPLA_ERR_TIMEOUT = -5,      /* device-latched: a kernel's bounded wait for one of its own asynchronous copies ran out;
                                 the kernel skipped the arithmetic that needed the data and returned (no trap, no hang);
                                 the outputs of that call are undefined */
  SPLA_ERR_BOUNDS = -6        /* device-latched: a length in seq_lens outside [0, max_context], an invalid entry of a
                                 caller-given selection, or (SPLA_DEBUG_BOUNDS) a block index / token offset outside
                                 the cache was met; the access was skipped or the value clamped, nothing out of range
                                 was addressed */
} spla_status_t;

typedef enum { SPLA_F32 = 0, SPLA_BF16 = 1 } spla_dtype_t;

/* flags */
#define SPLA_ADOPT_CONTENTS 1u /* spla_init_cache keeps stats / rla_state / tok_lse / seq_lens as they are */
#define SPLA_FIRST_ORDER 2u    /* block score without the covariance term (Eq. taylor-1st) */
#define SPLA_NO_RLA 4u         /* out = o_sparse; the residual branch is skipped (the paper's SPA ablation) */
#define SPLA_GENERAL_KERNELS 8u /* always use the general kernels (any group size up to 16, any length, fp32 or bf16)
                                   instead of the cluster / tensor-core ones: for testing and comparison */
#define SPLA_STATS_BF16 16u    /* the block statistics are stored as bfloat16: they are computed in fp32 as always and
                                   rounded once (to nearest even) when written; the Taylor score of Section 3.1 reads
                                   the rounded values (ln n_i stays exact).  Halves the bytes the score streams; the
                                   paper does not say in which precision its block summaries are kept. */
#define SPLA_DEBUG_BOUNDS 32u  /* checked mode (a stand-in for a memory checker): every kernel verifies the block index,
                                   record range or token offset of each access it derives itself before making it;
                                   a violation skips the access and latches SPLA_ERR_BOUNDS.  Same results otherwise.
                                   Checks on caller-provided data (seq_lens, sel_in, n_new) are always on. */

typedef struct {
  int32_t batch;          /* sequences per call, >= 1 */
  int32_t n_q_heads;      /* H_q */
  int32_t n_kv_heads;     /* H_kv; G = H_q / H_kv must be an integer in [1, 16] */
  int32_t head_dim;       /* d: 64 or 128 */
  int32_t block_size;     /* B: 16, 32, 64 or 128 tokens */
  int32_t top_k;          /* k: blocks read per unit per step, 1..64 */
  int32_t max_context;    /* capacity in tokens per sequence; ceil(max_context / B) <= 32768 */
  int32_t n_sink_blocks;  /* always-selected initial blocks (paper: 1) */
  int32_t n_local_blocks; /* always-selected most recent blocks (paper: 4); n_sink + n_local <= top_k */
  int32_t kv_dtype;       /* spla_dtype_t of k_cache, v_cache, k_new, v_new */
  int32_t q_dtype;        /* spla_dtype_t of q */
  float sm_scale;         /* multiplies q in the block score and in exact attention; 0 -> 1/sqrt(d) */
  float phi_scale;        /* multiplies q and k inside the feature map phi = softmax; 0 -> 1 */
  float rms_eps;          /* epsilon of the RMSNorm; 0 -> 1e-6 */
  uint32_t flags;
  int32_t window_size;    /* C: strided selection windows (Section 3.1, "Strided Block Selection"); 0 = whole blocks */
  int32_t window_stride;  /* s: distance between window starts; 0 with window_size 0.  The paper uses C = 32, s = 16.
                             Windows are the ones lying entirely inside a block: starts 0, s, 2s, ... while
                             start + C <= B; at most 8 per block.  A block's log mass is the maximum over its
                             windows, and the per-head normalisation over blocks comes after that pooling. */
} spla_config_t;

/* Device buffers of one cache, all caller-owned.  max_blocks = ceil(max_context / B). */
typedef struct {
  void *k_cache;      /* DEVICE [batch][H_kv][max_blocks][B][d] kv_dtype; token t of a unit lives in block t / B */
  void *v_cache;      /* DEVICE same layout */
  void *stats;        /* DEVICE [batch][H_kv][max_blocks][NW][2][d] fp32 (bfloat16 with SPLA_STATS_BF16): key mean, then
                         population variance, of each of the NW selection windows of a block (NW = 1: the whole block) */
  float *rla_state;   /* DEVICE [batch][H_kv][d][d] fp32 S_bar: row = feature of phi(k), column = value dim */
  float *tok_lse;     /* DEVICE [batch][H_kv][max_blocks * B] fp32: logsumexp_c(phi_scale * k_t[c]) per token */
  int32_t *seq_lens;  /* DEVICE [batch]: tokens cached per sequence */
  void *workspace;    /* DEVICE scratch of at least spla_sizes_t.workspace bytes; contents are the library's */
  size_t workspace_bytes;
} spla_buffers_t;

typedef struct {
  size_t k_cache, v_cache, stats, rla_state, tok_lse, seq_lens, workspace; /* bytes */
} spla_sizes_t;

typedef struct spla_cache spla_cache_t; /* opaque host-side descriptor */

/* Byte size of every buffer for a configuration.  HOST pointers.  Validates the configuration. */
int spla_query_sizes(const spla_config_t *config, spla_sizes_t *sizes_out);

/*
 * Bind caller-owned buffers to a descriptor: the KV cache k_{1:N}, v_{1:N} of Section 2, kept for all later
 * queries, together with the block statistics of Section 3.1 and the recurrent state of Eq. rla-impl-1.  Unless SPLA_ADOPT_CONTENTS is set, stats, rla_state, tok_lse,
 * seq_lens are zeroed on `stream`; the workspace is always initialised.  K/V contents are never cleared.
 * config, buffers: HOST, copied.  *cache_out: HOST, receives a descriptor to release with spla_destroy_cache.
 */
int spla_init_cache(const spla_config_t *config, const spla_buffers_t *buffers, void *stream, spla_cache_t **cache_out);

/*
 * Append tokens to every sequence (the cache growth of Section 2 plus the state update of Eq. rla-impl-1 and
 * the statistics of Eq. taylor-2nd).  For sequence b the first n_new[b] of the max_new provided tokens are
 * stored at positions seq_lens[b]..; the mean and population variance of every touched block are recomputed
 * from the cached keys; S_bar += phi(k_t)^T v_t for each new token in fp32; tok_lse is filled; seq_lens[b]
 * grows by n_new[b].
 *   k_new, v_new: DEVICE [batch][H_kv][max_new][d] kv_dtype.
 *   n_new: DEVICE int32 [batch], each in [0, max_new]; NULL means max_new for every sequence.
 *   max_new >= 1.  Returns SPLA_ERR_CAPACITY (nothing enqueued) if the host-side bound on the longest
 *   sequence plus max_new exceeds max_context; a sequence that overflows on the device only is skipped and
 *   reported by spla_sync_status.
 */
int spla_append_tokens(spla_cache_t *cache, const void *k_new, const void *v_new, const int32_t *n_new,
                       int32_t max_new, void *stream);

/*
 * One decode step for every sequence: steps 1-5 of the file comment.
 *   q:          DEVICE [batch][H_q][d] q_dtype, unscaled.
 *   rms_weight: DEVICE [H_q][d] fp32 RMSNorm scale (the only parameters the method adds, Section 3.3);
 *               may be NULL with SPLA_NO_RLA.
 *   out:        DEVICE [batch][H_q][d] fp32.
 *   sel_idx:    DEVICE int32 [batch][H_kv][top_k] or NULL: selected block indices, ascending, padded with -1.
 *   dbg_o_sparse, dbg_o_rla: DEVICE fp32 [batch][H_q][d] or NULL: the exact-attention output and the
 *               residual o_bar - o_tilde before the RMSNorm.
 * A sequence of length 0 yields out = 0.  Unselected blocks' K/V are never read.
 */
int spla_decode(spla_cache_t *cache, const void *q, const float *rms_weight, float *out, int32_t *sel_idx,
                float *dbg_o_sparse, float *dbg_o_rla, void *stream);

/*
 * One whole step of the order of use the file comment gives: spla_append_tokens(k_new, v_new, n_new, max_new)
 * followed by spla_decode(q, ...), with the same arguments, the same results and the same error behaviour.  Made as
 * one call, the library knows that the score kernel follows this step's append directly, and lets it stream the
 * statistics of the blocks that were already complete while the append is still running.  q (like k_new, v_new)
 * must be ready in stream order when the call is made.
 */
int spla_append_decode(spla_cache_t *cache, const void *k_new, const void *v_new, const int32_t *n_new, int32_t max_new,
                       const void *q, const float *rms_weight, float *out, int32_t *sel_idx, float *dbg_o_sparse,
                       float *dbg_o_rla, void *stream);

/*
 * Steps 1-2 of spla_decode only: scores the blocks (Section 3.1, Eq. taylor-2nd; Section 2.2, grouped BlockScore)
 * and selects top_k of them (Section 2.1, Select).  sel_idx: DEVICE int32 [batch][H_kv][top_k], ascending, padded
 * with -1.  The scores stay available to spla_copy_scores.  Together with spla_decode_selected this splits a
 * decode step in two, e.g. to reuse one selection for several queries.
 */
int spla_select(spla_cache_t *cache, const void *q, int32_t *sel_idx, void *stream);

/*
 * Same as spla_decode with the selection given instead of computed (steps 3-5 only): sel_in DEVICE int32
 * [batch][H_kv][top_k], valid block indices padded with -1 at the tail.  For testing against an oracle when a
 * tie makes several index sets correct, and for callers that select elsewhere.  The list is checked on the device:
 * an entry that is negative before the tail, not below ceil(seq_len / B), or repeated is dropped (the remaining
 * entries are attended to) and SPLA_ERR_BOUNDS is latched for spla_sync_status; nothing outside the cache is read.
 */
int spla_decode_selected(spla_cache_t *cache, const void *q, const float *rms_weight, const int32_t *sel_in,
                         float *out, float *dbg_o_sparse, float *dbg_o_rla, void *stream);

/*
 * Prefill- / training-shaped forward.  The paper develops the method on the decode step and says that it carries over
 * to training and prefilling (Section 2, opening paragraph; Section 3.3 "Kernel Design": its kernels serve both).  The
 * reading taken here is the causal one: T new tokens per sequence are appended, and the output of each of the T query
 * positions is what spla_append_decode would give if the tokens were appended one at a time - position i sees tokens
 * 0 .. L + i, with the block statistics (its own block as far as it is filled), the selection and the recurrent
 * state S_bar of that prefix.  Afterwards the cache is as after spla_append_tokens(k_new, v_new, NULL, T).
 *   k_new, v_new: DEVICE [batch][H_kv][T][d] kv_dtype (every sequence takes all T tokens).
 *   q:            DEVICE [batch][T][H_q][d] q_dtype, unscaled.
 *   rms_weight:   DEVICE [H_q][d] fp32 (may be NULL with SPLA_NO_RLA).
 *   out:          DEVICE [batch][T][H_q][d] fp32.
 *   sel_idx:      DEVICE int32 [batch][T][H_kv][top_k] or NULL: the blocks each position selected.
 *   workspace:    DEVICE scratch, 256-byte aligned, of at least the `min_bytes` that spla_query_prefill_workspace
 *                 reports for this T; with more (up to `good_bytes`) more positions are processed per kernel launch.
 * Built on the general kernels (any group size up to 16, fp32 or bf16, d 64 or 128); strided selection windows are not
 * supported (SPLA_ERR_UNSUPPORTED).  Returns SPLA_ERR_CAPACITY, with nothing enqueued, if the chunk does not fit.
 */
int spla_prefill(spla_cache_t *cache, const void *k_new, const void *v_new, const void *q, int32_t T,
                 const float *rms_weight, float *out, int32_t *sel_idx, void *workspace, size_t workspace_bytes,
                 void *stream);

/* Workspace of spla_prefill for chunks of T tokens: the least it runs with, and a size that lets it work efficiently.
 * HOST pointers; either may be NULL. */
int spla_query_prefill_workspace(const spla_config_t *config, int32_t T, size_t *min_bytes, size_t *good_bytes);

/* Block scores of the last spla_decode: DEVICE fp32 [batch][H_kv][max_blocks] copy-out (entries >= nblk are 0). */
int spla_copy_scores(spla_cache_t *cache, float *scores_out, void *stream);

/*
 * Waits for `stream`, then returns and clears the device-latched status: SPLA_OK, or the code of the last condition
 * a kernel latched since the previous call: SPLA_ERR_CAPACITY (an append skipped a sequence that would overflow),
 * SPLA_ERR_BOUNDS (a length, selection entry or index outside the cache was clamped or skipped), SPLA_ERR_TIMEOUT (a
 * bounded wait inside a kernel ran out).  SPLA_ERR_CUDA if the copy or the synchronisation itself fails.
 */
int spla_sync_status(spla_cache_t *cache, void *stream);

/*
 * Block scoring + top-k selection (steps 1-2 of spla_decode) for callers that cannot allocate device memory.
 * The paper has no counterpart to this call; it exists for deployment reasons only.  Some code that wants a
 * selection has no way to provide the workspace the regular path needs: it runs inside a memory pool that was
 * sized and frozen up front, or it is a plug-in that receives tensors but no allocator, or it sits in a loop where
 * cudaMalloc (which synchronises the device) is off limits.  This variant therefore takes only inputs and
 * outputs and keeps the kernel's scratch in a fixed array inside the library's device image.
 *   config:     HOST; batch, heads, head_dim, block_size, top_k, max_context, sink/local counts, q_dtype,
 *               sm_scale and SPLA_FIRST_ORDER are used.  The scratch needed, about
 *               batch * H_kv * max_blocks * (G + 1) * 4 bytes, must fit SPLA_NOALLOC_SCRATCH_BYTES, otherwise
 *               SPLA_ERR_UNSUPPORTED is returned and nothing is launched.  window_size must be 0 (whole-block
 *               statistics) and SPLA_STATS_BF16 unset (fp32 records), otherwise SPLA_ERR_UNSUPPORTED.
 *   stats:      DEVICE fp32 [batch][H_kv][max_blocks][2][d], as maintained by spla_append_tokens.
 *   seq_lens:   DEVICE int32 [batch].
 *   q:          DEVICE [batch][H_q][d] q_dtype.
 *   sel_idx:    DEVICE int32 [batch][H_kv][top_k] output, ascending, padded with -1.
 *   scores_out: DEVICE fp32 [batch][H_kv][max_blocks] output or NULL (entries past the last block are 0).
 *   status_out: DEVICE int32 [1] output or NULL: 0, or SPLA_ERR_BOUNDS if a length in seq_lens lay outside
 *               [0, max_context] (it was clamped; the caller owns that buffer, so a stale one is easy to pass).
 * The call allocates nothing: no cudaMalloc / cudaFree and no allocating library routine.  Every GPU that loads
 * the library carries the SPLA_NOALLOC_SCRATCH_BYTES array until the process exits.  The first call on each
 * device looks up the array's device address (with that device current); make that first call outside any
 * stream capture.  All calls share the one array, which still holds the previous call's contents (what must
 * start at zero is cleared on `stream` first): two of these calls that overlap on the GPU - different streams,
 * or different threads - race on it and give wrong selections.  Issue them on one stream, or order them yourself.
 */
#define SPLA_NOALLOC_SCRATCH_BYTES (4u << 20)
int spla_select_blocks_noalloc(const spla_config_t *config, const float *stats, const int32_t *seq_lens,
                               const void *q, int32_t *sel_idx, float *scores_out, int32_t *status_out, void *stream);

/*
 * Test hook for the failure path of the kernels' bounded waits (no counterpart in the paper).  Every wait of a decode
 * kernel on one of its asynchronous copies polls a barrier a bounded number of times (2^22 by default) and, when the
 * limit is reached, latches SPLA_ERR_TIMEOUT, skips the arithmetic and returns normally.  This call sets that limit
 * for the decode kernels of `cache` (max_wait_polls > 0; 0 restores the default) and makes their copy barriers expect
 * extra_expected_bytes more than will ever arrive (>= 0, a multiple of 16; 0 in normal use), so that a test can watch a
 * wait run out without any fault, trap or endless loop on the device.  HOST values; affects later calls only.
 */
int spla_debug_wait_hook(spla_cache_t *cache, int32_t max_wait_polls, int32_t extra_expected_bytes);

/* Tells the library an upper bound of the current sequence lengths after adopting contents (HOST value). */
int spla_set_length_bound(spla_cache_t *cache, int32_t max_seq_len);

/* Releases the descriptor only; caller buffers are untouched.  NULL is allowed. */
int spla_destroy_cache(spla_cache_t *cache);

/* Static, NUL-terminated description of a status code. */
const char *spla_status_string(int status);

/* Text of the last CUDA error this library saw on the calling thread ("" if none). */
const char *spla_last_cuda_error(void);

/* Number of kernels this library has launched (or recorded into a stream capture) from the calling thread so far. */
unsigned long long spla_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* SPLA_H_ */
