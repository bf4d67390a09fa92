// C ABI of the library: argument validation, workspace carve-up and kernel launches.  Host code only.
#include <math.h>
#include <stdlib.h>
#include <new>
#include <stdio.h>
#include <string.h>

#include <cuda.h>

#include "../../include/spla.h"
#include "spla_internal.h"

using namespace spla;

struct spla_cache {
  spla_config_t cfg;
  spla_buffers_t buf;
  Params p;
  int64_t len_bound;   // host-side upper bound of the longest sequence
  // clusters the device holds at once, as last queried: score kernel for (cs, chunk), attend kernel per log2(acs)
  int score_occ_chunk[2][17] = {}, score_occ_n[2][17] = {};   // resident clusters as last queried, by [kernel: score / fused decode][cluster size]
  int attend_occ[5] = {-2, -2, -2, -2, -2};   // by log2 of the cluster size
  int sm_count;
  AttendMaps maps;
  AttendMaps state_maps;   // the same caches in boxes of 64 tokens, for the tensor-core state kernel
};

static thread_local char g_cuda_err[256] = "";

namespace spla {
thread_local unsigned long long g_launch_count = 0;
int cuda_fail(cudaError_t e, const char* where) {
  snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", where, cudaGetErrorString(e));
  return SPLA_ERR_CUDA;
}
int device_sm_count() {
  int dev = 0, n = 0;
  if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0)
    return n;
  return 148;
}
}  // namespace spla

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// TMA tensor map over a K or V cache seen as a 2-D bf16 matrix [batch * H_kv * max_blocks * B rows][d columns]:
// boxes of B rows x 64 columns (128 bytes, the widest the 128-byte swizzle allows).
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static TensorMapEncodeFn tensor_map_encoder() {
  static TensorMapEncodeFn encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult st;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &st) != cudaSuccess || !fn) return nullptr;
    encode = (TensorMapEncodeFn)fn;
  }
  return encode;
}

// A K or V cache as a bf16 matrix [rows][d] with boxes of B rows x 64 columns (128-byte swizzle).
static bool make_kv_map(void* out128, void* base, int d, int B, unsigned long long rows) {
  TensorMapEncodeFn encode = tensor_map_encoder();
  if (!encode) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)d * 2};
  const cuuint32_t box[2] = {64u, (cuuint32_t)B};
  const cuuint32_t estr[2] = {1u, 1u};
  return encode(reinterpret_cast<CUtensorMap*>(out128), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same cache seen as [d / 64 column halves][rows][64 columns], so that ONE copy brings a whole tile of `tile_rows`
// rows: its box is all halves x tile_rows x 64, which lands in shared memory half by half, each half [rows][128 bytes]
// with the 128-byte swizzle - the layout the attend phase reads.  (An issue costs the issuing thread about 0.1 us.)
static bool make_kv_tile_map(void* out128, void* base, int d, int tile_rows, unsigned long long rows) {
  TensorMapEncodeFn encode = tensor_map_encoder();
  if (!encode || d % 64 != 0) return false;
  const cuuint64_t dims[3] = {64u, (cuuint64_t)rows, (cuuint64_t)(d / 64)};
  const cuuint64_t strides[2] = {(cuuint64_t)d * 2, 128u};
  const cuuint32_t box[3] = {64u, (cuuint32_t)tile_rows, (cuuint32_t)(d / 64)};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return encode(reinterpret_cast<CUtensorMap*>(out128), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, base, dims, strides, box, estr,
                CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Selection windows per block: the strided windows that lie entirely inside a block (1 without windows).
static int windows_per_block(const spla_config_t* c) {
  return c->window_size > 0 ? (c->block_size - c->window_size) / c->window_stride + 1 : 1;
}

static int validate_config(const spla_config_t* c) {
  if (!c) return SPLA_ERR_INVALID_ARG;
  if (c->batch < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->top_k < 1 || c->max_context < 1)
    return SPLA_ERR_INVALID_ARG;
  if (c->n_q_heads % c->n_kv_heads) return SPLA_ERR_INVALID_ARG;
  if (c->n_sink_blocks < 0 || c->n_local_blocks < 0 || c->n_sink_blocks + c->n_local_blocks > c->top_k)
    return SPLA_ERR_INVALID_ARG;
  if ((c->kv_dtype != SPLA_F32 && c->kv_dtype != SPLA_BF16) || (c->q_dtype != SPLA_F32 && c->q_dtype != SPLA_BF16))
    return SPLA_ERR_INVALID_ARG;
  if (c->sm_scale < 0.f || c->phi_scale < 0.f || c->rms_eps < 0.f) return SPLA_ERR_INVALID_ARG;
  if (c->flags & ~(SPLA_ADOPT_CONTENTS | SPLA_FIRST_ORDER | SPLA_NO_RLA | SPLA_GENERAL_KERNELS | SPLA_STATS_BF16 | SPLA_DEBUG_BOUNDS))
    return SPLA_ERR_INVALID_ARG;
  const int G = c->n_q_heads / c->n_kv_heads;
  if (G > kMaxGroup) return SPLA_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return SPLA_ERR_UNSUPPORTED;
  if (c->block_size != 16 && c->block_size != 32 && c->block_size != 64 && c->block_size != 128)
    return SPLA_ERR_UNSUPPORTED;
  if (c->top_k > kMaxTopK) return SPLA_ERR_UNSUPPORTED;
  const int64_t max_blocks = ((int64_t)c->max_context + c->block_size - 1) / c->block_size;
  if (max_blocks > kMaxBlocks) return SPLA_ERR_UNSUPPORTED;
  if ((int64_t)c->batch * c->n_kv_heads > 65535) return SPLA_ERR_UNSUPPORTED;
  if (c->window_size < 0 || c->window_stride < 0 || (c->window_size == 0) != (c->window_stride == 0))
    return SPLA_ERR_INVALID_ARG;
  if (c->window_size > c->block_size) return SPLA_ERR_INVALID_ARG;
  if (windows_per_block(c) > kMaxWindows) return SPLA_ERR_UNSUPPORTED;
  return SPLA_OK;
}

struct WorkspaceLayout {
  size_t ell, chunk_part, scores, obar_part, sel, n_sel, att_acc, att_ml, score_ticket, attend_ticket, append_ticket, state_part, state_ticket, status, total;
  int max_chunks;
};

static WorkspaceLayout workspace_layout(const spla_config_t* c) {
  WorkspaceLayout w;
  const size_t U = (size_t)c->batch * c->n_kv_heads, G = c->n_q_heads / c->n_kv_heads, d = c->head_dim;
  const size_t max_blocks = ((size_t)c->max_context + c->block_size - 1) / c->block_size;
  const size_t NW = windows_per_block(c);
  w.max_chunks = (int)((max_blocks * NW + kScoreChunkMin - 1) / kScoreChunkMin);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.ell = take(U * G * max_blocks * NW * 4);
  w.chunk_part = take(U * w.max_chunks * G * 2 * 4);
  w.scores = take(U * max_blocks * 4);
  w.obar_part = take(U * kStateSplits * G * d * 4);
  w.sel = take(U * c->top_k * 4);
  w.n_sel = take(U * 4);
  w.att_acc = take(U * c->top_k * 2 * G * d * 4);
  w.att_ml = take(U * c->top_k * G * 2 * 4);
  w.score_ticket = take(U * 4);
  w.attend_ticket = take(U * 4);
  w.append_ticket = take(256);
  w.state_part = take(state_umma_part_bytes((int)U, (int)d));
  w.state_ticket = take(U * 4);
  w.status = take(256);
  w.total = off;
  return w;
}

extern "C" int spla_query_sizes(const spla_config_t* config, spla_sizes_t* sizes_out) {
  int rc = validate_config(config);
  if (rc) return rc;
  if (!sizes_out) return SPLA_ERR_INVALID_ARG;
  const size_t U = (size_t)config->batch * config->n_kv_heads, d = config->head_dim, B = config->block_size;
  const size_t max_blocks = ((size_t)config->max_context + B - 1) / B;
  const size_t e = config->kv_dtype == SPLA_BF16 ? 2 : 4;
  sizes_out->k_cache = U * max_blocks * B * d * e;
  sizes_out->v_cache = sizes_out->k_cache;
  sizes_out->stats = U * max_blocks * windows_per_block(config) * 2 * d * ((config->flags & SPLA_STATS_BF16) ? 2 : 4);
  sizes_out->rla_state = U * d * d * 4;
  sizes_out->tok_lse = U * max_blocks * B * 4;
  sizes_out->seq_lens = (size_t)config->batch * 4;
  sizes_out->workspace = workspace_layout(config).total;
  return SPLA_OK;
}

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

extern "C" int spla_init_cache(const spla_config_t* config, const spla_buffers_t* b, void* stream,
                               spla_cache_t** cache_out) {
  int rc = validate_config(config);
  if (rc) return rc;
  if (!b || !cache_out) return SPLA_ERR_INVALID_ARG;
  if (!b->k_cache || !b->v_cache || !b->stats || !b->rla_state || !b->tok_lse || !b->seq_lens || !b->workspace)
    return SPLA_ERR_INVALID_ARG;
  if (!aligned(b->k_cache, 256) || !aligned(b->v_cache, 256) || !aligned(b->stats, 256) ||
      !aligned(b->rla_state, 256) || !aligned(b->tok_lse, 256) || !aligned(b->workspace, 256) ||
      !aligned(b->seq_lens, 4))
    return SPLA_ERR_INVALID_ARG;
  spla_sizes_t sz;
  spla_query_sizes(config, &sz);
  if (b->workspace_bytes < sz.workspace) return SPLA_ERR_INVALID_ARG;

  spla_cache* c = new (std::nothrow) spla_cache;
  if (!c) return SPLA_ERR_INVALID_ARG;
  c->cfg = *config;
  c->buf = *b;
  c->sm_count = device_sm_count();
  if (c->cfg.sm_scale == 0.f) c->cfg.sm_scale = 1.0f / sqrtf((float)config->head_dim);
  if (c->cfg.phi_scale == 0.f) c->cfg.phi_scale = 1.0f;
  if (c->cfg.rms_eps == 0.f) c->cfg.rms_eps = 1e-6f;

  Params& p = c->p;
  memset(&p, 0, sizeof(p));
  p.batch = config->batch; p.Hq = config->n_q_heads; p.Hkv = config->n_kv_heads; p.G = p.Hq / p.Hkv;
  p.d = config->head_dim; p.B = config->block_size; p.top_k = config->top_k;
  p.max_context = config->max_context;
  p.max_blocks = (config->max_context + config->block_size - 1) / config->block_size;
  p.n_sink = config->n_sink_blocks; p.n_local = config->n_local_blocks;
  p.NW = windows_per_block(config);
  p.win_C = config->window_size > 0 ? config->window_size : config->block_size;
  p.win_s = config->window_size > 0 ? config->window_stride : config->block_size;
  p.flags = config->flags; p.kv_bf16 = config->kv_dtype == SPLA_BF16;
  p.sm_scale = c->cfg.sm_scale; p.phi_scale = c->cfg.phi_scale; p.rms_eps = c->cfg.rms_eps;
  p.k_cache = b->k_cache; p.v_cache = b->v_cache; p.stats = reinterpret_cast<float*>(b->stats); p.state = b->rla_state;
  p.tok_lse = b->tok_lse; p.seq_lens = b->seq_lens;
  const WorkspaceLayout w = workspace_layout(config);
  char* ws = reinterpret_cast<char*>(b->workspace);
  p.ell = (float*)(ws + w.ell); p.chunk_part = (float*)(ws + w.chunk_part); p.scores = (float*)(ws + w.scores);
  p.obar_part = (float*)(ws + w.obar_part); p.sel = (int*)(ws + w.sel); p.n_sel = (int*)(ws + w.n_sel);
  p.att_acc = (float*)(ws + w.att_acc); p.att_ml = (float*)(ws + w.att_ml);
  p.score_ticket = (int*)(ws + w.score_ticket); p.attend_ticket = (int*)(ws + w.attend_ticket);
  p.append_ticket = (int*)(ws + w.append_ticket);
  p.state_part = (float*)(ws + w.state_part); p.state_ticket = (int*)(ws + w.state_ticket);
  p.status = (int*)(ws + w.status);
  p.max_chunks = w.max_chunks;
  p.tile_rows = (p.B * p.d * 2 > 16384 && p.B % 32 == 0) ? p.B / 2 : p.B;
  p.acs = 0;

  c->maps.valid = false;
  c->state_maps.valid = false;
  if (p.kv_bf16) {
    const unsigned long long rows = (unsigned long long)p.batch * p.Hkv * p.max_blocks * p.B;
    c->maps.valid = make_kv_tile_map(c->maps.k, b->k_cache, p.d, p.tile_rows, rows) &&
                    make_kv_tile_map(c->maps.v, b->v_cache, p.d, p.tile_rows, rows);
    c->state_maps.valid = p.d == 128 && rows >= 64 && rows < (1ull << 31) && !(config->flags & SPLA_GENERAL_KERNELS) &&
                          make_kv_map(c->state_maps.k, b->k_cache, p.d, 64, rows) &&
                          make_kv_map(c->state_maps.v, b->v_cache, p.d, 64, rows);
  }

  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(b->workspace, 0, w.total, s);
  if (e == cudaSuccess && !(config->flags & SPLA_ADOPT_CONTENTS)) {
    e = cudaMemsetAsync(b->stats, 0, sz.stats, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(b->rla_state, 0, sz.rla_state, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(b->tok_lse, 0, sz.tok_lse, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(b->seq_lens, 0, sz.seq_lens, s);
    c->len_bound = 0;
  } else {
    c->len_bound = config->max_context;   // adopted contents: lengths unknown to the host until told
  }
  if (e != cudaSuccess) {
    delete c;
    return cuda_fail(e, "spla_init_cache");
  }
  *cache_out = c;
  return SPLA_OK;
}

extern "C" int spla_set_length_bound(spla_cache_t* c, int32_t max_seq_len) {
  if (!c || max_seq_len < 0 || max_seq_len > c->cfg.max_context) return SPLA_ERR_INVALID_ARG;
  c->len_bound = max_seq_len;
  return SPLA_OK;
}

extern "C" int spla_append_tokens(spla_cache_t* c, const void* k_new, const void* v_new, const int32_t* n_new,
                                  int32_t max_new, void* stream) {
  if (!c || !k_new || !v_new || max_new < 1) return SPLA_ERR_INVALID_ARG;
  if (!aligned(k_new, 16) || !aligned(v_new, 16)) return SPLA_ERR_INVALID_ARG;
  if (c->len_bound + max_new > c->cfg.max_context) return SPLA_ERR_CAPACITY;
  cudaError_t e = launch_append(c->p, k_new, v_new, n_new, max_new, &c->state_maps, (cudaStream_t)stream);
  if (e != cudaSuccess) return cuda_fail(e, "spla_append_tokens");
  c->len_bound += max_new;
  return SPLA_OK;
}

// Sizes the score grid from the host-side bound of the sequence lengths: the CTAs per unit (cluster size) and the
// blocks per CTA.  Wanted: as many CTAs as the device holds at once (two per SM), so that every SM streams, but all
// of them resident together - a cluster's CTAs sit in one GPC, so the device may hold fewer clusters of a size than
// its CTA slots suggest, and a launch whose clusters do not all fit runs in two waves and takes twice as long.  The
// cluster size need not be a power of two (32 units x 9 CTAs fill 148 SMs where 32 x 8 leave 40 of them half empty).
// Candidates go from the largest that fits the slots down to the smallest the block count allows; the first whose
// clusters the occupancy query reports as all resident is taken.
// `fused`: the plan is for the fused decode kernel (score + attend in one launch), whose occupancy is asked for.
// Returns true with p->cs / chunk set if a cluster kernel can serve the launch.
static bool plan_score_clusters(spla_cache* c, Params* p, int64_t blocks, bool fused) {
  const int units = p->batch * p->Hkv;
  const int wi = fused ? 1 : 0;
  const long long slots = 2LL * c->sm_count;
  int cs_lo = 1;                                            // keep the local ranking short: at most 576 blocks per CTA
  while (cs_lo < 16 && blocks > 576LL * cs_lo) ++cs_lo;
  while (cs_lo < 16 && !score_cluster_chunk(blocks, cs_lo, p->NW, p->G, p->d)) ++cs_lo;
  if (!score_cluster_chunk(blocks, cs_lo, p->NW, p->G, p->d)) return false;
  int cs_hi = (int)(slots / units);
  if (cs_hi > 16) cs_hi = 16;
  if (cs_hi < cs_lo) cs_hi = cs_lo;                         // several waves by necessity
  int pick = cs_lo;
  for (int cs = cs_hi; cs >= cs_lo; --cs) {
    const int chunk = score_cluster_chunk(blocks, cs, p->NW, p->G, p->d);
    if (!chunk) continue;
    if (cs == 1 || (long long)units * cs > slots) { pick = cs; break; }   // nothing to ask
    if (c->score_occ_chunk[wi][cs] != chunk) {
      Params probe = *p;
      probe.cs = cs;
      probe.chunk = chunk;
      c->score_occ_n[wi][cs] = fused ? decode_fused_max_clusters(probe) : score_cluster_max_clusters(probe);
      c->score_occ_chunk[wi][cs] = chunk;
    }
    const int occ = c->score_occ_n[wi][cs];
    if (units <= occ || (occ < 0 && (cs & (cs - 1)) == 0)) { pick = cs; break; }   // all resident (or unknown, for the portable sizes)
  }
  p->cs = pick;
  p->chunk = score_cluster_chunk(blocks, pick, p->NW, p->G, p->d);
  p->n_chunks_cap = pick;
  return true;
}

// `fused`: plan for the fused decode kernel if a cluster plan exists (p->cs > 0 on return), else for the general kernel.
static void plan_score_grid(spla_cache* c, Params* p, bool fused = false) {
  int64_t blocks = (c->len_bound + c->cfg.block_size - 1) / c->cfg.block_size;
  if (blocks < 1) blocks = 1;
  p->cs = 0;
  if (!(c->cfg.flags & SPLA_GENERAL_KERNELS) && plan_score_clusters(c, p, blocks, fused)) return;
  p->cs = 0;
  p->chunk = score_chunk_for((long long)p->batch * p->Hkv, blocks * p->NW, c->sm_count);   // in records (windows)
  p->n_chunks_cap = (int)((blocks * p->NW + p->chunk - 1) / p->chunk);
}

// The fused decode kernel serves bf16 caches and queries with groups of up to 8 heads (what the tensor-core attend
// phase is built for) whenever the cluster score plan exists.
static bool fused_eligible(const spla_cache* c) {
  return !(c->cfg.flags & SPLA_GENERAL_KERNELS) && c->p.kv_bf16 && c->cfg.q_dtype == SPLA_BF16 &&
         c->p.G <= 8 && c->maps.valid && attend_mma_smem_bytes(c->p.tile_rows, c->p.d, 1) + 4096 <= (size_t)113 * 1024;
}


static cudaError_t launch_score(const Params& p, const void* q, int qb, int* sel_user, cudaStream_t s, int pending_new = 0) {
  return p.cs > 0 ? launch_score_cluster(p, q, qb, sel_user, pending_new, s) : launch_score_select(p, q, qb, sel_user, s);
}

// Cluster size of the tensor-core attend kernel as a launch of its own, written to p->acs: the largest power of two (at
// most 16 and at most top_k) for which all CTAs are resident at once; each CTA of a cluster then walks top_k / size
// selected blocks.
static void plan_attend(spla_cache* c, Params* p) {
  p->acs = 0;
  if (c->cfg.flags & SPLA_GENERAL_KERNELS) return;
  const long long U = (long long)c->p.batch * c->p.Hkv;
  const size_t smem = attend_mma_smem_bytes(c->p.tile_rows, c->p.d, 1) + 2048;
  long long per_sm = (227 * 1024) / (long long)smem;
  if (per_sm > 2) per_sm = 2;                     // the kernel is compiled for two CTAs per SM (no register spills)
  if (per_sm < 1) return;                         // the tiles do not fit: use the general kernel
  const long long slots = per_sm * c->sm_count;
  int cs = 1;
  while (cs * 2 <= 16 && cs * 2 <= c->p.top_k && U * cs * 2 <= slots) cs *= 2;
  // all clusters of the launch must be resident together (see plan_score_clusters): ask the device
  for (; cs > 1; cs /= 2) {
    int lg = 0;
    while ((1 << lg) < cs) ++lg;
    if (c->attend_occ[lg] == -2) {
      Params probe = c->p;
      probe.acs = cs;
      c->attend_occ[lg] = attend_mma_max_clusters(probe);
    }
    if (c->attend_occ[lg] < 0 || U <= c->attend_occ[lg]) break;
  }
  p->acs = cs;
}

// Steps a1-a5 for every unit: the fused kernel where it applies, else score + select and attend + merge as two launches.
// pending > 0: the call directly follows, in the stream, this step's append of at most that many tokens per sequence;
// the score phase then streams the statistics of the blocks that were complete before it while it still runs.
// (Starting that stream early in a plain spla_decode as well, before the wait for whatever kernel precedes, with the
// query read after the wait, was measured and is not done: decode at 128K 39.6 against 38.8 us.)
static int launch_decode(spla_cache* c, const void* q, const float* rms_weight, float* out, int32_t* sel_idx,
                         float* dbg_o_sparse, float* dbg_o_rla, int pending, cudaStream_t s, const char* where) {
  Params p = c->p;
  const int qb = c->cfg.q_dtype == SPLA_BF16;
  cudaError_t e;
  if (fused_eligible(c)) {
    // (a launch of several waves keeps the two-kernel form: measured faster there, the phases of different waves
    // would otherwise compete for the same SMs)
    plan_score_grid(c, &p, true);
    if (p.cs > 0 && (long long)p.batch * p.Hkv * p.cs <= 2LL * c->sm_count) {
      e = launch_decode_fused(p, c->maps, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, sel_idx, pending, s);
      return e == cudaSuccess ? SPLA_OK : cuda_fail(e, where);
    }
  }
  plan_score_grid(c, &p, false);
  plan_attend(c, &p);
  e = launch_score(p, q, qb, sel_idx, s, pending);
  if (e == cudaSuccess) e = launch_attend_merge(p, &c->maps, q, qb, rms_weight, nullptr, out, dbg_o_sparse, dbg_o_rla, s);
  return e == cudaSuccess ? SPLA_OK : cuda_fail(e, where);
}

extern "C" int spla_decode(spla_cache_t* c, const void* q, const float* rms_weight, float* out, int32_t* sel_idx,
                           float* dbg_o_sparse, float* dbg_o_rla, void* stream) {
  if (!c || !q || !out) return SPLA_ERR_INVALID_ARG;
  if (!rms_weight && !(c->cfg.flags & SPLA_NO_RLA)) return SPLA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16)) return SPLA_ERR_INVALID_ARG;
  return launch_decode(c, q, rms_weight, out, sel_idx, dbg_o_sparse, dbg_o_rla, 0, (cudaStream_t)stream, "spla_decode");
}

// One decode step, append then decode, as one call.  Because the score kernel then directly follows this step's
// append kernel in the stream, it is told so and streams the statistics of the blocks that were complete before
// the append while the append is still running; it waits for the append only before it reads the final lengths
// and the few blocks the append wrote to.  Same results as the two calls made one after the other.
extern "C" int spla_append_decode(spla_cache_t* c, const void* k_new, const void* v_new, const int32_t* n_new,
                                  int32_t max_new, const void* q, const float* rms_weight, float* out,
                                  int32_t* sel_idx, float* dbg_o_sparse, float* dbg_o_rla, void* stream) {
  if (!c || !q || !out) return SPLA_ERR_INVALID_ARG;
  if (!rms_weight && !(c->cfg.flags & SPLA_NO_RLA)) return SPLA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16)) return SPLA_ERR_INVALID_ARG;
  const int rc = spla_append_tokens(c, k_new, v_new, n_new, max_new, stream);
  if (rc != SPLA_OK) return rc;
  // only the fused decode-step append kernel (at most 32 tokens) opens the dependent launch early enough for the
  // early stream to matter
  return launch_decode(c, q, rms_weight, out, sel_idx, dbg_o_sparse, dbg_o_rla, max_new <= 32 ? max_new : 0,
                       (cudaStream_t)stream, "spla_append_decode");
}

extern "C" int spla_select(spla_cache_t* c, const void* q, int32_t* sel_idx, void* stream) {
  if (!c || !q || !sel_idx) return SPLA_ERR_INVALID_ARG;
  if (!aligned(q, 16)) return SPLA_ERR_INVALID_ARG;
  Params p = c->p;
  plan_score_grid(c, &p);
  cudaError_t e = launch_score(p, q, c->cfg.q_dtype == SPLA_BF16, sel_idx, (cudaStream_t)stream);
  return e == cudaSuccess ? SPLA_OK : cuda_fail(e, "spla_select");
}

extern "C" int spla_decode_selected(spla_cache_t* c, const void* q, const float* rms_weight, const int32_t* sel_in,
                                    float* out, float* dbg_o_sparse, float* dbg_o_rla, void* stream) {
  if (!c || !q || !out || !sel_in) return SPLA_ERR_INVALID_ARG;
  if (!rms_weight && !(c->cfg.flags & SPLA_NO_RLA)) return SPLA_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16)) return SPLA_ERR_INVALID_ARG;
  Params p = c->p;
  p.n_chunks_cap = 0;                      // only the o_bar CTAs of the first kernel run
  p.chunk = kScoreChunkMin;
  p.cs = 0;
  plan_attend(c, &p);
  const int qb = c->cfg.q_dtype == SPLA_BF16;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaSuccess;
  if (!(c->cfg.flags & SPLA_NO_RLA)) e = launch_score_select(p, q, qb, nullptr, s);
  if (e != cudaSuccess) return cuda_fail(e, "spla_decode_selected/o_bar");
  e = launch_attend_merge(p, &c->maps, q, qb, rms_weight, sel_in, out, dbg_o_sparse, dbg_o_rla, s);
  if (e != cudaSuccess) return cuda_fail(e, "spla_decode_selected/attend_merge");
  return SPLA_OK;
}

// ---- prefill-shaped forward --------------------------------------------------------------------------------------
// Workspace of spla_prefill: the per-position tables for the whole chunk, then the decode kernels' scratch for one
// batch of `tb` positions (U * tb virtual units).
struct PrefillLayout {
  size_t vstats, vobar, ell, chunk_part, scores, sel, n_sel, att_acc, att_ml, tickets, tickets_bytes, total;
  int max_chunks;
};

static PrefillLayout prefill_layout(const spla_config_t* c, int T, int tb) {
  PrefillLayout w;
  const size_t U = (size_t)c->batch * c->n_kv_heads, G = c->n_q_heads / c->n_kv_heads, d = c->head_dim;
  const size_t max_blocks = ((size_t)c->max_context + c->block_size - 1) / c->block_size;
  const size_t V = U * (size_t)tb;                 // virtual units per launch
  w.max_chunks = (int)((max_blocks + kScoreChunkMin - 1) / kScoreChunkMin);
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  w.vstats = take(U * T * 2 * d * 4);
  w.vobar = take(U * T * G * d * 4);
  w.ell = take(V * G * max_blocks * 4);
  w.chunk_part = take(V * w.max_chunks * G * 2 * 4);
  w.scores = take(V * max_blocks * 4);
  w.sel = take(V * c->top_k * 4);
  w.n_sel = take(V * 4);
  w.att_acc = take(V * c->top_k * 2 * G * d * 4);
  w.att_ml = take(V * c->top_k * G * 2 * 4);
  w.tickets = take(2 * V * 4);                      // score tickets, then attend tickets: zeroed by every call
  w.tickets_bytes = 2 * V * 4;
  w.total = off;
  return w;
}

static int prefill_batch_cap(const spla_config_t* c) {   // virtual units are the grid's y dimension
  const long long U = (long long)c->batch * c->n_kv_heads;
  return (int)(65535 / U);
}

extern "C" int spla_query_prefill_workspace(const spla_config_t* config, int32_t T, size_t* min_bytes, size_t* good_bytes) {
  int rc = validate_config(config);
  if (rc) return rc;
  if (T < 1 || (!min_bytes && !good_bytes)) return SPLA_ERR_INVALID_ARG;
  if (prefill_batch_cap(config) < 1) return SPLA_ERR_UNSUPPORTED;
  const size_t one = prefill_layout(config, T, 1).total;
  if (min_bytes) *min_bytes = one;
  if (good_bytes) {
    // about 256 MB of per-batch scratch, at most the whole chunk at once
    const size_t per_pos = prefill_layout(config, T, 2).total - one;
    long long tb = (long long)((256ull << 20) / (per_pos ? per_pos : 1));
    if (tb < 1) tb = 1;
    if (tb > T) tb = T;
    if (tb > prefill_batch_cap(config)) tb = prefill_batch_cap(config);
    *good_bytes = prefill_layout(config, T, (int)tb).total;
  }
  return SPLA_OK;
}

extern "C" int spla_prefill(spla_cache_t* c, const void* k_new, const void* v_new, const void* q, int32_t T,
                            const float* rms_weight, float* out, int32_t* sel_idx, void* workspace, size_t workspace_bytes,
                            void* stream) {
  if (!c || !k_new || !v_new || !q || !out || !workspace || T < 1) return SPLA_ERR_INVALID_ARG;
  if (!rms_weight && !(c->cfg.flags & SPLA_NO_RLA)) return SPLA_ERR_INVALID_ARG;
  if (!aligned(k_new, 16) || !aligned(v_new, 16) || !aligned(q, 16) || !aligned(out, 16) || !aligned(workspace, 256))
    return SPLA_ERR_INVALID_ARG;
  if (c->p.NW != 1) return SPLA_ERR_UNSUPPORTED;                 // whole-block statistics only
  if (c->len_bound + T > c->cfg.max_context) return SPLA_ERR_CAPACITY;
  // positions per launch: as many as the workspace holds
  const int cap = prefill_batch_cap(&c->cfg);
  if (cap < 1) return SPLA_ERR_UNSUPPORTED;
  const size_t one = prefill_layout(&c->cfg, T, 1).total;
  if (workspace_bytes < one) return SPLA_ERR_INVALID_ARG;
  const size_t per_pos = prefill_layout(&c->cfg, T, 2).total - one;
  long long tb = 1 + (long long)((workspace_bytes - one) / (per_pos ? per_pos : 1));
  if (tb > T) tb = T;
  if (tb > cap) tb = cap;
  while (tb > 1 && prefill_layout(&c->cfg, T, (int)tb).total > workspace_bytes) --tb;   // (alignment padding)
  const PrefillLayout w = prefill_layout(&c->cfg, T, (int)tb);
  char* ws = reinterpret_cast<char*>(workspace);
  cudaStream_t s = (cudaStream_t)stream;
  const int qb = c->cfg.q_dtype == SPLA_BF16;

  // 1. the chunk goes into the cache: K/V, per-token log-sum-exp, block statistics, lengths; the state is left for the
  //    scan (which needs S_bar as it was before the chunk)
  {
    Params pa = c->p;
    pa.flags |= SPLA_NO_RLA;
    cudaError_t e = launch_append(pa, k_new, v_new, nullptr, T, nullptr, s);
    if (e != cudaSuccess) return cuda_fail(e, "spla_prefill/append");
    c->len_bound += T;
  }
  // 2. per-position statistics of the growing block, o_bar of every position, S_bar advanced over the chunk
  float* vstats = reinterpret_cast<float*>(ws + w.vstats);
  float* vobar = reinterpret_cast<float*>(ws + w.vobar);
  cudaError_t e = launch_prefill_prepare(c->p, T, q, qb, vstats, vobar, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + w.tickets, 0, w.tickets_bytes, s);
  if (e != cudaSuccess) return cuda_fail(e, "spla_prefill/prepare");
  // 3. score, select, attend, merge: the general decode kernels over virtual units, a batch of positions per launch
  Params pv = c->p;
  pv.ell = (float*)(ws + w.ell); pv.chunk_part = (float*)(ws + w.chunk_part); pv.scores = (float*)(ws + w.scores);
  pv.sel = (int*)(ws + w.sel); pv.n_sel = (int*)(ws + w.n_sel);
  pv.att_acc = (float*)(ws + w.att_acc); pv.att_ml = (float*)(ws + w.att_ml);
  pv.score_ticket = (int*)(ws + w.tickets); pv.attend_ticket = pv.score_ticket + (size_t)c->p.batch * c->p.Hkv * tb;
  pv.max_chunks = w.max_chunks;
  pv.vTtot = T; pv.vstats = vstats; pv.vobar = vobar;
  pv.cs = 0; pv.acs = 0;
  int64_t blocks = (c->len_bound + c->cfg.block_size - 1) / c->cfg.block_size;
  if (blocks < 1) blocks = 1;
  for (int t0 = 0; t0 < T; t0 += (int)tb) {
    pv.vt0 = t0;
    pv.vT = (int)(tb < T - t0 ? tb : T - t0);
    pv.chunk = score_chunk_for((long long)pv.batch * pv.Hkv * pv.vT, blocks, c->sm_count);
    pv.n_chunks_cap = (int)((blocks + pv.chunk - 1) / pv.chunk);
    e = launch_score_select(pv, q, qb, sel_idx, s);
    if (e == cudaSuccess) e = launch_attend_merge(pv, nullptr, q, qb, rms_weight, nullptr, out, nullptr, nullptr, s);
    if (e != cudaSuccess) return cuda_fail(e, "spla_prefill/decode kernels");
  }
  return SPLA_OK;
}

extern "C" int spla_copy_scores(spla_cache_t* c, float* scores_out, void* stream) {
  if (!c || !scores_out) return SPLA_ERR_INVALID_ARG;
  const size_t bytes = (size_t)c->p.batch * c->p.Hkv * c->p.max_blocks * sizeof(float);
  cudaError_t e = cudaMemcpyAsync(scores_out, c->p.scores, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream);
  return e == cudaSuccess ? SPLA_OK : cuda_fail(e, "spla_copy_scores");
}

extern "C" int spla_sync_status(spla_cache_t* c, void* stream) {
  if (!c) return SPLA_ERR_INVALID_ARG;
  int st = 0;
  cudaStream_t s = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(&st, c->p.status, sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && st != 0) e = cudaMemsetAsync(c->p.status, 0, sizeof(int), s);
  if (e != cudaSuccess) return cuda_fail(e, "spla_sync_status");
  return st;
}

extern "C" int spla_debug_wait_hook(spla_cache_t* c, int32_t max_wait_polls, int32_t extra_expected_bytes) {
  if (!c || max_wait_polls < 0 || extra_expected_bytes < 0 || (extra_expected_bytes % 16)) return SPLA_ERR_INVALID_ARG;
  c->p.wait_limit = max_wait_polls;
  c->p.dbg_tx_extra = extra_expected_bytes;
  return SPLA_OK;
}

extern "C" int spla_destroy_cache(spla_cache_t* c) {
  delete c;
  return SPLA_OK;
}

extern "C" const char* spla_status_string(int status) {
  switch (status) {
    case SPLA_OK: return "ok";
    case SPLA_ERR_INVALID_ARG: return "invalid argument";
    case SPLA_ERR_CAPACITY: return "cache capacity exceeded";
    case SPLA_ERR_CUDA: return "CUDA error";
    case SPLA_ERR_UNSUPPORTED: return "unsupported configuration";
    case SPLA_ERR_TIMEOUT: return "a kernel's bounded wait ran out";
    case SPLA_ERR_BOUNDS: return "length or index outside the cache (clamped or skipped on the device)";
    default: return "unknown status";
  }
}

extern "C" const char* spla_last_cuda_error(void) { return g_cuda_err; }

extern "C" unsigned long long spla_launch_count(void) { return g_launch_count; }
