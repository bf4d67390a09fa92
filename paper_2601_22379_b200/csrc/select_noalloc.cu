// spla_select_blocks_noalloc: block scoring + top-k selection for callers that cannot allocate device memory.
//
// The regular path keeps the selection kernel's scratch (per-head log masses, per-chunk normalisers, scores,
// arrival tickets) in a workspace the caller allocates.  Some callers cannot do that: code running inside a
// memory pool that is already carved up and frozen, a plug-in that is handed tensors but no allocator, or a
// latency-critical loop where any cudaMalloc (an implicit device synchronisation) is forbidden.  For them this
// one entry point runs the same score + select kernel with its scratch in a fixed array that lives in the
// library's device image.  The price: a fixed upper size, 4 MiB of every GPU that loads the library held until
// the process exits, and one shared scratch, so two of these calls must never overlap on the GPU.
#include <math.h>
#include <string.h>

#include <mutex>

#include "../../include/spla.h"
#include "spla_internal.h"

using namespace spla;

namespace {

constexpr size_t kNoAllocScratchBytes = SPLA_NOALLOC_SCRATCH_BYTES;
constexpr int kMaxDevices = 64;

// File-scope device array.  In host code this name is only a handle for the runtime (a host-side shadow
// symbol), never a device pointer: the device address must be asked for with cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_dev_ptr[kMaxDevices] = {};   // per device: device address of g_noalloc_scratch
int g_sm_count[kMaxDevices] = {};            // per device: multiprocessor count (sizes the grid; the query allocates nothing)

// Once per device, with that device current: resolve the device address of the scratch array.
cudaError_t scratch_for_current_device(void** ptr_out, int* sm_count_out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_dev_ptr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_dev_ptr[dev] = ptr;
    g_sm_count[dev] = device_sm_count();
  }
  *ptr_out = g_scratch_dev_ptr[dev];
  *sm_count_out = g_sm_count[dev];
  return cudaSuccess;
}

size_t align256(size_t x) { return (x + 255) / 256 * 256; }

}  // namespace

extern "C" int spla_select_blocks_noalloc(const spla_config_t* cfg, const float* stats, const int32_t* seq_lens,
                                          const void* q, int32_t* sel_idx, float* scores_out, int32_t* status_out,
                                          void* stream) {
  if (!cfg || !stats || !seq_lens || !q || !sel_idx) return SPLA_ERR_INVALID_ARG;
  spla_sizes_t sz;
  const int rc = spla_query_sizes(cfg, &sz);                 // validates the configuration (host only)
  if (rc != SPLA_OK) return rc;
  if (cfg->window_size != 0 || (cfg->flags & SPLA_STATS_BF16)) return SPLA_ERR_UNSUPPORTED;   // whole-block fp32 statistics only
  if (((uintptr_t)stats % 16) || ((uintptr_t)q % 16) || ((uintptr_t)seq_lens % 4) || ((uintptr_t)sel_idx % 4))
    return SPLA_ERR_INVALID_ARG;

  // Carve the selection kernel's scratch out of the fixed array; refuse what does not fit.
  const size_t U = (size_t)cfg->batch * cfg->n_kv_heads, G = cfg->n_q_heads / cfg->n_kv_heads;
  const size_t max_blocks = ((size_t)cfg->max_context + cfg->block_size - 1) / cfg->block_size;
  const size_t max_chunks = (max_blocks + kScoreChunkMin - 1) / kScoreChunkMin;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align256(off + bytes); return o; };
  const size_t o_ticket = take(U * 4);                      // must be zero when the kernel starts
  const size_t o_status = take(256);
  const size_t zero_bytes = off;
  const size_t o_ell = take(U * G * max_blocks * 4);
  const size_t o_chunk = take(U * max_chunks * G * 2 * 4);
  const size_t o_scores = take(U * max_blocks * 4);
  const size_t o_sel = take(U * cfg->top_k * 4);
  const size_t o_nsel = take(U * 4);
  if (off > kNoAllocScratchBytes) return SPLA_ERR_UNSUPPORTED;   // beyond the fixed scratch: use spla_decode

  void* base_v = nullptr;
  int sm_count = 148;
  cudaError_t e = scratch_for_current_device(&base_v, &sm_count);
  if (e != cudaSuccess) return cuda_fail(e, "spla_select_blocks_noalloc/scratch address");
  char* base = reinterpret_cast<char*>(base_v);

  Params p;
  memset(&p, 0, sizeof(p));
  p.batch = cfg->batch; p.Hq = cfg->n_q_heads; p.Hkv = cfg->n_kv_heads; p.G = (int)G;
  p.d = cfg->head_dim; p.B = cfg->block_size; p.top_k = cfg->top_k;
  p.max_context = cfg->max_context; p.max_blocks = (int)max_blocks; p.max_chunks = (int)max_chunks;
  p.n_sink = cfg->n_sink_blocks; p.n_local = cfg->n_local_blocks;
  p.NW = 1; p.win_C = cfg->block_size; p.win_s = cfg->block_size;
  p.flags = (cfg->flags & SPLA_FIRST_ORDER) | SPLA_NO_RLA;      // score + select only: no o_bar CTAs
  p.kv_bf16 = cfg->kv_dtype == SPLA_BF16;
  p.sm_scale = cfg->sm_scale == 0.f ? 1.0f / sqrtf((float)cfg->head_dim) : cfg->sm_scale;
  p.phi_scale = 1.f; p.rms_eps = 1e-6f;
  p.chunk = score_chunk_for((long long)U, (long long)max_blocks, sm_count);
  p.n_chunks_cap = (int)((max_blocks + p.chunk - 1) / p.chunk);
  p.stats = const_cast<float*>(stats);
  p.seq_lens = const_cast<int*>(seq_lens);
  p.score_ticket = (int*)(base + o_ticket); p.status = (int*)(base + o_status);
  p.ell = (float*)(base + o_ell); p.chunk_part = (float*)(base + o_chunk); p.scores = (float*)(base + o_scores);
  p.sel = (int*)(base + o_sel); p.n_sel = (int*)(base + o_nsel);

  cudaStream_t s = (cudaStream_t)stream;
  // The array keeps whatever the previous call left: the tickets have to start at zero, and the score rows are
  // cleared so that entries past a sequence's last block read as 0 in scores_out.
  e = cudaMemsetAsync(base, 0, zero_bytes, s);
  if (e == cudaSuccess && scores_out) e = cudaMemsetAsync(base + o_scores, 0, U * max_blocks * 4, s);
  if (e == cudaSuccess) e = launch_score_select(p, q, cfg->q_dtype == SPLA_BF16, sel_idx, s);
  if (e == cudaSuccess && scores_out)
    e = cudaMemcpyAsync(scores_out, base + o_scores, U * max_blocks * 4, cudaMemcpyDeviceToDevice, s);
  if (e == cudaSuccess && status_out)
    e = cudaMemcpyAsync(status_out, base + o_status, sizeof(int), cudaMemcpyDeviceToDevice, s);
  return e == cudaSuccess ? SPLA_OK : cuda_fail(e, "spla_select_blocks_noalloc");
}
