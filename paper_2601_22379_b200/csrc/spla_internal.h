// Host-side declarations shared by the translation units of the library (not part of the public ABI).
#pragma once

#include "spla_device.cuh"

namespace spla {

// GQA group sizes are padded to the next power of two inside the kernels; padded heads carry zero queries
// and are never written out.
inline int padded_group(int G) {
  int gp = 1;
  while (gp < G) gp <<= 1;
  return gp;
}

// Kernels this library has launched from the calling thread (spla_launch_count): bumped at every launch site.
extern thread_local unsigned long long g_launch_count;

// Launch with optional thread-block-cluster shape and programmatic dependent launch: with `pdl` the grid may
// start while the preceding kernel of the stream drains; it must execute griddepcontrol.wait before it touches
// anything that kernel produces (every kernel launched this way does so in its prologue).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_ex(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream, int cluster_x,
                             bool pdl, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (cluster_x > 0) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x;
    attr[n].val.clusterDim.y = 1;
    attr[n].val.clusterDim.z = 1;
    ++n;
  }
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  cfg.attrs = attr;
  cfg.numAttrs = n;
  ++g_launch_count;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// How many clusters of `cluster_x` CTAs of this kernel the device holds at once (all CTAs of a cluster sit in one
// GPC, so this is less than CTA slots / cluster size); -1 if the query fails.
template <typename... KArgs>
inline int max_active_clusters(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, int cluster_x) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cluster_x;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return n;
}

// spla_api.cu: records the text of a failed CUDA call for spla_last_cuda_error and returns SPLA_ERR_CUDA
int cuda_fail(cudaError_t e, const char* where);
int device_sm_count();   // multiprocessors of the current device (148 if the query fails)
// score_select.cu
int score_chunk_for(long long units, long long max_seq_blocks, int sm_count);
cudaError_t launch_score_select(const Params& p, const void* q, int q_is_bf16, int* sel_user, cudaStream_t stream);
// score_cluster.cu (G <= 8, at most 16 x 1024 blocks per sequence)
int score_cluster_chunk(long long max_seq_blocks, int cs, int NW, int G, int d);   // blocks per CTA, 0: not servable
// Clusters of the score kernel (p.cs CTAs each, p.chunk blocks per CTA) the device holds at once; -1 if unknown.
int score_cluster_max_clusters(const Params& p);
cudaError_t launch_score_cluster(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new,
                                 cudaStream_t stream);
struct AttendMaps {                      // TMA tensor maps (CUtensorMap) of the K and V caches, opaque to the host code
  alignas(64) unsigned char k[128];
  alignas(64) unsigned char v[128];
  bool valid;
};
// state_umma.cu (bulk S_bar update on tcgen05 tensor cores: bf16 cache, d = 128; maps with boxes of 64 tokens)
int state_umma_splits(int units);
size_t state_umma_part_bytes(int units, int d);
cudaError_t launch_state_umma(const Params& p, const AttendMaps* maps, const int* n_new, int max_new, cudaStream_t stream);
// attend_merge.cu
cudaError_t launch_attend_merge(const Params& p, const AttendMaps* maps, const void* q, int q_is_bf16,
                                const float* rms_weight, const int* sel_in, float* out, float* dbg_o_sparse,
                                float* dbg_o_rla, cudaStream_t stream);
// attend_mma.cu (bf16 K/V and q, G <= 8)
size_t attend_mma_smem_bytes(int B, int D, int groups);
int attend_mma_max_clusters(const Params& p);   // clusters of p.acs CTAs resident at once; -1 if unknown
cudaError_t launch_attend_mma(const Params& p, const AttendMaps& maps, const void* q, const float* rms_weight, float* out,
                              float* dbg_o_sparse, float* dbg_o_rla, cudaStream_t stream);
// prefill.cu: prefix statistics of every chunk position's own block and the chunk scan (o_bar per position; advances S_bar)
cudaError_t launch_prefill_prepare(const Params& p, int Ttot, const void* q, int q_is_bf16, float* vstats, float* vobar,
                                   cudaStream_t stream);
// decode_fused.cu: score + select + attend + merge of one decode step as one cluster kernel (bf16 K/V and q, G <= 8;
// the cluster plan in p.cs / p.chunk).  pending_new as for launch_score_cluster.
cudaError_t launch_decode_fused(const Params& p, const AttendMaps& maps, const void* q, const float* rms_weight, float* out,
                                float* dbg_o_sparse, float* dbg_o_rla, int* sel_user, int pending_new, cudaStream_t stream);
int decode_fused_max_clusters(const Params& p);   // clusters of p.cs CTAs resident at once; -1 if unknown
// append.cu
// `state_maps` (may be null): tensor maps with boxes of 64 tokens; when given, bulk appends of a bf16 cache with
// d = 128 update S_bar on the tensor cores instead of the FMA kernel.
cudaError_t launch_append(const Params& p, const void* k_new, const void* v_new, const int* n_new, int max_new,
                          const AttendMaps* state_maps, cudaStream_t stream);

}  // namespace spla
