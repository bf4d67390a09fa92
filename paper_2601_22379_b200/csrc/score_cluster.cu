// The cluster score + select kernel as a launch of its own, and the planner of its grid.
#include "score_cluster.cuh"

namespace spla {

// Decides whether the cluster kernel can serve a launch and with which cluster size / records per CTA.
// Returns false when the general kernel has to be used (very long sequences, groups above 8).
// `cs_cap` bounds the cluster size from above where the block count leaves a choice (the caller lowers it when the
// device cannot hold all clusters of the first choice at once).  `warps` is the build size (8 or 16): the 16-warp
// build holds one CTA per SM, so the machine is full with half as many CTAs.
bool plan_score_cluster(int units, long long max_seq_blocks, int NW, int G, int d, int sm_count, int cs_cap, int warps,
                        int* cs_out, int* chunk_out) {
  if (G > 8) return false;
  if (max_seq_blocks < 1) max_seq_blocks = 1;
  if (cs_cap > kMaxCluster) cs_cap = kMaxCluster;
  const int per_sm = warps == 16 ? 1 : 2;
  const long long per_cta_max = warps == 16 ? 1024 : 576;                     // keep the local ranking short
  int cs = 1;
  while (cs < kMaxCluster && max_seq_blocks > per_cta_max * cs) cs *= 2;
  while (cs < cs_cap && (long long)units * cs * 2 <= (long long)per_sm * sm_count) cs *= 2;   // fill the machine once
  const long long chunk = (max_seq_blocks + cs - 1) / cs;
  const int chunk32 = (int)((chunk + 31) / 32 * 32);
  if (chunk32 > 1024) return false;
  const size_t ring = (size_t)kStages * warps * kRecPerWarp * 2 * d * 4;
  if (ring + 4096 + (size_t)G * chunk32 * 4 > (size_t)(warps == 16 ? 226 : 200) * 1024) return false;
  *cs_out = cs;
  *chunk_out = chunk32;
  return true;
}

// pending_new > 0: the kernel directly follows, in the stream, an append of at most that many tokens per sequence
// and may stream the older blocks' statistics before that append has completed.
cudaError_t launch_score_cluster(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new,
                                 cudaStream_t stream) {
  return launch_size<8>(p, q, q_is_bf16, sel_user, pending_new, stream, nullptr);
}

int score_cluster_max_clusters(const Params& p) {
  int n = -1;
  const cudaError_t e = launch_size<8>(p, nullptr, 0, nullptr, 0, nullptr, &n);
  if (e != cudaSuccess) { cudaGetLastError(); return -1; }
  return n;
}

}  // namespace spla
