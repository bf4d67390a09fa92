// The cluster score + select kernel as a launch of its own, and the planner of its grid.
#include "score_cluster.cuh"

namespace spla {

// Blocks per CTA when `cs` CTAs share a sequence of at most max_seq_blocks blocks, or 0 if the cluster kernel cannot
// serve that (groups above 8, more than 1024 blocks per CTA, shared memory).  The share is the exact quotient rounded
// up to a multiple of 8, so that the CTAs of a cluster stream equal amounts.
int score_cluster_chunk(long long max_seq_blocks, int cs, int NW, int G, int d) {
  if (G > 8 || cs < 1 || cs > kMaxCluster) return 0;
  if (max_seq_blocks < 1) max_seq_blocks = 1;
  const long long chunk = ((max_seq_blocks + cs - 1) / cs + 7) / 8 * 8;
  if (chunk > 1024) return 0;
  const size_t ring = (size_t)kStages * 8 * kRecPerWarp * 2 * d * 4;
  if (ring + 4096 + (size_t)G * chunk * 4 > (size_t)200 * 1024) return 0;
  (void)NW;
  return (int)chunk;
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
