// The 16-warp build of the cluster score kernel: one CTA per SM, a 192 KB statistics ring.
#include "score_cluster.cuh"

namespace spla {

cudaError_t launch_score_cluster16(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new,
                                   cudaStream_t stream, int* occ) {
  return launch_size<16>(p, q, q_is_bf16, sel_user, pending_new, stream, occ);
}

}  // namespace spla
