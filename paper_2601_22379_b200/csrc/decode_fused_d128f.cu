// Fused decode kernel: the instantiations for head dimension 128 and float statistics records.
#include "decode_fused.cuh"

namespace spla {

cudaError_t launch_decode_fused_d128f(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                                   float* dr, int* sel_user, int pending_new, cudaStream_t s, int* occ) {
  return fused_launch_dst<128, float>(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ);
}

}  // namespace spla
