// Fused decode kernel: the instantiations for head dimension 64 and __nv_bfloat16 statistics records.
#include "decode_fused.cuh"

namespace spla {

cudaError_t launch_decode_fused_d64h(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                                   float* dr, int* sel_user, int pending_new, cudaStream_t s, int* occ) {
  return fused_launch_dst<64, __nv_bfloat16>(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ);
}

}  // namespace spla
