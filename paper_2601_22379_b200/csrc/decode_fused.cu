// Dispatch of the fused decode kernel (decode_fused.cuh) over its four translation units.
#include "spla_internal.h"

namespace spla {

#define SPLA_DECL(name)                                                                                                     \
  cudaError_t name(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds, float* dr, \
                   int* sel_user, int pending_new, cudaStream_t s, int* occ);
SPLA_DECL(launch_decode_fused_d128f)
SPLA_DECL(launch_decode_fused_d128h)
SPLA_DECL(launch_decode_fused_d64f)
SPLA_DECL(launch_decode_fused_d64h)
#undef SPLA_DECL

static cudaError_t dispatch(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds, float* dr,
                            int* sel_user, int pending_new, cudaStream_t s, int* occ) {
  const bool half = (p.flags & kStatsBf16) != 0;
  if (p.d == 128)
    return half ? launch_decode_fused_d128h(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ)
                : launch_decode_fused_d128f(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ);
  return half ? launch_decode_fused_d64h(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ)
              : launch_decode_fused_d64f(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ);
}

// bf16 K/V and q, groups of up to 8 heads, a cluster plan in p.cs / p.chunk.
cudaError_t launch_decode_fused(const Params& p, const AttendMaps& maps, const void* q, const float* rms_weight, float* out,
                                float* dbg_o_sparse, float* dbg_o_rla, int* sel_user, int pending_new, cudaStream_t stream) {
  return dispatch(p, maps, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, sel_user, pending_new, stream, nullptr);
}

// Clusters of the fused kernel (p.cs CTAs each, p.chunk blocks per CTA) the device holds at once; -1 if unknown.
int decode_fused_max_clusters(const Params& p) {
  int n = -1;
  AttendMaps none;
  if (dispatch(p, none, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, 0, nullptr, &n) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return n;
}

}  // namespace spla
