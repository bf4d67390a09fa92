// The tensor-core attend + merge kernel as a launch of its own, and its launch shapes.
#include "attend_mma.cuh"

namespace spla {

template <int D, bool PACK, int NG>
__global__ void __launch_bounds__(NG * kAttendThreads, NG == 1 ? 2 : 1)
    attend_mma_kernel(const Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const __nv_bfloat16* __restrict__ q, const float* __restrict__ rms_weight, float* __restrict__ out,
                      float* __restrict__ dbg_sparse, float* __restrict__ dbg_rla) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  attend_mma_body<D, PACK, NG, false>(p, map_k, map_v, q, rms_weight, out, dbg_sparse, dbg_rla, smem_raw);
}

// Dynamic shared memory of the kernel: the two-slot tile ring, reused for the cross-warp fold, and the receive area of
// the merge behind it.
size_t attend_mma_smem_bytes(int B, int D, int groups) { return attend_mma_ring_bytes(B, D, groups) + attend_mma_recv_bytes(D); }

template <int D, bool PACK, int NG>
static cudaError_t launch_shape(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                                float* dr, cudaStream_t stream, int* occupancy) {
  const size_t smem = attend_mma_smem_bytes(p.tile_rows, D, NG);
  const dim3 grid(p.acs, p.batch * p.Hkv);
  auto kern = attend_mma_kernel<D, PACK, NG>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess && p.acs > 8) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  if (e != cudaSuccess) return e;
  if (occupancy) {
    *occupancy = max_active_clusters(kern, grid, dim3(NG * kAttendThreads), smem, p.acs);
    return cudaSuccess;
  }
  const CUtensorMap& mk = *reinterpret_cast<const CUtensorMap*>(maps.k);
  const CUtensorMap& mv = *reinterpret_cast<const CUtensorMap*>(maps.v);
  return launch_ex(kern, grid, dim3(NG * kAttendThreads), smem, stream, p.acs, true, p, mk, mv,
                   reinterpret_cast<const __nv_bfloat16*>(q), w, out, ds, dr);
}

template <int D>
static cudaError_t launch_mma(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                              float* dr, cudaStream_t stream, int* occ) {
  return p.G <= 4 ? launch_shape<D, true, 1>(p, maps, q, w, out, ds, dr, stream, occ)
                  : launch_shape<D, false, 1>(p, maps, q, w, out, ds, dr, stream, occ);
}

// Clusters of p.acs CTAs of the attend kernel the device holds at once; -1 if the query fails.
int attend_mma_max_clusters(const Params& p) {
  int n = -1;
  AttendMaps none;
  const cudaError_t e = p.d == 128 ? launch_mma<128>(p, none, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, &n)
                                   : launch_mma<64>(p, none, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, &n);
  if (e != cudaSuccess) { cudaGetLastError(); return -1; }
  return n;
}

cudaError_t launch_attend_mma(const Params& p, const AttendMaps& maps, const void* q, const float* rms_weight, float* out,
                              float* dbg_o_sparse, float* dbg_o_rla, cudaStream_t stream) {
  return p.d == 128 ? launch_mma<128>(p, maps, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream, nullptr)
                    : launch_mma<64>(p, maps, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream, nullptr);
}

}  // namespace spla
