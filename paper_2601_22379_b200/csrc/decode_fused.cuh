// One decode step's score + select + attend + merge as ONE kernel: a thread-block cluster per (sequence, KV head)
// unit runs the whole of spla_decode for it.
//
//   phase 1  block score and top-k selection (Section 3.1, Eq. taylor-2nd; Section 2.2 grouped BlockScore;
//            Section 2.1 Select) and o_bar = phi(q) S_bar (Section 3.2, Eq. rla-impl-1): the body of the cluster
//            score kernel, all eight warps of every CTA.  It ends with the selection of the unit (best block first) in
//            every CTA's own shared memory (each CTA computes it from its copy of the unit's keys), so nothing is handed
//            over and no cluster barrier stands between the phases;
//   phase 2  exact attention over the selected blocks with the selected linear term from the same tiles
//            (Section 2.2, Eq. gqa-sparse; Section 3.2, Eq. rla-impl-2), the subtraction and the RMSNorm merge
//            (Eq. rla-impl-3, Section 3.3): the body of the tensor-core attend kernel, on the first four warps, which
//            are also the ones that selected; the other four finish o_bar meanwhile and then only join the barriers.
// The two phases want different register budgets (about 120 registers x 8 warps, then about 220 x 4 warps).  After
// phase 1 the second warp group hands its registers back to the CTA's pool and the first takes them (setmaxnreg),
// so both phases run at two CTAs per SM without spilling.  What the fusion removes: one kernel boundary per step
// (several microseconds between the last CTA of the score grid and the first byte of the attend grid) and the
// wait of every unit's attention for the slowest unit's selection - a cluster starts on its K/V tiles as soon as
// its own selection is done.
#pragma once

#include "attend_mma.cuh"
#include "score_cluster.cuh"

namespace spla {

template <int D, int GP, bool WIN, bool EARLY, typename ST>
__global__ void __launch_bounds__(256, 2)
    decode_fused_kernel(const Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                        const __nv_bfloat16* __restrict__ q, const float* __restrict__ rms_weight, float* __restrict__ out,
                        float* __restrict__ dbg_sparse, float* __restrict__ dbg_rla, int* __restrict__ sel_user, int pending_new) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ __align__(16) int sel_share[kMaxTopK + 2];   // the unit's selection, its size, the length: phase 1 leaves them here
  __shared__ __align__(8) uint64_t tile_full[kMaxSlots + 1];   // the attend phase's tile barriers and its merge barrier
  // o_bar of the heads this CTA merges (at most 8 x D floats): behind the working space of the role that computes it
  float* obar_s = reinterpret_cast<float*>(smem_raw + Smem<D, GP, ST, 8>::kStateScratch + 2048);
  if (threadIdx.x == 0) {                   // the K/V tensor maps are needed late: have them fetched now
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    for (int s = 0; s <= kMaxSlots; ++s) mbar_init(&tile_full[s], 1);  // (phase 1's initialisation fence, same thread, covers them)
  }
  score_cluster_body<D, GP, WIN, EARLY, ST, 8>(p, q, 1, sel_user, pending_new, smem_raw, sel_share, obar_s);
  if ((threadIdx.x >> 5) < 4) {
    // Phase 2's tiles arrive through the asynchronous proxy (TMA) in shared memory that these warps have just read and
    // written through the generic proxy (the key table, the selection's work arrays): each of them orders its accesses
    // before the copies, then they meet.  (What all eight warps did there earlier was ordered before phase 1's last
    // cluster barrier.)
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("bar.sync 1, 128;" ::: "memory");
    warpgroup_reg_inc<232>();
    attend_mma_body<D, (GP <= 4), 1, true>(p, map_k, map_v, q, rms_weight, out, dbg_sparse, dbg_rla, smem_raw, sel_share, tile_full,
                                           smem_raw + Smem<D, GP, ST, 8>::kMergeRecv, obar_s);
  } else {
    warpgroup_reg_dec<24>();
    if (threadIdx.x == 128) {               // the tiles are a microsecond or two away: have the tensor maps at hand again
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_k) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&map_v) : "memory");
    }
    if (blockIdx.x == 0) write_selection(p, blockIdx.y, sel_share, -1, sel_user, (int)threadIdx.x - 128);
    cluster_sync_all();    // the closing barrier of phase 2 counts every thread of the cluster
  }
}

template <int D, int GP, bool WIN, bool EARLY, typename ST>
static cudaError_t fused_launch_win(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                                    float* dr, int* sel_user, int pending_new, cudaStream_t stream, int* occupancy) {
  using SM = Smem<D, GP, ST, 8>;
  const int U = p.batch * p.Hkv;
  size_t smem = (size_t)SM::kEll + (size_t)p.G * p.chunk * sizeof(float);
  const size_t smem_attend = attend_mma_ring_bytes(p.tile_rows, D, 1);     // (the merge's receive area lies in phase 1's layout)
  if (smem_attend > smem) smem = smem_attend;
  auto kern = decode_fused_kernel<D, GP, WIN, EARLY, ST>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e == cudaSuccess && p.cs > 8) e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
  if (e != cudaSuccess) return e;
  if (occupancy) {
    *occupancy = max_active_clusters(kern, dim3(p.cs, U, 1), dim3(256, 1, 1), smem, p.cs);
    return cudaSuccess;
  }
  const CUtensorMap& mk = *reinterpret_cast<const CUtensorMap*>(maps.k);
  const CUtensorMap& mv = *reinterpret_cast<const CUtensorMap*>(maps.v);
  return launch_ex(kern, dim3(p.cs, U, 1), dim3(256, 1, 1), smem, stream, p.cs, true, p, mk, mv,
                   reinterpret_cast<const __nv_bfloat16*>(q), w, out, ds, dr, sel_user, pending_new);
}

// All instantiations for one head dimension and one statistics type (one translation unit each).
template <int D, typename ST>
static cudaError_t fused_launch_dst(const Params& p, const AttendMaps& maps, const void* q, const float* w, float* out, float* ds,
                                    float* dr, int* sel_user, int pending_new, cudaStream_t s, int* occ) {
  const int GP = padded_group(p.G);
  const bool win = p.NW > 1, early = pending_new > 0;
#define SPLA_FUSED_CASE(GPV)                                                                                                   \
  case GPV:                                                                                                                    \
    if (win) return early ? fused_launch_win<D, GPV, true, true, ST>(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ) \
                          : fused_launch_win<D, GPV, true, false, ST>(p, maps, q, w, out, ds, dr, sel_user, 0, s, occ);         \
    return early ? fused_launch_win<D, GPV, false, true, ST>(p, maps, q, w, out, ds, dr, sel_user, pending_new, s, occ)         \
                 : fused_launch_win<D, GPV, false, false, ST>(p, maps, q, w, out, ds, dr, sel_user, 0, s, occ);
  switch (GP) {
    SPLA_FUSED_CASE(1)
    SPLA_FUSED_CASE(2)
    SPLA_FUSED_CASE(4)
    default:
    SPLA_FUSED_CASE(8)
  }
#undef SPLA_FUSED_CASE
}

}  // namespace spla
