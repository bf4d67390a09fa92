// Pieces shared by the two sparse-attend kernels: the per-unit arrival ticket and the split-K merge that the
// last CTA of a unit runs (Section 3.2, Eq. rla-impl-3 and Section 3.3 of the paper: o_rla = o_bar - o_tilde,
// out = o_sparse + RMSNorm(o_rla)).
#pragma once

#include "spla_device.cuh"

namespace spla {

// Called by all threads of the CTA after its partial results are written.  Returns true in every thread of
// the CTA that arrived last among `expected` CTAs of unit u (and re-arms the ticket).  Nobody waits.
__device__ __forceinline__ bool arrive_last(int* ticket, int expected, int* flag_smem) {
  __syncthreads();                                   // all partial-result stores precede thread 0's fence
  if (threadIdx.x == 0) {
    asm volatile("fence.acq_rel.gpu;" ::: "memory");   // release the CTA's stores (cumulative over the barrier above)
    const int t = atomicAdd(ticket, 1);
    const int last = (t == expected - 1);
    if (last) *ticket = 0;
    asm volatile("fence.acq_rel.gpu;" ::: "memory");   // acquire the other CTAs' stores
    *flag_smem = last;
  }
  __syncthreads();
  return *flag_smem != 0;
}

// Merge of the n_items partial results of unit u, by kAttendThreads threads.
//   att_ml [item][G][2]      : (max, sum) of the exact branch in the base-2 domain
//   att_acc[item][2][G][D]   : softmax numerators, then the selected linear term
// smem: at least kMaxTopK * kMaxGroup floats.
// When every block of the sequence is selected the unselected set is empty and o_bar - o_tilde is exactly zero;
// the difference of the two computed sums would only be rounding noise (which the RMSNorm would blow up), so
// the residual is set to zero in that case.
// `vu` indexes the workspace arrays, `ur` says which cache unit / query rows / length it stands for.
template <int D>
__device__ __forceinline__ void merge_unit(const Params& p, int vu, const UnitRef& ur, int n_items,
                                           const float* __restrict__ rms_weight, float* __restrict__ out,
                                           float* __restrict__ dbg_sparse, float* __restrict__ dbg_rla, float* smem) {
  constexpr int C4 = D / 4;                          // threads per head, one float4 of columns each
  constexpr int HG = kAttendThreads / C4;            // heads in flight
  constexpr int IU = 8;                              // items whose loads are in flight together
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.G;
  const int h = ur.h;
  const int nblk_u = (ur.L + p.B - 1) / p.B;
  const bool rla = !(p.flags & 4u) && p.n_sel[vu] < nblk_u;
  float* wt_s = smem;                                // [n_items][G]: exp2(m_it - M) / L

  // The first batch of partial results is requested before the weights are formed: the two are independent
  // and each costs one L2 round trip.
  const int hg = tid / C4, c4 = tid % C4;
  const float* parts = p.att_acc + (size_t)vu * p.top_k * 2 * G * D;
  float4 a[IU], t[IU];
  auto fetch = [&](int g, int it0) {
#pragma unroll
    for (int j = 0; j < IU; ++j) {
      const int it = it0 + j;
      if (it < n_items) {
        const float* pp = parts + (size_t)it * 2 * G * D;
        a[j] = __ldcg(reinterpret_cast<const float4*>(pp + (size_t)g * D) + c4);
        t[j] = rla ? __ldcg(reinterpret_cast<const float4*>(pp + (size_t)(G + g) * D) + c4) : make_float4(0.f, 0.f, 0.f, 0.f);
      } else {
        a[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        t[j] = a[j];
      }
    }
  };
  if (hg < G) fetch(hg, 0);

  // softmax weights of the items: one warp per head, lanes over items
  const float* ml_u = p.att_ml + (size_t)vu * p.top_k * G * 2;
  for (int g = warp; g < G; g += kAttendThreads / 32) {
    float m[2], l[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      const int it = lane + 32 * j;
      if (it < n_items) {
        const float2 v = __ldcg(reinterpret_cast<const float2*>(ml_u + ((size_t)it * G + g) * 2));
        m[j] = v.x; l[j] = v.y;
      } else {
        m[j] = -INFINITY; l[j] = 0.f;
      }
    }
    const float M = warp_max(fmaxf(m[0], m[1]));
    const float w0 = ex2(m[0] - M), w1 = ex2(m[1] - M);
    const float inv = 1.f / warp_sum(w0 * l[0] + w1 * l[1]);
    if (lane < n_items) wt_s[lane * G + g] = w0 * inv;
    if (lane + 32 < n_items) wt_s[(lane + 32) * G + g] = w1 * inv;
  }
  __syncthreads();

  for (int g0 = 0; g0 < G; g0 += HG) {
    const int g = g0 + hg;
    const bool live = g < G;
    float4 osp = make_float4(0.f, 0.f, 0.f, 0.f), otil = osp, obar = osp;
    if (live) {
      if (rla && ur.t >= 0) {                      // prefill: o_bar of this position, from the chunk scan
        obar = __ldcg(reinterpret_cast<const float4*>(p.vobar + (((size_t)ur.u * p.vTtot + ur.t) * G + g) * D) + c4);
      } else if (rla) {
#pragma unroll
        for (int s = 0; s < kStateSplits; ++s) {
          const float4 v = __ldcg(reinterpret_cast<const float4*>(p.obar_part + (((size_t)vu * kStateSplits + s) * G + g) * D) + c4);
          obar.x += v.x; obar.y += v.y; obar.z += v.z; obar.w += v.w;
        }
      }
      for (int it0 = 0; it0 < n_items; it0 += IU) {
        if (g0 > 0 || it0 > 0) fetch(g, it0);
#pragma unroll
        for (int j = 0; j < IU; ++j) {
          const int it = it0 + j;
          const float w = it < n_items ? wt_s[it * G + g] : 0.f;
          osp.x = fmaf(w, a[j].x, osp.x); osp.y = fmaf(w, a[j].y, osp.y);
          osp.z = fmaf(w, a[j].z, osp.z); osp.w = fmaf(w, a[j].w, osp.w);
          otil.x += t[j].x; otil.y += t[j].y; otil.z += t[j].z; otil.w += t[j].w;
        }
      }
    }
    const float4 r = make_float4(obar.x - otil.x, obar.y - otil.y, obar.z - otil.z, obar.w - otil.w);
    float sq = r.x * r.x + r.y * r.y + r.z * r.z + r.w * r.w;
#pragma unroll
    for (int o = C4 / 2; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);   // over the C4 lanes of this head
    if (live) {
      const size_t o = (ur.qrow + g) * D + c4 * 4;
      float4 res = osp;
      if (rla) {
        const float inv_rms = rsqrtf(sq / D + p.rms_eps);
        const float4 gm = *reinterpret_cast<const float4*>(rms_weight + ((size_t)h * G + g) * D + c4 * 4);
        res.x += gm.x * r.x * inv_rms; res.y += gm.y * r.y * inv_rms;
        res.z += gm.z * r.z * inv_rms; res.w += gm.w * r.w * inv_rms;
      }
      *reinterpret_cast<float4*>(out + o) = res;
      if (dbg_sparse) *reinterpret_cast<float4*>(dbg_sparse + o) = osp;
      if (dbg_rla) *reinterpret_cast<float4*>(dbg_rla + o) = r;
    }
  }
}

// Empty sequence: the output of the unit is zero.
template <int D>
__device__ __forceinline__ void write_zero_unit(const Params& p, const UnitRef& ur, float* out, float* dbg_sparse, float* dbg_rla) {
  for (int idx = threadIdx.x; idx < p.G * D; idx += blockDim.x) {
    const size_t o = ur.qrow * D + idx;
    out[o] = 0.f;
    if (dbg_sparse) dbg_sparse[o] = 0.f;
    if (dbg_rla) dbg_rla[o] = 0.f;
  }
}

}  // namespace spla
