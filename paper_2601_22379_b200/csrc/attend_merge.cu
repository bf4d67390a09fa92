// Sparse attention over the selected blocks with the residual-linear-attention subtraction fused in, and
// the split-K merge done by the last CTA of every unit.
//
// One CTA per (unit, selected block).  The block's K and V tiles (contiguous in the cache) and its per-token
// log-sum-exp are staged into shared memory with one bulk asynchronous copy each.  From the SAME tiles the CTA
// forms, for every query head of the group,
//   exact branch  (Section 2.2, Eq. gqa-sparse):  m, l = sum_t exp(s_t - m), acc = sum_t exp(s_t - m) v_t
//   linear branch (Section 3.2, Eq. rla-impl-2):  o_tilde partial = sum_t (phi(q) . phi(k_t)) v_t
// so the selected linear term costs no extra memory traffic and unselected blocks are never read.
// The last CTA of the unit (atomic ticket, nobody waits) merges the partials, subtracts o_tilde from
// o_bar = phi(q) S_bar (Eq. rla-impl-3), applies the RMSNorm and adds the two branches (Section 3.3).
#include "attend_common.cuh"
#include "spla_internal.h"

namespace spla {

template <typename T, int D, int GP>
__global__ void __launch_bounds__(kAttendThreads) attend_merge_kernel(const Params p, const void* __restrict__ q_raw,
                                                                      int q_is_bf16, const float* __restrict__ rms_weight,
                                                                      float* __restrict__ out, float* __restrict__ dbg_sparse,
                                                                      float* __restrict__ dbg_rla) {
  constexpr int VEC = D / 32;
  constexpr int NV = 2 * GP;
  constexpr int LPV = 32 / NV > 0 ? 32 / NV : 1;
  constexpr int NWARP = kAttendThreads / 32;
  constexpr int TS = kAttendThreads / D;        // token slices in the value pass
  extern __shared__ __align__(128) unsigned char smem_raw[];

  const int vu = blockIdx.y, item = blockIdx.x;     // vu: index into the workspace (a virtual unit in a prefill launch)
  const UnitRef ur = unit_ref(p, vu);
  const int u = ur.u;                               // the cache's unit
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.G, B = p.B;
  const bool rla = !(p.flags & 4u);

  const int nsel = p.n_sel[vu];
  if (item >= nsel) {
    if (nsel == 0 && item == 0) write_zero_unit<D>(p, ur, out, dbg_sparse, dbg_rla);   // empty sequence
    return;
  }
  const int blk = p.sel[(size_t)vu * p.top_k + item];
  const int L = ur.L;
  int n_tok = min(B, L - blk * B);
  if ((p.flags & kDebugBounds) && (blk < 0 || blk >= p.max_blocks || n_tok <= 0)) {
    // checked build: a block index that does not name a cached block is reported and the block is treated as empty
    if (tid == 0) atomicExch(p.status, kStatusBounds);
    n_tok = 0;
  }
  const bool fetch = n_tok > 0;

  // shared memory carve-up
  T* Ks = reinterpret_cast<T*>(smem_raw);
  T* Vs = Ks + (size_t)B * D;
  float* lse_s = reinterpret_cast<float*>(Vs + (size_t)B * D);   // [B]
  float* w_s = lse_s + B;                                         // [B][NV]: logits then weights, linear coefficients
  float* misc = w_s + (size_t)B * NV;                             // [2 * GP] (m, l) then scratch
  uint64_t* bar = reinterpret_cast<uint64_t*>(misc + 4 * GP + 2 * NWARP * GP);
  __shared__ int flag_s;

  if (tid == 0 && !fetch) { mbar_init(bar, 1); mbar_init_done(); }
  if (tid == 0 && fetch) {
    mbar_init(bar, 1);
    mbar_init_done();
    const size_t tile = (size_t)u * p.max_blocks + blk;
    const uint32_t tile_bytes = (uint32_t)((size_t)B * D * sizeof(T));
    mbar_expect_tx(bar, 2 * tile_bytes + (uint32_t)(B * sizeof(float)) + (uint32_t)p.dbg_tx_extra);
    bulk_g2s(Ks, reinterpret_cast<const T*>(p.k_cache) + tile * B * D, tile_bytes, bar);
    bulk_g2s(Vs, reinterpret_cast<const T*>(p.v_cache) + tile * B * D, tile_bytes, bar);
    bulk_g2s(lse_s, p.tok_lse + tile * B, (uint32_t)(B * sizeof(float)), bar);
  }

  // Query slices while the copies fly: q2 = q * sm_scale * log2(e) for the logits (base-2 domain),
  // fq = phi(q) = softmax(phi_scale * q) for the linear branch.
  float q2[GP][VEC], fq[GP][VEC];
  const float a2 = p.phi_scale * kLog2e;
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    if (g < G) {
      float x[VEC];
      const size_t qoff = (ur.qrow + g) * D + lane * VEC;
      if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
      else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
      float mx = -INFINITY;
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        q2[g][v] = x[v] * (p.sm_scale * kLog2e);
        fq[g][v] = x[v] * a2;
        mx = fmaxf(mx, fq[g][v]);
      }
      mx = warp_max(mx);
      float sum = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) { fq[g][v] = exp2f(fq[g][v] - mx); sum += fq[g][v]; }
      sum = warp_sum(sum);
      const float inv = rla ? 1.f / sum : 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) fq[g][v] *= inv;
    } else {
#pragma unroll
      for (int v = 0; v < VEC; ++v) { q2[g][v] = 0.f; fq[g][v] = 0.f; }
    }
  }
  __syncthreads();                               // barrier initialised before anyone polls it
  bool arrived = fetch && mbar_wait(bar, 0, p.wait_limit);
  if (fetch && !arrived) {                                // never expected: report it, give the copies a second bounded wait, skip the math
    if (tid == 0) atomicExch(p.status, kStatusTimeout);
    mbar_wait(bar, 0, p.wait_limit);
  }

  // ---- pass 1: logits and linear coefficients per token ----------------------------------------------
  const int my_idx = lane / LPV;
  const bool writer = (lane % LPV) == 0;
  if (arrived) {
    for (int t = warp; t < n_tok; t += NWARP) {
      float k[VEC];
      load_vec<VEC>(Ks + (size_t)t * D + lane * VEC, k);
      const float lse2 = lse_s[t] * kLog2e;
      float e[VEC];
#pragma unroll
      for (int v = 0; v < VEC; ++v) e[v] = ex2(fmaf(k[v], a2, -lse2));      // phi(k_t)[c]
      float vals[NV];
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        float s = 0.f, a = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          s = fmaf(q2[g][v], k[v], s);
          a = fmaf(fq[g][v], e[v], a);
        }
        vals[g] = s;
        vals[GP + g] = a;
      }
      warp_reduce_multi<NV>(vals, lane);
      if (writer) w_s[t * NV + my_idx] = vals[0];
    }
  }
  __syncthreads();

  // ---- per-head softmax statistics over the block's tokens -------------------------------------------
  float* m_s = misc;            // [GP]
  float* l_s = misc + GP;       // [GP]
  for (int g = warp; g < G; g += NWARP) {
    float m = -INFINITY;
    for (int t = lane; t < n_tok; t += 32) m = fmaxf(m, w_s[t * NV + g]);
    m = warp_max(m);
    float l = 0.f;
    for (int t = lane; t < n_tok; t += 32) {
      const float pw = ex2(w_s[t * NV + g] - m);
      w_s[t * NV + g] = pw;
      l += pw;
    }
    l = warp_sum(l);
    if (lane == 0) { m_s[g] = m; l_s[g] = l; }
  }
  __syncthreads();

  // (kept in registers: with small tiles the fold buffer of pass 2 reaches over the statistics in shared memory)
  float my_m = 0.f, my_l = 0.f;
  if (tid < G) { my_m = m_s[tid]; my_l = l_s[tid]; }

  // ---- pass 2: both branches share the V tile ---------------------------------------------------------
  const int ts = tid / D, col = tid % D;
  float acc[NV];
#pragma unroll
  for (int i = 0; i < NV; ++i) acc[i] = 0.f;
  if (arrived) {
    for (int t = ts; t < n_tok; t += TS) {
      const float v = to_float(Vs[(size_t)t * D + col]);
      float w[NV];                                                     // same address for every thread: broadcast
      if constexpr (NV % 4 == 0) {
#pragma unroll
        for (int i = 0; i < NV / 4; ++i) {
          const float4 x = reinterpret_cast<const float4*>(w_s + t * NV)[i];
          w[4 * i] = x.x; w[4 * i + 1] = x.y; w[4 * i + 2] = x.z; w[4 * i + 3] = x.w;
        }
      } else {
        const float2 x = *reinterpret_cast<const float2*>(w_s + t * NV);
        w[0] = x.x; w[1] = x.y;
      }
#pragma unroll
      for (int i = 0; i < NV; ++i) acc[i] = fmaf(w[i], v, acc[i]);
    }
  }
  if constexpr (TS > 1) {        // fold the token slices together through shared memory (tiles are no longer needed)
    float* red = reinterpret_cast<float*>(smem_raw);                 // [TS][NV][D]
    __syncthreads();
#pragma unroll
    for (int i = 0; i < NV; ++i) red[((size_t)ts * NV + i) * D + col] = acc[i];
    __syncthreads();
    if (ts == 0) {
#pragma unroll
      for (int i = 0; i < NV; ++i) {
        float t2 = 0.f;
        for (int s2 = 0; s2 < TS; ++s2) t2 += red[((size_t)s2 * NV + i) * D + col];
        acc[i] = t2;
      }
    }
  }

  // ---- partial results of this block -------------------------------------------------------------------
  float* part = p.att_acc + ((size_t)vu * p.top_k + item) * 2 * G * D;
  if (ts == 0) {
#pragma unroll
    for (int g = 0; g < GP; ++g) {
      if (g < G) {
        part[(size_t)g * D + col] = acc[g];
        part[(size_t)(G + g) * D + col] = acc[GP + g];
      }
    }
  }
  if (tid < G) {
    float* ml = p.att_ml + (((size_t)vu * p.top_k + item) * G + tid) * 2;
    ml[0] = my_m;
    ml[1] = my_l;
  }
  if (!arrive_last(&p.attend_ticket[vu], nsel, &flag_s)) return;

  // ---- merge (last CTA of the unit) ---------------------------------------------------------------------
  merge_unit<D>(p, vu, ur, nsel, rms_weight, out, dbg_sparse, dbg_rla, reinterpret_cast<float*>(smem_raw));
}

// Takes a caller-given selection into the workspace.  The list is not trusted: only entries that name an existing
// block of the sequence (0 <= index < ceil(L / B)) and that are not repeated are kept, in the order given, packed to
// the front; the rest of the row is padded with -1.  Anything dropped other than the -1 padding at the tail (a hole,
// an index past the last block, a duplicate) is reported through the status word, and nothing outside the cache is
// ever addressed because of it.  One CTA of kMaxTopK threads per unit.
__global__ void __launch_bounds__(kMaxTopK) adopt_selection_kernel(const Params p, const int* __restrict__ sel_in) {
  const int u = blockIdx.x, b = u / p.Hkv, t = threadIdx.x;
  __shared__ int raw_s[kMaxTopK];
  __shared__ int keep_s[kMaxTopK];
  const int nblk = (checked_len(p, b) + p.B - 1) / p.B;
  const int v = t < p.top_k ? sel_in[(size_t)u * p.top_k + t] : -1;
  raw_s[t] = v;
  __syncthreads();
  bool keep = v >= 0 && v < nblk;
  for (int j = 0; keep && j < t; ++j) keep = raw_s[j] != v;          // a repeated block would be attended to twice
  keep_s[t] = keep;
  __syncthreads();
  int pos = 0, total = 0, last_given = -1;
  for (int j = 0; j < p.top_k; ++j) {
    pos += (j < t) && keep_s[j];
    total += keep_s[j];
    if (raw_s[j] != -1) last_given = j;
  }
  if (keep) p.sel[(size_t)u * p.top_k + pos] = v;
  if (t >= total && t < p.top_k) p.sel[(size_t)u * p.top_k + t] = -1;
  if (t == 0) {
    p.n_sel[u] = total;
    if (total != last_given + 1) atomicExch(p.status, kStatusBounds);   // something other than tail padding was dropped
  }
}

template <typename T, int D, int GP>
static cudaError_t launch_one(const Params& p, const void* q, int qb, const float* w, float* out, float* ds, float* dr,
                              cudaStream_t stream) {
  constexpr int NV = 2 * GP;
  constexpr int NWARP = kAttendThreads / 32;
  size_t smem = (size_t)2 * p.B * D * sizeof(T) + (size_t)p.B * sizeof(float) + (size_t)p.B * NV * sizeof(float) +
                (size_t)(4 * GP + 2 * NWARP * GP) * sizeof(float) + 16;
  const size_t smem_merge = (size_t)(kMaxTopK * kMaxGroup) * sizeof(float);
  if (smem_merge > smem) smem = smem_merge;
  const size_t smem_red = (size_t)(kAttendThreads / D) * NV * D * sizeof(float);
  if (smem_red > smem) smem = smem_red;
  auto kern = attend_merge_kernel<T, D, GP>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid(p.top_k, p.batch * p.Hkv * (p.vT > 0 ? p.vT : 1));
  kern<<<grid, kAttendThreads, smem, stream>>>(p, q, qb, w, out, ds, dr);
  ++g_launch_count;
  return cudaGetLastError();
}

template <typename T, int D>
static cudaError_t launch_g(const Params& p, int GP, const void* q, int qb, const float* w, float* out, float* ds,
                            float* dr, cudaStream_t s) {
  switch (GP) {
    case 1: return launch_one<T, D, 1>(p, q, qb, w, out, ds, dr, s);
    case 2: return launch_one<T, D, 2>(p, q, qb, w, out, ds, dr, s);
    case 4: return launch_one<T, D, 4>(p, q, qb, w, out, ds, dr, s);
    case 8: return launch_one<T, D, 8>(p, q, qb, w, out, ds, dr, s);
    default: return launch_one<T, D, 16>(p, q, qb, w, out, ds, dr, s);
  }
}

cudaError_t launch_attend_merge(const Params& p, const AttendMaps* maps, const void* q, int q_is_bf16,
                                const float* rms_weight, const int* sel_in, float* out, float* dbg_o_sparse,
                                float* dbg_o_rla, cudaStream_t stream) {
  if (sel_in) {
    adopt_selection_kernel<<<p.batch * p.Hkv, kMaxTopK, 0, stream>>>(p, sel_in);
    ++g_launch_count;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
  }
  if (p.kv_bf16 && q_is_bf16 && p.G <= 8 && maps && maps->valid && p.acs > 0)
    return launch_attend_mma(p, *maps, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream);
  const int GP = padded_group(p.G);
  if (p.kv_bf16) {
    return p.d == 128 ? launch_g<__nv_bfloat16, 128>(p, GP, q, q_is_bf16, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream)
                      : launch_g<__nv_bfloat16, 64>(p, GP, q, q_is_bf16, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream);
  }
  return p.d == 128 ? launch_g<float, 128>(p, GP, q, q_is_bf16, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream)
                    : launch_g<float, 64>(p, GP, q, q_is_bf16, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream);
}

}  // namespace spla
