// Block score + selection kernel, with the o_bar = phi(q) S_bar partials riding along as extra CTAs.
//
// Score (Section 3.1 of the paper): for query head m of the group and block i with n_i tokens,
//   ell^m_i = ln n_i + q_hat^m . mean_i + ln(1 + 1/2 sum_c (q_hat^m_c)^2 var_i[c])
// is the log of the second-order Taylor estimate of the block's attention mass; per head the masses are
// normalised over all blocks and the G heads are summed (Section 2.2).  One warp consumes one 2d-float
// statistics record with a single 128-bit load per lane for the mean and one for the variance.
//
// Selection (Section 2.1 Select; Section 4 forced sink/local blocks): the last CTA of a unit to finish
// (atomic ticket, no waiting) reduces the per-chunk normalisers, forms the aggregated score, and picks the
// top-k by an 8-bit radix select on the score bits followed by an index-ordered compaction.
#include "spla_internal.h"

namespace spla {

template <int D, int GP>
__global__ void __launch_bounds__(kScoreThreads) score_select_kernel(const Params p, const void* __restrict__ q_raw,
                                                                     int q_is_bf16, int* __restrict__ sel_user) {
  constexpr int VEC = D / 32;
  constexpr int NV = 2 * GP;             // values reduced per record: GP mean dots, GP variance dots
  constexpr int LPV = 32 / NV > 0 ? 32 / NV : 1;  // lanes holding a copy of each reduced value
  constexpr int NWARP = kScoreThreads / 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];

  const int u = blockIdx.y;
  const int b = u / p.Hkv, h = u % p.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.G;
  const int L = p.seq_lens[b];
  const int nblk = (L + p.B - 1) / p.B;
  const int n_chunks = max(1, (nblk + kScoreChunk - 1) / kScoreChunk);
  const int c = blockIdx.x;

  // ------------------------------------------------------------------ o_bar role ----------------------
  if (c >= p.n_chunks_cap) {
    const int s = c - p.n_chunks_cap;                      // which slice of the state's rows
    float* phiq = reinterpret_cast<float*>(smem_raw);      // [GP][D]
    float* red = phiq + GP * D;                            // [kScoreThreads / D][GP][D]
    const float a2 = p.phi_scale * kLog2e;
    for (int g = warp; g < G; g += NWARP) {
      float x[VEC];
      const size_t qoff = ((size_t)b * p.Hq + (size_t)h * G + g) * D + lane * VEC;
      if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
      else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
      float mx = -INFINITY;
#pragma unroll
      for (int v = 0; v < VEC; ++v) { x[v] *= a2; mx = fmaxf(mx, x[v]); }
      mx = warp_max(mx);
      float sum = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) { x[v] = exp2f(x[v] - mx); sum += x[v]; }
      sum = warp_sum(sum);
      const float inv = 1.f / sum;
#pragma unroll
      for (int v = 0; v < VEC; ++v) phiq[g * D + lane * VEC + v] = x[v] * inv;
    }
    __syncthreads();
    constexpr int RG = kScoreThreads / D;                  // row groups working side by side
    const int rg = tid / D, j = tid % D;
    const int rows = D / kStateSplits;
    const float* S = p.state + (size_t)u * D * D;
    float acc[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) acc[g] = 0.f;
    for (int r = s * rows + rg; r < (s + 1) * rows; r += RG) {
      const float sv = S[(size_t)r * D + j];
#pragma unroll
      for (int g = 0; g < GP; ++g)
        if (g < G) acc[g] = fmaf(phiq[g * D + r], sv, acc[g]);
    }
#pragma unroll
    for (int g = 0; g < GP; ++g) red[(rg * GP + g) * D + j] = acc[g];
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += kScoreThreads) {
      const int g = idx / D, jj = idx % D;
      float t = 0.f;
#pragma unroll
      for (int r2 = 0; r2 < RG; ++r2) t += red[(r2 * GP + g) * D + jj];
      p.obar_part[(((size_t)u * kStateSplits + s) * G + g) * D + jj] = t;
    }
    return;
  }

  // ------------------------------------------------------------------ score role ----------------------
  if (c >= n_chunks) return;

  // q_hat slices for the mean dot and 1/2 q_hat^2 for the variance dot, in registers.
  float qm[GP][VEC], qv[GP][VEC];
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    if (g < G) {
      float x[VEC];
      const size_t qoff = ((size_t)b * p.Hq + (size_t)h * G + g) * D + lane * VEC;
      if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
      else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        qm[g][v] = x[v] * p.sm_scale;
        qv[g][v] = (p.flags & 2u) ? 0.f : 0.5f * qm[g][v] * qm[g][v];
      }
    } else {
#pragma unroll
      for (int v = 0; v < VEC; ++v) { qm[g][v] = 0.f; qv[g][v] = 0.f; }
    }
  }

  const float* stats_u = p.stats + (size_t)u * p.max_blocks * 2 * D;
  float* ell_u = p.ell + (size_t)u * G * p.max_blocks;
  // Lanes 0..15 end up with the mean dots, lanes 16..31 with the variance dots; value index = lane / LPV.
  const int my_g = (lane & 15) / LPV;
  const bool writer = lane < 16 && (lane % LPV) == 0 && my_g < G;
  float run_max = -INFINITY, run_sum = 0.f;

  constexpr int RPW = kScoreChunk / NWARP;   // records per warp
  constexpr int UNR = 4;                     // records in flight per warp
  const int rec0 = c * kScoreChunk + warp * RPW;
#pragma unroll 1
  for (int r0 = 0; r0 < RPW; r0 += UNR) {
    float mean[UNR][VEC], var[UNR][VEC];
#pragma unroll
    for (int r = 0; r < UNR; ++r) {
      const int i = rec0 + r0 + r;
      if (i < nblk) {
        const float* rec = stats_u + (size_t)i * 2 * D;
        load_vec<VEC>(rec + lane * VEC, mean[r]);
        load_vec<VEC>(rec + D + lane * VEC, var[r]);
      } else {
#pragma unroll
        for (int v = 0; v < VEC; ++v) { mean[r][v] = 0.f; var[r][v] = 0.f; }
      }
    }
#pragma unroll
    for (int r = 0; r < UNR; ++r) {
      const int i = rec0 + r0 + r;
      float vals[NV];
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        float dm = 0.f, dv = 0.f;
#pragma unroll
        for (int v = 0; v < VEC; ++v) {
          dm = fmaf(qm[g][v], mean[r][v], dm);
          dv = fmaf(qv[g][v], var[r][v], dv);
        }
        vals[g] = dm;
        vals[GP + g] = dv;
      }
      warp_reduce_multi<NV>(vals, lane);
      const float other = __shfl_xor_sync(0xffffffffu, vals[0], 16);   // variance dot of the same head
      if (writer && i < nblk) {
        const int n_i = min(p.B, L - i * p.B);
        const float ell = __logf((float)n_i) + vals[0] + log1pf(other);
        ell_u[(size_t)my_g * p.max_blocks + i] = ell;
        const float nm = fmaxf(run_max, ell);
        run_sum = run_sum * __expf(run_max - nm) + __expf(ell - nm);
        run_max = nm;
      }
    }
  }

  // per-chunk (max, sum exp) per head
  float* wred = reinterpret_cast<float*>(smem_raw);     // [NWARP][GP][2]
  __shared__ int is_last_s;
  if (writer) {
    wred[(warp * GP + my_g) * 2 + 0] = run_max;
    wred[(warp * GP + my_g) * 2 + 1] = run_sum;
  }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY, s = 0.f;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) {
      const float wm = wred[(w * GP + tid) * 2], ws = wred[(w * GP + tid) * 2 + 1];
      const float nm = fmaxf(m, wm);
      if (nm > -INFINITY) s = s * __expf(m - nm) + ws * __expf(wm - nm);
      m = nm;
    }
    float* cp = p.chunk_part + (((size_t)u * p.max_chunks + c) * G + tid) * 2;
    cp[0] = m;
    cp[1] = s;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int t = atomicAdd(&p.score_ticket[u], 1);
    is_last_s = (t == n_chunks - 1);
    if (is_last_s) p.score_ticket[u] = 0;                // ready for the next decode step
  }
  __syncthreads();
  if (!is_last_s) return;
  __threadfence();

  // ------------------------------------------------------------------ selection (one CTA per unit) ----
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);           // [max_blocks]
  __shared__ float lse_s[kMaxGroup];
  __shared__ int hist[256];
  __shared__ int wtot[2][NWARP];
  __shared__ uint32_t sel_digit_s;
  __shared__ int sel_k_s;

  for (int g = warp; g < G; g += NWARP) {
    float m = -INFINITY, s = 0.f;
    for (int cc = lane; cc < n_chunks; cc += 32) {
      const float* cp = p.chunk_part + (((size_t)u * p.max_chunks + cc) * G + g) * 2;
      const float cm = __ldcg(cp), cs = __ldcg(cp + 1);
      const float nm = fmaxf(m, cm);
      if (nm > -INFINITY) s = s * __expf(m - nm) + cs * __expf(cm - nm);
      m = nm;
    }
    const float M = warp_max(m);
    s = (m > -INFINITY) ? s * __expf(m - M) : 0.f;
    s = warp_sum(s);
    if (lane == 0) lse_s[g] = M + __logf(s);
  }
  __syncthreads();

  const int k_eff = min(p.top_k, nblk);
  float* scores_u = p.scores + (size_t)u * p.max_blocks;
  for (int i = tid; i < nblk; i += kScoreThreads) {
    float sc = 0.f;
    for (int g = 0; g < G; ++g) sc += __expf(__ldcg(ell_u + (size_t)g * p.max_blocks + i) - lse_s[g]);
    scores_u[i] = sc;
    const bool forced = (i < p.n_sink) || (i >= nblk - p.n_local);
    keys[i] = forced ? 0xffffffffu : __float_as_uint(sc);
  }
  __syncthreads();

  // radix select: the k_eff-th largest key
  uint32_t prefix = 0, mask = 0;
  int kk = k_eff;
  if (k_eff > 0) {
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      hist[tid] = 0;                                                   // kScoreThreads == 256 bins
      __syncthreads();
      for (int i = tid; i < nblk; i += kScoreThreads) {
        const uint32_t key = keys[i];
        if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1);
      }
      __syncthreads();
      if (warp == 0) {
        int bins[8], tot = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { bins[j] = hist[lane * 8 + j]; tot += bins[j]; }
        int above = tot;                                               // inclusive suffix sum over lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, above, o);
          if (lane + o < 32) above += t;
        }
        above -= tot;                                                  // keys in bins of higher lanes
        if (above < kk && kk <= above + tot) {
          int cum = above;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (cum < kk && kk <= cum + bins[j]) { sel_digit_s = lane * 8 + j; sel_k_s = kk - cum; }
            cum += bins[j];
          }
        }
      }
      __syncthreads();
      prefix |= sel_digit_s << shift;
      mask |= 0xffu << shift;
      kk = sel_k_s;
      __syncthreads();
    }
  }
  const uint32_t T = prefix;   // threshold key; kk = how many keys equal to T are taken (lowest indices first)

  // index-ordered compaction
  const int per = (nblk + kScoreThreads - 1) / kScoreThreads;
  const int i0 = tid * per, i1 = min(nblk, i0 + per);
  int n_gt = 0, n_eq = 0;
  for (int i = i0; i < i1; ++i) {
    const uint32_t key = keys[i];
    n_gt += key > T;
    n_eq += key == T;
  }
  int s_gt = n_gt, s_eq = n_eq;                                        // inclusive scans within the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, s_gt, o), e = __shfl_up_sync(0xffffffffu, s_eq, o);
    if (lane >= o) { s_gt += a; s_eq += e; }
  }
  if (lane == 31) { wtot[0][warp] = s_gt; wtot[1][warp] = s_eq; }
  __syncthreads();
  int gt_before = s_gt - n_gt, eq_before = s_eq - n_eq;
  for (int w = 0; w < warp; ++w) { gt_before += wtot[0][w]; eq_before += wtot[1][w]; }
  int* sel_u = p.sel + (size_t)u * p.top_k;
  int* sel_o = sel_user ? sel_user + (size_t)u * p.top_k : nullptr;
  if (k_eff > 0) {
    for (int i = i0; i < i1; ++i) {
      const uint32_t key = keys[i];
      const bool take = key > T || (key == T && eq_before < kk);
      if (take) {
        const int slot = gt_before + min(eq_before, kk);
        sel_u[slot] = i;
        if (sel_o) sel_o[slot] = i;
      }
      gt_before += key > T;
      eq_before += key == T;
    }
  }
  for (int t = k_eff + tid; t < p.top_k; t += kScoreThreads) {
    sel_u[t] = -1;
    if (sel_o) sel_o[t] = -1;
  }
  if (tid == 0) p.n_sel[u] = k_eff;
}

template <int D, int GP>
static cudaError_t launch_one(const Params& p, const void* q, int q_is_bf16, int* sel_user, cudaStream_t stream) {
  const int U = p.batch * p.Hkv;
  const bool rla = !(p.flags & 4u);
  dim3 grid(p.n_chunks_cap + (rla ? kStateSplits : 0), U);
  size_t smem = (size_t)p.max_blocks * sizeof(uint32_t);
  const size_t smem_state = (size_t)(GP * D + (kScoreThreads / D) * GP * D) * sizeof(float);
  if (smem_state > smem) smem = smem_state;
  const size_t smem_wred = (size_t)(kScoreThreads / 32) * GP * 2 * sizeof(float);
  if (smem_wred > smem) smem = smem_wred;
  auto kern = score_select_kernel<D, GP>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, kScoreThreads, smem, stream>>>(p, q, q_is_bf16, sel_user);
  return cudaGetLastError();
}

template <int D>
static cudaError_t launch_d(const Params& p, int GP, const void* q, int qb, int* sel_user, cudaStream_t s) {
  switch (GP) {
    case 1: return launch_one<D, 1>(p, q, qb, sel_user, s);
    case 2: return launch_one<D, 2>(p, q, qb, sel_user, s);
    case 4: return launch_one<D, 4>(p, q, qb, sel_user, s);
    case 8: return launch_one<D, 8>(p, q, qb, sel_user, s);
    default: return launch_one<D, 16>(p, q, qb, sel_user, s);
  }
}

cudaError_t launch_score_select(const Params& p, const void* q, int q_is_bf16, int* sel_user, cudaStream_t stream) {
  const int GP = padded_group(p.G);
  return p.d == 128 ? launch_d<128>(p, GP, q, q_is_bf16, sel_user, stream)
                    : launch_d<64>(p, GP, q, q_is_bf16, sel_user, stream);
}

}  // namespace spla
