// Prefill- / training-shaped forward: the output of every query position of a chunk of T new tokens.
//
// The paper develops the method on the decode step and says that it carries over to training and prefilling
// (Section 2, opening; Section 3.3 "Kernel Design": the kernels serve both).  The reading taken: the query at
// position t sees exactly the cache a decode step at t would see - tokens 0..t, the block statistics, the selection
// and the recurrent state of that prefix.  This file holds what that needs beyond the decode kernels:
//   * prefix statistics: for every position the mean / variance of its own, still growing block as of that position
//     (Section 3.1, Eq. taylor-2nd); completed blocks keep the records the append wrote;
//   * the chunk scan: o_bar_t = phi(q_t) S_bar_t for every position, S_bar_t = S_bar_{t-1} + phi(k_t)^T v_t
//     (Section 3.2, Eq. rla-impl-1), as a chunked linear-attention scan: per sub-chunk of 32 positions the part that
//     comes from the state before the sub-chunk is one product with the state, the causal part inside it a masked
//     32 x 32 product, and the state then takes the sub-chunk's rank-32 update; the scan also leaves S_bar of the
//     whole chunk in the cache, i.e. it is this call's state update.
// Scoring, selection, exact attention, the subtraction and the merge then run in the general decode kernels with
// one *virtual unit* per (sequence, KV head, position): same arithmetic, a per-position length.
#include "spla_internal.h"

namespace spla {

namespace {

constexpr int kPfThreads = 256;
constexpr int kSub = 32;                       // positions per sub-chunk of the scan

// One CTA per (block touched by the chunk, unit).  The block's keys (as cached: the append has run) are staged in
// shared memory as fp32; then, for every chunk position inside the block, the statistics of the block's tokens up to
// and including that position: mean, then population variance (1/n), two passes, the same summation order as the
// append kernels use for the cache's own records, so that a position's record equals what a token-by-token append
// would have left in the cache at that point.
template <typename T, int D>
__global__ void __launch_bounds__(kPfThreads) prefill_stats_kernel(const Params p, int Ttot, float* __restrict__ vstats) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* tile = reinterpret_cast<float*>(smem_raw);            // [B][D]
  __shared__ float red_s[kPfThreads / D][D];
  __shared__ float mean_s[D];
  constexpr int TG = kPfThreads / D;
  const int tid = threadIdx.x;
  const int u = blockIdx.y, b = u / p.Hkv;
  const int L_end = checked_len(p, b);
  const int L0 = max(0, L_end - Ttot);                          // first chunk position
  const int blk = L0 / p.B + blockIdx.x;
  const int t0 = blk * p.B;
  if (t0 >= L_end) return;                                      // CTA-uniform
  const int cnt = min(p.B, L_end - t0);
  const T* kc = reinterpret_cast<const T*>(p.k_cache) + ((size_t)u * p.max_blocks * p.B + t0) * D;
  for (int idx = tid; idx < cnt * D; idx += kPfThreads) tile[idx] = to_float(kc[idx]);
  __syncthreads();
  const int tg = tid / D, c = tid % D;
  const bool round16 = (p.flags & kStatsBf16) != 0;
  for (int pos = max(t0, L0); pos < t0 + cnt; ++pos) {
    const int n = pos - t0 + 1;                                 // tokens of the block as of this position
    float sum = 0.f;
    for (int t = tg; t < n; t += TG) sum += tile[(size_t)t * D + c];
    red_s[tg][c] = sum;
    __syncthreads();
    if (tg == 0) {
      float tot = 0.f;
#pragma unroll
      for (int g2 = 0; g2 < TG; ++g2) tot += red_s[g2][c];
      mean_s[c] = tot / (float)n;
    }
    __syncthreads();
    const float mean = mean_s[c];
    float ss = 0.f;
    for (int t = tg; t < n; t += TG) {
      const float dv = tile[(size_t)t * D + c] - mean;
      ss = fmaf(dv, dv, ss);
    }
    __syncthreads();
    red_s[tg][c] = ss;
    __syncthreads();
    if (tg == 0) {
      float tot = 0.f;
#pragma unroll
      for (int g2 = 0; g2 < TG; ++g2) tot += red_s[g2][c];
      float m = mean, v = tot / (float)n;
      if (round16) { m = __bfloat162float(__float2bfloat16_rn(m)); v = __bfloat162float(__float2bfloat16_rn(v)); }
      float* rec = vstats + ((size_t)u * Ttot + (pos - L0)) * 2 * D;
      rec[c] = m;
      rec[D + c] = v;
    }
    __syncthreads();
  }
}

// The chunk scan, one CTA per unit (sequential over the sub-chunks, the state in shared memory).
//   S      [D][D]      running state (row = feature of phi(k), column = value channel)
//   fk     [kSub][D]   phi(k_j) of the sub-chunk          vv [kSub][D]  v_j
//   fq     [kSub][D]   phi(q_i) of one head               aa [kSub][kSub]  phi(q_i) . phi(k_j), j <= i
// Thread (ig, c4): rows i = ig, ig + 8, ... of the sub-chunk, columns 4 c4 .. 4 c4 + 3 (D = 128: 32 column quads x 8
// row groups; D = 64: 16 quads x 16 groups).
template <typename T, int D>
__global__ void __launch_bounds__(kPfThreads) prefill_scan_kernel(const Params p, int Ttot, const void* __restrict__ q_raw,
                                                                  int q_is_bf16, float* __restrict__ vobar) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* S = reinterpret_cast<float*>(smem_raw);               // [D][D]
  float* fk = S + D * D;                                       // [kSub][D]
  float* vv = fk + kSub * D;                                   // [kSub][D]
  float* fq = vv + kSub * D;                                   // [kSub][D]
  float* aa = fq + kSub * D;                                   // [kSub][kSub + 1]
  constexpr int CQ = D / 4;                                    // column quads
  constexpr int IG = kPfThreads / CQ;                          // row groups
  constexpr int RPT = kSub / IG;                               // sub-chunk rows per thread
  constexpr int VEC = D / 32;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.x, b = u / p.Hkv, h = u % p.Hkv;
  const int G = p.G;
  const int L_end = checked_len(p, b);
  const int L0 = max(0, L_end - Ttot);
  const int n_pos = L_end - L0;                                // = Ttot unless the cache holds fewer tokens
  const float a2 = p.phi_scale * kLog2e;
  const size_t unit_tok0 = (size_t)u * p.max_blocks * p.B;
  const T* kc = reinterpret_cast<const T*>(p.k_cache) + unit_tok0 * D;
  const T* vc = reinterpret_cast<const T*>(p.v_cache) + unit_tok0 * D;
  float* Sg = p.state + (size_t)u * D * D;
  for (int idx = tid; idx < D * D; idx += kPfThreads) S[idx] = Sg[idx];
  const int c4 = tid % CQ, ig = tid / CQ;
  __syncthreads();

  for (int s0 = 0; s0 < n_pos; s0 += kSub) {
    const int ns = min(kSub, n_pos - s0);
    // phi(k_j) and v_j of the sub-chunk (rows past its end are zero)
    for (int idx = tid; idx < kSub * D; idx += kPfThreads) {
      const int j = idx / D, c = idx % D;
      float f = 0.f, v = 0.f;
      if (j < ns) {
        const size_t pos = (size_t)(L0 + s0 + j);
        f = ex2(fmaf(to_float(kc[pos * D + c]), a2, -p.tok_lse[unit_tok0 + pos] * kLog2e));
        v = to_float(vc[pos * D + c]);
      }
      fk[idx] = f;
      vv[idx] = v;
    }
    for (int g = 0; g < G; ++g) {
      __syncthreads();                                         // fk / vv written; the previous head is done with fq / aa
      // phi(q_i) of head g for the sub-chunk's positions: one warp per position
      for (int i = warp; i < kSub; i += kPfThreads / 32) {
        float x[VEC];
        if (i < ns) {
          const size_t qoff = (((size_t)b * Ttot + (s0 + i)) * p.Hq + (size_t)h * G + g) * D + lane * VEC;
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
          for (int v = 0; v < VEC; ++v) fq[i * D + lane * VEC + v] = x[v] * inv;
        } else {
#pragma unroll
          for (int v = 0; v < VEC; ++v) fq[i * D + lane * VEC + v] = 0.f;
        }
      }
      __syncthreads();
      // causal coefficients inside the sub-chunk: aa[i][j] = phi(q_i) . phi(k_j) for j <= i
      for (int idx = tid; idx < kSub * kSub; idx += kPfThreads) {
        const int i = idx / kSub, j = idx % kSub;
        float a = 0.f;
        if (j <= i && i < ns) {
          const float4* x = reinterpret_cast<const float4*>(fq + i * D);
          const float4* y = reinterpret_cast<const float4*>(fk + j * D);
#pragma unroll 8
          for (int c = 0; c < D / 4; ++c) {
            const int cc = (c + j) % (D / 4);                   // rotated start: the lanes of a warp (different j) hit different banks
            const float4 xa = x[cc], ya = y[cc];
            a = fmaf(xa.x, ya.x, a); a = fmaf(xa.y, ya.y, a); a = fmaf(xa.z, ya.z, a); a = fmaf(xa.w, ya.w, a);
          }
        }
        aa[i * (kSub + 1) + j] = a;
      }
      __syncthreads();
      // o_bar of the thread's rows and columns: the state before the sub-chunk, then the causal part
      float acc[RPT][4];
#pragma unroll
      for (int r = 0; r < RPT; ++r) { acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f; }
#pragma unroll 4
      for (int k = 0; k < D; ++k) {
        const float4 sv = *reinterpret_cast<const float4*>(S + (size_t)k * D + c4 * 4);
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
          const float f = fq[(ig + r * IG) * D + k];
          acc[r][0] = fmaf(f, sv.x, acc[r][0]); acc[r][1] = fmaf(f, sv.y, acc[r][1]);
          acc[r][2] = fmaf(f, sv.z, acc[r][2]); acc[r][3] = fmaf(f, sv.w, acc[r][3]);
        }
      }
      for (int j = 0; j < ns; ++j) {
        const float4 v4 = *reinterpret_cast<const float4*>(vv + (size_t)j * D + c4 * 4);
#pragma unroll
        for (int r = 0; r < RPT; ++r) {
          const float a = aa[(ig + r * IG) * (kSub + 1) + j];     // zero above the diagonal
          acc[r][0] = fmaf(a, v4.x, acc[r][0]); acc[r][1] = fmaf(a, v4.y, acc[r][1]);
          acc[r][2] = fmaf(a, v4.z, acc[r][2]); acc[r][3] = fmaf(a, v4.w, acc[r][3]);
        }
      }
#pragma unroll
      for (int r = 0; r < RPT; ++r) {
        const int i = ig + r * IG;
        if (i < ns)
          *reinterpret_cast<float4*>(vobar + (((size_t)u * Ttot + (s0 + i)) * G + g) * D + c4 * 4) =
              make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
      }
    }
    __syncthreads();                                           // every head has read S
    // state update: S[k][c] += sum_j phi(k_j)[k] v_j[c]; thread (ig, c4) takes rows k = ig, ig + IG, ...
    for (int k = ig; k < D; k += IG) {
      float4 sv = *reinterpret_cast<float4*>(S + (size_t)k * D + c4 * 4);
      for (int j = 0; j < ns; ++j) {
        const float f = fk[j * D + k];
        const float4 v4 = *reinterpret_cast<const float4*>(vv + (size_t)j * D + c4 * 4);
        sv.x = fmaf(f, v4.x, sv.x); sv.y = fmaf(f, v4.y, sv.y); sv.z = fmaf(f, v4.z, sv.z); sv.w = fmaf(f, v4.w, sv.w);
      }
      *reinterpret_cast<float4*>(S + (size_t)k * D + c4 * 4) = sv;
    }
    __syncthreads();
  }
  for (int idx = tid; idx < D * D; idx += kPfThreads) Sg[idx] = S[idx];
}

template <typename T, int D>
cudaError_t launch_typed(const Params& p, int Ttot, const void* q, int q_is_bf16, float* vstats, float* vobar, cudaStream_t stream) {
  const int U = p.batch * p.Hkv;
  {
    const size_t smem = (size_t)p.B * D * sizeof(float);
    auto kern = prefill_stats_kernel<T, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<dim3((Ttot + p.B - 1) / p.B + 1, U), kPfThreads, smem, stream>>>(p, Ttot, vstats);
    ++g_launch_count;
  }
  if (!(p.flags & 4u)) {
    const size_t smem = (size_t)(D * D + 3 * kSub * D + kSub * (kSub + 1)) * sizeof(float);
    auto kern = prefill_scan_kernel<T, D>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<U, kPfThreads, smem, stream>>>(p, Ttot, q, q_is_bf16, vobar);
    ++g_launch_count;
  }
  return cudaGetLastError();
}

}  // namespace

// Runs after the chunk's K/V, per-token log-sum-exp, block statistics and lengths are in the cache, with S_bar still the
// state BEFORE the chunk: fills vstats [U][T][2][d] and vobar [U][T][G][d] and advances S_bar over the chunk.
cudaError_t launch_prefill_prepare(const Params& p, int Ttot, const void* q, int q_is_bf16, float* vstats, float* vobar,
                                   cudaStream_t stream) {
  if (p.kv_bf16)
    return p.d == 128 ? launch_typed<__nv_bfloat16, 128>(p, Ttot, q, q_is_bf16, vstats, vobar, stream)
                      : launch_typed<__nv_bfloat16, 64>(p, Ttot, q, q_is_bf16, vstats, vobar, stream);
  return p.d == 128 ? launch_typed<float, 128>(p, Ttot, q, q_is_bf16, vstats, vobar, stream)
                    : launch_typed<float, 64>(p, Ttot, q, q_is_bf16, vstats, vobar, stream);
}

}  // namespace spla
