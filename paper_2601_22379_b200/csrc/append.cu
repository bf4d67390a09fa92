// KV append: store the new tokens, refresh the block statistics the Taylor score reads (Section 3.1,
// Eq. taylor-2nd: block key mean and diagonal population covariance) and advance the global linear-attention
// state S_bar += phi(k_t)^T v_t in fp32 (Section 3.2, Eq. rla-impl-1, "Numerical Stability").
//
// Four small kernels in stream order, all reading the OLD sequence lengths until the last one bumps them:
//   copy   : k_new, v_new -> cache; per-token logsumexp of phi_scale * k into tok_lse
//   stats  : mean / variance of every touched block recomputed from the cached keys (two exact passes, so the
//            result does not depend on how the tokens were split across append calls)
//   state  : rank-n update of S_bar, rows tiled over CTAs, phi(k) staged through shared memory
//   lengths: seq_lens += n_new
#include "spla_internal.h"

namespace spla {

constexpr int kCopyThreads = 256;
constexpr int kStateRows = 16;     // rows of S_bar per CTA
constexpr int kStateTokens = 32;   // tokens staged per inner step

__device__ __forceinline__ int tokens_to_add(const Params& p, const int* n_new, int max_new, int b, int L) {
  int n = n_new ? n_new[b] : max_new;
  n = max(0, min(n, max_new));
  if (L + n > p.max_context) return -1;      // would overflow: skip this sequence, the caller is told via status
  return n;
}

template <int BYTES>
__device__ __forceinline__ void copy_bytes(void* dst, const void* src) {
  if constexpr (BYTES == 16) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  else if constexpr (BYTES == 8) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
  else *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
}

template <typename T, int D>
__global__ void __launch_bounds__(kCopyThreads) append_copy_kernel(const Params p, const T* __restrict__ k_new,
                                                                   const T* __restrict__ v_new,
                                                                   const int* __restrict__ n_new, int max_new) {
  constexpr int VEC = D / 32;
  const int u = blockIdx.y, b = u / p.Hkv;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  if (n < 0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicExch(p.status, -2);
    return;
  }
  const int i = blockIdx.x * (kCopyThreads / 32) + warp;
  if (i >= n) return;
  const size_t src = ((size_t)u * max_new + i) * D + lane * VEC;
  const size_t pos = (size_t)u * p.max_blocks * p.B + (size_t)(L + i);
  T* kd = reinterpret_cast<T*>(p.k_cache) + pos * D + lane * VEC;
  T* vd = reinterpret_cast<T*>(p.v_cache) + pos * D + lane * VEC;
  float k[VEC];
  load_vec<VEC>(k_new + src, k);
  copy_bytes<VEC * sizeof(T)>(kd, k_new + src);
  copy_bytes<VEC * sizeof(T)>(vd, v_new + src);
  float mx = -INFINITY;
#pragma unroll
  for (int v = 0; v < VEC; ++v) { k[v] *= p.phi_scale; mx = fmaxf(mx, k[v]); }
  mx = warp_max(mx);
  float s = 0.f;
#pragma unroll
  for (int v = 0; v < VEC; ++v) s += expf(k[v] - mx);
  s = warp_sum(s);
  if (lane == 0) p.tok_lse[pos] = mx + logf(s);
}

template <typename T, int D>
__global__ void __launch_bounds__(D) append_stats_kernel(const Params p, const int* __restrict__ n_new, int max_new) {
  const int u = blockIdx.y, b = u / p.Hkv;
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  if (n <= 0) return;
  const int blk = L / p.B + blockIdx.x;                    // x-th touched block
  const int t0 = blk * p.B;
  if (t0 >= L + n) return;
  const int cnt = min(p.B, L + n - t0);
  const int c = threadIdx.x;
  const T* kb = reinterpret_cast<const T*>(p.k_cache) + ((size_t)u * p.max_blocks * p.B + t0) * D + c;
  float sum = 0.f;
  for (int t = 0; t < cnt; ++t) sum += to_float(kb[(size_t)t * D]);
  const float mean = sum / (float)cnt;
  float ss = 0.f;
  for (int t = 0; t < cnt; ++t) {
    const float dv = to_float(kb[(size_t)t * D]) - mean;
    ss = fmaf(dv, dv, ss);
  }
  float* rec = p.stats + ((size_t)u * p.max_blocks + blk) * 2 * D;
  rec[c] = mean;
  rec[D + c] = ss / (float)cnt;
}

template <typename T, int D>
__global__ void __launch_bounds__(D) append_state_kernel(const Params p, const T* __restrict__ k_new,
                                                         const T* __restrict__ v_new, const int* __restrict__ n_new,
                                                         int max_new) {
  __shared__ float phi_s[kStateTokens][kStateRows];
  const int u = blockIdx.y, b = u / p.Hkv;
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  if (n <= 0) return;
  const int row0 = blockIdx.x * kStateRows;
  const int j = threadIdx.x;
  const float a2 = p.phi_scale * kLog2e;
  const float* lse = p.tok_lse + (size_t)u * p.max_blocks * p.B + L;
  const T* kn = k_new + (size_t)u * max_new * D;
  const T* vn = v_new + (size_t)u * max_new * D;
  float acc[kStateRows];
#pragma unroll
  for (int r = 0; r < kStateRows; ++r) acc[r] = 0.f;
  for (int t0 = 0; t0 < n; t0 += kStateTokens) {
    const int nt = min(kStateTokens, n - t0);
    __syncthreads();
    for (int idx = j; idx < kStateTokens * kStateRows; idx += D) {
      const int t = idx / kStateRows, r = idx % kStateRows;
      float f = 0.f;
      if (t < nt) f = exp2f(fmaf(to_float(kn[(size_t)(t0 + t) * D + row0 + r]), a2, -lse[t0 + t] * kLog2e));
      phi_s[t][r] = f;
    }
    __syncthreads();
    for (int t = 0; t < nt; ++t) {
      const float v = to_float(vn[(size_t)(t0 + t) * D + j]);
#pragma unroll
      for (int r = 0; r < kStateRows; ++r) acc[r] = fmaf(phi_s[t][r], v, acc[r]);
    }
  }
  float* S = p.state + (size_t)u * D * D + (size_t)row0 * D + j;
#pragma unroll
  for (int r = 0; r < kStateRows; ++r) S[(size_t)r * D] += acc[r];
}

__global__ void append_lengths_kernel(const Params p, const int* __restrict__ n_new, int max_new) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= p.batch) return;
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  if (n > 0) p.seq_lens[b] = L + n;
}

template <typename T, int D>
static cudaError_t launch_typed(const Params& p, const void* k_new, const void* v_new, const int* n_new, int max_new,
                                cudaStream_t stream) {
  const int U = p.batch * p.Hkv;
  const T* kn = reinterpret_cast<const T*>(k_new);
  const T* vn = reinterpret_cast<const T*>(v_new);
  const int per_cta = kCopyThreads / 32;
  append_copy_kernel<T, D><<<dim3((max_new + per_cta - 1) / per_cta, U), kCopyThreads, 0, stream>>>(p, kn, vn, n_new, max_new);
  append_stats_kernel<T, D><<<dim3((max_new + p.B - 1) / p.B + 1, U), D, 0, stream>>>(p, n_new, max_new);
  if (!(p.flags & 4u))
    append_state_kernel<T, D><<<dim3(D / kStateRows, U), D, 0, stream>>>(p, kn, vn, n_new, max_new);
  append_lengths_kernel<<<(p.batch + 127) / 128, 128, 0, stream>>>(p, n_new, max_new);
  return cudaGetLastError();
}

cudaError_t launch_append(const Params& p, const void* k_new, const void* v_new, const int* n_new, int max_new,
                          cudaStream_t stream) {
  if (p.kv_bf16)
    return p.d == 128 ? launch_typed<__nv_bfloat16, 128>(p, k_new, v_new, n_new, max_new, stream)
                      : launch_typed<__nv_bfloat16, 64>(p, k_new, v_new, n_new, max_new, stream);
  return p.d == 128 ? launch_typed<float, 128>(p, k_new, v_new, n_new, max_new, stream)
                    : launch_typed<float, 64>(p, k_new, v_new, n_new, max_new, stream);
}

}  // namespace spla
