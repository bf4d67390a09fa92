// KV append: store the new tokens, refresh the block statistics the Taylor score reads (Section 3.1,
// Eq. taylor-2nd: block key mean and diagonal population covariance) and advance the global linear-attention
// state S_bar += phi(k_t)^T v_t in fp32 (Section 3.2, Eq. rla-impl-1, "Numerical Stability").
//
// Appends of up to 32 tokens per sequence (the decode loop) run as ONE fused kernel, see append_fused_kernel.
// Bulk appends (prefill) run as three kernels in stream order, all reading the OLD sequence lengths until the
// last one bumps them:
//   block  : one CTA per touched block: its keys (cached ones below the old length, new ones above) are staged in
//            shared memory once; from there the new tokens go to the cache (k_new, v_new -> cache), their
//            logsumexp of phi_scale * k to tok_lse, and the block's mean / variance records are recomputed (two
//            exact passes, so the result does not depend on how the tokens were split across append calls)
//   state  : rank-n update of S_bar (tensor cores for long bf16 appends, else rows tiled over CTAs on the FMA pipe)
//   lengths: seq_lens += n_new
#include "spla_internal.h"

namespace spla {

constexpr int kStateRows = 16;     // rows of S_bar per CTA
constexpr int kStateTokens = 32;   // tokens staged per inner step
constexpr int kStateUmmaMinTokens = 256;   // appends at least this long take the tensor-core state kernel

__device__ __forceinline__ int tokens_to_add(const Params& p, const int* n_new, int max_new, int b, int L) {
  int n = n_new ? n_new[b] : max_new;
  n = max(0, min(n, max_new));
  if (L < 0 || L + n > p.max_context) return -1;   // would overflow (or a corrupt length): skip this sequence, the caller is told via status
  return n;
}

template <int BYTES>
__device__ __forceinline__ void copy_bytes(void* dst, const void* src) {
  if constexpr (BYTES == 16) *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src);
  else if constexpr (BYTES == 8) *reinterpret_cast<uint2*>(dst) = *reinterpret_cast<const uint2*>(src);
  else *reinterpret_cast<uint32_t*>(dst) = *reinterpret_cast<const uint32_t*>(src);
}

// Mean and population variance of one selection window of one block (window w covers the block's tokens
// [w * win_s, w * win_s + win_C); without strided windows that is the whole block), two exact passes, by
// kStatThreads threads (groups of D threads take every TG-th token; the partial sums are combined in a fixed
// order, so every append path gives the same bits).  `key_at(t)` returns channel (tid % D) of the block's token t.
// A window that holds no token yet is left alone.
constexpr int kStatThreads = 256;
template <int D, bool WIN, typename KeyAt>
__device__ __forceinline__ void block_stats_core(const Params& p, int u, int blk, int w, int L_total, bool act,
                                                 float (*red_s)[D], float* mean_s, KeyAt key_at) {
  constexpr int TG = kStatThreads / D;
  const int tid = threadIdx.x;
  const int t0 = blk * p.B;
  const int t_lo = WIN ? w * p.win_s : 0;
  const int t_hi = act ? (WIN ? min(min(p.B, L_total - t0), t_lo + p.win_C) : min(p.B, L_total - t0)) : 0;   // tokens [t_lo, t_hi)
  const int cnt = max(0, t_hi - t_lo);
  act = act && cnt > 0;
  const int tg = tid / D, c = tid % D;
  float sum = 0.f;
#pragma unroll 8
  for (int t = t_lo + tg; t < t_hi; t += TG) sum += key_at(t);
  red_s[tg][c] = sum;
  __syncthreads();
  if (tg == 0) {
    float tot = 0.f;
#pragma unroll
    for (int g2 = 0; g2 < TG; ++g2) tot += red_s[g2][c];
    mean_s[c] = cnt > 0 ? tot / (float)cnt : 0.f;
  }
  __syncthreads();
  const float mean = mean_s[c];
  float ss = 0.f;
#pragma unroll 8
  for (int t = t_lo + tg; t < t_hi; t += TG) {
    const float dv = key_at(t) - mean;
    ss = fmaf(dv, dv, ss);
  }
  __syncthreads();
  red_s[tg][c] = ss;
  __syncthreads();
  if (tg == 0 && act) {
    float tot = 0.f;
#pragma unroll
    for (int g2 = 0; g2 < TG; ++g2) tot += red_s[g2][c];
    const size_t rec_off = (WIN ? ((size_t)u * p.max_blocks + blk) * p.NW + w : (size_t)u * p.max_blocks + blk) * 2 * D;
    if (p.flags & kStatsBf16) {                      // 16-bit records: rounded once, here
      __nv_bfloat16* rec = reinterpret_cast<__nv_bfloat16*>(p.stats) + rec_off;
      rec[c] = __float2bfloat16_rn(mean);
      rec[D + c] = __float2bfloat16_rn(tot / (float)cnt);
    } else {
      float* rec = p.stats + rec_off;
      rec[c] = mean;
      rec[D + c] = tot / (float)cnt;
    }
  }
}

// The same from global memory: token t of the block comes from the cache if its position is below `L_cached`,
// else from the new tokens `kn`.
template <typename T, int D, bool WIN>
__device__ __forceinline__ void block_stats_role(const Params& p, int u, int blk, int w, int L_cached, int L_total, const T* kn,
                                                 bool act, float (*red_s)[D], float* mean_s) {
  const int t0 = blk * p.B;
  const int c = threadIdx.x % D;
  const T* kc = reinterpret_cast<const T*>(p.k_cache) + ((size_t)u * p.max_blocks * p.B + t0) * D + c;
  // One address per token (cached or new) and one load from it: no branch around the loads, so that the
  // unrolled loop keeps several of them in flight.
  block_stats_core<D, WIN>(p, u, blk, w, L_total, act, red_s, mean_s, [&](int t) {
    const int pos = t0 + t;
    const T* src = pos < L_cached ? kc + (size_t)t * D : kn + (size_t)(pos - L_cached) * D + c;
    return to_float(*src);
  });
}

// Bulk append, one CTA per touched block (blockIdx.x-th block at or after the one the old length falls in).  The
// block's keys are staged once in shared memory, 16 bytes per thread and load, several loads in flight: cached
// keys below the old length, new keys above it; the new keys and values go on to the cache from the same
// registers.  Then, from shared memory: the per-token logsumexp of the new tokens (one warp per token) and the
// statistics records of all the block's windows.
constexpr int kBlockLoads = 4;                       // 16-byte loads of K (and of V) in flight per thread
template <typename T, int D>
__global__ void __launch_bounds__(kStatThreads) append_block_kernel(const Params p, const T* __restrict__ k_new,
                                                                    const T* __restrict__ v_new,
                                                                    const int* __restrict__ n_new, int max_new) {
  extern __shared__ __align__(16) unsigned char tile_raw[];
  __shared__ float red_s[kStatThreads / D][D];
  __shared__ float mean_s[D];
  constexpr int VEC = D / 32;
  constexpr int CH = D * (int)sizeof(T) / 16;        // 16-byte chunks per token
  T* tile = reinterpret_cast<T*>(tile_raw);          // [B][D]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y, b = u / p.Hkv;
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  if (n < 0) {
    if (blockIdx.x == 0 && tid == 0) atomicExch(p.status, kStatusCapacity);
    return;
  }
  const int blk = L / p.B + blockIdx.x;
  const int t0 = blk * p.B;
  if (n == 0 || t0 >= L + n) return;                 // CTA-uniform
  const int cnt = min(p.B, L + n - t0);              // tokens the block holds after the append
  if ((p.flags & kDebugBounds) && (blk < 0 || blk >= p.max_blocks)) {   // checked build: the block must exist (CTA-uniform)
    if (tid == 0) atomicExch(p.status, kStatusBounds);
    return;
  }
  const int t_new = max(0, L - t0);                  // its first new token

  const size_t blk_tok0 = (size_t)u * p.max_blocks * p.B + t0;
  uint4* kc = reinterpret_cast<uint4*>(reinterpret_cast<T*>(p.k_cache) + blk_tok0 * D);
  uint4* vc = reinterpret_cast<uint4*>(reinterpret_cast<T*>(p.v_cache) + blk_tok0 * D);
  // new token i of the unit sits at chunk (t0 - L + t) * CH + ch of kn / vn
  const uint4* kn = reinterpret_cast<const uint4*>(k_new + (size_t)u * max_new * D) + (ptrdiff_t)(t0 - L) * CH;
  const uint4* vn = reinterpret_cast<const uint4*>(v_new + (size_t)u * max_new * D) + (ptrdiff_t)(t0 - L) * CH;
  uint4* tile4 = reinterpret_cast<uint4*>(tile_raw);
  const int total = cnt * CH, first_new = t_new * CH;
  for (int base = 0; base < total; base += kBlockLoads * kStatThreads) {
    uint4 kk[kBlockLoads], vv[kBlockLoads];
#pragma unroll
    for (int j = 0; j < kBlockLoads; ++j) {
      const int idx = base + j * kStatThreads + tid;
      if (idx < total) {
        if (idx >= first_new) { kk[j] = __ldcs(kn + idx); vv[j] = __ldcs(vn + idx); }
        else kk[j] = kc[idx];
      }
    }
#pragma unroll
    for (int j = 0; j < kBlockLoads; ++j) {
      const int idx = base + j * kStatThreads + tid;
      if (idx < total) {
        tile4[idx] = kk[j];
        if (idx >= first_new) { kc[idx] = kk[j]; vc[idx] = vv[j]; }
      }
    }
  }
  __syncthreads();

  // per-token logsumexp of phi_scale * k, the value the decode and the state update read
  for (int t = t_new + warp; t < cnt; t += kStatThreads / 32) {
    float k[VEC];
    load_vec<VEC>(tile + (size_t)t * D + lane * VEC, k);
    float mx = -INFINITY;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { k[v] *= p.phi_scale; mx = fmaxf(mx, k[v]); }
    mx = warp_max(mx);
    float s = 0.f;
#pragma unroll
    for (int v = 0; v < VEC; ++v) s += expf(k[v] - mx);
    s = warp_sum(s);
    if (lane == 0) p.tok_lse[blk_tok0 + t] = mx + logf(s);
  }

  const int c = tid % D;
  for (int w = 0; w < p.NW; ++w) {
    block_stats_core<D, true>(p, u, blk, w, L + n, true, red_s, mean_s,
                              [&](int t) { return to_float(tile[(size_t)t * D + c]); });
    __syncthreads();                                 // the next window reuses the reduction buffers
  }
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

// ---------------------------------------------------------------------------------------------------------
// Decode-step appends (a few tokens per sequence): everything above in ONE launch.  CTAs take one of three roles
// by blockIdx.x; no role needs another's output, because the new tokens are read from k_new / v_new directly
// (statistics of the open block: cached keys below the old length, new keys above it; state: the per-token
// log-sum-exp is recomputed from the new keys).  Every CTA reads the old lengths; the last CTA to have read them
// (atomic ticket at the start, nobody waits) advances them.
constexpr int kFusedThreads = 256;
constexpr int kFusedMaxNew = 32;

template <typename T, int D, bool WIN>
__global__ void __launch_bounds__(kFusedThreads, 4) append_fused_kernel(const Params p, const T* __restrict__ k_new,
                                                                     const T* __restrict__ v_new,
                                                                     const int* __restrict__ n_new, int max_new, int n_copy,
                                                                     int n_stats) {
  constexpr int VEC = D / 32;
  constexpr int TG = kFusedThreads / D;            // thread groups of D threads
  __shared__ float red_s[TG][D];
  __shared__ float mean_s[D];
  __shared__ float phi_s[kFusedMaxNew][kStateRows];
  __shared__ float lse_s[kFusedMaxNew];
  __shared__ int last_s;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y, b = u / p.Hkv;
  int role = blockIdx.x;

  pdl_wait();                                      // the preceding decode still reads the cache and the lengths
  pdl_launch_dependents();
  const int L = p.seq_lens[b];
  const int n = tokens_to_add(p, n_new, max_new, b, L);
  const T* kn = k_new + (size_t)u * max_new * D;
  const T* vn = v_new + (size_t)u * max_new * D;
  const size_t unit_tok0 = (size_t)u * p.max_blocks * p.B;

  // ---- the lengths are advanced by whichever CTA is the last to have read them ----------------------------------
  // Every CTA works from the length it read above.  Once all CTAs of the launch hold theirs (the barrier below
  // consumes each thread's value, so no load of a length is still in flight), the last one to check in may store the
  // new lengths while the others are still busy: nothing in this launch reads them again, and the next kernel
  // starts after this grid has completed.  No fence and no wait at the end of the kernel.
  if (__syncthreads_or(L < 0)) return;               // (lengths are never negative)
  if (tid == 0) {
    const int t = atomicAdd(p.append_ticket, 1);
    last_s = (t == (int)(gridDim.x * gridDim.y) - 1);
    if (last_s) *p.append_ticket = 0;
  }
  __syncthreads();
  if (last_s) {
    for (int bb = tid; bb < p.batch; bb += kFusedThreads) {
      const int Lb = p.seq_lens[bb];
      const int nb = tokens_to_add(p, n_new, max_new, bb, Lb);
      if (nb > 0) p.seq_lens[bb] = Lb + nb;
    }
  }

  if (role < n_copy) {
    // ---- copy role: one warp per token; also the per-token log-sum-exp the decode reads ------------------
    if (n < 0 && role == 0 && tid == 0) atomicExch(p.status, kStatusCapacity);
    const int i = role * (kFusedThreads / 32) + warp;
    bool in_cache = true;
    if ((p.flags & kDebugBounds) && n > 0 && i < n && L + i >= p.max_blocks * p.B) {   // checked build
      if (lane == 0) atomicExch(p.status, kStatusBounds);
      in_cache = false;
    }
    if (n > 0 && i < n && in_cache) {
      const size_t pos = unit_tok0 + (size_t)(L + i);
      float k[VEC];
      load_vec<VEC>(kn + (size_t)i * D + lane * VEC, k);
      copy_bytes<VEC * sizeof(T)>(reinterpret_cast<T*>(p.k_cache) + pos * D + lane * VEC, kn + (size_t)i * D + lane * VEC);
      copy_bytes<VEC * sizeof(T)>(reinterpret_cast<T*>(p.v_cache) + pos * D + lane * VEC, vn + (size_t)i * D + lane * VEC);
      float mx = -INFINITY;
#pragma unroll
      for (int v = 0; v < VEC; ++v) { k[v] *= p.phi_scale; mx = fmaxf(mx, k[v]); }
      mx = warp_max(mx);
      float sm = 0.f;
#pragma unroll
      for (int v = 0; v < VEC; ++v) sm += expf(k[v] - mx);
      sm = warp_sum(sm);
      if (lane == 0) p.tok_lse[pos] = mx + logf(sm);
    }
  } else if ((role -= n_copy) < n_stats) {
    // ---- statistics role: one touched block; cached keys below the old length, new keys above it -----------
    const int blk = L / p.B + (WIN ? role / p.NW : role);
    block_stats_role<T, D, WIN>(p, u, blk, WIN ? role % p.NW : 0, L, L + max(n, 0), kn, n > 0 && blk * p.B < L + n, red_s, mean_s);
  } else if (!(p.flags & 4u)) {
    // ---- state role: S_bar[row0 .. row0 + 15][:] += sum_t phi(k_t)[row] v_t ------------------------------------
    role -= n_stats;
    const int row0 = role * kStateRows;
    const int nn = max(n, 0);
    const float a2 = p.phi_scale * kLog2e;
    // The rows of S_bar this thread will update are requested first: the load comes from DRAM and would
    // otherwise sit at the end of the role's dependency chain.
    constexpr int RPT = kStateRows / TG;                         // rows per thread
    const int tg = tid / D, j = tid % D;
    float* S = p.state + (size_t)u * D * D + (size_t)(row0 + tg * RPT) * D + j;
    float s_old[RPT];
#pragma unroll
    for (int r = 0; r < RPT; ++r) s_old[r] = nn > 0 ? __ldcs(S + (size_t)r * D) : 0.f;
    // log-sum-exp of every new token: 8 threads per token, D / 8 consecutive channels each, loaded up front
    {
      constexpr int CPT = D / 8;                                 // channels per thread
      const int t = tid >> 3, part = tid & 7;
      float x[CPT];
      if (t < nn) {
#pragma unroll
        for (int c4 = 0; c4 < CPT / 4; ++c4) {
          float y[4];
          load_vec<4>(kn + (size_t)t * D + part * CPT + c4 * 4, y);
#pragma unroll
          for (int v = 0; v < 4; ++v) x[c4 * 4 + v] = y[v] * a2;
        }
      } else {
#pragma unroll
        for (int v = 0; v < CPT; ++v) x[v] = -INFINITY;
      }
      float mx = -INFINITY, sm = 0.f;
#pragma unroll
      for (int v = 0; v < CPT; ++v) mx = fmaxf(mx, x[v]);
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
      if (t < nn) {
#pragma unroll
        for (int v = 0; v < CPT; ++v) sm += exp2f(x[v] - mx);
      }
      sm += __shfl_xor_sync(0xffffffffu, sm, 1);
      sm += __shfl_xor_sync(0xffffffffu, sm, 2);
      sm += __shfl_xor_sync(0xffffffffu, sm, 4);
      if (t < nn && part == 0) lse_s[t] = mx + log2f(sm);        // base-2 domain
    }
    __syncthreads();
    for (int idx = tid; idx < kFusedMaxNew * kStateRows; idx += kFusedThreads) {
      const int t = idx / kStateRows, r = idx % kStateRows;
      phi_s[t][r] = t < nn ? exp2f(to_float(kn[(size_t)t * D + row0 + r]) * a2 - lse_s[t]) : 0.f;
    }
    __syncthreads();
    float acc[RPT];
#pragma unroll
    for (int r = 0; r < RPT; ++r) acc[r] = 0.f;
    for (int t = 0; t < nn; ++t) {
      const float v = to_float(vn[(size_t)t * D + j]);
#pragma unroll
      for (int r = 0; r < RPT; ++r) acc[r] = fmaf(phi_s[t][tg * RPT + r], v, acc[r]);
    }
    if (nn > 0) {
#pragma unroll
      for (int r = 0; r < RPT; ++r) S[(size_t)r * D] = s_old[r] + acc[r];
    }
  }

}

template <typename T, int D>
static cudaError_t launch_typed(const Params& p, const void* k_new, const void* v_new, const int* n_new, int max_new,
                                const AttendMaps* state_maps, cudaStream_t stream) {
  const int U = p.batch * p.Hkv;
  const T* kn = reinterpret_cast<const T*>(k_new);
  const T* vn = reinterpret_cast<const T*>(v_new);
  if (max_new <= kFusedMaxNew) {
    const int n_copy = (max_new + kFusedThreads / 32 - 1) / (kFusedThreads / 32);
    const int n_stats = ((max_new + p.B - 1) / p.B + 1) * p.NW;   // one CTA per window of every block that can be touched
    const int n_state = (p.flags & 4u) ? 0 : D / kStateRows;
    // Same shared-memory carve-out as the decode kernels around it: a change of carve-out drains the SMs.
    auto kern = p.NW > 1 ? append_fused_kernel<T, D, true> : append_fused_kernel<T, D, false>;
    cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    return launch_ex(kern, dim3(n_copy + n_stats + n_state, U), dim3(kFusedThreads), 0, stream, 0, true,
                     p, kn, vn, n_new, max_new, n_copy, n_stats);
  }
  {
    const size_t tile_bytes = (size_t)p.B * D * sizeof(T);
    auto kern = append_block_kernel<T, D>;
    if (tile_bytes > 48 * 1024) cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tile_bytes);
    kern<<<dim3((max_new + p.B - 1) / p.B + 1, U), kStatThreads, tile_bytes, stream>>>(p, kn, vn, n_new, max_new);
    ++g_launch_count;
  }
  if (!(p.flags & 4u)) {
    // long appends of a bf16 cache with d = 128: the rank-n update is a dense contraction, done on the tensor cores
    // from the tokens the copy kernel has just stored; everything else on the FMA pipe
    if (sizeof(T) == 2 && D == 128 && state_maps && state_maps->valid && max_new >= kStateUmmaMinTokens) {
      const cudaError_t e = launch_state_umma(p, state_maps, n_new, max_new, stream);
      if (e != cudaSuccess) return e;
    } else {
      append_state_kernel<T, D><<<dim3(D / kStateRows, U), D, 0, stream>>>(p, kn, vn, n_new, max_new);
      ++g_launch_count;
    }
  }
  append_lengths_kernel<<<(p.batch + 127) / 128, 128, 0, stream>>>(p, n_new, max_new);
  ++g_launch_count;
  return cudaGetLastError();
}

cudaError_t launch_append(const Params& p, const void* k_new, const void* v_new, const int* n_new, int max_new,
                          const AttendMaps* state_maps, cudaStream_t stream) {
  if (p.kv_bf16)
    return p.d == 128 ? launch_typed<__nv_bfloat16, 128>(p, k_new, v_new, n_new, max_new, state_maps, stream)
                      : launch_typed<__nv_bfloat16, 64>(p, k_new, v_new, n_new, max_new, state_maps, stream);
  return p.d == 128 ? launch_typed<float, 128>(p, k_new, v_new, n_new, max_new, state_maps, stream)
                    : launch_typed<float, 64>(p, k_new, v_new, n_new, max_new, state_maps, stream);
}

}  // namespace spla
