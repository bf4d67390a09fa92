// Block-wide selection of the k best (key, index) pairs out of n held in shared memory, in O(n) work per pass
// instead of pairwise ranking.  Order: larger key first, then smaller index (Section 2.1 of the paper, Select =
// TopK; ties are broken by block index).  Keys equal to 0xffffffff mark forced blocks and always win.
//
// Method: forced keys are emitted first.  For the rest a 256-bin histogram over the live key interval [lo, hi]
// (bin = (key - lo) >> shift) locates the bin that holds the k-th largest key; everything in higher bins is
// emitted, and the interval shrinks to that bin.  This repeats until the bin holds at most kSmall keys, which are
// then ranked against each other exactly (or, if all of them are equal, by index against the whole input).
// With well-spread scores a single pass is enough.
#pragma once

#include "spla_device.cuh"

namespace spla {

constexpr int kSelSmall = 64;       // size below which the threshold bin is ranked pairwise

struct TopkScratch {                // shared memory work area, 16-byte aligned
  int hist[256];
  uint32_t small_key[kSelSmall];
  int small_idx[kSelSmall];
  uint32_t lo, hi;                  // live interval of free keys
  int n_forced, n_emit, n_small;
  int code_t, above, bin_count;
};

// `emit(slot, key, idx)` stores one selected pair (slots 0 .. return value - 1, in no particular order).
// `idx_of(i)` maps position i of `key` to the pair's index.  All threads of the CTA must call this; `nthreads`
// is blockDim.x.  Returns min(k, n).
template <class IdxFn, class EmitFn>
__device__ __forceinline__ int select_topk(const uint32_t* key, int n, int k, IdxFn idx_of, EmitFn emit, TopkScratch* sc) {
  const int tid = threadIdx.x, lane = tid & 31, nthreads = blockDim.x;
  k = min(k, n);
  if (k <= 0) return 0;
  if (tid == 0) { sc->lo = 0xffffffffu; sc->hi = 0u; sc->n_forced = 0; sc->n_emit = 0; sc->n_small = 0; }
  __syncthreads();

  // forced pairs out first; interval of the free keys
  {
    uint32_t mn = 0xffffffffu, mx = 0u;
    int nf = 0;
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x == 0xffffffffu) {
        ++nf;
        emit(atomicAdd(&sc->n_emit, 1), x, idx_of(i));
      } else {
        mn = min(mn, x);
        mx = max(mx, x);
      }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    nf = __reduce_add_sync(0xffffffffu, nf);
    if (lane == 0) {
      atomicMin(&sc->lo, mn);
      atomicMax(&sc->hi, mx);
      if (nf) atomicAdd(&sc->n_forced, nf);
    }
  }
  __syncthreads();
  const int n_forced = sc->n_forced;
  int need = k - n_forced;                    // free pairs still to pick
  if (need <= 0) return k;                    // (forced pairs never exceed k: the caller's configuration guarantees it)
  uint32_t lo = sc->lo, hi = sc->hi;
  if (need >= n - n_forced) {                 // everything is selected
    for (int i = tid; i < n; i += nthreads)
      if (key[i] != 0xffffffffu) emit(atomicAdd(&sc->n_emit, 1), key[i], idx_of(i));
    __syncthreads();
    return k;
  }

  int shift = 0, bin_count = 0;
  for (int pass = 0; pass < 5; ++pass) {      // at most four 8-bit levels exist in 32 bits
    const uint32_t range = hi - lo;
    shift = range < 256u ? 0 : (32 - __clz(range)) - 8;
    for (int i = tid; i < 256; i += nthreads) sc->hist[i] = 0;
    __syncthreads();
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x >= lo && x <= hi) atomicAdd(&sc->hist[(x - lo) >> shift], 1);
    }
    __syncthreads();
    if (tid < 32) {                           // the bin of the need-th largest live key
      int bins[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { bins[j] = sc->hist[lane * 8 + j]; tot += bins[j]; }
      int above = tot;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_down_sync(0xffffffffu, above, o);
        if (lane + o < 32) above += t;
      }
      above -= tot;
      if (above < need && need <= above + tot) {
        int cum = above;
#pragma unroll
        for (int j = 7; j >= 0; --j) {
          if (cum < need && need <= cum + bins[j]) { sc->code_t = lane * 8 + j; sc->above = cum; sc->bin_count = bins[j]; }
          cum += bins[j];
        }
      }
    }
    __syncthreads();
    const uint32_t code_t = (uint32_t)sc->code_t;
    bin_count = sc->bin_count;
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x >= lo && x <= hi && ((x - lo) >> shift) > code_t) emit(atomicAdd(&sc->n_emit, 1), x, idx_of(i));
    }
    need -= sc->above;
    const uint32_t lo2 = lo + (code_t << shift);
    const uint32_t span = shift == 0 ? 0u : ((1u << shift) - 1u);
    hi = min(hi, lo2 + span);
    lo = lo2;
    if (bin_count <= kSelSmall || shift == 0) break;
    __syncthreads();                          // everybody has read code_t / above before the next pass rewrites them
  }

  // `need` of the bin_count keys in [lo, hi] remain to be picked
  if (bin_count <= kSelSmall) {
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x >= lo && x <= hi) {
        const int s = atomicAdd(&sc->n_small, 1);
        sc->small_key[s] = x;
        sc->small_idx[s] = idx_of(i);
      }
    }
    __syncthreads();
    if (tid < bin_count) {
      const uint32_t a = sc->small_key[tid];
      const int ia = sc->small_idx[tid];
      int rk = 0;
      for (int j = 0; j < bin_count; ++j) {
        const uint32_t bkey = sc->small_key[j];
        rk += (bkey > a) || (bkey == a && sc->small_idx[j] < ia);
      }
      if (rk < need) emit(atomicAdd(&sc->n_emit, 1), a, ia);
    }
  } else {
    // many identical keys (shift == 0 means lo == hi): the smallest indices win; count equals before each one
    for (int i = tid; i < n; i += nthreads) {
      if (key[i] != lo) continue;
      const int ia = idx_of(i);
      int rk = 0;
      for (int j = 0; j < n; ++j) rk += (key[j] == lo) && (idx_of(j) < ia);
      if (rk < need) emit(atomicAdd(&sc->n_emit, 1), lo, ia);
    }
  }
  __syncthreads();
  return k;
}

}  // namespace spla
