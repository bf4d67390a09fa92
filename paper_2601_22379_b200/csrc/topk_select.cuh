// Block-wide selection of the k best (key, index) pairs out of n held in shared memory, in O(n) work per pass
// instead of pairwise ranking.  Order: larger key first, then smaller index (Section 2.1 of the paper, Select =
// TopK; ties are broken by block index).  Keys equal to 0xffffffff mark forced blocks and always win.
//
// Method: forced keys are emitted first.  For the rest a 256-bin histogram over the live key interval [lo, hi]
// (bin = (key - lo) >> shift) locates the bin that holds the k-th largest key; everything in higher bins is
// emitted, and the interval shrinks to that bin.  This repeats until the bin holds at most 32 keys, which one
// warp then ranks against each other exactly with shuffles (or, if the bin is a single repeated value, by index
// against the whole input).  With well-spread scores a single pass is enough.
#pragma once

#include "spla_device.cuh"

namespace spla {

constexpr int kSelSmall = 32;       // size at which the threshold bin is ranked by one warp

struct TopkScratch {                // shared memory work area
  int hist[256 + 32];               // bin b lives at b + b / 8: a lane that owns 8 consecutive bins reads without conflicts
  uint32_t small_key[kSelSmall];
  int small_idx[kSelSmall];
  uint32_t lo, hi;                  // live interval of the free keys
  int n_forced, n_emit, n_small;
  int code_t, above, bin_count;
};

// The threads that run a selection together: the whole CTA (barrier id 0), or its first `nthreads` threads (whole
// warps) meeting on a named barrier of their own while the rest of the CTA does something else.
struct TopkGroup {
  int tid, nthreads, bar_id;
  __device__ __forceinline__ void sync() const {
    if (bar_id == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "r"(nthreads) : "memory");
  }
};
__device__ __forceinline__ TopkGroup topk_whole_cta() { return TopkGroup{(int)threadIdx.x, (int)blockDim.x, 0}; }

__device__ __forceinline__ bool pair_before(uint32_t ka, int ia, uint32_t kb, int ib) { return ka > kb || (ka == kb && ia < ib); }

// Statistics pass for callers that have not gathered them while producing the keys: emits the forced pairs and
// leaves lo / hi / n_forced / n_emit in the scratch.  Ends with a barrier.
template <class IdxFn, class EmitFn>
__device__ __forceinline__ void topk_prepare(const uint32_t* key, int n, IdxFn idx_of, EmitFn emit, TopkScratch* sc,
                                             const TopkGroup grp = topk_whole_cta()) {
  const int tid = grp.tid, lane = tid & 31, nthreads = grp.nthreads;
  if (tid == 0) { sc->lo = 0xffffffffu; sc->hi = 0u; sc->n_forced = 0; sc->n_emit = 0; }
  grp.sync();
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
  grp.sync();
}

// Requires sc->lo, sc->hi, sc->n_forced, sc->n_emit to describe `key` (forced pairs already emitted) and a
// barrier since they were written.  `emit(slot, key, idx)` stores one selected pair (slots in no particular
// order); `idx_of(i)` maps position i of `key` to the pair's index.  All threads of the group must call this.
// Returns min(k, n).
template <class IdxFn, class EmitFn>
__device__ __forceinline__ int select_topk(const uint32_t* key, int n, int k, IdxFn idx_of, EmitFn emit, TopkScratch* sc,
                                          const TopkGroup grp = topk_whole_cta()) {
  const int tid = grp.tid, lane = tid & 31, nthreads = grp.nthreads;
  k = min(k, n);
  if (k <= 0) return 0;
  const int n_forced = sc->n_forced;
  int need = k - n_forced;                    // free pairs still to pick
  if (need <= 0) return k;                    // (forced pairs never exceed k: the configuration guarantees it)
  uint32_t lo = sc->lo, hi = sc->hi;
  if (need >= n - n_forced) {                 // everything is selected
    for (int i = tid; i < n; i += nthreads)
      if (key[i] != 0xffffffffu) emit(atomicAdd(&sc->n_emit, 1), key[i], idx_of(i));
    grp.sync();
    return k;
  }

  int shift = 0, bin_count = 0;
  for (int pass = 0; pass < 5; ++pass) {      // at most four 8-bit levels exist in 32 bits
    const uint32_t range = hi - lo;
    shift = range < 256u ? 0 : (32 - __clz(range)) - 8;
    for (int i = tid; i < 256 + 32; i += nthreads) sc->hist[i] = 0;
    if (tid == 0) sc->n_small = 0;
    grp.sync();
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x >= lo && x <= hi) {
        const uint32_t c = (x - lo) >> shift;
        atomicAdd(&sc->hist[c + (c >> 3)], 1);
      }
    }
    grp.sync();
    if (tid < 32) {                           // the bin of the need-th largest live key
      int bins[8], tot = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) { bins[j] = sc->hist[lane * 9 + j]; tot += bins[j]; }
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
    grp.sync();
    const uint32_t code_t = (uint32_t)sc->code_t;
    bin_count = sc->bin_count;
    const bool last = bin_count <= kSelSmall || shift == 0;
    for (int i = tid; i < n; i += nthreads) {
      const uint32_t x = key[i];
      if (x >= lo && x <= hi) {
        const uint32_t c = (x - lo) >> shift;
        if (c > code_t) {
          emit(atomicAdd(&sc->n_emit, 1), x, idx_of(i));
        } else if (c == code_t && last && bin_count <= kSelSmall) {   // collect the threshold bin for the exact ranking
          const int s = atomicAdd(&sc->n_small, 1);
          sc->small_key[s] = x;
          sc->small_idx[s] = idx_of(i);
        }
      }
    }
    need -= sc->above;
    const uint32_t lo2 = lo + (code_t << shift);
    const uint32_t span = shift == 0 ? 0u : ((1u << shift) - 1u);
    hi = min(hi, lo2 + span);
    lo = lo2;
    grp.sync();                          // small_* complete; code_t / above may be rewritten by the next pass
    if (last) break;
  }

  // `need` of the bin_count keys in [lo, hi] remain to be picked
  if (bin_count <= kSelSmall) {
    if (tid < 32) {                           // one warp ranks the bin with shuffles
      const bool have = lane < bin_count;
      const uint32_t a = have ? sc->small_key[lane] : 0u;
      const int ia = have ? sc->small_idx[lane] : 0x7fffffff;
      int rk = 0;
#pragma unroll
      for (int j = 0; j < kSelSmall; ++j) {
        const uint32_t bkey = __shfl_sync(0xffffffffu, a, j);
        const int bidx = __shfl_sync(0xffffffffu, ia, j);
        rk += (j < bin_count) && pair_before(bkey, bidx, a, ia);
      }
      if (have && rk < need) emit(atomicAdd(&sc->n_emit, 1), a, ia);
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
  grp.sync();
  return k;
}

}  // namespace spla
