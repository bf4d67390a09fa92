// Device-side helpers shared by the SPLA kernels: parameter block, type loads,
// warp reductions, mbarrier + bulk-copy (TMA) wrappers for sm_100a.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spla {

constexpr int kScoreThreads = 256;      // block-score kernel: 8 warps, one block record per warp at a time
constexpr int kScoreChunkMin = 32;      // block records per CTA: a power of two in [32, 512], chosen per launch
constexpr int kScoreChunkMax = 512;
constexpr int kStateSplits = 4;         // CTAs per unit that compute o_bar = phi(q) S_bar
constexpr int kAttendThreads = 128;     // sparse-attend kernel: 4 warps per selected block
constexpr int kMaxGroup = 16;
constexpr int kMaxWindows = 8;          // selection windows per block, at most
constexpr int kMaxTopK = 64;
constexpr unsigned kStatsBf16 = 16u;     // Params::flags bit: statistics records are bfloat16 (SPLA_STATS_BF16)
constexpr unsigned kDebugBounds = 32u;   // Params::flags bit: every block index / token offset is checked (SPLA_DEBUG_BOUNDS)
// Values a kernel may latch into the status word (the spla_status_t codes of the same meaning)
constexpr int kStatusCapacity = -2;      // an append would overflow max_context: that sequence was skipped
constexpr int kStatusTimeout = -5;       // a bounded wait on a copy barrier ran out: the math was skipped
constexpr int kStatusBounds = -6;        // an index or length outside the cache was met: the access was skipped
constexpr int kWaitLimitDefault = 1 << 22;
constexpr int kMaxBlocks = 32768;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Everything a kernel needs, passed by value.
struct Params {
  int batch, Hq, Hkv, G, d, B, top_k, max_blocks, max_context, n_sink, n_local;
  unsigned flags;
  int kv_bf16;                          // K/V cache element type: 1 = bf16, 0 = fp32
  float sm_scale, phi_scale, rms_eps;
  int NW, win_C, win_s;                 // selection windows per block, their size and stride (1, B, B: whole blocks)
  int n_chunks_cap;                     // score-kernel chunks launched per unit
  int chunk;                            // block records per score CTA
  int cs;                               // score kernel, cluster edition: CTAs per unit (0 = general kernel)
  int tile_rows;                        // tensor-core attend: rows of a K/V tile (the block size, or half of it where a block exceeds 16 KB)
  int acs;                              // tensor-core attend kernel: CTAs (cluster size) per unit
  // caller buffers
  void* k_cache;
  void* v_cache;
  float* stats;                         // fp32 records, or bfloat16 ones behind the same pointer (flags & kStatsBf16)
  float* state;
  float* tok_lse;
  int* seq_lens;
  // workspace regions
  float* ell;          // [U][G][max_blocks]      Taylor log-mass per head and block
  float* chunk_part;   // [U][max_chunks][G][2]   per-chunk (max, sum exp) of ell, natural log domain
  float* scores;       // [U][max_blocks]         aggregated BlockScore
  float* obar_part;    // [U][kStateSplits][G][d] partial phi(q) S_bar
  int* sel;            // [U][top_k]
  int* n_sel;          // [U]
  float* att_acc;      // [U][top_k][2][G][d]     per selected block: softmax numerator, then linear term
  float* att_ml;       // [U][top_k][G][2]        per selected block: (max, sum) in log2 domain
  int* score_ticket;   // [U]
  int* attend_ticket;  // [U]
  int* append_ticket;  // [1]
  float* state_part;   // [U][splits][d][d]  partial S_bar updates of the tensor-core state kernel
  int* state_ticket;   // [U]
  int* status;         // [1]
  int max_chunks;
  // Prefill-shaped forward (general kernels only): the grid's second dimension then counts *virtual* units, one per
  // (sequence, KV head, query position of the current batch of positions); vT == 0 in decode.
  int vT;                               // query positions per launch (0: decode)
  int vt0;                              // first position of this launch within the chunk
  int vTtot;                            // positions of the whole chunk (stride of q / out / vstats / vobar)
  const float* vstats;                  // [U][vTtot][2][d] statistics of each position's own (last, partial) block as of that position
  const float* vobar;                   // [U][vTtot][G][d] o_bar = phi(q_t) S_bar_t of every position
  int wait_limit;                       // iterations a bounded barrier wait polls before it gives up (0: kWaitLimitDefault)
  int dbg_tx_extra;                     // test hook: bytes added to what the decode kernels' copy barriers expect (0 in use)
};

__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }

// Loads VEC consecutive elements starting at p (aligned to VEC * sizeof(T)) as floats.
template <int VEC>
__device__ __forceinline__ void load_vec(const float* p, float (&out)[VEC]) {
  if constexpr (VEC == 4) {
    float4 v = *reinterpret_cast<const float4*>(p);
    out[0] = v.x; out[1] = v.y; out[2] = v.z; out[3] = v.w;
  } else if constexpr (VEC == 2) {
    float2 v = *reinterpret_cast<const float2*>(p);
    out[0] = v.x; out[1] = v.y;
  } else {
    out[0] = *p;
  }
}
template <int VEC>
__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float (&out)[VEC]) {
  if constexpr (VEC == 4) {
    uint2 raw = *reinterpret_cast<const uint2*>(p);
    out[0] = __uint_as_float(raw.x << 16); out[1] = __uint_as_float(raw.x & 0xffff0000u);
    out[2] = __uint_as_float(raw.y << 16); out[3] = __uint_as_float(raw.y & 0xffff0000u);
  } else if constexpr (VEC == 2) {
    uint32_t raw = *reinterpret_cast<const uint32_t*>(p);
    out[0] = __uint_as_float(raw << 16); out[1] = __uint_as_float(raw & 0xffff0000u);
  } else {
    out[0] = __bfloat162float(*p);
  }
}

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sums N (a power of two, <= 32) per-lane values across the warp with N - 1 + log2(32 / N) shuffles instead
// of 5 N: each halving step keeps one half of the values and hands the other half to the partner lane.
// On return v[0] of lane l holds the warp total of the input value with index l / (32 / N).
template <int N>
__device__ __forceinline__ void warp_reduce_multi(float (&v)[N], int lane) {
  static_assert(N >= 1 && N <= 32 && (N & (N - 1)) == 0, "N must be a power of two <= 32");
  int off = 16;
#pragma unroll
  for (int n = N; n > 1; n >>= 1) {
    const bool upper = (lane & off) != 0;
#pragma unroll
    for (int i = 0; i < n / 2; ++i) {
      const float send = upper ? v[i] : v[i + n / 2];
      const float keep = upper ? v[i + n / 2] : v[i];
      v[i] = keep + __shfl_xor_sync(0xffffffffu, send, off);
    }
    off >>= 1;
  }
#pragma unroll
  for (; off > 0; off >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], off);
}

// ---- mbarrier + bulk async copy (TMA, untiled) -------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Initialises one barrier; after the last of a batch the same thread calls mbar_init_done() once.
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_init_done() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Global -> shared bulk copy; src, dst 16-byte aligned, bytes a multiple of 16.  Never multicast.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst)),
               "l"(src), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
// Bounded wait: returns false if the phase did not complete within `limit` polls (0: the default limit).
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, int limit = 0) {
  const uint32_t addr = smem_u32(bar);
  if (limit <= 0) limit = kWaitLimitDefault;
  for (int it = 0; it < limit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(addr), "r"(parity)
        : "memory");
    if (done) return true;
    if (it > 64) __nanosleep(64);
  }
  return false;
}

// ---- thread-block clusters and distributed shared memory ---------------------------------------------------------
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Asynchronous 8-byte store into (possibly another CTA's) shared memory that counts its bytes on the mbarrier `bar` of
// the same CTA as `addr` (both shared::cluster addresses; addr 8-byte aligned).
__device__ __forceinline__ void st_async_v2(uint32_t addr, uint32_t a, uint32_t b, uint32_t bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v2.b32 [%0], {%1, %2}, [%3];" ::"r"(addr), "r"(a),
               "r"(b), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void st_async_v4(uint32_t addr, float a, float b, float c, float d, uint32_t bar) {   // 16 bytes, 16-byte aligned
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.f32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(addr),
               "f"(a), "f"(b), "f"(c), "f"(d), "r"(bar)
               : "memory");
}
// the two halves of the same barrier, for warps that have work to do between announcing and needing it (.aligned:
// executed by whole warps)
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void st_dsmem_u32(uint32_t addr, uint32_t v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void st_dsmem_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {   // 16-byte aligned
  asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// the two bf16 halves of a packed word, as floats
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

// ---- warp-level tensor-core product D += A B with fp32 accumulators (mma.m16n8k16, bf16 inputs) -------------------
// Fragment layout (PTX ISA; g = lane / 4, t = lane % 4): A rows g and g + 8, B column g, D rows g and g + 8 at
// columns 2t, 2t + 1.
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Register reallocation between the warp groups (4 warps) of a CTA: a group that needs fewer registers from here on
// gives them back to the CTA's pool, a group that needs more takes them (and waits until they are there).  Counts
// are multiples of 8 in [24, 256]; every warp of a group must execute the same instruction.
template <int N> __device__ __forceinline__ void warpgroup_reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N> __device__ __forceinline__ void warpgroup_reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// The cached length of sequence b as the decode kernels use it.  seq_lens is a caller-owned buffer (and may have been
// adopted with its contents): a value outside [0, max_context] would size loops and shared-memory arrays wrongly, so
// it is clamped and reported through the status word instead of being trusted.
__device__ __forceinline__ int checked_len(const Params& p, int b) {
  int L = __ldcg(p.seq_lens + b);
  if ((unsigned)L > (unsigned)p.max_context) {
    atomicExch(p.status, kStatusBounds);
    L = L < 0 ? 0 : p.max_context;
  }
  return L;
}

// What one value of the grid's unit dimension stands for.  Decode: unit u = (sequence b, KV head h), all cached
// tokens.  Prefill-shaped forward: a virtual unit = (u, position t of the chunk); it sees the first L tokens only,
// L = the cached length minus the chunk positions after t, which is what a decode step at that position would see.
struct UnitRef {
  int u, b, h, t, L;
  size_t qrow;                          // row of the group's first head in q / out (rows of d elements)
};
__device__ __forceinline__ UnitRef unit_ref(const Params& p, int vu) {
  UnitRef r;
  if (p.vT > 0) { r.u = vu / p.vT; r.t = p.vt0 + vu % p.vT; }
  else { r.u = vu; r.t = -1; }
  r.b = r.u / p.Hkv;
  r.h = r.u % p.Hkv;
  r.L = checked_len(p, r.b);
  if (r.t >= 0) r.L = max(0, r.L - (p.vTtot - 1 - r.t));
  r.qrow = ((size_t)r.b * (r.t >= 0 ? p.vTtot : 1) + (size_t)max(r.t, 0)) * p.Hq + (size_t)r.h * p.G;
  return r;
}

// A score launch is sized on the host from an upper bound of the lengths.  A length above what the launch covers (the
// host's bound was wrong, or seq_lens was overwritten) is cut to the covered part and reported, so that every block
// the selection may name has been scored.
__device__ __forceinline__ int cover_len(const Params& p, int L, long long cover_tokens) {
  if ((long long)L > cover_tokens) {
    atomicExch(p.status, kStatusBounds);
    L = (int)cover_tokens;
  }
  return L;
}

// Programmatic dependent launch: wait for the preceding grid's memory, allow the next grid to start.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

}  // namespace spla
