// Bulk update of the recurrent state on the 5th-generation tensor cores:  S_bar += phi(K)^T V  over all tokens a
// bulk append (prefill) adds (Section 3.2 of the paper, Eq. rla-impl-1; "Numerical Stability": the state is kept
// in fp32).  For one (sequence, KV head) unit this is a dense [d x n] . [n x d] contraction over the n new tokens,
// which is what tcgen05.mma is for: the accumulator (128 x 128 fp32) lives in tensor memory, both operands come
// from shared memory through matrix descriptors, one elected thread issues the instructions.
//
// Shapes: M = 128 features of phi(k), N = 128 value channels, K = tokens.  The cache stores a token's d channels
// contiguously, so both operands are "MN-major"; a TMA box of 64 tokens x 64 channels with the 128-byte swizzle
// lands exactly in the canonical layout the matrix descriptor names (rows of 128 bytes, swizzle atoms of 8 rows).
//
// Per CTA (one unit, one split of the unit's new tokens), 10 warps:
//   warp 0     : producer - tiled TMA loads of K and V tiles (64 tokens) into a 4-stage ring;
//   warps 2..9 : transform (two groups of four warps, alternating tiles) - phi(k) = exp(phi_scale k - lse_t) in place (lse_t from the per-token table the copy
//                kernel has just filled), split into a bf16 head (written over K) and a bf16 remainder (second
//                buffer), so that the product carries 16 significant bits of phi; rows past the last new token
//                are zeroed in all three tiles;
//   warp 1     : issues 2 x 4 tcgen05.mma (head and remainder, K = 16 tokens each) per tile, commits the stage
//                back to the producer, and owns the tensor-memory allocation;
//   warps 2..9 : also drain the accumulator: the tensor core does not add into its fp32 accumulator with
//                round-to-nearest, and the error grows with the length of the chain (measured against float64:
//                1e-4 relative after 4000 instructions), so a chain is cut after two tiles (16 instructions),
//                where the 16-bit representation of phi is what is left (1.8e-6 relative on S_bar, whose entries
//                are sums of signed terms, so per-term errors do not average out): the issuer alternates
//                between two accumulators, and the transform warps add a finished one into fp32 registers
//                (64 columns of one row per thread, round-to-nearest) while the other is being filled;
//                at the end the registers go to this split's partial buffer.
// The last CTA of a unit to finish (atomic ticket, nobody waits) adds the partials to S_bar in split order, so the
// result does not depend on the order in which CTAs ran.  With a single split the CTA adds to S_bar itself.
//
// Every wait is an mbarrier poll with an iteration limit; on expiry the CTA raises its abort flag, all roles
// leave their loops, tensor memory is released and the time-out status is latched.  No multicast anywhere.
#include <cuda.h>

#include "spla_internal.h"

namespace spla {

namespace {

constexpr int kSuD = 128;
constexpr int kSuTile = 64;                                  // tokens per stage
constexpr int kSuStages = 4;
constexpr int kSuTransformWarps = 8;
constexpr int kSuThreads = (2 + kSuTransformWarps) * 32;
constexpr int kSuHalfBytes = kSuTile * 128;                  // one TMA box: 64 tokens x 64 channels bf16
constexpr int kSuTileBytes = 2 * kSuHalfBytes;               // 16 KB: all 128 channels
constexpr int kSuStageBytes = 3 * kSuTileBytes;              // K (becomes the head of phi), remainder of phi, V
constexpr int kSuSmemBytes = kSuStages * kSuStageBytes;      // 192 KB
constexpr int kSuGroup = 2;                                  // tiles accumulated in tensor memory before a flush
constexpr int kSuTmemCols = 256;                             // two 128-column accumulators, used in turn

// tcgen05 instruction descriptor, kind::f16: fp32 accumulator (bit 4), A and B bf16 (bits 7, 10), A and B
// MN-major (bits 15, 16), N / 8 at bit 17, M / 16 at bit 24.
constexpr uint32_t kSuIdesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((kSuD / 8) << 17) | ((kSuD / 16) << 24);

// Shared-memory matrix descriptor of an MN-major bf16 operand in the 128-byte swizzle: start address / 16,
// leading byte offset / 16 at bit 16 (distance between the two 64-channel halves), stride byte offset / 16 at
// bit 32 (distance between groups of 8 tokens), descriptor version 1 at bit 46, layout type 2 at bit 61.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  const uint64_t lo = (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)(kSuHalfBytes >> 4) << 16);
  const uint64_t hi = (uint64_t)(1024 >> 4) | (1ull << 14) | (2ull << 29);
  return lo | (hi << 32);
}

__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
               "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void mbar_arrive1(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(kSuIdesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// Arrives on the barrier once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive accumulator columns of this thread's tensor-memory lane.
__device__ __forceinline__ void tmem_ld32(uint32_t addr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(addr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}


}  // namespace

__global__ void __launch_bounds__(kSuThreads, 1)
    state_umma_kernel(const Params p, const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
                      const int* __restrict__ n_new, int max_new) {
  constexpr int D = kSuD;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ __align__(8) uint64_t full[kSuStages];      // TMA -> transform
  __shared__ __align__(8) uint64_t ready[kSuStages];     // transform -> MMA
  __shared__ __align__(8) uint64_t empty[kSuStages];     // MMA (tcgen05.commit) -> TMA
  __shared__ __align__(8) uint64_t acc_full[2];          // MMA (tcgen05.commit) -> drain: a group's accumulator is complete
  __shared__ __align__(8) uint64_t acc_empty[2];         // drain -> MMA: the accumulator may be overwritten
  __shared__ uint32_t tmem_base_s;
  __shared__ int abort_s, last_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int u = blockIdx.y, b = u / p.Hkv;
  const int split = blockIdx.x, S = gridDim.x;

  // the tokens this call adds to the sequence (the lengths are advanced by a later kernel of the same append)
  const int L = p.seq_lens[b];
  int n = n_new ? n_new[b] : max_new;
  n = max(0, min(n, max_new));
  if (L + n > p.max_context) n = 0;                      // reported by the copy kernel; nothing is added
  const int tiles_total = (n + kSuTile - 1) / kSuTile;
  const int tps = (tiles_total + S - 1) / S;             // tiles per split
  const int t_begin = min(tiles_total, split * tps);
  const int my_tiles = min(tiles_total, t_begin + tps) - t_begin;
  const size_t unit_tok0 = (size_t)u * p.max_blocks * p.B;

  if (tid == 0) {
    for (int s = 0; s < kSuStages; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], kSuTransformWarps / 2); mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&acc_full[a], 1); mbar_init(&acc_empty[a], kSuTransformWarps); }
    mbar_init_done();
    abort_s = 0;
  }
  if (warp == 1) {                                       // tensor memory for the 128 x 128 fp32 accumulator
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(kSuTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_base_s;
  volatile int* abort_flag = &abort_s;

  if (my_tiles > 0) {
    if (warp == 0) {
      // ---------------------------------------------------------------- producer ---------------------------------
      if (lane == 0) {
        int issued = 0;
        for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
          const int s = i % kSuStages;
          if (i >= kSuStages && !mbar_wait(&empty[s], ((i / kSuStages) - 1) & 1)) { atomicExch(&abort_s, 1); break; }
          const uint32_t base = smem_u32(smem_raw + (size_t)s * kSuStageBytes);
          const int row = (int)(unit_tok0 + (size_t)L + (size_t)(t_begin + i) * kSuTile);
          mbar_expect_tx(&full[s], 2 * kSuTileBytes);
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            tma_load_box(base + h * kSuHalfBytes, &map_k, h * 64, row, &full[s]);
            tma_load_box(base + 2 * kSuTileBytes + h * kSuHalfBytes, &map_v, h * 64, row, &full[s]);
          }
          issued = i + 1;
        }
        if (*abort_flag)                                 // let the copies in flight land before the CTA leaves
          for (int j = max(0, issued - kSuStages); j < issued; ++j) mbar_wait(&full[j % kSuStages], (j / kSuStages) & 1);
      }
    } else if (warp == 1) {
      // ---------------------------------------------------------------- MMA issuer -------------------------------
      if (lane == 0) {
        for (int i = 0; i < my_tiles && !*abort_flag; ++i) {
          const int s = i % kSuStages;
          const int g = i / kSuGroup, ab = g & 1;        // group of tiles and the accumulator it goes to
          const bool first = i % kSuGroup == 0, last = i % kSuGroup == kSuGroup - 1 || i == my_tiles - 1;
          if (first && g >= 2 && !mbar_wait(&acc_empty[ab], ((g >> 1) - 1) & 1)) { atomicExch(&abort_s, 1); break; }
          if (!mbar_wait(&ready[s], (i / kSuStages) & 1)) { atomicExch(&abort_s, 1); break; }
          tc_fence_after();
          const uint32_t base = smem_u32(smem_raw + (size_t)s * kSuStageBytes);
#pragma unroll
          for (int part = 0; part < 2; ++part)           // head of phi, then its remainder
#pragma unroll
            for (int kk = 0; kk < kSuTile / 16; ++kk)    // 16 tokens (two swizzle atoms of 8 rows) per instruction
              umma_bf16(tmem + ab * kSuD, umma_desc(base + part * kSuTileBytes + kk * 2048),
                        umma_desc(base + 2 * kSuTileBytes + kk * 2048), (!first || part > 0 || kk > 0) ? 1u : 0u);
          umma_commit(&empty[s]);                        // the stage may be refilled once these have read it
          if (last) umma_commit(&acc_full[ab]);          // and the group's sum may be drained
        }
      }
    } else {
      // ---------------------------------------------------------------- transform --------------------------------
      // Two groups of four warps take the tiles in turn, so that one group's waits (tile landed, proxy fence, drain)
      // overlap the other's arithmetic.  Thread tg of a group owns the 16-byte chunks tg, tg + 128, ... of a tile
      // (consecutive lanes on consecutive chunks: no bank conflicts), which lie in the rows tg / 8 + 16 k of both
      // halves.  The swizzle moves chunks only inside their 128-byte row, and phi is elementwise given the
      // token's log-sum-exp, so which channels a chunk holds does not matter here.
      const int wg = (warp - 2) >> 2, tg = (tid - 64) & 127;
      const int r0 = tg >> 3;
      const float a2 = p.phi_scale * kLog2e;
      const float* lse = p.tok_lse + unit_tok0 + L;
      bool ok = true;
      // drain role: row 32 (warp % 4) + lane of the accumulator (a warp reaches only those tensor-memory lanes),
      // columns 64 half ... 64 half + 63
      const int q = warp & 3, half = (warp - 2) >> 2;
      const int n_groups = (my_tiles + kSuGroup - 1) / kSuGroup;
      int drained = 0;                                   // groups added into the registers so far
      float acc[64];
#pragma unroll
      for (int x = 0; x < 64; ++x) acc[x] = 0.f;
      auto drain = [&](int g) {
        const int ab = g & 1;
        if (!mbar_wait(&acc_full[ab], (g >> 1) & 1)) { ok = false; return; }
        __syncwarp();                                    // the aligned tensor-memory loads want the warp converged
        tc_fence_after();
#pragma unroll
        for (int cb = 0; cb < 2; ++cb) {
          float v[32];
          tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(ab * kSuD + half * 64 + cb * 32), v);
#pragma unroll
          for (int x = 0; x < 32; ++x) acc[cb * 32 + x] += v[x];
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive1(&acc_empty[ab]);
      };
      // the tokens' log-sum-exps are fetched one tile ahead: a global load in the loop would be its critical path
      float lse_next[4];
      auto load_lse = [&](int i) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int pos = (t_begin + i) * kSuTile + r0 + 16 * k;
          lse_next[k] = (i < my_tiles && pos < n) ? __ldg(lse + pos) : 0.f;
        }
      };
      load_lse(wg);
      for (int i = wg; i < my_tiles && !*abort_flag; i += 2) {
        const int s = i % kSuStages;
        float nl2[4];
        bool valid[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          nl2[k] = -lse_next[k] * kLog2e;
          valid[k] = (t_begin + i) * kSuTile + r0 + 16 * k < n;   // token index among the new ones
        }
        load_lse(i + 2);
        if (!mbar_wait(&full[s], (i / kSuStages) & 1)) { ok = false; break; }
        unsigned char* st = smem_raw + (size_t)s * kSuStageBytes + tg * 16;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          uint4* kp = reinterpret_cast<uint4*>(st + j * 2048);
          uint4* lp = reinterpret_cast<uint4*>(st + kSuTileBytes + j * 2048);
          uint4 hi4 = make_uint4(0u, 0u, 0u, 0u), lo4 = hi4;
          if (valid[j & 3]) {
            const uint4 raw = *kp;
            const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
            uint32_t ho[4], lo[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float f0 = ex2(fmaf(__uint_as_float(w[e] << 16), a2, nl2[j & 3]));
              const float f1 = ex2(fmaf(__uint_as_float(w[e] & 0xffff0000u), a2, nl2[j & 3]));
              ho[e] = pack_bf16(f0, f1);
              lo[e] = pack_bf16(f0 - __uint_as_float(ho[e] << 16), f1 - __uint_as_float(ho[e] & 0xffff0000u));
            }
            hi4 = make_uint4(ho[0], ho[1], ho[2], ho[3]);
            lo4 = make_uint4(lo[0], lo[1], lo[2], lo[3]);
          } else {
            *reinterpret_cast<uint4*>(st + 2 * kSuTileBytes + j * 2048) = hi4;   // V of a row that is not a new token
          }
          *kp = hi4;
          *lp = lo4;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic writes -> visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive1(&ready[s]);
        // one accumulator group behind the issuer: by now those instructions have long completed
        while (ok && drained < i / kSuGroup) { drain(drained); ++drained; }
        if (!ok) break;
      }
      while (ok && !*abort_flag && drained < n_groups) { drain(drained); ++drained; }
      if (!ok) atomicExch(&abort_s, 1);

      // ---------------------------------------------------------------- epilogue ---------------------------------
      if (!*abort_flag) {
        const int row = q * 32 + lane;
        float* dst = (S > 1 ? p.state_part + ((size_t)u * S + split) * D * D : p.state + (size_t)u * D * D) + (size_t)row * D + half * 64;
#pragma unroll
        for (int x = 0; x < 64; x += 4) {
          float4* d4 = reinterpret_cast<float4*>(dst + x);
          float4 o = make_float4(acc[x], acc[x + 1], acc[x + 2], acc[x + 3]);
          if (S == 1) { const float4 old = *d4; o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w; }
          *d4 = o;
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kSuTmemCols) : "memory");
  }
  if (tid == 0 && abort_s) atomicExch(p.status, kStatusTimeout);
  if (S == 1) return;

  // ------------------------------------------------------------------ last CTA of the unit: partials -> S_bar ----
  if (tid == 0) {
    __threadfence();
    const int t = atomicAdd(&p.state_ticket[u], 1);
    last_s = (t == S - 1);
    if (last_s) p.state_ticket[u] = 0;
    __threadfence();
  }
  __syncthreads();
  if (!last_s || tiles_total == 0 || abort_s) return;
  const int live = (tiles_total + tps - 1) / tps;        // splits that had tiles, in order
  const float4* part = reinterpret_cast<const float4*>(p.state_part + (size_t)u * S * D * D);
  float4* st4 = reinterpret_cast<float4*>(p.state + (size_t)u * D * D);
  for (int idx = tid; idx < D * D / 4; idx += kSuThreads) {
    float4 acc = __ldcg(part + idx);
    for (int s2 = 1; s2 < live; ++s2) {
      const float4 x = __ldcg(part + (size_t)s2 * (D * D / 4) + idx);
      acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    }
    float4 o = st4[idx];
    o.x += acc.x; o.y += acc.y; o.z += acc.z; o.w += acc.w;
    st4[idx] = o;
  }
}

// Splits of a unit's tokens: enough CTAs to fill a 148-SM part once (one CTA per SM), at most 16 per unit.  A
// fixed SM count, because the partial buffer is sized from the configuration alone, before any device is known.
int state_umma_splits(int units) {
  int s = 148 / (units > 0 ? units : 1);
  return s < 1 ? 1 : (s > 16 ? 16 : s);
}

size_t state_umma_part_bytes(int units, int d) {
  const int s = state_umma_splits(units);
  return s > 1 ? (size_t)units * s * d * d * 4 : 0;
}

cudaError_t launch_state_umma(const Params& p, const AttendMaps* maps, const int* n_new, int max_new, cudaStream_t stream) {
  const int U = p.batch * p.Hkv;
  const int S = state_umma_splits(U);
  cudaError_t e = cudaFuncSetAttribute(state_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSuSmemBytes);
  if (e != cudaSuccess) return e;
  state_umma_kernel<<<dim3(S, U), kSuThreads, kSuSmemBytes, stream>>>(
      p, *reinterpret_cast<const CUtensorMap*>(maps->k), *reinterpret_cast<const CUtensorMap*>(maps->v), n_new, max_new);
  ++g_launch_count;
  return cudaGetLastError();
}

}  // namespace spla
