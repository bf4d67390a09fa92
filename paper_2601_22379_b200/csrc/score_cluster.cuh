// Block score + selection, cluster edition: the CTAs that score one (sequence, KV head) unit form a thread-block
// cluster, so the selection no longer runs as a serial tail in one CTA behind a global-memory hand-off.
//
//   phase A  every CTA streams its share of the unit's statistics records through a ring of shared-memory
//            stages filled by bulk asynchronous copies (full/empty mbarriers; one thread feeds the ring) and keeps the
//            Taylor log masses ell^m_i (Section 3.1 of the paper, Eq. taylor-2nd, diagonal covariance) and its
//            per-head (max, sum exp) in shared memory;
//   sync 1   hardware cluster barrier;
//   phase B  every CTA reads the partial normalisers of its siblings over distributed shared memory, forms the
//            aggregated BlockScore of its own blocks (Section 2.2: per-head softmax over blocks, summed over the
//            group), picks its best min(k, n) blocks and pushes them into the leader CTA's memory;
//   sync 2   hardware cluster barrier;
//   phase C  the leader picks the top k of the <= 16 x 64 candidates (forced sink / local blocks carry the
//            maximal key; Section 4 "Sparsity Specifications") and writes them in ascending order, while its
//            siblings compute o_bar = phi(q) S_bar, the part of the residual branch that needs no selection.
// Ordering everywhere is (score descending, block index ascending).  The only waits are the two hardware
// barriers and bounded mbarrier polls.  No multicast is used.
//
// The body is a device function: it is the whole of the score + select kernel (spla_select, and spla_decode where the
// fused kernel does not apply) and the first half of the fused decode kernel (decode_fused.cuh).
#pragma once

#include "spla_internal.h"
#include "state_role.cuh"
#include "topk_select.cuh"

namespace spla {

namespace {

constexpr int kRecPerWarp = 4;                           // statistics records per warp per ring stage
constexpr int kStages = 3;
constexpr int kMaxCluster = 16;
constexpr int kSlotRec = 16;                             // records per slot of the tensor-core streaming path

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// Order-preserving map of a float onto an unsigned integer (larger float <=> larger key; every key is above 0).
__device__ __forceinline__ uint32_t float_order_key(float x) {
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float float_from_order_key(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
  const float nm = fmaxf(m, m2);
  if (nm > -INFINITY) s = s * __expf(m - nm) + s2 * __expf(m2 - nm);
  m = nm;
}

// Sums N per-lane values over aligned groups of W lanes (W = 16 or 32, N <= W a power of two) by halving:
// afterwards v[0] of lane l holds the group total of the value with index (l % W) / (W / N).
template <int N, int W>
__device__ __forceinline__ void group_reduce_multi(float (&v)[N], int lane) {
  int off = W / 2;
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

// Layout of the dynamic shared memory (identical in every CTA, which distributed shared memory relies on).
template <int D, int GP, typename ST, int NWP>
struct Smem {
  static constexpr int kStageRec = NWP * kRecPerWarp;              // statistics records per ring stage
  static constexpr int kRecBytes = 2 * D * (int)sizeof(ST);        // ST: element type of the statistics records
  static constexpr int kStageBytes = kStageRec * kRecBytes;
  // tensor-core streaming (groups of up to four heads): the ring is cut into slots of 16 records, one MMA tile each
  static constexpr bool kMma = GP <= 4 && sizeof(ST) == 2;         // 16-bit records, groups of up to four heads
  static constexpr int kSlotBytes = kSlotRec * kRecBytes;
  static constexpr int kSlots = NWP;                               // one ring position per warp
  static constexpr int kStreamBytes = kMma ? kSlots * kSlotBytes : kStages * kStageBytes;
  // after streaming the ring is dead and holds the selection's work arrays:
  static constexpr int kKeys = 0;                                   // uint32 [1024]        this CTA's block keys
  static constexpr int kCandKey = kKeys + 1024 * 4;                 // uint32 [16][64]      (the leader's copy is the live one)
  static constexpr int kCandIdx = kCandKey + kMaxCluster * kMaxTopK * 4;
  static constexpr int kCandCnt = kCandIdx + kMaxCluster * kMaxTopK * 4;   // int [16]
  static constexpr int kFlatKey = kCandCnt + 64;                    // uint32 [1024]
  static constexpr int kFlatIdx = kFlatKey + kMaxCluster * kMaxTopK * 4;
  static constexpr int kSelTmp = kFlatIdx + kMaxCluster * kMaxTopK * 4;    // int [64]
  static constexpr int kScratch = (kSelTmp + kMaxTopK * 4 + 15) / 16 * 16; // TopkScratch
  static constexpr int kWorkEnd = (kScratch + (int)sizeof(TopkScratch) + 1023) / 1024 * 1024;
  // the ring, padded where the work arrays need more than its stages
  // ... and, for the fused decode kernel, padded to 68 KB: the attend phase lays its K/V tile ring (at most 66 KB) over
  // this area, and the tile copies must stay clear of the fixed region below, which holds this phase's mbarrier
  // objects (never invalidated: overwriting them with tile data corrupted value rows, found with NaN-filled memory)
  static constexpr int kRingBytes0 = kStreamBytes > kWorkEnd ? kStreamBytes : kWorkEnd;
  static constexpr int kRingBytes = kRingBytes0 > 68 * 1024 ? kRingBytes0 : 68 * 1024;
  // fixed region after the ring:
  static constexpr int kPart = kRingBytes;                          // float [GP][2]  this CTA's (max, sum)
  static constexpr int kAllPart = kPart + GP * 2 * 4;               // float [16][GP][2]
  static constexpr int kLse = kAllPart + kMaxCluster * GP * 2 * 4;  // float [GP]
  static constexpr int kWred = kLse + GP * 4;                       // float [NWP][GP][2]
  static constexpr int kBars = (kWred + NWP * GP * 2 * 4 + 7) / 8 * 8;            // uint64: full / empty per stage, or one per slot
  static constexpr int kNumBars = NWP > 2 * kStages ? NWP : 2 * kStages;
  static constexpr int kEll = (kBars + kNumBars * 8 + 15) / 16 * 16;               // float [G][chunk]
};

}  // namespace

// WIN: strided selection windows (several statistics records per block, max-pooled); without them the kernel is
// compiled with one record per block as a constant.
// EARLY: the kernel follows the append of the same step in the stream and does not wait for it before streaming:
// the blocks that were complete before that append (at most `pending_new` tokens per sequence) cannot change any
// more, so their statistics are streamed while the append still runs; only then does the kernel wait for the
// append, read the final length and take the few remaining blocks (those the append wrote to) from global memory.
// ST: element type of the statistics records (float, or __nv_bfloat16 with half the bytes to stream).
// On return the selection of the unit is in p.sel / p.n_sel (and sel_user), written by the cluster's leader, and the
// o_bar partials in p.obar_part; every thread of every CTA of the cluster returns (nobody has left the kernel).
template <int D, int GP, bool WIN, bool EARLY, typename ST, int NWP>
// `sel_share` (fused kernel only, else null): a shared-memory array of kMaxTopK + 2 ints at the same place in every CTA
// of the cluster; the leader also writes the selection there, in every CTA, followed by the count and the length.
__device__ __forceinline__ void score_cluster_body(const Params& p, const void* __restrict__ q_raw, int q_is_bf16,
                                                   int* __restrict__ sel_user, int pending_new, unsigned char* smem_raw,
                                                   int* sel_share = nullptr) {
  using SM = Smem<D, GP, ST, NWP>;
  constexpr int kCsConsumers = NWP;             // warps; all consume, lane 0 of warp 0 also feeds the ring
  constexpr int kCsThreads = NWP * 32;
  constexpr int kStageRec = SM::kStageRec;
  constexpr int UNR = kRecPerWarp;              // records per warp per stage
  constexpr int W = GP <= 4 ? 16 : 32;          // lanes that share one record
  constexpr int NGRP = 32 / W;                  // records a warp works on side by side
  constexpr int PASSES = UNR / NGRP;
  constexpr int VECW = D / W;                   // floats of the mean (and of the variance) per lane
  constexpr int NV = 2 * GP;
  constexpr int LPV = W / NV;                   // lanes holding a copy of each reduced value
  constexpr int FB = LPV < PASSES ? LPV : PASSES;
  static_assert(LPV >= 1, "group too large for the lane layout");

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int CS = gridDim.x;
  const int rank = blockIdx.x;
  const int G = p.G;
  const int u = blockIdx.y;
  const int b = u / p.Hkv, h = u % p.Hkv;

  float* part_s = reinterpret_cast<float*>(smem_raw + SM::kPart);
  float* all_part = reinterpret_cast<float*>(smem_raw + SM::kAllPart);
  float* lse_s = reinterpret_cast<float*>(smem_raw + SM::kLse);
  float* wred = reinterpret_cast<float*>(smem_raw + SM::kWred);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + SM::kBars);
  uint64_t* empty = full + kStages;
  float* ell_s = reinterpret_cast<float*>(smem_raw + SM::kEll);          // [G][chunk] log mass per block
  __shared__ int err_s;

  const int chunk = p.chunk;                      // blocks per CTA
  const int NW = WIN ? p.NW : 1;                  // selection windows per block; a "record" is one window
  const int cta_blk0 = rank * chunk;              // first block of this CTA's share
  const int rec_begin = cta_blk0 * NW;            // (a CTA that has records starts at its share's first block)
  const ST* stats_u = reinterpret_cast<const ST*>(p.stats) + (size_t)u * p.max_blocks * NW * 2 * D;
  if (tid == 0) {                               // nothing here depends on the preceding kernel
    if constexpr (SM::kMma) { for (int s = 0; s < SM::kSlots; ++s) mbar_init(&full[s], 1); }
    else { for (int s = 0; s < kStages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kCsConsumers); } }
    err_s = 0;
  }
  if (!EARLY) {
    pdl_wait();                                 // everything the preceding kernels wrote (statistics, lengths, q) is visible
    pdl_launch_dependents();                    // only now may the next kernel begin its prologue: it reads q before its own wait
  }

  // ---- the query loads go out first and the ring is started as soon as the sequence length is known: a small
  // load issued into the streaming traffic would take several microseconds.
  // Lane layout: `hl` of W lanes covers d = c * 4 W + 4 hl .. + 3.
  const int hl = lane % W, grp = lane / W;
  constexpr int CW = VECW >= 4 ? 4 : VECW;      // floats per vector load
  constexpr int NC = VECW / CW;
  // Tensor-core streaming (16-bit records, groups of up to four heads): a slot of 16 records is the A operand of
  // mma.m16n8k16 (16 x d, row-major, as stored), the B operand's eight columns are the group's scaled queries, each
  // split in two bf16 parts, bf16(q) and bf16(q - bf16(q)) (column n: head n / 2, part n % 2), whose products are
  // added after the MMA: the query enters with 16 significant bits, the statistics exactly, the sums are fp32.
  // Thread (g8, t4) owns 16 consecutive bytes of every 64 of a record half (mean or variance), which it fetches with
  // one 128-bit load per row; the k index inside an MMA is a permutation of the channels, the same for A and B.
  constexpr bool MMA = SM::kMma;
  constexpr int NJ = D * (int)sizeof(ST) / 64;   // 16-byte chunks per thread and record half
  const int g8 = lane >> 2, t4 = lane & 3;
  uint32_t bq[MMA ? NJ : 1][4], bv[MMA ? NJ : 1][4];
  float qm[GP][VECW], qv[GP][VECW];
  if constexpr (MMA) {
    const int head = g8 >> 1, part = g8 & 1;
#pragma unroll
    for (int j = 0; j < NJ; ++j) {
      float x[8];                                // channels 32 j + 8 t4 .. + 7
      if (head < G) {
        const size_t qoff = ((size_t)b * p.Hq + (size_t)h * G + head) * D + (size_t)j * 32 + t4 * 8;
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float y[4];
          if (q_is_bf16) load_vec<4>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff + c * 4, y);
          else load_vec<4>(reinterpret_cast<const float*>(q_raw) + qoff + c * 4, y);
#pragma unroll
          for (int v = 0; v < 4; ++v) x[c * 4 + v] = y[v];
        }
      } else {
#pragma unroll
        for (int v = 0; v < 8; ++v) x[v] = 0.f;
      }
      float qa[8], qb2[8];                       // this thread's part of q_hat and of q_hat^2 / 2
#pragma unroll
      for (int v = 0; v < 8; ++v) {
        const float qh = x[v] * p.sm_scale;
        const float qq = (p.flags & 2u) ? 0.f : 0.5f * qh * qh;
        const float h1 = __bfloat162float(__float2bfloat16_rn(qh)), h2 = __bfloat162float(__float2bfloat16_rn(qq));
        qa[v] = part ? qh - h1 : h1;
        qb2[v] = part ? qq - h2 : h2;
      }
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        bq[j][v] = pack_bf16(qa[2 * v], qa[2 * v + 1]);
        bv[j][v] = pack_bf16(qb2[2 * v], qb2[2 * v + 1]);
      }
    }
  }
#pragma unroll
  for (int g = 0; g < GP && !MMA; ++g) {
    if (g < G) {
      const size_t qrow = ((size_t)b * p.Hq + (size_t)h * G + g) * D;
#pragma unroll
      for (int c = 0; c < NC; ++c) {
        float x[CW];
        const size_t qoff = qrow + (size_t)c * W * 4 + hl * CW;
        if (q_is_bf16) load_vec<CW>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
        else load_vec<CW>(reinterpret_cast<const float*>(q_raw) + qoff, x);
#pragma unroll
        for (int v = 0; v < CW; ++v) qm[g][c * CW + v] = x[v];
      }
    } else {
#pragma unroll
      for (int v = 0; v < VECW; ++v) qm[g][v] = 0.f;
    }
  }
  // EARLY: this length may be the one before or after the running append; minus `pending_new` it bounds from below
  // the tokens that were there before it
  int L0;
  if (EARLY) {                                    // one read for the whole CTA: the value may change under our feet
    __shared__ int l0_s;
    if (tid == 0) l0_s = cover_len(p, checked_len(p, b), (long long)CS * chunk * p.B);
    __syncthreads();
    L0 = l0_s;
  } else {
    L0 = cover_len(p, checked_len(p, b), (long long)CS * chunk * p.B);
  }
  int L = L0;
  int nblk = (L + p.B - 1) / p.B;
  const int nblk_stream = EARLY ? max(0, L0 - pending_new) / p.B : nblk;    // blocks whose records the ring may fetch
  const int n_stream = max(0, min(cta_blk0 + chunk, nblk_stream) - cta_blk0) * NW;
  int blk_begin = min(nblk, cta_blk0);
  int nb_my = min(nblk, blk_begin + chunk) - blk_begin;   // blocks of this CTA (EARLY: refreshed after the wait)
  int n_my = nb_my * NW;                          // records of this CTA
  const int n_rounds = (n_stream + kStageRec - 1) / kStageRec;

  auto issue = [&](int r) {                      // thread 0 only: one bulk copy fills stage r % kStages
    const int s = r % kStages;
    int nrec = min(kStageRec, n_stream - r * kStageRec);
    if (p.flags & kDebugBounds) {                // checked build: the copy must stay inside the unit's records
      const int room = p.max_blocks * NW - (rec_begin + r * kStageRec);
      if (nrec > room) { atomicExch(p.status, kStatusBounds); nrec = max(room, 0); }
    }
    const uint32_t bytes = (uint32_t)nrec * SM::kRecBytes;
    mbar_expect_tx(&full[s], bytes + (uint32_t)p.dbg_tx_extra);
    bulk_g2s(smem_raw + (size_t)s * SM::kStageBytes, stats_u + (size_t)(rec_begin + r * kStageRec) * 2 * D, bytes, &full[s]);
  };
  // tensor-core path: slot r (16 records) goes to ring position r % kSlots and is consumed by the warp of that
  // number, which then refills its position itself with slot r + kSlots (so every warp sees the phases of its
  // barrier in order)
  const int n_slots = (n_stream + kSlotRec - 1) / kSlotRec;
  auto issue_slot = [&](int r) {                // one thread
    const int pos = r % SM::kSlots;
    int nrec = min(kSlotRec, n_stream - r * kSlotRec);
    if (p.flags & kDebugBounds) {                // checked build: the copy must stay inside the unit's records
      const int room = p.max_blocks * NW - (rec_begin + r * kSlotRec);
      if (nrec > room) { atomicExch(p.status, kStatusBounds); nrec = max(room, 0); }
    }
    const uint32_t bytes = (uint32_t)nrec * SM::kRecBytes;
    mbar_expect_tx(&full[pos], bytes + (uint32_t)p.dbg_tx_extra);
    bulk_g2s(smem_raw + (size_t)pos * SM::kSlotBytes, stats_u + (size_t)(rec_begin + r * kSlotRec) * 2 * D, bytes, &full[pos]);
  };
  if (tid == 0) {
    if constexpr (MMA) { for (int r = 0; r < min(SM::kSlots, n_slots); ++r) issue_slot(r); }
    else { for (int r = 0; r < min(kStages, n_rounds); ++r) issue(r); }
  }
#pragma unroll
  for (int g = 0; g < GP && !MMA; ++g) {
#pragma unroll
    for (int v = 0; v < VECW; ++v) {
      qm[g][v] *= p.sm_scale;
      qv[g][v] = (p.flags & 2u) ? 0.f : 0.5f * qm[g][v] * qm[g][v];
    }
  }
  if (WIN)                                      // pooled slots start below every key
    for (int x = tid; x < G * chunk; x += kCsThreads) reinterpret_cast<uint32_t*>(ell_s)[x] = 0u;
  __syncthreads();                              // the barrier initialisation is visible to every consumer

  {
    // After the group reduction the first W/2 lanes of a group hold the mean dots and the others the variance
    // dots, value index (hl % (W/2)) / LPV, each on LPV lanes.  Copy lane `sub` keeps the result of pass `sub`,
    // so the log / exp work of FB passes runs side by side.
    const int my_g = (hl % (W / 2)) / LPV;
    const int sub = hl % LPV;
    const bool fin_lane = hl < W / 2 && sub < FB && my_g < G;
    const float ln_full = logf((float)p.B);
    // EARLY: while streaming, every block is a full one; the last block of the sequence comes after the wait
    int nblk_fin = EARLY ? 0x7fffffff : nblk;
    int n_last = L - (nblk - 1) * p.B;           // tokens of the last block
    float ln_last = logf((float)max(1, n_last));
    const float ln_win = logf((float)p.win_C);
    const unsigned nw_magic = 0xffffffffu / (unsigned)NW + 1u;   // floor(x / NW) = umulhi(x, magic) for x < 2^16, NW <= 8
    float run_max = -INFINITY, run_sum = 0.f;

    // Tensor-core path: one slot of 16 records -> dots of head t4 with records g8 and g8 + 8 of the slot -> log
    // masses.  `li0` is the CTA-local index of the slot's first record, `limit` the number of local records that
    // exist for this call.  Rows past the limit hold stale bytes; every row is independent and theirs are dropped.
    auto consume_slot = [&](const unsigned char* slot, int li0, int limit) {
      float cm[4] = {0.f, 0.f, 0.f, 0.f}, cv[4] = {0.f, 0.f, 0.f, 0.f};
      const unsigned char* r0 = slot + (size_t)g8 * SM::kRecBytes + t4 * 16;
      const unsigned char* r1 = r0 + 8 * SM::kRecBytes;
      constexpr int HALF = SM::kRecBytes / 2;                      // the variance follows the mean
#pragma unroll
      for (int j = 0; j < (MMA ? NJ : 0); ++j) {
        const uint4 m0 = *reinterpret_cast<const uint4*>(r0 + j * 64), m1 = *reinterpret_cast<const uint4*>(r1 + j * 64);
        const uint4 v0 = *reinterpret_cast<const uint4*>(r0 + HALF + j * 64), v1 = *reinterpret_cast<const uint4*>(r1 + HALF + j * 64);
        mma_bf16(cm, m0.x, m1.x, m0.y, m1.y, bq[j][0], bq[j][1]);
        mma_bf16(cv, v0.x, v1.x, v0.y, v1.y, bv[j][0], bv[j][1]);
        mma_bf16(cm, m0.z, m1.z, m0.w, m1.w, bq[j][2], bq[j][3]);
        mma_bf16(cv, v0.z, v1.z, v0.w, v1.w, bv[j][2], bv[j][3]);
      }
      // columns 2 t4 and 2 t4 + 1 are the two query parts of head t4
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
        const float dm = cm[2 * hf] + cm[2 * hf + 1], dv = cv[2 * hf] + cv[2 * hf + 1];
        const int li = li0 + g8 + 8 * hf;
        if (t4 < G && li < limit) {
          if (!WIN) {
            const float ell = (rec_begin + li == nblk_fin - 1 ? ln_last : ln_full) + dm + __logf(1.f + dv);
            ell_s[t4 * chunk + li] = ell;
            const float nm = fmaxf(run_max, ell);
            run_sum = run_sum * __expf(run_max - nm) + __expf(ell - nm);
            run_max = nm;
          } else {
            // strided windows (Section 3.1, "Strided Block Selection"): log mass of window w of a block,
            // max-pooled into the block's slot right away through an order-preserving integer key
            const int lb = (int)__umulhi((unsigned)li, nw_magic), w = li - lb * NW;   // li / NW without a division
            float ln_n = ln_win;
            if (cta_blk0 + lb == nblk_fin - 1) {
              const int cnt = min(p.win_C, n_last - w * p.win_s);
              ln_n = cnt > 0 ? logf((float)cnt) : -INFINITY;
            }
            atomicMax(reinterpret_cast<uint32_t*>(ell_s) + t4 * chunk + lb, float_order_key(ln_n + dm + __logf(1.f + dv)));
          }
        }
      }
    };
    if constexpr (MMA) {
#pragma unroll 1
      for (int r = warp; r < n_slots; r += SM::kSlots) {          // warp w owns ring position w
        const int pos = r % SM::kSlots;
        if (!mbar_wait(&full[pos], (r / SM::kSlots) & 1, p.wait_limit)) { if (lane == 0) atomicExch(&err_s, 1); break; }
        consume_slot(smem_raw + (size_t)pos * SM::kSlotBytes, r * kSlotRec, n_stream);
        __syncwarp();                                              // every lane has its operands: the slot is free
        if (lane == 0 && r + SM::kSlots < n_slots) issue_slot(r + SM::kSlots);
      }
    }

    // dots of the records a warp holds in registers -> log masses (and, with whole blocks, the running normaliser);
    // `limit` is the number of local records that exist for this call
    auto finish_passes = [&](int l0, int limit, float (&mean)[PASSES][VECW], float (&var)[PASSES][VECW]) {
#pragma unroll
        for (int p0 = 0; p0 < PASSES; p0 += FB) {
          float dm_keep = 0.f, dv_keep = 0.f;
#pragma unroll
          for (int pp = 0; pp < FB; ++pp) {
            float vals[NV];
#pragma unroll
            for (int g = 0; g < GP; ++g) {
              // packed fp32 FMAs (two products per instruction): even and odd channels accumulate side by side
              float2 am = make_float2(0.f, 0.f), av = make_float2(0.f, 0.f);
              if (GP <= 4 || g < G) {              // (groups of 5 to 7 heads: the padded heads' products are skipped)
#pragma unroll
                for (int v = 0; v < VECW; v += 2) {
                  am = __ffma2_rn(make_float2(qm[g][v], qm[g][v + 1]), make_float2(mean[p0 + pp][v], mean[p0 + pp][v + 1]), am);
                  av = __ffma2_rn(make_float2(qv[g][v], qv[g][v + 1]), make_float2(var[p0 + pp][v], var[p0 + pp][v + 1]), av);
                }
              }
              vals[g] = am.x + am.y;
              vals[GP + g] = av.x + av.y;
            }
            group_reduce_multi<NV, W>(vals, lane);
            const float other = __shfl_xor_sync(0xffffffffu, vals[0], W / 2);   // variance dot of the same head
            if (sub == pp) { dm_keep = vals[0]; dv_keep = other; }
          }
          const int li = l0 + (p0 + sub) * NGRP + grp;
          if (fin_lane && li < limit) {
            if (!WIN) {
              const float ell = (rec_begin + li == nblk_fin - 1 ? ln_last : ln_full) + dm_keep + __logf(1.f + dv_keep);
              ell_s[my_g * chunk + li] = ell;
              const float nm = fmaxf(run_max, ell);
              run_sum = run_sum * __expf(run_max - nm) + __expf(ell - nm);
              run_max = nm;
            } else {
              // strided windows (Section 3.1, "Strided Block Selection"): log mass of window w of a block,
              // max-pooled into the block's slot right away through an order-preserving integer key
              const int lb = (int)__umulhi((unsigned)li, nw_magic), w = li - lb * NW;   // li / NW without a division
              float ln_n = ln_win;
              if (cta_blk0 + lb == nblk_fin - 1) {
                const int cnt = min(p.win_C, n_last - w * p.win_s);
                ln_n = cnt > 0 ? logf((float)cnt) : -INFINITY;
              }
              atomicMax(reinterpret_cast<uint32_t*>(ell_s) + my_g * chunk + lb, float_order_key(ln_n + dm_keep + __logf(1.f + dv_keep)));
            }
          }
        }
    };
#pragma unroll 1
    for (int r = 0; r < (MMA ? 0 : n_rounds); ++r) {
      const int s = r % kStages;
      if (!mbar_wait(&full[s], (r / kStages) & 1, p.wait_limit)) { if (lane == 0) atomicExch(&err_s, 1); break; }
      const int l0 = r * kStageRec + warp * UNR;                       // first record of this warp, CTA-local
      const ST* st = reinterpret_cast<const ST*>(smem_raw + (size_t)s * SM::kStageBytes) + (size_t)(warp * UNR) * 2 * D;
      float mean[PASSES][VECW], var[PASSES][VECW];
#pragma unroll
      for (int ps = 0; ps < PASSES; ++ps) {
        const int rec = ps * NGRP + grp;
        if (l0 + rec < n_stream) {
#pragma unroll
          for (int c = 0; c < NC; ++c) {
            float a[CW], bb[CW];
            load_vec<CW>(st + (size_t)rec * 2 * D + c * W * 4 + hl * CW, a);
            load_vec<CW>(st + (size_t)rec * 2 * D + D + c * W * 4 + hl * CW, bb);
#pragma unroll
            for (int v = 0; v < CW; ++v) { mean[ps][c * CW + v] = a[v]; var[ps][c * CW + v] = bb[v]; }
          }
        } else {
#pragma unroll
          for (int v = 0; v < VECW; ++v) { mean[ps][v] = 0.f; var[ps][v] = 0.f; }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);                            // the stage is in registers: hand it back
      if (tid == 0 && r + kStages < n_rounds) {                         // refill it once every warp has done the same
        if (mbar_wait(&empty[s], (r / kStages) & 1, p.wait_limit)) issue(r + kStages);
        else atomicExch(&err_s, 1);
      }
      __syncwarp();
      if (l0 < n_stream) finish_passes(l0, n_stream, mean, var);
    }
    if constexpr (EARLY) {
      // now the append must be complete: final length, and the blocks it wrote to (the last ones of the sequence, a
      // handful of records) through plain loads into stage 0, one more round
      pdl_wait();
      pdl_launch_dependents();
      L = cover_len(p, checked_len(p, b), (long long)CS * chunk * p.B);
      nblk = (L + p.B - 1) / p.B;
      blk_begin = min(nblk, cta_blk0);
      nb_my = min(nblk, blk_begin + chunk) - blk_begin;
      n_my = nb_my * NW;
      nblk_fin = nblk;
      n_last = L - (nblk - 1) * p.B;
      ln_last = logf((float)max(1, n_last));
      const int n_late = n_my - n_stream;
      if (n_late > 0) {                            // CTA-uniform
        __syncthreads();                           // every warp is done with the ring
        float4* dst = reinterpret_cast<float4*>(smem_raw);
        const float4* src = reinterpret_cast<const float4*>(stats_u + (size_t)(rec_begin + n_stream) * 2 * D);
        for (int x = tid; x < n_late * (SM::kRecBytes / 16); x += kCsThreads) dst[x] = __ldcg(src + x);
        __syncthreads();
        if constexpr (MMA)
          for (int base = warp * kSlotRec; base < n_late; base += kCsConsumers * kSlotRec)
            consume_slot(smem_raw + (size_t)base * SM::kRecBytes, n_stream + base, n_my);
        for (int base = 0; base < (MMA ? 0 : n_late); base += kStageRec) {
          const int l0 = n_stream + base + warp * UNR;
          const ST* st = reinterpret_cast<const ST*>(smem_raw) + (size_t)(base + warp * UNR) * 2 * D;
          float mean[PASSES][VECW], var[PASSES][VECW];
#pragma unroll
          for (int ps = 0; ps < PASSES; ++ps) {
            const int rec = ps * NGRP + grp;
            if (l0 + rec < n_my) {
#pragma unroll
              for (int c = 0; c < NC; ++c) {
                float a[CW], bb[CW];
                load_vec<CW>(st + (size_t)rec * 2 * D + c * W * 4 + hl * CW, a);
                load_vec<CW>(st + (size_t)rec * 2 * D + D + c * W * 4 + hl * CW, bb);
#pragma unroll
                for (int v = 0; v < CW; ++v) { mean[ps][c * CW + v] = a[v]; var[ps][c * CW + v] = bb[v]; }
              }
            } else {
#pragma unroll
              for (int v = 0; v < VECW; ++v) { mean[ps][v] = 0.f; var[ps][v] = 0.f; }
            }
          }
          if (l0 < n_my) finish_passes(l0, n_my, mean, var);
        }
      }
    }
    if (WIN) {
      // the pooled keys back to floats, and this CTA's (max, sum exp) per head from them; lane 0 of every warp
      // then holds the warp's pair
      __syncthreads();
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        float m = -INFINITY, sm = 0.f;
        if (g < G)
          for (int lb = tid; lb < nb_my; lb += kCsThreads) {
            const float x = float_from_order_key(reinterpret_cast<const uint32_t*>(ell_s)[g * chunk + lb]);
            ell_s[g * chunk + lb] = x;
            lse_merge(m, sm, x, 1.f);
          }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, sm, o);
          lse_merge(m, sm, m2, s2);
        }
        if (lane == 0) { wred[(warp * GP + g) * 2 + 0] = m; wred[(warp * GP + g) * 2 + 1] = sm; }
      }
    }
    if constexpr (MMA) {
      // lanes with the same t4 hold partial normalisers of head t4: fold over g8
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, run_max, o), s2 = __shfl_xor_sync(0xffffffffu, run_sum, o);
        lse_merge(run_max, run_sum, m2, s2);
      }
      if (!WIN && lane < G) {
        wred[(warp * GP + lane) * 2 + 0] = run_max;
        wred[(warp * GP + lane) * 2 + 1] = run_sum;
      }
    }
    // fold the finalising lanes of a head: copy lanes (xor < LPV), then the record groups of the warp (xor W)
#pragma unroll
    for (int o = 1; o < (MMA ? 0 : FB); o <<= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, run_max, o), s2 = __shfl_xor_sync(0xffffffffu, run_sum, o);
      lse_merge(run_max, run_sum, m2, s2);
    }
    if constexpr (NGRP == 2 && !MMA) {
      const float m2 = __shfl_xor_sync(0xffffffffu, run_max, 16), s2 = __shfl_xor_sync(0xffffffffu, run_sum, 16);
      lse_merge(run_max, run_sum, m2, s2);
    }
    if (!MMA && !WIN && fin_lane && sub == 0 && grp == 0) {
      wred[(warp * GP + my_g) * 2 + 0] = run_max;
      wred[(warp * GP + my_g) * 2 + 1] = run_sum;
    }
  }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY, s = 0.f;
#pragma unroll
    for (int w = 0; w < kCsConsumers; ++w) lse_merge(m, s, wred[(w * GP + tid) * 2], wred[(w * GP + tid) * 2 + 1]);
    part_s[tid * 2] = m;
    part_s[tid * 2 + 1] = s;
  }
  if (tid == 0 && err_s) atomicExch(p.status, kStatusTimeout);

  cluster_sync_all();                                                   // ---- sync 1: partial normalisers visible

  // ------------------------------------------------------------------ phase B -------------------------------
  // Log-sum-exp of every head over the whole cluster, by each warp on its own (no block barrier): lane p
  // fetches the (max, sum) pair of CTA p / GP and head p % GP over distributed shared memory, then the lanes
  // of one head are folded with shuffles.
  float lse_r[GP];
  {
    float m = -INFINITY, sm = 0.f;
    for (int pr = lane; pr < CS * GP; pr += 32) {
      const int r = pr / GP, g = pr % GP;
      if (g < G) {
        const uint32_t remote = map_to_rank(smem_u32(part_s + g * 2), (uint32_t)r);
        lse_merge(m, sm, ld_dsmem_f32(remote), ld_dsmem_f32(remote + 4));
      }
    }
#pragma unroll
    for (int o = GP; o < 32; o <<= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, sm, o);
      lse_merge(m, sm, m2, s2);
    }
    const float lse = m + __logf(sm);
#pragma unroll
    for (int g = 0; g < GP; ++g) lse_r[g] = __shfl_sync(0xffffffffu, lse, g);
  }

  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + SM::kKeys);
  TopkScratch* scratch = reinterpret_cast<TopkScratch*>(smem_raw + SM::kScratch);
  const int k_eff = min(p.top_k, nblk);
  const uint32_t cand_key0 = map_to_rank(smem_u32(smem_raw + SM::kCandKey), 0u) + (uint32_t)rank * kMaxTopK * 4;
  const uint32_t cand_idx0 = map_to_rank(smem_u32(smem_raw + SM::kCandIdx), 0u) + (uint32_t)rank * kMaxTopK * 4;
  auto push = [&](int slot, uint32_t key, int idx) {                  // into the leader's candidate table
    st_dsmem_u32(cand_key0 + (uint32_t)slot * 4, key);
    st_dsmem_u32(cand_idx0 + (uint32_t)slot * 4, (uint32_t)idx);
  };
  if (tid == 0) { scratch->lo = 0xffffffffu; scratch->hi = 0u; scratch->n_forced = 0; scratch->n_emit = 0; }
  __syncthreads();
  {
    // aggregated score of this CTA's blocks; the statistics the selection needs are gathered on the way
    float* scores_u = p.scores + (size_t)u * p.max_blocks;
    uint32_t mn = 0xffffffffu, mx = 0u;
    int nf = 0;
    for (int li = tid; li < nb_my; li += kCsThreads) {
      float sc = 0.f;
#pragma unroll
      for (int g = 0; g < GP; ++g)
        if (g < G) sc += __expf(ell_s[g * chunk + li] - lse_r[g]);
      const int i = blk_begin + li;
      scores_u[i] = sc;
      const bool forced = (i < p.n_sink) || (i >= nblk - p.n_local);
      const uint32_t key = forced ? 0xffffffffu : __float_as_uint(sc);
      keys[li] = key;
      if (forced) {
        ++nf;
        push(atomicAdd(&scratch->n_emit, 1), key, i);
      } else {
        mn = min(mn, key);
        mx = max(mx, key);
      }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    nf = __reduce_add_sync(0xffffffffu, nf);
    if (lane == 0) {
      atomicMin(&scratch->lo, mn);
      atomicMax(&scratch->hi, mx);
      if (nf) atomicAdd(&scratch->n_forced, nf);
    }
  }
  __syncthreads();

  // this CTA's best min(k_eff, n_my) blocks go to the leader's candidate table
  {
    const int cnt = select_topk(keys, nb_my, k_eff, [&](int li) { return blk_begin + li; }, push, scratch);
    if (tid == 0) st_dsmem_u32(map_to_rank(smem_u32(smem_raw + SM::kCandCnt), 0u) + (uint32_t)rank * 4, (uint32_t)cnt);
  }

  cluster_sync_all();                                                   // ---- sync 2: candidates are in the leader
  const bool rla = !(p.flags & 4u);
  if (rank != 0) {
    // The siblings are done with the selection; while the leader finishes it they compute the part of the
    // residual branch that needs no selection, o_bar = phi(q) S_bar, one slice of the state's rows each.
    if (rla)
      for (int s = rank - 1; s < kStateSplits; s += CS - 1) {
        __syncthreads();                       // (the slices of one CTA reuse the same shared memory)
        state_role<D, GP, kCsThreads>(p, u, s, q_raw, q_is_bf16, reinterpret_cast<float*>(smem_raw));
      }
  } else {
  // ------------------------------------------------------------------ phase C (leader) ----------------------
  const uint32_t* cand_key = reinterpret_cast<const uint32_t*>(smem_raw + SM::kCandKey);
  const int* cand_idx = reinterpret_cast<const int*>(smem_raw + SM::kCandIdx);
  const int* cand_cnt = reinterpret_cast<const int*>(smem_raw + SM::kCandCnt);
  uint32_t* flat_key = reinterpret_cast<uint32_t*>(smem_raw + SM::kFlatKey);
  int* flat_idx = reinterpret_cast<int*>(smem_raw + SM::kFlatIdx);
  int* sel_tmp = reinterpret_cast<int*>(smem_raw + SM::kSelTmp);
  // Two lower bounds of the k_eff-th best key, so that most of the table drops out before any ranking.  With n_full
  // CTAs that sent a full list of k_eff candidates: (a) the smallest key of any one full list (that list alone holds
  // k_eff keys from there upwards: good when one part of the sequence dominates); (b) the smallest, over the full
  // lists, of each list's q-th best key, q = ceil(k_eff / n_full) (n_full q >= k_eff keys lie at or above it: good
  // when the lists look alike).  The larger of the two is used.
  uint32_t* list_min = reinterpret_cast<uint32_t*>(scratch->hist);      // [kMaxCluster] bound (a) per list
  uint32_t* list_qth = list_min + kMaxCluster;                          // [kMaxCluster] q-th best per list
  int* n_surv = scratch->hist + 2 * kMaxCluster;                        // survivor counter
  int n_full = 0;
  for (int r = 0; r < CS; ++r) n_full += cand_cnt[r] == k_eff;
  const int quota = n_full > 0 ? (k_eff + n_full - 1) / n_full : 0;
  for (int r = warp; r < CS; r += kCsConsumers) {
    const int cnt = cand_cnt[r];
    const bool is_full = cnt == k_eff;
    uint32_t v0 = lane < cnt ? cand_key[r * kMaxTopK + lane] : (is_full ? 0xffffffffu : 0u);
    uint32_t v1 = lane + 32 < cnt ? cand_key[r * kMaxTopK + lane + 32] : (is_full ? 0xffffffffu : 0u);
    const uint32_t lmin = __reduce_min_sync(0xffffffffu, min(v0, v1));  // (the padding of a full list is neutral here)
    if (lane >= cnt) v0 = 0u;
    if (lane + 32 >= cnt) v1 = 0u;
    uint32_t m = 0xffffffffu;                                           // "no bound from this list" for the minimum below
    if (is_full && quota <= 8) {
      for (int round = 0; round < quota; ++round) {                     // knock the largest out, quota times
        m = __reduce_max_sync(0xffffffffu, max(v0, v1));
        const uint32_t in0 = __ballot_sync(0xffffffffu, v0 == m);
        const uint32_t in1 = __ballot_sync(0xffffffffu, v1 == m);
        if (in0) { if (lane == __ffs(in0) - 1) v0 = 0u; }
        else if (lane == __ffs(in1) - 1) v1 = 0u;
      }
    }
    if (lane == 0) { list_min[r] = is_full ? lmin : 0u; list_qth[r] = m; }
  }
  if (tid == 0) *n_surv = 0;
  __syncthreads();
  uint32_t bound_a = 0u, bound_b = 0xffffffffu;
  for (int r = 0; r < CS; ++r) { bound_a = max(bound_a, list_min[r]); bound_b = min(bound_b, list_qth[r]); }
  if (bound_b == 0xffffffffu) bound_b = 0u;                             // no full list, or too large a quota
  const uint32_t bound = max(bound_a, bound_b);
  for (int c0 = 0; c0 < CS * kMaxTopK; c0 += kCsThreads) {             // the survivors, in no particular order
    const int c = c0 + tid, r = c / kMaxTopK, sl = c % kMaxTopK;
    const bool live = c < CS * kMaxTopK && sl < cand_cnt[r] && cand_key[c] >= bound;
    const uint32_t vote = __ballot_sync(0xffffffffu, live);
    int base = 0;
    if (lane == 0 && vote) base = atomicAdd(n_surv, __popc(vote));
    base = __shfl_sync(0xffffffffu, base, 0);
    if (live) {
      const int dst = base + __popc(vote & ((1u << lane) - 1u));
      flat_key[dst] = cand_key[c];
      flat_idx[dst] = cand_idx[c];
    }
  }
  __syncthreads();
  const int total = *n_surv;
  auto keep = [&](int slot, uint32_t, int idx) { sel_tmp[slot] = idx; };
  auto flat_of = [&](int c) { return flat_idx[c]; };
  if (total <= kCsThreads) {
    // few survivors (the usual case): every thread ranks its candidates against all others by counting, reading the
    // table with broadcast 128-bit loads; no shared-memory atomics, one barrier
    if (tid < 4) { flat_key[total + tid] = 0u; flat_idx[total + tid] = 0x7fffffff; }   // padding that precedes nothing
    __syncthreads();
    for (int c = tid; c < total; c += kCsThreads) {
      const uint32_t a = flat_key[c];
      const int ia = flat_idx[c];
      int rk = 0;
      for (int j = 0; j < total; j += 4) {
        const uint4 kk = *reinterpret_cast<const uint4*>(flat_key + j);
        const int4 ii = *reinterpret_cast<const int4*>(flat_idx + j);
        rk += pair_before(kk.x, ii.x, a, ia) + pair_before(kk.y, ii.y, a, ia) + pair_before(kk.z, ii.z, a, ia) +
              pair_before(kk.w, ii.w, a, ia);
      }
      if (rk < k_eff) sel_tmp[rk] = ia;
    }
    __syncthreads();
  } else {
    topk_prepare(flat_key, total, flat_of, keep, scratch);
    select_topk(flat_key, total, k_eff, flat_of, keep, scratch);
  }

  int* sel_u = p.sel + (size_t)u * p.top_k;
  int* sel_o = sel_user ? sel_user + (size_t)u * p.top_k : nullptr;
  for (int s = tid; s < p.top_k; s += kCsThreads) {
    if (s < k_eff) {
      const int ia = sel_tmp[s];
      int pos = 0;
#pragma unroll 8
      for (int j = 0; j < k_eff; ++j) pos += sel_tmp[j] < ia;
      sel_u[pos] = ia;
      if (sel_o) sel_o[pos] = ia;
      if (sel_share)
        for (int r = 0; r < CS; ++r) st_dsmem_u32(map_to_rank(smem_u32(sel_share + pos), (uint32_t)r), (uint32_t)ia);
    } else {
      sel_u[s] = -1;
      if (sel_o) sel_o[s] = -1;
    }
  }
  if (tid == 0) {
    p.n_sel[u] = k_eff;
    if (sel_share)
      for (int r = 0; r < CS; ++r) {
        st_dsmem_u32(map_to_rank(smem_u32(sel_share + kMaxTopK), (uint32_t)r), (uint32_t)k_eff);
        st_dsmem_u32(map_to_rank(smem_u32(sel_share + kMaxTopK + 1), (uint32_t)r), (uint32_t)L);
      }
  }
  if (rla && CS == 1)
    for (int s = 0; s < kStateSplits; ++s) {
      __syncthreads();
      state_role<D, GP, kCsThreads>(p, u, s, q_raw, q_is_bf16, reinterpret_cast<float*>(smem_raw));
    }
  }   // leader
}

template <int D, int GP, bool WIN, bool EARLY, typename ST, int NWP>
__global__ void __launch_bounds__(NWP * 32, 2) score_cluster_kernel(const Params p, const void* __restrict__ q_raw,
                                                                    int q_is_bf16, int* __restrict__ sel_user,
                                                                    int pending_new) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  score_cluster_body<D, GP, WIN, EARLY, ST, NWP>(p, q_raw, q_is_bf16, sel_user, pending_new, smem_raw);
}

// `occupancy` non-null: nothing is launched; it receives the number of clusters of this launch that the device holds
// at once (-1 if the query fails).
template <int D, int GP, bool WIN, bool EARLY, typename ST, int NWP>
static cudaError_t launch_win(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new, cudaStream_t stream,
                              int* occupancy) {
  using SM = Smem<D, GP, ST, NWP>;
  const int U = p.batch * p.Hkv;
  size_t smem = (size_t)SM::kEll + (size_t)p.G * p.chunk * sizeof(float);
  auto kern = score_cluster_kernel<D, GP, WIN, EARLY, ST, NWP>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  if (p.cs > 8) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
  }
  if (occupancy) {
    *occupancy = max_active_clusters(kern, dim3(p.cs, U, 1), dim3(NWP * 32, 1, 1), smem, p.cs);
    return cudaSuccess;
  }
  return launch_ex(kern, dim3(p.cs, U, 1), dim3(NWP * 32, 1, 1), smem, stream, p.cs, true, p, q, q_is_bf16, sel_user, pending_new);
}

template <int D, int GP, typename ST, int NWP>
static cudaError_t launch_st(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new, cudaStream_t stream,
                             int* occ) {
  if (pending_new > 0)
    return p.NW > 1 ? launch_win<D, GP, true, true, ST, NWP>(p, q, q_is_bf16, sel_user, pending_new, stream, occ)
                    : launch_win<D, GP, false, true, ST, NWP>(p, q, q_is_bf16, sel_user, pending_new, stream, occ);
  return p.NW > 1 ? launch_win<D, GP, true, false, ST, NWP>(p, q, q_is_bf16, sel_user, 0, stream, occ)
                  : launch_win<D, GP, false, false, ST, NWP>(p, q, q_is_bf16, sel_user, 0, stream, occ);
}

template <int D, int GP, int NWP>
static cudaError_t launch_one(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new, cudaStream_t stream,
                              int* occ) {
  return (p.flags & kStatsBf16) ? launch_st<D, GP, __nv_bfloat16, NWP>(p, q, q_is_bf16, sel_user, pending_new, stream, occ)
                                : launch_st<D, GP, float, NWP>(p, q, q_is_bf16, sel_user, pending_new, stream, occ);
}

template <int D, int NWP>
static cudaError_t launch_d(const Params& p, int GP, const void* q, int qb, int* sel_user, int pending_new, cudaStream_t s,
                            int* occ) {
  switch (GP) {
    case 1: return launch_one<D, 1, NWP>(p, q, qb, sel_user, pending_new, s, occ);
    case 2: return launch_one<D, 2, NWP>(p, q, qb, sel_user, pending_new, s, occ);
    case 4: return launch_one<D, 4, NWP>(p, q, qb, sel_user, pending_new, s, occ);
    default: return launch_one<D, 8, NWP>(p, q, qb, sel_user, pending_new, s, occ);
  }
}

// The entry of one build size: launches, or (occ non-null) only asks how many clusters are resident at once.
template <int NWP>
static cudaError_t launch_size(const Params& p, const void* q, int q_is_bf16, int* sel_user, int pending_new, cudaStream_t stream,
                               int* occ) {
  const int GP = padded_group(p.G);
  return p.d == 128 ? launch_d<128, NWP>(p, GP, q, q_is_bf16, sel_user, pending_new, stream, occ)
                    : launch_d<64, NWP>(p, GP, q, q_is_bf16, sel_user, pending_new, stream, occ);
}

}  // namespace spla
