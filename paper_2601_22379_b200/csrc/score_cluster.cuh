// Block score + selection, cluster edition: the CTAs that score one (sequence, KV head) unit form a thread-block
// cluster, so the selection no longer runs as a serial tail in one CTA behind a global-memory hand-off.
//
//   phase A     every CTA streams its share of the unit's statistics records through a ring of shared-memory
//               stages filled by bulk asynchronous copies (full/empty mbarriers; one thread feeds the ring) and keeps
//               the Taylor log masses ell^m_i (Section 3.1 of the paper, Eq. taylor-2nd, diagonal covariance) in shared
//               memory;
//   exchange 1  its per-head (max, sum exp) goes into every CTA of the cluster as asynchronous stores (st.async) that
//               count their bytes on a barrier of the receiver; a CTA goes on when all partials have reached it;
//   phase B     warps 0-3 form the normalisers and the aggregated BlockScore of the CTA's own blocks (Section 2.2:
//               per-head softmax over blocks, summed over the group); warps 4-7 compute o_bar = phi(q) S_bar, the
//               part of the residual branch that needs no selection, from here on;
//   exchange 2  each score goes, as an integer key, into the key table of every CTA that selects (all of them in the
//               fused decode kernel, the first otherwise), again as counted asynchronous stores;
//   phase C     warps 0-3 of a selecting CTA pick the top k on their own (Section 2.1 Select; the forced sink / local
//               blocks of Section 4 "Sparsity Specifications" are known from their indices).  No leader, no hand-off:
//               the selection of a unit is computed in as many copies as CTAs use it, which costs less than sending it.
// Ordering everywhere is (score descending, block index ascending).  No barrier of the whole cluster lies on the path:
// one is announced at the start and completed before the first exchange (everybody's barriers exist), and the kernel
// of its own closes with one.  All waits are bounded mbarrier polls or CTA barriers.  No multicast is used.
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
  // tensor-core streaming (16-bit records; fp32 records for groups of more than four heads, where the FMA pipe cannot
  // keep up): the ring is cut into slots of 16 records, one MMA row tile each
  static constexpr bool kMma = sizeof(ST) == 2 || GP > 4;
  static constexpr int kSlotBytes = kSlotRec * kRecBytes;
  static constexpr int kSlots = sizeof(ST) == 2 ? NWP : 6;         // one ring position per streaming warp (6 x 16 KB with fp32 records)
  static constexpr int kStreamBytes = kMma ? kSlots * kSlotBytes : kStages * kStageBytes;
  // after streaming the ring is dead and holds the selection's work arrays:
  static constexpr int kKeys = 0;                                   // uint32 [16 x 1024]   the keys of the whole unit, by block index
  static constexpr int kFlatCap = 512;                              // survivors that are ranked by counting
  static constexpr int kFlat = kKeys + kMaxCluster * 1024 * 4;      // uint64 [kFlatCap + 4]  (key, complement of the index)
  static constexpr int kLaneMax = kFlat + (kFlatCap + 4) * 8;       // uint32 [128]         best key of every pair of selecting threads (64 used)
  static constexpr int kSelTmp = kLaneMax + 128 * 4;                // int [64]             the picks, best first (where the caller gives no array)
  static constexpr int kSelOut = kSelTmp + kMaxTopK * 4;            // int [64 + 2]         work array of the histogram selection
  static constexpr int kScratch = (kSelOut + (kMaxTopK + 2) * 4 + 15) / 16 * 16;   // TopkScratch
  static constexpr int kWorkEnd = (kScratch + (int)sizeof(TopkScratch) + 1023) / 1024 * 1024;
  // ... followed by the scratch of the o_bar role, which runs beside the selection
  static constexpr int kStateScratch = kWorkEnd;                    // float [GP * D + (128 / D) * GP * D]
  static constexpr int kStateBytes0 = (GP * D + (128 / D > 0 ? 128 / D : 1) * GP * D) * 4;
  static constexpr int kStateBytes = kStateBytes0 > 2048 + 8 * D * 4 ? kStateBytes0 : 2048 + 8 * D * 4;   // (fused kernel: 2 KB of working space, then o_bar of up to 8 heads)
  static constexpr int kAreaEnd = (kStateScratch + kStateBytes + 1023) / 1024 * 1024;
  // The ring area is padded to hold all of that.  The fused decode kernel relies on it too: its attend phase lays the
  // K/V tile ring (at most 66 KB) over this area, and the tile copies must stay clear of the fixed region below, which
  // holds this phase's mbarrier objects (never invalidated: overwriting them with tile data corrupted value rows, found
  // with NaN-filled memory), and of the o_bar scratch, which may still be in use when the first tiles arrive.
  static constexpr int kMergeRecv = kAreaEnd;                       // the attend phase's receive area (fused kernel)
  static constexpr int kMergeRecvBytes = (16 * (2 * D + 2) * 4 + 1023) / 1024 * 1024;
  static constexpr int kRingBytes = kStreamBytes > kMergeRecv + kMergeRecvBytes ? kStreamBytes : kMergeRecv + kMergeRecvBytes;
  static_assert(kStateScratch >= 68 * 1024, "the attend phase's tile ring must end below the o_bar scratch");
  // fixed region after the ring:
  static constexpr int kAllPart = kRingBytes;                       // float [16][GP][2]  every CTA's (max, sum exp) per head
  static constexpr int kWred = kAllPart + kMaxCluster * GP * 2 * 4; // float [NWP][GP][2] the warps' partials
  static constexpr int kBars = (kWred + NWP * GP * 2 * 4 + 7) / 8 * 8;            // uint64: full / empty per stage, or one per slot
  static constexpr int kRingBars = kMma ? kSlots : 2 * kStages;
  static constexpr int kNumBars = kRingBars + 2;                    // ... and one each for the two exchanges of the cluster
  // (tensor-core path with two column tiles: the B fragments of the variance dots, one word per lane and (tile, chunk,
  // word), kept here instead of in 32 more registers per thread)
  static constexpr int kBfrag = (kBars + kNumBars * 8 + 15) / 16 * 16;
  static constexpr int kBfragBytes = (sizeof(ST) == 2 && GP > 4) ? 2 * (D * 2 / 64) * 4 * 32 * 4 : 0;
  static constexpr int kEll = kBfrag + kBfragBytes;                                // float [G][chunk]
};

}  // namespace

// WIN: strided selection windows (several statistics records per block, max-pooled); without them the kernel is
// compiled with one record per block as a constant.
// EARLY: the kernel follows the append of the same step in the stream and does not wait for it before streaming:
// the blocks that were complete before that append (at most `pending_new` tokens per sequence) cannot change any
// more, so their statistics are streamed while the append still runs; only then does the kernel wait for the
// append, read the final length and take the few remaining blocks (those the append wrote to) from global memory.
// ST: element type of the statistics records (float, or __nv_bfloat16 with half the bytes to stream).
// On return the selection of the unit is in p.sel / p.n_sel (and sel_user), written by the cluster's first CTA, and the
// o_bar partials are in p.obar_part or on their way there (warps 4-7 return on their own, without a barrier with the
// selecting warps 0-3); every thread of every CTA of the cluster returns (nobody has left the kernel).
// The picks of a unit, held best first in shared memory (`picks`, padded to a multiple of four with entries that precede
// nothing), go to the workspace and the caller's array in ascending order.  Run by warps 4-7 of the unit's first CTA
// (`t` = 0 .. 127), which first wait for warps 0-3 to announce the list on named barrier 3.  k_eff < 0: the count
// follows the list, at picks[kMaxTopK].
__device__ __forceinline__ void write_selection(const Params& p, int u, const int* picks, int k_eff, int* __restrict__ sel_user,
                                                int t) {
  asm volatile("bar.sync 3, 256;" ::: "memory");
  if (k_eff < 0) k_eff = picks[kMaxTopK];
  int* sel_u = p.sel + (size_t)u * p.top_k;
  int* sel_o = sel_user ? sel_user + (size_t)u * p.top_k : nullptr;
  for (int s = t; s < p.top_k; s += 128) {
    int pos = s, ia = -1;
    if (s < k_eff) {
      ia = picks[s];
      pos = 0;
      for (int j = 0; j < k_eff; j += 4) {
        const int4 ii = *reinterpret_cast<const int4*>(picks + j);
        pos += (ii.x < ia) + (ii.y < ia) + (ii.z < ia) + (ii.w < ia);
      }
    }
    sel_u[pos] = ia;
    if (sel_o) sel_o[pos] = ia;
  }
  if (t == 0) p.n_sel[u] = k_eff;
}

template <int D, int GP, bool WIN, bool EARLY, typename ST, int NWP>
// `sel_share` (fused kernel only, else null): a shared-memory array of kMaxTopK + 2 ints; warps 0-3 of every CTA leave
// the selection there, best block first, followed by the count and the length, and have met on a barrier since.
// `obar_local` (fused kernel only, else null): shared memory for o_bar of the heads this CTA merges, [heads][D].
__device__ __forceinline__ void score_cluster_body(const Params& p, const void* __restrict__ q_raw, int q_is_bf16,
                                                   int* __restrict__ sel_user, int pending_new, unsigned char* smem_raw,
                                                   int* sel_share = nullptr, float* obar_local = nullptr) {
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

  float* all_part = reinterpret_cast<float*>(smem_raw + SM::kAllPart);
  float* wred = reinterpret_cast<float*>(smem_raw + SM::kWred);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + SM::kBars);
  uint64_t* empty = full + kStages;
  uint64_t* pbar = full + SM::kRingBars;        // completes when every CTA's partial normalisers have arrived here
  uint64_t* kbar = pbar + 1;                    // completes when every CTA's keys have arrived here
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
    mbar_init(pbar, 1);
    mbar_init(kbar, 1);
    mbar_init_done();
    err_s = 0;
  }
  cluster_arrive();                             // the siblings may store here once everybody's barriers exist: completed before the first exchange
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
  // Tensor-core streaming (16-bit records): a slot of 16 records is the A operand of mma.m16n8k16 (16 x d, row-major,
  // as stored), the B operand's eight columns are four heads' scaled queries, each split in two bf16 parts, bf16(q) and
  // bf16(q - bf16(q)) (column n: head n / 2, part n % 2; a second column tile serves heads 4..7), whose products are
  // added after the MMA: the query enters with 16 significant bits, the statistics exactly, the sums are fp32.
  // Thread (g8, t4) owns 16 consecutive bytes of every 64 of a record half (mean or variance), which it fetches with
  // one 128-bit load per row; the k index inside an MMA is a permutation of the channels, the same for A and B.
  constexpr bool MMA = SM::kMma;
  // With fp32 records each element is split the same way, bf16(x) + bf16(x - bf16(x)) (16 significant bits, the
  // rounding of the second part 2^-17 relative), and each part gets its own MMA against the same columns.
  constexpr bool MMAF = MMA && sizeof(ST) == 4;
  constexpr int NJ = D * (int)sizeof(ST) / 64;   // 16-byte chunks per thread and record half
  constexpr int CPC = 16 / (int)sizeof(ST);      // channels per chunk: 8 (two MMA k-steps) or 4 (one)
  constexpr int BW = MMAF ? 2 : 4;               // B-fragment words per chunk
  const int g8 = lane >> 2, t4 = lane & 3;
  constexpr int NT2 = GP > 4 ? 2 : 1;            // column tiles of eight: four heads x two query parts each
  // 16-bit records with two column tiles: the variance fragments live in shared memory (the same for every warp).
  // (With fp32 records they stay in registers although that costs the GP = 8 builds a few spilled words: fetching them
  // per MMA made the already latency-bound slot loop 2 us slower per decode.)
  constexpr bool BVS = MMA && NT2 == 2 && !MMAF;
  uint32_t bq[MMA ? NT2 : 1][MMA ? NJ : 1][BW], bv[(MMA && !BVS) ? NT2 : 1][(MMA && !BVS) ? NJ : 1][BW];
  uint32_t* bv_s = reinterpret_cast<uint32_t*>(smem_raw + SM::kBfrag);   // [NT2][NJ][BW][32 lanes]
  float qm[GP][VECW], qv[GP][VECW];
  if constexpr (MMA) {
#pragma unroll
    for (int nt = 0; nt < NT2; ++nt) {
      const int head = nt * 4 + (g8 >> 1), part = g8 & 1;
#pragma unroll
      for (int j = 0; j < NJ; ++j) {
        float x[CPC];                              // channels j * 4 * CPC + t4 * CPC .. + CPC - 1
        if (head < G) {
          const size_t qoff = ((size_t)b * p.Hq + (size_t)h * G + head) * D + (size_t)j * 4 * CPC + t4 * CPC;
#pragma unroll
          for (int c = 0; c < CPC / 4; ++c) {
            float y[4];
            if (q_is_bf16) load_vec<4>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff + c * 4, y);
            else load_vec<4>(reinterpret_cast<const float*>(q_raw) + qoff + c * 4, y);
#pragma unroll
            for (int v = 0; v < 4; ++v) x[c * 4 + v] = y[v];
          }
        } else {
#pragma unroll
          for (int v = 0; v < CPC; ++v) x[v] = 0.f;
        }
        float qa[CPC], qb2[CPC];                   // this thread's part of q_hat and of q_hat^2 / 2
#pragma unroll
        for (int v = 0; v < CPC; ++v) {
          const float qh = x[v] * p.sm_scale;
          const float qq = (p.flags & 2u) ? 0.f : 0.5f * qh * qh;
          const float h1 = __bfloat162float(__float2bfloat16_rn(qh)), h2 = __bfloat162float(__float2bfloat16_rn(qq));
          qa[v] = part ? qh - h1 : h1;
          qb2[v] = part ? qq - h2 : h2;
        }
#pragma unroll
        for (int v = 0; v < BW; ++v) {
          bq[nt][j][v] = pack_bf16(qa[2 * v], qa[2 * v + 1]);
          if constexpr (BVS) { if (warp == 0) bv_s[((nt * NJ + j) * BW + v) * 32 + lane] = pack_bf16(qb2[2 * v], qb2[2 * v + 1]); }
          else bv[nt][j][v] = pack_bf16(qb2[2 * v], qb2[2 * v + 1]);
        }
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
    float run_max2 = -INFINITY, run_sum2 = 0.f;  // (tensor-core path, groups of more than four heads: head 4 + t4)

    // Tensor-core path: one slot of 16 records -> dots of heads t4 (and 4 + t4) with records g8 and g8 + 8 of the
    // slot -> log masses.  `li0` is the CTA-local index of the slot's first record, `limit` the number of local records
    // that exist for this call.  Rows past the limit hold stale bytes; every row is independent and theirs are dropped.
    auto consume_slot = [&](const unsigned char* slot, int li0, int limit) {
      float cm[NT2][4], cv[NT2][4];
#pragma unroll
      for (int nt = 0; nt < NT2; ++nt) { cm[nt][0] = cm[nt][1] = cm[nt][2] = cm[nt][3] = 0.f; cv[nt][0] = cv[nt][1] = cv[nt][2] = cv[nt][3] = 0.f; }
      const unsigned char* r0 = slot + (size_t)g8 * SM::kRecBytes + t4 * 16;
      const unsigned char* r1 = r0 + 8 * SM::kRecBytes;
      constexpr int HALF = SM::kRecBytes / 2;                      // the variance follows the mean
      if constexpr (MMA && !MMAF) {
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          const uint4 m0 = *reinterpret_cast<const uint4*>(r0 + j * 64), m1 = *reinterpret_cast<const uint4*>(r1 + j * 64);
          const uint4 v0 = *reinterpret_cast<const uint4*>(r0 + HALF + j * 64), v1 = *reinterpret_cast<const uint4*>(r1 + HALF + j * 64);
#pragma unroll
          for (int nt = 0; nt < NT2; ++nt) {
            mma_bf16(cm[nt], m0.x, m1.x, m0.y, m1.y, bq[nt][j][0], bq[nt][j][1]);
            uint32_t w0, w1, w2, w3;
            if constexpr (BVS) {
              const uint32_t* t = bv_s + ((nt * NJ + j) * BW) * 32 + lane;
              w0 = t[0]; w1 = t[32]; w2 = t[64]; w3 = t[96];
            } else {
              w0 = bv[nt][j][0]; w1 = bv[nt][j][1]; w2 = bv[nt][j][2]; w3 = bv[nt][j][3];
            }
            mma_bf16(cv[nt], v0.x, v1.x, v0.y, v1.y, w0, w1);
            mma_bf16(cm[nt], m0.z, m1.z, m0.w, m1.w, bq[nt][j][2], bq[nt][j][3]);
            mma_bf16(cv[nt], v0.z, v1.z, v0.w, v1.w, w2, w3);
          }
        }
      }
      if constexpr (MMAF) {
        // fp32 records: this thread's four channels of the chunk, rows g8 and g8 + 8, are the A fragment of one k-step
        // (k indices 2 t4, 2 t4 + 1, 2 t4 + 8, 2 t4 + 9); first the mean, then the variance, each as two bf16 parts
        auto split_mma = [&](const unsigned char* a_lo, const unsigned char* a_hi, float (&acc)[NT2][4], const bool var, int j) {
          const float4 x0 = *reinterpret_cast<const float4*>(a_lo + j * 64), x1 = *reinterpret_cast<const float4*>(a_hi + j * 64);
          const uint32_t h0 = pack_bf16(x0.x, x0.y), h1 = pack_bf16(x1.x, x1.y), h2 = pack_bf16(x0.z, x0.w), h3 = pack_bf16(x1.z, x1.w);
          const uint32_t l0 = pack_bf16(x0.x - bf16_lo(h0), x0.y - bf16_hi(h0)), l1 = pack_bf16(x1.x - bf16_lo(h1), x1.y - bf16_hi(h1));
          const uint32_t l2 = pack_bf16(x0.z - bf16_lo(h2), x0.w - bf16_hi(h2)), l3 = pack_bf16(x1.z - bf16_lo(h3), x1.w - bf16_hi(h3));
#pragma unroll
          for (int nt = 0; nt < NT2; ++nt) {
            uint32_t w0, w1;
            if (!var) { w0 = bq[nt][j][0]; w1 = bq[nt][j][1]; }
            else if constexpr (BVS) { const uint32_t* t = bv_s + ((nt * NJ + j) * BW) * 32 + lane; w0 = t[0]; w1 = t[32]; }
            else { w0 = bv[nt][j][0]; w1 = bv[nt][j][1]; }
            mma_bf16(acc[nt], h0, h1, h2, h3, w0, w1);
            mma_bf16(acc[nt], l0, l1, l2, l3, w0, w1);
          }
        };
#pragma unroll
        for (int j = 0; j < NJ; ++j) {
          split_mma(r0, r1, cm, false, j);
          split_mma(r0 + HALF, r1 + HALF, cv, true, j);
        }
      }
      // columns 2 t4 and 2 t4 + 1 of column tile nt are the two query parts of head 4 nt + t4
#pragma unroll
      for (int nt = 0; nt < NT2; ++nt) {
        const int hd = nt * 4 + t4;
        float& rmax = nt == 0 ? run_max : run_max2;
        float& rsum = nt == 0 ? run_sum : run_sum2;
#pragma unroll
        for (int hf = 0; hf < 2; ++hf) {
          const float dm = cm[nt][2 * hf] + cm[nt][2 * hf + 1], dv = cv[nt][2 * hf] + cv[nt][2 * hf + 1];
          const int li = li0 + g8 + 8 * hf;
          if (hd < G && li < limit) {
            if (!WIN) {
              const float ell = (rec_begin + li == nblk_fin - 1 ? ln_last : ln_full) + dm + __logf(1.f + dv);
              ell_s[hd * chunk + li] = ell;
              const float nm = fmaxf(rmax, ell);
              rsum = rsum * __expf(rmax - nm) + __expf(ell - nm);
              rmax = nm;
            } else {
              // strided windows (Section 3.1, "Strided Block Selection"): log mass of window w of a block,
              // max-pooled into the block's slot right away through an order-preserving integer key
              const int lb = (int)__umulhi((unsigned)li, nw_magic), w = li - lb * NW;   // li / NW without a division
              float ln_n = ln_win;
              if (cta_blk0 + lb == nblk_fin - 1) {
                const int cnt = min(p.win_C, n_last - w * p.win_s);
                ln_n = cnt > 0 ? logf((float)cnt) : -INFINITY;
              }
              atomicMax(reinterpret_cast<uint32_t*>(ell_s) + hd * chunk + lb, float_order_key(ln_n + dm + __logf(1.f + dv)));
            }
          }
        }
      }
    };
    if constexpr (MMA) {
#pragma unroll 1
      for (int r = warp; warp < SM::kSlots && r < n_slots; r += SM::kSlots) {   // warp w < kSlots owns ring position w
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
      // lanes with the same t4 hold partial normalisers of head t4 (and 4 + t4): fold over g8
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, run_max, o), s2 = __shfl_xor_sync(0xffffffffu, run_sum, o);
        lse_merge(run_max, run_sum, m2, s2);
        if constexpr (NT2 == 2) {
          const float m3 = __shfl_xor_sync(0xffffffffu, run_max2, o), s3 = __shfl_xor_sync(0xffffffffu, run_sum2, o);
          lse_merge(run_max2, run_sum2, m3, s3);
        }
      }
      if (!WIN && lane < 4) {
        if (lane < G) {
          wred[(warp * GP + lane) * 2 + 0] = run_max;
          wred[(warp * GP + lane) * 2 + 1] = run_sum;
        }
        if (NT2 == 2 && 4 + lane < G) {
          wred[(warp * GP + 4 + lane) * 2 + 0] = run_max2;
          wred[(warp * GP + 4 + lane) * 2 + 1] = run_sum2;
        }
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
  // (fused decode kernel: TMA tiles will overwrite the ring area; what all eight warps did there is ordered before
  // those copies here, the barrier passes the order on)
  if (sel_share) asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncthreads();
  cluster_wait();                               // every CTA of the cluster has its barriers in place (announced at the top)

  // ---- exchange 1: this CTA's (max, sum exp) of every head goes into every CTA of the cluster, as asynchronous
  // stores that count their bytes on the receiver's barrier: a CTA goes on as soon as all partials have reached it,
  // without a barrier of the whole cluster.  (All partials here also means: every CTA is done with its ring.)
  const bool key_dest = sel_share || rank == 0;   // a kernel of its own: only the first CTA selects
  if (warp == 0) {
    // lane w * GP + g takes the pair of warp w and head g; the warps of a head are folded with shuffles (32 / GP >= 8
    // warps fit a pass for groups of up to four heads, else two passes); lanes 0 .. G - 1 then send head `lane`
    float m = -INFINITY, s = 0.f;
    for (int e = lane; e < kCsConsumers * GP; e += 32) lse_merge(m, s, wred[e * 2], wred[e * 2 + 1]);
#pragma unroll
    for (int o = GP; o < 32; o <<= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, m, o), s2 = __shfl_xor_sync(0xffffffffu, s, o);
      lse_merge(m, s, m2, s2);
    }
    if (lane < G) {
      const uint32_t mine = smem_u32(all_part + ((size_t)rank * GP + lane) * 2), bar = smem_u32(pbar);
      for (int r = 0; r < CS; ++r)
        st_async_v2(map_to_rank(mine, (uint32_t)r), __float_as_uint(m), __float_as_uint(s), map_to_rank(bar, (uint32_t)r));
    }
  }
  const int nblk_pad = min(nblk, CS * chunk);
  if (tid == 32) {
    mbar_expect_tx(pbar, (uint32_t)(CS * G * 8));
    if (key_dest) {                               // the keys arrive two at a time: every CTA sends ceil(its blocks / 2) pairs
      uint32_t bytes = 0;
      for (int r = 0; r < CS; ++r) bytes += (uint32_t)((max(0, min(nblk_pad, (r + 1) * chunk) - min(nblk_pad, r * chunk)) + 1) / 2) * 8u;
      mbar_expect_tx(kbar, bytes);
    }
  }
  if (tid == 0 && err_s) atomicExch(p.status, kStatusTimeout);
  const bool rla = !(p.flags & 4u);
  const int n = nblk;
  const int k_eff = min(p.top_k, n);
  int* sel_tmp = sel_share ? sel_share : reinterpret_cast<int*>(smem_raw + SM::kSelTmp);   // the picks, best first

  if (warp >= 4) {
    // Warps 4-7: o_bar = phi(q) S_bar (one slice of the state's rows per CTA) beside the scoring and the selection;
    // then, in the first CTA, the selection in ascending order for the workspace and the caller.
    if (!sel_share) cluster_arrive();             // (closing barrier of the kernel of its own, see below: these warps send nothing)
    if (rla && obar_local) {
      // fused decode kernel: this CTA will merge heads rank, rank + CS, ... and computes their o_bar in full, into its
      // own shared memory
      for (int hd = rank, i = 0; hd < G; hd += CS, ++i)
        state_head<D, 128>(p, u, hd, q_raw, q_is_bf16, obar_local + (size_t)i * D,
                           reinterpret_cast<float*>(smem_raw + SM::kStateScratch), tid - 128, 2);
    } else if (rla) {
      for (int s = rank; s < kStateSplits; s += CS) {
        if (s != rank) asm volatile("bar.sync 2, 128;" ::: "memory");   // (the slices of one CTA reuse the same scratch)
        state_role<D, GP, 128>(p, u, s, q_raw, q_is_bf16, reinterpret_cast<float*>(smem_raw + SM::kStateScratch), tid - 128, 2);
      }
    }
    if (obar_local) asm volatile("bar.arrive 2, 256;" ::: "memory");   // o_bar of this CTA's heads is in place (warps 0-3 wait there before the merge)
    // (the fused decode kernel calls this itself, once these warps have given their registers to the others)
    if (rank == 0 && !sel_share) write_selection(p, u, sel_tmp, k_eff, sel_user, tid - 128);
    if (!sel_share) cluster_wait();
    return;
  }

  // ------------------------------------------------------------------ phase B (warps 0-3) -------------------
  const TopkGroup selg{tid, 128, 1};
  if (!mbar_wait(pbar, 0, p.wait_limit) && lane == 0) atomicExch(p.status, kStatusTimeout);
  // Log-sum-exp of every head over the whole cluster, by each warp on its own (no block barrier): lane p takes the
  // (max, sum) pair of CTA p / GP and head p % GP, then the lanes of one head are folded with shuffles.
  float lse_r[GP];
  {
    float m = -INFINITY, sm = 0.f;
    for (int pr = lane; pr < CS * GP; pr += 32) {
      const int g = pr % GP;
      if (g < G) lse_merge(m, sm, all_part[pr * 2], all_part[pr * 2 + 1]);
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

  // ---- exchange 2: the aggregated score of this CTA's blocks goes to global memory (spla_copy_scores) and, as an
  // integer key, into the key table of every selecting CTA (two blocks per thread and store; the share of a CTA is a
  // multiple of 8 blocks; entries past the sequence's last block are never read)
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw + SM::kKeys);
  {
    float* scores_u = p.scores + (size_t)u * p.max_blocks;
    const uint32_t keys0 = smem_u32(keys), bar = smem_u32(kbar);
    const int n_dest = sel_share ? CS : 1;
    for (int li = tid * 2; li < nb_my; li += 128 * 2) {
      float sc0 = 0.f, sc1 = 0.f;
#pragma unroll
      for (int g = 0; g < GP; ++g)
        if (g < G) {
          const float2 e = *reinterpret_cast<const float2*>(ell_s + g * chunk + li);
          sc0 += __expf(e.x - lse_r[g]);
          sc1 += __expf(e.y - lse_r[g]);
        }
      const int i = blk_begin + li;
      scores_u[i] = sc0;
      if (li + 1 < nb_my) scores_u[i + 1] = sc1; else sc1 = 0.f;
      for (int r = 0; r < n_dest; ++r)
        st_async_v2(map_to_rank(keys0 + (uint32_t)i * 4u, (uint32_t)r), __float_as_uint(sc0), __float_as_uint(sc1),
                    map_to_rank(bar, (uint32_t)r));
    }
  }
  // As a kernel of its own the cluster closes with a barrier that every thread announces once it has sent its last
  // store and completes before it leaves: no CTA is gone while a sibling may still store into it, even after a wait
  // that gave up.  (In the fused decode kernel the barriers of the attend phase do that.)
  if (!sel_share) cluster_arrive();
  if (!key_dest) {
    cluster_wait();
    return;
  }

  // the selection's fixed parts need no key: the forced blocks behind the `need` ranked ones, padding that precedes
  // nothing behind them, an empty survivor table
  unsigned long long* flat = reinterpret_cast<unsigned long long*>(smem_raw + SM::kFlat);
  const int n_forced = (p.n_sink + p.n_local >= n) ? n : p.n_sink + p.n_local;
  const int need = k_eff - n_forced;
  const int n_sink = p.n_sink, local0 = n - p.n_local;             // free blocks: n_sink <= i < local0
  for (int s = tid; s < kMaxTopK; s += 128) {
    int v = 0x7fffffff;
    if (k_eff == n) { if (s < k_eff) v = s; }                      // everything is selected
    else if (s >= max(need, 0) && s < k_eff) { const int f = s - max(need, 0); v = f < n_sink ? f : local0 + (f - n_sink); }
    sel_tmp[s] = v;
  }
  for (int s = tid; s < SM::kFlatCap + 4; s += 128) flat[s] = 0ull;
  if (tid == 0) {
    reinterpret_cast<TopkScratch*>(smem_raw + SM::kScratch)->n_small = 0;   // (the survivor count)
    if (sel_share) { sel_share[kMaxTopK] = k_eff; sel_share[kMaxTopK + 1] = L; }
  }

  if (!mbar_wait(kbar, 0, p.wait_limit) && lane == 0) atomicExch(p.status, kStatusTimeout);   // ---- all keys are here

  // ------------------------------------------------------------------ phase C (warps 0-3) -------------------
  // Top k_eff of the unit's n blocks.  The forced blocks (the first n_sink, the last n_local) are known from their
  // indices; `need` free blocks remain to be picked.  The need-th best of 64 sampled maxima is a lower bound of the
  // need-th best key overall (they belong to different blocks), and little more than `need` keys reach it.  The survivors
  // are ranked by counting, as 64-bit words (key, complement of the index) that one comparison orders; the picks stay
  // in that order (best first, then the forced blocks): every CTA computes the same list, and the attention does not
  // care.  Where too many survive (equal scores) or the sequence has more than 128 x 64 blocks, the histogram selection
  // runs over the whole table instead and its picks are put in ascending order.
  if (k_eff < n && need > 0) {
    TopkScratch* scratch = reinterpret_cast<TopkScratch*>(smem_raw + SM::kScratch);
    int* n_surv = &scratch->n_small;
    uint32_t* bound_s = &scratch->lo;
    const int n_free = local0 - n_sink;
    const int nr = (n_free + 127) / 128;                              // free blocks per thread
    const uint32_t* my_keys = keys + n_sink + tid;
    const int my_n = n_free > tid ? (n_free - tid + 127) / 128 : 0;   // ... of this thread
    int total = SM::kFlatCap + 1;
    if (nr <= 64) {
      // Thread t looks at the free blocks t, t + 128, ... (spread over the whole sequence, whatever its structure);
      // every pair of threads notes the best key it sees, made unique and comparable in one go: the low six bits give
      // way to the pair's number (rounding the key down keeps the bound a lower bound).
      uint32_t* pair_max = reinterpret_cast<uint32_t*>(smem_raw + SM::kLaneMax);
      uint32_t mx = 0u;
#pragma unroll 8
      for (int r = 0; r < my_n; ++r) mx = max(mx, my_keys[128 * r]);
      mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      const int pr = tid >> 1, half = tid & 1;
      const uint32_t mine = (mx & ~63u) | (uint32_t)(63 - pr);
      if (!half) pair_max[pr] = mine;
      selg.sync();                                // (also: the survivor count was cleared before the keys came)
      {
        int rk = 0;                               // rank of this pair's best key among the 64, half of them per thread
#pragma unroll
        for (int j = 0; j < 32; j += 4) {
          const uint4 kk = *reinterpret_cast<const uint4*>(pair_max + half * 32 + j);
          rk += (kk.x > mine) + (kk.y > mine) + (kk.z > mine) + (kk.w > mine);
        }
        rk += __shfl_xor_sync(0xffffffffu, rk, 1);
        if (!half && rk == need - 1) *bound_s = mine & ~63u;
      }
      selg.sync();
      const uint32_t bound = *bound_s;
      {
        // the survivors, in no particular order: mark, count, reserve a range per warp, write
        unsigned long long mask = 0ull;
#pragma unroll 8
        for (int r = 0; r < my_n; ++r) mask |= (unsigned long long)(my_keys[128 * r] >= bound) << r;
        const int cnt = __popcll(mask);
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += t;
        }
        int base = 0;
        if (lane == 31) base = atomicAdd(n_surv, incl);
        int dst = __shfl_sync(0xffffffffu, base, 31) + incl - cnt;
        while (mask) {
          const int r = __ffsll((long long)mask) - 1;
          mask &= mask - 1ull;
          if (dst < SM::kFlatCap)
            flat[dst] = ((unsigned long long)my_keys[128 * r] << 32) | (uint32_t)(0x7fffffff - (n_sink + tid + 128 * r));
          ++dst;
        }
      }
      selg.sync();
      total = *n_surv;
    }
    if (total <= SM::kFlatCap) {
      // P = 4, 2 or 1 neighbouring lanes share a candidate and a part of the table each (broadcast 128-bit loads; the
      // empty entries behind the survivors precede nothing)
      const int lg = total <= 32 ? 2 : total <= 64 ? 1 : 0, P = 1 << lg;
      const int span = (((total + P - 1) >> lg) + 1) & ~1;            // entries per part, even
      for (int c0 = 0; c0 < total; c0 += 128 >> lg) {
        const int c = c0 + (tid >> lg), part = tid & (P - 1);
        const unsigned long long a = c < total ? flat[c] : ~0ull;
        int rk = 0;
#pragma unroll 4
        for (int j = part * span; j < (part + 1) * span; j += 2) {
          const ulonglong2 kk = *reinterpret_cast<const ulonglong2*>(flat + j);
          rk += (kk.x > a) + (kk.y > a);
        }
        if (lg >= 1) rk += __shfl_xor_sync(0xffffffffu, rk, 1);
        if (lg >= 2) rk += __shfl_xor_sync(0xffffffffu, rk, 2);
        if (part == 0 && c < total && rk < need) sel_tmp[rk] = 0x7fffffff - (int)(uint32_t)a;
      }
    } else {
      // forced blocks get the maximal key and the histogram selection picks all k_eff, in no reproducible order:
      // they are put in ascending order, so that every CTA of the cluster holds the same list
      for (int i = tid; i < n_forced; i += 128) keys[i < n_sink ? i : local0 + (i - n_sink)] = 0xffffffffu;
      int* pick = reinterpret_cast<int*>(smem_raw + SM::kSelOut);
      selg.sync();
      auto keep = [&](int slot, uint32_t, int idx) { pick[slot] = idx; };
      auto same = [&](int i) { return i; };
      topk_prepare(keys, n, same, keep, scratch, selg);
      select_topk(keys, n, k_eff, same, keep, scratch, selg);
      for (int s = tid; s < k_eff; s += 128) {
        const int ia = pick[s];
        int pos = 0;
        for (int j = 0; j < k_eff; ++j) pos += pick[j] < ia;
        sel_tmp[pos] = ia;
      }
    }
  }
  selg.sync();
  if (rank == 0) asm volatile("bar.arrive 3, 256;" ::: "memory");       // warps 4-7 write the list out
  if (!sel_share) cluster_wait();
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
