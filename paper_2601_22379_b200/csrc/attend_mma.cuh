// Sparse attention + fused residual-linear term for bf16 K/V on tensor cores (GQA groups of up to 8 heads).
//
// The CTAs that serve one (sequence, KV head) unit form a thread-block cluster; CTA r of the cluster walks the
// selected blocks r, r + CS, r + 2 CS, ... through a shared-memory ring that TMA fills (tiled tensor copies with
// the 128-byte swizzle, so the ldmatrix reads below are bank-conflict free).  A CTA holds NG groups of four warps;
// group j takes every NG-th block of the CTA's list and its warps take the block's 16-token slices.  Two shapes are
// built: one group and a two-slot ring for launches with many units (two CTAs share an SM), and two groups with a
// ring as deep as shared memory allows for launches that fit the machine with one CTA per SM, where what counts is
// how many tiles are in flight at once.  Per slice the query group is the M side of two thin products that share one accumulator,
//     rows 0..7  :  S = Q K^T            (exact branch,  Section 2.2 of the paper, Eq. gqa-sparse)
//     rows 8..15 :  A = phi(Q) phi(K)^T  (linear branch, Section 3.2, Eq. rla-impl-2)
// where phi(K) is formed element-wise from the very K fragments just used (one ex2 per element, with the cached
// per-token log-sum-exp), so the selected linear term reads nothing extra.  After the online softmax on rows
// 0..7 the tile [P ; A] is the left operand of one product with the V tile, which accumulates the softmax
// numerator and o_tilde together.  The linear branch keeps far more than the 8 or 11 bits of one 16-bit operand,
// because o_bar - o_tilde cancels when most of the context is selected and the RMSNorm then rescales the
// difference (Section 3.2, "Numerical Stability": the states stay in high precision): phi(q) and phi(k) enter
// their product as an fp16 head plus an fp16 remainder each, and the coefficients phi(q).phi(k_t) enter the
// product with V as three bf16 parts.  For groups of up to 4 heads the
// extra parts ride in the accumulator rows that would otherwise be padding.
//
// Merge (Eq. rla-impl-3, Section 3.3): every CTA sends its partial results of head g into CTA g % CS of the cluster as
// asynchronous stores (st.async) that count their bytes on a barrier there; that CTA goes on when all of them have
// arrived, subtracts o_tilde from o_bar, applies the RMSNorm and writes the output.  No barrier of the whole cluster
// lies on the path (one closes the kernel: nobody leaves while a sibling may still store into it); all waits are
// bounded mbarrier polls or CTA barriers.
//
// The body is a device function: it is the whole of the attend + merge kernel (spla_decode_selected, and spla_decode
// where the fused kernel does not apply) and the second half of the fused decode kernel (decode_fused.cuh), where it
// runs on the first four warps of a larger CTA (FUSED: its CTA-wide barriers then count those 128 threads only, and
// the kernel around it has already made the selection visible).
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>

#include "spla_internal.h"

namespace spla {

namespace {

constexpr int kMaxSlots = 4;       // ring positions at most (two per warp group)

// Tiled TMA load of one K or V tile (never multicast): the map sees the cache as [column halves][rows][64 columns]; the
// box starts at column 0 of `row` and takes every half.
__device__ __forceinline__ void tma_load_tile(uint32_t dst, const CUtensorMap* map, int row, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
               "l"(map), "r"(0), "r"(row), "r"(0), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// Same shape with fp16 inputs: used for phi(q) phi(k)^T, whose operands lie in [0, 1] and are produced here, so
// the 11-bit fp16 significand can be chosen over bf16's 8 bits (the residual o_bar - o_tilde cancels heavily
// when a large share of the context is selected, which amplifies the rounding of o_tilde).
__device__ __forceinline__ void mma_f16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
  __half2 v = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float f16_lo(uint32_t x) { return __low2float(*reinterpret_cast<const __half2*>(&x)); }
__device__ __forceinline__ float f16_hi(uint32_t x) { return __high2float(*reinterpret_cast<const __half2*>(&x)); }

constexpr int kPad = 8;   // floats of padding per row of the cross-warp reduction buffer

// Bytes of the tile ring (reused for the cross-warp fold); as a kernel of its own the receive area of the merge follows.
__host__ __device__ constexpr size_t attend_mma_ring_bytes(int B, int D, int groups) {
  const size_t ring = (size_t)(2 * groups) * ((2 * (size_t)B * D * 2 + (size_t)B * 4 + 1023) / 1024 * 1024);
  const size_t fold = (size_t)(groups * (kAttendThreads / 32) * (16 * (D + kPad) + 16)) * sizeof(float);
  return (ring > fold ? ring : fold);
}
constexpr size_t attend_mma_recv_bytes(int D) { return (size_t)16 * (2 * D + 2) * 4; }

}  // namespace

// PACK: the group has at most 4 heads, so accumulator rows 4..7 and 12..15 are padding; rows 12..15 then carry
// the bf16 remainder of the linear coefficients and no extra products are needed for it.
template <int D, bool PACK, int NG, bool FUSED>
__device__ __forceinline__ void attend_mma_body(const Params& p, const CUtensorMap& map_k, const CUtensorMap& map_v,
                                                const __nv_bfloat16* __restrict__ q, const float* __restrict__ rms_weight,
                                                float* __restrict__ out, float* __restrict__ dbg_sparse,
                                                float* __restrict__ dbg_rla, unsigned char* smem_raw,
                                                const int* sel_share = nullptr, uint64_t* full_ext = nullptr,
                                                unsigned char* recv_raw = nullptr, const float* obar_local = nullptr) {
  constexpr int KS = D / 16;        // k-steps of the two QK-type products
  constexpr int NT = D / 8;         // n-tiles of the PV-type product
  constexpr int NTHR = NG * kAttendThreads;
  constexpr int NWARP = NTHR / 32;
  __shared__ __align__(8) uint64_t full_own[kMaxSlots + 1];
  uint64_t* full = full_ext ? full_ext : full_own;      // (the fused kernel initialises its barriers at its start)
  uint64_t* mbar_merge = full + kMaxSlots;              // completes when every sibling's partial results have arrived here
  __shared__ float red_s[NWARP];
  __shared__ int sel_s[kMaxTopK];
  __shared__ int err_s;

  const int u = blockIdx.y;
  const int rank = blockIdx.x, CS = gridDim.x;
  const int b = u / p.Hkv, h = u % p.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int gi = warp >> 2, wg = warp & 3, gtid = tid & (kAttendThreads - 1);   // group, warp in group, thread in group
  const int g = lane >> 2, t = lane & 3;
  const int G = p.G, B = p.B;
  const int TB = p.tile_rows, TPB = B / TB;   // rows of a K/V tile, tiles per block (blocks of 128 tokens at d = 128 come as two tiles)
  const bool rla_on = !(p.flags & 4u);
  constexpr int ns = 2 * NG;                    // ring positions in use (a multiple of NG: a group refills what it frees)
  auto cta_sync = [&]() {                      // barrier over the threads that run this body
    if constexpr (FUSED) asm volatile("bar.sync 1, %0;" ::"n"(NG * kAttendThreads) : "memory");
    else __syncthreads();
  };
  auto group_sync = [&]() {                    // barrier over the four warps of this group
    if constexpr (NG == 1) cta_sync();
    else asm volatile("bar.sync %0, %1;" ::"r"(2 + gi), "r"(kAttendThreads) : "memory");
  };

  if constexpr (!FUSED) pdl_launch_dependents();
  // ---- query fragments first: they depend on nothing the preceding kernel writes, so under programmatic
  // dependent launch this part overlaps that kernel's tail.  Rows = heads of the group, held in registers.
  // qa: rows 0..7 of the first product (raw q; the softmax scale is applied to the fp32 logits);
  // fa: rows 8..15 of the second product, phi(q) = softmax(phi_scale * q) in fp16.
  // fl_s (groups of more than 4 heads only): the fp16 remainder of phi(q), a second left operand, kept in shared
  // memory (the same for every warp) to stay clear of the register limit; in the packed layout rows 12..15 of fa
  // carry that remainder for heads 0..3 instead.
  __shared__ uint32_t fl_s[PACK ? 1 : KS][2][32];
  uint32_t qa[KS][2], fa[KS][2];
  auto make_fragments = [&]() {
    const bool hv = g < G;
    const bool rem_row = PACK && g >= 4;                  // this lane's row 8 + g holds the remainder of head g - 4
    const int hq = rem_row ? g - 4 : g;                   // head whose phi(q) this lane forms
    const bool hp = hq < G;
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)b * p.Hq + (size_t)h * G + (hp ? hq : 0)) * D);
    const float a2 = p.phi_scale * kLog2e;
    float mx = -INFINITY;
    uint32_t qr[KS][2];
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      qr[kk][0] = hp ? __ldg(qrow + 8 * kk + t) : 0u;
      qr[kk][1] = hp ? __ldg(qrow + 8 * kk + 4 + t) : 0u;
      qa[kk][0] = hv ? qr[kk][0] : 0u;                    // rows of padding carry zero queries in the exact branch
      qa[kk][1] = hv ? qr[kk][1] : 0u;
    }
#pragma unroll
    for (int kk = 0; kk < KS; ++kk)
      mx = fmaxf(mx, fmaxf(fmaxf(bf16_lo(qr[kk][0]), bf16_hi(qr[kk][0])), fmaxf(bf16_lo(qr[kk][1]), bf16_hi(qr[kk][1]))));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    float e[KS][4], sum = 0.f;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      e[kk][0] = exp2f((bf16_lo(qr[kk][0]) - mx) * a2); e[kk][1] = exp2f((bf16_hi(qr[kk][0]) - mx) * a2);
      e[kk][2] = exp2f((bf16_lo(qr[kk][1]) - mx) * a2); e[kk][3] = exp2f((bf16_hi(qr[kk][1]) - mx) * a2);
      sum += (e[kk][0] + e[kk][1]) + (e[kk][2] + e[kk][3]);
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    const float inv = (hp && rla_on) ? 1.f / sum : 0.f;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      const float f0 = e[kk][0] * inv, f1 = e[kk][1] * inv, f2 = e[kk][2] * inv, f3 = e[kk][3] * inv;
      const uint32_t h0 = pack_f16(f0, f1), h1 = pack_f16(f2, f3);
      const uint32_t l0 = pack_f16(f0 - f16_lo(h0), f1 - f16_hi(h0)), l1 = pack_f16(f2 - f16_lo(h1), f3 - f16_hi(h1));
      if constexpr (PACK) {
        fa[kk][0] = rem_row ? l0 : h0;
        fa[kk][1] = rem_row ? l1 : h1;
      } else {
        fa[kk][0] = h0; fa[kk][1] = h1;
        if (warp == 0) { fl_s[kk][0][lane] = l0; fl_s[kk][1][lane] = l1; }   // (visible after a barrier below)
      }
    }
  };
  // As a kernel of its own the fragments are formed first (under programmatic dependent launch this overlaps the
  // preceding kernel's tail); inside the fused kernel the selection is already there, so the first tiles are
  // requested first and the fragments are formed while they are on their way.
  if constexpr (!FUSED) make_fragments();
  if (tid == 0) {
    if (!full_ext) {
      for (int s = 0; s <= kMaxSlots; ++s) mbar_init(&full[s], 1);
      mbar_init_done();
    }
    err_s = 0;
  }
  // As a kernel of its own: the siblings may store here once everybody's merge barrier exists; announced now,
  // completed before the first such store.  (In the fused kernel the score phase has done that.)
  if constexpr (!FUSED) cluster_arrive();

  if constexpr (!FUSED) pdl_wait();             // the selection of this step is complete and visible from here on

  // the selection, its size and the length: from the workspace, or (fused kernel) from where the score phase's leader
  // left them in this CTA's shared memory
  int nsel = sel_share ? sel_share[kMaxTopK] : __ldcg(p.n_sel + u);
  const int L = sel_share ? sel_share[kMaxTopK + 1] : checked_len(p, b);
  for (int i = tid; i < p.top_k; i += NTHR) sel_s[i] = sel_share ? (i < nsel ? sel_share[i] : -1) : __ldcg(p.sel + (size_t)u * p.top_k + i);
  if (p.flags & kDebugBounds) {
    // checked build: the list must name nsel existing blocks; it is cut at the first entry that does not, and the
    // status word says so (every CTA of the cluster sees the same list and cuts it at the same place)
    __shared__ int first_bad_s;
    if (tid == 0) first_bad_s = min(max(nsel, 0), p.top_k);
    cta_sync();
    const int nblk_chk = (L + B - 1) / B;
    for (int i = tid; i < min(nsel, p.top_k); i += NTHR)
      if (sel_s[i] < 0 || sel_s[i] >= nblk_chk) atomicMin(&first_bad_s, i);
    cta_sync();
    if (first_bad_s != nsel) {
      if (tid == 0 && rank == 0) atomicExch(p.status, kStatusBounds);
      nsel = first_bad_s;
    }
  }
  cta_sync();                              // selection list and barrier initialisation visible to the CTA

  const int n_tiles = nsel * TPB;                                    // tile j: part j % TPB of pick j / TPB
  const int nb = n_tiles > rank ? (n_tiles - rank + CS - 1) / CS : 0;   // my tiles: j = rank + i * CS
  const int tile_bytes = TB * D * 2;
  const int slot_bytes = (2 * tile_bytes + TB * 4 + 1023) & ~1023;  // K tile, V tile, per-token lse; the swizzle needs 1 KB alignment
  // The copies of tile i of this CTA (K, V, the tokens' log-sum-exp): `part` < 0 issues all of them from one thread;
  // otherwise the caller spreads the parts 0 .. kTileParts - 1 over lanes (part 0 also announces the bytes; the
  // barrier's transaction count may run ahead of that announcement).
  constexpr int kTileParts = 3;
  auto issue = [&](int i, int part = -1) {
    const int slot = i % ns;
    const int j = rank + i * CS;
    const int blk = min(max(sel_s[j / TPB], 0), p.max_blocks - 1);   // (a list entry can never address outside the cache)
    const uint32_t base = smem_u32(smem_raw + (size_t)slot * slot_bytes);
    const int row0 = (int)(((size_t)u * p.max_blocks + blk) * B) + (j % TPB) * TB;
    if (part <= 0) mbar_expect_tx(&full[slot], (uint32_t)(2 * tile_bytes + TB * 4 + p.dbg_tx_extra));
    if (part <= 0) tma_load_tile(base, &map_k, row0, &full[slot]);
    if (part < 0 || part == 1) tma_load_tile(base + tile_bytes, &map_v, row0, &full[slot]);
    if (part < 0 || part == 2)
      bulk_g2s(smem_raw + (size_t)slot * slot_bytes + 2 * tile_bytes, p.tok_lse + (size_t)row0, (uint32_t)(TB * 4), &full[slot]);
  };
  if (tid < ns * kTileParts && tid / kTileParts < nb) issue(tid / kTileParts, tid % kTileParts);   // the first tiles, one copy per lane
  if constexpr (FUSED) {
    make_fragments();
    if constexpr (!PACK) cta_sync();          // fl_s is read by every warp
  }

  // ---- per-warp running state over its slices -----------------------------------------------------------
  float m_run = -INFINITY, l_run = 0.f;      // row g of the exact branch (l: this lane's share)
  float o[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
  const float sc2 = p.sm_scale * kLog2e;
  const float a2 = p.phi_scale * kLog2e;
  const int spb = TB / 16;                   // slices per tile
  const int mi = lane >> 3, r8 = lane & 7;   // ldmatrix: which 8x8 matrix this lane addresses, and which row
  const int half_bytes = TB * 128;

  // A wait that runs out marks the warp dead: it skips the arithmetic from then on but still joins every barrier of
  // its group, so that the barrier counts match whatever the other warps saw.
  bool dead = false;
#pragma unroll 1
  for (int i = gi; i < nb; i += NG) {
    const int slot = i % ns;
    if (!dead && !__all_sync(0xffffffffu, mbar_wait(&full[slot], (i / ns) & 1, p.wait_limit))) {
      dead = true;
      if (lane == 0) atomicExch(&err_s, 1);
    }
    unsigned char* sb = smem_raw + (size_t)slot * slot_bytes;
    const uint32_t ks = smem_u32(sb);
    const uint32_t vs = ks + tile_bytes;
    const float* lse_s = reinterpret_cast<const float*>(sb + 2 * tile_bytes);
    const int jt = rank + i * CS;
    const int blk = sel_s[jt / TPB];
    const int ntok = max(0, min(TB, L - blk * B - (jt % TPB) * TB));   // (0: a tile of the open block wholly past the end)
    if (ntok < TB) {
      // the open block of the sequence: rows past its end hold whatever the cache memory holds; the value rows
      // must be zero so that (probability 0) x (garbage) cannot produce a NaN
      for (int idx = gtid; idx < (TB - ntok) * (D / 8) && !dead; idx += kAttendThreads) {
        const int row = ntok + idx / (D / 8), ch = idx % (D / 8);
        *reinterpret_cast<uint4*>(sb + tile_bytes + (ch >> 3) * half_bytes + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) =
            make_uint4(0u, 0u, 0u, 0u);
      }
      group_sync();
    }
#pragma unroll 1
    for (int sl = wg; sl < spb; sl += 4) {
      const int tok0 = sl * 16;
      if (tok0 >= ntok || dead) break;
      const float lse2_0 = lse_s[tok0 + g] * kLog2e, lse2_1 = lse_s[tok0 + 8 + g] * kLog2e;
      // two accumulator tiles per n-tile (one per product) so that the dependent chain of each is half as long;
      // rows 0..7 of the first and rows 8..15 of the second are the meaningful halves
      float sacc[2][4], aacc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f;
        aacc[nt][0] = aacc[nt][1] = aacc[nt][2] = aacc[nt][3] = 0.f;
      }
      const uint32_t krow = ks + (tok0 + (mi >> 1) * 8 + r8) * 128;
#pragma unroll
      for (int kk = 0; kk < KS; ++kk) {
        uint32_t kb[4];
        const int ch = 2 * kk + (mi & 1);
        ldmatrix_x4(kb, krow + (ch >> 3) * half_bytes + (((ch & 7) ^ r8) << 4));
        mma_bf16(sacc[0], qa[kk][0], 0u, qa[kk][1], 0u, kb[0], kb[1]);
        mma_bf16(sacc[1], qa[kk][0], 0u, qa[kk][1], 0u, kb[2], kb[3]);
        // phi(k) of the same fragments, as an fp16 head and an fp16 remainder (together 17 or more significant bits)
        uint32_t pb[4], pl[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const float ls = x < 2 ? lse2_0 : lse2_1;
          const float e0 = ex2(fmaf(bf16_lo(kb[x]), a2, -ls)), e1 = ex2(fmaf(bf16_hi(kb[x]), a2, -ls));
          pb[x] = pack_f16(e0, e1);
          pl[x] = pack_f16(e0 - f16_lo(pb[x]), e1 - f16_hi(pb[x]));
        }
        mma_f16(aacc[0], 0u, fa[kk][0], 0u, fa[kk][1], pb[0], pb[1]);
        mma_f16(aacc[1], 0u, fa[kk][0], 0u, fa[kk][1], pb[2], pb[3]);
        mma_f16(aacc[0], 0u, fa[kk][0], 0u, fa[kk][1], pl[0], pl[1]);
        mma_f16(aacc[1], 0u, fa[kk][0], 0u, fa[kk][1], pl[2], pl[3]);
        if constexpr (!PACK) {                         // remainder of phi(q) times the head of phi(k)
          const uint32_t fl0 = fl_s[kk][0][lane], fl1 = fl_s[kk][1][lane];
          mma_f16(aacc[0], 0u, fl0, 0u, fl1, pb[0], pb[1]);
          mma_f16(aacc[1], 0u, fl0, 0u, fl1, pb[2], pb[3]);
        }
      }
      if constexpr (PACK) {                            // rows 12..15 (remainder of phi(q)) onto rows 8..11
#pragma unroll
        for (int nt = 0; nt < 2; ++nt) {
          aacc[nt][2] += __shfl_down_sync(0xffffffffu, aacc[nt][2], 16);
          aacc[nt][3] += __shfl_down_sync(0xffffffffu, aacc[nt][3], 16);
        }
      }
      // online softmax on rows 0..7; rows 8..15 stay linear.  Tokens past the end of the sequence are masked.
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const bool valid = tok0 + nt * 8 + 2 * t + c < ntok;
          sacc[nt][c] = valid ? sacc[nt][c] * sc2 : -INFINITY;
          sacc[nt][2 + c] = valid ? aacc[nt][2 + c] : 0.f;
          mx = fmaxf(mx, sacc[nt][c]);
        }
      }
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);            // finite: the slice has at least one valid token
      const float corr = ex2(m_run - m_new);
      m_run = m_new;
      float psum = 0.f;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        sacc[nt][0] = ex2(sacc[nt][0] - m_new);
        sacc[nt][1] = ex2(sacc[nt][1] - m_new);
        psum += sacc[nt][0] + sacc[nt][1];
      }
      l_run = fmaf(l_run, corr, psum);
      // [P ; A] as the left operand of the product with V (bf16, like V).  The linear coefficients are split
      // into three bf16 parts (head, remainder, remainder of that) so that o_tilde keeps ~24 bits of them.
      uint32_t pa0 = pack_bf16(sacc[0][0], sacc[0][1]), pa2 = pack_bf16(sacc[1][0], sacc[1][1]);
      uint32_t pa1 = pack_bf16(sacc[0][2], sacc[0][3]), pa3 = pack_bf16(sacc[1][2], sacc[1][3]);
      const float r00 = sacc[0][2] - bf16_lo(pa1), r01 = sacc[0][3] - bf16_hi(pa1);
      const float r10 = sacc[1][2] - bf16_lo(pa3), r11 = sacc[1][3] - bf16_hi(pa3);
      const uint32_t ra1 = pack_bf16(r00, r01), ra3 = pack_bf16(r10, r11);
      const uint32_t rb1 = pack_bf16(r00 - bf16_lo(ra1), r01 - bf16_hi(ra1));
      const uint32_t rb3 = pack_bf16(r10 - bf16_lo(ra3), r11 - bf16_hi(ra3));
      float corr_o = corr;
      if constexpr (PACK) {
        // rows 12..15 <- second parts of heads 0..3, rows 4..7 <- their third parts (from the lanes 16 below);
        // rows 4..7 then accumulate a linear term and must not take the softmax rescaling
        const uint32_t u1 = __shfl_up_sync(0xffffffffu, ra1, 16), u3 = __shfl_up_sync(0xffffffffu, ra3, 16);
        const uint32_t w1 = __shfl_up_sync(0xffffffffu, rb1, 16), w3 = __shfl_up_sync(0xffffffffu, rb3, 16);
        if (g >= 4) { pa1 = u1; pa3 = u3; pa0 = w1; pa2 = w3; corr_o = 1.f; }
      }
      const uint32_t vrow = vs + (tok0 + (mi & 1) * 8 + r8) * 128;
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t vb[4];
        const int ch = 2 * np + (mi >> 1);
        ldmatrix_x4_trans(vb, vrow + (ch >> 3) * half_bytes + (((ch & 7) ^ r8) << 4));
        o[2 * np][0] *= corr_o; o[2 * np][1] *= corr_o;
        o[2 * np + 1][0] *= corr_o; o[2 * np + 1][1] *= corr_o;
        mma_bf16(o[2 * np], pa0, pa1, pa2, pa3, vb[0], vb[1]);
        mma_bf16(o[2 * np + 1], pa0, pa1, pa2, pa3, vb[2], vb[3]);
        if constexpr (!PACK) {
          if (rla_on) {
            mma_bf16(o[2 * np], 0u, ra1, 0u, ra3, vb[0], vb[1]);
            mma_bf16(o[2 * np + 1], 0u, ra1, 0u, ra3, vb[2], vb[3]);
            mma_bf16(o[2 * np], 0u, rb1, 0u, rb3, vb[0], vb[1]);
            mma_bf16(o[2 * np + 1], 0u, rb1, 0u, rb3, vb[2], vb[3]);
          }
        }
      }
    }
    group_sync();                                      // every warp of the group is done with this slot
    if (gtid == 0 && i + ns < nb && !dead) {
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy reads before the async-proxy refill
      issue(i + ns);
    }
  }
  if (tid == 0 && err_s) atomicExch(p.status, kStatusTimeout);

  // (a kernel input the merge needs at its very end: requested now, it arrives under the fold)
  const float gamma0 = (rank < G && tid < D) ? __ldg(rms_weight + ((size_t)h * G + rank) * D + tid) : 0.f;

  // ---- fold the four warps together ------------------------------------------------------------------------
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  cta_sync();                                   // the ring is dead: its space becomes the reduction buffer
  float* red_o = reinterpret_cast<float*>(smem_raw);                    // [NWARP][16][D + kPad]
  float* red_m = red_o + NWARP * 16 * (D + kPad);                       // [NWARP][8]
  float* red_l = red_m + NWARP * 8;                                     // [NWARP][8]
  // Where the partial results of head hd go: into the CTA that merges it, hd % CS, entry (hd / CS) * CS + sender of
  // its receive area (at most 16 entries: [2][D] floats each, then the (max, sum) pairs), as asynchronous stores that
  // count their bytes on that CTA's merge barrier.
  constexpr int kRecvEntries = 16;
  float* recv = recv_raw ? reinterpret_cast<float*>(recv_raw)
                         : reinterpret_cast<float*>(smem_raw + attend_mma_ring_bytes(TB, D, NG));  // [16][2][D], [16][2]
  float* recv_ml = recv + kRecvEntries * 2 * D;
  const int my_heads = G > rank ? (G - rank + CS - 1) / CS : 0;         // heads this CTA merges
  if (tid == 0 && my_heads > 0) mbar_expect_tx(mbar_merge, (uint32_t)(my_heads * CS * (2 * D * 4 + 8)));
  // every warp leaves its rows as they are, with its running maximum and sum; the combiner rescales (one barrier less
  // than agreeing on the maximum first)
  if (t == 0) { red_m[warp * 8 + g] = m_run; red_l[warp * 8 + g] = l_run; }
  {
    float* ro = red_o + (size_t)warp * 16 * (D + kPad);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      *reinterpret_cast<float2*>(ro + (size_t)g * (D + kPad) + nt * 8 + 2 * t) = make_float2(o[nt][0], o[nt][1]);
      *reinterpret_cast<float2*>(ro + (size_t)(g + 8) * (D + kPad) + nt * 8 + 2 * t) = make_float2(o[nt][2], o[nt][3]);
    }
  }
  cta_sync();
  if constexpr (!FUSED) cluster_wait();         // (every CTA's merge barrier exists: announced at the top)
  const uint32_t recv0 = smem_u32(recv), recv_ml0 = smem_u32(recv_ml), bar0 = smem_u32(mbar_merge);
  for (int idx = tid; idx < 2 * G * (D / 4); idx += NTHR) {             // four columns per thread and step
    const int br = idx / (G * (D / 4)), hd = (idx / (D / 4)) % G, c4 = (idx % (D / 4)) * 4;   // branch, head, first column
    const int rr = br * 8 + hd;
    float fw[NWARP];                                                    // 0 for a warp that saw no token
    {
      float M = red_m[hd];
#pragma unroll
      for (int w = 1; w < NWARP; ++w) M = fmaxf(M, red_m[w * 8 + hd]);
#pragma unroll
      for (int w = 0; w < NWARP; ++w) fw[w] = (br == 0 && M > -INFINITY) ? ex2(red_m[w * 8 + hd] - M) : (br == 0 ? 0.f : 1.f);
    }
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int w = 0; w < NWARP; ++w) {
      const float4 a = *reinterpret_cast<const float4*>(red_o + ((size_t)w * 16 + rr) * (D + kPad) + c4);
      s.x += a.x * fw[w]; s.y += a.y * fw[w]; s.z += a.z * fw[w]; s.w += a.w * fw[w];
      if (PACK && br == 1) {                                              // the second and third parts of the coefficients
        const float4 b2 = *reinterpret_cast<const float4*>(red_o + ((size_t)w * 16 + rr + 4) * (D + kPad) + c4);
        const float4 b3 = *reinterpret_cast<const float4*>(red_o + ((size_t)w * 16 + hd + 4) * (D + kPad) + c4);
        s.x += b2.x + b3.x; s.y += b2.y + b3.y; s.z += b2.z + b3.z; s.w += b2.w + b3.w;
      }
    }
    const uint32_t dest = (uint32_t)(hd % CS);
    const int entry = (hd / CS) * CS + rank;
    st_async_v4(map_to_rank(recv0 + (uint32_t)(((entry * 2 + br) * D + c4) * 4), dest), s.x, s.y, s.z, s.w,
                map_to_rank(bar0, dest));
  }
  if (tid < G) {
    float Mg = red_m[tid], Lg = 0.f;
#pragma unroll
    for (int w = 1; w < NWARP; ++w) Mg = fmaxf(Mg, red_m[w * 8 + tid]);
#pragma unroll
    for (int w = 0; w < NWARP; ++w) Lg += Mg > -INFINITY ? red_l[w * 8 + tid] * ex2(red_m[w * 8 + tid] - Mg) : 0.f;
    const uint32_t dest = (uint32_t)(tid % CS);
    const int entry = (tid / CS) * CS + rank;
    st_async_v2(map_to_rank(recv_ml0 + (uint32_t)(entry * 8), dest), __float_as_uint(Mg), __float_as_uint(Lg),
                map_to_rank(bar0, dest));
  }

  // ---- merge: CTA r of the cluster owns heads r, r + CS, ...; one thread per output column ---------------
  const int nblk_u = (L + B - 1) / B;
  const bool rla = rla_on && nsel < nblk_u;          // everything selected: the residual is exactly zero
  if (my_heads > 0) {
    // as a kernel of its own o_bar comes from the workspace (written by the preceding kernel): requested before the wait
    float ob0[kStateSplits];
#pragma unroll
    for (int s = 0; s < kStateSplits; ++s)
      ob0[s] = (!FUSED && rla && tid < D) ? __ldcg(p.obar_part + (((size_t)u * kStateSplits + s) * G + rank) * D + tid) : 0.f;
    if (!__all_sync(0xffffffffu, mbar_wait(mbar_merge, 0, p.wait_limit)) && lane == 0) atomicExch(p.status, kStatusTimeout);
    if constexpr (FUSED) asm volatile("bar.sync 2, 256;" ::: "memory");   // warps 4-7 have left o_bar of this CTA's heads
    for (int hd = rank, hi = 0; hd < G; hd += CS, ++hi) {
      const int col = tid;
      float o_sp = 0.f, o_til = 0.f, o_bar = 0.f;
      if (nsel > 0) {
        const float* e_ml = recv_ml + (size_t)hi * CS * 2;
        const float* e_o = recv + (size_t)hi * CS * 2 * D;
        float Mx = -INFINITY;
        for (int r = 0; r < CS; ++r) Mx = fmaxf(Mx, e_ml[r * 2]);
        float Ls = 0.f;
        for (int r = 0; r < CS; ++r) {
          const float w = ex2(e_ml[r * 2] - Mx);
          Ls = fmaf(w, e_ml[r * 2 + 1], Ls);
          if (col < D) {
            o_sp = fmaf(w, e_o[(size_t)(r * 2) * D + col], o_sp);
            if (rla) o_til += e_o[(size_t)(r * 2 + 1) * D + col];
          }
        }
        o_sp /= Ls;
        if (rla && col < D) {
          if constexpr (FUSED) {
            o_bar = obar_local[(size_t)hi * D + col];
          } else if (hi == 0) {
#pragma unroll
            for (int s = 0; s < kStateSplits; ++s) o_bar += ob0[s];
          } else {
#pragma unroll
            for (int s = 0; s < kStateSplits; ++s)
              o_bar += __ldcg(p.obar_part + (((size_t)u * kStateSplits + s) * G + hd) * D + col);
          }
        }
      }
      const float r_ = (rla && col < D) ? o_bar - o_til : 0.f;
      float sq = warp_sum(r_ * r_);
      cta_sync();
      if (lane == 0) red_s[warp] = sq;
      cta_sync();
      float tot = 0.f;
#pragma unroll
      for (int w = 0; w < NWARP; ++w) tot += red_s[w];
      if (col < D) {
        const size_t oidx = ((size_t)b * p.Hq + (size_t)h * G + hd) * D + col;
        float res = o_sp;
        const float gamma = hd == rank ? gamma0 : rms_weight[((size_t)h * G + hd) * D + col];
        if (rla) res += gamma * r_ * rsqrtf(tot / D + p.rms_eps);
        out[oidx] = res;
        if (dbg_sparse) dbg_sparse[oidx] = o_sp;
        if (dbg_rla) dbg_rla[oidx] = r_;
      }
    }
  } else if constexpr (FUSED) {
    asm volatile("bar.sync 2, 256;" ::: "memory");   // (the barrier with warps 4-7 counts every thread)
  }
  // ---- the closing barrier: nobody leaves while a sibling may still store into it; and the CTAs of a cluster leave
  // together (when some left earlier than others, the next launch's clusters no longer all found room at once)
  cluster_sync_all();
}

}  // namespace spla
