// Sparse attention + fused residual-linear term for bf16 K/V on tensor cores (GQA groups of up to 8 heads).
//
// For one (unit, group of selected blocks) the CTA stages the K and V tiles with 16-byte asynchronous copies
// into an XOR-swizzled shared-memory layout, and each warp walks 16-token slices.  Per slice the query group
// is the M side of two thin products that share one accumulator tile,
//     rows 0..7  :  S   = Q K^T           (exact branch,  Section 2.2, Eq. gqa-sparse)
//     rows 8..15 :  A   = phi(Q) phi(K)^T (linear branch, Section 3.2, Eq. rla-impl-2)
// where phi(K) is formed element-wise from the very K fragments just used (one ex2 per element, with the
// cached per-token log-sum-exp), so the selected linear term reads nothing extra.  After the online softmax
// on rows 0..7 the tile [P ; A] is the left operand of one product with the V tile, which accumulates the
// softmax numerator (rows 0..7) and o_tilde (rows 8..15) together.  The last CTA of the unit merges.
#include <cuda_fp16.h>

#include "attend_common.cuh"
#include "spla_internal.h"

namespace spla {

namespace {

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_pending(int n) {   // at most n groups still in flight
  switch (n) {
    case 0: asm volatile("cp.async.wait_group 0;" ::: "memory"); break;
    case 1: asm volatile("cp.async.wait_group 1;" ::: "memory"); break;
    case 2: asm volatile("cp.async.wait_group 2;" ::: "memory"); break;
    default: asm volatile("cp.async.wait_group 3;" ::: "memory"); break;
  }
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// D += A(16x16, row) * B(16x8, col), bf16 inputs, fp32 accumulate.
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }

constexpr int kPad = 8;   // floats of padding per row of the cross-warp reduction buffer

}  // namespace

template <int D>
__global__ void __launch_bounds__(kAttendThreads, 3) attend_mma_kernel(const Params p, const __nv_bfloat16* __restrict__ q,
                                                                    const float* __restrict__ rms_weight,
                                                                    float* __restrict__ out, float* __restrict__ dbg_sparse,
                                                                    float* __restrict__ dbg_rla) {
  constexpr int KS = D / 16;        // k-steps of the two QK-type products
  constexpr int NT = D / 8;         // n-tiles of the PV-type product
  constexpr int CPR = D / 8;        // 16-byte chunks per K/V row
  constexpr int ROWB = D * 2;       // bytes per K/V row
  constexpr int NWARP = kAttendThreads / 32;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int flag_s;

  const int u = blockIdx.y, item = blockIdx.x;
  const int b = u / p.Hkv, h = u % p.Hkv;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const int G = p.G, B = p.B, bpc = p.bpc;
  const bool rla = !(p.flags & 4u);

  pdl_launch_dependents();
  // ---- query fragments first: they depend on nothing the preceding kernel writes, so under programmatic
  // dependent launch this part overlaps that kernel's tail.  Rows = heads of the group, held in registers.
  // qa: rows 0..7 of the first product (raw q; the softmax scale is applied to the fp32 logits);
  // fa: rows 8..15 of the second product, phi(q) = softmax(phi_scale * q) in fp16.
  uint32_t qa[KS][2], fa[KS][2];
  {
    const bool hv = g < G;
    const uint32_t* qrow = reinterpret_cast<const uint32_t*>(q + ((size_t)b * p.Hq + (size_t)h * G + (hv ? g : 0)) * D);
    const float a2 = p.phi_scale * kLog2e;
    float mx = -INFINITY;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      qa[kk][0] = hv ? __ldg(qrow + 8 * kk + t) : 0u;
      qa[kk][1] = hv ? __ldg(qrow + 8 * kk + 4 + t) : 0u;
    }
#pragma unroll
    for (int kk = 0; kk < KS; ++kk)
      mx = fmaxf(mx, fmaxf(fmaxf(bf16_lo(qa[kk][0]), bf16_hi(qa[kk][0])), fmaxf(bf16_lo(qa[kk][1]), bf16_hi(qa[kk][1]))));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
    float e[KS][4], sum = 0.f;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      e[kk][0] = exp2f((bf16_lo(qa[kk][0]) - mx) * a2); e[kk][1] = exp2f((bf16_hi(qa[kk][0]) - mx) * a2);
      e[kk][2] = exp2f((bf16_lo(qa[kk][1]) - mx) * a2); e[kk][3] = exp2f((bf16_hi(qa[kk][1]) - mx) * a2);
      sum += (e[kk][0] + e[kk][1]) + (e[kk][2] + e[kk][3]);
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    const float inv = (hv && rla) ? 1.f / sum : 0.f;
#pragma unroll
    for (int kk = 0; kk < KS; ++kk) {
      fa[kk][0] = pack_f16(e[kk][0] * inv, e[kk][1] * inv);
      fa[kk][1] = pack_f16(e[kk][2] * inv, e[kk][3] * inv);
    }
  }

  pdl_wait();                                   // the selection of this step is complete and visible from here on

  // one round trip: the count, the (speculatively addressed) block indices of this CTA, the sequence length
  const int j0 = item * bpc;
  const int nsel = __ldcg(p.n_sel + u);
  const int L = __ldcg(p.seq_lens + b);
  int blk_j[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) blk_j[j] = __ldcg(p.sel + (size_t)u * p.top_k + min(j0 + j, p.top_k - 1));
  const int n_items = (nsel + bpc - 1) / bpc;
  if (item >= n_items) {
    if (nsel == 0 && item == 0) write_zero_unit<D>(p, u, out, dbg_sparse, dbg_rla);
    return;
  }
  SPLA_MARK(p, u, 32 + item, 0);
  const int nb = min(bpc, nsel - j0);
  const int tile_bytes = B * ROWB;
  unsigned char* lse_base = smem_raw + (size_t)bpc * 2 * tile_bytes;

  // ---- stage the tiles: 16-byte async copies, chunk index XOR (row & 7), rows past the sequence end zero-filled
  int n_tok[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    n_tok[j] = 0;
    if (j < nb) {
      const int blk = blk_j[j];
      n_tok[j] = min(B, L - blk * B);
      const size_t tile = (size_t)u * p.max_blocks + blk;
      const __nv_bfloat16* ksrc = reinterpret_cast<const __nv_bfloat16*>(p.k_cache) + tile * B * D;
      const __nv_bfloat16* vsrc = reinterpret_cast<const __nv_bfloat16*>(p.v_cache) + tile * B * D;
      const uint32_t kdst = smem_u32(smem_raw + (size_t)j * 2 * tile_bytes);
      const uint32_t vdst = kdst + tile_bytes;
      for (int idx = tid; idx < B * CPR; idx += kAttendThreads) {
        const int row = idx / CPR, ch = idx % CPR;
        const uint32_t off = row * ROWB + ((ch ^ (row & 7)) << 4);
        const int sz = row < n_tok[j] ? 16 : 0;
        cp_async16(kdst + off, ksrc + (size_t)row * D + ch * 8, sz);
        cp_async16(vdst + off, vsrc + (size_t)row * D + ch * 8, sz);
      }
      if (tid < B / 4) cp_async16(smem_u32(lse_base + (size_t)j * B * 4) + tid * 16, p.tok_lse + tile * B + tid * 4, 16);
    }
    cp_async_commit();
  }

  SPLA_MARK(p, u, 32 + item, 1);
  // ---- per-warp running state over its slices -----------------------------------------------------------
  float m_run = -INFINITY, l_run = 0.f;      // row g of the exact branch (l: this lane's share)
  float o[NT][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
  const float sc2 = p.sm_scale * kLog2e;
  const float a2 = p.phi_scale * kLog2e;
  const int spb = B / 16;                    // slices per block
  const int mi = lane >> 3, r8 = lane & 7;   // ldmatrix: which 8x8 matrix this lane addresses, and which row

#pragma unroll 1
  for (int j = 0; j < nb; ++j) {
    cp_async_wait_pending(4 - 1 - j);        // four groups were committed; block j is group j
    __syncthreads();
    if (j == 0) SPLA_MARK(p, u, 32 + item, 2);
    const uint32_t ks = smem_u32(smem_raw + (size_t)j * 2 * tile_bytes);
    const uint32_t vs = ks + tile_bytes;
    const float* lse_s = reinterpret_cast<const float*>(lse_base + (size_t)j * B * 4);
    const int ntok = n_tok[j];
#pragma unroll 1
    for (int sl = warp; sl < spb; sl += NWARP) {
      const int tok0 = sl * 16;
      if (tok0 >= ntok) break;
      const float lse2_0 = lse_s[tok0 + g] * kLog2e, lse2_1 = lse_s[tok0 + 8 + g] * kLog2e;
      float sacc[2][4];
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) { sacc[nt][0] = sacc[nt][1] = sacc[nt][2] = sacc[nt][3] = 0.f; }
      const uint32_t krow = ks + (tok0 + (mi >> 1) * 8 + r8) * ROWB;
#pragma unroll
      for (int kk = 0; kk < KS; ++kk) {
        uint32_t kb[4];
        ldmatrix_x4(kb, krow + (((2 * kk + (mi & 1)) ^ r8) << 4));
        mma_bf16(sacc[0], qa[kk][0], 0u, qa[kk][1], 0u, kb[0], kb[1]);
        mma_bf16(sacc[1], qa[kk][0], 0u, qa[kk][1], 0u, kb[2], kb[3]);
        uint32_t pb[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float ls = i < 2 ? lse2_0 : lse2_1;
          pb[i] = pack_f16(ex2(fmaf(bf16_lo(kb[i]), a2, -ls)), ex2(fmaf(bf16_hi(kb[i]), a2, -ls)));
        }
        mma_f16(sacc[0], 0u, fa[kk][0], 0u, fa[kk][1], pb[0], pb[1]);
        mma_f16(sacc[1], 0u, fa[kk][0], 0u, fa[kk][1], pb[2], pb[3]);
      }
      // online softmax on rows 0..7; rows 8..15 stay linear.  Tokens past the end of the sequence are masked.
      float mx = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const bool valid = tok0 + nt * 8 + 2 * t + c < ntok;
          sacc[nt][c] = valid ? sacc[nt][c] * sc2 : -INFINITY;
          sacc[nt][2 + c] = valid ? sacc[nt][2 + c] : 0.f;
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
      // into a bf16 head and a bf16 remainder so that o_tilde keeps ~16 bits of them.
      const uint32_t pa0 = pack_bf16(sacc[0][0], sacc[0][1]), pa1 = pack_bf16(sacc[0][2], sacc[0][3]);
      const uint32_t pa2 = pack_bf16(sacc[1][0], sacc[1][1]), pa3 = pack_bf16(sacc[1][2], sacc[1][3]);
      const uint32_t ra1 = pack_bf16(sacc[0][2] - bf16_lo(pa1), sacc[0][3] - bf16_hi(pa1));
      const uint32_t ra3 = pack_bf16(sacc[1][2] - bf16_lo(pa3), sacc[1][3] - bf16_hi(pa3));
      const uint32_t vrow = vs + (tok0 + (mi & 1) * 8 + r8) * ROWB;
#pragma unroll
      for (int np = 0; np < NT / 2; ++np) {
        uint32_t vb[4];
        ldmatrix_x4_trans(vb, vrow + (((2 * np + (mi >> 1)) ^ r8) << 4));
        o[2 * np][0] *= corr; o[2 * np][1] *= corr;
        o[2 * np + 1][0] *= corr; o[2 * np + 1][1] *= corr;
        mma_bf16(o[2 * np], pa0, pa1, pa2, pa3, vb[0], vb[1]);
        mma_bf16(o[2 * np + 1], pa0, pa1, pa2, pa3, vb[2], vb[3]);
        if (rla) {
          mma_bf16(o[2 * np], 0u, ra1, 0u, ra3, vb[0], vb[1]);
          mma_bf16(o[2 * np + 1], 0u, ra1, 0u, ra3, vb[2], vb[3]);
        }
      }
    }
  }
  cp_async_wait_pending(0);

  SPLA_MARK(p, u, 32 + item, 3);
  // ---- fold the four warps together ------------------------------------------------------------------------
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 1);
  l_run += __shfl_xor_sync(0xffffffffu, l_run, 2);
  __syncthreads();                                   // the tiles are dead: their space becomes the reduction buffer
  float* red_o = reinterpret_cast<float*>(smem_raw);                    // [NWARP][16][D + kPad]
  float* red_m = red_o + NWARP * 16 * (D + kPad);                       // [NWARP][8]
  float* red_l = red_m + NWARP * 8;                                     // [NWARP][8]
  if (t == 0) red_m[warp * 8 + g] = m_run;
  __syncthreads();
  float M = red_m[g];
#pragma unroll
  for (int w = 1; w < NWARP; ++w) M = fmaxf(M, red_m[w * 8 + g]);
  const float f = ex2(m_run - M);                    // 0 for a warp that saw no token
  if (t == 0) red_l[warp * 8 + g] = l_run * f;
  {
    float* ro = red_o + (size_t)warp * 16 * (D + kPad);
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      *reinterpret_cast<float2*>(ro + (size_t)g * (D + kPad) + nt * 8 + 2 * t) = make_float2(o[nt][0] * f, o[nt][1] * f);
      *reinterpret_cast<float2*>(ro + (size_t)(g + 8) * (D + kPad) + nt * 8 + 2 * t) = make_float2(o[nt][2], o[nt][3]);
    }
  }
  __syncthreads();
  float* part = p.att_acc + ((size_t)u * p.top_k + item) * 2 * G * D;
  for (int idx = tid; idx < 2 * G * D; idx += kAttendThreads) {
    const int row = idx / D, col = idx % D;            // row < G: exact branch of head row; else linear branch
    const int rr = row < G ? row : 8 + (row - G);
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) s += red_o[((size_t)w * 16 + rr) * (D + kPad) + col];
    part[idx] = s;
  }
  if (tid < G) {
    float Mg = red_m[tid], Lg = 0.f;
#pragma unroll
    for (int w = 1; w < NWARP; ++w) Mg = fmaxf(Mg, red_m[w * 8 + tid]);
#pragma unroll
    for (int w = 0; w < NWARP; ++w) Lg += red_l[w * 8 + tid];
    float* ml = p.att_ml + (((size_t)u * p.top_k + item) * G + tid) * 2;
    ml[0] = Mg;
    ml[1] = Lg;
  }

  SPLA_MARK(p, u, 32 + item, 4);
  if (!arrive_last(&p.attend_ticket[u], n_items, &flag_s)) return;
  SPLA_MARK(p, u, 32 + item, 5);
  merge_unit<D>(p, u, n_items, rms_weight, out, dbg_sparse, dbg_rla, reinterpret_cast<float*>(smem_raw));
  SPLA_MARK(p, u, 32 + item, 6);
}

template <int D>
static cudaError_t launch_mma(const Params& p, const void* q, const float* w, float* out, float* ds, float* dr,
                              cudaStream_t stream) {
  const size_t tiles = (size_t)p.bpc * (2 * (size_t)p.B * D * 2 + (size_t)p.B * 4);
  const size_t red = (size_t)(kAttendThreads / 32) * (16 * (D + kPad) + 16) * sizeof(float);
  size_t smem = tiles > red ? tiles : red;
  const size_t merge = (size_t)kMaxTopK * kMaxGroup * sizeof(float);
  if (merge > smem) smem = merge;
  auto kern = attend_mma_kernel<D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((p.top_k + p.bpc - 1) / p.bpc, p.batch * p.Hkv);
  return launch_ex(kern, grid, dim3(kAttendThreads), smem, stream, 0, true, p, reinterpret_cast<const __nv_bfloat16*>(q), w, out,
                   ds, dr);
}

cudaError_t launch_attend_mma(const Params& p, const void* q, const float* rms_weight, float* out, float* dbg_o_sparse,
                              float* dbg_o_rla, cudaStream_t stream) {
  return p.d == 128 ? launch_mma<128>(p, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream)
                    : launch_mma<64>(p, q, rms_weight, out, dbg_o_sparse, dbg_o_rla, stream);
}

}  // namespace spla
