// Block score + selection kernel, with the o_bar = phi(q) S_bar partials riding along as extra CTAs.
//
// Score (Section 3.1 of the paper): for query head m of the group and block i with n_i tokens,
//   ell^m_i = ln n_i + q_hat^m . mean_i + ln(1 + 1/2 sum_c (q_hat^m_c)^2 var_i[c])
// is the log of the second-order Taylor estimate of the block's attention mass; per head the masses are
// normalised over all blocks and the G heads are summed (Section 2.2).  One warp consumes one 2d-float
// statistics record with a single 128-bit load per lane for the mean and one for the variance; a CTA streams
// `chunk` consecutive records, 32 at a time, with the next 32 already in flight (register double buffer), and
// the grid is sized to about one resident wave so that the per-CTA fixed cost is paid once.
//
// Selection (Section 2.1 Select; Section 4 forced sink/local blocks): the last CTA of a unit to finish
// (atomic ticket, no waiting) reduces the per-chunk normalisers, forms the aggregated score, and picks the
// top-k by an 8-bit radix select on the score bits followed by an index-ordered compaction.
#include "spla_internal.h"
#include "state_role.cuh"

namespace spla {

namespace {

constexpr int UNR = 4;                                  // records per warp per round
constexpr int kRound = (kScoreThreads / 32) * UNR;      // records per CTA per round (32)

// One statistics record (mean, then variance; fp32 or bfloat16 elements) spread over a warp, VEC channels per lane.
template <int VEC>
__device__ __forceinline__ void load_record(const float* stats, size_t rec_elem, bool rec_bf16, int D, int lane, bool valid,
                                            float (&mean)[VEC], float (&var)[VEC]) {
  if (valid && rec_bf16) {
    const __nv_bfloat16* rec = reinterpret_cast<const __nv_bfloat16*>(stats) + rec_elem;
    load_vec<VEC>(rec + lane * VEC, mean);
    load_vec<VEC>(rec + D + lane * VEC, var);
  } else if (valid) {
    const float* rec = stats + rec_elem;
    if constexpr (VEC == 4) {
      const float4 a = __ldcs(reinterpret_cast<const float4*>(rec + lane * 4));
      const float4 b = __ldcs(reinterpret_cast<const float4*>(rec + D + lane * 4));
      mean[0] = a.x; mean[1] = a.y; mean[2] = a.z; mean[3] = a.w;
      var[0] = b.x; var[1] = b.y; var[2] = b.z; var[3] = b.w;
    } else {
      const float2 a = __ldcs(reinterpret_cast<const float2*>(rec + lane * 2));
      const float2 b = __ldcs(reinterpret_cast<const float2*>(rec + D + lane * 2));
      mean[0] = a.x; mean[1] = a.y;
      var[0] = b.x; var[1] = b.y;
    }
  } else {
#pragma unroll
    for (int v = 0; v < VEC; ++v) { mean[v] = 0.f; var[v] = 0.f; }
  }
}

// Merge two (max, sum-of-exp) pairs.
__device__ __forceinline__ void lse_merge(float& m, float& s, float m2, float s2) {
  const float nm = fmaxf(m, m2);
  if (nm > -INFINITY) s = s * __expf(m - nm) + s2 * __expf(m2 - nm);
  m = nm;
}

}  // namespace

template <int D, int GP>
__global__ void __launch_bounds__(kScoreThreads, GP >= 2 ? 1 : 2) score_select_kernel(const Params p, const void* __restrict__ q_raw,
                                                                        int q_is_bf16, int* __restrict__ sel_user) {
  constexpr int VEC = D / 32;
  constexpr int NV = 2 * GP;             // values reduced per record: GP mean dots, GP variance dots
  constexpr int LPV = 32 / NV > 0 ? 32 / NV : 1;  // lanes holding a copy of each reduced value
  constexpr int FB = LPV < UNR ? LPV : UNR;       // records finalised together, one per copy lane
  constexpr int NWARP = kScoreThreads / 32;
  extern __shared__ __align__(16) unsigned char smem_raw[];

  const int vu = blockIdx.y;                        // index into the workspace arrays (a virtual unit in a prefill launch)
  const UnitRef ur = unit_ref(p, vu);
  const int u = ur.u;                               // the cache's unit: statistics, K/V, state
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int G = p.G;
  const int c = blockIdx.x;

  // ------------------------------------------------------------------ o_bar role ----------------------
  if (c >= p.n_chunks_cap) {
    state_role<D, GP, kScoreThreads>(p, u, c - p.n_chunks_cap, q_raw, q_is_bf16, reinterpret_cast<float*>(smem_raw), (int)threadIdx.x, 0);
    return;
  }

  // ------------------------------------------------------------------ score role ----------------------
  const int NW = p.NW;                              // selection windows per block; a "record" is one window
  const int L = cover_len(p, ur.L, (long long)p.n_chunks_cap * p.chunk / NW * p.B);
  const int nblk = (L + p.B - 1) / p.B;
  const int nrec = nblk * NW;
  const int chunk = p.chunk;                        // records per CTA
  const int n_chunks = max(1, (nrec + chunk - 1) / chunk);
  if (c >= n_chunks) return;

  // q_hat slices for the mean dot and 1/2 q_hat^2 for the variance dot, in registers.
  float qm[GP][VEC], qv[GP][VEC];
#pragma unroll
  for (int g = 0; g < GP; ++g) {
    if (g < G) {
      float x[VEC];
      const size_t qoff = (ur.qrow + g) * D + lane * VEC;
      if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
      else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
#pragma unroll
      for (int v = 0; v < VEC; ++v) {
        qm[g][v] = x[v] * p.sm_scale;
        qv[g][v] = (p.flags & 2u) ? 0.f : 0.5f * qm[g][v] * qm[g][v];
      }
    } else {
#pragma unroll
      for (int v = 0; v < VEC; ++v) { qm[g][v] = 0.f; qv[g][v] = 0.f; }
    }
  }

  const size_t ell_stride = (size_t)p.max_blocks * NW;
  const size_t stats_u = (size_t)u * ell_stride * 2 * D;      // first element of the unit's records
  const bool rec_bf16 = (p.flags & kStatsBf16) != 0;
  float* ell_u = p.ell + (size_t)vu * G * ell_stride;
  // prefill: a position's own (last) block holds fewer tokens than the cache's record of it describes: its
  // statistics as of that position come from the per-position table (whole-block statistics only)
  const float* own_rec = ur.t >= 0 ? p.vstats + ((size_t)u * p.vTtot + ur.t) * 2 * D : nullptr;
  // After the warp reduction lanes 0..15 hold the mean dots and lanes 16..31 the variance dots, value index
  // lane / LPV, each replicated on LPV lanes.  Copy lane `sub` finalises record `sub` of the batch, so the
  // log / exp work of FB records runs side by side instead of one record at a time.
  const int my_g = (lane & 15) / LPV;
  const int sub = lane % LPV;
  const bool fin_lane = lane < 16 && sub < FB && my_g < G;
  const float ln_full = logf((float)p.B);
  const int n_last = L - (nblk - 1) * p.B;          // tokens of the last block
  const float ln_last = logf((float)max(1, n_last));
  const float ln_win = logf((float)p.win_C);
  float run_max = -INFINITY, run_sum = 0.f;

  const int rounds = chunk / kRound;
  const int base = c * chunk + warp * UNR;                 // record of (round 0, r = 0) for this warp

  float mean[2][UNR][VEC], var[2][UNR][VEC];
  auto load_round = [&](int round, int buf) {
#pragma unroll
    for (int r = 0; r < UNR; ++r) {
      const int i = base + round * kRound + r;
      bool valid = i < nrec;
      if ((p.flags & kDebugBounds) && valid && i >= p.max_blocks * NW) {   // checked build: the record must exist
        atomicExch(p.status, kStatusBounds);
        valid = false;
      }
      if (own_rec && i == nblk - 1) load_record<VEC>(own_rec, 0, false, D, lane, valid, mean[buf][r], var[buf][r]);
      else load_record<VEC>(p.stats, stats_u + (size_t)i * 2 * D, rec_bf16, D, lane, valid, mean[buf][r], var[buf][r]);
    }
  };
  auto compute_round = [&](int round, int buf) {
    const int i0 = base + round * kRound;
    if (i0 >= nrec) return;                                // warp-uniform
#pragma unroll
    for (int r0 = 0; r0 < UNR; r0 += FB) {
      float dm_keep = 0.f, dv_keep = 0.f;
#pragma unroll
      for (int rr = 0; rr < FB; ++rr) {
        const int r = r0 + rr;
        float vals[NV];
#pragma unroll
        for (int g = 0; g < GP; ++g) {
          float dm = 0.f, dv = 0.f;
#pragma unroll
          for (int v = 0; v < VEC; ++v) {
            dm = fmaf(qm[g][v], mean[buf][r][v], dm);
            dv = fmaf(qv[g][v], var[buf][r][v], dv);
          }
          vals[g] = dm;
          vals[GP + g] = dv;
        }
        warp_reduce_multi<NV>(vals, lane);
        const float other = __shfl_xor_sync(0xffffffffu, vals[0], 16);   // variance dot of the same head
        if (sub == rr) { dm_keep = vals[0]; dv_keep = other; }
      }
      const int i = i0 + r0 + sub;
      if (fin_lane && i < nrec) {
        if (NW == 1) {
          const float ell = (i == nblk - 1 ? ln_last : ln_full) + dm_keep + __logf(1.f + dv_keep);
          ell_u[(size_t)my_g * ell_stride + i] = ell;
          const float nm = fmaxf(run_max, ell);
          run_sum = run_sum * __expf(run_max - nm) + __expf(ell - nm);
          run_max = nm;
        } else {
          // strided windows (Section 3.1, "Strided Block Selection"): the log mass of window w of block blk; the
          // pooling over a block's windows and the normalisers are left to the selecting CTA
          const int blk = i / NW, w = i - blk * NW;
          float ln_n = ln_win;
          if (blk == nblk - 1) {
            const int cnt = min(p.win_C, n_last - w * p.win_s);
            ln_n = cnt > 0 ? logf((float)cnt) : -INFINITY;
          }
          ell_u[(size_t)my_g * ell_stride + i] = ln_n + dm_keep + __logf(1.f + dv_keep);
        }
      }
    }
  };

  load_round(0, 0);
#pragma unroll 1
  for (int round = 0; round < rounds; round += 2) {
    if (round + 1 < rounds) load_round(round + 1, 1);
    compute_round(round, 0);
    if (round + 1 < rounds) {
      if (round + 2 < rounds) load_round(round + 2, 0);
      compute_round(round + 1, 1);
    }
  }

  // per-chunk (max, sum exp) per head: fold the FB finalising lanes, then the warps
#pragma unroll
  for (int o = 1; o < FB; o <<= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, run_max, o), s2 = __shfl_xor_sync(0xffffffffu, run_sum, o);
    lse_merge(run_max, run_sum, m2, s2);
  }
  float* wred = reinterpret_cast<float*>(smem_raw);     // [NWARP][GP][2]
  __shared__ int is_last_s;
  if (fin_lane && sub == 0) {
    wred[(warp * GP + my_g) * 2 + 0] = run_max;
    wred[(warp * GP + my_g) * 2 + 1] = run_sum;
  }
  __syncthreads();
  if (tid < G) {
    float m = -INFINITY, s = 0.f;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) lse_merge(m, s, wred[(w * GP + tid) * 2], wred[(w * GP + tid) * 2 + 1]);
    float* cp = p.chunk_part + (((size_t)vu * p.max_chunks + c) * G + tid) * 2;
    cp[0] = m;
    cp[1] = s;
  }
  __syncthreads();                                       // every thread's stores precede thread 0's fence
  if (tid == 0) {
    __threadfence();
    const int t = atomicAdd(&p.score_ticket[vu], 1);
    is_last_s = (t == n_chunks - 1);
    if (is_last_s) p.score_ticket[vu] = 0;               // ready for the next decode step
    __threadfence();
  }
  __syncthreads();
  if (!is_last_s) return;

  // ------------------------------------------------------------------ selection (one CTA per unit) ----
  uint32_t* keys = reinterpret_cast<uint32_t*>(smem_raw);           // [max_blocks]
  __shared__ float lse_s[kMaxGroup];
  __shared__ int hist[256];
  __shared__ int wtot[2][NWARP];
  __shared__ uint32_t sel_digit_s;
  __shared__ int sel_k_s;

  // The first batch of log masses is requested before the normalisers are reduced: the two do not depend on
  // each other and each is one L2 round trip.
  constexpr int SB = 4;                                             // blocks per thread with loads in flight together
  float e[SB][GP];
  auto load_batch = [&](int i0) {
#pragma unroll
    for (int j = 0; j < SB; ++j) {
      const int i = i0 + j * kScoreThreads + tid;
#pragma unroll
      for (int g = 0; g < GP; ++g) {
        float x = -INFINITY;
        if (g < G && i < nblk)
          for (int w = 0; w < NW; ++w) x = fmaxf(x, __ldcg(ell_u + (size_t)g * ell_stride + (size_t)i * NW + w));   // max-pool
        e[j][g] = x;
      }
    }
  };
  load_batch(0);

  if (NW > 1) {
    // windows: the normalisers are those of the pooled log masses, which only exist here
    float* wred2 = reinterpret_cast<float*>(smem_raw);                // [NWARP][GP][2]; the keys are written later
    float m[GP], sm[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) { m[g] = -INFINITY; sm[g] = 0.f; }
    for (int i0 = 0; i0 < nblk; i0 += kScoreThreads * SB) {
      if (i0 > 0) load_batch(i0);
#pragma unroll
      for (int j = 0; j < SB; ++j)
#pragma unroll
        for (int g = 0; g < GP; ++g) lse_merge(m[g], sm[g], e[j][g], e[j][g] > -INFINITY ? 1.f : 0.f);
    }
#pragma unroll
    for (int g = 0; g < GP; ++g) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m[g], o), s2 = __shfl_xor_sync(0xffffffffu, sm[g], o);
        lse_merge(m[g], sm[g], m2, s2);
      }
      if (lane == 0) { wred2[(warp * GP + g) * 2] = m[g]; wred2[(warp * GP + g) * 2 + 1] = sm[g]; }
    }
    __syncthreads();
    if (tid < G) {
      float mm = -INFINITY, ss = 0.f;
#pragma unroll
      for (int w = 0; w < NWARP; ++w) lse_merge(mm, ss, wred2[(w * GP + tid) * 2], wred2[(w * GP + tid) * 2 + 1]);
      lse_s[tid] = mm + __logf(ss);
    }
    __syncthreads();
    load_batch(0);
  }
  for (int g = warp; g < G && NW == 1; g += NWARP) {
    float m = -INFINITY, s = 0.f;
#pragma unroll 4
    for (int cc = lane; cc < n_chunks; cc += 32) {
      const float2 ms = __ldcg(reinterpret_cast<const float2*>(p.chunk_part + (((size_t)vu * p.max_chunks + cc) * G + g) * 2));
      lse_merge(m, s, ms.x, ms.y);
    }
    const float M = warp_max(m);
    s = (m > -INFINITY) ? s * __expf(m - M) : 0.f;
    s = warp_sum(s);
    if (lane == 0) lse_s[g] = M + __logf(s);
  }
  __syncthreads();

  const int k_eff = min(p.top_k, nblk);
  float* scores_u = p.scores + (size_t)vu * p.max_blocks;
  float lse_r[GP];
#pragma unroll
  for (int g = 0; g < GP; ++g) lse_r[g] = g < G ? lse_s[g] : 0.f;
  for (int i0 = 0; i0 < nblk; i0 += kScoreThreads * SB) {
    if (i0 > 0) load_batch(i0);
#pragma unroll
    for (int j = 0; j < SB; ++j) {
      const int i = i0 + j * kScoreThreads + tid;
      if (i < nblk) {
        float sc = 0.f;
#pragma unroll
        for (int g = 0; g < GP; ++g)
          if (g < G) sc += __expf(e[j][g] - lse_r[g]);
        scores_u[i] = sc;
        const bool forced = (i < p.n_sink) || (i >= nblk - p.n_local);
        keys[i] = forced ? 0xffffffffu : __float_as_uint(sc);
      }
    }
  }
  __syncthreads();

  // radix select: the k_eff-th largest key, 8 bits per pass.  A warp whose active lanes all hold the same
  // digit (the rule in the exponent pass) adds its count once; otherwise each lane adds for itself.
  uint32_t prefix = 0, mask = 0;
  int kk = k_eff;
  if (k_eff > 0) {
#pragma unroll 1
    for (int shift = 24; shift >= 0; shift -= 8) {
      hist[tid] = 0;                                                   // kScoreThreads == 256 bins
      __syncthreads();
#pragma unroll 4
      for (int i0 = 0; i0 < nblk; i0 += kScoreThreads) {
        const int i = i0 + tid;
        const uint32_t key = i < nblk ? keys[i] : 0u;
        const bool in = i < nblk && (key & mask) == prefix;
        const unsigned act = __ballot_sync(0xffffffffu, in);
        if (act) {
          const uint32_t digit = (key >> shift) & 255u;
          const uint32_t first = __shfl_sync(0xffffffffu, digit, __ffs(act) - 1);
          const unsigned same = __ballot_sync(0xffffffffu, in && digit == first);
          if (same == act) {
            if (lane == __ffs(act) - 1) atomicAdd(&hist[first], __popc(act));
          } else if (in) {
            atomicAdd(&hist[digit], 1);
          }
        }
      }
      __syncthreads();
      if (warp == 0) {
        int bins[8], tot = 0;
#pragma unroll
        for (int j = 0; j < 8; ++j) { bins[j] = hist[lane * 8 + j]; tot += bins[j]; }
        int above = tot;                                               // inclusive suffix sum over lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int t = __shfl_down_sync(0xffffffffu, above, o);
          if (lane + o < 32) above += t;
        }
        above -= tot;                                                  // keys in bins of higher lanes
        if (above < kk && kk <= above + tot) {
          int cum = above;
#pragma unroll
          for (int j = 7; j >= 0; --j) {
            if (cum < kk && kk <= cum + bins[j]) { sel_digit_s = lane * 8 + j; sel_k_s = kk - cum; }
            cum += bins[j];
          }
        }
      }
      __syncthreads();
      prefix |= sel_digit_s << shift;
      mask |= 0xffu << shift;
      kk = sel_k_s;
    }
  }
  const uint32_t T = prefix;   // threshold key; kk = how many keys equal to T are taken (lowest indices first)

  // index-ordered compaction
  const int per = (nblk + kScoreThreads - 1) / kScoreThreads;
  const int i0 = tid * per, i1 = min(nblk, i0 + per);
  int n_gt = 0, n_eq = 0;
  for (int i = i0; i < i1; ++i) {
    const uint32_t key = keys[i];
    n_gt += key > T;
    n_eq += key == T;
  }
  int s_gt = n_gt, s_eq = n_eq;                                        // inclusive scans within the warp
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int a = __shfl_up_sync(0xffffffffu, s_gt, o), e = __shfl_up_sync(0xffffffffu, s_eq, o);
    if (lane >= o) { s_gt += a; s_eq += e; }
  }
  if (lane == 31) { wtot[0][warp] = s_gt; wtot[1][warp] = s_eq; }
  __syncthreads();
  int gt_before = s_gt - n_gt, eq_before = s_eq - n_eq;
  for (int w = 0; w < warp; ++w) { gt_before += wtot[0][w]; eq_before += wtot[1][w]; }
  int* sel_u = p.sel + (size_t)vu * p.top_k;
  int* sel_o = sel_user ? sel_user + (ur.qrow / G) * p.top_k : nullptr;   // [batch][H_kv][k], or [batch][T][H_kv][k]
  if (k_eff > 0 && n_gt + n_eq > 0) {
    for (int i = i0; i < i1; ++i) {
      const uint32_t key = keys[i];
      const bool take = key > T || (key == T && eq_before < kk);
      if (take) {
        const int slot = gt_before + min(eq_before, kk);
        sel_u[slot] = i;
        if (sel_o) sel_o[slot] = i;
      }
      gt_before += key > T;
      eq_before += key == T;
    }
  }
  for (int t = k_eff + tid; t < p.top_k; t += kScoreThreads) {
    sel_u[t] = -1;
    if (sel_o) sel_o[t] = -1;
  }
  if (tid == 0) p.n_sel[vu] = k_eff;
}

template <int D, int GP>
static cudaError_t launch_one(const Params& p, const void* q, int q_is_bf16, int* sel_user, cudaStream_t stream) {
  const int U = p.batch * p.Hkv * (p.vT > 0 ? p.vT : 1);
  const bool rla = !(p.flags & 4u) && p.vT == 0;          // (a prefill launch gets o_bar from the chunk scan instead)
  dim3 grid(p.n_chunks_cap + (rla ? kStateSplits : 0), U);
  size_t smem = (size_t)p.max_blocks * sizeof(uint32_t);
  const size_t smem_state = (size_t)(GP * D + (kScoreThreads / D) * GP * D) * sizeof(float);
  if (smem_state > smem) smem = smem_state;
  const size_t smem_wred = (size_t)(kScoreThreads / 32) * GP * 2 * sizeof(float);
  if (smem_wred > smem) smem = smem_wred;
  auto kern = score_select_kernel<D, GP>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<grid, kScoreThreads, smem, stream>>>(p, q, q_is_bf16, sel_user);
  ++g_launch_count;
  return cudaGetLastError();
}

template <int D>
static cudaError_t launch_d(const Params& p, int GP, const void* q, int qb, int* sel_user, cudaStream_t s) {
  switch (GP) {
    case 1: return launch_one<D, 1>(p, q, qb, sel_user, s);
    case 2: return launch_one<D, 2>(p, q, qb, sel_user, s);
    case 4: return launch_one<D, 4>(p, q, qb, sel_user, s);
    case 8: return launch_one<D, 8>(p, q, qb, sel_user, s);
    default: return launch_one<D, 16>(p, q, qb, sel_user, s);
  }
}

int score_chunk_for(long long units, long long max_seq_blocks, int sm_count) {
  // Smallest chunk (a multiple of the 32 records a CTA consumes per round) for which all score CTAs are
  // resident at once (two CTAs per SM); long ragged batches simply take several waves of the largest chunk.
  int chunk = kScoreChunkMin;
  while (chunk < kScoreChunkMax && units * ((max_seq_blocks + chunk - 1) / chunk) > 2LL * sm_count) chunk *= 2;
  return chunk;
}

cudaError_t launch_score_select(const Params& p, const void* q, int q_is_bf16, int* sel_user, cudaStream_t stream) {
  const int GP = padded_group(p.G);
  return p.d == 128 ? launch_d<128>(p, GP, q, q_is_bf16, sel_user, stream)
                    : launch_d<64>(p, GP, q, q_is_bf16, sel_user, stream);
}

}  // namespace spla
