// o_bar = phi(q) S_bar for one slice of the state's rows (Section 3.2 of the paper, Eq. rla-impl-1): the part of
// the residual branch that needs neither the selection nor any K/V tile.  Run by spare CTAs of the score kernels.
#pragma once

#include "spla_device.cuh"

namespace spla {

// NT threads take part.  bar_id 0: they are the first NT threads of the CTA, whose other threads only join the
// barriers.  Otherwise they are NT consecutive threads (whole warps) with local numbers `tid` = 0 .. NT - 1 that meet
// on the named barrier `bar_id`, and the rest of the CTA is elsewhere.
// smem: (GP * D + (NT / D) * GP * D) floats.
template <int D, int GP, int NT>
__device__ __forceinline__ void state_role(const Params& p, int u, int s, const void* __restrict__ q_raw, int q_is_bf16,
                                           float* smem, const int tid, const int bar_id) {
  auto meet = [&]() {
    if (bar_id == 0) __syncthreads();
    else asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory");
  };
  const int stride = bar_id == 0 ? (int)blockDim.x : NT;
  constexpr int VEC = D / 32;
  constexpr int RG = NT / D;                             // row groups working side by side
  constexpr int ROWS = D / kStateSplits / RG;            // rows per thread
  const int lane = tid & 31, warp = tid >> 5;
  const int b = u / p.Hkv, h = u % p.Hkv, G = p.G;
  const bool act = tid < NT;
  float* phiq = smem;                                    // [GP][D]
  float* red = phiq + GP * D;                            // [RG][GP][D]
  const float a2 = p.phi_scale * kLog2e;
  const int rg = tid / D, j = tid % D;
  const float* S = p.state + (size_t)u * D * D + (size_t)(s * (D / kStateSplits) + rg) * D + j;
  constexpr int RB = ROWS > 16 ? 16 : ROWS;              // rows in flight per thread (bounds the registers)
  float sv[RB];
#pragma unroll
  for (int r = 0; r < RB; ++r) sv[r] = act ? __ldcs(S + (size_t)r * RG * D) : 0.f;   // in flight while phi(q) is formed
  for (int g = warp; g < G; g += NT / 32) {
    float x[VEC];
    const size_t qoff = ((size_t)b * p.Hq + (size_t)h * G + g) * D + lane * VEC;
    if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
    else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
    float mx = -INFINITY;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { x[v] *= a2; mx = fmaxf(mx, x[v]); }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { x[v] = exp2f(x[v] - mx); sum += x[v]; }
    sum = warp_sum(sum);
    const float inv = 1.f / sum;
#pragma unroll
    for (int v = 0; v < VEC; ++v) phiq[g * D + lane * VEC + v] = x[v] * inv;
  }
  meet();
  if (act) {
    float acc[GP];
#pragma unroll
    for (int g = 0; g < GP; ++g) acc[g] = 0.f;
#pragma unroll
    for (int r0 = 0; r0 < ROWS; r0 += RB) {
      if (r0 > 0) {
#pragma unroll
        for (int r = 0; r < RB; ++r) sv[r] = __ldcs(S + (size_t)(r0 + r) * RG * D);
      }
#pragma unroll
      for (int r = 0; r < RB; ++r) {
        const int row = s * (D / kStateSplits) + rg + (r0 + r) * RG;
#pragma unroll
        for (int g = 0; g < GP; ++g)
          if (g < G) acc[g] = fmaf(phiq[g * D + row], sv[r], acc[g]);
      }
    }
#pragma unroll
    for (int g = 0; g < GP; ++g) red[(rg * GP + g) * D + j] = acc[g];
  }
  meet();
  for (int idx = tid; idx < G * D; idx += stride) {
    const int g = idx / D, jj = idx % D;
    float t = 0.f;
#pragma unroll
    for (int r2 = 0; r2 < RG; ++r2) t += red[(r2 * GP + g) * D + jj];
    p.obar_part[(((size_t)u * kStateSplits + s) * G + g) * D + jj] = t;
  }
}

// o_bar of ONE query head over all rows of the state, left in shared memory (`obar`, D floats): the fused decode
// kernel's form, where the CTA that merges a head computes that head's o_bar itself, so that it neither travels nor has
// to be made visible to another CTA.  NT threads with local numbers `tid` meet on the named barrier `bar_id`.
// smem: (D + (NT / D) * D) floats.
template <int D, int NT>
__device__ __forceinline__ void state_head(const Params& p, int u, int head, const void* __restrict__ q_raw, int q_is_bf16,
                                           float* __restrict__ obar, float* smem, const int tid, const int bar_id) {
  auto meet = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(bar_id), "n"(NT) : "memory"); };
  constexpr int VEC = D / 32;
  constexpr int RG = NT / D;                             // row groups working side by side
  constexpr int ROWS = D / RG;                           // rows per thread
  constexpr int RB = ROWS < 32 ? ROWS : 32;              // rows in flight per thread (the role is latency-bound: few, deep batches)
  const int lane = tid & 31, warp = tid >> 5;
  const int b = u / p.Hkv, h = u % p.Hkv;
  float* phiq = smem;                                    // [D]
  float* red = phiq + D;                                 // [RG][D]
  const int rg = tid / D, j = tid % D;
  const float* S = p.state + (size_t)u * D * D + (size_t)rg * D + j;
  float sv[RB];
#pragma unroll
  for (int r = 0; r < RB; ++r) sv[r] = __ldcs(S + (size_t)r * RG * D);       // in flight while phi(q) is formed
  if (warp == 0) {
    const float a2 = p.phi_scale * kLog2e;
    float x[VEC];
    const size_t qoff = ((size_t)b * p.Hq + (size_t)h * p.G + head) * D + lane * VEC;
    if (q_is_bf16) load_vec<VEC>(reinterpret_cast<const __nv_bfloat16*>(q_raw) + qoff, x);
    else load_vec<VEC>(reinterpret_cast<const float*>(q_raw) + qoff, x);
    float mx = -INFINITY;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { x[v] *= a2; mx = fmaxf(mx, x[v]); }
    mx = warp_max(mx);
    float sum = 0.f;
#pragma unroll
    for (int v = 0; v < VEC; ++v) { x[v] = exp2f(x[v] - mx); sum += x[v]; }
    sum = warp_sum(sum);
    const float inv = 1.f / sum;
#pragma unroll
    for (int v = 0; v < VEC; ++v) phiq[lane * VEC + v] = x[v] * inv;
  }
  meet();
  float acc = 0.f;
#pragma unroll 1
  for (int r0 = 0; r0 < ROWS; r0 += RB) {
    if (r0 > 0) {
#pragma unroll
      for (int r = 0; r < RB; ++r) sv[r] = __ldcs(S + (size_t)(r0 + r) * RG * D);
    }
#pragma unroll
    for (int r = 0; r < RB; ++r) acc = fmaf(phiq[rg + (r0 + r) * RG], sv[r], acc);
  }
  red[rg * D + j] = acc;
  meet();
  if (tid < D) {
    float t = 0.f;
#pragma unroll
    for (int r2 = 0; r2 < RG; ++r2) t += red[r2 * D + tid];
    obar[tid] = t;
  }
  meet();                                                // (the scratch may be reused)
}

}  // namespace spla
