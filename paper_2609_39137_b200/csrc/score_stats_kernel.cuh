// Statistics of the router's score distribution over a dumped logit matrix:
//   * full-pool selection-score entropy H = -sum_e p_e ln p_e per token
//     (Section 4.3), for both score families the paper evaluates:
//       biased sigmoid  p_e = max(sigmoid(z_e) + b_e, 0) / sum (clamped, normalised)
//       softmax         p_e = softmax_e(z)
//     reported as the mean over the tokens of a layer;
//   * the forward statistics of the auxiliary balancing loss (Eq. 8):
//     P_i = mean over tokens of softmax_i(z), f_i = n_i / T, aux = sum_i f_i P_i.
//
// One pass over the dump, HBM-bound: a warp takes one token row at a time, lane
// l holds experts l, l+32, ... in registers (coalesced 128-byte loads), the row
// sums are warp shuffles.  Per row the entropies come from
//   H = ln S - (sum_e c_e ln c_e) / S,  S = sum_e c_e
// so the softmax family needs no logarithm per element (ln c_e = z_e - max).
// Partial sums per CTA go to scratch in the workspace and are added in a fixed
// order by two small kernels, in binary64: results do not depend on timing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "route_math.cuh"

namespace moe {

constexpr int kStatThreads = 256;
constexpr int kStatWarps = kStatThreads / 32;
constexpr int kStatCtaTarget = 592;      // CTAs over all layers (4 per SM on 148 SMs)
constexpr int kStatCtaMaxPerLayer = 592;

__host__ __device__ inline int stat_ctas_per_layer(int L) {
  int c = kStatCtaTarget / (L < 1 ? 1 : L);
  if (c < 1) c = 1;
  if (c > kStatCtaMaxPerLayer) c = kStatCtaMaxPerLayer;
  return c;
}

struct StatParams {
  const float* logits;   // [L][T][E]
  const float* bias;     // [L][E]
  int L, T, E, C;        // C = CTAs per layer
  float* part_P;         // [L][C][E] partial sums of softmax probabilities
  float* part_H;         // [L][C][2] partial sums of (biased-sigmoid, softmax) entropies
  double* aux_part;      // [L][16] shares of sum_i f_i P_i per group of 64 experts
  // second kernel
  const int* loads;      // [L][E] or null
  float* h_biased;       // [L] or null
  float* h_softmax;      // [L] or null
  float* mean_prob;      // [L][E] or null
  float* aux;            // [L] or null
};

__device__ __forceinline__ float exp2f_fast(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float rcp_fast(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float lg2_fast(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, d));
  return v;
}

// NPL = experts per lane (E <= 32 * NPL).  grid = (C, L)
template <int NPL>
__global__ void __launch_bounds__(kStatThreads, 4) score_stats_kernel(StatParams p) {
  chained_launch_enter();
  // per-warp accumulators of the softmax probabilities and the layer's bias live in shared memory so that
  // a thread's registers hold little more than its NPL logits of the current row (4 CTAs per SM)
  __shared__ float sP[kStatWarps][32 * NPL];
  __shared__ float sB[32 * NPL];
  __shared__ float sH[kStatWarps][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int layer = blockIdx.y;
  const float* zl = p.logits + (size_t)layer * p.T * p.E;
  for (int e = threadIdx.x; e < 32 * NPL; e += kStatThreads) {
    sB[e] = (e < p.E) ? p.bias[(size_t)layer * p.E + e] : 0.0f;
#pragma unroll
    for (int w = 0; w < kStatWarps; ++w) sP[w][e] = 0.0f;
  }
  __syncthreads();
  float* myP = sP[warp];
  float acc_hb = 0.0f, acc_hs = 0.0f;
  for (int row = blockIdx.x * kStatWarps + warp; row < p.T; row += p.C * kStatWarps) {
    const float* zr = zl + (size_t)row * p.E;
    float z[NPL];
#pragma unroll
    for (int j = 0; j < NPL; ++j) {
      const int e = lane + 32 * j;
      z[j] = (e < p.E) ? __ldg(zr + e) : -INFINITY;
    }
    float m = z[0];
#pragma unroll
    for (int j = 1; j < NPL; ++j) m = fmaxf(m, z[j]);
    m = warp_max(m);
    float S = 0.0f, A = 0.0f, R = 0.0f, B = 0.0f;
#pragma unroll
    for (int j = 0; j < NPL; ++j) {
      const int e = lane + 32 * j;
      if (e < p.E) {
        // hardware exp2 / log2 approximations (about 2 ulp each): these are statistics with a 1e-5 relative
        // budget, not the routing decision, so the bit-exact score chain is not needed here
        const float sg = rcp_fast(1.0f + exp2f_fast(z[j] * -1.44269504f));
        const float c = fmaxf(sg + sB[e], 0.0f);
        R += c;
        B = fmaf(c, (c > 0.0f) ? lg2_fast(c) : 0.0f, B);         // sum c log2 c; scaled to nats once per row
        const float d = z[j] - m;
        const float q = exp2f_fast(d * 1.44269504f);
        S += q;
        A = fmaf(q, d, A);
        z[j] = q;
      } else {
        z[j] = 0.0f;
      }
    }
    S = warp_sum(S); A = warp_sum(A); R = warp_sum(R); B = warp_sum(B);
    acc_hs += logf(S) - A / S;                                   // once per row: full-precision logf
    acc_hb += (R > 0.0f) ? (logf(R) - (B * 0.693147181f) / R) : 0.0f;
    const float inv = 1.0f / S;
#pragma unroll
    for (int j = 0; j < NPL; ++j) myP[lane + 32 * j] = fmaf(z[j], inv, myP[lane + 32 * j]);   // only this warp touches its row of sP
  }
  if (lane == 0) { sH[warp][0] = acc_hb; sH[warp][1] = acc_hs; }
  __syncthreads();
  float* outP = p.part_P + ((size_t)layer * p.C + blockIdx.x) * p.E;
  for (int e = threadIdx.x; e < p.E; e += kStatThreads) {
    float s = 0.0f;
#pragma unroll
    for (int w = 0; w < kStatWarps; ++w) s += sP[w][e];
    outP[e] = s;
  }
  if (threadIdx.x < 2) {
    float s = 0.0f;
#pragma unroll
    for (int w = 0; w < kStatWarps; ++w) s += sH[w][threadIdx.x];
    p.part_H[((size_t)layer * p.C + blockIdx.x) * 2 + threadIdx.x] = s;
  }
}

// Second step, grid = (ceil(E / 64), L), 1024 threads = 64 experts x 16 slices of the per-CTA partial sums:
// every thread adds its slice in index order (binary64), the 16 slice sums are added in order, P_i is stored and
// the group's share of sum_i f_i P_i is reduced with a fixed tree into aux_part[layer][group].
constexpr int kStatFinExperts = 64;
constexpr int kStatFinSlices = 16;
constexpr int kStatMaxGroups = 16;   // 1024 experts / 64

__global__ void __launch_bounds__(1024) score_stats_finish_kernel(StatParams p) {
  chained_launch_enter();
  __shared__ double y[kStatFinSlices][kStatFinExperts];
  const int layer = blockIdx.y, group = blockIdx.x;
  const int el = threadIdx.x % kStatFinExperts, sl = threadIdx.x / kStatFinExperts;
  const int e = group * kStatFinExperts + el;
  double s = 0.0;
  if (e < p.E)
    for (int c = sl; c < p.C; c += kStatFinSlices) s += (double)p.part_P[((size_t)layer * p.C + c) * p.E + e];
  y[sl][el] = s;
  __syncthreads();
  if (sl == 0) {
    double tot = 0.0;
#pragma unroll
    for (int k = 0; k < kStatFinSlices; ++k) tot += y[k][el];
    const double P = tot / (double)p.T;
    double term = 0.0;
    if (e < p.E) {
      if (p.mean_prob) p.mean_prob[(size_t)layer * p.E + e] = (float)P;
      if (p.loads) term = ((double)p.loads[(size_t)layer * p.E + e] / (double)p.T) * P;
    }
    y[0][el] = term;
  }
  for (int stride = kStatFinExperts / 2; stride >= 1; stride >>= 1) {
    __syncthreads();
    if (sl == 0 && el < stride) y[0][el] = y[0][el] + y[0][el + stride];
  }
  __syncthreads();
  if (threadIdx.x == 0) p.aux_part[(size_t)layer * kStatMaxGroups + group] = y[0][0];
}

// Third step, one warp per layer: the groups' aux shares and the per-CTA entropy sums, added in index order.
__global__ void score_stats_scalar_kernel(StatParams p, int groups) {
  chained_launch_enter();
  const int layer = blockIdx.x, lane = threadIdx.x;
  double hb = 0.0, hs = 0.0;
  for (int c = lane; c < p.C; c += 32) {
    hb += (double)p.part_H[((size_t)layer * p.C + c) * 2 + 0];
    hs += (double)p.part_H[((size_t)layer * p.C + c) * 2 + 1];
  }
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    hb += __shfl_xor_sync(0xffffffffu, hb, d);
    hs += __shfl_xor_sync(0xffffffffu, hs, d);
  }
  if (lane == 0) {
    if (p.h_biased) p.h_biased[layer] = (float)(hb / (double)p.T);
    if (p.h_softmax) p.h_softmax[layer] = (float)(hs / (double)p.T);
    if (p.aux && p.loads) {
      double a = 0.0;
      for (int g = 0; g < groups; ++g) a += p.aux_part[(size_t)layer * kStatMaxGroups + g];
      p.aux[layer] = (float)a;
    }
  }
}

}  // namespace moe
