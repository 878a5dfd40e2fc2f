// Statistics of the router's score distribution over a dumped logit matrix:
//   * full-pool selection-score entropy H = -sum_e p_e ln p_e per token
//     (Section 4.3), for both score families the paper evaluates:
//       biased sigmoid  p_e = max(sigmoid(z_e) + b_e, 0) / sum (clamped, normalised)
//       softmax         p_e = softmax_e(z)
//     reported as the mean over the tokens of a layer;
//   * the forward statistics of the auxiliary balancing loss (Eq. 8):
//     P_i = mean over tokens of softmax_i(z), f_i = n_i / T, aux = sum_i f_i P_i.
//
// One pass over the dump: a warp takes one token row at a time, lane l holds
// the groups of four experts 4 (l + 32 k) .. + 3 in registers (coalesced 16-byte
// loads), the row sums are warp shuffles.  Per row the entropies come from
//   H = ln S - (sum_e c_e ln c_e) / S,  S = sum_e c_e
// so the softmax family needs no logarithm per element (ln c_e = z_e - max).
// Partial sums per CTA go to scratch in the workspace and are added in a fixed
// order by a second small kernel, in binary64: results do not depend on timing.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <type_traits>

#include "route_math.cuh"

namespace moe {

constexpr int kStatThreads = 256;
constexpr int kStatWarps = kStatThreads / 32;
constexpr int kStatCtaTarget = 444;      // CTAs over all layers (3 per SM on 148 SMs)
constexpr int kStatCtaMaxPerLayer = 444;

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
  unsigned int* arrivals; // [L] finished groups of the second kernel; zero between calls
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

// Sums of four per-lane values over the warp with 6 + 4 shuffles instead of 20: after two exchange rounds every
// lane carries one of the four values (chosen by lane bits 4 and 3) summed over 4 lanes, three more rounds
// finish the sums inside the groups of 8 lanes, and the totals are broadcast from lanes 0, 8, 16, 24.
__device__ __forceinline__ void warp_sum4(float& a, float& b, float& c, float& d, int lane) {
  const bool h1 = (lane & 16) != 0, h2 = (lane & 8) != 0;
  float k0 = h1 ? c : a, k1 = h1 ? d : b;
  k0 += __shfl_xor_sync(0xffffffffu, h1 ? a : c, 16);
  k1 += __shfl_xor_sync(0xffffffffu, h1 ? b : d, 16);
  float k = h2 ? k1 : k0;
  k += __shfl_xor_sync(0xffffffffu, h2 ? k0 : k1, 8);
  k += __shfl_xor_sync(0xffffffffu, k, 4);
  k += __shfl_xor_sync(0xffffffffu, k, 2);
  k += __shfl_xor_sync(0xffffffffu, k, 1);
  a = __shfl_sync(0xffffffffu, k, 0);
  b = __shfl_sync(0xffffffffu, k, 8);
  c = __shfl_sync(0xffffffffu, k, 16);
  d = __shfl_sync(0xffffffffu, k, 24);
}

// dynamic shared memory of score_stats_kernel<NV>: per warp two staged rows, then the layer's bias
__host__ __device__ inline size_t stat_smem_bytes(int nv) { return (size_t)(kStatWarps * 2 + 1) * 32 * nv * 16; }

// NV = 16-byte groups of four experts per lane (E <= 128 * NV, E a multiple of 4, rows 16-byte aligned); kFull:
// E == 128 * NV, no group needs a bounds test.  grid = (C, L)
//
// The pass is bound by the special-function pipe (one warp instruction per 8 cycles per SM sub-partition) and by
// instruction issue about equally, so the per-logit work is arranged around as few of both as possible.  Three
// special-function instructions: with q = exp(z - m), the softmax numerator that is needed anyway,
// sigmoid(z) = q / (q + exp(-m)) costs one reciprocal instead of an exponential and a reciprocal, and the
// logarithm of the clamped biased score is the third.  exp(-m) is computed once per row; rows with |m| > 40
// (where exp(-m) or q + exp(-m) could leave the binary32 range) take the direct form with four.  The plain
// arithmetic runs on pairs of logits with the packed two-float instructions of sm_100.
// Rows arrive through asynchronous 16-byte copies into a two-row ring per warp (each lane reads back exactly the
// words it copied, so no warp synchronisation is involved): the next row is in flight while this one is worked on.
template <int NV, bool kFull>
__global__ void __launch_bounds__(kStatThreads, 3) score_stats_kernel(StatParams p) {
  chained_launch_enter();
  constexpr int NP = 2 * NV;                   // pairs of logits per lane
  extern __shared__ float4 stat_smem[];
  __shared__ float sH[kStatWarps][2];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int layer = blockIdx.y;
  float4* ring = stat_smem + (size_t)warp * 2 * 32 * NV;
  const float4* sB = stat_smem + (size_t)kStatWarps * 2 * 32 * NV;
  const float* zl = p.logits + (size_t)layer * p.T * p.E;
  for (int e = threadIdx.x; e < 128 * NV; e += kStatThreads)
    reinterpret_cast<float*>(stat_smem + (size_t)kStatWarps * 2 * 32 * NV)[e] = (e < p.E) ? p.bias[(size_t)layer * p.E + e] : 0.0f;
  __syncthreads();
  constexpr float kLog2e = 1.44269504f, kLn2 = 0.693147181f;
  f32x2 P[NP];                                 // probability sums of the lane's experts
#pragma unroll
  for (int j = 0; j < NP; ++j) P[j] = pack2(0.0f, 0.0f);
  float acc_hb = 0.0f, acc_hs = 0.0f;
  // lane l holds experts 4 (l + 32 k) .. + 3: consecutive lanes, consecutive 16-byte words
  auto mine = [&](int k) { return kFull || 4 * (lane + 32 * k) < p.E; };
  auto fetch = [&](int row, int buf) {
    const float4* zr = reinterpret_cast<const float4*>(zl + (size_t)row * p.E) + lane;
    const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(ring + buf * 32 * NV + lane));
#pragma unroll
    for (int k = 0; k < NV; ++k)
      if (mine(k))
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + k * 512), "l"(zr + 32 * k) : "memory");
  };
  const int row_step = p.C * kStatWarps;
  int row = blockIdx.x * kStatWarps + warp;
  if (row < p.T) fetch(row, 0);
  asm volatile("cp.async.commit_group;" ::: "memory");
  for (int it = 0; row < p.T; row += row_step, ++it) {
    if (row + row_step < p.T) fetch(row + row_step, (it + 1) & 1);
    asm volatile("cp.async.commit_group;" ::: "memory");       // possibly empty: the wait below counts groups
    asm volatile("cp.async.wait_group 1;" ::: "memory");
    const float4* zs = ring + (it & 1) * 32 * NV + lane;
    float4 z[NV];
    float m = -INFINITY;
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      z[k] = mine(k) ? zs[32 * k] : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      m = fmax3(m, fmaxf(z[k].x, z[k].y), fmaxf(z[k].z, z[k].w));
    }
    m = warp_max(m);
    // hardware exp2 / log2 / reciprocal approximations (a few ulp each): these are statistics with a 1e-5
    // relative budget, not the routing decision, so the bit-exact score chain is not needed here.
    // The two forms are two complete copies of the row's work, so that neither carries the other's registers.
    auto finish_row = [&](auto fast_tag) {
      constexpr bool kFast = decltype(fast_tag)::value;
      // lane-pair partial sums; A = sum q log2 q, B = sum c log2 c: scaled to nats once per row
      f32x2 S2 = pack2(0.0f, 0.0f), A2 = S2, R2 = S2, B2 = S2;
      const float mL = m * kLog2e;
      const float c0 = kFast ? exp2f_fast(-mL) : 1.0f;   // exp(-m), in [4e-18, 3e17]
      const f32x2 l2e = pack2(kLog2e, kLog2e), nmL = pack2(-mL, -mL), c02 = pack2(c0, c0);
      const f32x2 nl2e = pack2(-kLog2e, -kLog2e), zero2 = pack2(0.0f, 0.0f), tiny2 = pack2(1e-37f, 1e-37f);
      f32x2 q2[NP];
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        if (mine(k)) {
          const float4 b4 = sB[lane + 32 * k];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const f32x2 zz = h ? pack2(z[k].z, z[k].w) : pack2(z[k].x, z[k].y);
            const f32x2 bb = h ? pack2(b4.z, b4.w) : pack2(b4.x, b4.y);
            const f32x2 t = fma2(zz, l2e, nmL);                     // (z - m) log2 e
            float t0, t1;
            unpack2(t, t0, t1);
            const f32x2 q = pack2(exp2f_fast(t0), exp2f_fast(t1));
            S2 = add2(S2, q);
            A2 = fma2(q, t, A2);
            f32x2 sg;
            if (kFast) {
              float u0, u1;
              unpack2(add2(q, c02), u0, u1);
              sg = mul2(q, pack2(rcp_fast(u0), rcp_fast(u1)));
            } else {
              float u0, u1;
              unpack2(mul2(zz, nl2e), u0, u1);
              unpack2(add2(pack2(exp2f_fast(u0), exp2f_fast(u1)), c02), u0, u1);   // c02 = 1 here
              sg = pack2(rcp_fast(u0), rcp_fast(u1));
            }
            float c0_, c1_;
            unpack2(add2(sg, bb), c0_, c1_);
            const f32x2 c = pack2(fmaxf(c0_, 0.0f), fmaxf(c1_, 0.0f));
            R2 = add2(R2, c);
            // log2(c + 1e-37) equals log2 c for every c that is not tiny and is finite at c = 0, where the
            // product with c is 0
            float g0, g1;
            unpack2(add2(c, tiny2), g0, g1);
            B2 = fma2(c, pack2(lg2_fast(g0), lg2_fast(g1)), B2);
            q2[2 * k + h] = q;
          }
        } else {
          q2[2 * k] = zero2;
          q2[2 * k + 1] = zero2;
        }
      }
      float S, Sh, A, Ah, R, Rh, B, Bh;
      unpack2(S2, S, Sh); unpack2(A2, A, Ah); unpack2(R2, R, Rh); unpack2(B2, B, Bh);
      S += Sh; A += Ah; R += Rh; B += Bh;
      warp_sum4(S, A, R, B, lane);
      // once per row, in log2 units: H = ln 2 (log2 S - A / S); S >= 1 (the row maximum contributes q = 1)
      const float inv = rcp_fast(S);
      acc_hs += kLn2 * (lg2_fast(S) - A * inv);
      acc_hb += (R > 0.0f) ? kLn2 * (lg2_fast(R) - B * rcp_fast(R)) : 0.0f;
      const f32x2 inv2 = pack2(inv, inv);
#pragma unroll
      for (int j = 0; j < NP; ++j) P[j] = fma2(q2[j], inv2, P[j]);
    };
    if (fabsf(m) <= 40.0f) finish_row(std::true_type{});   // warp-uniform
    else finish_row(std::false_type{});
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();                                  // every warp is done with its ring: it now takes the warps' sums
  float* sP = reinterpret_cast<float*>(stat_smem);  // [warps][128 NV]
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    float4 o;
    unpack2(P[2 * k], o.x, o.y);
    unpack2(P[2 * k + 1], o.z, o.w);
    *reinterpret_cast<float4*>(sP + (size_t)warp * 128 * NV + 4 * (lane + 32 * k)) = o;
  }
  if (lane == 0) { sH[warp][0] = acc_hb; sH[warp][1] = acc_hs; }
  __syncthreads();
  float* outP = p.part_P + ((size_t)layer * p.C + blockIdx.x) * p.E;
  for (int e = threadIdx.x; e < p.E; e += kStatThreads) {
    float s = 0.0f;
#pragma unroll
    for (int w = 0; w < kStatWarps; ++w) s += sP[(size_t)w * 128 * NV + e];
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
  if (e < p.E) {
#pragma unroll 4
    for (int c = sl; c < p.C; c += kStatFinSlices) s += (double)p.part_P[((size_t)layer * p.C + c) * p.E + e];
  }
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
  // The layer's scalars are written by whichever CTA of the layer finishes last (it waits for nothing): the
  // groups' aux shares and the per-CTA entropy sums are added in a fixed order, so the result does not depend on
  // which CTA that is.  The counter wraps to zero at the last arrival.
  __shared__ bool last;
  if (threadIdx.x == 0) {
    p.aux_part[(size_t)layer * kStatMaxGroups + group] = y[0][0];
    __threadfence();
    last = atomicInc(&p.arrivals[layer], gridDim.x - 1) == gridDim.x - 1;
  }
  __syncthreads();
  if (!last || threadIdx.x >= 32) return;
  __threadfence();
  const int lane = threadIdx.x;
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
      for (int g = 0; g < (int)gridDim.x; ++g) a += __ldcg(&p.aux_part[(size_t)layer * kStatMaxGroups + g]);
      p.aux[layer] = (float)a;
    }
  }
}

}  // namespace moe
