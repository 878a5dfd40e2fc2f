// Bias-controller step for all layers in one launch: one CTA of 1024 threads
// per layer, thread i owns expert i.
//   error        e_i = (nbar - n_i) / nbar                    Eq. 3
//   ID           Algorithm 1 lines 8-13 (Eq. 9-12)
//   fixed step   b += eta * sign(e)                           Eq. 5
//   quantile     b = rho * b + (1 - rho) * Q                  Eq. 6-7 + EMA (Section 3)
//   frozen       b unchanged
//   metrics      MaxVio, MinVio                               Eq. 13
// Arithmetic: error and metrics in binary64 rounded once to binary32; the
// update in binary32 with explicitly rounded operations (nothing contracted);
// the centring mean is a binary64 pairwise sum over 1024 padded entries with
// strides 512, 256, ..., 1.
#pragma once
#include <cuda_runtime.h>
#include <limits.h>
#include <stdint.h>

#include "route_math.cuh"

namespace moe {

constexpr int kCtrlThreads = 1024;
constexpr int kStatusState = 4;  // = MOE_ERR_STATE

struct CtrlParams {
  int L, E;
  int controller;  // MOE_CTRL_*
  float ki, kd, eta, rho;
  int center;
  float* bias;        // [L][E] in/out
  float* e_prev;      // [L][E] in/out
  float* bias_prev;   // [L][E] out: bias before this update (for the drift diagnostic)
  int* loads_acc;     // [L][E] consumed and zeroed
  int* loads_last;    // [L][E] out
  float* maxvio;      // [L] out
  float* minvio;      // [L] out
  int* gate_count;    // [L] out
  const float* qb_target;  // [L][E], quantile controller only
  int* status;
};

// Shared-memory scratch of one controller step.
struct CtrlScratch {
  double y[1024];
  long long red_sum[32];
  int red_max[32], red_min[32], red_gate[32];
  long long total_s;
  int max_s, min_s;
};

// One controller step of one layer by the CTA's 1024 threads, one expert per thread, tid in [0, 1024).  `sync`
// is a barrier over exactly these threads.  The integer reductions are order-free; the centring sum has a
// fixed order (y[i] += y[i + stride], strides 512 ... 1).  Loads are read from L2 (they were accumulated
// there with atomics by the routing kernel's CTAs).
template <typename Sync>
__device__ __forceinline__ void controller_layer(const CtrlParams& p, int layer, int tid, CtrlScratch* sc, Sync sync) {
  constexpr int NT = kCtrlThreads;
  constexpr int PER = 1024 / NT;
  const int lane = tid & 31, warp = tid >> 5;
  int n[PER];
  long long s = 0;
  int mx = INT_MIN, mn = INT_MAX;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = tid + j * NT;
    const bool live = i < p.E;
    n[j] = live ? __ldcg(p.loads_acc + (size_t)layer * p.E + i) : 0;
    s += n[j];
    mx = max(mx, live ? n[j] : INT_MIN);
    mn = min(mn, live ? n[j] : INT_MAX);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    s += __shfl_xor_sync(0xffffffffu, s, d);
    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, d));
    mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, d));
  }
  if (lane == 0) { sc->red_sum[warp] = s; sc->red_max[warp] = mx; sc->red_min[warp] = mn; }
  sync();
  if (warp == 0) {
    const bool has = lane < NT / 32;
    s = has ? sc->red_sum[lane] : 0; mx = has ? sc->red_max[lane] : INT_MIN; mn = has ? sc->red_min[lane] : INT_MAX;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      s += __shfl_xor_sync(0xffffffffu, s, d);
      mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, d));
      mn = min(mn, __shfl_xor_sync(0xffffffffu, mn, d));
    }
    if (lane == 0) { sc->total_s = s; sc->max_s = mx; sc->min_s = mn; }
  }
  sync();
  const long long total = sc->total_s;
  if (total <= 0) {
    // empty batch: the error of Eq. 3 is undefined; leave the layer untouched
    if (tid == 0) atomicCAS(p.status, 0, kStatusState);
    return;
  }
  const double nbar = __ddiv_rn((double)total, (double)p.E);
  float b[PER], e[PER];
  int gsum = 0;
#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = tid + j * NT;
    const bool live = i < p.E;
    const size_t o = (size_t)layer * p.E + i;
    e[j] = live ? (float)__ddiv_rn(__dsub_rn(nbar, (double)n[j]), nbar) : 0.0f;
    b[j] = live ? p.bias[o] : 0.0f;
    const float ep = live ? p.e_prev[o] : 0.0f;
    int gate = 0;
    if (p.controller == 0) {                       // ID Balancing
      const float de = __fsub_rn(e[j], ep);
      gate = ((ep > 0.0f && de > 0.0f) || (ep < 0.0f && de < 0.0f)) ? 1 : 0;
      const float t1 = __fmul_rn(p.ki, e[j]);
      const float t2 = gate ? __fmul_rn(p.kd, de) : 0.0f;
      b[j] = __fadd_rn(__fadd_rn(b[j], t1), t2);
    } else if (p.controller == 1) {                // fixed-step integral
      const float step = (e[j] > 0.0f) ? p.eta : (e[j] < 0.0f) ? -p.eta : 0.0f;
      b[j] = __fadd_rn(b[j], step);
    } else if (p.controller == 2) {                // quantile target (+ EMA)
      const float q = live ? p.qb_target[o] : 0.0f;
      if (p.rho == 0.0f) {
        b[j] = q;
      } else {
        const float keep = __fmul_rn(p.rho, b[j]);
        const float take = __fmul_rn(__fsub_rn(1.0f, p.rho), q);
        b[j] = __fadd_rn(keep, take);
      }
    }
    if (live) gsum += gate;
  }

  if (p.center) {
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int i = tid + j * NT;
      sc->y[i] = (i < p.E) ? (double)b[j] : 0.0;
    }
    sync();
#pragma unroll 1
    for (int stride = 512; stride >= 32; stride >>= 1) {
      // y[i + stride] is not written during this pass, so one barrier suffices
      for (int i = tid; i < stride; i += NT) sc->y[i] = __dadd_rn(sc->y[i], sc->y[i + stride]);
      sync();
    }
    if (tid < 32) {
      // strides 16 ... 1 stay inside the first warp: same additions, warp barriers instead of block barriers
#pragma unroll
      for (int stride = 16; stride >= 1; stride >>= 1) {
        double v = 0.0;
        if (tid < stride) v = __dadd_rn(sc->y[tid], sc->y[tid + stride]);
        __syncwarp();
        if (tid < stride) sc->y[tid] = v;
        __syncwarp();
      }
    }
    sync();
    const float mean = (float)__ddiv_rn(sc->y[0], (double)p.E);
#pragma unroll
    for (int j = 0; j < PER; ++j) b[j] = __fsub_rn(b[j], mean);
  }

#pragma unroll
  for (int d = 16; d > 0; d >>= 1) gsum += __shfl_xor_sync(0xffffffffu, gsum, d);
  if (lane == 0) sc->red_gate[warp] = gsum;
  sync();

#pragma unroll
  for (int j = 0; j < PER; ++j) {
    const int i = tid + j * NT;
    if (i < p.E) {
      const size_t o = (size_t)layer * p.E + i;
      p.bias_prev[o] = p.bias[o];
      p.bias[o] = b[j];
      p.e_prev[o] = e[j];
      p.loads_last[o] = n[j];
      p.loads_acc[o] = 0;
    }
  }
  if (tid == 0) {
    int gtot = 0;
    for (int w = 0; w < NT / 32; ++w) gtot += sc->red_gate[w];
    p.gate_count[layer] = gtot;
    p.maxvio[layer] = (float)__ddiv_rn(__dsub_rn((double)sc->max_s, nbar), nbar);
    p.minvio[layer] = (float)__ddiv_rn(__dsub_rn(nbar, (double)sc->min_s), nbar);
  }
}

__global__ void __launch_bounds__(kCtrlThreads) controller_kernel(const CtrlParams p) {
  __shared__ CtrlScratch sc;
  // launched with programmatic stream serialisation: the block may already be resident while the
  // routing kernel before it drains; nothing of that kernel's output is touched before this returns
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // the next routing kernel may be scheduled now; it waits for this grid before it reads anything
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  controller_layer(p, blockIdx.x, threadIdx.x, &sc, [] { __syncthreads(); });
}

// Diagnostics the paper plots for the load controller (figure captions of Section 3, Section 4.3), per layer,
// from the state the last controller update left: out[layer][0] fraction of open worsening gates, [1] share of
// all assignments that went to the busiest 10 % of the experts (m = round(E/10) experts), [2] fraction of experts
// without any token, [3] mean |bias change| of the last update.  Integer counts, binary64 ratios rounded once.
struct DiagParams {
  int L, E;
  const int* loads_last;    // [L][E]
  const int* gate_count;    // [L]
  const float* bias;        // [L][E]
  const float* bias_prev;   // [L][E]
  float* out;               // [L][4]
};

__global__ void __launch_bounds__(kCtrlThreads) diagnostics_kernel(const DiagParams p) {
  chained_launch_enter();
  __shared__ unsigned int hist[256];
  __shared__ unsigned int sel_prefix, sel_rank;
  __shared__ long long red_a[32], red_b[32];
  __shared__ int red_c[32], red_d[32];
  __shared__ double y[kCtrlThreads];
  const int layer = blockIdx.x, i = threadIdx.x, lane = i & 31, warp = i >> 5;
  const bool live = i < p.E;
  const size_t o = (size_t)layer * p.E + i;
  const int n = live ? p.loads_last[o] : -1;
  y[i] = live ? fabs((double)p.bias[o] - (double)p.bias_prev[o]) : 0.0;
  // The share of the busiest m experts needs the sum of the m largest loads: the m-th largest load v* is
  // found by a radix select (four 8-bit digits, most significant first, shared-memory histogram of the
  // values that still match the digits fixed so far); the sum is then that of the loads above v* plus
  // v* for the remaining places -- equal loads are interchangeable, so no order among them is needed.
  int m = (p.E + 5) / 10;
  if (m < 1) m = 1;
  const unsigned int key = live ? (unsigned int)n : 0u;        // loads are non-negative
  if (i == 0) { sel_prefix = 0u; sel_rank = (unsigned int)m; }
#pragma unroll 1
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    if (i < 256) hist[i] = 0u;
    __syncthreads();
    const unsigned int pre = sel_prefix;
    if (live && (pass == 0 || ((key ^ pre) >> (shift + 8)) == 0u)) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    __syncthreads();
    if (warp == 0) {
      // lane l owns bins 255 - 8l ... 248 - 8l (descending): find the bin where the count from the top reaches the rank
      unsigned int c[8], mine = 0;
#pragma unroll
      for (int t = 0; t < 8; ++t) { c[t] = hist[255 - (lane * 8 + t)]; mine += c[t]; }
      unsigned int incl = mine;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
      }
      const unsigned int rank = sel_rank, excl = incl - mine;
      if (rank > excl && rank <= incl) {
        unsigned int run = excl;
#pragma unroll
        for (int t = 0; t < 8; ++t) {
          if (rank > run && rank <= run + c[t]) {
            sel_prefix = pre | ((unsigned int)(255 - (lane * 8 + t)) << shift);
            sel_rank = rank - run;
          }
          run += c[t];
        }
      }
    }
    __syncthreads();
  }
  const int vstar = (int)sel_prefix;            // the m-th largest load
  long long tot = live ? n : 0, top = (live && n > vstar) ? n : 0;
  int above = (live && n > vstar) ? 1 : 0;
  int empty = (live && n == 0) ? 1 : 0;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    tot += __shfl_xor_sync(0xffffffffu, tot, d);
    top += __shfl_xor_sync(0xffffffffu, top, d);
    empty += __shfl_xor_sync(0xffffffffu, empty, d);
    above += __shfl_xor_sync(0xffffffffu, above, d);
  }
  if (lane == 0) { red_a[warp] = tot; red_b[warp] = top; red_c[warp] = empty; red_d[warp] = above; }
  for (int stride = kCtrlThreads / 2; stride >= 1; stride >>= 1) {
    __syncthreads();
    if (i < stride) y[i] = __dadd_rn(y[i], y[i + stride]);
  }
  __syncthreads();
  if (i == 0) {
    long long t = 0, tp = 0;
    int em = 0, ab = 0;
    for (int w = 0; w < kCtrlThreads / 32; ++w) { t += red_a[w]; tp += red_b[w]; em += red_c[w]; ab += red_d[w]; }
    tp += (long long)(m - ab) * vstar;          // the places among the m busiest that are held by loads equal to v*
    float* out = p.out + (size_t)layer * 4;
    out[0] = (float)__ddiv_rn((double)p.gate_count[layer], (double)p.E);
    out[1] = t > 0 ? (float)__ddiv_rn((double)tp, (double)t) : 0.0f;
    out[2] = (float)__ddiv_rn((double)em, (double)p.E);
    out[3] = (float)__ddiv_rn(y[0], (double)p.E);
  }
}

// Mean over tokens of the top-K gating-score entropy H = -sum_k w_k ln w_k (nats, Section 4.3).  Two steps with a
// fixed summation order, binary64 throughout: grid (kEntropySlices, L) CTAs each sum a contiguous slice of the
// layer's tokens (per thread: tokens tid, tid+256, ... of the slice; then a pairwise tree) into part[layer][slice];
// one warp per layer adds the slices in index order.
constexpr int kEntropySlices = 64;
constexpr int kEntropyThreads = 256;

__global__ void __launch_bounds__(kEntropyThreads) gate_entropy_kernel(const float* gate, int T, int K, double* part) {
  chained_launch_enter();
  __shared__ double y[kEntropyThreads];
  const int layer = blockIdx.y, slice = blockIdx.x, i = threadIdx.x;
  const int per = (T + kEntropySlices - 1) / kEntropySlices;
  const int t0 = slice * per, t1 = min(T, t0 + per);
  const float* g = gate + (size_t)layer * T * K;
  double acc = 0.0;
  for (int t = t0 + i; t < t1; t += kEntropyThreads) {
    double h = 0.0;
    for (int k = 0; k < K; ++k) {
      const double w = (double)g[(size_t)t * K + k];
      if (w > 0.0) h -= w * log(w);
    }
    acc += h;
  }
  y[i] = acc;
  for (int stride = kEntropyThreads / 2; stride >= 1; stride >>= 1) {
    __syncthreads();
    if (i < stride) y[i] = y[i] + y[i + stride];
  }
  __syncthreads();
  if (i == 0) part[(size_t)layer * kEntropySlices + slice] = y[0];
}

__global__ void gate_entropy_finish_kernel(const double* part, int T, float* out) {
  chained_launch_enter();
  const int layer = blockIdx.x;
  if (threadIdx.x == 0) {
    double s = 0.0;
    for (int c = 0; c < kEntropySlices; ++c) s += part[(size_t)layer * kEntropySlices + c];
    out[layer] = (float)(s / (double)T);
  }
}

// Router weights given expert-contiguous, in [L][H][E] bf16 -> out [L][E][H] (hidden contiguous, the layout the
// routing kernel's tensor maps describe).  64 x 64 tiles through shared memory; grid (ceil(E/64), ceil(H/64), L),
// 256 threads; reads and writes are 128-byte rows.
__global__ void __launch_bounds__(256) transpose_w_kernel(const uint16_t* in, uint16_t* out, int H, int E) {
  chained_launch_enter();
  __shared__ uint16_t tile[64][66];
  const int layer = blockIdx.z, e0 = blockIdx.x * 64, h0 = blockIdx.y * 64;
  const uint16_t* src = in + (size_t)layer * H * E;
  uint16_t* dst = out + (size_t)layer * E * H;
  const int c = threadIdx.x & 63, r4 = threadIdx.x >> 6;
  for (int r = r4; r < 64; r += 4) {
    const int h = h0 + r, e = e0 + c;
    tile[r][c] = (h < H && e < E) ? src[(size_t)h * E + e] : (uint16_t)0;
  }
  __syncthreads();
  for (int r = r4; r < 64; r += 4) {
    const int e = e0 + r, h = h0 + c;
    if (e < E && h < H) dst[(size_t)e * H + h] = tile[c][r];
  }
}

// loads_acc[i] += add[i]
__global__ void loads_add_kernel(int* acc, const int* add, int n) {
  chained_launch_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) acc[i] += add[i];
}

}  // namespace moe
