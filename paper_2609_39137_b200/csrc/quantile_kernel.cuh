// Quantile Balancing target (Eq. 6-7): for every expert j the r-th smallest
// margin d_ij = s_ij - alpha_i over the m tokens of the step, Q_j = -d, with
// the nearest-rank position r = m - floor(m K / E) (no interpolation).
//
// Exact selection by a most-significant-digit radix select over the
// order-preserving 32-bit image of the margin: four passes of 8 bits.  Each
// pass streams the dumped logits once (HBM-bound, coalesced: a warp reads 32
// consecutive experts of one token), recomputes the score, and counts -- per
// expert -- the margins that still match the digits fixed so far, in a
// shared-memory histogram that is flushed to the global scratch histogram with
// one atomic per non-empty bin per CTA.  A small scan kernel then fixes the
// next digit per expert, updates the remaining rank and clears the histogram.
// With a key scratch (contexts of the quantile controller have one) the first
// pass stores the 32-bit image of every margin and the three later passes
// stream those 4 bytes back instead of recomputing the score, which makes them
// memory-bound instead of instruction-bound.
//
// Contexts with the key scratch replace the last two digit passes by a gather:
// after two passes the keys sharing the answer's 16-bit prefix are few (their
// number is the count of the bin the second scan chose); one more stream over
// the keys appends them to a per-expert list, and a warp per expert selects the
// answer among them (two 8-bit digits in shared memory).
//
// Scratch per context: hist [E][256] u32, prefix [E] u32, rank [E] u32, keys [max_tokens][E] u32,
// match [E] u32, fill [E] u32, list [E][1024] u16.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "route_math.cuh"

namespace moe {

constexpr int kQbCols = 32;       // experts per CTA (one per lane)
constexpr int kQbThreads = 256;   // 8 warps, each takes every 8th row of the CTA's row range
constexpr int kQbRowsInFlight = 8;

struct QbParams {
  const float* logits;  // [m][E]
  const float* alpha;   // [m]
  int m, E, K;
  uint32_t* hist;       // [E][256], zero on entry of every histogram pass
  uint32_t* prefix;     // [E] digits fixed so far (high bits)
  uint32_t* rank;       // [E] remaining 1-based rank inside the matching set
  float* target;        // [E] out: Q_j
  uint32_t* keys;       // [m][E] scratch or null: pass 0 stores every margin's key, later passes read it back
  // gather form of the last two digits (contexts with a key scratch): after two passes the keys that share the
  // 16-bit prefix of the answer are few; they are gathered per expert and the answer is selected among them
  uint32_t* match;      // [E] number of keys sharing the prefix (the count of the bin chosen by the second scan)
  uint32_t* fill;       // [E] entries gathered so far
  uint16_t* list;       // [E][kQbListCap] low 16 bits of the gathered keys
  // Margins with a large common offset (a bias that has drifted as a whole) share their sign, exponent and leading
  // mantissa bits, so the keys that share a 16-bit prefix can be many more than a list holds; the second scan then
  // raises this flag and a third digit pass runs before the gather (its two kernels return at once otherwise)
  uint32_t* deep;       // [1] or null
};
constexpr int kQbListCap = 1024;

// Monotone map float -> uint32 (a < b as floats  <=>  key(a) < key(b)); -0 is
// canonicalised to +0 first so equal values get equal keys.
__device__ __forceinline__ uint32_t margin_key(float d) {
  d = __fadd_rn(d, 0.0f);
  const uint32_t u = __float_as_uint(d);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float margin_from_key(uint32_t k) {
  const uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}

__global__ void qb_init_kernel(QbParams p) {
  chained_launch_enter();
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < p.E) {
    long long r = (long long)p.m - ((long long)p.m * p.K) / p.E;
    if (r < 1) r = 1;
    if (r > p.m) r = p.m;
    p.prefix[j] = 0u;
    p.rank[j] = (uint32_t)r;
  }
  if (j == 0 && p.deep != nullptr) *p.deep = 0u;
  for (int i = j; i < p.E * 256; i += gridDim.x * blockDim.x) p.hist[i] = 0u;
}

// pass = 0..3, most significant byte first.  grid = (ceil(E/32), row_splits)
__global__ void __launch_bounds__(kQbThreads) qb_hist_kernel(QbParams p, int pass) {
  chained_launch_enter();
  if (p.deep != nullptr && pass == 2 && *p.deep == 0u) return;   // the third digit is not needed
  __shared__ uint32_t h[256 * kQbCols];  // [bin][col]: lanes hit distinct banks
  for (int i = threadIdx.x; i < 256 * kQbCols; i += kQbThreads) h[i] = 0u;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col = blockIdx.x * kQbCols + lane;
  const bool live = col < p.E;
  const int shift = 24 - 8 * pass;
  const uint32_t pre = live ? p.prefix[col] : 0u;
  const int rows_per = (p.m + gridDim.y - 1) / gridDim.y;
  const int r0 = blockIdx.y * rows_per;
  const int r1 = min(p.m, r0 + rows_per);
  // kQbRowsInFlight independent 128-byte row segments per warp are requested before any is used
  constexpr int kWarps = kQbThreads / 32;
  if (p.keys != nullptr && pass > 0) {
    // keys of pass 0 are read back: no score arithmetic, the pass is a plain stream over 4 bytes per margin
    for (int i0 = r0 + warp; i0 < r1; i0 += kWarps * kQbRowsInFlight) {
      uint32_t key[kQbRowsInFlight];
#pragma unroll
      for (int u = 0; u < kQbRowsInFlight; ++u) {
        const int i = i0 + u * kWarps;
        key[u] = (live && i < r1) ? __ldg(p.keys + (size_t)i * p.E + col) : 0u;
      }
#pragma unroll
      for (int u = 0; u < kQbRowsInFlight; ++u) {
        const int i = i0 + u * kWarps;
        if (live && i < r1 && ((key[u] ^ pre) >> (shift + 8)) == 0u)
          atomicAdd(&h[((key[u] >> shift) & 255u) * kQbCols + lane], 1u);
      }
    }
  } else {
    for (int i0 = r0 + warp; i0 < r1; i0 += kWarps * kQbRowsInFlight) {
      float z[kQbRowsInFlight], a[kQbRowsInFlight];
#pragma unroll
      for (int u = 0; u < kQbRowsInFlight; ++u) {
        const int i = i0 + u * kWarps;
        const bool ok = live && i < r1;
        z[u] = ok ? __ldg(p.logits + (size_t)i * p.E + col) : 0.0f;
        a[u] = ok ? __ldg(p.alpha + i) : 0.0f;
      }
#pragma unroll
      for (int u = 0; u < kQbRowsInFlight; ++u) {
        const int i = i0 + u * kWarps;
        if (live && i < r1) {
          const float s = sigmoid_score(z[u]);
          const uint32_t key = margin_key(__fsub_rn(s, a[u]));
          if (p.keys != nullptr) p.keys[(size_t)i * p.E + col] = key;      // pass 0 only
          const bool match = (pass == 0) || (((key ^ pre) >> (shift + 8)) == 0u);
          if (match) atomicAdd(&h[((key >> shift) & 255u) * kQbCols + lane], 1u);
        }
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < 256 * kQbCols; i += kQbThreads) {
    const int c = blockIdx.x * kQbCols + (i % kQbCols);
    const uint32_t cnt = h[i];
    if (cnt != 0u && c < p.E) atomicAdd(&p.hist[(size_t)c * 256 + i / kQbCols], cnt);
  }
}

// One warp per expert: find the bin holding the remaining rank, fix that
// digit, clear the histogram; after the last pass emit Q_j = -margin.
__global__ void qb_scan_kernel(QbParams p, int pass) {
  chained_launch_enter();
  if (p.deep != nullptr && pass == 2 && *p.deep == 0u) return;
  const int j = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int lane = threadIdx.x & 31;
  if (j >= p.E) return;
  uint32_t* hj = p.hist + (size_t)j * 256;
  uint32_t c[8];
  uint32_t mine = 0;
#pragma unroll
  for (int t = 0; t < 8; ++t) { c[t] = hj[lane * 8 + t]; mine += c[t]; }
  uint32_t incl = mine;  // inclusive prefix sum over lanes
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  const uint32_t rank = p.rank[j];
  const uint32_t excl = incl - mine;
  const bool holder = (rank > excl) && (rank <= incl);   // exactly one lane when 1 <= rank <= total
  uint32_t bin = 0, below = 0, count = 0;
  if (holder) {
    uint32_t run = excl;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (rank > run && rank <= run + c[t]) { bin = lane * 8 + t; below = run; count = c[t]; }
      run += c[t];
    }
  }
  const uint32_t who = __ballot_sync(0xffffffffu, holder);
  const int src = who ? (__ffs(who) - 1) : 0;
  bin = __shfl_sync(0xffffffffu, bin, src);
  below = __shfl_sync(0xffffffffu, below, src);
  count = __shfl_sync(0xffffffffu, count, src);
#pragma unroll
  for (int t = 0; t < 8; ++t) hj[lane * 8 + t] = 0u;
  if (lane == 0) {
    const uint32_t pre = p.prefix[j] | (bin << (24 - 8 * pass));
    p.prefix[j] = pre;
    p.rank[j] = rank - below;
    if (pass == 3) p.target[j] = -margin_from_key(pre);
    if ((pass == 1 || pass == 2) && p.match != nullptr) {
      p.match[j] = count;
      p.fill[j] = 0u;
      if (pass == 1 && p.deep != nullptr && count > (uint32_t)kQbListCap) atomicOr(p.deep, 1u);
    }
  }
}

// Gather (after two digit passes): one more stream over the stored keys; a key that shares the 16-bit prefix of
// its expert's answer is appended to that expert's list (its low 16 bits).  Experts whose matching set is larger
// than the list (long runs of equal margins) are left to the selection kernel, which then reads their keys itself.
// grid and row split as for qb_hist_kernel.
__global__ void __launch_bounds__(kQbThreads) qb_gather_kernel(QbParams p) {
  chained_launch_enter();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int col = blockIdx.x * kQbCols + lane;
  const bool live = col < p.E && p.match[col] <= (uint32_t)kQbListCap;
  const uint32_t pre = live ? p.prefix[col] : 0u;
  const int fixed_shift = (*p.deep != 0u) ? 8 : 16;     // bits of the key not fixed yet
  const int rows_per = (p.m + gridDim.y - 1) / gridDim.y;
  const int r0 = blockIdx.y * rows_per;
  const int r1 = min(p.m, r0 + rows_per);
  constexpr int kWarps = kQbThreads / 32;
  for (int i0 = r0 + warp; i0 < r1; i0 += kWarps * kQbRowsInFlight) {
    uint32_t key[kQbRowsInFlight];
#pragma unroll
    for (int u = 0; u < kQbRowsInFlight; ++u) {
      const int i = i0 + u * kWarps;
      key[u] = (live && i < r1) ? __ldg(p.keys + (size_t)i * p.E + col) : 0u;
    }
#pragma unroll
    for (int u = 0; u < kQbRowsInFlight; ++u) {
      const int i = i0 + u * kWarps;
      if (live && i < r1 && ((key[u] ^ pre) >> fixed_shift) == 0u) {
        const uint32_t pos = atomicAdd(&p.fill[col], 1u);
        if (pos < (uint32_t)kQbListCap) p.list[(size_t)col * kQbListCap + pos] = (uint16_t)(key[u] & 0xffffu);
      }
    }
  }
}

// Selection among the gathered keys: one warp per expert.  Two 8-bit digits over the low 16 bits, each a
// warp-private shared-memory histogram followed by the same scan as qb_scan_kernel.  An expert whose matching
// set did not fit the list walks its own column of the key scratch instead (strided reads: slow, but only long
// runs of equal margins get there).  Emits Q_j = -margin.
constexpr int kQbSelectWarps = 4;

__global__ void __launch_bounds__(kQbSelectWarps * 32) qb_select_kernel(QbParams p) {
  chained_launch_enter();
  __shared__ uint32_t hs[kQbSelectWarps][256];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int j = blockIdx.x * kQbSelectWarps + warp;
  if (j >= p.E) return;
  uint32_t* h = hs[warp];
  const uint32_t n_match = p.match[j];
  const bool listed = n_match <= (uint32_t)kQbListCap;
  const uint32_t n = listed ? n_match : (uint32_t)p.m;
  const bool deep = *p.deep != 0u;
  const int fixed_shift = deep ? 8 : 16;
  uint32_t pre = p.prefix[j];          // top 16 (24 after a third digit pass) bits fixed
  uint32_t rank = p.rank[j];           // 1-based rank inside the matching set
  const uint16_t* lst = p.list + (size_t)j * kQbListCap;
  auto value = [&](uint32_t i, bool& match) -> uint32_t {
    // low 16 bits of candidate i and whether it belongs to the matching set at all
    if (listed) { match = true; return (uint32_t)lst[i]; }
    const uint32_t key = __ldg(p.keys + (size_t)i * p.E + j);
    match = ((key ^ pre) >> fixed_shift) == 0u;
    return key & 0xffffu;
  };
#pragma unroll 1
  for (int digit = deep ? 1 : 0; digit < 2; ++digit) {
    const int shift = 8 - 8 * digit;
#pragma unroll
    for (int t = 0; t < 8; ++t) h[lane * 8 + t] = 0u;
    __syncwarp();
    for (uint32_t i = lane; i < n; i += 32) {
      bool match;
      const uint32_t v = value(i, match);
      if (match && (digit == 0 || ((v ^ pre) & 0xff00u) == 0u)) atomicAdd(&h[(v >> shift) & 255u], 1u);
    }
    __syncwarp();
    uint32_t c[8], mine = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) { c[t] = h[lane * 8 + t]; mine += c[t]; }
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    const uint32_t excl = incl - mine;
    const bool holder = (rank > excl) && (rank <= incl);
    uint32_t bin = 0, below = 0;
    if (holder) {
      uint32_t run = excl;
#pragma unroll
      for (int t = 0; t < 8; ++t) {
        if (rank > run && rank <= run + c[t]) { bin = lane * 8 + t; below = run; }
        run += c[t];
      }
    }
    const uint32_t who = __ballot_sync(0xffffffffu, holder);
    const int src = who ? (__ffs(who) - 1) : 0;
    bin = __shfl_sync(0xffffffffu, bin, src);
    below = __shfl_sync(0xffffffffu, below, src);
    pre |= bin << shift;
    rank -= below;
    __syncwarp();
  }
  if (lane == 0) p.target[j] = -margin_from_key(pre);
}

// ---------------------------------------------------------------------------
// Quantile target estimated from a per-expert margin histogram (footnote to
// Eq. 7: the estimate the paper mentions for use "at scale"; bins, range and
// the rule inside a bin are this library's choice).  One pass over the dump:
//   bin k = floor((d + range) * inv_h) clamped to [0, B-1], d = sigmoid(z) - alpha
//   (two rounded binary32 operations), B uniform bins over [-range, range);
// the counts of a CTA's 8 experts are kept in shared memory ([expert][B + 4] words, the 4 extra words skew the
// experts' rows by four banks) and flushed with one global atomic per non-empty bin,
// consecutive lanes on consecutive bins of one expert (contiguous addresses); the number of row splits is kept
// small, because every split flushes its own copy of the non-empty bins.  A second kernel (one warp
// per expert) finds the bin k* of the r-th smallest margin, r = m - floor(mK/E),
// and interpolates in binary64: est = -range + (k* + ((r - below) - 0.5) / cnt) * h.
// The counts are integers, so histograms of several ranks can be added before
// the second kernel runs (that is what makes the estimate usable when the
// tokens of a step are spread over data-parallel ranks).
constexpr int kQhCols = 8;         // experts per CTA: 32 bytes of a row, one DRAM sector
constexpr int kQhThreads = 512;
constexpr int kQhRowsInFlight = 8;
constexpr int kQhMaxBins = 2048;   // 8 experts x 2052 words = 64 KB of shared memory

struct QhParams {
  const float* logits;  // [m][E]
  const float* alpha;   // [m]
  int m, E, K, B;
  float range, inv_h;   // inv_h = (float)B / (2 * range)
  float edge_eps;       // distance to a bin edge (in bins) below which the quick score is not trusted
  uint32_t* hist;       // [E][B], zero on entry of the histogram kernel, cleared again by the finish kernel
  float* target;        // [E] out: Q_j
};

__device__ __forceinline__ int margin_bin(float d, float range, float inv_h, int B) {
  const float u = __fmul_rn(__fadd_rn(d, range), inv_h);
  if (!(u >= 0.0f)) return 0;
  const float fl = floorf(u);
  return (fl >= (float)B) ? B - 1 : (int)fl;
}

// Quick score for binning: sigmoid(z) = 1 / (1 + 2^(-z log2 e)) with the hardware exponential and reciprocal
// approximations.  Its distance to sigmoid_score is measured over every finite binary32 logit
// (moe_debug_quick_score_gap) and stays below kQuickScoreGap; a margin whose quick bin position is closer than
// that (scaled to bins, plus the rounding of the position itself) to an edge is binned again from the exact score.
constexpr float kQuickScoreGap = 3e-7f;
__device__ __forceinline__ float quick_score(float z) {
  float u, r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(u) : "f"(z * -1.44269504f));
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(1.0f + u));
  return r;
}
// In bins: the quick score's distance to the exact one, doubled, plus 3e-4 for the roundings that separate the two
// positions (one of d + range, one of the product, one of the fused form, one of range * inv_h: each at most
// half an ulp of a value below 2048, 6.1e-5).
__host__ __device__ inline float qh_edge_eps(float inv_h) { return 2.0f * kQuickScoreGap * inv_h + 3e-4f; }

__device__ __noinline__ int exact_margin_bin(float z, float a, float range, float inv_h, int B) {
  return margin_bin(__fsub_rn(sigmoid_score(z), a), range, inv_h, B);
}

__host__ __device__ inline int qh_row_words(int B) { return B + 4; }
__host__ __device__ inline size_t qh_smem_bytes(int B) { return (size_t)kQhCols * qh_row_words(B) * 4; }

// grid = (ceil(E / 8), row_splits); dynamic shared memory qh_smem_bytes(B).  A lane takes four experts of a row
// (one 16-byte load), a warp 16 rows of the CTA's 8 experts per load; kQhRowsInFlight loads are issued before the
// first is used.  Every logit is binned from the quick score (two special-function instructions and about twenty
// others); the few whose position is within edge_eps of a bin edge, and non-finite ones, are binned again with the
// exact score chain, so the counts are those of the exact rule.
__global__ void __launch_bounds__(kQhThreads) qb_margin_hist_kernel(QhParams p) {
  chained_launch_enter();
  extern __shared__ uint32_t hs[];   // [col][B + 4] counters
  const int row_words = qh_row_words(p.B);
  for (int i = threadIdx.x; i < kQhCols * row_words; i += kQhThreads) hs[i] = 0u;
  __syncthreads();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int c0 = (lane & 1) * 4, sub = lane >> 1;         // first of the lane's four columns, row inside the warp's 16
  const int col0 = blockIdx.x * kQhCols + c0;
  const bool live = col0 < p.E;                           // E is a multiple of 4: a group is live or dead as a whole
  const int rows_per = (p.m + gridDim.y - 1) / gridDim.y;
  const int r0 = blockIdx.y * rows_per;
  const int r1 = min(p.m, r0 + rows_per);
  constexpr int kRowsPerIter = (kQhThreads / 32) * 16;    // rows taken by the CTA per load
  constexpr float kMagic = 12582912.0f;                   // 1.5 * 2^23: adding it rounds to an integer in the low mantissa bits
  const float r_ih_half = p.range * p.inv_h - 0.5f;
  const float trust = 0.5f - p.edge_eps;
  uint32_t* my = hs + c0 * row_words;
  for (int i0 = r0 + warp * 16 + sub; i0 < r1; i0 += kRowsPerIter * kQhRowsInFlight) {
    float4 z[kQhRowsInFlight];
    float a[kQhRowsInFlight];
#pragma unroll
    for (int u = 0; u < kQhRowsInFlight; ++u) {
      const int i = i0 + u * kRowsPerIter;
      const bool ok = live && i < r1;
      z[u] = ok ? __ldg(reinterpret_cast<const float4*>(p.logits + (size_t)i * p.E + col0)) : make_float4(0.f, 0.f, 0.f, 0.f);
      a[u] = ok ? __ldg(p.alpha + i) : 0.0f;
    }
#pragma unroll
    for (int u = 0; u < kQhRowsInFlight; ++u) {
      const int i = i0 + u * kRowsPerIter;
      if (live && i < r1) {
        const float zz[4] = {z[u].x, z[u].y, z[u].z, z[u].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          // position in bins, minus 1/2, from the quick score; rounding it to the nearest integer is the floor
          // of the position unless that lies close to an edge, which the test below catches (NaN included)
          const float ph = fmaf(quick_score(zz[j]) - a[u], p.inv_h, r_ih_half);
          const float tm = ph + kMagic;
          const float off = ph - (tm - kMagic);                   // in [-1/2, 1/2]: distance to the bin's middle
          int bin = __float_as_int(tm) - __float_as_int(kMagic);
          bin = max(0, min(p.B - 1, bin));
          if (!(fabsf(off) <= trust)) bin = exact_margin_bin(zz[j], a[u], p.range, p.inv_h, p.B);
          atomicAdd(&my[j * row_words + bin], 1u);
        }
      }
    }
  }
  __syncthreads();
  // flush: a warp stays inside one expert, consecutive lanes on consecutive bins
  for (int cl = 0; cl < kQhCols; ++cl) {
    const int cc = blockIdx.x * kQhCols + cl;
    if (cc >= p.E) break;
    for (int bin = threadIdx.x; bin < p.B; bin += kQhThreads) {
      const uint32_t cnt = hs[cl * row_words + bin];
      if (cnt != 0u) atomicAdd(&p.hist[(size_t)cc * p.B + bin], cnt);
    }
  }
}

// One CTA of 256 threads per expert: thread t owns the bins [t * per, (t + 1) * per), per = ceil(B / 256); a block
// scan of the threads' sums gives the count before each thread's range, and the thread whose range takes the
// cumulative count to the rank or beyond walks its bins and interpolates.  Every thread clears its bins (ready
// for the next update).
constexpr int kQhFinishThreads = 256;

__global__ void __launch_bounds__(kQhFinishThreads) qb_margin_hist_finish_kernel(QhParams p) {
  chained_launch_enter();
  __shared__ uint32_t warp_tot[kQhFinishThreads / 32];
  const int j = blockIdx.x;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t* hj = p.hist + (size_t)j * p.B;
  const int per = (p.B + kQhFinishThreads - 1) / kQhFinishThreads;    // <= 8 for B <= 2048
  const int b0 = tid * per;
  uint32_t c[8];
  uint32_t mine = 0;
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    c[t] = (t < per && b0 + t < p.B) ? hj[b0 + t] : 0u;
    mine += c[t];
  }
#pragma unroll
  for (int t = 0; t < 8; ++t)
    if (t < per && b0 + t < p.B) hj[b0 + t] = 0u;
  uint32_t incl = mine;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) warp_tot[warp] = incl;
  __syncthreads();
  uint32_t before = incl - mine;                          // count of the bins before this thread's range
  for (int w = 0; w < warp; ++w) before += warp_tot[w];
  long long r = (long long)p.m - ((long long)p.m * p.K) / p.E;
  if (r < 1) r = 1;
  if (r > p.m) r = p.m;
  const uint32_t rank = (uint32_t)r;
  if (rank > before && rank <= before + mine) {           // exactly one thread: the counts of an expert sum to m >= rank
    uint32_t run = before;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (rank > run && rank <= run + c[t]) {
        const int kstar = b0 + t;
        const double h = __ddiv_rn(__dmul_rn(2.0, (double)p.range), (double)p.B);
        const double inside = __ddiv_rn(__dsub_rn((double)(rank - run), 0.5), (double)c[t]);
        const double est = __dadd_rn(-(double)p.range, __dmul_rn(__dadd_rn((double)kstar, inside), h));
        p.target[j] = -(float)est;
      }
      run += c[t];
    }
  }
}

}  // namespace moe
