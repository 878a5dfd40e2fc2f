// Second half of a routing step under chunk-split scheduling.
//
// When the token tiles are long (hidden > 2048) the routing kernel gives the
// expert chunks of one tile to different CTA pairs that run at the same time,
// so the tile is streamed from HBM once and the other readers find it in L2.
// Each (tile, chunk) item leaves, per token, its chunk's best `cand_len`
// experts as (score s, expert e) pairs in ranking order (biased score
// descending, expert ascending).  The chunks cover disjoint experts, so the
// K best of the row (Eq. 2) are the first K of the merge of those sorted
// lists: this kernel recomputes the biased score v = s + b_e (one rounded
// addition, the same operation the routing kernel ordered by), merges, and
// produces what the fused epilogue produces otherwise -- indices, gates
// (selected scores normalised without the bias, sequential fp32 sum in output
// order), alpha = rank K+1 on request, and the load histogram (Algorithm 1
// line 4: shared-memory counts, one global atomic per non-zero expert per CTA).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "route_math.cuh"

namespace moe {

constexpr int kMergeThreads = 256;
constexpr int kMergeRowsPerCta = 1024;
constexpr int kMergeMaxChunks = 4;     // 1024 experts / 256 per chunk

struct MergeParams {
  int T, E, K, num_chunks, cand_len;
  const float2* cand;   // [L][num_chunks][T][cand_len]
  const float* bias;    // [L][E]
  int* loads;           // [L][E] accumulators (added to)
  int32_t* topk_idx;    // [L][T][K]
  float* topk_gate;     // [L][T][K]
  float* alpha_out;     // [L][T] or nullptr
};

// grid = (ceil(T / kMergeRowsPerCta), L); one thread per token row, kMergeRowsPerCta / kMergeThreads rows each
__global__ void __launch_bounds__(kMergeThreads) route_merge_kernel(const MergeParams p) {
  __shared__ float bias_s[1024];
  __shared__ int hist_s[1024];
  const int layer = blockIdx.y;
  // launched with programmatic stream serialisation behind the routing kernel: its lists are complete and
  // visible only after this wait
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int i = threadIdx.x; i < 1024; i += kMergeThreads) {
    bias_s[i] = (i < p.E) ? p.bias[(size_t)layer * p.E + i] : -INFINITY;
    hist_s[i] = 0;
  }
  __syncthreads();
  const int row_end = min(p.T, (int)(blockIdx.x + 1) * kMergeRowsPerCta);
  for (int tok = blockIdx.x * kMergeRowsPerCta + threadIdx.x; tok < row_end; tok += kMergeThreads) {
    // heads of the chunk lists
    const float2* lst[kMergeMaxChunks];
    float hv[kMergeMaxChunks], hs[kMergeMaxChunks];
    int he[kMergeMaxChunks], pos[kMergeMaxChunks];
#pragma unroll
    for (int c = 0; c < kMergeMaxChunks; ++c) {
      pos[c] = (c < p.num_chunks) ? 0 : p.cand_len;       // a chunk that does not exist is an exhausted list
      lst[c] = p.cand + (((size_t)layer * p.num_chunks + (c < p.num_chunks ? c : 0)) * p.T + tok) * p.cand_len;
    }
    auto load_head = [&](int c) {
      // an exhausted list, an entry without an expert and a padding column all rank after every real entry
      float2 se = make_float2(0.0f, __int_as_float(0x7fffffff));
      if (pos[c] < p.cand_len) se = lst[c][pos[c]];
      const int e = __float_as_int(se.y);
      const bool real = (unsigned)e < (unsigned)p.E;
      hs[c] = se.x;
      he[c] = real ? e : 0x7fffffff;
      hv[c] = real ? __fadd_rn(se.x, bias_s[e]) : -INFINITY;
    };
#pragma unroll
    for (int c = 0; c < kMergeMaxChunks; ++c) load_head(c);
    float sel_s[16];
    int sel_e[16];
    float alpha = __int_as_float(0x7fc00000);
#pragma unroll
    for (int k = 0; k < 17; ++k) {
      if (k <= p.K) {           // rank K is only needed for alpha
        int best = 0;
#pragma unroll
        for (int c = 1; c < kMergeMaxChunks; ++c)
          if (ranks_before(hv[c], he[c], hv[best], he[best])) best = c;
        float bv = hv[0], bs = hs[0];
        int be = he[0];
#pragma unroll
        for (int c = 1; c < kMergeMaxChunks; ++c)
          if (best == c) { bv = hv[c]; bs = hs[c]; be = he[c]; }
        if (k < 16 && k < p.K) { sel_s[k] = bs; sel_e[k] = be; }
        if (k == p.K) alpha = bv;
#pragma unroll
        for (int c = 0; c < kMergeMaxChunks; ++c)
          if (best == c) { pos[c] += 1; load_head(c); }
      }
    }
    float denom = sel_s[0];
#pragma unroll
    for (int k = 1; k < 16; ++k)
      if (k < p.K) denom = __fadd_rn(denom, sel_s[k]);
    const float uniform = __fdiv_rn(1.0f, (float)p.K);
    const size_t o = ((size_t)layer * p.T + tok) * p.K;
#pragma unroll
    for (int k = 0; k < 16; ++k) {
      if (k < p.K) {
        p.topk_idx[o + k] = sel_e[k];
        p.topk_gate[o + k] = (denom == 0.0f) ? uniform : __fdiv_rn(sel_s[k], denom);
        if ((unsigned)sel_e[k] < (unsigned)p.E) atomicAdd(&hist_s[sel_e[k]], 1);
      }
    }
    if (p.alpha_out != nullptr) p.alpha_out[(size_t)layer * p.T + tok] = alpha;
  }
  __syncthreads();
  for (int i = threadIdx.x; i < p.E; i += kMergeThreads) {
    const int n = hist_s[i];
    if (n != 0) atomicAdd(&p.loads[(size_t)layer * p.E + i], n);
  }
}

}  // namespace moe
