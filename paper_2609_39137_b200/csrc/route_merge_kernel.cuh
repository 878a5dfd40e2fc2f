// Second half of a routing step under chunk-split scheduling.
//
// When the token tiles are long the routing kernel gives the expert chunks of
// one tile to different CTA pairs that run at the same time, so the tile is
// streamed from HBM once and the other readers find it in L2.  Each (tile,
// chunk) item leaves, per token, its chunk's best `cand_len` experts as
// (score s, expert e) pairs in ranking order (biased score descending, expert
// ascending); the lists of a token are contiguous: cand[layer][token][chunk][cand_len].
// The chunks cover disjoint experts, so the K best of the row (Eq. 2) are the
// first K of the merge of those sorted lists: this kernel recomputes the biased
// score v = s + b_e (one rounded addition, the same operation the routing
// kernel ordered by), merges, and produces what the fused epilogue produces
// otherwise -- indices, gates (selected scores normalised without the bias,
// sequential fp32 sum in output order), alpha = rank K+1 on request, and the
// load histogram (Algorithm 1 line 4).
//
// Memory-bound: per token it reads num_chunks * cand_len * 8 bytes and writes
// 8 K (+4) bytes.  A warp takes 32 consecutive tokens: their lists are one
// contiguous block, which the lanes fetch with coalesced asynchronous copies
// (all in flight at once) into the warp's part of shared memory, one row
// per token with an odd row stride (conflict-free both for the staging and for
// the lanes reading different entries of their own rows); then each lane
// merges its own token from there and stores its outputs.  A CTA walks tokens
// of ONE layer and flushes its histogram once at its end (one global atomic per
// non-zero expert per CTA); inside the token loop only warps synchronise.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "route_math.cuh"

namespace moe {

constexpr int kMergeThreads = 256;
constexpr int kMergeMaxChunks = 4;     // 1024 experts / 256 per chunk
constexpr int kMergeMaxK = 16;

struct MergeParams {
  int T, E, K, num_chunks, cand_len;
  const float2* cand;   // [L][T][num_chunks][cand_len]
  const float* bias;    // [L][E]
  int* loads;           // [L][E] accumulators (added to)
  int32_t* topk_idx;    // [L][T][K]
  float* topk_gate;     // [L][T][K]
  float* alpha_out;     // [L][T] or nullptr
};

// row stride of the staged lists in float2 units (odd)
__host__ __device__ inline int merge_row_stride(int n_all) { return n_all | 1; }
__host__ __device__ inline size_t merge_smem_bytes(int n_all) {
  return (size_t)kMergeThreads * merge_row_stride(n_all) * sizeof(float2);
}

// grid = (slices, L); dynamic shared memory merge_smem_bytes(num_chunks * cand_len)
__global__ void __launch_bounds__(kMergeThreads, 3) route_merge_kernel(const MergeParams p) {
  extern __shared__ float2 lists_s[];                       // [entry][thread]
  __shared__ float bias_s[1024];
  __shared__ int hist_s[1024];
  const int layer = blockIdx.y;
  const int tid = threadIdx.x;
  const int n_all = p.num_chunks * p.cand_len;
  // launched with programmatic stream serialisation behind the routing kernel: its lists are complete and
  // visible only after this wait
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int i = tid; i < 1024; i += kMergeThreads) {
    bias_s[i] = (i < p.E) ? p.bias[(size_t)layer * p.E + i] : -INFINITY;
    hist_s[i] = 0;
  }
  __syncthreads();
  const int lane = tid & 31;
  const int stride = merge_row_stride(n_all);
  float2* warp_s = lists_s + (size_t)(tid - lane) * stride;  // rows of this warp's 32 tokens
  const float2* mine = warp_s + lane * stride;
  const float uniform = __fdiv_rn(1.0f, (float)p.K);
  // warp-uniform loop: tok0 = first token of the warp's group of 32
  for (int tok0 = blockIdx.x * kMergeThreads + (tid - lane); tok0 < p.T; tok0 += gridDim.x * kMergeThreads) {
    const int rows = min(32, p.T - tok0);
    const int total = rows * n_all;                        // float2 elements of the group, contiguous
    const float2* src = p.cand + ((size_t)layer * p.T + tok0) * n_all;
    __syncwarp();                                          // the previous group's merges have read the rows
    int r = 0, n = lane;                                   // element lane + 32 j as (row, entry)
    while (n >= n_all) { n -= n_all; r += 1; }
    const int dr = 32 / n_all, dn = 32 - dr * n_all;       // advancing the element by 32
    // asynchronous 8-byte copies global -> shared, all of the group's entries in flight at once (no registers
    // are held for them); consecutive lanes, consecutive entries
#pragma unroll 1
    for (int i = lane; i < total; i += 32) {
      const uint32_t dst = static_cast<uint32_t>(__cvta_generic_to_shared(warp_s + r * stride + n));
      asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(dst), "l"(src + i) : "memory");
      r += dr; n += dn;
      if (n >= n_all) { n -= n_all; r += 1; }
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    const int tok = tok0 + lane;
    if (lane < rows) {
    // Heads of the (up to four) lists; a step picks the best head by a two-round tournament and replaces it
    // with its list's next entry.  Everything is selections under predicates: lanes differ in which list wins,
    // and a branch per list would run all four bodies one after the other in every step.
    float hv[kMergeMaxChunks], hs[kMergeMaxChunks];
    int he[kMergeMaxChunks];
    uint32_t pos_all = 0;                                    // four 8-bit positions
    auto entry = [&](int c, int pos, float& v, float& sc, int& e) {
      // an exhausted list, an entry without an expert and a padding column all rank after every real entry
      const bool in = c < p.num_chunks && pos < p.cand_len;
      const float2 se = mine[min(c, p.num_chunks - 1) * p.cand_len + min(pos, p.cand_len - 1)];
      const int ei = __float_as_int(se.y);
      const bool real = in && (unsigned)ei < (unsigned)p.E;
      sc = se.x;
      e = real ? ei : 0x7fffffff;
      v = real ? __fadd_rn(se.x, bias_s[real ? ei : 0]) : -INFINITY;
    };
#pragma unroll
    for (int c = 0; c < kMergeMaxChunks; ++c) entry(c, 0, hv[c], hs[c], he[c]);
    float alpha = __int_as_float(0x7fc00000);
    float denom = 0.0f;
    float sel_s[kMergeMaxK];
    int sel_e[kMergeMaxK];
#pragma unroll
    for (int k = 0; k < kMergeMaxK + 1; ++k) {
      if (k < p.cand_len) {                                // rank K is only needed for alpha
        float v01, s01, v23, s23, bv, bs;
        int e01, e23, be;
        const bool t01 = ranks_before(hv[1], he[1], hv[0], he[0]);
        const bool t23 = ranks_before(hv[3], he[3], hv[2], he[2]);
        select_triple(t01, hv[0], hv[1], hs[0], hs[1], he[0], he[1], v01, s01, e01);
        select_triple(t23, hv[2], hv[3], hs[2], hs[3], he[2], he[3], v23, s23, e23);
        const bool tb = ranks_before(v23, e23, v01, e01);
        select_triple(tb, v01, v23, s01, s23, e01, e23, bv, bs, be);
        const int best = tb ? (t23 ? 3 : 2) : (t01 ? 1 : 0);
        if (k < kMergeMaxK && k < p.K) {
          sel_s[k] = bs;
          sel_e[k] = be;
          denom = (k == 0) ? bs : __fadd_rn(denom, bs);     // D = ((s_0 + s_1) + s_2) + ... in output order
        }
        if (k == p.K) alpha = bv;
        const int npos = (int)((pos_all >> (8 * best)) & 0xffu) + 1;
        pos_all += 1u << (8 * best);
        float nv, ns;
        int ne;
        entry(best, npos, nv, ns, ne);
#pragma unroll
        for (int c = 0; c < kMergeMaxChunks; ++c) select_triple(best == c, hv[c], nv, hs[c], ns, he[c], ne, hv[c], hs[c], he[c]);
      }
    }
    // every entry of the row has been read: the row now takes the outputs, (expert, gate) at position k
    float2* out_row = warp_s + lane * stride;
    // one reciprocal of the denominator and a branch-free correctly rounded division per gate; a token whose
    // denominator or smallest score is outside the range where that holds takes the library's division
    float smin = INFINITY;
#pragma unroll
    for (int k = 0; k < kMergeMaxK; ++k)
      if (k < p.K) smin = fminf(smin, sel_s[k]);
    const bool safe = gate_division_safe(smin, denom);
    const float rden = rcp_rn_normal(safe ? denom : 1.0f);
#pragma unroll
    for (int k = 0; k < kMergeMaxK; ++k) {
      if (k < p.K) {
        float gk = div_rn_by(sel_s[k], denom, rden);
        if (!safe) gk = (denom == 0.0f) ? uniform : __fdiv_rn(sel_s[k], denom);
        out_row[k] = make_float2(__int_as_float(sel_e[k]), gk);
        if ((unsigned)sel_e[k] < (unsigned)p.E) atomicAdd(&hist_s[sel_e[k]], 1);
      }
    }
    if (p.alpha_out != nullptr) p.alpha_out[(size_t)layer * p.T + tok] = alpha;
    }   // lane < rows
    __syncwarp();
    // the group's outputs are contiguous in global memory (rows x K words): consecutive lanes, consecutive words
    {
      const size_t o0 = ((size_t)layer * p.T + tok0) * p.K;
      int rr = 0, kk = lane;
      while (kk >= p.K) { kk -= p.K; rr += 1; }
      const int drr = 32 / p.K, dkk = 32 - drr * p.K;
      for (int j = lane; j < rows * p.K; j += 32) {
        const float2 eg = warp_s[rr * stride + kk];
        p.topk_idx[o0 + j] = __float_as_int(eg.x);
        p.topk_gate[o0 + j] = eg.y;
        rr += drr; kk += dkk;
        if (kk >= p.K) { kk -= p.K; rr += 1; }
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < p.E; i += kMergeThreads) {
    const int n = hist_s[i];
    if (n != 0) atomicAdd(&p.loads[(size_t)layer * p.E + i], n);
  }
}

}  // namespace moe
