// Host side of the C ABI declared in include/moe_route.h: argument checks,
// workspace layout, TMA descriptors, kernel launches.  No device memory is
// allocated here; all state lives in the caller's workspace.
#include "../../include/moe_route.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "controller_kernel.cuh"
#include "quantile_kernel.cuh"
#include "score_stats_kernel.cuh"
#include "route_kernel.cuh"
#include "route_merge_kernel.cuh"

namespace {

using namespace moe;

constexpr size_t kAlign = 256;
constexpr size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t status, bias, e_prev, bias_prev, loads_acc, loads_last, maxvio, minvio, gate_count;
  size_t qb_target, qb_hist, qb_prefix, qb_rank, qb_keys, qb_match, qb_fill, qb_list, qb_deep;
  size_t state_end;  // everything before this is cleared at init
  size_t stat_cnt;   // [L] arrival counters of score_stats_finish_kernel (wrap to zero by themselves)
  size_t stat_P, stat_H, stat_aux, ent_part;   // per-CTA partial sums of moe_score_stats (written before they are read)
  size_t stage_x, stage_w, stage_idx, stage_gate;
  size_t w_t;   // [L][E][H] bf16 copy of the weights when they are given as [L][H][E]
  size_t cand;  // [L][chunks][max_tokens][K+1] (score, expert) pairs, chunk-split scheduling only
  size_t total;
#ifdef MOE_DEBUG
  // debug build: every section is followed by a 256-byte canary that moe_route_poll checks
  int num_guards;
  size_t guard[48];
#endif
};
#ifdef MOE_DEBUG
constexpr unsigned char kCanaryByte = 0xC5;
#endif

// Chunk-split scheduling (the expert chunks of a token tile go to different CTA pairs, a merge kernel
// finishes): chosen when one CTA pair re-reading its tile once per chunk would push the tiles of all
// resident pairs out of L2 -- 74 pairs x 256 tokens x hidden x 2 bytes exceeds the 126 MB L2 beyond
// hidden ~ 3300 -- and there is more than one chunk.  Also chosen for launches so small that every (tile, chunk)
// gets a CTA pair of its own (at most 64 such items at max_tokens): the chunks of a tile are then scanned side by
// side instead of one after the other, which is worth more than the merge launch costs.
bool use_chunk_split(const moe_route_config& c) {
  if (c.num_experts <= kBN) return false;
  if (c.chunk_split == 1) return false;
  if (c.chunk_split == 2) return true;
  const long long chunks = (c.num_experts + kBN - 1) / kBN;
  const long long tile_pairs = ((long long)c.max_tokens + 2 * kBM - 1) / (2 * kBM);
  return c.hidden > 3072 || (long long)c.num_layers * tile_pairs * chunks <= 64;
}

Layout make_layout(const moe_route_config& c) {
  Layout l{};
  size_t o = 0;
  const size_t LE = (size_t)c.num_layers * c.num_experts;
#ifdef MOE_DEBUG
  auto take = [&](size_t bytes) {
    size_t at = o;
    o = align_up(o + bytes);
    if (l.num_guards < 48) l.guard[l.num_guards++] = o;
    o += kAlign;
    return at;
  };
#else
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes); return at; };
#endif
  l.status = take(64);
  l.bias = take(LE * 4);
  l.e_prev = take(LE * 4);
  l.bias_prev = take(LE * 4);
  l.loads_acc = take(LE * 4);
  l.loads_last = take(LE * 4);
  l.maxvio = take((size_t)c.num_layers * 4);
  l.minvio = take((size_t)c.num_layers * 4);
  l.gate_count = take((size_t)c.num_layers * 4);
  l.qb_target = take(LE * 4);
  l.stat_cnt = take((size_t)c.num_layers * 4);
  if (c.controller == MOE_CTRL_QUANTILE) {
    // exact selection: radix histogram [E][256]; histogram estimate: margin histogram [E][qb_hist_bins]
    l.qb_hist = take((size_t)c.num_experts * (c.qb_hist_bins > 0 ? c.qb_hist_bins : 256) * 4);
    l.qb_prefix = take((size_t)c.num_experts * 4);
    l.qb_rank = take((size_t)c.num_experts * 4);
  }
  l.state_end = o;
  if (c.controller == MOE_CTRL_QUANTILE && c.qb_hist_bins == 0) {
    l.qb_keys = take((size_t)c.max_tokens * c.num_experts * 4);
    l.qb_match = take((size_t)c.num_experts * 4);
    l.qb_fill = take((size_t)c.num_experts * 4);
    l.qb_list = take((size_t)c.num_experts * kQbListCap * 2);
    l.qb_deep = take(4);
  }
  {
    const size_t LC = (size_t)c.num_layers * stat_ctas_per_layer(c.num_layers);
    l.stat_P = take(LC * c.num_experts * 4);
    l.stat_H = take(LC * 2 * 4);
    l.stat_aux = take((size_t)c.num_layers * kStatMaxGroups * 8);
    l.ent_part = take((size_t)c.num_layers * kEntropySlices * 8);
  }
  if (c.host_staging) {
    const size_t LT = (size_t)c.num_layers * c.max_tokens;
    l.stage_x = take(LT * c.hidden * 2);
    l.stage_w = take(LE * c.hidden * 2);
    l.stage_idx = take(LT * c.top_k * 4);
    l.stage_gate = take(LT * c.top_k * 4);
  }
  if (c.w_layout == 1) l.w_t = take(LE * c.hidden * 2);
  if (use_chunk_split(c)) {
    const size_t chunks = (size_t)(c.num_experts + kBN - 1) / kBN;
    l.cand = take((size_t)c.num_layers * chunks * c.max_tokens * (c.top_k + 1) * sizeof(float2));
  }
  l.total = o;
  return l;
}

bool config_ok(const moe_route_config* c) {
  if (!c || c->struct_size != (int32_t)sizeof(moe_route_config)) return false;
  if (c->num_layers < 1 || c->num_layers > 65535) return false;
  if (c->num_experts < 8 || c->num_experts > kMaxE || (c->num_experts % 8) != 0) return false;
  if (c->top_k < 1 || c->top_k > 16 || c->top_k >= c->num_experts) return false;
  if (c->hidden < 8 || (c->hidden % 8) != 0) return false;
  if (c->max_tokens < 1) return false;
  if (c->controller < MOE_CTRL_ID || c->controller > MOE_CTRL_FROZEN) return false;
  if (!(c->ki >= 0.0f) || !(c->kd >= 0.0f) || !(c->eta >= 0.0f)) return false;
  if (!(c->qb_ema_rho >= 0.0f) || !(c->qb_ema_rho < 1.0f)) return false;
  if (c->center < -1 || c->center > 1) return false;
  if (c->spin_limit < 0) return false;
  if (c->w_layout != 0 && c->w_layout != 1) return false;
  if (c->chunk_split < 0 || c->chunk_split > 2) return false;
  if (c->qb_hist_bins != 0 && (c->qb_hist_bins < 32 || c->qb_hist_bins > kQhMaxBins || (c->qb_hist_bins % 32) != 0))
    return false;
  if (c->qb_hist_bins != 0 && !(c->qb_hist_range > 0.0f && c->qb_hist_range <= 1e6f)) return false;
  return true;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// Scratch of moe_quantile_target_static: radix histogram [1024][256] u32, then prefix [1024] and
// rank [1024] u32.  Lives in every device that loads the library, until the process exits.
constexpr int kStaticMaxExperts = 1024;
constexpr int kStaticMaxDevices = 64;
constexpr size_t kStaticScratchBytes = (size_t)kStaticMaxExperts * 256 * 4 + 2 * (size_t)kStaticMaxExperts * 4;
static __device__ __align__(256) unsigned char moe_static_quantile_scratch[kStaticScratchBytes];
static void* g_static_scratch_dev[kStaticMaxDevices];   // device address of the array, per device
static int g_static_sms[kStaticMaxDevices];
static std::mutex g_static_mu;

struct moe_route_ctx {
  moe_route_config cfg;
  Layout lay;
  uint8_t* ws;
  int device;
  int num_sms;
  int center_on;
  EncodeTiledFn encode;
  cudaStream_t last_stream;
  int64_t launches;
  int64_t ctrl_steps;   // controller updates enqueued so far (exported / restored with the controller state)
  int stall_next;       // moe_debug_route_stall: applies to the next routing launch only
  size_t merge_occ_smem;   // resident CTAs per SM of route_merge_kernel, cached per shared-memory size
  int merge_occ;
  int qh_occ;              // resident CTAs per SM of qb_margin_hist_kernel (0: not asked yet)
  // cached TMA descriptors
  const void* map_x_ptr;
  const void* map_w_ptr;
  int map_tokens;
  CUtensorMap tm_x, tm_w;
  // quantile controller: dump of the last routing step
  const float* qb_logits;
  const float* qb_alpha;
  int qb_tokens;
  bool staged_w;
  char err[256];
};

namespace {

int fail(moe_route_ctx* ctx, int code, const char* fmt, ...) {
  if (ctx) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
    va_end(ap);
  }
  return code;
}

int cuda_fail(moe_route_ctx* ctx, cudaError_t e, const char* what) {
  return fail(ctx, MOE_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

template <typename T>
T* at(moe_route_ctx* ctx, size_t off) { return reinterpret_cast<T*>(ctx->ws + off); }

int* status_ptr(moe_route_ctx* ctx) { return at<int>(ctx, ctx->lay.status); }

// 3-D bf16 tensor map: dims (inner, rows, layers), box (64, box_rows, 1), 128-byte swizzle,
// out-of-range elements read as zero.
int encode_map(moe_route_ctx* ctx, CUtensorMap* out, const void* base, uint64_t inner, uint64_t rows,
               uint64_t layers, uint32_t box_rows) {
  cuuint64_t dims[3] = {inner, rows, layers};
  cuuint64_t strides[2] = {inner * 2, inner * rows * 2};
  cuuint32_t box[3] = {(cuuint32_t)kBK, box_rows, 1};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = ctx->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                           CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return fail(ctx, MOE_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", (int)r);
  return MOE_OK;
}

// Launch with programmatic stream serialisation: the kernel's launch latency and prologue overlap the tail of the
// kernel queued before it; every kernel launched this way starts with chained_launch_enter().
template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t lc{};
  lc.gridDim = grid;
  lc.blockDim = block;
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

template <int KL>
int launch_route(moe_route_ctx* ctx, const RouteParams& rp, int grid, cudaStream_t st) {
  static bool attr_set[64] = {};
  const size_t smem = route_smem_bytes();
  if (!attr_set[ctx->device & 63]) {
    cudaError_t e = cudaFuncSetAttribute(route_step_kernel<KL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaFuncSetAttribute(route_step_kernel)");
    attr_set[ctx->device & 63] = true;
  }
  // programmatic stream serialisation: prologue, TMA loads and MMAs may overlap the tail of the kernel
  // queued before this one; the epilogue waits for that kernel before it reads the bias
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(grid);
  lc.blockDim = dim3(kRouteThreads);
  lc.dynamicSmemBytes = smem;
  lc.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, route_step_kernel<KL>, ctx->tm_x, ctx->tm_w, rp);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "route_step_kernel launch");
  ctx->launches += 1;
  return MOE_OK;
}

int route_device(moe_route_ctx* ctx, const void* x, const void* w, int32_t T, int32_t* idx, float* gate,
                 float* logits, float* alpha, cudaStream_t st) {
  const moe_route_config& c = ctx->cfg;
  if (c.w_layout == 1) {
    // expert-contiguous weights: bring them into the layout of the tensor map first (same stream; the routing
    // kernel's producer waits for the preceding grid before its first load)
    if (reinterpret_cast<uintptr_t>(w) & 1) return fail(ctx, MOE_ERR_INVALID_ARG, "w must be 2-byte aligned");
    uint16_t* wt = at<uint16_t>(ctx, ctx->lay.w_t);
    const dim3 tg((c.num_experts + 63) / 64, (c.hidden + 63) / 64, c.num_layers);
    launch_chained(transpose_w_kernel, tg, dim3(256), 0, st, static_cast<const uint16_t*>(w), wt, c.hidden, c.num_experts);
    cudaError_t te = cudaGetLastError();
    if (te != cudaSuccess) return cuda_fail(ctx, te, "transpose_w_kernel launch");
    ctx->launches += 1;
    w = wt;
  }
  if (ctx->map_x_ptr != x || ctx->map_w_ptr != w || ctx->map_tokens != T) {
    if ((reinterpret_cast<uintptr_t>(x) & 15) || (reinterpret_cast<uintptr_t>(w) & 15))
      return fail(ctx, MOE_ERR_INVALID_ARG, "x and w must be 16-byte aligned");
    int rc = encode_map(ctx, &ctx->tm_x, x, c.hidden, T, c.num_layers, kBM);
    if (rc) return rc;
    rc = encode_map(ctx, &ctx->tm_w, w, c.hidden, c.num_experts, c.num_layers, kBN / 2);
    if (rc) return rc;
    ctx->map_x_ptr = x; ctx->map_w_ptr = w; ctx->map_tokens = T;
  }
  RouteParams rp{};
  rp.L = c.num_layers; rp.T = T; rp.H = c.hidden; rp.E = c.num_experts; rp.K = c.top_k;
  rp.pairs_per_layer = (T + 2 * kBM - 1) / (2 * kBM);
  rp.num_items = rp.pairs_per_layer * c.num_layers;
  rp.num_kblocks = (c.hidden + kBK - 1) / kBK;
  // fp32 accumulation error of the tensor core grows with the length of the accumulation chain: chains
  // longer than 2048 hidden elements are split in two and added once in fp32 by the epilogue
  rp.num_segs = (c.hidden > 2048) ? 2 : 1;
  rp.seg_kblocks = (rp.num_kblocks + rp.num_segs - 1) / rp.num_segs;
  rp.num_chunks = (c.num_experts + kBN - 1) / kBN;
  rp.bias = at<float>(ctx, ctx->lay.bias);
  rp.loads = at<int>(ctx, ctx->lay.loads_acc);
  rp.topk_idx = idx; rp.topk_gate = gate; rp.logits_out = logits; rp.alpha_out = alpha;
  rp.status = status_ptr(ctx);
  rp.spin_limit = c.spin_limit > 0 ? (uint32_t)c.spin_limit : 0x7fffffffu;
  const int need = c.top_k + (alpha ? 1 : 0);
  rp.stall_after = ctx->stall_next;
  ctx->stall_next = 0;
  rp.split = use_chunk_split(c) ? 1 : 0;
  if (rp.split) {
    rp.num_items *= rp.num_chunks;
    rp.cand_len = need;
    rp.cand = at<float2>(ctx, ctx->lay.cand);
  }
  const int max_pairs = ctx->num_sms / 2;
  const int grid = 2 * (rp.num_items < max_pairs ? rp.num_items : max_pairs);   // clusters of 2 CTAs
  int rc;
  if (need <= 3) rc = launch_route<3>(ctx, rp, grid, st);
  else if (need <= 5) rc = launch_route<5>(ctx, rp, grid, st);
  else if (need <= 8) rc = launch_route<8>(ctx, rp, grid, st);
  else if (need <= 10) rc = launch_route<10>(ctx, rp, grid, st);
  else if (need <= 11) rc = launch_route<11>(ctx, rp, grid, st);   // Top-10 with the alpha output (quantile controller)
  else rc = launch_route<17>(ctx, rp, grid, st);
  if (rc != MOE_OK || !rp.split) return rc;
  // chunk-split scheduling: merge the chunks' candidate lists into indices, gates, alpha and loads
  MergeParams mp{};
  mp.T = T; mp.E = c.num_experts; mp.K = c.top_k; mp.num_chunks = rp.num_chunks; mp.cand_len = need;
  mp.cand = rp.cand; mp.bias = rp.bias; mp.loads = rp.loads;
  mp.topk_idx = idx; mp.topk_gate = gate; mp.alpha_out = alpha;
  {
    static bool attr_set[64] = {};
    if (!attr_set[ctx->device & 63]) {
      cudaError_t ae = cudaFuncSetAttribute(route_merge_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)merge_smem_bytes(kMergeMaxChunks * (kMergeMaxK + 1)));
      if (ae != cudaSuccess) return cuda_fail(ctx, ae, "cudaFuncSetAttribute(route_merge_kernel)");
      attr_set[ctx->device & 63] = true;
    }
  }
  // a CTA walks tokens of one layer and flushes its histogram once; the grid is at most what is resident at
  // once (a grid slightly above that would run a second, almost empty wave)
  const size_t merge_smem = merge_smem_bytes(rp.num_chunks * need);
  if (ctx->merge_occ < 1 || ctx->merge_occ_smem != merge_smem) {
    int occ = 0;
    cudaError_t oe = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, route_merge_kernel, kMergeThreads, merge_smem);
    if (oe != cudaSuccess || occ < 1) return cuda_fail(ctx, oe, "occupancy of route_merge_kernel");
    ctx->merge_occ = occ;
    ctx->merge_occ_smem = merge_smem;
  }
  const int per_sm = ctx->merge_occ;
  const int num_tiles = (T + kMergeThreads - 1) / kMergeThreads;
  int slices = (per_sm * ctx->num_sms) / c.num_layers;
  if (slices > num_tiles) slices = num_tiles;
  if (slices < 1) slices = 1;
  cudaLaunchConfig_t lc{};
  lc.gridDim = dim3(slices, c.num_layers);
  lc.blockDim = dim3(kMergeThreads);
  lc.dynamicSmemBytes = merge_smem;
  lc.stream = st;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  lc.attrs = &attr;
  lc.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&lc, route_merge_kernel, mp);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "route_merge_kernel launch");
  ctx->launches += 1;
  return MOE_OK;
}

}  // namespace

extern "C" {

void moe_route_default_config(moe_route_config* cfg, int32_t num_layers, int32_t num_experts, int32_t top_k,
                              int32_t hidden, int32_t max_tokens) {
  if (!cfg) return;
  memset(cfg, 0, sizeof *cfg);
  cfg->struct_size = (int32_t)sizeof *cfg;
  cfg->num_layers = num_layers;
  cfg->num_experts = num_experts;
  cfg->top_k = top_k;
  cfg->hidden = hidden;
  cfg->max_tokens = max_tokens;
  cfg->controller = MOE_CTRL_ID;
  cfg->ki = 6e-3f;
  cfg->kd = 6e-3f;
  cfg->eta = 1e-3f;
  cfg->qb_ema_rho = 0.0f;
  cfg->center = -1;
  cfg->spin_limit = 0;
  cfg->host_staging = 0;
  cfg->w_layout = 0;
  cfg->chunk_split = 0;
  cfg->qb_hist_bins = 0;
  cfg->qb_hist_range = 1.0f;
}

size_t moe_route_workspace_bytes(const moe_route_config* cfg) {
  if (!config_ok(cfg)) return 0;
  return make_layout(*cfg).total;
}

int moe_route_init(const moe_route_config* cfg, void* dev_workspace, size_t workspace_bytes, moe_route_ctx** out) {
  if (!out) return MOE_ERR_INVALID_ARG;
  *out = nullptr;
  if (!config_ok(cfg)) return MOE_ERR_INVALID_ARG;
  const Layout lay = make_layout(*cfg);
  if (!dev_workspace || workspace_bytes < lay.total || (reinterpret_cast<uintptr_t>(dev_workspace) % kAlign) != 0)
    return MOE_ERR_WORKSPACE;
  moe_route_ctx* ctx = new (std::nothrow) moe_route_ctx();
  if (!ctx) return MOE_ERR_CUDA;
  ctx->cfg = *cfg;
  ctx->lay = lay;
  ctx->ws = static_cast<uint8_t*>(dev_workspace);
  ctx->center_on = cfg->center >= 0 ? cfg->center : (cfg->controller == MOE_CTRL_ID ? 1 : 0);
  if (cfg->controller == MOE_CTRL_FROZEN) ctx->center_on = 0;
  cudaError_t e = cudaGetDevice(&ctx->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&ctx->num_sms, cudaDevAttrMultiProcessorCount, ctx->device);
  int major = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, ctx->device);
  if (e != cudaSuccess) { delete ctx; return MOE_ERR_CUDA; }
  if (major != 10) { delete ctx; return MOE_ERR_UNSUPPORTED; }   // sm_100a code only
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || !fn || qres != cudaDriverEntryPointSuccess) { delete ctx; return MOE_ERR_CUDA; }
  ctx->encode = reinterpret_cast<EncodeTiledFn>(fn);
  e = cudaMemset(dev_workspace, 0, lay.state_end);
#ifdef MOE_DEBUG
  for (int g = 0; g < lay.num_guards && e == cudaSuccess; ++g)
    e = cudaMemset(static_cast<uint8_t*>(dev_workspace) + lay.guard[g], kCanaryByte, kAlign);
#endif
  if (e == cudaSuccess) e = cudaDeviceSynchronize();
  if (e != cudaSuccess) { delete ctx; return MOE_ERR_CUDA; }
  *out = ctx;
  return MOE_OK;
}

int moe_route_step(moe_route_ctx* ctx, const void* x_bf16, const void* w_bf16, int32_t num_tokens,
                   int32_t* topk_idx, float* topk_gate, float* logits_out, float* alpha_out, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (!x_bf16 || !w_bf16 || !topk_idx || !topk_gate) return fail(ctx, MOE_ERR_INVALID_ARG, "null tensor pointer");
  if (num_tokens < 1 || num_tokens > ctx->cfg.max_tokens)
    return fail(ctx, MOE_ERR_INVALID_ARG, "num_tokens %d outside [1, %d]", num_tokens, ctx->cfg.max_tokens);
  // the dump is written with 16-byte vector stores, the other outputs with 4-byte stores
  if (reinterpret_cast<uintptr_t>(logits_out) & 15)
    return fail(ctx, MOE_ERR_INVALID_ARG, "logits_out must be 16-byte aligned");
  if ((reinterpret_cast<uintptr_t>(topk_idx) & 3) || (reinterpret_cast<uintptr_t>(topk_gate) & 3) ||
      (reinterpret_cast<uintptr_t>(alpha_out) & 3))
    return fail(ctx, MOE_ERR_INVALID_ARG, "topk_idx, topk_gate and alpha_out must be 4-byte aligned");
  if (ctx->cfg.controller == MOE_CTRL_QUANTILE && (!logits_out || !alpha_out))
    return fail(ctx, MOE_ERR_INVALID_ARG, "the quantile controller needs logits_out and alpha_out");
  if (ctx->cfg.controller == MOE_CTRL_QUANTILE && ctx->qb_logits != nullptr) {
    // Eq. 7 ranks the margins of ONE score matrix; a second routing call
    // before the update would need a merged dump.
    return fail(ctx, MOE_ERR_UNSUPPORTED, "quantile controller: one routing step per controller update");
  }
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  int rc = route_device(ctx, x_bf16, w_bf16, num_tokens, topk_idx, topk_gate, logits_out, alpha_out, st);
  if (rc == MOE_OK && ctx->cfg.controller == MOE_CTRL_QUANTILE) {
    ctx->qb_logits = logits_out; ctx->qb_alpha = alpha_out; ctx->qb_tokens = num_tokens;
  }
  return rc;
}

int moe_route_step_host(moe_route_ctx* ctx, const void* x_bf16_host, const void* w_bf16_host, int32_t num_tokens,
                        int32_t* topk_idx_host, float* topk_gate_host, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  const moe_route_config& c = ctx->cfg;
  if (!c.host_staging) return fail(ctx, MOE_ERR_STATE, "context was created without host_staging");
  if (c.controller == MOE_CTRL_QUANTILE) return fail(ctx, MOE_ERR_UNSUPPORTED, "host step: no quantile controller");
  if (!x_bf16_host || !topk_idx_host || !topk_gate_host) return fail(ctx, MOE_ERR_INVALID_ARG, "null host pointer");
  if (!w_bf16_host && !ctx->staged_w) return fail(ctx, MOE_ERR_STATE, "no router weights staged yet");
  if (num_tokens < 1 || num_tokens > c.max_tokens) return fail(ctx, MOE_ERR_INVALID_ARG, "num_tokens out of range");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  const size_t LT = (size_t)c.num_layers * num_tokens;
  cudaError_t e = cudaMemcpyAsync(ctx->ws + ctx->lay.stage_x, x_bf16_host, LT * c.hidden * 2, cudaMemcpyHostToDevice, st);
  if (e == cudaSuccess && w_bf16_host) {
    e = cudaMemcpyAsync(ctx->ws + ctx->lay.stage_w, w_bf16_host, (size_t)c.num_layers * c.num_experts * c.hidden * 2,
                        cudaMemcpyHostToDevice, st);
    ctx->staged_w = true;
  }
  if (e != cudaSuccess) return cuda_fail(ctx, e, "host to device copy");
  int rc = route_device(ctx, ctx->ws + ctx->lay.stage_x, ctx->ws + ctx->lay.stage_w, num_tokens,
                        at<int32_t>(ctx, ctx->lay.stage_idx), at<float>(ctx, ctx->lay.stage_gate), nullptr, nullptr, st);
  if (rc) return rc;
  e = cudaMemcpyAsync(topk_idx_host, ctx->ws + ctx->lay.stage_idx, LT * c.top_k * 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(topk_gate_host, ctx->ws + ctx->lay.stage_gate, LT * c.top_k * 4, cudaMemcpyDeviceToHost, st);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "device to host copy");
  return MOE_OK;
}

int moe_controller_update(moe_route_ctx* ctx, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  const moe_route_config& c = ctx->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  if (c.controller == MOE_CTRL_QUANTILE) {
    if (!ctx->qb_logits) return fail(ctx, MOE_ERR_STATE, "quantile controller: no routing step since the last update");
    if (c.qb_hist_bins > 0) {
      // footnote to Eq. 7: the target estimated from a per-expert margin histogram, one pass over the dump
      const size_t smem = qh_smem_bytes(c.qb_hist_bins);
      static bool attr_set[64] = {};
      if (!attr_set[ctx->device & 63]) {
        cudaError_t ae = cudaFuncSetAttribute(qb_margin_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                              (int)qh_smem_bytes(kQhMaxBins));
        if (ae != cudaSuccess) return cuda_fail(ctx, ae, "cudaFuncSetAttribute(qb_margin_hist_kernel)");
        attr_set[ctx->device & 63] = true;
      }
      const int groups = (c.num_experts + kQhCols - 1) / kQhCols;
      // one resident wave: every row split flushes its own copy of the non-empty bins, and a grid a little
      // above what is resident runs a second, almost empty wave
      if (ctx->qh_occ < 1) {
        int occ = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, qb_margin_hist_kernel, kQhThreads, smem) != cudaSuccess || occ < 1)
          occ = 1;
        ctx->qh_occ = occ;
      }
      int splits = ctx->qh_occ * ctx->num_sms / groups;
      const int max_splits = (ctx->qb_tokens + 127) / 128;
      if (splits > max_splits) splits = max_splits;
      if (splits < 1) splits = 1;
      for (int l = 0; l < c.num_layers; ++l) {
        QhParams q{};
        q.logits = ctx->qb_logits + (size_t)l * ctx->qb_tokens * c.num_experts;
        q.alpha = ctx->qb_alpha + (size_t)l * ctx->qb_tokens;
        q.m = ctx->qb_tokens; q.E = c.num_experts; q.K = c.top_k; q.B = c.qb_hist_bins;
        q.range = c.qb_hist_range;
        q.inv_h = (float)c.qb_hist_bins / (2.0f * c.qb_hist_range);
        q.edge_eps = qh_edge_eps(q.inv_h);
        q.hist = at<uint32_t>(ctx, ctx->lay.qb_hist);
        q.target = at<float>(ctx, ctx->lay.qb_target) + (size_t)l * c.num_experts;
        launch_chained(qb_margin_hist_kernel, dim3(groups, splits), dim3(kQhThreads), smem, st, q);
        launch_chained(qb_margin_hist_finish_kernel, dim3(c.num_experts), dim3(kQhFinishThreads), 0, st, q);
        ctx->launches += 2;
      }
      cudaError_t qe = cudaGetLastError();
      if (qe != cudaSuccess) return cuda_fail(ctx, qe, "margin histogram kernels launch");
      ctx->qb_logits = nullptr;
    }
    const int col_groups = (c.num_experts + kQbCols - 1) / kQbCols;
    int splits = (6 * ctx->num_sms + col_groups - 1) / col_groups;
    const int max_splits = (ctx->qb_tokens + 63) / 64;
    if (splits > max_splits) splits = max_splits;
    if (splits < 1) splits = 1;
    // Eq. 7 is per layer: the layers take turns on the one radix-select scratch (same stream, so in order)
    for (int l = 0; c.qb_hist_bins == 0 && l < c.num_layers; ++l) {
      QbParams q{};
      q.logits = ctx->qb_logits + (size_t)l * ctx->qb_tokens * c.num_experts;
      q.alpha = ctx->qb_alpha + (size_t)l * ctx->qb_tokens;
      q.m = ctx->qb_tokens; q.E = c.num_experts; q.K = c.top_k;
      q.hist = at<uint32_t>(ctx, ctx->lay.qb_hist);
      q.prefix = at<uint32_t>(ctx, ctx->lay.qb_prefix);
      q.rank = at<uint32_t>(ctx, ctx->lay.qb_rank);
      q.target = at<float>(ctx, ctx->lay.qb_target) + (size_t)l * c.num_experts;
      q.keys = at<uint32_t>(ctx, ctx->lay.qb_keys);
      q.match = at<uint32_t>(ctx, ctx->lay.qb_match);
      q.fill = at<uint32_t>(ctx, ctx->lay.qb_fill);
      q.list = at<uint16_t>(ctx, ctx->lay.qb_list);
      q.deep = at<uint32_t>(ctx, ctx->lay.qb_deep);
      launch_chained(qb_init_kernel, dim3(64), dim3(256), 0, st, q);
      // two digit passes; the third one's kernels return at once unless the second scan found a set that does not
      // fit the list
      for (int pass = 0; pass < 3; ++pass) {
        launch_chained(qb_hist_kernel, dim3(col_groups, splits), dim3(kQbThreads), 0, st, q, pass);
        launch_chained(qb_scan_kernel, dim3((c.num_experts * 32 + 255) / 256), dim3(256), 0, st, q, pass);
      }
      // the last two digits: gather the keys that share the 16-bit prefix, select among them
      launch_chained(qb_gather_kernel, dim3(col_groups, splits), dim3(kQbThreads), 0, st, q);
      launch_chained(qb_select_kernel, dim3((c.num_experts + kQbSelectWarps - 1) / kQbSelectWarps),
                     dim3(kQbSelectWarps * 32), 0, st, q);
      ctx->launches += 9;
    }
    {
      cudaError_t qe = cudaGetLastError();
      if (qe != cudaSuccess) return cuda_fail(ctx, qe, "quantile kernels launch");
    }
    ctx->qb_logits = nullptr;
  }
  CtrlParams p{};
  p.L = c.num_layers; p.E = c.num_experts; p.controller = c.controller;
  p.ki = c.ki; p.kd = c.kd; p.eta = c.eta; p.rho = c.qb_ema_rho; p.center = ctx->center_on;
  p.bias = at<float>(ctx, ctx->lay.bias);
  p.e_prev = at<float>(ctx, ctx->lay.e_prev);
  p.bias_prev = at<float>(ctx, ctx->lay.bias_prev);
  p.loads_acc = at<int>(ctx, ctx->lay.loads_acc);
  p.loads_last = at<int>(ctx, ctx->lay.loads_last);
  p.maxvio = at<float>(ctx, ctx->lay.maxvio);
  p.minvio = at<float>(ctx, ctx->lay.minvio);
  p.gate_count = at<int>(ctx, ctx->lay.gate_count);
  p.qb_target = at<float>(ctx, ctx->lay.qb_target);
  p.status = status_ptr(ctx);
  {
    // programmatic stream serialisation: the launch latency overlaps the tail of the kernel before it
    cudaLaunchConfig_t lc{};
    lc.gridDim = dim3(c.num_layers);
    lc.blockDim = dim3(kCtrlThreads);
    lc.dynamicSmemBytes = 0;
    lc.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = &attr;
    lc.numAttrs = 1;
    cudaError_t le = cudaLaunchKernelEx(&lc, controller_kernel, p);
    if (le != cudaSuccess) return cuda_fail(ctx, le, "controller_kernel launch");
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "controller_kernel launch");
  ctx->launches += 1;
  ctx->ctrl_steps += 1;
  return MOE_OK;
}

static int copy_out(moe_route_ctx* ctx, void* dst, size_t off, size_t bytes, cudaStream_t st) {
  if (!dst) return MOE_OK;
  cudaError_t e = cudaMemcpyAsync(dst, ctx->ws + off, bytes, cudaMemcpyDeviceToDevice, st);
  return e == cudaSuccess ? MOE_OK : cuda_fail(ctx, e, "device copy");
}

int moe_load_stats(moe_route_ctx* ctx, int32_t* loads, float* bias, float* maxvio, float* minvio, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  const size_t LE = (size_t)ctx->cfg.num_layers * ctx->cfg.num_experts * 4, Lb = (size_t)ctx->cfg.num_layers * 4;
  int rc = copy_out(ctx, loads, ctx->lay.loads_last, LE, st);
  if (!rc) rc = copy_out(ctx, bias, ctx->lay.bias, LE, st);
  if (!rc) rc = copy_out(ctx, maxvio, ctx->lay.maxvio, Lb, st);
  if (!rc) rc = copy_out(ctx, minvio, ctx->lay.minvio, Lb, st);
  return rc;
}

int moe_gate_stats(moe_route_ctx* ctx, int32_t* gate_count, void* cuda_stream) {
  if (!ctx || !gate_count) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  return copy_out(ctx, gate_count, ctx->lay.gate_count, (size_t)ctx->cfg.num_layers * 4, st);
}

int moe_load_diagnostics(moe_route_ctx* ctx, float* diag, void* cuda_stream) {
  if (!ctx || !diag) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  DiagParams d{};
  d.L = ctx->cfg.num_layers; d.E = ctx->cfg.num_experts;
  d.loads_last = at<int>(ctx, ctx->lay.loads_last);
  d.gate_count = at<int>(ctx, ctx->lay.gate_count);
  d.bias = at<float>(ctx, ctx->lay.bias);
  d.bias_prev = at<float>(ctx, ctx->lay.bias_prev);
  d.out = diag;
  launch_chained(diagnostics_kernel, dim3(d.L), dim3(kCtrlThreads), 0, st, d);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "diagnostics_kernel launch");
  ctx->launches += 1;
  return MOE_OK;
}

int moe_gate_entropy(moe_route_ctx* ctx, const float* topk_gate, int32_t num_tokens, float* entropy, void* cuda_stream) {
  if (!ctx || !topk_gate || !entropy) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (num_tokens < 1) return fail(ctx, MOE_ERR_INVALID_ARG, "num_tokens must be positive");
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  double* part = at<double>(ctx, ctx->lay.ent_part);
  launch_chained(gate_entropy_kernel, dim3(kEntropySlices, ctx->cfg.num_layers), dim3(kEntropyThreads), 0, st, topk_gate,
                 num_tokens, ctx->cfg.top_k, part);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "gate_entropy_kernel launch");
  launch_chained(gate_entropy_finish_kernel, dim3(ctx->cfg.num_layers), dim3(32), 0, st, part, num_tokens, entropy);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "gate_entropy_finish_kernel launch");
  ctx->launches += 2;
  return MOE_OK;
}

int moe_score_stats(moe_route_ctx* ctx, const float* logits, int32_t num_tokens, const int32_t* loads,
                    float* entropy_biased, float* entropy_softmax, float* mean_prob, float* aux, void* cuda_stream) {
  if (!ctx || !logits) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (num_tokens < 1) return fail(ctx, MOE_ERR_INVALID_ARG, "num_tokens must be positive");
  if (aux && !loads) return fail(ctx, MOE_ERR_INVALID_ARG, "aux needs the loads of the same tokens");
  if (reinterpret_cast<uintptr_t>(logits) % 16 != 0) return fail(ctx, MOE_ERR_INVALID_ARG, "logits must be 16-byte aligned");
  const moe_route_config& c = ctx->cfg;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  StatParams p{};
  p.logits = logits;
  p.bias = at<float>(ctx, ctx->lay.bias);
  p.L = c.num_layers; p.T = num_tokens; p.E = c.num_experts; p.C = stat_ctas_per_layer(c.num_layers);
  p.part_P = at<float>(ctx, ctx->lay.stat_P);
  p.part_H = at<float>(ctx, ctx->lay.stat_H);
  p.aux_part = at<double>(ctx, ctx->lay.stat_aux);
  p.arrivals = at<unsigned int>(ctx, ctx->lay.stat_cnt);
  p.loads = loads; p.h_biased = entropy_biased; p.h_softmax = entropy_softmax; p.mean_prob = mean_prob; p.aux = aux;
  const dim3 grid(p.C, p.L);
  {
    const int nv = p.E <= 256 ? 2 : p.E <= 512 ? 4 : p.E <= 768 ? 6 : 8;
    const bool full = (p.E == 128 * nv);
    void (*kern)(StatParams) =
        nv == 2 ? (full ? score_stats_kernel<2, true> : score_stats_kernel<2, false>)
      : nv == 4 ? (full ? score_stats_kernel<4, true> : score_stats_kernel<4, false>)
      : nv == 6 ? (full ? score_stats_kernel<6, true> : score_stats_kernel<6, false>)
                : (full ? score_stats_kernel<8, true> : score_stats_kernel<8, false>);
    static bool attr_set[64][8] = {};
    bool& done = attr_set[ctx->device & 63][(nv / 2 - 1) * 2 + (full ? 1 : 0)];
    if (!done) {
      cudaError_t ae = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)stat_smem_bytes(nv));
      if (ae != cudaSuccess) return cuda_fail(ctx, ae, "cudaFuncSetAttribute(score_stats_kernel)");
      done = true;
    }
    launch_chained(kern, grid, dim3(kStatThreads), stat_smem_bytes(nv), st, p);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "score_stats_kernel launch");
  const int groups = (p.E + kStatFinExperts - 1) / kStatFinExperts;
  launch_chained(score_stats_finish_kernel, dim3(groups, p.L), dim3(1024), 0, st, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "score_stats_finish_kernel launch");
  ctx->launches += 2;
  return MOE_OK;
}

int moe_loads_peek(moe_route_ctx* ctx, int32_t* loads, void* cuda_stream) {
  if (!ctx || !loads) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  return copy_out(ctx, loads, ctx->lay.loads_acc, (size_t)ctx->cfg.num_layers * ctx->cfg.num_experts * 4, st);
}

int moe_loads_buffer(moe_route_ctx* ctx, int32_t** dev_loads) {
  if (!ctx || !dev_loads) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  *dev_loads = at<int32_t>(ctx, ctx->lay.loads_acc);
  return MOE_OK;
}

int moe_loads_add(moe_route_ctx* ctx, const int32_t* loads, void* cuda_stream) {
  if (!ctx || !loads) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  const int n = ctx->cfg.num_layers * ctx->cfg.num_experts;
  launch_chained(loads_add_kernel, dim3((n + 255) / 256), dim3(256), 0, st, at<int>(ctx, ctx->lay.loads_acc), loads, n);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "loads_add_kernel launch");
  ctx->launches += 1;
  return MOE_OK;
}

int moe_state_export(moe_route_ctx* ctx, float* bias, float* e_prev, int64_t* step_host, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (step_host) *step_host = ctx->ctrl_steps;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  const size_t LE = (size_t)ctx->cfg.num_layers * ctx->cfg.num_experts * 4;
  int rc = copy_out(ctx, bias, ctx->lay.bias, LE, st);
  if (!rc) rc = copy_out(ctx, e_prev, ctx->lay.e_prev, LE, st);
  return rc;
}

int moe_state_import(moe_route_ctx* ctx, const float* bias, const float* e_prev, int64_t step, void* cuda_stream) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  if (step < -1) return fail(ctx, MOE_ERR_INVALID_ARG, "step must be >= 0 (or -1 to keep the counter)");
  if (step >= 0) ctx->ctrl_steps = step;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  const size_t LE = (size_t)ctx->cfg.num_layers * ctx->cfg.num_experts * 4;
  cudaError_t e = cudaSuccess;
  if (bias) e = cudaMemcpyAsync(ctx->ws + ctx->lay.bias, bias, LE, cudaMemcpyDeviceToDevice, st);
  if (e == cudaSuccess && e_prev) e = cudaMemcpyAsync(ctx->ws + ctx->lay.e_prev, e_prev, LE, cudaMemcpyDeviceToDevice, st);
  return e == cudaSuccess ? MOE_OK : cuda_fail(ctx, e, "device copy");
}

int moe_route_poll(moe_route_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  cudaError_t e = cudaStreamSynchronize(ctx->last_stream);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
  int st[2] = {0, 0};
  e = cudaMemcpy(st, status_ptr(ctx), sizeof st, cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(ctx, e, "status read");
#ifdef MOE_DEBUG
  for (int g = 0; g < ctx->lay.num_guards && st[0] == MOE_OK; ++g) {
    unsigned char canary[kAlign];
    if (cudaMemcpy(canary, ctx->ws + ctx->lay.guard[g], kAlign, cudaMemcpyDeviceToHost) != cudaSuccess)
      return cuda_fail(ctx, cudaGetLastError(), "canary read");
    for (size_t i = 0; i < kAlign; ++i)
      if (canary[i] != kCanaryByte)
        return fail(ctx, MOE_ERR_INTERNAL, "workspace canary %d (offset %zu) overwritten at byte %zu", g,
                    ctx->lay.guard[g], i);
  }
#endif
  if (st[0] != MOE_OK) {
    cudaMemset(status_ptr(ctx), 0, sizeof st);
    if (st[0] == MOE_ERR_TIMEOUT) {
      // the step that gave up is void: its outputs are incomplete and whatever it (and earlier microbatches of
      // the same step) counted is dropped, so a later controller update cannot consume a partial histogram
      cudaMemset(ctx->ws + ctx->lay.loads_acc, 0, (size_t)ctx->cfg.num_layers * ctx->cfg.num_experts * 4);
      ctx->qb_logits = nullptr;
      return fail(ctx, MOE_ERR_TIMEOUT, "a bounded device-side wait expired (wait id %d); load accumulators cleared", st[1]);
    }
    if (st[0] == MOE_ERR_STATE)
      return fail(ctx, MOE_ERR_STATE, "controller update on a layer with no routed tokens");
    if (st[0] == MOE_ERR_INTERNAL)
      return fail(ctx, MOE_ERR_INTERNAL, "debug build: index guard %d of the routing kernel tripped", st[1] - 1000);
    return fail(ctx, st[0], "device status %d", st[0]);
  }
  return MOE_OK;
}

// grid-stride sweep over all 2^32 fp32 bit patterns (NaN and infinities skipped)
__global__ void score_gap_kernel(unsigned int* out) {
  float worst = 0.0f;
  const unsigned long long n = 1ull << 32;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned int bits = (unsigned int)i;
    if ((bits & 0x7f800000u) == 0x7f800000u) continue;
    const float z = __uint_as_float(bits);
    worst = fmaxf(worst, fabsf(moe::approx_score(z) - moe::sigmoid_score(z)));
  }
  for (int d = 16; d > 0; d >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, d));
  if ((threadIdx.x & 31) == 0) atomicMax(out, __float_as_uint(worst));
}

// out[0]: number of binary32 inputs (all 2^32 bit patterns) for which the score chain with the branch-free
// reciprocal differs in any bit from the chain with the library's correctly rounded reciprocal;
// out[1]: number of normal d in [2^-126, 2^126] for which rcp_rn_normal(d) differs from __frcp_rn(d)
__global__ void rcp_check_kernel(unsigned int* out) {
  unsigned int bad_score = 0, bad_rcp = 0;
  const unsigned long long n = 1ull << 32;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned int bits = (unsigned int)i;
    const float z = __uint_as_float(bits);
    if (__float_as_uint(moe::sigmoid_score_t<false>(z)) != __float_as_uint(moe::sigmoid_score_t<true>(z))) bad_score += 1;
    const unsigned int ex = (bits >> 23) & 0xffu;
    if (ex >= 1u && ex <= 252u && !(ex == 252u && (bits & 0x7fffffu) != 0u)) {     // |d| in [2^-126, 2^126]
      if (__float_as_uint(moe::rcp_rn_normal(z)) != __float_as_uint(__frcp_rn(z))) bad_rcp += 1;
    }
  }
  for (int d = 16; d > 0; d >>= 1) {
    bad_score += __shfl_xor_sync(0xffffffffu, bad_score, d);
    bad_rcp += __shfl_xor_sync(0xffffffffu, bad_rcp, d);
  }
  if ((threadIdx.x & 31) == 0) {
    if (bad_score) atomicAdd(&out[0], bad_score);
    if (bad_rcp) atomicAdd(&out[1], bad_rcp);
  }
}

int moe_debug_rcp_check(uint32_t* dev_result, void* cuda_stream) {
  if (!dev_result) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(dev_result, 0, 2 * sizeof(uint32_t), st) != cudaSuccess) return MOE_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return MOE_ERR_CUDA;
  rcp_check_kernel<<<sms * 8, 256, 0, st>>>(dev_result);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

// out[0]: pairs (a, b) for which div_rn_by differs from __fdiv_rn.  b runs over every binary32 number in
// [2^-20, 32]; for each b, 48 numerators a in (0, b]: b scaled by factors just below 1 and by pseudo-random
// factors over 40 binades (the shapes a gate has: one score over a sum that contains it).
__global__ void division_check_kernel(unsigned int* out) {
  unsigned int bad = 0;
  const unsigned int b_lo = 0x35800000u /* 2^-20 */, b_hi = 0x42000000u /* 32 */;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x + b_lo; i <= b_hi;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const float b = __uint_as_float((unsigned int)i);
    const float r = moe::rcp_rn_normal(b);
    unsigned int h = (unsigned int)i * 2654435761u + 12345u;
    for (int k = 0; k < 48; ++k) {
      h = h * 1664525u + 1013904223u;
      float a;
      if (k < 8) a = b * (1.0f - (float)k * 5.9604645e-8f);                       // just below b
      else if (k < 16) a = __uint_as_float(((unsigned int)i & 0xff800000u) | (h >> 9));   // same binade, random mantissa
      else a = b * __uint_as_float(((87u + (h >> 27)) << 23) | (h & 0x7fffffu));  // b * [2^-40, 2^-8)
      if (!(a > 0.0f) || a > b || !moe::gate_division_safe(a, b)) continue;
      if (__float_as_uint(moe::div_rn_by(a, b, r)) != __float_as_uint(__fdiv_rn(a, b))) bad += 1;
    }
  }
  for (int d = 16; d > 0; d >>= 1) bad += __shfl_xor_sync(0xffffffffu, bad, d);
  if ((threadIdx.x & 31) == 0 && bad) atomicAdd(&out[0], bad);
}

int moe_debug_division_check(uint32_t* dev_result, void* cuda_stream) {
  if (!dev_result) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(dev_result, 0, sizeof(uint32_t), st) != cudaSuccess) return MOE_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return MOE_ERR_CUDA;
  division_check_kernel<<<sms * 8, 256, 0, st>>>(dev_result);
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

__global__ void quick_score_gap_kernel(unsigned int* out) {
  float worst = 0.0f;
  const unsigned long long n = 1ull << 32;
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned int bits = (unsigned int)i;
    if ((bits & 0x7f800000u) == 0x7f800000u) continue;
    const float z = __uint_as_float(bits);
    worst = fmaxf(worst, fabsf(moe::quick_score(z) - moe::sigmoid_score(z)));
  }
  for (int d = 16; d > 0; d >>= 1) worst = fmaxf(worst, __shfl_xor_sync(0xffffffffu, worst, d));
  if ((threadIdx.x & 31) == 0) atomicMax(out, __float_as_uint(worst));
}

int moe_debug_quick_score_gap(float* dev_result, void* cuda_stream) {
  if (!dev_result) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(dev_result, 0, sizeof(float), st) != cudaSuccess) return MOE_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return MOE_ERR_CUDA;
  quick_score_gap_kernel<<<sms * 8, 256, 0, st>>>(reinterpret_cast<unsigned int*>(dev_result));
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_debug_score_gap(float* dev_result, void* cuda_stream) {
  if (!dev_result) return MOE_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemsetAsync(dev_result, 0, sizeof(float), st) != cudaSuccess) return MOE_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
    return MOE_ERR_CUDA;
  score_gap_kernel<<<sms * 8, 256, 0, st>>>(reinterpret_cast<unsigned int*>(dev_result));
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

#ifdef MOE_KERNEL_TIMERS
// debug builds only: cycle accounting of the route kernel, 32 counters, optionally reset
int moe_debug_read_marks(unsigned long long* host_out) {
  cudaDeviceSynchronize();
  return cudaMemcpyFromSymbol(host_out, moe::g_route_marks, sizeof(unsigned long long) * 32) == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_debug_read_timers(long long* host_out, int reset) {
  cudaDeviceSynchronize();
  if (host_out && cudaMemcpyFromSymbol(host_out, moe::g_route_timers, sizeof(long long) * 32) != cudaSuccess)
    return MOE_ERR_CUDA;
  if (reset) {
    long long z[32] = {0};
    z[24] = 0x7fffffffffffffffll;   // running minimum of the CTA start times
    if (cudaMemcpyToSymbol(moe::g_route_timers, z, sizeof z) != cudaSuccess) return MOE_ERR_CUDA;
  }
  return MOE_OK;
}
#endif

// One warp waits, with the routing kernel's bounded wait, on an mbarrier phase that nothing completes.
__global__ void wait_timeout_probe_kernel(int* status, uint32_t spin_limit) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    moe::ptx::mbar_init(moe::ptx::smem_u32(&bar), 1);
    abort_flag = 0;
    moe::ptx::fence_mbar_init();
  }
  __syncthreads();
  moe::WaitCtl wc{&abort_flag, status, spin_limit};
  const bool ok = moe::wait_phase(moe::ptx::smem_u32(&bar), 0u, wc, 99);
  if (ok && threadIdx.x == 0) status[1] = -1;   // must not happen: nobody arrives on the barrier
}

int moe_debug_wait_timeout(moe_route_ctx* ctx, int32_t spin_limit, void* cuda_stream) {
  if (!ctx || spin_limit < 1) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  ctx->last_stream = st;
  wait_timeout_probe_kernel<<<1, 32, 0, st>>>(status_ptr(ctx), (uint32_t)spin_limit);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(ctx, e, "wait_timeout_probe_kernel launch");
  ctx->launches += 1;
  return MOE_OK;
}

int moe_debug_route_stall(moe_route_ctx* ctx, int32_t after_loads) {
  if (!ctx || after_loads < 1) return MOE_ERR_INVALID_ARG;
  ctx->err[0] = 0;
  ctx->stall_next = after_loads;
  return MOE_OK;
}

int moe_quantile_target_static(const float* logits, const float* alpha, int32_t num_tokens, int32_t num_experts,
                               int32_t top_k, float* target_out, void* cuda_stream) {
  if (!logits || !alpha || !target_out) return MOE_ERR_INVALID_ARG;
  if (num_tokens < 1 || num_experts < 1 || top_k < 1 || top_k >= num_experts) return MOE_ERR_INVALID_ARG;
  if (num_experts > kStaticMaxExperts) return MOE_ERR_WORKSPACE;   // beyond the built-in scratch
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return MOE_ERR_CUDA;
  if (dev < 0 || dev >= kStaticMaxDevices) return MOE_ERR_UNSUPPORTED;
  {
    // once per device, with that device current: turn the host-side stand-in of the array into its
    // device address (the symbol itself is not a device pointer and must never reach a kernel argument)
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (g_static_scratch_dev[dev] == nullptr) {
      void* ptr = nullptr;
      cudaError_t e = cudaGetSymbolAddress(&ptr, moe_static_quantile_scratch);
      if (e != cudaSuccess || ptr == nullptr) return MOE_ERR_CUDA;
      int sms = 0;
      if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
        return MOE_ERR_CUDA;
      g_static_sms[dev] = sms;
      g_static_scratch_dev[dev] = ptr;
    }
  }
  uint8_t* base = static_cast<uint8_t*>(g_static_scratch_dev[dev]);
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  QbParams q{};
  q.logits = logits; q.alpha = alpha; q.m = num_tokens; q.E = num_experts; q.K = top_k;
  q.hist = reinterpret_cast<uint32_t*>(base);
  q.prefix = reinterpret_cast<uint32_t*>(base + (size_t)kStaticMaxExperts * 256 * 4);
  q.rank = q.prefix + kStaticMaxExperts;
  q.target = target_out;
  // the array keeps whatever the previous call left: the init kernel clears the histogram and
  // resets prefix and rank before anything is counted
  launch_chained(qb_init_kernel, dim3(64), dim3(256), 0, st, q);
  const int col_groups = (num_experts + kQbCols - 1) / kQbCols;
  int splits = (6 * g_static_sms[dev] + col_groups - 1) / col_groups;
  const int max_splits = (num_tokens + 63) / 64;
  if (splits > max_splits) splits = max_splits;
  if (splits < 1) splits = 1;
  for (int pass = 0; pass < 4; ++pass) {
    launch_chained(qb_hist_kernel, dim3(col_groups, splits), dim3(kQbThreads), 0, st, q, pass);
    launch_chained(qb_scan_kernel, dim3((num_experts * 32 + 255) / 256), dim3(256), 0, st, q, pass);
  }
  return cudaGetLastError() == cudaSuccess ? MOE_OK : MOE_ERR_CUDA;
}

int moe_debug_build(void) {
#ifdef MOE_DEBUG
  return 1;
#else
  return 0;
#endif
}

int64_t moe_route_launch_count(const moe_route_ctx* ctx) { return ctx ? ctx->launches : 0; }

const char* moe_last_error(const moe_route_ctx* ctx) { return ctx ? ctx->err : "null context"; }

int moe_route_destroy(moe_route_ctx* ctx) {
  if (!ctx) return MOE_ERR_INVALID_ARG;
  delete ctx;
  return MOE_OK;
}

}  // extern "C"
