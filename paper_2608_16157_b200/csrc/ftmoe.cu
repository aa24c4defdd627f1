// Host side of the C ABI declared in include/ftmoe.h: handle, validation, launches, streams, events.
#include "../../include/ftmoe.h"

#include <cuda_runtime.h>

#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"
#include "ffn_stream.cuh"
#include "dequant_w4.cuh"
#include "ffn_mx4.cuh"
#include "ffn_mx4tc.cuh"
#include "ffn_w4.cuh"
#include "ffn_w4_half.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc2.cuh"
#include "fill.cuh"
#include "route_plan.cuh"

using namespace ftmoe;

namespace {

enum LayerPhase { PH_IDLE = 0, PH_ROUTED, PH_PLANNED, PH_FILLED };
constexpr int kFinalizeInKernelMaxTokens = 16;
constexpr int kMaxTableSlots = 6144;   // slots of one residency table (per layer, or the shared pool)

struct LayerState {
  int32_t *slot_expert = nullptr;
  int64_t *slot_stamp = nullptr;
  int32_t *expert_slot = nullptr;
  int64_t *step = nullptr;     // plan calls of this layer
  int64_t *clock = nullptr;    // the LRU clock the layer's plans advance (its own step counter, or the shared one)
  unsigned long long *stats = nullptr;
  int phase = PH_IDLE;
  int T = 0;
  uint32_t seq = 0;            // plans launched for this layer (stale-record check of the host mirror)
  cudaEvent_t ev_fill = nullptr;   // recorded on the copy stream after the layer's latest fills (or whole-layer prefetch)
  bool fill_recorded = false;
};

// Per-layer scratch: the routing arrays, the plan record and the work lists of the layer's latest step.  Every
// layer has its own set, so route/plan/fill of several layers may be issued before their forward calls.
struct Scratch {
  int32_t *ids, *count, *offset, *perm, *inv;
  float *topk_w;
  PlanHeader *plan_dev, *plan_host, *plan_host_devptr;
  WorkItem *items_res, *items_zc, *items_gemm;
  int32_t *res_pref, *gemm_pref;
  uint8_t *is_gemm;
};

}  // namespace

struct ft_moe {
  ft_moe_config_t cfg;
  size_t S = 0;
  int sm_count = 148;
  // memory
  uint8_t *slots = nullptr;         // [L][N_s][S]
  uint8_t *shared_dev = nullptr;    // [L][n_shared][S]
  const uint8_t *pool_dev = nullptr;  // device alias of host_pool
  uint8_t *tables = nullptr;        // one allocation for all tables (per layer, or shared by all layers)
  size_t tables_bytes = 0;
  uint8_t *stats_mem = nullptr;     // per-layer step counters and statistics (survive a resize)
  int table_slots = 0;              // slots per table: slots_per_layer, or n_layers*slots_per_layer when shared
  std::vector<LayerState> layers;
  // scratch: one set per layer (see Scratch), allocated as [L] x stride arrays
  size_t pair_stride = 0, plan_stride = 0;   // bytes per layer of the pair arrays / the plan record
  int32_t *ids = nullptr, *count = nullptr, *offset = nullptr, *perm = nullptr, *inv = nullptr;
  float *topk_w = nullptr;
  int32_t *route_hist = nullptr;        // [blocks of tokens][E] histograms of the blocked route / permute kernels
  float *y_acc = nullptr;
  PlanHeader *plan_dev = nullptr;
  PlanHeader *plan_host = nullptr;      // pinned, mapped
  PlanHeader *plan_host_devptr = nullptr;
  size_t plan_bytes = 0;
  WorkItem *items_res = nullptr, *items_zc = nullptr, *items_gemm = nullptr;
  int32_t *res_pref = nullptr;
  bool plan_mirrored = false;
  // prefill (grouped GEMM) path, allocated only when gemm_min_tokens > 0
  bool gemm = false;
  int32_t *gemm_pref = nullptr;
  uint8_t *is_gemm = nullptr;
  __nv_bfloat16 *xs = nullptr, *hbuf = nullptr, *obuf = nullptr;   // [P][d], [P][I], [P][d]
  CUtensorMap tm_xs, tm_h;       // x rows, H rows (128-row boxes, 128-byte swizzle)
  CUtensorMap tm_wgu, tm_wd;     // the slot pool as [unit][1 KiB gate/up tile] and [unit][2 KiB of down tiles]
  uint8_t *wq_scratch = nullptr; // 4-bit experts on the GEMM path: [slots_per_layer] bf16 records (tile order) of the call's layer
  uint32_t *status_dev = nullptr;
  uint32_t *seq_dev = nullptr;
  uint32_t *done_dev = nullptr;          // CTA completion counter of the streaming MMA kernel
  long long *trace_dev = nullptr;        // per-CTA clocks of the latest streaming-kernel launch
  // int4 path: h as fp32 [pass][16-neuron unit][token 8][neuron 16]; arrival counters, fixed-point h and its
  // (scale, bias) per (pass, 128-neuron group)
  float *w4_hraw = nullptr;
  int32_t *w4_hcount = nullptr;
  uint8_t *w4_hq = nullptr;
  uint8_t *tc_xq = nullptr;      // FT_W_MXFP4_TC: the bit-sliced activation images of a call
  int *tc_pass_done = nullptr;   // FT_W_MXFP4_TC: per pass, the groups whose h is written (hand-over between the two kernels)
  int *tc_gen = nullptr;         // FT_W_MXFP4_TC: cumulative counts of finished gate/up and down CTAs
  uint32_t tc_calls = 0;         // FT_W_MXFP4_TC: forward calls so far
  float2 *w4_hs = nullptr;
  int last_fill_layer = -1;
  int overlap = 0;                      // launch mode of the streaming kernel (see FfnStreamParams::overlap)
  float *stage_logits = nullptr;
  __nv_bfloat16 *stage_x = nullptr, *stage_y = nullptr;
  // streams / events
  cudaStream_t copy_stream = nullptr, aux_stream = nullptr;
  cudaEvent_t ev_plan = nullptr, ev_fill = nullptr, ev_fork = nullptr, ev_join = nullptr;
  cudaEvent_t ev_fill_t0 = nullptr, ev_fill_t1 = nullptr;
  uint64_t last_fill_bytes = 0;
  bool fill_timed = false;
  uint64_t launches = 0;
  // optional per-kernel timing (CUDA events on the launching stream)
  bool timing = false;
  struct Pending { int kind; cudaEvent_t e0, e1; };
  std::vector<Pending> pending;
  std::vector<cudaEvent_t> free_events;
  double time_us[FT_TIME_COUNT] = {0};
  uint64_t time_n[FT_TIME_COUNT] = {0};
};

namespace {

cudaError_t g_last_cuda_error = cudaSuccess;   // the CUDA error behind the latest FT_ERR_CUDA / FT_ERR_OOM

#define FT_CUDA(expr)                                                                     \
  do {                                                                                    \
    cudaError_t e_ = (expr);                                                              \
    if (e_ != cudaSuccess) {                                                              \
      g_last_cuda_error = e_;                                                             \
      if (e_ == cudaErrorMemoryAllocation) { (void)cudaGetLastError(); return FT_ERR_OOM; } \
      return FT_ERR_CUDA;                                                                 \
    }                                                                                     \
  } while (0)

Scratch scratch_of(const ft_moe *h, int layer) {
  const size_t E = h->cfg.n_experts, l = (size_t)layer;
  auto at = [&](auto *base, size_t bytes_per_layer) {
    using T = decltype(base);
    return base ? reinterpret_cast<T>(reinterpret_cast<uint8_t *>(base) + l * bytes_per_layer) : base;
  };
  Scratch s;
  s.ids = at(h->ids, h->pair_stride); s.perm = at(h->perm, h->pair_stride); s.inv = at(h->inv, h->pair_stride);
  s.topk_w = at(h->topk_w, h->pair_stride);
  s.count = at(h->count, E * 4); s.offset = at(h->offset, (E + 1) * 4);
  s.plan_dev = at(h->plan_dev, h->plan_stride);
  s.plan_host = at(h->plan_host, h->plan_stride);
  s.plan_host_devptr = at(h->plan_host_devptr, h->plan_stride);
  s.items_res = at(h->items_res, (2 * E + 1) * sizeof(WorkItem));
  s.items_zc = at(h->items_zc, E * sizeof(WorkItem));
  s.items_gemm = at(h->items_gemm, E * sizeof(WorkItem));
  s.res_pref = at(h->res_pref, (2 * E + 2) * 4);
  s.gemm_pref = at(h->gemm_pref, (E + 1) * 4);
  s.is_gemm = at(h->is_gemm, E);
  return s;
}

size_t expert_bytes_of(const ft_moe_config_t *c) {
  if (!c || c->hidden <= 0 || c->inter <= 0) return 0;
  const size_t d = (size_t)c->hidden, I = (size_t)c->inter;
  if (c->wdtype == FT_W_BF16) {
    if ((d != 256 && d != 512 && d != 1024 && d != 2048) || I % 16) return 0;
    return 3 * I * d * 2;
  }
  if (c->wdtype == FT_W_MXFP4 || c->wdtype == FT_W_MXFP4_TC) {
    if (d % 512 || d > 8192 || I % 128) return 0;   // (same shapes as int4)
    return 3 * I * d / 2 + 3 * I * d / 32;
  }
  if (c->wdtype == FT_W_NVFP4) {
    if (d % 512 || d > 8192 || I % 128) return 0;   // (same shapes as int4)
    return 3 * I * d / 2 + 3 * I * d / 16 + 256;
  }
  if (c->wdtype == FT_W_INT4_G128) {
    if (d % 512 || d > 8192 || I % 128) return 0;   // (the kernels further restrict d, see w4_shape_ok)
    return 3 * I * d / 2 + (2 * I * (d / 128) + (I / 128) * d) * 2;
  }
  return 0;
}

// shapes the int4 kernels are instantiated for
bool w4_shape_ok(const ft_moe_config_t &c) {
  const int d = c.hidden;
  return (d == 512 || d == 1024 || d == 2048 || d == 4096 || d == 7168 || d == 8192) && c.inter % 128 == 0;
}

ft_status_t drain_status(ft_moe *h) {
  uint32_t st = 0;
  FT_CUDA(cudaMemcpy(&st, h->status_dev, sizeof(st), cudaMemcpyDeviceToHost));
  if (st) {
    FT_CUDA(cudaMemset(h->status_dev, 0, sizeof(st)));
    if (st & kStatNonFinite) return FT_ERR_NONFINITE;
    if (st & kStatTimeout) return FT_ERR_TIMEOUT;
    return FT_ERR_CUDA;
  }
  return FT_OK;
}

cudaEvent_t timing_event(ft_moe *h) {
  if (!h->free_events.empty()) {
    cudaEvent_t e = h->free_events.back();
    h->free_events.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

void timing_flush(ft_moe *h) {
  for (auto &p : h->pending) {
    float ms = 0.f;
    if (cudaEventSynchronize(p.e1) == cudaSuccess && cudaEventElapsedTime(&ms, p.e0, p.e1) == cudaSuccess) {
      h->time_us[p.kind] += (double)ms * 1000.0;
      h->time_n[p.kind] += 1;
    }
    h->free_events.push_back(p.e0);
    h->free_events.push_back(p.e1);
  }
  h->pending.clear();
  (void)cudaGetLastError();
}

// Brackets the launches issued in its lifetime on `st` with two events when timing is on.
struct TimeScope {
  ft_moe *h;
  cudaStream_t st;
  int kind;
  cudaEvent_t e0 = nullptr;
  TimeScope(ft_moe *h_, cudaStream_t st_, int kind_) : h(h_), st(st_), kind(kind_) {
    if (h->timing) {
      if (h->pending.size() >= 4096) timing_flush(h);
      e0 = timing_event(h);
      cudaEventRecord(e0, st);
    }
  }
  ~TimeScope() {
    if (e0) {
      cudaEvent_t e1 = timing_event(h);
      cudaEventRecord(e1, st);
      h->pending.push_back({kind, e0, e1});
    }
  }
};

// Empties the residency tables `l` uses (with a shared pool: everybody's) and, unless keep_counters, the layer's
// step counter and statistics.
ft_status_t reset_layer(ft_moe *h, int l, bool keep_counters = false) {
  LayerState &L = h->layers[l];
  const int Ns = h->table_slots, E = h->cfg.n_experts;
  if (Ns > 0) {
    FT_CUDA(cudaMemset(L.slot_expert, 0xff, sizeof(int32_t) * Ns));
    FT_CUDA(cudaMemset(L.slot_stamp, 0xff, sizeof(int64_t) * Ns));
  }
  FT_CUDA(cudaMemset(h->cfg.global_pool ? L.expert_slot + (size_t)l * E : L.expert_slot, 0xff, sizeof(int32_t) * E));
  if (!keep_counters) {
    FT_CUDA(cudaMemset(L.step, 0, sizeof(int64_t)));
    FT_CUDA(cudaMemset(L.stats, 0, sizeof(unsigned long long) * FT_STAT_COUNT));
  }
  L.phase = PH_IDLE;
  L.T = 0;
  return FT_OK;
}

// (Re)allocates the slot pool and the residency tables for h->cfg.slots_per_layer and empties them.
ft_status_t alloc_cache(ft_moe *h) {
  const ft_moe_config_t &c = h->cfg;
  const size_t E = c.n_experts, Ns = c.slots_per_layer, L = c.n_layers;
  cudaFree(h->slots); h->slots = nullptr;
  cudaFree(h->tables); h->tables = nullptr;
  (void)cudaGetLastError();
  h->table_slots = c.global_pool ? (int)(L * Ns) : (int)Ns;
  if (Ns > 0) FT_CUDA(cudaMalloc(&h->slots, L * Ns * h->S));
  auto up = [](size_t v) { return (v + 255) & ~(size_t)255; };
  if (c.global_pool) {
    // one table for all layers, keyed by the flattened id layer*E + expert; one clock
    const size_t Nt = L * Ns;
    h->tables_bytes = up(Nt * 4) + up(Nt * 8) + up(L * E * 4) + up(8);
    FT_CUDA(cudaMalloc(&h->tables, h->tables_bytes));
    uint8_t *b = h->tables;
    int32_t *se = reinterpret_cast<int32_t *>(b); b += up(Nt * 4);
    int64_t *ss = reinterpret_cast<int64_t *>(b); b += up(Nt * 8);
    int32_t *es = reinterpret_cast<int32_t *>(b); b += up(L * E * 4);
    int64_t *clock = reinterpret_cast<int64_t *>(b);
    FT_CUDA(cudaMemset(clock, 0, 8));
    for (size_t l = 0; l < L; ++l) {
      LayerState &ls = h->layers[l];
      ls.slot_expert = se; ls.slot_stamp = ss; ls.expert_slot = es; ls.clock = clock;
    }
  } else {
    const size_t per_layer = up(Ns * 4) + up(Ns * 8) + up(E * 4);
    h->tables_bytes = per_layer * L;
    FT_CUDA(cudaMalloc(&h->tables, h->tables_bytes));
    for (size_t l = 0; l < L; ++l) {
      uint8_t *b = h->tables + l * per_layer;
      LayerState &ls = h->layers[l];
      ls.slot_expert = reinterpret_cast<int32_t *>(b); b += up(Ns * 4);
      ls.slot_stamp = reinterpret_cast<int64_t *>(b); b += up(Ns * 8);
      ls.expert_slot = reinterpret_cast<int32_t *>(b);
      ls.clock = ls.step;     // the layer's own step counter is its LRU clock
    }
  }
  for (size_t l = 0; l < L; ++l) {
    ft_status_t rc = reset_layer(h, (int)l, true);
    if (rc != FT_OK) return rc;
  }
  // (the limit belongs to the function on this device, not to the handle: always the largest table)
  FT_CUDA(cudaFuncSetAttribute(plan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxTableSlots * 16));
  FT_CUDA(cudaFuncSetAttribute(route_plan_small_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxTableSlots * 16));
  return FT_OK;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 row-major tensor [rows][cols] with a [box_rows][box_cols] tile, 128-byte swizzle.
bool make_tensor_map(EncodeTiledFn fn, CUtensorMap *tm, void *base, uint64_t rows, uint64_t cols, uint32_t box_rows,
                     uint32_t box_cols) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {box_cols, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
         CUDA_SUCCESS;
}

// The slot pool as a 3-D tensor of 8-byte words: [16-neuron unit][piece of `piece_bytes` inside the unit][words of
// the piece]; a box is `box_pieces` consecutive pieces of `box_units` consecutive units.
bool make_unit_map(EncodeTiledFn fn, CUtensorMap *tm, void *base, uint64_t n_units, uint64_t unit_bytes,
                   uint32_t piece_bytes, uint32_t box_pieces, uint32_t box_units) {
  const cuuint64_t dims[3] = {piece_bytes / 8, unit_bytes / piece_bytes, n_units};
  const cuuint64_t strides[2] = {piece_bytes, unit_bytes};
  const cuuint32_t box[3] = {piece_bytes / 8, box_pieces, box_units};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 3, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) ==
         CUDA_SUCCESS;
}

// Tensor maps of the weight operands of the prefill GEMMs over the current slot pool.
ft_status_t build_weight_maps(ft_moe *h) {
  const ft_moe_config_t &c = h->cfg;
  void *fnp = nullptr;
  cudaDriverEntryPointQueryResult qres;
  FT_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres));
  if (!fnp || qres != cudaDriverEntryPointSuccess) return FT_ERR_CUDA;
  EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fnp);
  // bf16 experts are read from their slots; 4-bit experts from the bf16 scratch records of the call's layer
  const bool scratch = c.wdtype != FT_W_BF16;
  const uint64_t n_units = (uint64_t)(scratch ? 1 : c.n_layers) * c.slots_per_layer * (c.inter / 16);
  const uint64_t unit_bytes = 96ull * c.hidden;
  uint8_t *base = scratch ? h->wq_scratch : h->slots;
  if (n_units == 0) return FT_OK;   // no slots: nothing goes through the GEMMs
  // gate/up: one 1 KiB tile (16 neurons x 32 hidden indices) of 8 consecutive units = 128 neurons;
  // down: 4 KiB (the tiles of 128 output columns) of 4 consecutive units = 64 neurons
  if (!make_unit_map(enc, &h->tm_wgu, base, n_units, unit_bytes, 1024, 1, 8) ||
      !make_unit_map(enc, &h->tm_wd, base, n_units, unit_bytes, 2048, 2, 4))
    return FT_ERR_CUDA;
  return FT_OK;
}

// The experts with many tokens (the plan's GEMM list): gather x rows into expert order, two grouped tcgen05 GEMMs
// over the weight tensor maps, fused gather-combine that also rounds y.
ft_status_t launch_gemm_path(ft_moe *h, int layer, const LayerState &L, const Scratch &sc, const __nv_bfloat16 *x_bf,
                             void *y_dev, cudaStream_t st) {
  const ft_moe_config_t &c = h->cfg;
    // experts with many tokens: gather x rows into expert order, two grouped tcgen05 GEMMs, fused combine
    {
      TimeScope ts(h, st, FT_TIME_GATHER);
      gather_rows_kernel<<<h->sm_count * 8, 256, 0, st>>>(x_bf, sc.perm, c.top_k, c.hidden, sc.offset + c.n_experts, h->xs);
    }
    GemmParams gp;
    gp.items = sc.items_gemm; gp.n_items = &sc.plan_dev->n_gemm_items; gp.mt_pref = sc.gemm_pref;
    gp.inter = c.inter; gp.d = c.hidden;
    gp.layer_unit0 = (c.global_pool || c.wdtype != FT_W_BF16) ? 0 : (long long)layer * c.slots_per_layer * (c.inter / 16);
    gp.status = h->status_dev;
    // CTA pairs (clusters of two) share every 256x256 tile
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(h->sm_count & ~1));
    lc.blockDim = dim3(kGemmThreads);
    lc.stream = st;
    cudaLaunchAttribute la[1];
    la[0].id = cudaLaunchAttributeClusterDimension;
    la[0].val.clusterDim.x = 2; la[0].val.clusterDim.y = 1; la[0].val.clusterDim.z = 1;
    lc.attrs = la;
    lc.numAttrs = 1;
    // gate/up + SwiGLU: one CTA per 128 x 256 tile (A = x rows, B = 128 gate + 128 up rows); measured faster
    // than the CTA-pair form for this GEMM, whose fused epilogue needs gate and up in the same TMEM
    gp.K = c.hidden; gp.n_tiles = c.inter / 128; gp.out = h->hbuf;
    {
      TimeScope ts(h, st, FT_TIME_GEMM1);
      gateup_gemm_kernel<<<h->sm_count, kGemmThreads, gateup_gemm_smem_bytes(), st>>>(h->tm_xs, h->tm_wgu, gp);
    }
    // down: A = the down tiles of 128 columns x 64 neurons per CTA, B = H rows (box 64 x 128 per CTA)
    gp.K = c.inter; gp.out = h->obuf;
    lc.dynamicSmemBytes = down_gemm2_smem_bytes();
    {
      TimeScope ts(h, st, FT_TIME_GEMM2);
      FT_CUDA(cudaLaunchKernelEx(&lc, down_gemm2_kernel, h->tm_wd, h->tm_h, gp));
    }
    {
      TimeScope ts(h, st, FT_TIME_COMBINE);
      combine_kernel<<<h->sm_count * 8, 256, 0, st>>>(h->obuf, sc.ids, sc.topk_w, sc.inv, sc.is_gemm, h->y_acc,
                                                      static_cast<__nv_bfloat16 *>(y_dev), L.T, c.top_k, c.hidden);
    }
    h->launches += 4;
    FT_CUDA(cudaGetLastError());
  return FT_OK;
}

}  // namespace

extern "C" {

size_t ft_moe_expert_bytes(const ft_moe_config_t *cfg) { return expert_bytes_of(cfg); }

const char *ft_moe_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

const char *ft_moe_status_string(ft_status_t s) {
  switch (s) {
    case FT_OK: return "ok";
    case FT_ERR_INVALID_ARG: return "invalid argument";
    case FT_ERR_NOT_PINNED: return "host pool is not pinned and mapped";
    case FT_ERR_OOM: return "out of memory";
    case FT_ERR_CUDA: return "CUDA error";
    case FT_ERR_STATE: return "call out of order";
    case FT_ERR_TIMEOUT: return "device-side wait timed out";
    case FT_ERR_NONFINITE: return "non-finite router logits";
    case FT_ERR_UNSUPPORTED: return "unsupported";
  }
  return "unknown status";
}

ft_status_t ft_moe_host_alloc(size_t bytes, void **out_host) {
  if (!out_host || bytes == 0) return FT_ERR_INVALID_ARG;
  *out_host = nullptr;
  cudaError_t e = cudaHostAlloc(out_host, bytes, cudaHostAllocPortable | cudaHostAllocMapped);
  if (e != cudaSuccess) {
    (void)cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? FT_ERR_OOM : FT_ERR_CUDA;
  }
  return FT_OK;
}

ft_status_t ft_moe_host_free(void *host) {
  if (!host) return FT_OK;
  FT_CUDA(cudaFreeHost(host));
  return FT_OK;
}

ft_status_t ft_moe_host_register(void *host, size_t bytes) {
  if (!host || bytes == 0) return FT_ERR_INVALID_ARG;
  cudaError_t e = cudaHostRegister(host, bytes, cudaHostRegisterPortable | cudaHostRegisterMapped);
  if (e != cudaSuccess) {
    g_last_cuda_error = e;
    (void)cudaGetLastError();
    return e == cudaErrorMemoryAllocation ? FT_ERR_OOM : FT_ERR_CUDA;
  }
  return FT_OK;
}

ft_status_t ft_moe_host_unregister(void *host) {
  if (!host) return FT_OK;
  FT_CUDA(cudaHostUnregister(host));
  return FT_OK;
}

ft_status_t ft_moe_destroy(ft_moe_t *h) {
  if (!h) return FT_OK;
  cudaSetDevice(h->cfg.device);
  cudaDeviceSynchronize();
  cudaFree(h->slots);
  cudaFree(h->shared_dev);
  cudaFree(h->tables);
  cudaFree(h->stats_mem);
  cudaFree(h->ids);
  cudaFree(h->count);
  cudaFree(h->offset);
  cudaFree(h->perm);
  cudaFree(h->inv);
  cudaFree(h->topk_w);
  cudaFree(h->route_hist);
  cudaFree(h->y_acc);
  cudaFree(h->plan_dev);
  if (h->plan_host) cudaFreeHost(h->plan_host);
  cudaFree(h->items_res);
  cudaFree(h->items_zc);
  cudaFree(h->items_gemm);
  cudaFree(h->res_pref);
  cudaFree(h->gemm_pref);
  cudaFree(h->is_gemm);
  cudaFree(h->xs);
  cudaFree(h->wq_scratch);
  cudaFree(h->hbuf);
  cudaFree(h->obuf);
  cudaFree(h->status_dev);
  cudaFree(h->seq_dev);
  cudaFree(h->done_dev);
  cudaFree(h->w4_hraw);
  cudaFree(h->w4_hcount);
  cudaFree(h->w4_hq);
  cudaFree(h->tc_xq);
  cudaFree(h->tc_pass_done);
  cudaFree(h->tc_gen);
  cudaFree(h->w4_hs);
  cudaFree(h->trace_dev);
  cudaFree(h->stage_logits);
  cudaFree(h->stage_x);
  cudaFree(h->stage_y);
  if (h->copy_stream) cudaStreamDestroy(h->copy_stream);
  if (h->aux_stream) cudaStreamDestroy(h->aux_stream);
  cudaEvent_t evs[] = {h->ev_plan, h->ev_fill, h->ev_fork, h->ev_join, h->ev_fill_t0, h->ev_fill_t1};
  for (cudaEvent_t e : evs)
    if (e) cudaEventDestroy(e);
  for (auto &ls : h->layers)
    if (ls.ev_fill) cudaEventDestroy(ls.ev_fill);
  for (auto &p : h->pending) { cudaEventDestroy(p.e0); cudaEventDestroy(p.e1); }
  for (cudaEvent_t e : h->free_events) cudaEventDestroy(e);
  (void)cudaGetLastError();
  delete h;
  return FT_OK;
}

ft_status_t ft_moe_create(const ft_moe_config_t *cfg, ft_moe_t **out) {
  if (!out) return FT_ERR_INVALID_ARG;
  *out = nullptr;
  if (!cfg || cfg->struct_size != sizeof(ft_moe_config_t)) return FT_ERR_INVALID_ARG;
  const ft_moe_config_t &c = *cfg;
  if (c.n_layers <= 0 || c.n_experts <= 0 || c.n_experts > kMaxExperts || c.top_k <= 0 ||
      c.top_k > c.n_experts || c.top_k > kMaxTopK || c.slots_per_layer < 0 ||
      (c.global_pool != 0 && c.global_pool != 1) ||
      (long long)c.slots_per_layer * (c.global_pool ? c.n_layers : 1) > kMaxTableSlots ||
      c.max_tokens <= 0 || (c.n_shared != 0 && c.n_shared != 1) || c.device < 0 ||
      (c.fill_mode != FT_FILL_COPY_ENGINE && c.fill_mode != FT_FILL_SM))
    return FT_ERR_INVALID_ARG;
  if (c.wdtype != FT_W_BF16 && c.wdtype != FT_W_INT4_G128 && c.wdtype != FT_W_MXFP4 && c.wdtype != FT_W_NVFP4 &&
      c.wdtype != FT_W_MXFP4_TC)
    return FT_ERR_INVALID_ARG;
  if (c.bw_fill_MBps == 0 || c.bw_zc_MBps == 0 || c.bw_hbm_MBps == 0 || c.reuse_credit < 0 ||
      c.zc_tokens_per_pass < 1 || c.hbm_tokens_per_pass < 1 || c.gemm_min_tokens < 0 || c.split_min_pairs < 0)
    return FT_ERR_INVALID_ARG;
  const size_t S = expert_bytes_of(cfg);
  if (S == 0 || (c.wdtype != FT_W_BF16 && !w4_shape_ok(c))) return FT_ERR_UNSUPPORTED;
  if (c.gemm_min_tokens != 0 &&
      (c.slots_per_layer == 0 || c.hidden % 256 || c.inter % 256 || c.gemm_min_tokens < 8 ||
       (c.wdtype != FT_W_BF16 && c.global_pool)))   // (4-bit: the bf16 scratch mirrors one layer's slots)
    return FT_ERR_UNSUPPORTED;
  if (!c.host_pool || c.host_pool_bytes < (size_t)c.n_layers * c.n_experts * S) return FT_ERR_INVALID_ARG;
  if (c.n_shared && !c.shared_weights) return FT_ERR_INVALID_ARG;
  if ((long long)c.max_tokens * c.top_k > (1ll << 30)) return FT_ERR_INVALID_ARG;

  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_CUDA; }
  if (c.device >= ndev) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(c.device));

  // The pool must be pinned and mapped: there is deliberately no pageable / CPU fallback.
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, c.host_pool) != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_NOT_PINNED; }
  if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return FT_ERR_NOT_PINNED;
  {
    const char *last = static_cast<const char *>(c.host_pool) + (size_t)c.n_layers * c.n_experts * S - 1;
    cudaPointerAttributes a2;
    if (cudaPointerGetAttributes(&a2, last) != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_NOT_PINNED; }
    if (a2.type != cudaMemoryTypeHost) return FT_ERR_NOT_PINNED;
  }

  ft_moe *h = new (std::nothrow) ft_moe();
  if (!h) return FT_ERR_OOM;
  h->cfg = c;
  h->S = S;
  h->pool_dev = static_cast<const uint8_t *>(attr.devicePointer);
  h->layers.resize(c.n_layers);
  ft_status_t rc = FT_OK;
  auto fail = [&](ft_status_t s) { ft_moe_destroy(h); return s; };
#define FT_TRY(expr)                                            \
  do {                                                          \
    cudaError_t e_ = (expr);                                    \
    if (e_ != cudaSuccess) {                                    \
      (void)cudaGetLastError();                                 \
      return fail(e_ == cudaErrorMemoryAllocation ? FT_ERR_OOM : FT_ERR_CUDA); \
    }                                                           \
  } while (0)

  int smc = 0;
  FT_TRY(cudaDeviceGetAttribute(&smc, cudaDevAttrMultiProcessorCount, c.device));
  h->sm_count = smc > 0 ? smc : 148;

  const size_t E = c.n_experts, Ns = c.slots_per_layer, L = c.n_layers;
  const size_t P = (size_t)c.max_tokens * c.top_k;
  if (c.n_shared) {
    FT_TRY(cudaMalloc(&h->shared_dev, L * S));
    FT_TRY(cudaMemcpy(h->shared_dev, c.shared_weights, L * S, cudaMemcpyHostToDevice));
  }
  // per-layer step counters and statistics
  {
    const size_t per = 256 + ((FT_STAT_COUNT * 8 + 255) & ~(size_t)255);
    FT_TRY(cudaMalloc(&h->stats_mem, per * L));
    FT_TRY(cudaMemset(h->stats_mem, 0, per * L));
    for (size_t l = 0; l < L; ++l) {
      h->layers[l].step = reinterpret_cast<int64_t *>(h->stats_mem + l * per);
      h->layers[l].stats = reinterpret_cast<unsigned long long *>(h->stats_mem + l * per + 256);
    }
  }
  rc = alloc_cache(h);
  if (rc != FT_OK) return fail(rc);
  h->pair_stride = (P * 4 + 16 + 15) & ~(size_t)15;
  FT_TRY(cudaMalloc(&h->ids, L * h->pair_stride));
  FT_TRY(cudaMalloc(&h->topk_w, L * h->pair_stride));
  FT_TRY(cudaMalloc(&h->count, L * E * 4));
  FT_TRY(cudaMalloc(&h->offset, L * (E + 1) * 4));
  FT_TRY(cudaMalloc(&h->perm, L * h->pair_stride));
  FT_TRY(cudaMalloc(&h->inv, L * h->pair_stride));
  FT_TRY(cudaMalloc(&h->route_hist, ((size_t)c.max_tokens / kRouteBlockTokens + 1) * E * 4));
  FT_TRY(cudaMalloc(&h->y_acc, (size_t)c.max_tokens * c.hidden * 4));
  FT_TRY(cudaMemset(h->y_acc, 0, (size_t)c.max_tokens * c.hidden * 4));
  h->plan_bytes = sizeof(PlanHeader) + 8 * E * 4;
  h->plan_stride = (h->plan_bytes + 63) & ~(size_t)63;
  FT_TRY(cudaMalloc(&h->plan_dev, L * h->plan_stride));
  FT_TRY(cudaMemset(h->plan_dev, 0, L * h->plan_stride));
  FT_TRY(cudaHostAlloc(&h->plan_host, L * h->plan_stride, cudaHostAllocMapped));
  memset(h->plan_host, 0, L * h->plan_stride);
  FT_TRY(cudaHostGetDevicePointer(reinterpret_cast<void **>(&h->plan_host_devptr), h->plan_host, 0));
  FT_TRY(cudaMalloc(&h->items_res, L * (2 * E + 1) * sizeof(WorkItem)));
  FT_TRY(cudaMemset(h->items_res, 0, L * (2 * E + 1) * sizeof(WorkItem)));
  FT_TRY(cudaMalloc(&h->items_zc, L * E * sizeof(WorkItem)));
  FT_TRY(cudaMalloc(&h->items_gemm, L * E * sizeof(WorkItem)));
  FT_TRY(cudaMalloc(&h->res_pref, L * (2 * E + 2) * 4));
  FT_TRY(cudaMemset(h->res_pref, 0, L * (2 * E + 2) * 4));
  if (c.gemm_min_tokens > 0) {
    const size_t Pr = P + 256;   // spare rows so that full boxes stay inside the tensors
    FT_TRY(cudaMalloc(&h->gemm_pref, L * (E + 1) * 4));
    FT_TRY(cudaMemset(h->gemm_pref, 0, L * (E + 1) * 4));
    FT_TRY(cudaMalloc(&h->is_gemm, L * E));
    FT_TRY(cudaMemset(h->is_gemm, 0, L * E));
    FT_TRY(cudaMalloc(&h->xs, Pr * c.hidden * 2));
    FT_TRY(cudaMalloc(&h->hbuf, Pr * c.inter * 2));
    FT_TRY(cudaMalloc(&h->obuf, Pr * c.hidden * 2));
    FT_TRY(cudaMemset(h->xs, 0, Pr * c.hidden * 2));
    FT_TRY(cudaMemset(h->hbuf, 0, Pr * c.inter * 2));
    void *fnp = nullptr;
    cudaDriverEntryPointQueryResult qres;
    FT_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fnp, cudaEnableDefault, &qres));
    if (!fnp || qres != cudaDriverEntryPointSuccess) return fail(FT_ERR_CUDA);
    EncodeTiledFn enc = reinterpret_cast<EncodeTiledFn>(fnp);
    if (!make_tensor_map(enc, &h->tm_xs, h->xs, Pr, c.hidden, 128, 64) ||
        !make_tensor_map(enc, &h->tm_h, h->hbuf, Pr, c.inter, 128, 64))
      return fail(FT_ERR_CUDA);
    if (c.wdtype != FT_W_BF16)
      FT_TRY(cudaMalloc(&h->wq_scratch, (size_t)c.slots_per_layer * 3 * c.inter * c.hidden * 2));
    rc = build_weight_maps(h);
    if (rc != FT_OK) return fail(rc);
    FT_TRY(cudaFuncSetAttribute(gateup_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)gateup_gemm_smem_bytes()));
    FT_TRY(cudaFuncSetAttribute(down_gemm2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)down_gemm2_smem_bytes()));
    h->gemm = true;
  }
  FT_TRY(cudaMalloc(&h->status_dev, 4));
  FT_TRY(cudaMemset(h->status_dev, 0, 4));
  FT_TRY(cudaMalloc(&h->seq_dev, 4));
  FT_TRY(cudaMemset(h->seq_dev, 0, 4));
  FT_TRY(cudaMalloc(&h->trace_dev, (size_t)h->sm_count * 4 * sizeof(long long)));
  FT_TRY(cudaMemset(h->trace_dev, 0, (size_t)h->sm_count * 4 * sizeof(long long)));
  FT_TRY(cudaMalloc(&h->done_dev, 4));
  FT_TRY(cudaMemset(h->done_dev, 0, 4));
  FT_TRY(cudaFuncSetAttribute(fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kFillStages * (int)kFillChunk));
  if (c.wdtype != FT_W_BF16) {
    const size_t passes = (P + 7) / 8 + 2 * E + 2;
    FT_TRY(cudaMalloc(&h->w4_hraw, passes * (c.inter / 16) * 1024));
    FT_TRY(cudaMemset(h->w4_hraw, 0, passes * (c.inter / 16) * 1024));
    FT_TRY(cudaMalloc(&h->w4_hcount, passes * (c.inter / 128) * 4));
    FT_TRY(cudaMemset(h->w4_hcount, 0, passes * (c.inter / 128) * 4));
    FT_TRY(cudaMalloc(&h->w4_hq, c.wdtype == FT_W_MXFP4_TC ? passes * tc_h_pass_bytes(c.inter) : passes * (c.inter / 128) * 2048));
    if (c.wdtype == FT_W_MXFP4_TC) {
      FT_TRY(cudaMemset(h->w4_hq, 0, passes * tc_h_pass_bytes(c.inter)));
      // one activation image per pass, or a single one for handles that never see more than 8 tokens
      const size_t n_img = c.max_tokens <= kQ4Tokens ? 1 : passes;
      FT_TRY(cudaMalloc(&h->tc_xq, n_img * kTcParts * tc_x_part_bytes(c.hidden)));
      FT_TRY(cudaMemset(h->tc_xq, 0, n_img * kTcParts * tc_x_part_bytes(c.hidden)));
      FT_TRY(cudaMalloc(&h->tc_pass_done, passes * sizeof(int)));
      FT_TRY(cudaMemset(h->tc_pass_done, 0, passes * sizeof(int)));
      FT_TRY(cudaMalloc(&h->tc_gen, 2 * sizeof(int)));
      FT_TRY(cudaMemset(h->tc_gen, 0, 2 * sizeof(int)));
      if (tc_gateup_fixed_bytes(c.hidden) + 3 * kTcStageA > kTcSmem ||
          tc_down_fixed_bytes(c.inter) + 3 * kTcStageD > kTcSmem || c.inter / 128 > 48 || h->sm_count < kTcParts)
        return fail(FT_ERR_UNSUPPORTED);
      FT_TRY(cudaFuncSetAttribute(tc_gateup_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmem));
      FT_TRY(cudaFuncSetAttribute(tc_down_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTcSmem));
    }
    FT_TRY(cudaMalloc(&h->w4_hs, passes * (c.inter / 128) * 64));
    // (limits are per function and device, not per handle: always the largest a CTA can have, and the handle's own
    // need is checked against it)
    const int sa = 232448, sb = (int)w4_down_smem_bytes(2 * kMaxExperts + 1);
    if (w4_gateup_smem_bytes(2 * c.n_experts + 1, c.hidden) > (size_t)sa) return fail(FT_ERR_UNSUPPORTED);
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<56>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_down_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb));
    FT_TRY(cudaFuncSetAttribute(w4_down_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<56>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_gateup_half_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_TRY(cudaFuncSetAttribute(w4_down_half_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb));
    FT_TRY(cudaFuncSetAttribute(w4_down_half_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, sb));
    const int sbm = (int)mx4_down_smem_bytes(2 * kMaxExperts + 1, false), sbn = (int)mx4_down_smem_bytes(2 * kMaxExperts + 1, true);
#define FT_MX_ATTR(G)                                                                                                   \
  FT_TRY(cudaFuncSetAttribute(mx4_gateup_kernel<G, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));           \
  FT_TRY(cudaFuncSetAttribute(mx4_gateup_kernel<G, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sa));
    FT_MX_ATTR(4) FT_MX_ATTR(8) FT_MX_ATTR(16) FT_MX_ATTR(32) FT_MX_ATTR(56) FT_MX_ATTR(64)
#undef FT_MX_ATTR
    FT_TRY(cudaFuncSetAttribute(mx4_down_kernel<8, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sbm));
    FT_TRY(cudaFuncSetAttribute(mx4_down_kernel<16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, sbm));
    FT_TRY(cudaFuncSetAttribute(mx4_down_kernel<8, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sbn));
    FT_TRY(cudaFuncSetAttribute(mx4_down_kernel<16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, sbn));
  }
  if (c.wdtype == FT_W_BF16) {
    // the limit is a property of the function on this device, not of the handle: always the largest size any
    // handle can ask for, so that handles of different shapes can live side by side
    const int smem = (int)ffn_stream_smem_bytes(2 * kMaxExperts + 1, 2048);
    FT_TRY(cudaFuncSetAttribute(ffn_stream_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    FT_TRY(cudaFuncSetAttribute(ffn_stream_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    FT_TRY(cudaFuncSetAttribute(ffn_stream_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    FT_TRY(cudaFuncSetAttribute(ffn_stream_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
  }
  FT_TRY(cudaMalloc(&h->stage_logits, (size_t)c.max_tokens * E * 4));
  FT_TRY(cudaMalloc(&h->stage_x, (size_t)c.max_tokens * c.hidden * 2));
  FT_TRY(cudaMalloc(&h->stage_y, (size_t)c.max_tokens * c.hidden * 2));
  FT_TRY(cudaStreamCreateWithFlags(&h->copy_stream, cudaStreamNonBlocking));
  FT_TRY(cudaStreamCreateWithFlags(&h->aux_stream, cudaStreamNonBlocking));
  FT_TRY(cudaEventCreateWithFlags(&h->ev_plan, cudaEventDisableTiming));
  FT_TRY(cudaEventCreateWithFlags(&h->ev_fill, cudaEventDisableTiming));
  for (auto &ls : h->layers) FT_TRY(cudaEventCreateWithFlags(&ls.ev_fill, cudaEventDisableTiming));
  FT_TRY(cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming));
  FT_TRY(cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming));
  FT_TRY(cudaEventCreate(&h->ev_fill_t0));
  FT_TRY(cudaEventCreate(&h->ev_fill_t1));
  for (int l = 0; l < c.n_layers; ++l) {
    rc = reset_layer(h, l);
    if (rc != FT_OK) return fail(rc);
  }
  FT_TRY(cudaDeviceSynchronize());
#undef FT_TRY
  *out = h;
  return FT_OK;
}

ft_status_t ft_moe_reset(ft_moe_t *h, int layer) {
  if (!h || layer < -1 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  if (h->cfg.global_pool && layer >= 0) return FT_ERR_UNSUPPORTED;   // the shared pool has no per-layer part
  for (int l = 0; l < h->cfg.n_layers; ++l)
    if (layer < 0 || l == layer) {
      ft_status_t rc = reset_layer(h, l);
      if (rc != FT_OK) return rc;
    }
  if (h->cfg.global_pool) FT_CUDA(cudaMemset(h->layers[0].clock, 0, 8));
  FT_CUDA(cudaMemset(h->y_acc, 0, (size_t)h->cfg.max_tokens * h->cfg.hidden * 4));
  FT_CUDA(cudaMemset(h->done_dev, 0, 4));
  if (h->w4_hraw) {   // the hand-over buffers of the 4-bit kernels (a call that gave up may have left partial sums)
    const ft_moe_config_t &c = h->cfg;
    const size_t passes = ((size_t)c.max_tokens * c.top_k + 7) / 8 + 2 * (size_t)c.n_experts + 2;
    FT_CUDA(cudaMemset(h->w4_hraw, 0, passes * (c.inter / 16) * 1024));
    FT_CUDA(cudaMemset(h->w4_hcount, 0, passes * (c.inter / 128) * 4));
    if (h->tc_pass_done) {
      FT_CUDA(cudaMemset(h->tc_pass_done, 0, passes * sizeof(int)));
      FT_CUDA(cudaMemset(h->tc_gen, 0, 2 * sizeof(int)));
      h->tc_calls = 0;
    }
  }
  FT_CUDA(cudaDeviceSynchronize());
  return FT_OK;
}

// Threads of the single-CTA route / plan kernels: one per expert, one warp per token, at least 256.
static int single_cta_threads(int E, int T) {
  int n = E > 32 * T ? E : 32 * T;
  n = ((n + 31) / 32) * 32;
  if (n < 256) n = 256;
  if (n > 1024) n = 1024;
  return n;
}

static RouteParams make_route_params(ft_moe *h, int layer, const float *logits_dev, int T) {
  const Scratch sc = scratch_of(h, layer);
  RouteParams rp;
  rp.logits = logits_dev;
  rp.T = T; rp.E = h->cfg.n_experts; rp.k = h->cfg.top_k;
  rp.ids = sc.ids; rp.w = sc.topk_w; rp.count = sc.count; rp.offset = sc.offset;
  rp.perm = sc.perm; rp.inv = sc.inv; rp.status = h->status_dev;
  return rp;
}

static PlanParams make_plan_params(ft_moe *h, int layer, bool mirror_to_host) {
  const ft_moe_config_t &c = h->cfg;
  LayerState &L = h->layers[layer];
  const Scratch sc = scratch_of(h, layer);
  PlanParams pp;
  pp.count = sc.count; pp.offset = sc.offset;
  pp.E = c.n_experts; pp.n_slots = h->table_slots;
  pp.id_base = c.global_pool ? layer * c.n_experts : 0;
  pp.cm.ns_fill = (int64_t)(h->S * 1000 / c.bw_fill_MBps);
  pp.cm.ns_zc = (int64_t)(h->S * 1000 / c.bw_zc_MBps);
  pp.cm.ns_hbm = (int64_t)(h->S * 1000 / c.bw_hbm_MBps);
  pp.cm.bw_fill = c.bw_fill_MBps; pp.cm.bw_res = c.bw_zc_residual_MBps;
  pp.cm.reuse_credit = c.reuse_credit; pp.cm.tz = c.zc_tokens_per_pass; pp.cm.tg = c.hbm_tokens_per_pass;
  pp.cm.gemm_min_tokens = c.gemm_min_tokens;
  pp.slot_expert = L.slot_expert; pp.slot_stamp = L.slot_stamp; pp.expert_slot = L.expert_slot;
  pp.step = L.clock; pp.layer_steps = L.step; pp.stats = L.stats;
  pp.pool_layer_dev = h->pool_dev + (size_t)layer * c.n_experts * h->S;
  pp.slots_layer = h->slots ? h->slots + (c.global_pool ? 0 : (size_t)layer * c.slots_per_layer * h->S) : nullptr;
  pp.shared_rec = c.n_shared ? h->shared_dev + (size_t)layer * h->S : nullptr;
  pp.S = h->S; pp.T = L.T;
  pp.tokens_per_pass = (c.wdtype == FT_W_BF16) ? kFsResTokensPerPass : kQ4Tokens;
  pp.zc_tokens_per_pass = (c.wdtype == FT_W_BF16) ? kFsZcTokensPerPass : kQ4Tokens;
  pp.hdr_dev = sc.plan_dev;
  pp.hdr_host = mirror_to_host ? sc.plan_host_devptr : nullptr;
  pp.items_res = sc.items_res; pp.res_pref = sc.res_pref;
  pp.items_zc = sc.items_zc; pp.items_gemm = sc.items_gemm;
  pp.gemm_pref = sc.gemm_pref; pp.is_gemm = sc.is_gemm;
  // decode-sized calls on a prefill-capable handle keep every expert on the streaming kernels
  if (L.T < c.gemm_min_tokens) pp.cm.gemm_min_tokens = 0;
  pp.seq_value = L.seq + 1;
  pp.prefetch = 0;
  return pp;
}

ft_status_t ft_moe_route(ft_moe_t *h, int layer, const float *logits_dev, int T, void *stream) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers || T < 0 || T > h->cfg.max_tokens) return FT_ERR_INVALID_ARG;
  if (T > 0 && !logits_dev) return FT_ERR_INVALID_ARG;
  LayerState &L = h->layers[layer];
  L.phase = PH_ROUTED;
  L.T = T;
  if (T == 0) return FT_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const RouteParams rp = make_route_params(h, layer, logits_dev, T);
  TimeScope ts(h, st, FT_TIME_ROUTE);
  if (T <= kRouteSmallMaxTokens) {
    route_small_kernel<<<1, single_cta_threads(h->cfg.n_experts, T), 0, st>>>(rp);
    h->launches++;
  } else {
    const int n_blocks = (T + kRouteBlockTokens - 1) / kRouteBlockTokens;
    route_block_kernel<<<n_blocks, 1024, 0, st>>>(rp, h->route_hist);
    permute_block_kernel<<<n_blocks, 1024, 0, st>>>(rp, h->route_hist, n_blocks);
    h->launches += 2;
  }
  FT_CUDA(cudaGetLastError());
  return FT_OK;
}

ft_status_t ft_moe_plan(ft_moe_t *h, int layer, ft_moe_plan_t *out, void *stream) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  LayerState &L = h->layers[layer];
  if (L.phase != PH_ROUTED) return FT_ERR_STATE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ft_moe_config_t &c = h->cfg;
  if (L.T > 0) {
    const bool mirror = (out != nullptr) || c.fill_mode == FT_FILL_COPY_ENGINE;
    const PlanParams pp = make_plan_params(h, layer, mirror);
    const size_t smem = (size_t)h->table_slots * 16;
    int threads = ((c.n_experts + 31) / 32) * 32;
    if (threads < 128) threads = 128;
    {
      TimeScope ts(h, st, FT_TIME_PLAN);
      plan_kernel<<<1, threads, smem, st>>>(pp);
    }
    h->launches++;
    L.seq++;
    h->plan_mirrored = mirror;
    FT_CUDA(cudaGetLastError());
    FT_CUDA(cudaEventRecord(h->ev_plan, st));
  }
  L.phase = PH_PLANNED;
  if (out) {
    const Scratch sc = scratch_of(h, layer);
    const int E = c.n_experts;
    if (L.T == 0) {
      out->step = -1;
      out->n_routed = out->n_hit = out->n_miss = out->n_fill = out->n_zc = 0;
      if (out->loc) for (int e = 0; e < E; ++e) out->loc[e] = kLocNotRouted;
      return FT_OK;
    }
    FT_CUDA(cudaEventSynchronize(h->ev_plan));
    const PlanHeader hd = *sc.plan_host;
    if (hd.seq != L.seq) return FT_ERR_CUDA;
    const int32_t *a = reinterpret_cast<const int32_t *>(sc.plan_host + 1);
    out->step = hd.step;
    out->n_routed = hd.n_routed; out->n_hit = hd.n_hit; out->n_miss = hd.n_miss;
    out->n_fill = hd.n_fill; out->n_zc = hd.n_zc;
    if (out->hit) memcpy(out->hit, a + 0 * E, sizeof(int32_t) * hd.n_hit);
    if (out->miss) memcpy(out->miss, a + 1 * E, sizeof(int32_t) * hd.n_miss);
    if (out->fill) memcpy(out->fill, a + 2 * E, sizeof(int32_t) * hd.n_fill);
    if (out->zc) memcpy(out->zc, a + 3 * E, sizeof(int32_t) * hd.n_zc);
    if (out->fill_order) memcpy(out->fill_order, a + 4 * E, sizeof(int32_t) * hd.n_fill);
    if (out->fill_slot) memcpy(out->fill_slot, a + 5 * E, sizeof(int32_t) * hd.n_fill);
    if (out->fill_evicted) memcpy(out->fill_evicted, a + 6 * E, sizeof(int32_t) * hd.n_fill);
    if (out->loc) memcpy(out->loc, a + 7 * E, sizeof(int32_t) * E);
    return drain_status(h);
  }
  return FT_OK;
}

ft_status_t ft_moe_prefetch_layer(ft_moe_t *h, int layer, void *stream, void *copy_stream) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  const ft_moe_config_t &c = h->cfg;
  LayerState &L = h->layers[layer];
  if (L.phase != PH_IDLE) return FT_ERR_STATE;
  // two full-layer buffers must fit: the layer being computed and the one being loaded
  if (c.global_pool ? (h->table_slots < 2 * c.n_experts) : (c.slots_per_layer < c.n_experts)) return FT_ERR_UNSUPPORTED;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const Scratch sc = scratch_of(h, layer);
  all_experts_kernel<<<1, 256, 0, st>>>(sc.count, sc.offset, c.n_experts);
  L.T = c.n_experts <= c.max_tokens ? c.n_experts : c.max_tokens;   // (only sizes the shared expert's passes: unused here)
  const bool mirror = c.fill_mode == FT_FILL_COPY_ENGINE;
  PlanParams pp = make_plan_params(h, layer, mirror);
  pp.prefetch = 1;
  pp.cm.gemm_min_tokens = 0;
  int threads = ((c.n_experts + 31) / 32) * 32;
  if (threads < 128) threads = 128;
  plan_kernel<<<1, threads, (size_t)h->table_slots * 16, st>>>(pp);
  h->launches += 2;
  L.seq++;
  h->plan_mirrored = mirror;
  FT_CUDA(cudaGetLastError());
  FT_CUDA(cudaEventRecord(h->ev_plan, st));
  L.phase = PH_PLANNED;
  ft_status_t rc = ft_moe_fill(h, layer, copy_stream ? copy_stream : h->copy_stream);
  L.phase = PH_IDLE;
  L.T = 0;
  return rc;
}

ft_status_t ft_moe_fill(ft_moe_t *h, int layer, void *copy_stream) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  LayerState &L = h->layers[layer];
  if (L.phase != PH_PLANNED) return FT_ERR_STATE;
  L.phase = PH_FILLED;
  h->fill_timed = false;
  h->last_fill_bytes = 0;
  h->last_fill_layer = layer;
  const Scratch sc = scratch_of(h, layer);
  if (L.T == 0 || h->cfg.slots_per_layer == 0) return FT_OK;
  cudaStream_t cs = static_cast<cudaStream_t>(copy_stream);
  const ft_moe_config_t &c = h->cfg;
  uint8_t *slots_layer = h->slots + (c.global_pool ? 0 : (size_t)layer * c.slots_per_layer * h->S);
  if (c.fill_mode == FT_FILL_COPY_ENGINE) {
    // the host needs the fill list: wait for the plan record (one host round trip per layer)
    FT_CUDA(cudaEventSynchronize(h->ev_plan));
    const PlanHeader hd = *sc.plan_host;
    if (hd.seq != L.seq) return FT_ERR_CUDA;
    if (hd.n_fill > 0) {
      const int E = c.n_experts;
      const int32_t *a = reinterpret_cast<const int32_t *>(sc.plan_host + 1);
      const int32_t *forder = a + 4 * E, *fslot = a + 5 * E;
      const uint8_t *pool_layer = static_cast<const uint8_t *>(c.host_pool) + (size_t)layer * E * h->S;
      FT_CUDA(cudaStreamWaitEvent(cs, h->ev_plan, 0));
      FT_CUDA(cudaEventRecord(h->ev_fill_t0, cs));
      {
        TimeScope ts(h, cs, FT_TIME_FILL);
        for (int i = 0; i < hd.n_fill; ++i) {
          if (forder[i] < 0 || forder[i] >= E || fslot[i] < 0 || fslot[i] >= h->table_slots) return FT_ERR_CUDA;
          FT_CUDA(cudaMemcpyAsync(slots_layer + (size_t)fslot[i] * h->S, pool_layer + (size_t)forder[i] * h->S,
                                  h->S, cudaMemcpyHostToDevice, cs));
        }
      }
      FT_CUDA(cudaEventRecord(h->ev_fill_t1, cs));
      FT_CUDA(cudaEventRecord(L.ev_fill, cs));
      L.fill_recorded = true;
      h->fill_timed = true;
      h->last_fill_bytes = (uint64_t)hd.n_fill * h->S;
    } else {
      // nothing to copy: the fill event of an earlier layer must not be waited on needlessly
      FT_CUDA(cudaStreamWaitEvent(cs, h->ev_plan, 0));
      FT_CUDA(cudaEventRecord(L.ev_fill, cs));
      L.fill_recorded = true;
    }
  } else {
    FillParams fp;
    fp.hdr = sc.plan_dev; fp.E = c.n_experts;
    fp.pool_layer_dev = h->pool_dev + (size_t)layer * c.n_experts * h->S;
    fp.slots_layer = slots_layer; fp.S = h->S;
    FT_CUDA(cudaStreamWaitEvent(cs, h->ev_plan, 0));
    FT_CUDA(cudaEventRecord(h->ev_fill_t0, cs));
    {
      TimeScope ts(h, cs, FT_TIME_FILL);
      fill_kernel<<<kFillCtas, kFillThreads, kFillStages * kFillChunk, cs>>>(fp, h->status_dev);
    }
    h->launches++;
    FT_CUDA(cudaGetLastError());
    FT_CUDA(cudaEventRecord(h->ev_fill_t1, cs));
    FT_CUDA(cudaEventRecord(L.ev_fill, cs));
    L.fill_recorded = true;
    h->fill_timed = true;
    h->last_fill_bytes = ~0ull;  // resolved from the plan record when asked
  }
  return FT_OK;
}

ft_status_t ft_moe_forward(ft_moe_t *h, int layer, const void *x_dev, void *y_dev, void *stream) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  LayerState &L = h->layers[layer];
  if (L.phase != PH_FILLED) return FT_ERR_STATE;
  L.phase = PH_IDLE;
  if (L.T == 0) return FT_OK;
  if (!x_dev || !y_dev) return FT_ERR_INVALID_ARG;
  if (((uintptr_t)x_dev | (uintptr_t)y_dev) & 15) return FT_ERR_INVALID_ARG;   // the kernels use 16-byte vector accesses
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ft_moe_config_t &c = h->cfg;
  const __nv_bfloat16 *x_bf = static_cast<const __nv_bfloat16 *>(x_dev);
  const bool use_gemm = h->gemm && L.T >= c.gemm_min_tokens;
  const Scratch sc = scratch_of(h, layer);
  if (c.wdtype == FT_W_BF16) {
    // bulk-copy pipelined tensor-core streaming kernel; the last CTA of the last launch finalizes y
    FfnStreamParams mp;
    mp.items = sc.items_res;
    mp.n_items = &sc.plan_dev->n_res_items;
    mp.n_hit = &sc.plan_dev->n_hit_items;
    mp.n_zc = &sc.plan_dev->n_zc_items;
    mp.pref = sc.res_pref;
    mp.max_items = 2 * c.n_experts + 1;
    mp.trace = h->trace_dev;
    mp.x = x_bf; mp.perm = sc.perm; mp.topk_w = sc.topk_w; mp.y_acc = h->y_acc;
    mp.y = static_cast<__nv_bfloat16 *>(y_dev);
    mp.done = h->done_dev; mp.status = h->status_dev;
    mp.inter = c.inter; mp.top_k = c.top_k; mp.T = L.T;
    const size_t smem = ffn_stream_smem_bytes(mp.max_items, c.hidden);
    cudaError_t launch_err = cudaSuccess;
    auto launch = [&](int part, int finalize) {
      mp.part = part;
      mp.finalize = finalize;
      mp.overlap = h->overlap;
      TimeScope ts(h, st, part == 1 ? FT_TIME_FFN_ZC : FT_TIME_FFN_RES);
      // while the device-driven fill holds kFillCtas SMs, the overlapping launch takes the others
      const int grid = (part == 1 && c.fill_mode == FT_FILL_SM) ? h->sm_count - kFillCtas : h->sm_count;
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3((unsigned)grid);
      lc.blockDim = dim3(kFsThreads);
      lc.dynamicSmemBytes = smem;
      lc.stream = st;
      cudaLaunchAttribute la[1];
      la[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      la[0].val.programmaticStreamSerializationAllowed = 1;
      lc.attrs = la;
      lc.numAttrs = h->overlap ? 1 : 0;
      cudaError_t e;
      switch (c.hidden / 256) {
        case 1: e = cudaLaunchKernelEx(&lc, ffn_stream_kernel<1>, mp); break;
        case 2: e = cudaLaunchKernelEx(&lc, ffn_stream_kernel<2>, mp); break;
        case 4: e = cudaLaunchKernelEx(&lc, ffn_stream_kernel<4>, mp); break;
        default: e = cudaLaunchKernelEx(&lc, ffn_stream_kernel<8>, mp); break;
      }
      if (e != cudaSuccess) launch_err = e;
      h->launches++;
    };
    // With enough tokens in the call the hits (and the zero-copy experts) are worth a launch of their own that
    // overlaps the fills; the filled experts follow once the fill event has fired.  With few tokens the extra
    // launch costs more than the overlap buys, so everything goes in one launch after the fills.
    const bool split = c.slots_per_layer > 0 && (long long)L.T * c.top_k >= c.split_min_pairs && c.split_min_pairs > 0;
    // the last CTA of the last launch rounds y itself unless the call has so many tokens that a launch of its own,
    // spread over the whole GPU, is quicker (or the GEMM path's combine does it)
    const bool own_finalize = !use_gemm && L.T > kFinalizeInKernelMaxTokens;
    const int fin = (use_gemm || own_finalize) ? 0 : 1;
    if (split) {
      launch(1, 0);
      if (L.fill_recorded) FT_CUDA(cudaStreamWaitEvent(st, L.ev_fill, 0));
      launch(2, fin);
    } else {
      if (c.slots_per_layer > 0 && L.fill_recorded) FT_CUDA(cudaStreamWaitEvent(st, L.ev_fill, 0));
      launch(0, fin);
    }
    if (own_finalize) {
      TimeScope ts(h, st, FT_TIME_FINALIZE);
      const int n4 = L.T * (c.hidden / 4);
      int grid = (n4 + 255) / 256;
      if (grid > h->sm_count * 4) grid = h->sm_count * 4;
      finalize_kernel<<<grid, 256, 0, st>>>(h->y_acc, static_cast<__nv_bfloat16 *>(y_dev), n4);
      h->launches++;
    }
    FT_CUDA(launch_err);
    FT_CUDA(cudaGetLastError());
    if (use_gemm) return launch_gemm_path(h, layer, L, sc, x_bf, y_dev, st);
    return FT_OK;
  }
  // int4 / mxfp4: gate/up kernel writes h, down kernel accumulates, its last CTA finalizes y
  if (c.slots_per_layer > 0 && L.fill_recorded) FT_CUDA(cudaStreamWaitEvent(st, L.ev_fill, 0));
  W4Params qp;
  qp.items = sc.items_res;
  qp.n_items = &sc.plan_dev->n_res_items;
  qp.n_zc = &sc.plan_dev->n_zc_items;
  qp.pref = sc.res_pref;
  qp.max_items = 2 * c.n_experts + 1;
  qp.x = x_bf; qp.perm = sc.perm; qp.topk_w = sc.topk_w;
  const bool nv = c.wdtype == FT_W_NVFP4;
  const bool mx = c.wdtype == FT_W_MXFP4 || nv;   // the floating-point 4-bit formats share their kernels
  qp.overlap = h->overlap;
  if (mx) { qp.mask = 0x1C1C1C1Cu; qp.flip = 0x80808080u; }   // (see ffn_mx4.cuh)
  else { qp.mask = 0x0F0F0F0Fu; qp.flip = 0x08080808u; }
  qp.hraw = h->w4_hraw; qp.hcount = h->w4_hcount; qp.hq = h->w4_hq; qp.hs = h->w4_hs;
  qp.y_acc = h->y_acc; qp.y = static_cast<__nv_bfloat16 *>(y_dev);
  qp.done = h->done_dev; qp.status = h->status_dev;
  qp.inter = c.inter; qp.top_k = c.top_k; qp.T = L.T;
  const bool own_finalize = !use_gemm && L.T > kFinalizeInKernelMaxTokens;
  qp.finalize = (use_gemm || own_finalize) ? 0 : 1;   // (the GEMM path's combine rounds y)
  if (c.wdtype == FT_W_MXFP4_TC) {
    // bit-sliced activation images, then the two block-scaled tensor-core kernels (programmatic dependents: their
    // set-up and first weight copies overlap the kernel before them)
    const bool dense = L.T <= kQ4Tokens, tc_own_finalize = !use_gemm && L.T > kFinalizeInKernelMaxTokens;
    qp.finalize = (use_gemm || tc_own_finalize) ? 0 : 1;   // (the GEMM path's combine rounds y)
    TcQuantParams tq;
    const int grid = h->sm_count - h->sm_count % kTcParts;   // CTA i works on part i % kTcParts of the hidden dimension
    const int expect_gu = (int)(h->tc_calls * (uint32_t)grid), expect_dn = (int)(h->tc_calls * (uint32_t)h->sm_count);
    h->tc_calls++;
    tq.w = qp; tq.x = x_bf; tq.xq = h->tc_xq; tq.d = c.hidden; tq.dense = dense ? 1 : 0;
    tq.gen = h->tc_gen; tq.expect_gu = expect_gu;
    // overlap mode 2: the call's first kernels start while the call before is finishing (the completion counts order
    // what they share); only for calls whose down kernel rounds y itself and that have a single activation image
    tq.early = (h->overlap == 2 && dense && !tc_own_finalize && !use_gemm) ? 1 : 0;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    {
      TimeScope ts(h, st, FT_TIME_GATHER);
      cudaLaunchConfig_t lc = {};
      // (the number of passes is known on the device only: one block row per possible pass, the surplus returns at once)
      const size_t max_passes = ((size_t)L.T * c.top_k + 7) / 8 + 2 * (size_t)c.n_experts + 2;
      lc.gridDim = dim3(c.hidden / 256, dense ? 1u : (unsigned)max_passes); lc.blockDim = dim3(256); lc.stream = st;
      lc.attrs = at; lc.numAttrs = h->overlap ? 1 : 0;   // (it waits for the kernels before it by itself)
      FT_CUDA(cudaLaunchKernelEx(&lc, tc_quant_x_kernel, tq));
    }
    TcParams tp;
    tp.w = qp; tp.xq = h->tc_xq; tp.d = c.hidden; tp.pass_done = h->tc_pass_done; tp.dense = dense ? 1 : 0;
    tp.gen = h->tc_gen; tp.expect_gu = expect_gu; tp.expect_dn = expect_dn;
    {
      TimeScope ts(h, st, FT_TIME_FFN_ZC);
      const size_t fixed = tc_gateup_fixed_bytes(c.hidden);
      tp.n_stages = (int)std::min<size_t>(kTcMaxStages, (kTcSmem - fixed) / kTcStageA);
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(grid); lc.blockDim = dim3(kTcThreads); lc.stream = st;
      lc.dynamicSmemBytes = fixed + (size_t)tp.n_stages * kTcStageA;
      lc.attrs = at; lc.numAttrs = 1;
      FT_CUDA(cudaLaunchKernelEx(&lc, tc_gateup_kernel, tp));
    }
    {
      TimeScope ts(h, st, FT_TIME_FFN_RES);
      const size_t fixed = tc_down_fixed_bytes(c.inter);
      tp.n_stages = (int)std::min<size_t>(kTcMaxStages, (kTcSmem - fixed) / kTcStageD);
      cudaLaunchConfig_t lc = {};
      lc.gridDim = dim3(h->sm_count); lc.blockDim = dim3(kTcThreads); lc.stream = st;
      lc.dynamicSmemBytes = fixed + (size_t)tp.n_stages * kTcStageD;
      lc.attrs = at; lc.numAttrs = 1;
      FT_CUDA(cudaLaunchKernelEx(&lc, tc_down_kernel, tp));
    }
    h->launches += 3;
    if (tc_own_finalize) {
      TimeScope ts(h, st, FT_TIME_FINALIZE);
      const int n4 = L.T * (c.hidden / 4);
      finalize_kernel<<<std::min((n4 + 255) / 256, h->sm_count * 8), 256, 0, st>>>(h->y_acc, qp.y, n4);
      h->launches++;
    }
    if (use_gemm) {
      // the experts of the GEMM list: expanded from their operand images to bf16 records, then the grouped GEMMs
      DequantParams dp;
      dp.items = sc.items_gemm; dp.n_items = &sc.plan_dev->n_gemm_items; dp.scratch = h->wq_scratch;
      dp.d = c.hidden; dp.inter = c.inter;
      {
        TimeScope ts(h, st, FT_TIME_GATHER);
        const dim3 dg((unsigned)(c.inter / 16), (unsigned)std::min(c.n_experts, c.slots_per_layer));
        dequant_w4_kernel<3><<<dg, 256, 0, st>>>(dp);
      }
      h->launches++;
      return launch_gemm_path(h, layer, L, sc, x_bf, y_dev, st);
    }
    return FT_OK;
  }
  const bool half = !mx && L.T <= kW4HalfTokens;   // int4 with at most 4 tokens: one MMA per pair of weight words
  const size_t sa = mx ? mx4_gateup_smem_bytes(qp.max_items, c.hidden)
                       : half ? w4_gateup_half_smem_bytes(qp.max_items, c.hidden) : w4_gateup_smem_bytes(qp.max_items, c.hidden);
  const size_t sb = mx ? mx4_down_smem_bytes(qp.max_items, nv)
                       : half ? w4_down_half_smem_bytes(qp.max_items) : w4_down_smem_bytes(qp.max_items);
  const int grid = h->sm_count;
  {
    TimeScope ts(h, st, FT_TIME_FFN_ZC);   // (timing slot reused for the gate/up kernel of the 4-bit paths)
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid); lc.blockDim = dim3(kW4Threads); lc.dynamicSmemBytes = sa; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = h->overlap ? 1 : 0;
    cudaError_t le;
    if (mx) {
#define FT_MX_LAUNCH(G) (nv ? cudaLaunchKernelEx(&lc, mx4_gateup_kernel<G, true>, qp) : cudaLaunchKernelEx(&lc, mx4_gateup_kernel<G, false>, qp))
      switch (c.hidden) {
        case 512: le = FT_MX_LAUNCH(4); break;
        case 1024: le = FT_MX_LAUNCH(8); break;
        case 2048: le = FT_MX_LAUNCH(16); break;
        case 4096: le = FT_MX_LAUNCH(32); break;
        case 7168: le = FT_MX_LAUNCH(56); break;
        default: le = FT_MX_LAUNCH(64); break;
      }
#undef FT_MX_LAUNCH
    } else if (half) {
      switch (c.hidden) {
        case 512: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<4>, qp); break;
        case 1024: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<8>, qp); break;
        case 2048: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<16>, qp); break;
        case 4096: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<32>, qp); break;
        case 7168: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<56>, qp); break;
        default: le = cudaLaunchKernelEx(&lc, w4_gateup_half_kernel<64>, qp); break;
      }
    } else {
      switch (c.hidden) {
        case 512: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<4>, qp); break;
        case 1024: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<8>, qp); break;
        case 2048: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<16>, qp); break;
        case 4096: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<32>, qp); break;
        case 7168: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<56>, qp); break;
        default: le = cudaLaunchKernelEx(&lc, w4_gateup_kernel<64>, qp); break;
      }
    }
    FT_CUDA(le);
  }
  {
    TimeScope ts(h, st, FT_TIME_FFN_RES);
    // a programmatic dependent of the gate/up kernel: its blocks set themselves up while that kernel drains and
    // wait for its completion before they read h
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(grid); lc.blockDim = dim3(kW4Threads); lc.dynamicSmemBytes = sb; lc.stream = st;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = at; lc.numAttrs = 1;
    if (nv) {
      if (c.hidden == 512) FT_CUDA(cudaLaunchKernelEx(&lc, mx4_down_kernel<8, true>, qp, c.hidden));
      else FT_CUDA(cudaLaunchKernelEx(&lc, mx4_down_kernel<16, true>, qp, c.hidden));
    } else if (mx) {
      if (c.hidden == 512) FT_CUDA(cudaLaunchKernelEx(&lc, mx4_down_kernel<8, false>, qp, c.hidden));
      else FT_CUDA(cudaLaunchKernelEx(&lc, mx4_down_kernel<16, false>, qp, c.hidden));
    } else if (half) {
      if (c.hidden == 512) FT_CUDA(cudaLaunchKernelEx(&lc, w4_down_half_kernel<8>, qp, c.hidden));
      else FT_CUDA(cudaLaunchKernelEx(&lc, w4_down_half_kernel<16>, qp, c.hidden));
    } else {
      if (c.hidden == 512) FT_CUDA(cudaLaunchKernelEx(&lc, w4_down_kernel<8>, qp, c.hidden));
      else FT_CUDA(cudaLaunchKernelEx(&lc, w4_down_kernel<16>, qp, c.hidden));
    }
    if (own_finalize) {
      const int n4 = L.T * (c.hidden / 4);
      finalize_kernel<<<std::min((n4 + 255) / 256, h->sm_count * 8), 256, 0, st>>>(h->y_acc, qp.y, n4);
      h->launches++;
    }
  }
  h->launches += 2;
  FT_CUDA(cudaGetLastError());
  if (use_gemm) {
    // the experts of the GEMM list are expanded to bf16 records in the layer's scratch pool first
    DequantParams dp;
    dp.items = sc.items_gemm; dp.n_items = &sc.plan_dev->n_gemm_items; dp.scratch = h->wq_scratch;
    dp.d = c.hidden; dp.inter = c.inter;
    {
      TimeScope ts(h, st, FT_TIME_GATHER);
      const dim3 dg((unsigned)(c.inter / 16), (unsigned)std::min(c.n_experts, c.slots_per_layer));
      if (nv) dequant_w4_kernel<2><<<dg, 256, 0, st>>>(dp);
      else if (mx) dequant_w4_kernel<1><<<dg, 256, 0, st>>>(dp);
      else dequant_w4_kernel<0><<<dg, 256, 0, st>>>(dp);
    }
    h->launches++;
    return launch_gemm_path(h, layer, L, sc, x_bf, y_dev, st);
  }
  return FT_OK;
}

ft_status_t ft_moe_layer(ft_moe_t *h, int layer, const float *logits_dev, const void *x_dev, void *y_dev,
                         int T, void *stream) {
  ft_status_t rc;
  if (h && layer >= 0 && layer < h->cfg.n_layers && T > 0 && T <= kRouteSmallMaxTokens && T <= h->cfg.max_tokens &&
      logits_dev) {
    // decode-sized call: route, permute and plan in one single-CTA launch
    LayerState &L = h->layers[layer];
    const ft_moe_config_t &c = h->cfg;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    L.T = T;
    const bool mirror = c.fill_mode == FT_FILL_COPY_ENGINE;
    const RouteParams rp = make_route_params(h, layer, logits_dev, T);
    const PlanParams pp = make_plan_params(h, layer, mirror);
    {
      TimeScope ts(h, st, FT_TIME_PLAN);
      route_plan_small_kernel<<<1, single_cta_threads(c.n_experts, T), (size_t)h->table_slots * 16, st>>>(rp, pp);
    }
    h->launches++;
    L.seq++;
    h->plan_mirrored = mirror;
    FT_CUDA(cudaGetLastError());
    FT_CUDA(cudaEventRecord(h->ev_plan, st));
    L.phase = PH_PLANNED;
  } else {
    rc = ft_moe_route(h, layer, logits_dev, T, stream);
    if (rc != FT_OK) return rc;
    rc = ft_moe_plan(h, layer, nullptr, stream);
    if (rc != FT_OK) return rc;
  }
  rc = ft_moe_fill(h, layer, h->copy_stream);
  if (rc != FT_OK) return rc;
  return ft_moe_forward(h, layer, x_dev, y_dev, stream);
}

ft_status_t ft_moe_layer_host(ft_moe_t *h, int layer, const float *logits_host, const void *x_host,
                              void *y_host, int T, void *stream) {
  if (!h || T < 0 || T > h->cfg.max_tokens) return FT_ERR_INVALID_ARG;
  if (T > 0 && (!logits_host || !x_host || !y_host)) return FT_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const ft_moe_config_t &c = h->cfg;
  if (T > 0) {
    FT_CUDA(cudaMemcpyAsync(h->stage_logits, logits_host, (size_t)T * c.n_experts * 4, cudaMemcpyHostToDevice, st));
    FT_CUDA(cudaMemcpyAsync(h->stage_x, x_host, (size_t)T * c.hidden * 2, cudaMemcpyHostToDevice, st));
  }
  ft_status_t rc = ft_moe_layer(h, layer, h->stage_logits, h->stage_x, h->stage_y, T, stream);
  if (rc != FT_OK) return rc;
  if (T > 0) {
    FT_CUDA(cudaMemcpyAsync(y_host, h->stage_y, (size_t)T * c.hidden * 2, cudaMemcpyDeviceToHost, st));
    FT_CUDA(cudaStreamSynchronize(st));
  }
  return FT_OK;
}

ft_status_t ft_moe_get_routing(ft_moe_t *h, int layer, int32_t *ids, float *w, int32_t *count,
                               int32_t *offset, int32_t *perm, int32_t *inv) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  const Scratch sc = scratch_of(h, layer);
  const size_t P = (size_t)h->layers[layer].T * h->cfg.top_k, E = h->cfg.n_experts;
  if (P == 0) {
    if (count) memset(count, 0, E * 4);
    if (offset) memset(offset, 0, (E + 1) * 4);
    return FT_OK;
  }
  if (ids) FT_CUDA(cudaMemcpy(ids, sc.ids, P * 4, cudaMemcpyDeviceToHost));
  if (w) FT_CUDA(cudaMemcpy(w, sc.topk_w, P * 4, cudaMemcpyDeviceToHost));
  if (count) FT_CUDA(cudaMemcpy(count, sc.count, E * 4, cudaMemcpyDeviceToHost));
  if (offset) FT_CUDA(cudaMemcpy(offset, sc.offset, (E + 1) * 4, cudaMemcpyDeviceToHost));
  if (perm) FT_CUDA(cudaMemcpy(perm, sc.perm, P * 4, cudaMemcpyDeviceToHost));
  if (inv) FT_CUDA(cudaMemcpy(inv, sc.inv, P * 4, cudaMemcpyDeviceToHost));
  return drain_status(h);
}

ft_status_t ft_moe_get_slot_table(ft_moe_t *h, int layer, int32_t *slot_expert, int64_t *slot_stamp,
                                  int32_t *expert_slot) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  const LayerState &L = h->layers[layer];
  const size_t Ns = h->table_slots;
  if (slot_expert && Ns) FT_CUDA(cudaMemcpy(slot_expert, L.slot_expert, Ns * 4, cudaMemcpyDeviceToHost));
  if (slot_stamp && Ns) FT_CUDA(cudaMemcpy(slot_stamp, L.slot_stamp, Ns * 8, cudaMemcpyDeviceToHost));
  if (expert_slot)
    FT_CUDA(cudaMemcpy(expert_slot, L.expert_slot + (h->cfg.global_pool ? (size_t)layer * h->cfg.n_experts : 0),
                       (size_t)h->cfg.n_experts * 4, cudaMemcpyDeviceToHost));
  return FT_OK;
}

ft_status_t ft_moe_read_slot(ft_moe_t *h, int layer, int slot, void *host_dst) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers || slot < 0 || slot >= h->table_slots || !host_dst)
    return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  FT_CUDA(cudaMemcpy(host_dst, h->slots + ((h->cfg.global_pool ? 0 : (size_t)layer * h->cfg.slots_per_layer) + slot) * h->S, h->S,
                     cudaMemcpyDeviceToHost));
  return FT_OK;
}

ft_status_t ft_moe_get_stats(ft_moe_t *h, int layer, uint64_t *counters, int n) {
  if (!h || layer < 0 || layer >= h->cfg.n_layers || !counters || n < 0) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  unsigned long long tmp[FT_STAT_COUNT];
  FT_CUDA(cudaMemcpy(tmp, h->layers[layer].stats, sizeof(tmp), cudaMemcpyDeviceToHost));
  for (int i = 0; i < n && i < FT_STAT_COUNT; ++i) counters[i] = tmp[i];
  return FT_OK;
}

ft_status_t ft_moe_sync_status(ft_moe_t *h) {
  if (!h) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  return drain_status(h);
}

ft_status_t ft_moe_last_fill(ft_moe_t *h, float *out_us, uint64_t *out_bytes) {
  if (!h) return FT_ERR_INVALID_ARG;
  if (out_us) *out_us = 0.f;
  if (out_bytes) *out_bytes = 0;
  if (!h->fill_timed) return FT_OK;
  FT_CUDA(cudaEventSynchronize(h->ev_fill_t1));
  float ms = 0.f;
  FT_CUDA(cudaEventElapsedTime(&ms, h->ev_fill_t0, h->ev_fill_t1));
  if (out_us) *out_us = ms * 1000.f;
  uint64_t bytes = h->last_fill_bytes;
  if (bytes == ~0ull) {
    PlanHeader hd;
    FT_CUDA(cudaMemcpy(&hd, scratch_of(h, h->last_fill_layer < 0 ? 0 : h->last_fill_layer).plan_dev, sizeof(hd),
                       cudaMemcpyDeviceToHost));
    bytes = (uint64_t)hd.n_fill * h->S;
  }
  if (out_bytes) *out_bytes = bytes;
  return FT_OK;
}

ft_status_t ft_moe_get_cta_trace(ft_moe_t *h, int64_t *out, int n_ctas) {
  if (!h || !out || n_ctas < 0) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  const int n = n_ctas < h->sm_count ? n_ctas : h->sm_count;
  FT_CUDA(cudaMemcpy(out, h->trace_dev, (size_t)n * 4 * sizeof(long long), cudaMemcpyDeviceToHost));
  return FT_OK;
}

ft_status_t ft_moe_resize(ft_moe_t *h, int slots_per_layer) {
  if (!h || slots_per_layer < 0) return FT_ERR_INVALID_ARG;
  if ((long long)slots_per_layer * (h->cfg.global_pool ? h->cfg.n_layers : 1) > kMaxTableSlots) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  for (auto &L : h->layers) L.phase = PH_IDLE;
  h->cfg.slots_per_layer = slots_per_layer;
  ft_status_t rc = alloc_cache(h);
  if (rc != FT_OK) {
    h->cfg.slots_per_layer = 0;
    (void)alloc_cache(h);
    return rc;
  }
  if (h->gemm) {   // the weight tensor maps of the prefill path are bound to the slot pool (bf16) or to the
                   // scratch pool of one layer's slots (4-bit), which follows the new slot count
    if (h->cfg.wdtype != FT_W_BF16) {
      cudaFree(h->wq_scratch);
      h->wq_scratch = nullptr;
      if (slots_per_layer > 0) {
        const cudaError_t e = cudaMalloc(&h->wq_scratch, (size_t)slots_per_layer * 3 * h->cfg.inter * h->cfg.hidden * 2);
        if (e != cudaSuccess) { (void)cudaGetLastError(); return FT_ERR_OOM; }
      }
    }
    rc = build_weight_maps(h);
    if (rc != FT_OK) return rc;
  }
  FT_CUDA(cudaDeviceSynchronize());
  return FT_OK;
}

ft_status_t ft_moe_set_split_min_pairs(ft_moe_t *h, int pairs) {
  if (!h || pairs < 0) return FT_ERR_INVALID_ARG;
  h->cfg.split_min_pairs = pairs;
  return FT_OK;
}

ft_status_t ft_moe_set_launch_overlap(ft_moe_t *h, int mode) {
  if (!h || mode < 0 || mode > 2) return FT_ERR_INVALID_ARG;
  h->overlap = mode;
  return FT_OK;
}

ft_status_t ft_moe_debug_inject(ft_moe_t *h, uint32_t withhold_mask, uint32_t wait_polls) {
  if (!h || (withhold_mask & ~15u)) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  const uint32_t polls = wait_polls ? wait_polls : kDefaultWaitPolls;
  FT_CUDA(cudaMemcpyToSymbol(g_debug_withhold, &withhold_mask, sizeof(uint32_t)));
  FT_CUDA(cudaMemcpyToSymbol(g_wait_polls, &polls, sizeof(uint32_t)));
  FT_CUDA(cudaDeviceSynchronize());
  return FT_OK;
}

ft_status_t ft_moe_launch_count(ft_moe_t *h, uint64_t *out) {
  if (!h || !out) return FT_ERR_INVALID_ARG;
  *out = h->launches;
  return FT_OK;
}

ft_status_t ft_moe_timing_enable(ft_moe_t *h, int on) {
  if (!h) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  timing_flush(h);
  for (int i = 0; i < FT_TIME_COUNT; ++i) { h->time_us[i] = 0.0; h->time_n[i] = 0; }
  h->timing = on != 0;
  return FT_OK;
}

ft_status_t ft_moe_timing_read(ft_moe_t *h, double *out_us, uint64_t *out_n, int n) {
  if (!h || !out_us || !out_n || n < 0) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  timing_flush(h);
  for (int i = 0; i < n && i < FT_TIME_COUNT; ++i) { out_us[i] = h->time_us[i]; out_n[i] = h->time_n[i]; }
  return FT_OK;
}

ft_status_t ft_moe_calibrate(ft_moe_t *h, uint32_t out_MBps[4]) {
  if (!h || !out_MBps) return FT_ERR_INVALID_ARG;
  FT_CUDA(cudaSetDevice(h->cfg.device));
  FT_CUDA(cudaDeviceSynchronize());
  const ft_moe_config_t &c = h->cfg;
  const size_t pool_records = (size_t)c.n_layers * c.n_experts;
  // sample: up to 256 MiB of pool records, at least one
  size_t n_rec = (256ull << 20) / h->S;
  if (n_rec < 1) n_rec = 1;
  if (n_rec > pool_records) n_rec = pool_records;
  const size_t bytes = n_rec * h->S;
  uint8_t *scratch = nullptr;
  uint32_t *sink = nullptr;
  FT_CUDA(cudaMalloc(&scratch, bytes));
  if (cudaMalloc(&sink, 4) != cudaSuccess) { cudaFree(scratch); (void)cudaGetLastError(); return FT_ERR_OOM; }
  cudaMemset(sink, 0, 4);
  cudaEvent_t e0, e1, e2, e3;
  cudaEventCreate(&e0); cudaEventCreate(&e1); cudaEventCreate(&e2); cudaEventCreate(&e3);
  const uint8_t *hp = static_cast<const uint8_t *>(c.host_pool);
  auto mbps = [](size_t b, float ms) { return (uint32_t)(ms > 0.f ? (double)b / (ms * 1e-3) / 1e6 : 0.0); };
  float best[4] = {1e30f, 1e30f, 1e30f, 1e30f};
  const int grid = h->sm_count * 4;
  for (int rep = 0; rep < 4; ++rep) {
    float ms;
    // (0) copy-engine fill rate: record-sized pinned H2D copies back to back
    cudaEventRecord(e0, h->copy_stream);
    for (size_t r = 0; r < n_rec; ++r)
      cudaMemcpyAsync(scratch + r * h->S, hp + r * h->S, h->S, cudaMemcpyHostToDevice, h->copy_stream);
    cudaEventRecord(e1, h->copy_stream);
    cudaEventSynchronize(e1);
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && ms < best[0]) best[0] = ms;
    // (1) zero-copy reads alone
    cudaEventRecord(e0, h->aux_stream);
    read_kernel<<<grid, 256, 0, h->aux_stream>>>(h->pool_dev, bytes, sink);
    cudaEventRecord(e1, h->aux_stream);
    cudaEventSynchronize(e1);
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && ms < best[1]) best[1] = ms;
    // (2) zero-copy reads while the copy engine is kept busy for the whole kernel
    cudaEventRecord(e2, h->copy_stream);
    for (int k = 0; k < 3; ++k)
      for (size_t r = 0; r < n_rec; ++r)
        cudaMemcpyAsync(scratch + r * h->S, hp + r * h->S, h->S, cudaMemcpyHostToDevice, h->copy_stream);
    cudaEventRecord(e3, h->copy_stream);
    cudaEventRecord(e0, h->aux_stream);
    read_kernel<<<grid, 256, 0, h->aux_stream>>>(h->pool_dev, bytes, sink);
    cudaEventRecord(e1, h->aux_stream);
    cudaEventSynchronize(e1);
    cudaEventSynchronize(e3);
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && ms < best[2]) best[2] = ms;
    // (3) HBM streaming reads
    cudaEventRecord(e0, h->aux_stream);
    read_kernel<<<grid, 256, 0, h->aux_stream>>>(scratch, bytes, sink);
    cudaEventRecord(e1, h->aux_stream);
    cudaEventSynchronize(e1);
    cudaEventElapsedTime(&ms, e0, e1);
    if (rep > 0 && ms < best[3]) best[3] = ms;
    h->launches += 3;
  }
  for (int i = 0; i < 4; ++i) out_MBps[i] = mbps(bytes, best[i]);
  cudaEventDestroy(e0); cudaEventDestroy(e1); cudaEventDestroy(e2); cudaEventDestroy(e3);
  cudaFree(scratch);
  cudaFree(sink);
  FT_CUDA(cudaDeviceSynchronize());
  FT_CUDA(cudaGetLastError());
  return FT_OK;
}

}  // extern "C"
