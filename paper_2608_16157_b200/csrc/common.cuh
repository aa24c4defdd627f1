// Shared device-side declarations of the expert-cached MoE layer library.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ftmoe {

constexpr int kMaxExperts = 1024;
constexpr int kMaxTopK = 32;
constexpr int kGroup = 128;  // int4 quantisation group

// Bits of the device status word (latched, reported by the next synchronising call).
constexpr uint32_t kStatNonFinite = 1u;
constexpr uint32_t kStatTimeout = 2u;
constexpr uint32_t kStatBadIndex = 4u;

constexpr int32_t kLocNotRouted = -1;
constexpr int32_t kLocZeroCopy = -2;

// One expert to evaluate: where its record is (slot in HBM, or the mapped host pool), which rows of
// the expert-sorted pair order belong to it.  expert < 0 marks the shared expert: its tokens are
// 0..n_tok-1 with gate weight 1.
struct __align__(16) WorkItem {
  const uint8_t *w;
  int32_t expert;
  int32_t n_tok;
  int32_t off;
  int32_t slot;
};

// Header of the plan record; 8 int32 arrays of n_experts entries follow it
// (hit, miss, fill, zc, fill_order, fill_slot, fill_evicted, loc).
struct PlanHeader {
  int64_t step;
  int32_t n_routed, n_hit, n_miss, n_fill, n_zc;
  int32_t n_res_items, n_zc_items, n_gemm_items;   // streaming list: [hits][shared][fills] = n_res_items, then zc
  uint32_t seq;      // incremented by every plan kernel; lets the host detect a stale record
  int32_t n_hit_items;   // leading entries of the streaming list that do not depend on this step's fills
  int32_t pad[4];
};
static_assert(sizeof(PlanHeader) == 64, "PlanHeader layout");

struct CostModelDev {
  int64_t ns_fill, ns_zc, ns_hbm;
  int64_t bw_fill, bw_res;
  int32_t reuse_credit, tz, tg, gemm_min_tokens;
};

__device__ __forceinline__ float bf16_bits_to_float(uint32_t hi16) { return __uint_as_float(hi16 << 16); }

__device__ __forceinline__ uint4 ld_stream_16(const void *p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld_stream_8(const void *p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

}  // namespace ftmoe
