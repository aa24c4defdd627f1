// Step 4, device-driven variant: one fixed-shape launch applies the device-resident fill list
// (expert -> slot) of the plan record; the valid count masks unused work (paper Sec. 4.1).
// Also the read kernels used by the bandwidth calibration.
#pragma once
#include "common.cuh"
#include "async.cuh"

namespace ftmoe {

struct FillParams {
  const PlanHeader *hdr;          // device plan record
  int E;
  const uint8_t *pool_layer_dev;  // device alias of the host pool, first record of the layer
  uint8_t *slots_layer;
  size_t S;                       // multiple of 16
};

constexpr int kFillCtas = 2;             // the copy needs bytes in flight, not SMs: 2 CTAs x 4 x 32 KiB saturate the link
constexpr int kFillStages = 4;
constexpr uint32_t kFillChunk = 32768;   // bytes per bulk copy
constexpr int kFillThreads = 32;

// A few single-warp CTAs move the records with the bulk-copy engine: host pool -> shared memory
// (cp.async.bulk, completion on an mbarrier) -> slot (cp.async.bulk shared -> global).  No SM arithmetic, no
// registers per byte, and only kFillCtas SMs are touched (more CTAs were measured to slow the concurrent expert kernel without raising the link rate), so the expert kernel keeps the rest of the GPU
// while records stream in over the host link.
__global__ void __launch_bounds__(kFillThreads) fill_kernel(FillParams p, uint32_t *status) {
  extern __shared__ __align__(128) unsigned char smem[];
  __shared__ uint64_t s_bar[kFillStages];
  __shared__ volatile int s_abort;
  const int n_fill = p.hdr->n_fill;
  if (n_fill == 0 || threadIdx.x != 0) return;
  const int32_t *forder = reinterpret_cast<const int32_t *>(p.hdr + 1) + 4 * p.E;
  const int32_t *fslot = forder + p.E;
  const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(s_bar);
  for (int s = 0; s < kFillStages; ++s) mbar_init(bar_base + 8 * s, 1);
  s_abort = 0;
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  const long long chunks_per = (long long)((p.S + kFillChunk - 1) / kFillChunk);
  const long long total = chunks_per * n_fill;
  // chunk c of the call -> CTA c % gridDim.x; this CTA's i-th chunk is c = blockIdx.x + i * gridDim.x
  const long long mine = (total > blockIdx.x) ? (total - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
  auto locate = [&](long long i, const uint8_t *&src, uint8_t *&dst, uint32_t &bytes) {
    const long long c = blockIdx.x + i * gridDim.x;
    const int f = (int)(c / chunks_per);
    const size_t off = (size_t)(c - (long long)f * chunks_per) * kFillChunk;
    bytes = (uint32_t)((p.S - off < kFillChunk) ? (p.S - off) : kFillChunk);
    src = p.pool_layer_dev + (size_t)forder[f] * p.S + off;
    dst = p.slots_layer + (size_t)fslot[f] * p.S + off;
  };
  auto issue_load = [&](long long i) {
    const uint8_t *src; uint8_t *dst; uint32_t bytes;
    locate(i, src, dst, bytes);
    const int s = (int)(i % kFillStages);
    mbar_expect_tx(bar_base + 8 * s, bytes);
    if ((g_debug_withhold & kWithholdFill) && i == 0) return;   // test hook: this copy never arrives
    bulk_g2s(smem_base + s * kFillChunk, src, bytes, bar_base + 8 * s);
  };
  for (long long i = 0; i < mine && i < kFillStages; ++i) issue_load(i);
  for (long long i = 0; i < mine; ++i) {
    const int s = (int)(i % kFillStages);
    if (!mbar_wait(bar_base + 8 * s, (uint32_t)((i / kFillStages) & 1), &s_abort, status)) break;
    const uint8_t *src; uint8_t *dst; uint32_t bytes;
    locate(i, src, dst, bytes);
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(smem_base + s * kFillChunk),
                 "r"(bytes)
                 : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    if (i + kFillStages < mine) {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");   // the store has read the stage: refill it
      issue_load(i + kFillStages);
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  abort_drain(&s_abort);
}

// Reads `bytes` (multiple of 16) and folds them into one word so the loads cannot be elided.
__global__ void __launch_bounds__(256) read_kernel(const uint8_t *src, size_t bytes, uint32_t *sink) {
  const size_t n = bytes / 16;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  uint32_t acc = 0;
  size_t c = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (; c + 3 * stride < n; c += 4 * stride) {
    uint4 v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = ld_stream_16(src + (c + i * stride) * 16);
#pragma unroll
    for (int i = 0; i < 4; ++i) acc ^= v[i].x ^ v[i].y ^ v[i].z ^ v[i].w;
  }
  for (; c < n; c += stride) {
    const uint4 v = ld_stream_16(src + c * 16);
    acc ^= v.x ^ v.y ^ v.z ^ v.w;
  }
  if (acc == 0x9e3779b9u) atomicAdd(sink, 1u);
}

}  // namespace ftmoe
