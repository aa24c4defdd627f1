// Step 4, SM-driven variant: one fixed-shape launch applies the device-resident fill list
// (expert -> slot) of the plan record; the valid count masks unused work (paper Sec. 4.1).
// Also the read kernels used by the bandwidth calibration.
#pragma once
#include "common.cuh"

namespace ftmoe {

struct FillParams {
  const PlanHeader *hdr;          // device plan record
  int E;
  const uint8_t *pool_layer_dev;  // device alias of the host pool, first record of the layer
  uint8_t *slots_layer;
  size_t S;                       // multiple of 16
};

__global__ void __launch_bounds__(256) fill_kernel(FillParams p) {
  const int n_fill = p.hdr->n_fill;
  if (n_fill == 0) return;
  const int32_t *forder = reinterpret_cast<const int32_t *>(p.hdr + 1) + 4 * p.E;
  const int32_t *fslot = forder + p.E;
  const size_t chunks_per = p.S / 16;
  const size_t total = chunks_per * (size_t)n_fill;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  size_t c = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  // four independent 16-byte loads in flight per thread
  for (; c + 3 * stride < total; c += 4 * stride) {
    uint4 v[4];
    size_t dsti[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const size_t cc = c + i * stride;
      const int f = (int)(cc / chunks_per);
      const size_t within = cc - (size_t)f * chunks_per;
      v[i] = ld_stream_16(p.pool_layer_dev + (size_t)forder[f] * p.S + within * 16);
      dsti[i] = (size_t)fslot[f] * p.S + within * 16;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4 *>(p.slots_layer + dsti[i]) = v[i];
  }
  for (; c < total; c += stride) {
    const int f = (int)(c / chunks_per);
    const size_t within = c - (size_t)f * chunks_per;
    const uint4 v = ld_stream_16(p.pool_layer_dev + (size_t)forder[f] * p.S + within * 16);
    *reinterpret_cast<uint4 *>(p.slots_layer + (size_t)fslot[f] * p.S + within * 16) = v;
  }
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
