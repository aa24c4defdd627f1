// Steps 5+6 for int4 (group 128, bf16 scales) experts at decode-sized token counts: two HBM-streaming kernels whose
// weight loads go straight from global memory into registers.  At 4 bits per weight the bound next to HBM is the
// integer/logic pipe that unpacks the codes, so the arithmetic is arranged for the cheapest unpacking there is:
//   * a 32-bit word holds 8 two's-complement codes; (w & 0x0F0F0F0F) ^ 0x08080808 and the same of w >> 4 are two
//     A-fragment registers of the int8 tensor-core instruction mma.sync.m16n8k32 (three logic instructions per 8
//     weights), holding code + 8;
//   * the bf16 activations of a (token, 128-element quantisation group) are re-expressed exactly once as 15-bit
//     fixed point against the group's largest magnitude m:  a ~ (m / 16256) * (128 hi + lo),  hi in [-127, 127],
//     lo in [0, 127]; hi and lo are the int8 B operands of two MMAs whose int32 sums are exact.  The representation
//     error is at most m / 32512 per element, i.e. below the rounding of the largest element to bf16 (m / 512);
//   * per group and output:  scale_w * ( (m / 16256) * (128 S_hi + S_lo) - 8 (m / 16256) sum(128 hi + lo) )  in fp32
//     (the second term removes the + 8 of the codes).
//   w4_gateup_kernel : 16 warps per SM; the work is cut into pieces = (16-neuron unit, half of the hidden dimension)
//                      and every warp streams its share of consecutive pieces by itself (gate tiles, up tiles and
//                      their scales of a unit are contiguous): no block-level synchronisation while a call has at
//                      most 8 tokens, and an even share per warp at every batch size.  A lane's two 16-byte loads
//                      per quantisation group are rows g and g+8 of the group's tile; a rolling register buffer is
//                      refilled as soon as a step has been consumed.  A piece's partial gate and up sums are added
//                      (red.global.add) into the unit's fp32 accumulators; the warp that completes a group of 128
//                      neurons of a pass (an arrival counter per group; nobody waits) applies SiLU(g) * u, converts
//                      the group to the fixed-point form above for the down kernel and clears the accumulators.
//   w4_down_kernel   : walks chunks (expert pass, block of 64*NWD output columns, group of 128 neurons) = 8 steps
//                      of 16 neurons x 512 bytes per warp.  Every warp owns four 16-column tiles: its 16-byte load
//                      per step is their A fragments.  No block-level synchronisation: a warp stages the chunk's h
//                      operands and scales for itself with cp.async.  The fold to fp32 happens when the chunk (= one
//                      neuron group) ends; the totals persist while consecutive chunks belong to the same pass and
//                      column block.  The gate-weighted combine is a red.global.add into the fp32 accumulator; the
//                      last CTA rounds it once to bf16.  Launched as a programmatic dependent of the gate/up
//                      kernel: its set-up overlaps that kernel's tail.
// Zero-copy experts (records in the mapped host pool) go through the same kernels.
#pragma once
#include "async.cuh"
#include "common.cuh"
#include "ffn_stream.cuh"   // red_add_f32

namespace ftmoe {

constexpr int kQ4Tokens = 8;         // tokens per weight pass
constexpr int kW4Threads = 512;
constexpr int kW4Warps = kW4Threads / 32;
constexpr float kW4Levels = 16256.f; // 127 * 128: |fixed-point activation| <= this
#ifndef W4_BS
#define W4_BS 2
#endif
constexpr int kW4KSplit = 2;             // a unit's hidden dimension is split into this many pieces of work
constexpr int kW4BlockSteps = W4_BS;     // depth of the gate/up kernel's rolling register buffer, in quantisation groups

struct W4Params {
  const WorkItem *items;
  const int32_t *n_items;   // resident items
  const int32_t *n_zc;      // zero-copy items appended after them
  const int32_t *pref;      // exclusive prefix of the weight passes (8 tokens each) per item
  int max_items;
  const __nv_bfloat16 *x;   // [T][d]
  const int32_t *perm;
  const float *topk_w;
  float *hraw;              // [pass][16-neuron unit][gate sums | up sums][token 8][neuron 16] fp32, zero between calls
  int32_t *hcount;          // [pass][128-neuron group]: pieces of the group added so far (self-resetting)
  uint8_t *hq;              // [pass][group][unit pair 4][token 8][q 4][hi u0, hi u1, lo u0, lo u1 : 4 neurons each]
  float2 *hs;               // [pass][group][token 8]: (m / 16256, 8 (m / 16256) sum of the fixed-point values)
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;
  uint32_t *done;
  uint32_t *status;
  int inter, top_k, T, finalize;
  int overlap;              // launch mode of the gate/up kernel, as FfnStreamParams::overlap (0 plain, 1, 2)
  // 0x0F0F0F0F and 0x08080808, passed as data: as literals the compiler encodes both as immediates and needs two
  // logic instructions per register (an instruction carries one immediate); as values it cannot see through they
  // live in registers and (x & mask) ^ flip is a single three-input logic instruction
  uint32_t mask, flip;
};

__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ void mma_s8(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                       uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+r"(c[0]), "+r"(c[1]), "+r"(c[2]), "+r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
// d = a * b (no accumulator to clear first)
__device__ __forceinline__ void mma_s8_first(int (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=r"(c[0]), "=r"(c[1]), "=r"(c[2]), "=r"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "r"(0));
}

// 8 values of one (token, group) -> fixed point against the group's largest magnitude `m` (already reduced over the
// group): hi/lo bytes of elements (0,2,4,6) and (1,3,5,7) -- the order in which w & 0x0F0F0F0F and (w >> 4) & ...
// deliver the codes of a word -- and the sum of the 8 fixed-point values.
struct W4Fixed { uint32_t hi_even, hi_odd, lo_even, lo_odd; int sum; };
__device__ __forceinline__ W4Fixed w4_to_fixed(const float (&f)[8], float inv) {
  int v[8];
  W4Fixed r;
  r.sum = 0;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    v[i] = __float2int_rn(f[i] * inv);
    r.sum += v[i];
  }
  auto pack = [](int a, int b, int c, int d_) {
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) | ((uint32_t)(d_ & 0xff) << 24);
  };
  r.hi_even = pack(v[0] >> 7, v[2] >> 7, v[4] >> 7, v[6] >> 7);
  r.hi_odd = pack(v[1] >> 7, v[3] >> 7, v[5] >> 7, v[7] >> 7);
  r.lo_even = pack(v[0] & 127, v[2] & 127, v[4] & 127, v[6] & 127);
  r.lo_odd = pack(v[1] & 127, v[3] & 127, v[5] & 127, v[7] & 127);
  return r;
}
// Scale of a group with largest magnitude m (non-finite inputs flagged by `bad`): value = scale * fixed, fixed =
// rint(value * inv).  A non-finite input makes the scale NaN, so that it reaches the output as it would in bf16.
__device__ __forceinline__ void w4_group_scale(float m, bool bad, float &scale, float &inv) {
  if (bad) { scale = __int_as_float(0x7fc00000); inv = 0.f; }
  else if (m < 1e-30f) { scale = 0.f; inv = 0.f; }
  else { scale = m * (1.f / kW4Levels); inv = kW4Levels / m; }
}

// Share number `who` of `total` work items split over `n`: total/n each, the first total%n one more.
__device__ __forceinline__ uint32_t w4_first(uint32_t total, uint32_t n, uint32_t who) {
  const uint32_t per = total / n, rem = total - per * n;
  return who * per + min(who, rem);
}
// Largest i in [0, n) with pref[i] <= v  (pref is non-decreasing, pref[0] = 0).
__device__ __forceinline__ int w4_find_item(const int32_t *pref, int n, uint32_t v) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((uint32_t)pref[mid] <= v) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Dynamic shared memory of the gate/up kernel: x [8][2d + 64] bytes (per run of 8 elements: hi bytes of elements
// 0,2,4,6 | hi of 1,3,5,7 | lo of 0,2,4,6 | lo of 1,3,5,7) | per (token, group): scale [8][G], bias [8][G] f32 |
// items [max_items] | pref [max_items + 1].
inline size_t w4_gateup_smem_bytes(int max_items, int d) {
  return (size_t)8 * (2 * d + 64) + (size_t)2 * 8 * (d / kGroup) * 4 + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}
// ... of the down kernel: per warp 2 slots of (h operands 2048 | 128 bytes of weight scales | 64 bytes of
// (scale, bias) per token) | items | pref.
constexpr uint32_t kW4DownSlot = 2048 + 128 + 64;
inline size_t w4_down_smem_bytes(int max_items) {
  return (size_t)kW4Warps * 2 * kW4DownSlot + (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}

template <int G>   // quantisation groups of the hidden dimension: d = 128 G, G a multiple of 4
__global__ void __launch_bounds__(kW4Threads, 1) w4_gateup_kernel(W4Params p) {
  constexpr int d = kGroup * G;
  constexpr uint32_t kUA = 2112u * G;               // bytes of a unit: gate tiles, up tiles, gate scales, up scales
  constexpr uint32_t kXStride = 2u * d + 64u;
  constexpr int kBS = kW4BlockSteps;                // steps of a block = depth of the rolling register buffer
  constexpr int kBlocks = G / kBS;                  // blocks of a unit
  constexpr int kKS = kW4KSplit, kBlocksP = kBlocks / kKS;   // blocks of a piece
  static_assert(G % kBS == 0 && kBlocks % kKS == 0, "whole blocks, whole pieces");
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_x = smem;
  float *s_sx = reinterpret_cast<float *>(s_x + 8 * kXStride);             // [8][G] m / 16256
  float *s_xb = s_sx + 8 * G;                                              // [8][G] 8 (m / 16256) sum(fixed)
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_xb + 8 * G);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the down kernel may set itself up meanwhile
  if (p.overlap == 1) asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  for (int i = tid; i <= p.max_items; i += kW4Threads) s_pref[i] = p.pref[i];
  {
    const uint4 *src = reinterpret_cast<const uint4 *>(p.items);
    uint4 *dst = reinterpret_cast<uint4 *>(s_items);
    for (int i = tid; i < 2 * p.max_items; i += kW4Threads) dst[i] = src[i];
  }
  __syncthreads();
  const uint32_t NBLK = (uint32_t)p.inter / 16u;
  const bool dense = p.T <= kQ4Tokens;

  // x rows of the MMA columns into shared memory as fixed point per (token, quantisation group)
  auto stage_x = [&](auto tok_of_column) {
    for (int i = tid; i < 8 * (d / 8); i += kW4Threads) {
      const int j = i / (d / 8), c8 = i - j * (d / 8);
      const int tok = tok_of_column(j);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok >= 0) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 8 * c8);
      const float f[8] = {bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y), bf16lo(v.z), bf16hi(v.z), bf16lo(v.w), bf16hi(v.w)};
      float m = 0.f;
      bool bad = false;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        m = fmaxf(m, fabsf(f[e]));
        bad |= !(fabsf(f[e]) <= 3.0e38f);
      }
#pragma unroll
      for (int o2 = 1; o2 < 16; o2 <<= 1) {   // 16 chunks = one group
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o2));
        bad |= __shfl_xor_sync(0xffffffffu, (int)bad, o2) != 0;
      }
      float scale, inv;
      w4_group_scale(m, bad, scale, inv);
      const W4Fixed fx = w4_to_fixed(f, inv);
      *reinterpret_cast<uint4 *>(s_x + j * kXStride + 16 * c8) = make_uint4(fx.hi_even, fx.hi_odd, fx.lo_even, fx.lo_odd);
      int sum = fx.sum;
#pragma unroll
      for (int o2 = 1; o2 < 16; o2 <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
      if ((lane & 15) == 0) {
        s_sx[j * G + c8 / 16] = scale;
        s_xb[j * G + c8 / 16] = 8.f * (float)sum * scale;
      }
    }
  };

  const uint32_t my_x = smem_u32(s_x) + g * kXStride + 16u * q;
  const uint32_t km = p.mask, kf = p.flip;
  const float *my_s0 = s_sx + (2 * q) * G, *my_s1 = s_sx + (2 * q + 1) * G;
  const float *my_b0 = s_xb + (2 * q) * G, *my_b1 = s_xb + (2 * q + 1) * G;

  // The warp that completes a group of 128 neurons of a pass converts it to fixed point for the down kernel:
  // lane = (token, quarter): the quarter's two units of 16 neurons.
  auto convert_group = [&](uint32_t grp) {
    const int tok = lane >> 2, qt = lane & 3;
    float *src = p.hraw + ((size_t)grp * 8 + 2 * qt) * 256 + tok * 16;   // per unit: gate sums [8][16], up sums [8][16]
    float v[2][16];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        float4 *pg = reinterpret_cast<float4 *>(src + u * 256) + k4, *pu_ = reinterpret_cast<float4 *>(src + u * 256 + 128) + k4;
        const float4 a = __ldcg(pg), b = __ldcg(pu_);
        __stcg(pg, make_float4(0.f, 0.f, 0.f, 0.f));   // the sums start from zero in the next call
        __stcg(pu_, make_float4(0.f, 0.f, 0.f, 0.f));
        v[u][4 * k4] = __fdividef(a.x, 1.f + __expf(-a.x)) * b.x;
        v[u][4 * k4 + 1] = __fdividef(a.y, 1.f + __expf(-a.y)) * b.y;
        v[u][4 * k4 + 2] = __fdividef(a.z, 1.f + __expf(-a.z)) * b.z;
        v[u][4 * k4 + 3] = __fdividef(a.w, 1.f + __expf(-a.w)) * b.w;
      }
    float m = 0.f;
    bool bad = false;
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
      for (int k = 0; k < 16; ++k) {
        m = fmaxf(m, fabsf(v[u][k]));
        bad |= !(fabsf(v[u][k]) <= 3.0e38f);
      }
#pragma unroll
    for (int o = 1; o < 4; o <<= 1) {   // the token's four quarters
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      bad |= __shfl_xor_sync(0xffffffffu, (int)bad, o) != 0;
    }
    float scale, inv;
    w4_group_scale(m, bad, scale, inv);
    int sum = 0;
    uint8_t *dst = p.hq + (size_t)grp * 2048 + qt * 512 + tok * 64;
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {   // neurons 4qq..4qq+3 of both units: (hi u0, hi u1, lo u0, lo u1)
      int w[8];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        w[k] = __float2int_rn(v[0][4 * qq + k] * inv);
        w[4 + k] = __float2int_rn(v[1][4 * qq + k] * inv);
      }
      uint32_t o[4] = {0u, 0u, 0u, 0u};
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        sum += w[k] + w[4 + k];
        o[0] |= (uint32_t)((w[k] >> 7) & 0xff) << (8 * k);
        o[1] |= (uint32_t)((w[4 + k] >> 7) & 0xff) << (8 * k);
        o[2] |= (uint32_t)(w[k] & 127) << (8 * k);
        o[3] |= (uint32_t)(w[4 + k] & 127) << (8 * k);
      }
      *reinterpret_cast<uint4 *>(dst + qq * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    if (qt == 0) p.hs[(size_t)grp * 8 + tok] = make_float2(scale, 8.f * (float)sum * scale);
  };

  // One warp streams `n_pieces` consecutive pieces (a unit's hidden dimension in kKS parts), starting with part ks0
  // of the unit at `base`; the pieces' partial gate / up sums are added into rows hrow0.. of the h buffer.
  // A step is one quantisation group of the hidden dimension: the gate tile and the up tile of that group, which
  // share their activation fragments.  Registers hold kBS steps; a step's registers are refilled with the step
  // kBS further on as soon as it has been consumed.
  auto run = [&](const uint8_t *base, int ks0, int n_pieces, uint32_t hrow0) {
    uint4 buf[4 * kBS];     // per step: gate rows g, g+8; up rows g, g+8
    uint32_t sc[2 * kBS];   // and their scales
    const uint8_t *nptr = base + ks0 * (G / kKS) * 1024 + g * 64 + q * 16;   // next block to request (its gate tiles)
    const uint8_t *nsc = base + 2048u * G + ks0 * (G / kKS) * 32 + g * 4;
    int nblk = ks0 * kBlocksP, blocks_left = n_pieces * kBlocksP;   // its index in its unit; blocks not yet requested
    auto advance = [&]() {
      nptr += kBS * 1024;
      nsc += kBS * 32;
      --blocks_left;
      if (++nblk == kBlocks) {   // on to the next unit
        nblk = 0;
        nptr += kUA - 1024u * G;
        nsc += kUA - 32u * G;
      }
    };
    auto request = [&](int si, const uint8_t *tp, const uint8_t *sp) {
      buf[4 * si] = ld_stream_16(tp + si * 1024);
      buf[4 * si + 1] = ld_stream_16(tp + si * 1024 + 512);
      buf[4 * si + 2] = ld_stream_16(tp + si * 1024 + 1024 * G);
      buf[4 * si + 3] = ld_stream_16(tp + si * 1024 + 1024 * G + 512);
      asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(sc[2 * si]) : "l"(sp + si * 32));
      asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(sc[2 * si + 1]) : "l"(sp + si * 32 + 32 * G));
    };
#pragma unroll
    for (int si = 0; si < kBS; ++si) request(si, nptr, nsc);
    advance();
    int ks = ks0;
    uint32_t hrow_i = hrow0;
    for (int piece = 0; piece < n_pieces; ++piece) {
      float tg[4] = {0.f, 0.f, 0.f, 0.f}, tot[4] = {0.f, 0.f, 0.f, 0.f};   // gate sums, up sums
      for (int blk = 0; blk < kBlocksP; ++blk) {
        const bool more = blocks_left > 0;
        const uint8_t *rp = nptr, *rs = nsc;         // the block that refills this one's registers
        if (more) advance();
        const int xg = ks * (G / kKS) + blk * kBS;   // first group of the block
        const uint32_t xa = my_x + xg * 256u;
#pragma unroll
        for (int si = 0; si < kBS; ++si) {
          int gh[4], gl[4], uh[4], ul[4];
          const uint32_t glo[4] = {buf[4 * si].x, buf[4 * si].y, buf[4 * si].z, buf[4 * si].w};
          const uint32_t ghi[4] = {buf[4 * si + 1].x, buf[4 * si + 1].y, buf[4 * si + 1].z, buf[4 * si + 1].w};
          const uint32_t ulo[4] = {buf[4 * si + 2].x, buf[4 * si + 2].y, buf[4 * si + 2].z, buf[4 * si + 2].w};
          const uint32_t uhi[4] = {buf[4 * si + 3].x, buf[4 * si + 3].y, buf[4 * si + 3].z, buf[4 * si + 3].w};
          const uint32_t gscale = sc[2 * si], uscale = sc[2 * si + 1];
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // word j: hidden indices 32j + 8q + 0..7 of the group, rows g and g+8
            const uint4 xv = lds_v4(xa + si * 256u + j * 64u);
            const uint32_t a0 = (glo[j] & km) ^ kf, a1 = (ghi[j] & km) ^ kf;
            const uint32_t a2 = ((glo[j] >> 4) & km) ^ kf, a3 = ((ghi[j] >> 4) & km) ^ kf;
            const uint32_t c0 = (ulo[j] & km) ^ kf, c1 = (uhi[j] & km) ^ kf;
            const uint32_t c2 = ((ulo[j] >> 4) & km) ^ kf, c3 = ((uhi[j] >> 4) & km) ^ kf;
            if (j == 0) {
              mma_s8_first(gh, a0, a1, a2, a3, xv.x, xv.y);
              mma_s8_first(gl, a0, a1, a2, a3, xv.z, xv.w);
              mma_s8_first(uh, c0, c1, c2, c3, xv.x, xv.y);
              mma_s8_first(ul, c0, c1, c2, c3, xv.z, xv.w);
            } else {
              mma_s8(gh, a0, a1, a2, a3, xv.x, xv.y);
              mma_s8(gl, a0, a1, a2, a3, xv.z, xv.w);
              mma_s8(uh, c0, c1, c2, c3, xv.x, xv.y);
              mma_s8(ul, c0, c1, c2, c3, xv.z, xv.w);
            }
          }
          if (more) request(si, rp, rs);   // refill the step just consumed
          const float sx0 = my_s0[xg + si], sx1 = my_s1[xg + si], b0 = my_b0[xg + si], b1 = my_b1[xg + si];
          {
            const float s_lo = bf16lo(gscale), s_hi = bf16hi(gscale);
            tg[0] += s_lo * ((float)(gh[0] * 128 + gl[0]) * sx0 - b0);
            tg[1] += s_lo * ((float)(gh[1] * 128 + gl[1]) * sx1 - b1);
            tg[2] += s_hi * ((float)(gh[2] * 128 + gl[2]) * sx0 - b0);
            tg[3] += s_hi * ((float)(gh[3] * 128 + gl[3]) * sx1 - b1);
          }
          {
            const float s_lo = bf16lo(uscale), s_hi = bf16hi(uscale);
            tot[0] += s_lo * ((float)(uh[0] * 128 + ul[0]) * sx0 - b0);
            tot[1] += s_lo * ((float)(uh[1] * 128 + ul[1]) * sx1 - b1);
            tot[2] += s_hi * ((float)(uh[2] * 128 + ul[2]) * sx0 - b0);
            tot[3] += s_hi * ((float)(uh[3] * 128 + ul[3]) * sx1 - b1);
          }
        }
      }
      // the piece's gate and up sums of neurons g, g+8 and tokens 2q, 2q+1 join the unit's sums
      float *hacc = p.hraw + (size_t)hrow_i * 256;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int at = (2 * q + (i & 1)) * 16 + g + 8 * (i >> 1);
        red_add_f32(hacc + at, tg[i]);
        red_add_f32(hacc + 128 + at, tot[i]);
      }
      // the last piece of a 128-neuron group (8 units x kKS pieces) to arrive converts the group
      __threadfence();
      __syncwarp();
      int old = 0;
      if (lane == 0) old = atomicAdd(p.hcount + (hrow_i >> 3), 1);
      old = __shfl_sync(0xffffffffu, old, 0);
      if (old == 8 * kKS - 1) {
        __threadfence();
        convert_group(hrow_i >> 3);
        if (lane == 0) p.hcount[hrow_i >> 3] = 0;
      }
      if (++ks == kKS) { ks = 0; ++hrow_i; }
    }
  };

  if (dense) {
    stage_x([&](int j) { return j < p.T ? j : -1; });
    __syncthreads();
  }
  // launched as a programmatic dependent with the caller's word that x and the plan are not produced by the
  // preceding kernel: only from here on (the h buffers, shared with that kernel) must it have completed
  if (p.overlap == 2) asm volatile("griddepcontrol.wait;" ::: "memory");
  // Pieces (pass, 16-neuron unit, part of the hidden dimension) in one flat order, split evenly over all warps of
  // the grid: the slot-resident range first, then the host-resident range.
  const uint32_t n_warps = gridDim.x * kW4Warps, wi = blockIdx.x * kW4Warps + warp;
  for (int range = 0; range < 2; ++range) {
    const uint32_t pass0 = range ? (uint32_t)s_pref[n_items] : 0u;
    const uint32_t pass1 = range ? (uint32_t)s_pref[n_items + n_zc] : (uint32_t)s_pref[n_items];
    const uint32_t PP = NBLK * kKS;                  // pieces of a pass
    const uint32_t total = (pass1 - pass0) * PP, ubase = pass0 * PP;
    if (total == 0) continue;
    const uint32_t wf = ubase + w4_first(total, n_warps, wi), we = ubase + w4_first(total, n_warps, wi + 1);
    const uint32_t cf = ubase + w4_first(total, n_warps, blockIdx.x * kW4Warps);
    const uint32_t ce = ubase + w4_first(total, n_warps, (blockIdx.x + 1) * kW4Warps);
    if (cf >= ce) continue;
    for (uint32_t pu = cf / PP; pu * PP < ce; ++pu) {   // the passes this CTA's warps touch
      const int item = w4_find_item(s_pref, n_items + n_zc, pu);
      const WorkItem &it = s_items[item];
      if (!dense) {   // MMA column j is the pass's j-th pair: stage those tokens' rows
        const int tok0 = (int)(pu - (uint32_t)s_pref[item]) * kQ4Tokens, nt = min(kQ4Tokens, it.n_tok - tok0);
        const int off_ = it.off + tok0, expert_ = it.expert;
        __syncthreads();   // the previous pass's readers are done
        stage_x([&](int j) {
          if (j >= nt) return -1;
          return expert_ >= 0 ? p.perm[off_ + j] / p.top_k : tok0 + j;
        });
        __syncthreads();
      }
      const uint32_t lo = max(wf, pu * PP), hi = min(we, (pu + 1) * PP);
      if (lo < hi) {
        const uint32_t rel = lo - pu * PP;
        run(it.w + (size_t)(rel / kKS) * kUA, (int)(rel % kKS), (int)(hi - lo), pu * NBLK + rel / kKS);
      }
    }
  }
}

template <int NWD>   // warps that own output columns: a column block is 64 * NWD columns
__global__ void __launch_bounds__(kW4Threads, 1) w4_down_kernel(W4Params p, int d) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_h = smem;                                                // [16 warps][2 slots]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(smem + kW4Warps * 2 * kW4DownSlot);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  for (int i = tid; i <= p.max_items; i += kW4Threads) s_pref[i] = p.pref[i];
  {
    const uint4 *src = reinterpret_cast<const uint4 *>(p.items);
    uint4 *dst = reinterpret_cast<uint4 *>(s_items);
    for (int i = tid; i < 2 * p.max_items; i += kW4Threads) dst[i] = src[i];
  }
  __syncthreads();
  const uint32_t NBLK = (uint32_t)p.inter / 16u, NG = (uint32_t)p.inter / 128u;
  const uint32_t G = (uint32_t)d / 128u, CB = (uint32_t)d / (64u * NWD);
  const size_t sec_b = (size_t)NBLK * 2112u * G, sec_c = sec_b + (size_t)p.inter * d / 2;
  const uint32_t per_pass = CB * NG;                // chunks of one pass, neuron group fastest
  const bool dense = p.T <= kQ4Tokens;
  // everything above reads only what was ready before the gate/up kernel; from here on its h is needed
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < NWD) {
    const uint32_t t0 = (uint32_t)s_pref[n_items] * per_pass;
    const uint32_t t1 = (uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * per_pass;
    const uint32_t rfirst0 = w4_first(t0, gridDim.x, blockIdx.x), rcount0 = w4_first(t0, gridDim.x, blockIdx.x + 1) - rfirst0;
    const uint32_t rfirst1 = t0 + w4_first(t1, gridDim.x, blockIdx.x);
    const uint32_t rcount1 = t0 + w4_first(t1, gridDim.x, blockIdx.x + 1) - rfirst1;
    const uint32_t my_h = smem_u32(s_h) + (uint32_t)warp * 2u * kW4DownSlot;
    const uint32_t km = p.mask, kf = p.flip;

    // chunk cursor: (pass pu, column block cb, neuron group ng), advanced without divisions
    struct Ck { const uint8_t *rec; uint32_t pu, cb, ng; int item; };
    int range = 0, item = 0;
    uint32_t left = 0;
    Ck cur;
    cur.pu = cur.cb = cur.ng = 0; cur.item = 0; cur.rec = nullptr;
    auto next_chunk = [&](Ck &c) -> bool {
      if (left == 0) {
        while (left == 0) {
          if (range == 2) return false;
          left = range ? rcount1 : rcount0;
          const uint32_t first = range ? rfirst1 : rfirst0;
          ++range;
          if (left) {
            cur.pu = first / per_pass;
            const uint32_t r = first - cur.pu * per_pass;
            cur.cb = r / NG;
            cur.ng = r - cur.cb * NG;
          }
        }
      } else if (++cur.ng == NG) {
        cur.ng = 0;
        if (++cur.cb == CB) { cur.cb = 0; ++cur.pu; }
      }
      while ((uint32_t)s_pref[item + 1] <= cur.pu) ++item;
      cur.item = item;
      cur.rec = s_items[item].w;
      c = cur;
      --left;
      return true;
    };
    // the chunk's h operands (2 KiB, contiguous), its weight scales and the per-token (scale, bias) for this warp alone
    auto stage = [&](const Ck &c, uint32_t slot) {
      const size_t grp = (size_t)c.pu * NG + c.ng;
      const uint8_t *hsrc = p.hq + grp * 2048;
      const uint32_t dst = my_h + slot * kW4DownSlot;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (i * 32 + lane) * 16u), "l"(hsrc + (i * 32 + lane) * 16)
                     : "memory");
      if (lane < 8)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2048u + lane * 16u),
                     "l"(c.rec + sec_c + ((size_t)(c.ng * CB + c.cb) * NWD + warp) * 128u + lane * 16u)
                     : "memory");
      else if (lane < 12)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2176u + (lane - 8) * 16u),
                     "l"(reinterpret_cast<const uint8_t *>(p.hs + grp * 8) + (lane - 8) * 16)
                     : "memory");
    };
    auto weights_of = [&](const Ck &c) -> const uint8_t * {
      return c.rec + sec_b + ((size_t)(c.cb * NG + c.ng) * 8u * NWD + warp) * 512u + lane * 16u;
    };

    float dtot[4][4];
    auto zero_tot = [&]() {
#pragma unroll
      for (int j = 0; j < 4; ++j) { dtot[j][0] = dtot[j][1] = dtot[j][2] = dtot[j][3] = 0.f; }
    };
    int my_tok = -1;
    float my_w = 0.f;
    int nt = 0;
    auto begin_pass = [&](const Ck &c) {   // tokens and gate weights of the pass (used at the flush)
      const WorkItem &it = s_items[c.item];
      const int tok0 = (int)(c.pu - (uint32_t)s_pref[c.item]) * kQ4Tokens;
      nt = min(kQ4Tokens, it.n_tok - tok0);
      my_tok = -1;
      my_w = 0.f;
      if (lane < nt) {
        if (it.expert >= 0) {
          const int pr = p.perm[it.off + tok0 + lane];
          my_tok = pr / p.top_k;
          my_w = p.topk_w[pr];
        } else {
          my_tok = tok0 + lane;
          my_w = 1.f;
        }
      }
    };
    auto flush = [&](uint32_t cb) {
      int tok_a, tok_b;
      float gw_a, gw_b;
      if (dense) {
        tok_a = tok_b = -1;
        gw_a = gw_b = 0.f;
        for (int i = 0; i < nt; ++i) {
          const int ti = __shfl_sync(0xffffffffu, my_tok, i);
          const float wi = __shfl_sync(0xffffffffu, my_w, i);
          if (ti == 2 * q) { tok_a = ti; gw_a = wi; }
          if (ti == 2 * q + 1) { tok_b = ti; gw_b = wi; }
        }
      } else {
        tok_a = __shfl_sync(0xffffffffu, my_tok, 2 * q);
        tok_b = __shfl_sync(0xffffffffu, my_tok, 2 * q + 1);
        gw_a = __shfl_sync(0xffffffffu, my_w, 2 * q);
        gw_b = __shfl_sync(0xffffffffu, my_w, 2 * q + 1);
      }
      const int col0 = (int)cb * 64 * NWD + warp * 64 + g;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (tok_a >= 0) {
          red_add_f32(p.y_acc + (size_t)tok_a * d + col0 + 16 * j, gw_a * dtot[j][0]);
          red_add_f32(p.y_acc + (size_t)tok_a * d + col0 + 16 * j + 8, gw_a * dtot[j][2]);
        }
        if (tok_b >= 0) {
          red_add_f32(p.y_acc + (size_t)tok_b * d + col0 + 16 * j, gw_b * dtot[j][1]);
          red_add_f32(p.y_acc + (size_t)tok_b * d + col0 + 16 * j + 8, gw_b * dtot[j][3]);
        }
      }
    };

    uint4 buf[8];             // the chunk's eight steps; a step's register is refilled with the same step of the
                              // next chunk as soon as it has been consumed
    Ck c0, c1;                // the chunk being consumed and the one after it
    bool h0 = next_chunk(c0), h1 = h0 && next_chunk(c1);
    if (h0) {
      stage(c0, 0);
      const uint8_t *w = weights_of(c0);
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) buf[uu] = ld_stream_16(w + (size_t)uu * NWD * 512u);
      begin_pass(c0);
      zero_tot();
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    uint32_t slot = 0;
    while (h0) {
      if (h1) stage(c1, slot ^ 1u);
      asm volatile("cp.async.commit_group;" ::: "memory");
      const uint8_t *refill = h1 ? weights_of(c1) : nullptr;
      asm volatile("cp.async.wait_group 1;" ::: "memory");   // this chunk's staged data have landed
      __syncwarp();
      const uint32_t hs_base = my_h + slot * kW4DownSlot;
      int ah[4][4], al[4][4];
#pragma unroll
      for (int m = 0; m < 4; ++m) {   // unit pair m: neurons 32m .. 32m+31 of the group
        const uint4 hv = lds_v4(hs_base + m * 512u + g * 64u + q * 16u);   // token g: (hi u0, hi u1, lo u0, lo u1)
        const uint32_t w0[4] = {buf[2 * m].x, buf[2 * m].y, buf[2 * m].z, buf[2 * m].w};
        const uint32_t w1[4] = {buf[2 * m + 1].x, buf[2 * m + 1].y, buf[2 * m + 1].z, buf[2 * m + 1].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {   // tile j: columns g (even codes) and g+8 (odd codes)
          const uint32_t a0 = (w0[j] & km) ^ kf, a1 = ((w0[j] >> 4) & km) ^ kf;
          const uint32_t a2 = (w1[j] & km) ^ kf, a3 = ((w1[j] >> 4) & km) ^ kf;
          if (m == 0) {
            mma_s8_first(ah[j], a0, a1, a2, a3, hv.x, hv.y);
            mma_s8_first(al[j], a0, a1, a2, a3, hv.z, hv.w);
          } else {
            mma_s8(ah[j], a0, a1, a2, a3, hv.x, hv.y);
            mma_s8(al[j], a0, a1, a2, a3, hv.z, hv.w);
          }
        }
        if (refill) {
          buf[2 * m] = ld_stream_16(refill + (size_t)(2 * m) * NWD * 512u);
          buf[2 * m + 1] = ld_stream_16(refill + (size_t)(2 * m + 1) * NWD * 512u);
        }
      }
      const uint4 sc = lds_v4(hs_base + 2048u + g * 16u);   // (column g, column g + 8) of the warp's four tiles
      const uint4 tb = lds_v4(hs_base + 2176u + q * 16u);   // tokens 2q, 2q+1: (scale, bias) each
      __syncwarp();   // every lane has read the slot: it may be overwritten
      const float sh0 = __uint_as_float(tb.x), b0 = __uint_as_float(tb.y), sh1 = __uint_as_float(tb.z), b1 = __uint_as_float(tb.w);
      const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float s_lo = bf16lo(sw[j]), s_hi = bf16hi(sw[j]);
        dtot[j][0] += s_lo * ((float)(ah[j][0] * 128 + al[j][0]) * sh0 - b0);
        dtot[j][1] += s_lo * ((float)(ah[j][1] * 128 + al[j][1]) * sh1 - b1);
        dtot[j][2] += s_hi * ((float)(ah[j][2] * 128 + al[j][2]) * sh0 - b0);
        dtot[j][3] += s_hi * ((float)(ah[j][3] * 128 + al[j][3]) * sh1 - b1);
      }
      if (!h1 || c1.pu != c0.pu || c1.cb != c0.cb) {
        flush(c0.cb);
        zero_tot();
        if (h1 && c1.pu != c0.pu) begin_pass(c1);
      }
      c0 = c1;
      h0 = h1;
      h1 = h0 && next_chunk(c1);
      slot ^= 1u;
    }
  }

  // ---- the last CTA to finish rounds the accumulator to bf16 and clears it ----
  if (!p.finalize) return;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t prev = atomicAdd(p.done, 1u);
    s_last = (prev == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  const int n4 = p.T * (d / 4);
  for (int i = tid; i < n4; i += kW4Threads) {
    const float4 v = __ldcg(reinterpret_cast<const float4 *>(p.y_acc) + i);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b2 = __floats2bfloat162_rn(v.z, v.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t *>(&a);
    o.y = *reinterpret_cast<uint32_t *>(&b2);
    reinterpret_cast<uint2 *>(p.y)[i] = o;
    reinterpret_cast<float4 *>(p.y_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  if (tid == 0) *p.done = 0u;
}

}  // namespace ftmoe
