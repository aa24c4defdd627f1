// Steps 5+6 for MXFP4 experts (e2m1 codes, one power-of-two scale byte per 32 elements of the contraction
// dimension; paper Sec. 5.1) at decode-sized token counts.  Same structure, work distribution and buffers as the int4 kernels of
// ffn_w4.cuh (every warp of the gate/up kernel streams its share of half-unit pieces; the down kernel walks chunks of 128
// neurons x 1024 columns; weights go from global memory straight into registers); what differs is the arithmetic:
//   * an e2m1 code is a 4-bit float, and placing its bits (s, e1 e0, m) at bits (7, 4 3, 2) of a byte gives the fp8
//     e4m3 number code * 2^-6 exactly, subnormals included.  ((w << 4) & 0x80808080) | ((w << 2) & 0x1C1C1C1C) does
//     that for the four even codes of a word, (w & 0x80808080) | ((w >> 2) & 0x1C1C1C1C) for the odd ones: seven
//     logic instructions per 8 weights, the two masks passed as data (see W4Params);
//   * the registers are A fragments of the fp8 tensor-core instruction mma.sync.m16n8k32 (e4m3 x e4m3 -> fp32), whose
//     K = 32 is exactly one scale block, so the block scale 2^(b-127) multiplies the fp32 result of every MMA, per row;
//   * the bf16 activations of a (token, group of 128) are scaled to |a| <= 256 and split into two e4m3 numbers,
//     a = hi + lo with lo the e4m3 rounding of a - hi (7-8 significant bits, like bf16, down to 2^-17 of the group's
//     largest magnitude); both MMAs accumulate into the same registers.
// NVFP4 experts (an unsigned e4m3 scale per 16 elements, a float32 scale per matrix) run through the same kernels
// (template flag NV): their records keep the codes of one 16-element block in the even nibbles of a word row and
// those of the next block in the odd nibbles, so that each block is one K = 16 fp8 MMA; the scale byte becomes a
// float by a shift, a mask and a multiplication by 2^120.
// The per-MMA scale multiplications and the seven-instruction unpack make these kernels bound by the logic pipe, not
// by HBM (about half the rate of the int4 kernels); the hardware's own route for this format is the block-scaled
// tcgen05 MMA, which reads packed fp4 and scale factors without any unpacking.
#pragma once
#include <cuda_fp8.h>

#include <type_traits>

#include "ffn_w4.cuh"

namespace ftmoe {

__device__ __forceinline__ void mma_e4m3(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_e4m3_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k32.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}

// K = 16 form (one 16-element scale block of an NVFP4 record): a0 = row g, a1 = row g+8, b0 = the token's 4 bytes.
__device__ __forceinline__ void mma_e4m3_k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(b0));
}
__device__ __forceinline__ void mma_e4m3_k16_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t b0) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.e4m3.e4m3.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%7,%7,%7,%7};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(b0), "f"(0.f));
}

constexpr float kMx4ActMax = 256.f;        // activations of a group are scaled so that the largest magnitude is this
constexpr float kMx4CodeScale = 64.f;      // the e4m3 placement of a code is code * 2^-6

// The even / odd codes of a word as e4m3 bytes.  k80 = 0x80808080, k1c = 0x1C1C1C1C (register constants).
__device__ __forceinline__ uint32_t mx4_even(uint32_t w, uint32_t k80, uint32_t k1c) {
  return ((w << 4) & k80) | ((w << 2) & k1c);
}
__device__ __forceinline__ uint32_t mx4_odd(uint32_t w, uint32_t k80, uint32_t k1c) {
  return (w & k80) | ((w >> 2) & k1c);
}
// 2^(b - 127) of byte j of a word of four scale bytes.
__device__ __forceinline__ float mx4_scale(uint32_t w, int j) {
  return __uint_as_float(j < 3 ? ((w << (23 - 8 * j)) & 0x7F800000u) : ((w >> 1) & 0x7F800000u));
}
// The unsigned e4m3 number of byte k of a word of four NVFP4 block scales: its bits moved to the float's exponent
// and mantissa top give the value * 2^-120 (an exact float, subnormal bytes included), the product restores it.
__device__ __forceinline__ float nv4_scale(uint32_t w, int k) {
  const uint32_t bits = (k < 3 ? (w << (20 - 8 * k)) : (w >> 4)) & 0x07F00000u;
  return __uint_as_float(bits) * 0x1p120f;
}
// e4m3 rounding of two floats (satfinite), low byte = a.
__device__ __forceinline__ uint32_t mx4_to_e4m3x2(float a, float b) {
  return (uint32_t)__nv_cvt_float2_to_fp8x2(make_float2(a, b), __NV_SATFINITE, __NV_E4M3);
}
__device__ __forceinline__ float2 mx4_from_e4m3x2(uint32_t v) {
  const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2((__nv_fp8x2_storage_t)v, __NV_E4M3);
  return __half22float2(*reinterpret_cast<const __half2 *>(&h));
}
// 8 scaled values -> (hi of elements 0,2,4,6 | hi of 1,3,5,7 | lo of 0,2,4,6 | lo of 1,3,5,7), value = hi + lo.
__device__ __forceinline__ uint4 mx4_split8(const float (&f)[8]) {
  uint32_t hi[4], lo[4];   // pair k = elements (2k, 2k+1)
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    hi[k] = mx4_to_e4m3x2(f[2 * k], f[2 * k + 1]);
    const float2 back = mx4_from_e4m3x2(hi[k]);
    lo[k] = mx4_to_e4m3x2(f[2 * k] - back.x, f[2 * k + 1] - back.y);
  }
  uint4 o;
  o.x = (hi[0] & 0xff) | ((hi[1] & 0xff) << 8) | ((hi[2] & 0xff) << 16) | ((hi[3] & 0xff) << 24);
  o.y = ((hi[0] >> 8) & 0xff) | (((hi[1] >> 8) & 0xff) << 8) | (((hi[2] >> 8) & 0xff) << 16) | (((hi[3] >> 8) & 0xff) << 24);
  o.z = (lo[0] & 0xff) | ((lo[1] & 0xff) << 8) | ((lo[2] & 0xff) << 16) | ((lo[3] & 0xff) << 24);
  o.w = ((lo[0] >> 8) & 0xff) | (((lo[1] >> 8) & 0xff) << 8) | (((lo[2] >> 8) & 0xff) << 16) | (((lo[3] >> 8) & 0xff) << 24);
  return o;
}
// 8 scaled values (consecutive elements) -> hi bytes of elements 0..3, of 4..7, lo bytes of 0..3, of 4..7.
__device__ __forceinline__ uint4 nv4_split8(const float (&f)[8]) {
  uint32_t hi[4], lo[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    hi[k] = mx4_to_e4m3x2(f[2 * k], f[2 * k + 1]);
    const float2 back = mx4_from_e4m3x2(hi[k]);
    lo[k] = mx4_to_e4m3x2(f[2 * k] - back.x, f[2 * k + 1] - back.y);
  }
  return make_uint4((hi[0] & 0xffff) | (hi[1] << 16), (hi[2] & 0xffff) | (hi[3] << 16),
                    (lo[0] & 0xffff) | (lo[1] << 16), (lo[2] & 0xffff) | (lo[3] << 16));
}
__device__ __forceinline__ void mx4_group_scale(float m, bool bad, float &scale, float &inv) {
  if (bad) { scale = __int_as_float(0x7fc00000); inv = 0.f; }
  else if (m < 1e-30f) { scale = 0.f; inv = 0.f; }
  else { scale = m * (1.f / kMx4ActMax); inv = kMx4ActMax / m; }
}

// Dynamic shared memory of the gate/up kernel: x [8][2d + 64] bytes (the split activations) | scale [8][G] f32 |
// items | pref.
inline size_t mx4_gateup_smem_bytes(int max_items, int d) {
  return (size_t)8 * (2 * d + 64) + (size_t)8 * (d / kGroup) * 4 + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}
// ... of the down kernel: per warp 2 slots of (h operands 2048 | 256 bytes of weight scales | 64 bytes of per-token
// scales) | items | pref.
constexpr uint32_t kMx4DownSlot = 2048 + 256 + 64;
constexpr uint32_t kNv4DownSlot = 2048 + 512 + 64;   // NVFP4: 512 bytes of weight scales (one per 16 neurons)
inline size_t mx4_down_smem_bytes(int max_items, bool nv) {
  return (size_t)kW4Warps * 2 * (nv ? kNv4DownSlot : kMx4DownSlot) + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}

// NV: NVFP4 records (an e4m3 scale per 16 elements, a float32 scale per matrix; the even codes of a word row are
// one scale block, the odd codes the next, see include/ftmoe.h) instead of MXFP4 ones.
template <int G, bool NV>   // groups of 128 of the hidden dimension: d = 128 G
__global__ void __launch_bounds__(kW4Threads, 1) mx4_gateup_kernel(W4Params p) {
  constexpr int d = kGroup * G;
  constexpr uint32_t kST = NV ? 128u : 64u;         // scale bytes of a tile
  constexpr uint32_t kUA = (2048u + 2u * kST) * G;  // bytes of a unit: gate tiles, up tiles, gate scales, up scales
  constexpr uint32_t kXStride = 2u * d + 64u;
  constexpr int kBS = kW4BlockSteps;
  constexpr int kBlocks = G / kBS;
  constexpr int kKS = kW4KSplit, kBlocksP = kBlocks / kKS;   // blocks of a piece
  static_assert(G % kBS == 0 && kBlocks % kKS == 0, "whole blocks, whole pieces");
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_x = smem;
  float *s_sx = reinterpret_cast<float *>(s_x + 8 * kXStride);             // [8][G] m / 256
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_sx + 8 * G);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
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

  auto stage_x = [&](auto tok_of_column) {
    for (int i = tid; i < 8 * (d / 8); i += kW4Threads) {
      const int j = i / (d / 8), c8 = i - j * (d / 8);
      const int tok = tok_of_column(j);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok >= 0) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 8 * c8);
      float f[8] = {bf16lo(v.x), bf16hi(v.x), bf16lo(v.y), bf16hi(v.y), bf16lo(v.z), bf16hi(v.z), bf16lo(v.w), bf16hi(v.w)};
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
      mx4_group_scale(m, bad, scale, inv);
#pragma unroll
      for (int e = 0; e < 8; ++e) f[e] *= inv;
      if constexpr (NV) {
        // elements 8 c8 .. 8 c8 + 7 are in half hf of their block of 32; lane q of the MMA reads, for word j4, the 16
        // bytes (hi of half 0 | hi of half 1 | lo of half 0 | lo of half 1) of elements 4q .. 4q+3 of each half
        const uint4 sp = nv4_split8(f);
        const int blk32 = c8 >> 2, hf = (c8 >> 1) & 1, q0 = 2 * (c8 & 1);
        uint32_t *row = reinterpret_cast<uint32_t *>(s_x + j * kXStride + 64 * blk32);
        row[4 * q0 + hf] = sp.x;
        row[4 * (q0 + 1) + hf] = sp.y;
        row[4 * q0 + 2 + hf] = sp.z;
        row[4 * (q0 + 1) + 2 + hf] = sp.w;
      } else {
        *reinterpret_cast<uint4 *>(s_x + j * kXStride + 16 * c8) = mx4_split8(f);
      }
      if ((lane & 15) == 0) s_sx[j * G + c8 / 16] = scale;
    }
  };

  const uint32_t my_x = smem_u32(s_x) + g * kXStride + 16u * q;
  const float *my_s0 = s_sx + (2 * q) * G, *my_s1 = s_sx + (2 * q + 1) * G;
  const uint32_t k1c = p.mask, k80 = p.flip;

  // The warp that completes a group of 128 neurons of a pass splits its h for the down kernel:
  // lane = (token, quarter): the quarter's two units of 16 neurons = one scale block of the down weights.
  const size_t tail = (size_t)(p.inter / 16) * kUA + (size_t)p.inter * d / 2 + (size_t)p.inter * d / 16;   // NV only
  auto convert_group = [&](uint32_t grp, const uint8_t *rec) {
    const int tok = lane >> 2, qt = lane & 3;
    float cs_g = kMx4CodeScale, cs_u = kMx4CodeScale;
    if constexpr (NV) {
      const float2 ms = __ldg(reinterpret_cast<const float2 *>(rec + tail));   // matrix scales of gate and up
      cs_g *= ms.x;
      cs_u *= ms.y;
    }
    float *src = p.hraw + ((size_t)grp * 8 + 2 * qt) * 256 + tok * 16;   // per unit: gate sums [8][16], up sums [8][16]
    float v[2][16];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        float4 *pg = reinterpret_cast<float4 *>(src + u * 256) + k4, *pu_ = reinterpret_cast<float4 *>(src + u * 256 + 128) + k4;
        float4 a = __ldcg(pg), b = __ldcg(pu_);
        __stcg(pg, make_float4(0.f, 0.f, 0.f, 0.f));   // the sums start from zero in the next call
        __stcg(pu_, make_float4(0.f, 0.f, 0.f, 0.f));
        a.x *= cs_g; a.y *= cs_g; a.z *= cs_g; a.w *= cs_g;
        b.x *= cs_u; b.y *= cs_u; b.z *= cs_u; b.w *= cs_u;
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
    mx4_group_scale(m, bad, scale, inv);
    uint8_t *dst = p.hq + (size_t)grp * 2048 + qt * 512 + tok * 64;
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {   // neurons 4qq..4qq+3 of both units: (hi u0, hi u1, lo u0, lo u1)
      uint32_t o[4];
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const float a0 = v[u][4 * qq] * inv, a1 = v[u][4 * qq + 1] * inv, a2 = v[u][4 * qq + 2] * inv, a3 = v[u][4 * qq + 3] * inv;
        const uint32_t h01 = mx4_to_e4m3x2(a0, a1), h23 = mx4_to_e4m3x2(a2, a3);
        const float2 b01 = mx4_from_e4m3x2(h01), b23 = mx4_from_e4m3x2(h23);
        const uint32_t l01 = mx4_to_e4m3x2(a0 - b01.x, a1 - b01.y), l23 = mx4_to_e4m3x2(a2 - b23.x, a3 - b23.y);
        o[u] = (h01 & 0xffff) | (h23 << 16);
        o[2 + u] = (l01 & 0xffff) | (l23 << 16);
      }
      *reinterpret_cast<uint4 *>(dst + qq * 16) = make_uint4(o[0], o[1], o[2], o[3]);
    }
    if (qt == 0) p.hs[(size_t)grp * 8 + tok] = make_float2(scale, 0.f);
  };

  auto run = [&](const uint8_t *rec, const uint8_t *base, int ks0, int n_pieces, uint32_t hrow0) {
    uint4 buf[4 * kBS];     // per step: gate rows g, g+8; up rows g, g+8
    // per step: the block scales of rows g and g+8, gate then up (MXFP4: four each in .x and .y; NVFP4: eight each
    // in .x .y and .z .w)
    using ScaleT = typename std::conditional<NV, uint4, uint2>::type;
    ScaleT sc[2 * kBS];
    const uint8_t *nptr = base + ks0 * (G / kKS) * 1024 + g * 64 + q * 16;
    const uint8_t *nsc = base + 2048u * G + ks0 * (G / kKS) * kST + g * (kST / 8);
    int nblk = ks0 * kBlocksP, blocks_left = n_pieces * kBlocksP;
    auto advance = [&]() {
      nptr += kBS * 1024;
      nsc += kBS * kST;
      --blocks_left;
      if (++nblk == kBlocks) {   // on to the next unit
        nblk = 0;
        nptr += kUA - 1024u * G;
        nsc += kUA - kST * G;
      }
    };
    auto request = [&](int si, const uint8_t *tp, const uint8_t *sp) {
      buf[4 * si] = ld_stream_16(tp + si * 1024);
      buf[4 * si + 1] = ld_stream_16(tp + si * 1024 + 512);
      buf[4 * si + 2] = ld_stream_16(tp + si * 1024 + 1024 * G);
      buf[4 * si + 3] = ld_stream_16(tp + si * 1024 + 1024 * G + 512);
      if constexpr (NV) {
        sc[2 * si] = ld_stream_16(sp + si * kST);
        sc[2 * si + 1] = ld_stream_16(sp + si * kST + kST * G);
      } else {
        sc[2 * si] = ld_stream_8(sp + si * kST);
        sc[2 * si + 1] = ld_stream_8(sp + si * kST + kST * G);
      }
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
        const uint8_t *rp = nptr, *rs = nsc;
        if (more) advance();
        const int xg = ks * (G / kKS) + blk * kBS;
        const uint32_t xa = my_x + xg * 256u;
#pragma unroll
        for (int si = 0; si < kBS; ++si) {
          const uint32_t glo[4] = {buf[4 * si].x, buf[4 * si].y, buf[4 * si].z, buf[4 * si].w};
          const uint32_t ghi[4] = {buf[4 * si + 1].x, buf[4 * si + 1].y, buf[4 * si + 1].z, buf[4 * si + 1].w};
          const uint32_t ulo[4] = {buf[4 * si + 2].x, buf[4 * si + 2].y, buf[4 * si + 2].z, buf[4 * si + 2].w};
          const uint32_t uhi[4] = {buf[4 * si + 3].x, buf[4 * si + 3].y, buf[4 * si + 3].z, buf[4 * si + 3].w};
          const ScaleT gs = sc[2 * si], us = sc[2 * si + 1];
          float sg[4] = {0.f, 0.f, 0.f, 0.f}, su[4] = {0.f, 0.f, 0.f, 0.f};   // the step's sums, before the activation scale
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // word j = scale block j of the group: hidden indices 32j + 8q + 0..7
            const uint4 xv = lds_v4(xa + si * 256u + j * 64u);
            if constexpr (NV) {
              // even codes = block 2j, odd codes = block 2j+1 of the group, each with its own scale per row
              float e0[4], e1[4];
              {
                const uint32_t a0 = mx4_even(glo[j], k80, k1c), a1 = mx4_even(ghi[j], k80, k1c);
                const uint32_t a2 = mx4_odd(glo[j], k80, k1c), a3 = mx4_odd(ghi[j], k80, k1c);
                mma_e4m3_k16_first(e0, a0, a1, xv.x);
                mma_e4m3_k16(e0, a0, a1, xv.z);
                mma_e4m3_k16_first(e1, a2, a3, xv.y);
                mma_e4m3_k16(e1, a2, a3, xv.w);
              }
              const uint32_t wlo = j < 2 ? gs.x : gs.y, whi = j < 2 ? gs.z : gs.w;
              const float l0 = nv4_scale(wlo, 2 * (j & 1)), l1 = nv4_scale(wlo, 2 * (j & 1) + 1);
              const float h0 = nv4_scale(whi, 2 * (j & 1)), h1 = nv4_scale(whi, 2 * (j & 1) + 1);
              sg[0] += l0 * e0[0] + l1 * e1[0]; sg[1] += l0 * e0[1] + l1 * e1[1];
              sg[2] += h0 * e0[2] + h1 * e1[2]; sg[3] += h0 * e0[3] + h1 * e1[3];
              {
                const uint32_t a0 = mx4_even(ulo[j], k80, k1c), a1 = mx4_even(uhi[j], k80, k1c);
                const uint32_t a2 = mx4_odd(ulo[j], k80, k1c), a3 = mx4_odd(uhi[j], k80, k1c);
                mma_e4m3_k16_first(e0, a0, a1, xv.x);
                mma_e4m3_k16(e0, a0, a1, xv.z);
                mma_e4m3_k16_first(e1, a2, a3, xv.y);
                mma_e4m3_k16(e1, a2, a3, xv.w);
              }
              const uint32_t vlo = j < 2 ? us.x : us.y, vhi = j < 2 ? us.z : us.w;
              const float m0 = nv4_scale(vlo, 2 * (j & 1)), m1 = nv4_scale(vlo, 2 * (j & 1) + 1);
              const float n0 = nv4_scale(vhi, 2 * (j & 1)), n1 = nv4_scale(vhi, 2 * (j & 1) + 1);
              su[0] += m0 * e0[0] + m1 * e1[0]; su[1] += m0 * e0[1] + m1 * e1[1];
              su[2] += n0 * e0[2] + n1 * e1[2]; su[3] += n0 * e0[3] + n1 * e1[3];
            } else {
            float ga[4], ua[4];
            {
              const uint32_t a0 = mx4_even(glo[j], k80, k1c), a1 = mx4_even(ghi[j], k80, k1c);
              const uint32_t a2 = mx4_odd(glo[j], k80, k1c), a3 = mx4_odd(ghi[j], k80, k1c);
              mma_e4m3_first(ga, a0, a1, a2, a3, xv.x, xv.y);
              mma_e4m3(ga, a0, a1, a2, a3, xv.z, xv.w);
            }
            {
              const uint32_t a0 = mx4_even(ulo[j], k80, k1c), a1 = mx4_even(uhi[j], k80, k1c);
              const uint32_t a2 = mx4_odd(ulo[j], k80, k1c), a3 = mx4_odd(uhi[j], k80, k1c);
              mma_e4m3_first(ua, a0, a1, a2, a3, xv.x, xv.y);
              mma_e4m3(ua, a0, a1, a2, a3, xv.z, xv.w);
            }
            const float g_lo = mx4_scale(gs.x, j), g_hi = mx4_scale(gs.y, j);
            const float u_lo = mx4_scale(us.x, j), u_hi = mx4_scale(us.y, j);
            sg[0] += g_lo * ga[0]; sg[1] += g_lo * ga[1]; sg[2] += g_hi * ga[2]; sg[3] += g_hi * ga[3];
            su[0] += u_lo * ua[0]; su[1] += u_lo * ua[1]; su[2] += u_hi * ua[2]; su[3] += u_hi * ua[3];
            }
          }
          if (more) request(si, rp, rs);   // refill the step just consumed
          const float sx0 = my_s0[xg + si], sx1 = my_s1[xg + si];
          tg[0] += sg[0] * sx0; tg[1] += sg[1] * sx1; tg[2] += sg[2] * sx0; tg[3] += sg[3] * sx1;
          tot[0] += su[0] * sx0; tot[1] += su[1] * sx1; tot[2] += su[2] * sx0; tot[3] += su[3] * sx1;
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
        convert_group(hrow_i >> 3, rec);
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
    for (uint32_t pu = cf / PP; pu * PP < ce; ++pu) {
      const int item = w4_find_item(s_pref, n_items + n_zc, pu);
      const WorkItem &it = s_items[item];
      if (!dense) {
        const int tok0 = (int)(pu - (uint32_t)s_pref[item]) * kQ4Tokens, nt = min(kQ4Tokens, it.n_tok - tok0);
        const int off_ = it.off + tok0, expert_ = it.expert;
        __syncthreads();
        stage_x([&](int j) {
          if (j >= nt) return -1;
          return expert_ >= 0 ? p.perm[off_ + j] / p.top_k : tok0 + j;
        });
        __syncthreads();
      }
      const uint32_t lo = max(wf, pu * PP), hi = min(we, (pu + 1) * PP);
      if (lo < hi) {
        const uint32_t rel = lo - pu * PP;
        run(it.w, it.w + (size_t)(rel / kKS) * kUA, (int)(rel % kKS), (int)(hi - lo), pu * NBLK + rel / kKS);
      }
    }
  }
}

template <int NWD, bool NV>   // warps that own output columns: a column block is 64 * NWD columns
__global__ void __launch_bounds__(kW4Threads, 1) mx4_down_kernel(W4Params p, int d) {
  constexpr uint32_t kSlot = NV ? kNv4DownSlot : kMx4DownSlot;
  constexpr uint32_t kSW = NV ? 512u : 256u;   // weight scale bytes of a chunk and warp
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_h = smem;                                                // [16 warps][2 slots]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(smem + kW4Warps * 2 * kSlot);
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
  const size_t sec_b = (size_t)NBLK * (NV ? 2304u : 2176u) * G, sec_c = sec_b + (size_t)p.inter * d / 2;
  const size_t tail = sec_c + (size_t)p.inter * d / 16;   // NV only: the matrix scales
  const uint32_t per_pass = CB * NG;
  const bool dense = p.T <= kQ4Tokens;
  asm volatile("griddepcontrol.wait;" ::: "memory");   // from here on the gate/up kernel's h is needed

  if (warp < NWD) {
    const uint32_t t0 = (uint32_t)s_pref[n_items] * per_pass;
    const uint32_t t1 = (uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * per_pass;
    const uint32_t rfirst0 = w4_first(t0, gridDim.x, blockIdx.x), rcount0 = w4_first(t0, gridDim.x, blockIdx.x + 1) - rfirst0;
    const uint32_t rfirst1 = t0 + w4_first(t1, gridDim.x, blockIdx.x);
    const uint32_t rcount1 = t0 + w4_first(t1, gridDim.x, blockIdx.x + 1) - rfirst1;
    const uint32_t my_h = smem_u32(s_h) + (uint32_t)warp * 2u * kSlot;
    const uint32_t k1c = p.mask, k80 = p.flip;

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
    auto stage = [&](const Ck &c, uint32_t slot) {
      const size_t grp = (size_t)c.pu * NG + c.ng;
      const uint8_t *hsrc = p.hq + grp * 2048;
      const uint32_t dst = my_h + slot * kSlot;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (i * 32 + lane) * 16u), "l"(hsrc + (i * 32 + lane) * 16)
                     : "memory");
      if (NV || lane < 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2048u + lane * 16u),
                     "l"(c.rec + sec_c + ((size_t)(c.ng * CB + c.cb) * NWD + warp) * kSW + lane * 16u)
                     : "memory");
      if (lane >= 16 && lane < 20)   // (scale, unused) of the 8 tokens: 64 bytes, of which the scales are used
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2048u + kSW + (lane - 16) * 16u),
                     "l"(reinterpret_cast<const uint8_t *>(p.hs + grp * 8) + (lane - 16) * 16)
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
    auto begin_pass = [&](const Ck &c) {
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
    auto flush = [&](uint32_t cb, const uint8_t *rec) {
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
      float cs = kMx4CodeScale;
      if constexpr (NV) cs *= __ldg(reinterpret_cast<const float *>(rec + tail) + 2);   // matrix scale of down
      gw_a *= cs;
      gw_b *= cs;
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

    uint4 buf[8];
    Ck c0, c1;
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
      asm volatile("cp.async.wait_group 1;" ::: "memory");
      __syncwarp();
      const uint32_t hs_base = my_h + slot * kSlot;
      // weight scales of the chunk.  MXFP4: word 2j + half = the four 32-neuron blocks of (tile j, column g + 8 half);
      // NVFP4: words 4j + 2 half, + 1 = the eight 16-neuron blocks
      uint32_t sw[NV ? 16 : 8];
#pragma unroll
      for (int i = 0; i < (NV ? 4 : 2); ++i) {
        const uint4 sv = lds_v4(hs_base + 2048u + g * (kSW / 8u) + 16u * i);
        sw[4 * i] = sv.x; sw[4 * i + 1] = sv.y; sw[4 * i + 2] = sv.z; sw[4 * i + 3] = sv.w;
      }
      float ct[4][4];   // the chunk's sums, before the activation scale
#pragma unroll
      for (int j = 0; j < 4; ++j) { ct[j][0] = ct[j][1] = ct[j][2] = ct[j][3] = 0.f; }
#pragma unroll
      for (int m = 0; m < 4; ++m) {   // unit pair m = scale block m: neurons 32m .. 32m+31 of the group
        const uint4 hv = lds_v4(hs_base + m * 512u + g * 64u + q * 16u);   // token g: (hi u0, hi u1, lo u0, lo u1)
        const uint32_t w0[4] = {buf[2 * m].x, buf[2 * m].y, buf[2 * m].z, buf[2 * m].w};
        const uint32_t w1[4] = {buf[2 * m + 1].x, buf[2 * m + 1].y, buf[2 * m + 1].z, buf[2 * m + 1].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {   // tile j: columns g (even codes) and g+8 (odd codes)
          const uint32_t a0 = mx4_even(w0[j], k80, k1c), a1 = mx4_odd(w0[j], k80, k1c);
          const uint32_t a2 = mx4_even(w1[j], k80, k1c), a3 = mx4_odd(w1[j], k80, k1c);
          if constexpr (NV) {
            float e0[4], e1[4];   // unit 2m and unit 2m+1: one scale block each
            mma_e4m3_k16_first(e0, a0, a1, hv.x);
            mma_e4m3_k16(e0, a0, a1, hv.z);
            mma_e4m3_k16_first(e1, a2, a3, hv.y);
            mma_e4m3_k16(e1, a2, a3, hv.w);
            const uint32_t wlo = sw[4 * j + (m >> 1)], whi = sw[4 * j + 2 + (m >> 1)];
            const float l0 = nv4_scale(wlo, 2 * (m & 1)), l1 = nv4_scale(wlo, 2 * (m & 1) + 1);
            const float h0 = nv4_scale(whi, 2 * (m & 1)), h1 = nv4_scale(whi, 2 * (m & 1) + 1);
            ct[j][0] += l0 * e0[0] + l1 * e1[0]; ct[j][1] += l0 * e0[1] + l1 * e1[1];
            ct[j][2] += h0 * e0[2] + h1 * e1[2]; ct[j][3] += h0 * e0[3] + h1 * e1[3];
          } else {
          float acc[4];
          mma_e4m3_first(acc, a0, a1, a2, a3, hv.x, hv.y);
          mma_e4m3(acc, a0, a1, a2, a3, hv.z, hv.w);
          const float s_lo = mx4_scale(sw[2 * j], m), s_hi = mx4_scale(sw[2 * j + 1], m);
          ct[j][0] += s_lo * acc[0]; ct[j][1] += s_lo * acc[1]; ct[j][2] += s_hi * acc[2]; ct[j][3] += s_hi * acc[3];
          }
        }
        if (refill) {
          buf[2 * m] = ld_stream_16(refill + (size_t)(2 * m) * NWD * 512u);
          buf[2 * m + 1] = ld_stream_16(refill + (size_t)(2 * m + 1) * NWD * 512u);
        }
      }
      const uint4 tb = lds_v4(hs_base + 2048u + kSW + q * 16u);   // tokens 2q, 2q+1: (scale, unused) each
      __syncwarp();   // every lane has read the slot: it may be overwritten
      const float sh0 = __uint_as_float(tb.x), sh1 = __uint_as_float(tb.z);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        dtot[j][0] += ct[j][0] * sh0; dtot[j][1] += ct[j][1] * sh1; dtot[j][2] += ct[j][2] * sh0; dtot[j][3] += ct[j][3] * sh1;
      }
      if (!h1 || c1.pu != c0.pu || c1.cb != c0.cb) {
        flush(c0.cb, c0.rec);
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
