// Many-token calls on 4-bit experts: the experts that go through the tensor-core GEMMs are first expanded, once per
// call, from their slot into a bf16 record in tile order (the layout the GEMMs' tensor maps read, see
// include/ftmoe.h) in a per-layer scratch pool.  With hundreds of tokens per expert the expansion (one pass over
// the record) is small beside the GEMMs, and the GEMMs then run on exact bf16 activations: int4 weights are rounded
// to bf16 after the multiplication by their scale (11-12 significant bits -> 8), MXFP4 weights (in either record
// order) are exact in bf16,
// NVFP4 weights are rounded after the multiplication by the block scale and the matrix scale.
// One thread produces one 16-byte chunk of the destination (8 weights), in destination order, so that the writes
// are coalesced; the 4-byte source words come from L2.
#pragma once
#include "common.cuh"
#include "ffn_w4.cuh"
#include "gemm_tc.cuh"   // pack_bf16

namespace ftmoe {

struct DequantParams {
  const WorkItem *items;    // the GEMM work list: record pointer (slot) and slot index per expert
  const int32_t *n_items;
  uint8_t *scratch;         // [slots_per_layer][3 * inter * d * 2] bf16 records in tile order
  int d, inter;
};

__device__ __forceinline__ float w4_code_value(uint32_t nib, bool mx) {
  if (!mx) return (float)((int)(nib ^ 8u) - 8);                 // two's-complement nibble
  const uint32_t e = (nib >> 1) & 3u, m = nib & 1u;             // e2m1: 0, 0.5 | (1 + m/2) * 2^(e-1)
  const float mag = e == 0 ? 0.5f * (float)m : __uint_as_float(((e + 126u) << 23) | (m << 22));
  return (nib & 8u) ? -mag : mag;
}

// value of an unsigned e4m3 byte (see nv4_scale in ffn_mx4.cuh)
__device__ __forceinline__ float w4_ue4m3(uint32_t b) { return __uint_as_float((b & 0x7Fu) << 20) * 0x1p120f; }

template <int FMT>   // 0: int4-g128, 1: MXFP4, 2: NVFP4, 3: MXFP4 stored as tensor-core operand images
__global__ void __launch_bounds__(256) dequant_w4_kernel(DequantParams p) {
  constexpr bool MX = FMT != 0, NV = FMT == 2, TC = FMT == 3;
  const int d = p.d, I = p.inter;
  const uint32_t G = (uint32_t)d / 128u, NG = (uint32_t)I / 128u, NBLK = (uint32_t)I / 16u;
  const uint32_t NWD = min(16u, (uint32_t)d / 64u), CBW = 64u * NWD, CB = (uint32_t)d / CBW;
  const size_t UA = (size_t)(NV ? 2304u : MX ? 2176u : 2112u) * G;
  const size_t sec_b = (size_t)NBLK * UA, sec_c = sec_b + (size_t)I * d / 2;
  const size_t S16 = (size_t)3 * I * d * 2;
  const uint32_t chunks_unit = 6u * (uint32_t)d;                // 16-byte chunks of a 96*d-byte destination unit
  const uint32_t cbw_shift = 31u - (uint32_t)__clz((int)CBW);   // CBW is 512 or 1024
  // one block per (16-neuron unit, expert of the GEMM list); the list's length is known on the device only
  const int item = blockIdx.y;
  if (item >= *p.n_items) return;
  const uint32_t u = blockIdx.x;
  const uint8_t *rec = p.items[item].w;
  float ms[3] = {1.f, 1.f, 1.f};   // NVFP4: the matrix scales
  if (NV) {
    const float *tail = reinterpret_cast<const float *>(rec + sec_c + (size_t)I * d / 16);
    ms[0] = tail[0]; ms[1] = tail[1]; ms[2] = tail[2];
  }
  uint8_t *dst_unit = p.scratch + (size_t)p.items[item].slot * S16 + (size_t)u * 96u * d;
  for (uint32_t k = threadIdx.x; k < chunks_unit; k += blockDim.x) {
    uint8_t *dst = dst_unit + (size_t)k * 16u;
    float v[8];
    if (k < 4u * (uint32_t)d) {
      // ---- gate (k < 2d) or up part: tile t of 16 neurons x 32 hidden indices, rows of 64 bytes, swizzled ----
      const uint32_t mm = k >= 2u * (uint32_t)d ? 1u : 0u, kk = k - mm * 2u * d;
      const uint32_t t = kk >> 6, r = (kk >> 2) & 15u, pos = kk & 3u;
      const uint32_t q = pos ^ ((r & 7u) >> 1);                 // chunk q of the row is stored at position pos
      const uint32_t grp = t >> 2, j = t & 3u;                  // hidden indices 128 grp + 32 j + 8 q + 0..7
      const uint8_t *unit = rec + (size_t)u * UA;
      if (TC) {
        // operand images: block of (128 neurons ng, 128 hidden indices st) = gate image, up image, gate scales, up
        // scales; the 8 codes of hidden indices 8q .. 8q+7 of block j are one word of the row
        const uint32_t row = 16u * (u & 7u) + r, kb = 32u * j + 8u * q;       // row of the 128, index in the 128
        const uint8_t *blk = rec + ((size_t)(u >> 3) * G + grp) * 17408u;
        const uint32_t w = *reinterpret_cast<const uint32_t *>(blk + mm * 8192u + 4096u * (kb >> 6) + 2048u * ((kb & 63u) >> 5) +
                                                               128u * (row >> 3) + 16u * (row & 7u) + ((kb & 31u) >> 1));
        const float scale = __uint_as_float((uint32_t)blk[16384u + mm * 512u + 16u * (row & 31u) + 4u * (row >> 5) + j] << 23);
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = scale * w4_code_value((w >> (4 * e)) & 15u, true);
      } else if (NV) {
        // hidden indices 8q .. 8q+7 of block j: half q>>1 of the block (= the nibble parity), bytes 0..3 of word j of
        // the source chunks 2(q&1) and 2(q&1)+1
        const uint8_t *row = unit + (size_t)mm * 1024u * G + grp * 1024u + r * 64u + j * 4u;
        const uint32_t wa = *reinterpret_cast<const uint32_t *>(row + (2u * (q & 1u)) * 16u);
        const uint32_t wb = *reinterpret_cast<const uint32_t *>(row + (2u * (q & 1u) + 1u) * 16u);
        const uint32_t hf = q >> 1;
        const uint32_t b = unit[2048u * G + mm * 128u * G + grp * 128u + (r & 7u) * 16u + (r >> 3) * 8u + 2u * j + hf];
        const float scale = w4_ue4m3(b) * ms[mm];
#pragma unroll
        for (int e = 0; e < 8; ++e) v[e] = scale * w4_code_value(((e < 4 ? wa : wb) >> (8 * (e & 3) + 4 * (int)hf)) & 15u, true);
      } else {
      const uint32_t w = *reinterpret_cast<const uint32_t *>(unit + (size_t)mm * 1024u * G + grp * 1024u + r * 64u + q * 16u + j * 4u);
      float scale;
      if (MX) {
        const uint32_t b = unit[2048u * G + mm * 64u * G + grp * 64u + (r & 7u) * 8u + (r >> 3) * 4u + j];
        scale = __uint_as_float(b << 23);
      } else {
        const uint16_t s = *reinterpret_cast<const uint16_t *>(unit + 2048u * G + mm * 32u * G + grp * 32u + (r & 7u) * 4u + (r >> 3) * 2u);
        scale = __uint_as_float((uint32_t)s << 16);
      }
#pragma unroll
      for (int e = 0; e < 8; ++e) v[e] = scale * w4_code_value((w >> (4 * e)) & 15u, MX);
      }
    } else {
      // ---- down part: tile ct of 16 columns x the unit's 16 neurons, rows of 32 bytes, swizzled ----
      const uint32_t kk = k - 4u * d;
      const uint32_t ct = kk >> 5, cg = (kk >> 4) & 1u, rr = (kk >> 1) & 7u, pos = kk & 1u;
      const uint32_t nhalf = pos ^ (rr >> 2);                   // neurons 8 nhalf .. 8 nhalf + 7 of the unit
      const uint32_t c = 16u * ct + 8u * cg + rr;               // output column
      const uint32_t ng = u >> 3, uu = u & 7u;
      const uint32_t cb = c >> cbw_shift, tt = (c - (cb << cbw_shift)) >> 4, wq = tt >> 2, j = tt & 3u;
      const uint8_t *src = rec + sec_b + ((((size_t)(cb * NG + ng) * 8u + uu) * NWD + wq) * 32u + 4u * rr + 2u * nhalf) * 16u + 4u * j;
      uint32_t w0 = 0u, w1 = 0u;
      if (!TC) { w0 = *reinterpret_cast<const uint32_t *>(src); w1 = *reinterpret_cast<const uint32_t *>(src + 16); }
      float scale;
      if (TC) {
        // section B: block of (128 columns cgp, 128 neurons ng); the unit's 16 neurons are 8 bytes of the column's row
        const uint32_t rowc = c & 127u, kb = 16u * uu + 8u * nhalf;            // column of the 128, first neuron in the 128
        const uint8_t *blk = rec + (size_t)(I / 128u) * G * 17408u + ((size_t)(c >> 7) * NG + ng) * 8704u;
        const uint32_t wv = *reinterpret_cast<const uint32_t *>(blk + 4096u * (kb >> 6) + 2048u * ((kb & 63u) >> 5) + 128u * (rowc >> 3) +
                                                                16u * (rowc & 7u) + ((kb & 31u) >> 1));
        scale = __uint_as_float((uint32_t)blk[8192u + 16u * (rowc & 31u) + 4u * (rowc >> 5) + (kb >> 5)] << 23);
#pragma unroll
        for (int i = 0; i < 8; ++i) v[i] = scale * w4_code_value((wv >> (4 * i)) & 15u, true);
        uint4 o;
        o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]); o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
        *reinterpret_cast<uint4 *>(dst) = o;
        continue;
      } else if (NV) {
        scale = w4_ue4m3(rec[sec_c + ((size_t)(ng * CB + cb) * NWD + wq) * 512u + 64u * rr + 16u * j + 8u * cg + uu]) * ms[2];
      } else if (MX) {
        const uint32_t b = rec[sec_c + ((size_t)(ng * CB + cb) * NWD + wq) * 256u + 32u * rr + 8u * j + 4u * cg + (uu >> 1)];
        scale = __uint_as_float(b << 23);
      } else {
        const uint16_t s = *reinterpret_cast<const uint16_t *>(rec + sec_c + ((size_t)(ng * CB + cb) * NWD + wq) * 128u + 16u * rr + 4u * j + 2u * cg);
        scale = __uint_as_float((uint32_t)s << 16);
      }
#pragma unroll
      for (int i = 0; i < 8; ++i) {   // neuron 8 nhalf + i: word i / 4, nibble 2 (i % 4) + column half
        const uint32_t w = i < 4 ? w0 : w1;
        v[i] = scale * w4_code_value((w >> (4 * (2 * (i & 3) + (int)cg))) & 15u, MX);
      }
    }
    uint4 o;
    o.x = pack_bf16(v[0], v[1]); o.y = pack_bf16(v[2], v[3]); o.z = pack_bf16(v[4], v[5]); o.w = pack_bf16(v[6], v[7]);
    *reinterpret_cast<uint4 *>(dst) = o;
  }
}

}  // namespace ftmoe
