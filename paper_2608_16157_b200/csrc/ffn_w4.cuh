// Steps 5+6 for int4 (group 128, bf16 scales) experts at decode-sized token counts: two HBM-streaming kernels whose
// weight loads go straight from global memory into registers, with the group dequantisation done there, so the
// path stays bound by the bytes it streams.
//
// The record is stored in tile order (include/ftmoe.h).  A 32-bit word holds 8 codes; (w >> 4k) & 0x000F000F puts
// codes k and k+4 into the two halves of a register and XOR 0x43084308 turns them into the bf16 numbers 136 + code
// (exact: 128..143 have one-unit spacing in bf16), i.e. one A-fragment register of mma.sync.m16n8k16 per two
// instructions.  The constant is removed in fp32: sum (136 + c) a = 136 sum a + sum c a, with the sums of the
// activations over a group computed once; the group scale multiplies the fp32 partial sum once per group.  Weights
// and activations are bf16 operands, so the activation range is that of bf16.
//   w4_gateup_kernel : one persistent CTA of 16 warps per SM walks 16-neuron units (gate tiles, up tiles and their
//                      scales, contiguous).  Warp w owns GW quantisation groups of the hidden dimension; a lane's two
//                      16-byte loads per group are rows g and g+8 of the group's tile.  Partial [16 x 8] sums are
//                      reduced across warps through (double-buffered) shared memory: one barrier per unit.
//                      h = SiLU(g) * u goes to a small global buffer, bf16 [pass][unit][token][neuron].
//   w4_down_kernel   : walks chunks (expert pass, block of 64*NWD output columns, group of 128 neurons) = 8 steps
//                      of 16 neurons x 512 bytes per warp.  Every warp owns four 16-column tiles: its 16-byte load
//                      per step is their four A fragments.  No block-level synchronisation at all: a warp stages
//                      the chunk's h fragments for itself with cp.async.  Scale and bias are folded when the
//                      chunk (= one neuron group) ends; the scaled totals persist while consecutive chunks belong
//                      to the same pass and column block.  The gate-weighted combine is a red.global.add into the
//                      fp32 accumulator; the last CTA rounds it once to bf16.
// Zero-copy experts (records in the mapped host pool) go through the same kernels.
#pragma once
#include "async.cuh"
#include "common.cuh"
#include "ffn_stream.cuh"   // red_add_f32

namespace ftmoe {

constexpr int kQ4Tokens = 8;         // tokens per weight pass
constexpr int kW4Threads = 512;
constexpr float kW4Bias = 136.f;     // the dequantised operand is 136 + code

struct W4Params {
  const WorkItem *items;
  const int32_t *n_items;   // resident items
  const int32_t *n_zc;      // zero-copy items appended after them
  const int32_t *pref;      // exclusive prefix of the weight passes (8 tokens each) per item
  int max_items;
  const __nv_bfloat16 *x;   // [T][d]
  const int32_t *perm;
  const float *topk_w;
  __nv_bfloat16 *hbuf;      // [pass][16-neuron unit][token 8][neuron 16]
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;
  uint32_t *done;
  uint32_t *status;
  int inter, top_k, T, finalize;
};

// 8 codes of one word -> four bf16x2 registers holding 136 + code: pairs (0,4) (1,5) (2,6) (3,7).
struct W4Frag { uint32_t p04, p15, p26, p37; };
__device__ __forceinline__ W4Frag w4_unpack(uint32_t w) {
  W4Frag f;
  f.p04 = (w & 0x000F000Fu) ^ 0x43084308u;
  f.p15 = ((w >> 4) & 0x000F000Fu) ^ 0x43084308u;
  f.p26 = ((w >> 8) & 0x000F000Fu) ^ 0x43084308u;
  f.p37 = ((w >> 12) & 0x000F000Fu) ^ 0x43084308u;
  return f;
}
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// This CTA's share of `total` work items: total/grid each, the first total%grid CTAs one more.
__device__ __forceinline__ void w4_share(uint32_t total, uint32_t &first, uint32_t &count) {
  const uint32_t per = total / gridDim.x, rem = total - per * gridDim.x;
  first = blockIdx.x * per + min((uint32_t)blockIdx.x, rem);
  count = per + (blockIdx.x < rem ? 1u : 0u);
}

// Dynamic shared memory of the gate/up kernel: red [2][16 warps][2][16 x 8] f32 | x [8][2d + 64] bytes (every run of 8
// elements stored as 0,4,1,5,2,6,3,7) | xsum [8][G] f32 | items [max_items] | pref [max_items + 1].
inline size_t w4_gateup_smem_bytes(int max_items, int d) {
  return (size_t)2 * 16 * 2 * 128 * 4 + (size_t)8 * (2 * d + 64) + (size_t)8 * (d / kGroup) * 4 +
         (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}
// ... of the down kernel: h [16 warps][2][8 units x 8 tokens x 16 neurons] bf16 | items | pref.
inline size_t w4_down_smem_bytes(int max_items) {
  return (size_t)16 * 2 * 2048 + (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}

template <int GW, int NW>   // GW quantisation groups per warp, NW warps take part: d = 128 * GW * NW
__global__ void __launch_bounds__(kW4Threads, 1) w4_gateup_kernel(W4Params p) {
  constexpr int G = GW * NW, d = kGroup * G;
  constexpr uint32_t kUA = 2112u * G;               // bytes of a unit: gate tiles, up tiles, gate scales, up scales
  constexpr uint32_t kXStride = 2u * d + 64u;
  extern __shared__ __align__(128) unsigned char smem[];
  float *s_red = reinterpret_cast<float *>(smem);                         // [2][16][2][128]
  unsigned char *s_x = smem + 2 * 16 * 2 * 128 * 4;
  float *s_xsum = reinterpret_cast<float *>(s_x + 8 * kXStride);          // [8][G]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_xsum + 8 * G);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);

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
  const uint32_t NBLK = (uint32_t)p.inter / 16u;
  const bool dense = p.T <= kQ4Tokens;
  const bool k_warp = (NW == 16) || warp < NW;

  // x rows of the MMA columns into shared memory, every run of 8 stored as 0,4,1,5,2,6,3,7 (the order in which the
  // dequantiser produces the codes of a word), and their sums over each quantisation group
  auto stage_x = [&](auto tok_of_column) {
    for (int i = tid; i < 8 * (d / 8); i += kW4Threads) {
      const int j = i / (d / 8), c8 = i - j * (d / 8);
      const int tok = tok_of_column(j);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok >= 0) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 8 * c8);
      uint4 o;
      o.x = __byte_perm(v.x, v.z, 0x5410);   // (x0, x4)
      o.y = __byte_perm(v.x, v.z, 0x7632);   // (x1, x5)
      o.z = __byte_perm(v.y, v.w, 0x5410);   // (x2, x6)
      o.w = __byte_perm(v.y, v.w, 0x7632);   // (x3, x7)
      *reinterpret_cast<uint4 *>(s_x + j * kXStride + 16 * c8) = o;
      float sum = bf16lo(v.x) + bf16hi(v.x) + bf16lo(v.y) + bf16hi(v.y) + bf16lo(v.z) + bf16hi(v.z) + bf16lo(v.w) +
                  bf16hi(v.w);
#pragma unroll
      for (int o2 = 1; o2 < 16; o2 <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);   // 16 chunks = one group
      if ((lane & 15) == 0) s_xsum[j * G + c8 / 16] = sum;
    }
  };

  // ---- per-lane constants ----
  const uint32_t t_off = (uint32_t)(warp * GW) * 1024u + g * 64u + q * 16u;      // row g, chunk q of the warp's first tile
  const uint32_t s_off = 2048u * G + (uint32_t)(warp * GW) * 32u + g * 4u;       // (scale of row g, of row g + 8)
  const uint32_t my_x = smem_u32(s_x) + g * kXStride + (uint32_t)(warp * GW) * 256u + 16u * q;

  uint4 bufg[2 * GW], bufu[2 * GW];
  uint32_t scg[GW], scu[GW];
  auto load_part = [&](uint4 (&buf)[2 * GW], uint32_t (&sc)[GW], const uint8_t *unit, uint32_t which) {
    if (k_warp) {
      const uint8_t *t = unit + which * (1024u * G) + t_off;
#pragma unroll
      for (int gw = 0; gw < GW; ++gw) {
        buf[2 * gw] = ld_stream_16(t + gw * 1024);
        buf[2 * gw + 1] = ld_stream_16(t + gw * 1024 + 512);
      }
      const uint8_t *s = unit + which * (32u * G) + s_off;
#pragma unroll
      for (int gw = 0; gw < GW; ++gw)
        asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(sc[gw]) : "l"(s + gw * 32));
    }
  };
  // scaled partial sums of one part over this warp's groups -> shared memory
  auto part_sums = [&](const uint4 (&buf)[2 * GW], const uint32_t (&sc)[GW], float *r) {
    if (k_warp) {
      float tot[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int gw = 0; gw < GW; ++gw) {
        float a1[4] = {0.f, 0.f, 0.f, 0.f}, a2[4] = {0.f, 0.f, 0.f, 0.f};
        const uint32_t lo[4] = {buf[2 * gw].x, buf[2 * gw].y, buf[2 * gw].z, buf[2 * gw].w};
        const uint32_t hi[4] = {buf[2 * gw + 1].x, buf[2 * gw + 1].y, buf[2 * gw + 1].z, buf[2 * gw + 1].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {   // word j: hidden indices 32j + 8q + 0..7 of the group
          const W4Frag fl = w4_unpack(lo[j]), fh = w4_unpack(hi[j]);
          const uint4 xv = lds_v4(my_x + gw * 256u + j * 64u);
          mma_bf16(a1, fl.p04, fh.p04, fl.p15, fh.p15, xv.x, xv.y);
          mma_bf16(a2, fl.p26, fh.p26, fl.p37, fh.p37, xv.z, xv.w);
        }
        const float s_lo = bf16lo(sc[gw]), s_hi = bf16hi(sc[gw]);
        const int grp = warp * GW + gw;
        const float b0 = kW4Bias * s_xsum[(2 * q) * G + grp], b1 = kW4Bias * s_xsum[(2 * q + 1) * G + grp];
        tot[0] += s_lo * (a1[0] + a2[0] - b0);
        tot[1] += s_lo * (a1[1] + a2[1] - b1);
        tot[2] += s_hi * (a1[2] + a2[2] - b0);
        tot[3] += s_hi * (a1[3] + a2[3] - b1);
      }
      *reinterpret_cast<float2 *>(r + g * 8 + 2 * q) = make_float2(tot[0], tot[1]);
      *reinterpret_cast<float2 *>(r + (g + 8) * 8 + 2 * q) = make_float2(tot[2], tot[3]);
    }
  };

  // ---- this CTA's share of the units: resident range, then host-resident range ----
  uint32_t rfirst0, rcount0, rfirst1, rcount1;
  w4_share((uint32_t)s_pref[n_items] * NBLK, rfirst0, rcount0);
  w4_share((uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * NBLK, rfirst1, rcount1);
  rfirst1 += (uint32_t)s_pref[n_items] * NBLK;
  struct Seg { const uint8_t *unit0; int item, pass, n_units; uint32_t hrow; };
  int range = 0, item = 0;
  uint32_t pu = 0, b = 0, left = 0;
  auto next_segment = [&](Seg &s) -> bool {
    while (left == 0) {
      if (range == 2) return false;
      left = range ? rcount1 : rcount0;
      if (left > 0) {
        const uint32_t first = range ? rfirst1 : rfirst0;
        pu = first / NBLK;
        b = first - pu * NBLK;
      }
      ++range;
    }
    while ((uint32_t)s_pref[item + 1] <= pu) ++item;
    s.item = item;
    s.pass = (int)(pu - (uint32_t)s_pref[item]);
    s.n_units = (int)min(left, NBLK - b);
    s.unit0 = s_items[item].w + (size_t)b * kUA;
    s.hrow = pu * NBLK + b;
    left -= s.n_units;
    ++pu;
    b = 0;
    return true;
  };

  Seg sg, nsg;
  bool more = next_segment(sg);
  if (more) {
    load_part(bufg, scg, sg.unit0, 0);
    load_part(bufu, scu, sg.unit0, 1);
  }
  if (dense) {
    stage_x([&](int j) { return j < p.T ? j : -1; });
    __syncthreads();
  }
  uint32_t par = 0;
  while (more) {
    more = next_segment(nsg);
    const uint8_t *after = more ? nsg.unit0 : nullptr;
    if (!dense) {   // MMA column j is the pass's j-th pair: stage those tokens' rows
      const WorkItem &it = s_items[sg.item];
      const int tok0 = sg.pass * kQ4Tokens, nt = min(kQ4Tokens, it.n_tok - tok0);
      const int off_ = it.off + tok0, expert_ = it.expert;
      __syncthreads();   // the previous segment's readers of s_x / s_xsum are done
      stage_x([&](int j) {
        if (j >= nt) return -1;
        return expert_ >= 0 ? p.perm[off_ + j] / p.top_k : tok0 + j;
      });
      __syncthreads();
    }
    const uint8_t *unit = sg.unit0;
    for (int k = 0; k < sg.n_units; ++k, unit += kUA) {
      const uint8_t *nunit = (k + 1 < sg.n_units) ? unit + kUA : after;
      float *red = s_red + par * (16 * 2 * 128);
      part_sums(bufg, scg, red + (warp * 2 + 0) * 128);
      if (nunit) load_part(bufg, scg, nunit, 0);
      part_sums(bufu, scu, red + (warp * 2 + 1) * 128);
      if (nunit) load_part(bufu, scu, nunit, 1);
      __syncthreads();
      {   // h = SiLU(sum gate) * (sum up): four threads per value, each sums a quarter of the warps' partial sums
        const int r = tid >> 2, qu = tid & 3;   // r = neuron * 8 + token
        float a = 0.f, c = 0.f;
#pragma unroll
        for (int w = 0; w < NW / 4; ++w) {
          a += red[((qu * (NW / 4) + w) * 2 + 0) * 128 + r];
          c += red[((qu * (NW / 4) + w) * 2 + 1) * 128 + r];
        }
        if (NW % 4 != 0 && qu < NW % 4) {   // (NW = 14: two warps left over)
          a += red[(((NW / 4) * 4 + qu) * 2 + 0) * 128 + r];
          c += red[(((NW / 4) * 4 + qu) * 2 + 1) * 128 + r];
        }
        a += __shfl_xor_sync(0xffffffffu, a, 1);
        c += __shfl_xor_sync(0xffffffffu, c, 1);
        a += __shfl_xor_sync(0xffffffffu, a, 2);
        c += __shfl_xor_sync(0xffffffffu, c, 2);
        if (qu == 0)
          p.hbuf[((size_t)sg.hrow + k) * 128 + (r & 7) * 16 + (r >> 3)] = __float2bfloat16_rn(__fdividef(a, 1.f + __expf(-a)) * c);
      }
      par ^= 1u;   // the next unit writes the other buffer: one barrier per unit is enough
    }
    sg = nsg;
  }
}

template <int NWD>   // warps that own output columns: a column block is 64 * NWD columns
__global__ void __launch_bounds__(kW4Threads, 1) w4_down_kernel(W4Params p, int d) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_h = smem;                                                // [16 warps][2][2048 bytes]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(smem + 16 * 2 * 2048);
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

  if (warp < NWD) {
    uint32_t rfirst0, rcount0, rfirst1, rcount1;
    w4_share((uint32_t)s_pref[n_items] * per_pass, rfirst0, rcount0);
    w4_share((uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * per_pass, rfirst1, rcount1);
    rfirst1 += (uint32_t)s_pref[n_items] * per_pass;
    const uint32_t my_h = smem_u32(s_h) + (uint32_t)warp * 4096u;

    // chunk cursor: (pass pu, column block cb, neuron group ng)
    struct Ck { const uint8_t *rec; uint32_t pu, cb, ng; int item; };
    int range = 0, item = 0;
    uint32_t cur = 0, left = 0;
    auto next_chunk = [&](Ck &c) -> bool {
      while (left == 0) {
        if (range == 2) return false;
        left = range ? rcount1 : rcount0;
        cur = range ? rfirst1 : rfirst0;
        ++range;
      }
      c.pu = cur / per_pass;
      const uint32_t r = cur - c.pu * per_pass;
      c.cb = r / NG;
      c.ng = r - c.cb * NG;
      while ((uint32_t)s_pref[item + 1] <= c.pu) ++item;
      c.item = item;
      c.rec = s_items[item].w;
      ++cur;
      --left;
      return true;
    };
    uint4 bufa[8], bufb[8];   // this chunk's / the next chunk's eight steps
    uint4 sca, scb;           // and their scales: (column g, column g + 8) of the warp's four tiles
    auto load_chunk = [&](uint4 (&buf)[8], uint4 &sc, const Ck &c, int hslot) {
      const uint8_t *t = c.rec + sec_b + ((size_t)(c.cb * NG + c.ng) * 8u * NWD + warp) * 512u + lane * 16u;
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) buf[uu] = ld_stream_16(t + (size_t)uu * NWD * 512u);
      sc = ld_stream_16(c.rec + sec_c + ((size_t)(c.ng * CB + c.cb) * NWD + warp) * 128u + g * 16u);
      // h of the chunk's 8 units (2 KiB, contiguous) for this warp alone
      const unsigned char *hsrc = reinterpret_cast<const unsigned char *>(p.hbuf) + ((size_t)c.pu * NBLK + c.ng * 8u) * 256u;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(my_h + hslot * 2048u + (i * 32 + lane) * 16u),
                     "l"(hsrc + (i * 32 + lane) * 16)
                     : "memory");
      asm volatile("cp.async.commit_group;" ::: "memory");
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
    // one chunk: 8 steps of 16 neurons for the warp's four column tiles, then scale and bias
    auto consume = [&](const uint4 (&buf)[8], const uint4 &sc, int hslot) {
      asm volatile("cp.async.wait_group 1;" ::: "memory");   // this chunk's h has landed (the next one's may be in flight)
      __syncwarp();
      float acc[4][4];
#pragma unroll
      for (int j = 0; j < 4; ++j) { acc[j][0] = acc[j][1] = acc[j][2] = acc[j][3] = 0.f; }
      float hs = 0.f;
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) {
        uint2 hb;   // h of token g, neurons 4q..4q+3 of the step
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(hb.x), "=r"(hb.y) : "r"(my_h + hslot * 2048u + uu * 256u + g * 32u + q * 8u));
        hs += bf16lo(hb.x) + bf16hi(hb.x) + bf16lo(hb.y) + bf16hi(hb.y);
        const uint32_t wv[4] = {buf[uu].x, buf[uu].y, buf[uu].z, buf[uu].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const W4Frag f = w4_unpack(wv[j]);
          mma_bf16(acc[j], f.p04, f.p15, f.p26, f.p37, hb.x, hb.y);
        }
      }
      __syncwarp();   // every lane has read the slot: it may be overwritten by the chunk after the next
      hs += __shfl_xor_sync(0xffffffffu, hs, 1);      // sum over the four lanes of token g: its 128 neurons
      hs += __shfl_xor_sync(0xffffffffu, hs, 2);
      const float b0 = kW4Bias * __shfl_sync(0xffffffffu, hs, (2 * q) * 4);
      const float b1 = kW4Bias * __shfl_sync(0xffffffffu, hs, (2 * q + 1) * 4);
      const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float s_lo = bf16lo(sw[j]), s_hi = bf16hi(sw[j]);
        dtot[j][0] += s_lo * (acc[j][0] - b0);
        dtot[j][1] += s_lo * (acc[j][1] - b1);
        dtot[j][2] += s_hi * (acc[j][2] - b0);
        dtot[j][3] += s_hi * (acc[j][3] - b1);
      }
    };

    Ck ck, nk;
    bool have = next_chunk(ck);
    if (have) {
      load_chunk(bufa, sca, ck, 0);
      begin_pass(ck);
      zero_tot();
    }
    int slot = 0;
    while (have) {
      const bool more = next_chunk(nk);
      // even steps: current chunk in bufa; odd steps: in bufb
      if (slot == 0) {
        if (more) load_chunk(bufb, scb, nk, 1); else asm volatile("cp.async.commit_group;" ::: "memory");
        consume(bufa, sca, 0);
      } else {
        if (more) load_chunk(bufa, sca, nk, 0); else asm volatile("cp.async.commit_group;" ::: "memory");
        consume(bufb, scb, 1);
      }
      if (!more || nk.pu != ck.pu || nk.cb != ck.cb) {
        flush(ck.cb);
        zero_tot();
        if (more && nk.pu != ck.pu) begin_pass(nk);
      }
      ck = nk;
      have = more;
      slot ^= 1;
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
