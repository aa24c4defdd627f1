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
//   w4_gateup_kernel : 16 warps per SM, every warp streams whole 16-neuron units (gate tiles, up tiles and their
//                      scales: contiguous) by itself: no partial sums to exchange, no block-level synchronisation
//                      while a call has at most 8 tokens.  A lane's two 16-byte loads per quantisation group are rows
//                      g and g+8 of the group's tile; a rolling buffer of 16 such loads per lane is refilled as soon
//                      as a pair has been consumed, so about 128 KiB per SM stay in flight.  h = SiLU(g) * u goes
//                      to a small global buffer, bf16 [pass][unit][token][neuron].
//   w4_down_kernel   : walks chunks (expert pass, block of 64*NWD output columns, group of 128 neurons) = 8 steps
//                      of 16 neurons x 512 bytes per warp.  Every warp owns four 16-column tiles: its 16-byte load
//                      per step is their four A fragments; the same rolling buffer, two chunks deep.  No block-level
//                      synchronisation: a warp stages the chunk's h fragments and scales for itself with cp.async.
//                      Scale and bias are folded when the chunk (= one neuron group) ends; the scaled totals persist
//                      while consecutive chunks belong to the same pass and column block.  The gate-weighted combine
//                      is a red.global.add into the fp32 accumulator; the last CTA rounds it once to bf16.  Launched
//                      as a programmatic dependent of the gate/up kernel: its set-up overlaps that kernel's tail.
// Zero-copy experts (records in the mapped host pool) go through the same kernels.
#pragma once
#include "async.cuh"
#include "common.cuh"
#include "ffn_stream.cuh"   // red_add_f32

namespace ftmoe {

constexpr int kQ4Tokens = 8;         // tokens per weight pass
constexpr int kW4Threads = 512;
constexpr int kW4Warps = kW4Threads / 32;
constexpr float kW4Bias = 136.f;
#ifndef W4_BLOCK_PAIRS
#define W4_BLOCK_PAIRS 4
#endif     // the dequantised operand is 136 + code

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
  float *hbias;             // [pass][16-neuron unit][token 8]: 136 x the sum of the unit's 16 (rounded) h values
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;
  uint32_t *done;
  uint32_t *status;
  int inter, top_k, T, finalize;
  uint32_t mask, magic;     // 0x000F000F, 0x43084308 (see w4_unpack)
};

// 8 codes of one word -> four bf16x2 registers holding 136 + code: pairs (0,4) (1,5) (2,6) (3,7).
struct W4Frag { uint32_t p04, p15, p26, p37; };
// mask = 0x000F000F and magic = 0x43084308 arrive as kernel arguments: as literals the compiler encodes both as
// immediates and needs two logic instructions per register (an instruction carries one immediate); as values it
// cannot see through they live in registers and (x & mask) ^ magic is a single three-input logic instruction.
struct W4Const { uint32_t mask, magic; };
__device__ __forceinline__ W4Frag w4_unpack(uint32_t w, const W4Const &k) {
  W4Frag f;
  f.p04 = (w & k.mask) ^ k.magic;
  f.p15 = ((w >> 4) & k.mask) ^ k.magic;
  f.p26 = ((w >> 8) & k.mask) ^ k.magic;
  f.p37 = ((w >> 12) & k.mask) ^ k.magic;
  return f;
}
// d = a * b (no accumulator to clear first)
__device__ __forceinline__ void mma_bf16_first(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(c[0]), "=f"(c[1]), "=f"(c[2]), "=f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1), "f"(0.f));
}
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

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

// Dynamic shared memory of the gate/up kernel: x [8][2d + 64] bytes (every run of 8 elements stored as
// 0,4,1,5,2,6,3,7) | xbias [8][G] f32 (136 x the sum of x over a group) | items [max_items] | pref [max_items + 1].
inline size_t w4_gateup_smem_bytes(int max_items, int d) {
  return (size_t)8 * (2 * d + 64) + (size_t)8 * (d / kGroup) * 4 + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}
// ... of the down kernel: per warp 3 slots of (h [8 units x 8 tokens x 16 neurons] bf16 | 128 bytes of scales |
// h bias [8 units][8 tokens] f32) | items | pref.
constexpr uint32_t kW4DownSlot = 2048 + 128 + 256;
inline size_t w4_down_smem_bytes(int max_items) {
  return (size_t)kW4Warps * 3 * kW4DownSlot + (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}

template <int G>   // quantisation groups of the hidden dimension: d = 128 G, G a multiple of 4
__global__ void __launch_bounds__(kW4Threads, 1) w4_gateup_kernel(W4Params p) {
  constexpr int d = kGroup * G;
  constexpr int kPairs = 2 * G;                     // (row g, row g+8) load pairs of a unit: G gate groups, G up groups
  constexpr uint32_t kUA = 2112u * G;               // bytes of a unit: gate tiles, up tiles, gate scales, up scales
  constexpr uint32_t kXStride = 2u * d + 64u;
  static_assert(G % 4 == 0, "the rolling buffer holds 8 pairs");
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_x = smem;
  float *s_xbias = reinterpret_cast<float *>(s_x + 8 * kXStride);          // [8][G]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_xbias + 8 * G);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the down kernel may set itself up meanwhile
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

  // x rows of the MMA columns into shared memory, every run of 8 stored as 0,4,1,5,2,6,3,7 (the order in which the
  // dequantiser produces the codes of a word), and 136 x their sums over each quantisation group
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
      if ((lane & 15) == 0) s_xbias[j * G + c8 / 16] = kW4Bias * sum;
    }
  };

  const uint32_t my_x = smem_u32(s_x) + g * kXStride + 16u * q;
  const float *my_b0 = s_xbias + (2 * q) * G, *my_b1 = s_xbias + (2 * q + 1) * G;

  const W4Const ks = {p.mask, p.magic};
  // One warp streams `n_units` consecutive units starting at `base`; their h goes to rows hrow0.. of the h buffer.
  // Work proceeds in blocks of 8 (row g, row g+8) load pairs = 8 quantisation groups of the gate or the up part.
  constexpr int kBP = W4_BLOCK_PAIRS;               // pairs of a block = depth of the rolling register buffer
  constexpr int kBlocks = kPairs / kBP;             // blocks of a unit
  static_assert(G % kBP == 0, "a block lies in the gate or in the up part");
  auto run = [&](const uint8_t *base, int n_units, uint32_t hrow0) {
    uint4 buf[2 * kBP];
    uint32_t sc[kBP];   // and the two rows' scales
    const uint8_t *nptr = base + g * 64 + q * 16;              // next block to request
    const uint8_t *nsc = base + 2048u * G + g * 4;
    int nblk = 0, blocks_left = n_units * kBlocks;             // its index in its unit; blocks not yet requested
    auto advance = [&]() {
      nptr += kBP * 1024;
      nsc += kBP * 32;
      --blocks_left;
      if (++nblk == kBlocks) {   // on to the next unit: skip this unit's scales / the next unit's tiles
        nblk = 0;
        nptr += 64 * G;
        nsc += 2048u * G;
      }
    };
#pragma unroll
    for (int pi = 0; pi < kBP; ++pi) {
      buf[2 * pi] = ld_stream_16(nptr + pi * 1024);
      buf[2 * pi + 1] = ld_stream_16(nptr + pi * 1024 + 512);
      asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(sc[pi]) : "l"(nsc + pi * 32));
    }
    advance();
    for (int u = 0; u < n_units; ++u) {
      float tot[4] = {0.f, 0.f, 0.f, 0.f}, tg[4] = {0.f, 0.f, 0.f, 0.f};
      int xg = 0;                                    // first group of the block
      for (int blk = 0; blk < kBlocks; ++blk) {
        const bool more = blocks_left > 0;
        const uint8_t *rp = nptr, *rs = nsc;         // the block that refills this one's registers
        if (more) advance();
        const uint32_t xa = my_x + xg * 256u;
        const float *b0p = my_b0 + xg, *b1p = my_b1 + xg;
#pragma unroll
        for (int pi = 0; pi < kBP; ++pi) {
          float a1[4], a2[4];
          const uint32_t lo[4] = {buf[2 * pi].x, buf[2 * pi].y, buf[2 * pi].z, buf[2 * pi].w};
          const uint32_t hi[4] = {buf[2 * pi + 1].x, buf[2 * pi + 1].y, buf[2 * pi + 1].z, buf[2 * pi + 1].w};
          const uint32_t scale = sc[pi];
#pragma unroll
          for (int j = 0; j < 4; ++j) {   // word j: hidden indices 32j + 8q + 0..7 of the group
            const W4Frag fl = w4_unpack(lo[j], ks), fh = w4_unpack(hi[j], ks);
            const uint4 xv = lds_v4(xa + pi * 256u + j * 64u);
            if (j == 0) {
              mma_bf16_first(a1, fl.p04, fh.p04, fl.p15, fh.p15, xv.x, xv.y);
              mma_bf16_first(a2, fl.p26, fh.p26, fl.p37, fh.p37, xv.z, xv.w);
            } else {
              mma_bf16(a1, fl.p04, fh.p04, fl.p15, fh.p15, xv.x, xv.y);
              mma_bf16(a2, fl.p26, fh.p26, fl.p37, fh.p37, xv.z, xv.w);
            }
          }
          if (more) {   // refill the pair just consumed
            buf[2 * pi] = ld_stream_16(rp + pi * 1024);
            buf[2 * pi + 1] = ld_stream_16(rp + pi * 1024 + 512);
            asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(sc[pi]) : "l"(rs + pi * 32));
          }
          const float s_lo = bf16lo(scale), s_hi = bf16hi(scale);
          const float b0 = b0p[pi], b1 = b1p[pi];
          tot[0] += s_lo * (a1[0] + a2[0] - b0);
          tot[1] += s_lo * (a1[1] + a2[1] - b1);
          tot[2] += s_hi * (a1[2] + a2[2] - b0);
          tot[3] += s_hi * (a1[3] + a2[3] - b1);
        }
        xg += kBP;
        if (xg == G) {
          xg = 0;
          if (blk < kBlocks - 1) {   // the gate sums are complete: the up groups follow
#pragma unroll
            for (int i = 0; i < 4; ++i) { tg[i] = tot[i]; tot[i] = 0.f; }
          }
        }
      }
      // h = SiLU(gate) * up of neurons g, g+8 and tokens 2q, 2q+1, rounded to bf16; and 136 x its sums over the
      // unit's 16 neurons, which the down kernel subtracts
      __nv_bfloat16 *hrow = p.hbuf + ((size_t)hrow0 + u) * 128;
      float hr[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float a = tg[i];
        const __nv_bfloat16 hv = __float2bfloat16_rn(__fdividef(a, 1.f + __expf(-a)) * tot[i]);
        hrow[(2 * q + (i & 1)) * 16 + g + 8 * (i >> 1)] = hv;
        hr[i] = __bfloat162float(hv);
      }
      float s0 = hr[0] + hr[2], s1 = hr[1] + hr[3];
#pragma unroll
      for (int o = 4; o < 32; o <<= 1) {
        s0 += __shfl_xor_sync(0xffffffffu, s0, o);
        s1 += __shfl_xor_sync(0xffffffffu, s1, o);
      }
      if (g == 0) *reinterpret_cast<float2 *>(p.hbias + ((size_t)hrow0 + u) * 8 + 2 * q) = make_float2(kW4Bias * s0, kW4Bias * s1);
    }
  };

  if (dense) {
    stage_x([&](int j) { return j < p.T ? j : -1; });
    __syncthreads();
  }
  // Units (pass, 16-neuron block) in one flat order, split evenly over all warps of the grid: the slot-resident
  // range first, then the host-resident range.
  const uint32_t n_warps = gridDim.x * kW4Warps, wi = blockIdx.x * kW4Warps + warp;
  for (int range = 0; range < 2; ++range) {
    const uint32_t pass0 = range ? (uint32_t)s_pref[n_items] : 0u;
    const uint32_t pass1 = range ? (uint32_t)s_pref[n_items + n_zc] : (uint32_t)s_pref[n_items];
    const uint32_t total = (pass1 - pass0) * NBLK, ubase = pass0 * NBLK;
    if (total == 0) continue;
    const uint32_t wf = ubase + w4_first(total, n_warps, wi), we = ubase + w4_first(total, n_warps, wi + 1);
    const uint32_t cf = ubase + w4_first(total, n_warps, blockIdx.x * kW4Warps);
    const uint32_t ce = ubase + w4_first(total, n_warps, (blockIdx.x + 1) * kW4Warps);
    if (cf >= ce) continue;
    for (uint32_t pu = cf / NBLK; pu * NBLK < ce; ++pu) {   // the passes this CTA's warps touch
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
      const uint32_t lo = max(wf, pu * NBLK), hi = min(we, (pu + 1) * NBLK);
      if (lo < hi) run(it.w + (size_t)(lo - pu * NBLK) * kUA, (int)(hi - lo), lo);
    }
  }
}

template <int NWD>   // warps that own output columns: a column block is 64 * NWD columns
__global__ void __launch_bounds__(kW4Threads, 1) w4_down_kernel(W4Params p, int d) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_h = smem;                                                // [16 warps][3][h 2048 | scales 128]
  WorkItem *s_items = reinterpret_cast<WorkItem *>(smem + kW4Warps * 3 * kW4DownSlot);
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
    const uint32_t my_h = smem_u32(s_h) + (uint32_t)warp * 3u * kW4DownSlot;
    const W4Const ks = {p.mask, p.magic};

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
    // h of the chunk's 8 units (2 KiB, contiguous) and the chunk's scales for this warp alone
    auto stage = [&](const Ck &c, uint32_t slot) {
      const unsigned char *hsrc = reinterpret_cast<const unsigned char *>(p.hbuf) + ((size_t)c.pu * NBLK + c.ng * 8u) * 256u;
      const uint32_t dst = my_h + slot * kW4DownSlot;
#pragma unroll
      for (int i = 0; i < 4; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (i * 32 + lane) * 16u), "l"(hsrc + (i * 32 + lane) * 16)
                     : "memory");
      if (lane < 8)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2048u + lane * 16u),
                     "l"(c.rec + sec_c + ((size_t)(c.ng * CB + c.cb) * NWD + warp) * 128u + lane * 16u)
                     : "memory");
      else if (lane < 24)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 2176u + (lane - 8) * 16u),
                     "l"(reinterpret_cast<const unsigned char *>(p.hbias) + ((size_t)c.pu * NBLK + c.ng * 8u) * 32u + (lane - 8) * 16)
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
    // one chunk: 8 steps of 16 neurons for the warp's four column tiles, then scale and bias; every step's
    // register is refilled with the same step of the chunk two ahead as soon as it has been consumed
    auto consume = [&](uint4 (&buf)[8], uint32_t slot, const uint8_t *refill) {
      asm volatile("cp.async.wait_group 2;" ::: "memory");   // this chunk's h, scales and biases have landed
      __syncwarp();
      const uint32_t hs_base = my_h + slot * kW4DownSlot;
      float acc[4][4];
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) {
        uint2 hb;   // h of token g, neurons 4q..4q+3 of the step
        asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(hb.x), "=r"(hb.y) : "r"(hs_base + uu * 256u + g * 32u + q * 8u));
        const uint32_t wv[4] = {buf[uu].x, buf[uu].y, buf[uu].z, buf[uu].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const W4Frag f = w4_unpack(wv[j], ks);
          if (uu == 0) mma_bf16_first(acc[j], f.p04, f.p15, f.p26, f.p37, hb.x, hb.y);
          else mma_bf16(acc[j], f.p04, f.p15, f.p26, f.p37, hb.x, hb.y);
        }
        if (refill) buf[uu] = ld_stream_16(refill + (size_t)uu * NWD * 512u);
      }
      const uint4 sc = lds_v4(hs_base + 2048u + g * 16u);   // (column g, column g + 8) of the warp's four tiles
      float b0 = 0.f, b1 = 0.f;                             // 136 x the sums of h over the chunk's 128 neurons
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) {
        float2 hb2;
        asm volatile("ld.shared.v2.f32 {%0,%1}, [%2];" : "=f"(hb2.x), "=f"(hb2.y) : "r"(hs_base + 2176u + uu * 32u + q * 8u));
        b0 += hb2.x;
        b1 += hb2.y;
      }
      __syncwarp();   // every lane has read the slot: it may be overwritten
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

    uint4 bufa[8], bufb[8];   // even / odd chunks of this CTA's sequence
    Ck c0, c1, c2;            // the chunk being consumed and the two after it
    bool h0 = next_chunk(c0), h1 = h0 && next_chunk(c1), h2 = h1 && next_chunk(c2);
    if (h0) {
      stage(c0, 0);
      const uint8_t *w = weights_of(c0);
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) bufa[uu] = ld_stream_16(w + (size_t)uu * NWD * 512u);
      begin_pass(c0);
      zero_tot();
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    if (h1) {
      stage(c1, 1);
      const uint8_t *w = weights_of(c1);
#pragma unroll
      for (int uu = 0; uu < 8; ++uu) bufb[uu] = ld_stream_16(w + (size_t)uu * NWD * 512u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    uint32_t slot = 0;
    int half = 0;
    while (h0) {
      const uint32_t slot2 = slot >= 1 ? slot - 1 : 2;   // (slot + 2) % 3
      if (h2) stage(c2, slot2);
      asm volatile("cp.async.commit_group;" ::: "memory");
      const uint8_t *refill = h2 ? weights_of(c2) : nullptr;
      if (half == 0) consume(bufa, slot, refill); else consume(bufb, slot, refill);
      if (!h1 || c1.pu != c0.pu || c1.cb != c0.cb) {
        flush(c0.cb);
        zero_tot();
        if (h1 && c1.pu != c0.pu) begin_pass(c1);
      }
      c0 = c1; c1 = c2;
      h0 = h1; h1 = h2;
      h2 = h1 && next_chunk(c2);
      slot = slot == 2 ? 0 : slot + 1;
      half ^= 1;
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
