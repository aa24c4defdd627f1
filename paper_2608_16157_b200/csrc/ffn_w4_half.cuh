// The int4 kernels of ffn_w4.cuh for calls with at most 4 tokens.  The MMA has 8 columns whatever the token count;
// with <= 4 tokens column 2t holds the hi bytes and column 2t+1 the lo bytes of token t's fixed-point activations,
// so ONE int8 MMA per pair of weight words yields both partial sums (128 S_hi + S_lo are neighbours in a lane's
// accumulator fragment), where the 8-token kernels issue two.  Half the tensor-core instructions, half the
// activation-fragment loads and half the folding arithmetic per weight; everything else (record layout, work
// distribution, buffers, the hand-over of h through global memory) is as in ffn_w4.cuh.  Calls with <= 4 tokens have
// one pass per expert and MMA column pair t = token t, so none of the many-token machinery is needed here.
#pragma once
#include "ffn_w4.cuh"

namespace ftmoe {

constexpr int kW4HalfTokens = 4;
#ifndef W4_HALF_BS
#define W4_HALF_BS 2
#endif
constexpr int kW4HalfBlockSteps = W4_HALF_BS;   // quantisation-group steps a warp of the gate/up kernel keeps in flight

// gate/up: x [8 columns][d + 32] bytes (per run of 8 elements 8 bytes: the column's bytes of elements 0,2,4,6 |
// 1,3,5,7) | scale [4][G], bias [4][G] f32 | items | pref.
inline size_t w4_gateup_half_smem_bytes(int max_items, int d) {
  return (size_t)8 * (d + 32) + (size_t)2 * 4 * (d / kGroup) * 4 + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}
// down: per warp 2 slots of (h operands 1024 | 128 bytes of weight scales | 64 bytes of (scale, bias) per token).
constexpr uint32_t kW4HalfDownSlot = 1024 + 128 + 64;
inline size_t w4_down_half_smem_bytes(int max_items) {
  return (size_t)kW4Warps * 2 * kW4HalfDownSlot + (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}

__device__ __forceinline__ uint2 lds_v2(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}

template <int G>
__global__ void __launch_bounds__(kW4Threads, 1) w4_gateup_half_kernel(W4Params p) {
  constexpr int d = kGroup * G;
  constexpr uint32_t kUA = 2112u * G;
  constexpr uint32_t kXStride = (uint32_t)d + 32u;   // = 32 mod 128: conflict-free 8-byte fragment loads
  constexpr int kBS = kW4HalfBlockSteps;
  constexpr int kBlocks = G / kBS;
  constexpr int kKS = kW4KSplit, kBlocksP = kBlocks / kKS;   // blocks of a piece
  static_assert(G % kBS == 0 && kBlocks % kKS == 0, "whole blocks, whole pieces");
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_x = smem;
  float *s_sx = reinterpret_cast<float *>(s_x + 8 * kXStride);             // [4][G] m / 16256
  float *s_xb = s_sx + 4 * G;                                              // [4][G] 8 (m / 16256) sum(fixed)
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_xb + 4 * G);
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
  // token t -> columns 2t (hi bytes) and 2t+1 (lo bytes)
  for (int i = tid; i < kW4HalfTokens * (d / 8); i += kW4Threads) {
    const int t = i / (d / 8), c8 = i - t * (d / 8);
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (t < p.T) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)t * d + 8 * c8);
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
    *reinterpret_cast<uint2 *>(s_x + (2 * t) * kXStride + 8 * c8) = make_uint2(fx.hi_even, fx.hi_odd);
    *reinterpret_cast<uint2 *>(s_x + (2 * t + 1) * kXStride + 8 * c8) = make_uint2(fx.lo_even, fx.lo_odd);
    int sum = fx.sum;
#pragma unroll
    for (int o2 = 1; o2 < 16; o2 <<= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o2);
    if ((lane & 15) == 0) {
      s_sx[t * G + c8 / 16] = scale;
      s_xb[t * G + c8 / 16] = 8.f * (float)sum * scale;
    }
  }
  __syncthreads();
  if (p.overlap == 2) asm volatile("griddepcontrol.wait;" ::: "memory");   // (see the 8-token kernel)
  const uint32_t NBLK = (uint32_t)p.inter / 16u;
  const uint32_t my_x = smem_u32(s_x) + g * kXStride + 8u * q;      // column g, run q of a 32-wide slice
  const float *my_s = s_sx + q * G, *my_b = s_xb + q * G;           // this lane's accumulator columns 2q, 2q+1 = token q
  const uint32_t km = p.mask, kf = p.flip;

  // the warp that completes a group of 128 neurons converts it: lane = (token, quarter); tokens >= 4 do not exist
  auto convert_group = [&](uint32_t grp) {
    const int tok = lane >> 2, qt = lane & 3;
    const bool live = tok < kW4HalfTokens;
    float *src = p.hraw + ((size_t)grp * 8 + 2 * qt) * 256 + (live ? tok : 0) * 16;   // per unit: gate sums | up sums
    float v[2][16];
#pragma unroll
    for (int u = 0; u < 2; ++u)
#pragma unroll
      for (int k4 = 0; k4 < 4; ++k4) {
        float4 *pg = reinterpret_cast<float4 *>(src + u * 256) + k4, *pu_ = reinterpret_cast<float4 *>(src + u * 256 + 128) + k4;
        const float4 a = __ldcg(pg), b = __ldcg(pu_);
        if (live) {   // the sums start from zero in the next call
          __stcg(pg, make_float4(0.f, 0.f, 0.f, 0.f));
          __stcg(pu_, make_float4(0.f, 0.f, 0.f, 0.f));
        }
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
    for (int o = 1; o < 4; o <<= 1) {
      m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
      bad |= __shfl_xor_sync(0xffffffffu, (int)bad, o) != 0;
    }
    float scale, inv;
    w4_group_scale(m, bad, scale, inv);
    int sum = 0;
    // [unit pair 4][column 8][q 4][4 neurons of u0 | 4 neurons of u1]: hi bytes in column 2 tok, lo in 2 tok + 1
    uint8_t *dst = p.hq + (size_t)grp * 1024 + qt * 256 + (2 * tok) * 32;
#pragma unroll
    for (int qq = 0; qq < 4; ++qq) {
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
      if (live) {
        *reinterpret_cast<uint2 *>(dst + qq * 8) = make_uint2(o[0], o[1]);
        *reinterpret_cast<uint2 *>(dst + 32 + qq * 8) = make_uint2(o[2], o[3]);
      }
    }
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    sum += __shfl_xor_sync(0xffffffffu, sum, 2);
    if (qt == 0 && live) p.hs[(size_t)grp * 8 + tok] = make_float2(scale, 8.f * (float)sum * scale);
  };

  auto run = [&](const uint8_t *base, int ks0, int n_pieces, uint32_t hrow0) {
    uint4 buf[4 * kBS];     // per step: gate rows g, g+8; up rows g, g+8
    uint32_t sc[2 * kBS];
    const uint8_t *nptr = base + ks0 * (G / kKS) * 1024 + g * 64 + q * 16;
    const uint8_t *nsc = base + 2048u * G + ks0 * (G / kKS) * 32 + g * 4;
    int nblk = ks0 * kBlocksP, blocks_left = n_pieces * kBlocksP;
    auto advance = [&]() {
      nptr += kBS * 1024;
      nsc += kBS * 32;
      --blocks_left;
      if (++nblk == kBlocks) {
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
      float tg[2] = {0.f, 0.f}, tot[2] = {0.f, 0.f};   // gate / up sums of neurons g, g+8 for token q
      for (int blk = 0; blk < kBlocksP; ++blk) {
        const bool more = blocks_left > 0;
        const uint8_t *rp = nptr, *rs = nsc;
        if (more) advance();
        const int xg = ks * (G / kKS) + blk * kBS;
        const uint32_t xa = my_x + xg * 128u;
#pragma unroll
        for (int si = 0; si < kBS; ++si) {
          int ga[4], ua[4];   // [0] = 128-weighted part, [1] = unit part of row g; [2], [3] of row g+8
          const uint32_t glo[4] = {buf[4 * si].x, buf[4 * si].y, buf[4 * si].z, buf[4 * si].w};
          const uint32_t ghi[4] = {buf[4 * si + 1].x, buf[4 * si + 1].y, buf[4 * si + 1].z, buf[4 * si + 1].w};
          const uint32_t ulo[4] = {buf[4 * si + 2].x, buf[4 * si + 2].y, buf[4 * si + 2].z, buf[4 * si + 2].w};
          const uint32_t uhi[4] = {buf[4 * si + 3].x, buf[4 * si + 3].y, buf[4 * si + 3].z, buf[4 * si + 3].w};
          const uint32_t gscale = sc[2 * si], uscale = sc[2 * si + 1];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const uint2 xv = lds_v2(xa + si * 128u + j * 32u);
            const uint32_t a0 = (glo[j] & km) ^ kf, a1 = (ghi[j] & km) ^ kf;
            const uint32_t a2 = ((glo[j] >> 4) & km) ^ kf, a3 = ((ghi[j] >> 4) & km) ^ kf;
            const uint32_t c0 = (ulo[j] & km) ^ kf, c1 = (uhi[j] & km) ^ kf;
            const uint32_t c2 = ((ulo[j] >> 4) & km) ^ kf, c3 = ((uhi[j] >> 4) & km) ^ kf;
            if (j == 0) {
              mma_s8_first(ga, a0, a1, a2, a3, xv.x, xv.y);
              mma_s8_first(ua, c0, c1, c2, c3, xv.x, xv.y);
            } else {
              mma_s8(ga, a0, a1, a2, a3, xv.x, xv.y);
              mma_s8(ua, c0, c1, c2, c3, xv.x, xv.y);
            }
          }
          if (more) request(si, rp, rs);
          const float sx = my_s[xg + si], xb = my_b[xg + si];
          tg[0] += bf16lo(gscale) * ((float)(ga[0] * 128 + ga[1]) * sx - xb);
          tg[1] += bf16hi(gscale) * ((float)(ga[2] * 128 + ga[3]) * sx - xb);
          tot[0] += bf16lo(uscale) * ((float)(ua[0] * 128 + ua[1]) * sx - xb);
          tot[1] += bf16hi(uscale) * ((float)(ua[2] * 128 + ua[3]) * sx - xb);
        }
      }
      // the piece's gate and up sums of neurons g, g+8 and token q join the unit's sums
      float *hacc = p.hraw + (size_t)hrow_i * 256 + q * 16;
      red_add_f32(hacc + g, tg[0]);
      red_add_f32(hacc + g + 8, tg[1]);
      red_add_f32(hacc + 128 + g, tot[0]);
      red_add_f32(hacc + 128 + g + 8, tot[1]);
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

  const uint32_t n_warps = gridDim.x * kW4Warps, wi = blockIdx.x * kW4Warps + warp;
  for (int range = 0; range < 2; ++range) {
    const uint32_t pass0 = range ? (uint32_t)s_pref[n_items] : 0u;
    const uint32_t pass1 = range ? (uint32_t)s_pref[n_items + n_zc] : (uint32_t)s_pref[n_items];
    const uint32_t PP = NBLK * kKS;                  // pieces of a pass
    const uint32_t total = (pass1 - pass0) * PP, ubase = pass0 * PP;
    if (total == 0) continue;
    const uint32_t wf = ubase + w4_first(total, n_warps, wi), we = ubase + w4_first(total, n_warps, wi + 1);
    for (uint32_t pu = wf / PP; pu * PP < we; ++pu) {   // the passes (= experts) this warp touches
      const WorkItem &it = s_items[w4_find_item(s_pref, n_items + n_zc, pu)];
      const uint32_t lo = max(wf, pu * PP), hi = min(we, (pu + 1) * PP);
      if (lo < hi) {
        const uint32_t rel = lo - pu * PP;
        run(it.w + (size_t)(rel / kKS) * kUA, (int)(rel % kKS), (int)(hi - lo), pu * NBLK + rel / kKS);
      }
    }
  }
}

template <int NWD>
__global__ void __launch_bounds__(kW4Threads, 1) w4_down_half_kernel(W4Params p, int d) {
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_h = smem;
  WorkItem *s_items = reinterpret_cast<WorkItem *>(smem + kW4Warps * 2 * kW4HalfDownSlot);
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
  const uint32_t per_pass = CB * NG;
  asm volatile("griddepcontrol.wait;" ::: "memory");

  if (warp < NWD) {
    const uint32_t t0 = (uint32_t)s_pref[n_items] * per_pass;
    const uint32_t t1 = (uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * per_pass;
    const uint32_t rfirst0 = w4_first(t0, gridDim.x, blockIdx.x), rcount0 = w4_first(t0, gridDim.x, blockIdx.x + 1) - rfirst0;
    const uint32_t rfirst1 = t0 + w4_first(t1, gridDim.x, blockIdx.x);
    const uint32_t rcount1 = t0 + w4_first(t1, gridDim.x, blockIdx.x + 1) - rfirst1;
    const uint32_t my_h = smem_u32(s_h) + (uint32_t)warp * 2u * kW4HalfDownSlot;
    const uint32_t km = p.mask, kf = p.flip;

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
      const uint8_t *hsrc = p.hq + grp * 1024;
      const uint32_t dst = my_h + slot * kW4HalfDownSlot;
#pragma unroll
      for (int i = 0; i < 2; ++i)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + (i * 32 + lane) * 16u), "l"(hsrc + (i * 32 + lane) * 16)
                     : "memory");
      if (lane < 8)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 1024u + lane * 16u),
                     "l"(c.rec + sec_c + ((size_t)(c.ng * CB + c.cb) * NWD + warp) * 128u + lane * 16u)
                     : "memory");
      else if (lane < 12)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst + 1152u + (lane - 8) * 16u),
                     "l"(reinterpret_cast<const uint8_t *>(p.hs + grp * 8) + (lane - 8) * 16)
                     : "memory");
    };
    auto weights_of = [&](const Ck &c) -> const uint8_t * {
      return c.rec + sec_b + ((size_t)(c.cb * NG + c.ng) * 8u * NWD + warp) * 512u + lane * 16u;
    };

    float dtot[4][2];   // tile j: columns g, g+8 for token q
    auto zero_tot = [&]() {
#pragma unroll
      for (int j = 0; j < 4; ++j) { dtot[j][0] = dtot[j][1] = 0.f; }
    };
    float gw = 0.f;     // gate weight of token q in the current pass, 0 if the expert does not serve it
    bool served = false;
    auto begin_pass = [&](const Ck &c) {
      const WorkItem &it = s_items[c.item];
      gw = 0.f;
      served = false;
      for (int i = 0; i < it.n_tok; ++i) {   // <= 4 pairs
        int tk;
        float w;
        if (it.expert >= 0) {
          const int pr = p.perm[it.off + i];
          tk = pr / p.top_k;
          w = p.topk_w[pr];
        } else {
          tk = i;
          w = 1.f;
        }
        if (tk == q) { gw = w; served = true; }
      }
    };
    auto flush = [&](uint32_t cb) {
      if (!served) return;
      float *ya = p.y_acc + (size_t)q * d + (int)cb * 64 * NWD + warp * 64 + g;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        red_add_f32(ya + 16 * j, gw * dtot[j][0]);
        red_add_f32(ya + 16 * j + 8, gw * dtot[j][1]);
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
      const uint32_t hs_base = my_h + slot * kW4HalfDownSlot;
      int acc[4][4];
#pragma unroll
      for (int m = 0; m < 4; ++m) {   // unit pair m: neurons 32m .. 32m+31 of the group
        const uint2 hv = lds_v2(hs_base + m * 256u + g * 32u + q * 8u);   // column g: 4 neurons of u0 | of u1
        const uint32_t w0[4] = {buf[2 * m].x, buf[2 * m].y, buf[2 * m].z, buf[2 * m].w};
        const uint32_t w1[4] = {buf[2 * m + 1].x, buf[2 * m + 1].y, buf[2 * m + 1].z, buf[2 * m + 1].w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t a0 = (w0[j] & km) ^ kf, a1 = ((w0[j] >> 4) & km) ^ kf;
          const uint32_t a2 = (w1[j] & km) ^ kf, a3 = ((w1[j] >> 4) & km) ^ kf;
          if (m == 0) mma_s8_first(acc[j], a0, a1, a2, a3, hv.x, hv.y);
          else mma_s8(acc[j], a0, a1, a2, a3, hv.x, hv.y);
        }
        if (refill) {
          buf[2 * m] = ld_stream_16(refill + (size_t)(2 * m) * NWD * 512u);
          buf[2 * m + 1] = ld_stream_16(refill + (size_t)(2 * m + 1) * NWD * 512u);
        }
      }
      const uint4 sc = lds_v4(hs_base + 1024u + g * 16u);
      const uint2 tb = lds_v2(hs_base + 1152u + q * 8u);   // token q: (scale, bias)
      __syncwarp();
      const float sh = __uint_as_float(tb.x), hb = __uint_as_float(tb.y);
      const uint32_t sw[4] = {sc.x, sc.y, sc.z, sc.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        dtot[j][0] += bf16lo(sw[j]) * ((float)(acc[j][0] * 128 + acc[j][1]) * sh - hb);
        dtot[j][1] += bf16hi(sw[j]) * ((float)(acc[j][2] * 128 + acc[j][3]) * sh - hb);
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
