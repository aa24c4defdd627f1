// Steps 5+6 for int4 (group 128, bf16 scales) experts at decode-sized token counts, with the group
// dequantisation done in registers so the path stays bound by the bytes it streams.
//
// Two persistent kernels per layer, both fed by a bulk-copy (cp.async.bulk + mbarrier) shared-memory ring and
// both computing with mma.sync m16n8k16 (bf16 x bf16 -> fp32, up to 8 tokens in N):
//   q4_gateup_kernel : streams Wg_q / Wu_q rows and their scales.  A 32-bit word holds 8 codes of one row;
//                      (w >> s) & 0x000F000F puts codes i and i+4 into the two halves of a register,
//                      XOR 0x43084308 turns them into the bf16 numbers 128 + (code ^ 8), and one bf16x2
//                      subtract of 136 gives the signed codes exactly: three instructions per fragment
//                      register.  The contraction index is permuted identically for the weights and for x,
//                      so each lane's 16-byte load covers one quantisation group of its row and the scale is
//                      applied once per group to the fp32 partial sums.  h = SiLU(g) * u is written to a
//                      small global buffer in the B-fragment order of the second kernel.
//   q4_down_kernel   : streams Wd_q, which the record stores in fragment order (one coalesced 128-byte load
//                      per 16x16 tile), so no transposition is needed; groups of four CTAs split the output columns;
//                      bias and scale sd[n/128][c] are folded when a 128-neuron group ends; the gate-weighted combine is a
//                      red.global.add into the fp32 accumulator and the last CTA rounds it once to bf16.
// Zero-copy experts (records in the mapped host pool) go through the same kernels.
#pragma once
#include "common.cuh"
#include "async.cuh"

namespace ftmoe {

constexpr int kQ4Tokens = 8;        // tokens per weight pass
constexpr int kQ4Threads = 288;     // 8 consumer warps + 1 producer warp
constexpr int kQ4StagesA = 3;
constexpr int kQ4StagesB = 8;

struct Q4Params {
  const WorkItem *items;
  const int32_t *n_items;   // resident items
  const int32_t *n_zc;      // zero-copy items appended after them
  const int32_t *pref;      // exclusive prefix of the weight passes (8 tokens each) per item
  int max_items;
  const __nv_bfloat16 *x;   // [T][d]
  const int32_t *perm;
  const float *topk_w;
  uint2 *hbuf;              // [pass][16-neuron block][lane]: (h[q],h[q+4]) , (h[8+q],h[12+q])/16 of token g as fp16x2
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;
  uint32_t *done;
  uint32_t *status;
  int d, inter, top_k, T, finalize;
};

// In-register dequantisation of one 32-bit word (8 codes c_0..c_7, two's complement) into four fp16x2 fragment
// registers with five instructions (one shift, four LOP3) and no arithmetic:
//   r0 = (w      & 0x000F000F) ^ 0x64086408  ->  (1024 + u_0,    1024 + u_4)       u_i = c_i + 8 in [0, 15]
//   r1 = (w      & 0x00F000F0) ^ 0x64806480  ->  (1024 + 16 u_1, 1024 + 16 u_5)
//   r2 = (w >> 8 & 0x000F000F) ^ 0x64086408  ->  (1024 + u_2,    1024 + u_6)
//   r3 = (w >> 8 & 0x00F000F0) ^ 0x64806480  ->  (1024 + 16 u_3, 1024 + 16 u_7)
// (0x6400 is 1024.0 in fp16, whose mantissa LSB there is 1.)  The other MMA operand carries a/16 wherever the
// weight register is scaled by 16, so the products are (1032 + c) a for the even codes and (72 + c) a for the odd
// ones; the constants are removed in fp32:  sum c a = acc - 1032 * sum_even a - 72 * sum_odd a.
constexpr float kQ4BiasEven = 1032.f, kQ4BiasOdd = 72.f;
struct Q4Frag { uint32_t r0, r1, r2, r3; };
__device__ __forceinline__ Q4Frag q4_unpack(uint32_t w) {
  Q4Frag f;
  const uint32_t w8 = w >> 8;
  f.r0 = (w & 0x000F000Fu) ^ 0x64086408u;
  f.r1 = (w & 0x00F000F0u) ^ 0x64806480u;
  f.r2 = (w8 & 0x000F000Fu) ^ 0x64086408u;
  f.r3 = (w8 & 0x00F000F0u) ^ 0x64806480u;
  return f;
}
__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float bf16lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_h2(float a, float b) {
  __half2 h = __floats2half2_rn(a, b);
  return *reinterpret_cast<uint32_t *>(&h);
}
__device__ __forceinline__ float h2sum(uint32_t v) {
  const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&v));
  return f.x + f.y;
}

// token g of a pass: row of x, gate weight
__device__ __forceinline__ void q4_token(const Q4Params &p, const WorkItem &it, int pass, int g, int &tok, float &gw) {
  const int nt = min(8, it.n_tok - 8 * pass);
  tok = -1;
  gw = 0.f;
  if (g < nt) {
    if (it.expert >= 0) {
      const int pr = p.perm[it.off + 8 * pass + g];
      tok = pr / p.top_k;
      gw = p.topk_w[pr];
    } else {
      tok = 8 * pass + g;
      gw = 1.f;
    }
  }
}

inline size_t q4_gateup_stage_bytes(int d) { return (size_t)16 * (d / 2 + 64) + d / 4; }
inline size_t q4_gateup_smem_bytes(int d) {
  return kQ4StagesA * q4_gateup_stage_bytes(d) + 8 * 2 * 16 * 8 * 4 + (2 * kMaxExperts + 2) * 4 + 2 * kQ4StagesA * 8 + 16;
}
inline size_t q4_down_smem_bytes(int d) {
  return (size_t)kQ4StagesB * 2 * d + (2 * kMaxExperts + 2) * 4 + 2 * kQ4StagesB * 8 + 16;
}

// SB = 128-wide groups of the contraction index per warp; KW = d / 128 / SB warps take part in the MMAs.
template <int SB>
__global__ void __launch_bounds__(kQ4Threads, 1) q4_gateup_kernel(Q4Params p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = p.d;
  const uint32_t row_bytes = d / 2;
  const uint32_t stride = row_bytes + 64;          // = 64 mod 128: conflict-free 16-byte fragment loads
  const uint32_t scale_row = (d / kGroup) * 2;     // bytes of one row of scales
  const uint32_t stage_bytes = 16 * stride + 16 * scale_row;
  unsigned char *sp = smem + (size_t)kQ4StagesA * stage_bytes;
  float *s_red = reinterpret_cast<float *>(sp); sp += 8 * 2 * 16 * 8 * 4;
  int32_t *s_pref = reinterpret_cast<int32_t *>(sp); sp += (2 * kMaxExperts + 2) * 4;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(sp); sp += 2 * kQ4StagesA * 8;
  volatile int *s_abort = reinterpret_cast<volatile int *>(sp);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  const int NBLK = p.inter / 16;
  const int KW = d / kGroup / SB;
  const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kQ4StagesA + s); };
  if (tid == 0) {
    for (int s = 0; s < kQ4StagesA; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 8); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i <= p.max_items; i += blockDim.x) s_pref[i] = p.pref[i];
  __syncthreads();
  const long long total_res = (long long)s_pref[n_items] * NBLK;
  const long long total_all = (long long)s_pref[n_items + n_zc] * NBLK;
  const size_t mat_bytes = (size_t)row_bytes * p.inter;
  const size_t smat_bytes = (size_t)scale_row * p.inter;
  int item = 0;
  uint32_t tile = 0;

  for (int range = 0; range < 2; ++range) {
    const long long r0 = range ? total_res : 0, rn = range ? total_all - total_res : total_res;
    long long u = r0 + rn * blockIdx.x / gridDim.x;
    const long long u1 = r0 + rn * (blockIdx.x + 1) / gridDim.x;
    while (u < u1) {
      const long long pu = u / NBLK;
      while (s_pref[item + 1] <= pu) ++item;
      const int pass = (int)(pu - s_pref[item]);
      const int b_begin = (int)(u - pu * NBLK);
      const long long left = u1 - u;
      const int b_end = (left < (long long)(NBLK - b_begin)) ? b_begin + (int)left : NBLK;
      const WorkItem it = p.items[item];
      if (warp == 8) {
        // ---------------- producer: lanes 0..15 copy one row each, lane 16 the block's scales ----------------
        for (int b = b_begin; b < b_end; ++b) {
          for (int which = 0; which < 2; ++which, ++tile) {
            const int s = tile % kQ4StagesA;
            const uint32_t ph = (tile / kQ4StagesA) & 1u;
            if (lane == 0) {
              mbar_wait(empty_bar(s), ph ^ 1u, s_abort, p.status);
              mbar_expect_tx(full_bar(s), 16 * row_bytes + 16 * scale_row);
            }
            __syncwarp();
            const bool withhold = (g_debug_withhold & kWithholdQ4) && tile == 0;   // test hook
            if (!*s_abort && !withhold) {
              const uint32_t dst = smem_base + s * stage_bytes;
              if (lane < 16)
                bulk_g2s(dst + lane * stride, it.w + which * mat_bytes + (size_t)(b * 16 + lane) * row_bytes, row_bytes,
                         full_bar(s));
              else if (lane == 16)
                bulk_g2s(dst + 16 * stride, it.w + 3 * mat_bytes + which * smat_bytes + (size_t)b * 16 * scale_row,
                         16 * scale_row, full_bar(s));
            }
          }
        }
      } else {
        // ---------------- consumers ----------------
        const int g = lane >> 2, q = lane & 3;
        int tok_g;
        float gw_g;
        q4_token(p, it, pass, g, tok_g, gw_g);
        // x fragments: lane (g, q) holds token g, contraction indices [128*(warp*SB+sb) + 32q, +32), each run of 8
        // rearranged as the pairs (0,4) (1,5) (2,6) (3,7) the dequantiser produces
        uint32_t xf[SB][4][4];
        float xs[SB][2];   // bias term of the group's dot products (1032 * even-code x sum + 72 * odd-code x sum), tokens 2q, 2q+1
#pragma unroll
        for (int sb = 0; sb < SB; ++sb) {
          float part = 0.f;
#pragma unroll
          for (int wi = 0; wi < 4; ++wi) {
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (tok_g >= 0 && warp < KW)
              v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok_g * d + (warp * SB + sb) * kGroup + 32 * q + 8 * wi);
            // e0..e7 = the 8 consecutive x values of this word; fp16 operands (e0,e4) (e1,e5)/16 (e2,e6) (e3,e7)/16
            xf[sb][wi][0] = pack_h2(bf16lo(v.x), bf16lo(v.z));
            xf[sb][wi][1] = pack_h2(bf16hi(v.x) * 0.0625f, bf16hi(v.z) * 0.0625f);
            xf[sb][wi][2] = pack_h2(bf16lo(v.y), bf16lo(v.w));
            xf[sb][wi][3] = pack_h2(bf16hi(v.y) * 0.0625f, bf16hi(v.w) * 0.0625f);
            part += kQ4BiasEven * (h2sum(xf[sb][wi][0]) + h2sum(xf[sb][wi][2])) +
                    kQ4BiasOdd * 16.f * (h2sum(xf[sb][wi][1]) + h2sum(xf[sb][wi][3]));
          }
          part += __shfl_xor_sync(0xffffffffu, part, 1);
          part += __shfl_xor_sync(0xffffffffu, part, 2);    // all four lanes of token g hold its group's bias term
          xs[sb][0] = __shfl_sync(0xffffffffu, part, (2 * q) * 4);
          xs[sb][1] = __shfl_sync(0xffffffffu, part, (2 * q + 1) * 4);
        }
        for (int b = b_begin; b < b_end; ++b) {
          float cgu[2][4];
#pragma unroll
          for (int which = 0; which < 2; ++which, ++tile) {
            const int s = tile % kQ4StagesA;
            const uint32_t ph = (tile / kQ4StagesA) & 1u;
            cgu[which][0] = cgu[which][1] = cgu[which][2] = cgu[which][3] = 0.f;
            const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
            if (ok && warp < KW) {
              const unsigned char *tile_ptr = smem + (size_t)s * stage_bytes;   // plain loads: freely schedulable
              const __nv_bfloat16 *sc = reinterpret_cast<const __nv_bfloat16 *>(smem + (size_t)s * stage_bytes + 16 * stride);
#pragma unroll
              for (int sb = 0; sb < SB; ++sb) {
                const int grp = warp * SB + sb;
                const uint4 lo = *reinterpret_cast<const uint4 *>(tile_ptr + g * stride + grp * 64 + 16 * q);
                const uint4 hi = *reinterpret_cast<const uint4 *>(tile_ptr + (g + 8) * stride + grp * 64 + 16 * q);
                const uint32_t wl[4] = {lo.x, lo.y, lo.z, lo.w}, wh[4] = {hi.x, hi.y, hi.z, hi.w};
                // two accumulators so that consecutive MMAs do not wait for each other
                float acc[4] = {0.f, 0.f, 0.f, 0.f}, acc2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int wi = 0; wi < 4; ++wi) {
                  const Q4Frag fl = q4_unpack(wl[wi]), fh = q4_unpack(wh[wi]);
                  mma_f16(acc, fl.r0, fh.r0, fl.r1, fh.r1, xf[sb][wi][0], xf[sb][wi][1]);    // codes (0,4) and (1,5)
                  mma_f16(acc2, fl.r2, fh.r2, fl.r3, fh.r3, xf[sb][wi][2], xf[sb][wi][3]);   // codes (2,6) and (3,7)
                }
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[i] += acc2[i];
                const float s_lo = __bfloat162float(sc[g * (d / kGroup) + grp]);
                const float s_hi = __bfloat162float(sc[(g + 8) * (d / kGroup) + grp]);
                cgu[which][0] = fmaf(s_lo, acc[0] - xs[sb][0], cgu[which][0]);
                cgu[which][1] = fmaf(s_lo, acc[1] - xs[sb][1], cgu[which][1]);
                cgu[which][2] = fmaf(s_hi, acc[2] - xs[sb][0], cgu[which][2]);
                cgu[which][3] = fmaf(s_hi, acc[3] - xs[sb][1], cgu[which][3]);
              }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty_bar(s));
          }
          // cross-warp reduction, SwiGLU, h in the B-fragment order of the down kernel
          {
            float *r0 = s_red + ((warp * 2 + 0) * 16) * 8;
            float *r1 = s_red + ((warp * 2 + 1) * 16) * 8;
            *reinterpret_cast<float2 *>(r0 + g * 8 + 2 * q) = make_float2(cgu[0][0], cgu[0][1]);
            *reinterpret_cast<float2 *>(r0 + (g + 8) * 8 + 2 * q) = make_float2(cgu[0][2], cgu[0][3]);
            *reinterpret_cast<float2 *>(r1 + g * 8 + 2 * q) = make_float2(cgu[1][0], cgu[1][1]);
            *reinterpret_cast<float2 *>(r1 + (g + 8) * 8 + 2 * q) = make_float2(cgu[1][2], cgu[1][3]);
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          if (tid < 128) {
            const int n = tid >> 3, t = tid & 7;
            float a = 0.f, c = 0.f;
#pragma unroll
            for (int w = 0; w < 8; ++w) {
              a += s_red[((w * 2 + 0) * 16 + n) * 8 + t];
              c += s_red[((w * 2 + 1) * 16 + n) * 8 + t];
            }
            const float h = a / (1.f + __expf(-a)) * c;
            // neuron n = 4*slot + qq of the block goes to lane 4*t + qq, half-word `slot` of its two words
            // (fp16; the second word, neurons 8..15, is stored divided by 16 to match the x16 weight registers)
            const int qq = n & 3, slot = n >> 2;
            __half *dst = reinterpret_cast<__half *>(p.hbuf + ((size_t)pu * NBLK + b) * 32 + 4 * t + qq);
            dst[slot] = __float2half_rn(slot >= 2 ? h * 0.0625f : h);
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
        }
      }
      u += (b_end - b_begin);
    }
  }
  abort_drain(s_abort);
}

// CTW = 16-column tiles per warp; four CTAs (blockIdx.x & 3) share a range of blocks and split the columns in
// quarters, which leaves registers for a scaled total next to the per-group accumulators.
template <int CTW>
__global__ void __launch_bounds__(kQ4Threads, 1) q4_down_kernel(Q4Params p) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = p.d;
  const uint32_t stage_bytes = 2u * d;      // (d/64) tiles x 128 bytes: a quarter of one block's columns
  unsigned char *sp = smem + (size_t)kQ4StagesB * stage_bytes;
  int32_t *s_pref = reinterpret_cast<int32_t *>(sp); sp += (2 * kMaxExperts + 2) * 4;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(sp); sp += 2 * kQ4StagesB * 8;
  volatile int *s_abort = reinterpret_cast<volatile int *>(sp);
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  const int NBLK = p.inter / 16;
  const int slice = blockIdx.x >> 2, hf = blockIdx.x & 3, n_slices = gridDim.x >> 2;   // hf: column quarter
  const uint32_t smem_base = smem_u32(smem), bar_base = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kQ4StagesB + s); };
  if (tid == 0) {
    for (int s = 0; s < kQ4StagesB; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 8); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i <= p.max_items; i += blockDim.x) s_pref[i] = p.pref[i];
  __syncthreads();
  const long long total_res = (long long)s_pref[n_items] * NBLK;
  const long long total_all = (long long)s_pref[n_items + n_zc] * NBLK;
  const size_t mat_bytes = (size_t)(d / 2) * p.inter;
  const size_t smat_bytes = (size_t)(d / kGroup) * 2 * p.inter;
  int item = 0;
  uint32_t tile = 0;

  for (int range = 0; range < 2; ++range) {
    const long long r0 = range ? total_res : 0, rn = range ? total_all - total_res : total_res;
    long long u = r0 + rn * slice / n_slices;
    const long long u1 = r0 + rn * (slice + 1) / n_slices;
    while (u < u1) {
      const long long pu = u / NBLK;
      while (s_pref[item + 1] <= pu) ++item;
      const int pass = (int)(pu - s_pref[item]);
      const int b_begin = (int)(u - pu * NBLK);
      const long long left = u1 - u;
      const int b_end = (left < (long long)(NBLK - b_begin)) ? b_begin + (int)left : NBLK;
      const WorkItem it = p.items[item];
      const uint8_t *wd = it.w + 2 * mat_bytes;
      if (warp == 8) {
        if (lane == 0) {
          for (int b = b_begin; b < b_end; ++b, ++tile) {
            const int s = tile % kQ4StagesB;
            const uint32_t ph = (tile / kQ4StagesB) & 1u;
            mbar_wait(empty_bar(s), ph ^ 1u, s_abort, p.status);
            if (*s_abort) break;
            mbar_expect_tx(full_bar(s), stage_bytes);
            bulk_g2s(smem_base + s * stage_bytes, wd + ((size_t)b * (d / 16) + (size_t)hf * (d / 64)) * 128, stage_bytes,
                     full_bar(s));
          }
        }
      } else {
        const int g = lane >> 2, q = lane & 3;
        int tok_g;
        float gw_g;
        q4_token(p, it, pass, g, tok_g, gw_g);
        const __nv_bfloat16 *sd = reinterpret_cast<const __nv_bfloat16 *>(it.w + 3 * mat_bytes + 2 * smat_bytes);
        const int col0 = hf * (d / 4) + warp * CTW * 16;   // first column of this warp
        // dacc: sum_n (bias + code) h over the blocks of the current 128-neuron group; dtot: the scaled total.
        // Within one group the scale is a per-column constant, so bias and scale are folded into dtot when the
        // group (or the CTA's range) ends:  dtot += scale[c] * (dacc - bias term of the h values).
        float dacc[CTW][4], dtot[CTW][4];
        float hsum = 0.f;   // bias term so far for token g: 1032 * sum of h over neurons 0..7 + 72 * sum over 8..15 of each block
#pragma unroll
        for (int c = 0; c < CTW; ++c) {
          dacc[c][0] = dacc[c][1] = dacc[c][2] = dacc[c][3] = 0.f;
          dtot[c][0] = dtot[c][1] = dtot[c][2] = dtot[c][3] = 0.f;
        }
        const int tok_a = __shfl_sync(0xffffffffu, tok_g, (2 * q) * 4);
        const int tok_b = __shfl_sync(0xffffffffu, tok_g, (2 * q + 1) * 4);
        const float gw_a = __shfl_sync(0xffffffffu, gw_g, (2 * q) * 4);
        const float gw_b = __shfl_sync(0xffffffffu, gw_g, (2 * q + 1) * 4);
        uint32_t sdr[CTW];   // scales of the current group: (column g, column g+8) of every tile, two bf16
        auto load_scales = [&](int grp) {
#pragma unroll
          for (int c = 0; c < CTW; ++c) {
            const __nv_bfloat16 *sp2 = sd + (size_t)grp * d + col0 + 16 * c + g;
            sdr[c] = (uint32_t)__bfloat16_as_ushort(sp2[0]) | ((uint32_t)__bfloat16_as_ushort(sp2[8]) << 16);
          }
        };
        auto fold = [&]() {
          float hs = hsum;
          hs += __shfl_xor_sync(0xffffffffu, hs, 1);
          hs += __shfl_xor_sync(0xffffffffu, hs, 2);
          const float ha = __shfl_sync(0xffffffffu, hs, (2 * q) * 4);
          const float hb2 = __shfl_sync(0xffffffffu, hs, (2 * q + 1) * 4);
#pragma unroll
          for (int c = 0; c < CTW; ++c) {
            const float s_lo = bf16lo(sdr[c]), s_hi = bf16hi(sdr[c]);
            dtot[c][0] = fmaf(s_lo, dacc[c][0] - ha, dtot[c][0]);
            dtot[c][1] = fmaf(s_lo, dacc[c][1] - hb2, dtot[c][1]);
            dtot[c][2] = fmaf(s_hi, dacc[c][2] - ha, dtot[c][2]);
            dtot[c][3] = fmaf(s_hi, dacc[c][3] - hb2, dtot[c][3]);
            dacc[c][0] = dacc[c][1] = dacc[c][2] = dacc[c][3] = 0.f;
          }
          hsum = 0.f;
        };
        int cur_grp = (b_begin * 16) / kGroup;
        load_scales(cur_grp);
        // h fragments are fetched two blocks ahead (they sit in L2; a block is consumed faster than one L2 round trip)
        const uint2 *hsrc = p.hbuf + (size_t)pu * NBLK * 32 + lane;
        uint2 hb0 = hsrc[(size_t)b_begin * 32];
        uint2 hb1 = (b_begin + 1 < b_end) ? hsrc[(size_t)(b_begin + 1) * 32] : make_uint2(0u, 0u);
        for (int b = b_begin; b < b_end; ++b, ++tile) {
          const uint2 hb = hb0;
          hb0 = hb1;
          if (b + 2 < b_end) hb1 = hsrc[(size_t)(b + 2) * 32];
          const int grp = (b * 16) / kGroup;
          if (grp != cur_grp) {
            fold();
            cur_grp = grp;
            load_scales(cur_grp);
          }
          const int s = tile % kQ4StagesB;
          const uint32_t ph = (tile / kQ4StagesB) & 1u;
          const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
          if (ok) {
            hsum += kQ4BiasEven * h2sum(hb.x) + kQ4BiasOdd * 16.f * h2sum(hb.y);
            // plain loads (not volatile asm) so that the compiler can issue all of a block's loads up front
            const uint32_t *wsrc = reinterpret_cast<const uint32_t *>(smem + (size_t)s * stage_bytes) + (warp * CTW) * 32 + lane;
            uint32_t wv[CTW];
#pragma unroll
            for (int c = 0; c < CTW; ++c) wv[c] = wsrc[c * 32];
#pragma unroll
            for (int c = 0; c < CTW; ++c) {
              const uint32_t w = wv[c];
              const Q4Frag f = q4_unpack(w);   // r0: column g, neurons (q,q+4); r1: column g, (8+q,12+q) x16; r2,r3: column g+8
              mma_f16(dacc[c], f.r0, f.r2, f.r1, f.r3, hb.x, hb.y);
            }
          }
          __syncwarp();
          if (lane == 0) mbar_arrive(empty_bar(s));
        }
        fold();
        // gate-weighted combine
#pragma unroll
        for (int c = 0; c < CTW; ++c) {
          const int col = col0 + 16 * c + g;
          if (tok_a >= 0) {
            atomicAdd(p.y_acc + (size_t)tok_a * d + col, gw_a * dtot[c][0]);
            atomicAdd(p.y_acc + (size_t)tok_a * d + col + 8, gw_a * dtot[c][2]);
          }
          if (tok_b >= 0) {
            atomicAdd(p.y_acc + (size_t)tok_b * d + col, gw_b * dtot[c][1]);
            atomicAdd(p.y_acc + (size_t)tok_b * d + col + 8, gw_b * dtot[c][3]);
          }
        }
      }
      u += (b_end - b_begin);
    }
  }
  abort_drain(s_abort);

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
  const long long n4 = (long long)p.T * d / 4;
  // eight independent L2 loads in flight per thread: the round trips overlap instead of adding up
  for (long long i0 = tid; i0 < n4; i0 += 8LL * blockDim.x) {
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long i = i0 + (long long)j * blockDim.x;
      v[j] = (i < n4) ? __ldcg(reinterpret_cast<const float4 *>(p.y_acc) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long i = i0 + (long long)j * blockDim.x;
      if (i < n4) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[j].x, v[j].y), b = __floats2bfloat162_rn(v[j].z, v[j].w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t *>(&a);
        o.y = *reinterpret_cast<uint32_t *>(&b);
        reinterpret_cast<uint2 *>(p.y)[i] = o;
        reinterpret_cast<float4 *>(p.y_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
  if (tid == 0) *p.done = 0u;
}

}  // namespace ftmoe
