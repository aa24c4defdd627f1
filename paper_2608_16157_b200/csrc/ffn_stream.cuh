// Steps 5+6 for decode-sized token counts: a streaming SwiGLU expert FFN.  Every routed expert's
// record is read exactly once per pass of up to TC tokens with 16-byte (bf16) or 8-byte (int4)
// coalesced loads, from an HBM slot or, for the zero-copy set, from the mapped host pool.  All three
// matrices are stored one row per intermediate neuron, so a CTA that owns a block of neurons
// computes gate and up for them, applies SiLU * up * gate-weight, and immediately adds their
// down-projection rows into per-thread fp32 accumulators; the gate-weighted combine is a
// red.global.add into an fp32 [T][d] accumulator that a finalize kernel rounds once to bf16.
#pragma once
#include "common.cuh"

namespace ftmoe {

struct FfnParams {
  const WorkItem *items;
  const int32_t *n_items;      // device-resident valid count
  const __nv_bfloat16 *x;      // [T][d]
  const int32_t *perm;         // [P]
  const float *topk_w;         // [P]
  float *y_acc;                // [T][d] fp32, zero on entry of the first kernel of a forward
  int d, inter, top_k;
};

template <int WD>
struct WTraits;
template <>
struct WTraits<0> {  // bf16
  static constexpr int EPL = 8;    // elements per load
  static constexpr int VEC = 16;   // bytes per load
};
template <>
struct WTraits<1> {  // int4, group 128
  static constexpr int EPL = 16;
  static constexpr int VEC = 8;
};

template <int WD>
__device__ __forceinline__ void load_w(const uint8_t *row, int ct, float (&out)[WTraits<WD>::EPL]) {
  if constexpr (WD == 0) {
    const uint4 v = ld_stream_16(row + (size_t)ct * 16);
    const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(r[i] << 16);
      out[2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
    }
  } else {
    const uint2 v = ld_stream_8(row + (size_t)ct * 8);
    const uint32_t r[2] = {v.x, v.y};
#pragma unroll
    for (int i = 0; i < 2; ++i)
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int q = (int)((r[i] >> (4 * j)) & 0xFu);
        out[8 * i + j] = (float)((q ^ 8) - 8);   // two's-complement nibble
      }
  }
}

template <int WD, int TC, int NR>
__global__ void __launch_bounds__(WD == 0 ? 256 : 512) ffn_stream_kernel(FfnParams p) {
  using WT = WTraits<WD>;
  constexpr int EPL = WT::EPL;
  const int tid = threadIdx.x, lane = tid & 31;
  const int CT = p.d / EPL;                 // threads across one row
  const int G = blockDim.x / CT;            // row groups
  const int g = tid / CT, ct = tid - g * CT;
  const int nwrg = CT >> 5;
  const int col0 = ct * EPL;
  const int n_items = *p.n_items;
  const int rows_per_unit = NR * G;
  const int NBLK = p.inter / rows_per_unit;
  const long long total = (long long)n_items * NBLK;
  long long u = total * blockIdx.x / gridDim.x;
  const long long u1 = total * (blockIdx.x + 1) / gridDim.x;
  const size_t row_bytes = (size_t)p.d * (WD == 0 ? 2 : 1) / (WD == 0 ? 1 : 2);
  const size_t mat_bytes = row_bytes * p.inter;

  __shared__ int s_tok[TC];
  __shared__ float s_gw[TC];
  __shared__ float s_red[16 * NR * 2 * TC];   // [warp][r][2][t]
  __shared__ float s_h[16 * NR * TC];         // [g][r][t]   (G <= 16)

  while (u < u1) {
    const int item = (int)(u / NBLK);
    const int b_begin = (int)(u - (long long)item * NBLK);
    const long long left = u1 - u;
    const int b_end = (left < (long long)(NBLK - b_begin)) ? b_begin + (int)left : NBLK;
    const WorkItem it = p.items[item];
    const uint8_t *Wg = it.w, *Wu = it.w + mat_bytes, *Wd = it.w + 2 * mat_bytes;
    const __nv_bfloat16 *sg = nullptr, *su = nullptr, *sd = nullptr;
    if constexpr (WD == 1) {
      sg = reinterpret_cast<const __nv_bfloat16 *>(it.w + 3 * mat_bytes);
      su = sg + (size_t)p.inter * (p.d / kGroup);
      sd = su + (size_t)p.inter * (p.d / kGroup);
    }
    for (int t0 = 0; t0 < it.n_tok; t0 += TC) {
      const int nt = min(TC, it.n_tok - t0);
      __syncthreads();
      if (tid < TC) {
        int tok = 0;
        float gw = 0.f;
        if (tid < nt) {
          if (it.expert >= 0) {
            const int pr = p.perm[it.off + t0 + tid];
            tok = pr / p.top_k;
            gw = p.topk_w[pr];
          } else {
            tok = t0 + tid;
            gw = 1.f;
          }
        }
        s_tok[tid] = tok;
        s_gw[tid] = gw;
      }
      __syncthreads();
      float xr[TC][EPL];
      float acc[TC][EPL];
#pragma unroll
      for (int t = 0; t < TC; ++t) {
#pragma unroll
        for (int j = 0; j < EPL; ++j) { xr[t][j] = 0.f; acc[t][j] = 0.f; }
        if (t < nt) {
          const uint4 *xp = reinterpret_cast<const uint4 *>(p.x + (size_t)s_tok[t] * p.d + col0);
#pragma unroll
          for (int v = 0; v < EPL / 8; ++v) {
            const uint4 xv = xp[v];
            const uint32_t r[4] = {xv.x, xv.y, xv.z, xv.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              xr[t][8 * v + 2 * i] = __uint_as_float(r[i] << 16);
              xr[t][8 * v + 2 * i + 1] = __uint_as_float(r[i] & 0xffff0000u);
            }
          }
        }
      }
      for (int b = b_begin; b < b_end; ++b) {
        const int n_base = b * rows_per_unit + g * NR;
        float pg[NR][TC], pu[NR][TC];
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          float wg[EPL], wu[EPL];
          load_w<WD>(Wg + (size_t)(n_base + r) * row_bytes, ct, wg);
          load_w<WD>(Wu + (size_t)(n_base + r) * row_bytes, ct, wu);
          float scg = 1.f, scu = 1.f;
          if constexpr (WD == 1) {
            const size_t si = (size_t)(n_base + r) * (p.d / kGroup) + col0 / kGroup;
            scg = __bfloat162float(sg[si]);
            scu = __bfloat162float(su[si]);
          }
#pragma unroll
          for (int t = 0; t < TC; ++t) {
            float a = 0.f, c = 0.f;
#pragma unroll
            for (int j = 0; j < EPL; ++j) {
              a = fmaf(wg[j], xr[t][j], a);
              c = fmaf(wu[j], xr[t][j], c);
            }
            pg[r][t] = a * scg;
            pu[r][t] = c * scu;
          }
        }
        // reduce over the CT threads of the row group: warp shuffles, then across warps via smem
#pragma unroll
        for (int r = 0; r < NR; ++r)
#pragma unroll
          for (int t = 0; t < TC; ++t) {
            const float a = warp_sum(pg[r][t]);
            const float c = warp_sum(pu[r][t]);
            if (lane == 0) {
              const int wglob = tid >> 5;
              s_red[((wglob * NR + r) * 2 + 0) * TC + t] = a;
              s_red[((wglob * NR + r) * 2 + 1) * TC + t] = c;
            }
          }
        __syncthreads();
        if (ct < NR * TC) {
          const int r = ct / TC, t = ct - r * TC;
          float a = 0.f, c = 0.f;
          for (int w = 0; w < nwrg; ++w) {
            const int wglob = g * nwrg + w;
            a += s_red[((wglob * NR + r) * 2 + 0) * TC + t];
            c += s_red[((wglob * NR + r) * 2 + 1) * TC + t];
          }
          const float h = a / (1.f + __expf(-a)) * c * s_gw[t];
          s_h[(g * NR + r) * TC + t] = h;
        }
        __syncthreads();
#pragma unroll
        for (int r = 0; r < NR; ++r) {
          float wd[EPL];
          load_w<WD>(Wd + (size_t)(n_base + r) * row_bytes, ct, wd);
          if constexpr (WD == 1) {
            const __nv_bfloat16 *sp = sd + (size_t)((n_base + r) / kGroup) * p.d + col0;
#pragma unroll
            for (int j = 0; j < EPL; ++j) wd[j] *= __bfloat162float(sp[j]);
          }
#pragma unroll
          for (int t = 0; t < TC; ++t) {
            const float h = s_h[(g * NR + r) * TC + t];
#pragma unroll
            for (int j = 0; j < EPL; ++j) acc[t][j] = fmaf(h, wd[j], acc[t][j]);
          }
        }
      }
      // gate-weighted combine: add this CTA's partial into the fp32 accumulator
#pragma unroll
      for (int t = 0; t < TC; ++t) {
        if (t < nt) {
          float *dst = p.y_acc + (size_t)s_tok[t] * p.d + col0;
#pragma unroll
          for (int j = 0; j < EPL; j += 4) {
            asm volatile("red.global.add.v4.f32 [%0], {%1,%2,%3,%4};" ::"l"(dst + j), "f"(acc[t][j]),
                         "f"(acc[t][j + 1]), "f"(acc[t][j + 2]), "f"(acc[t][j + 3])
                         : "memory");
          }
        }
      }
    }
    u += (b_end - b_begin);
  }
}

// y = bf16(y_acc); y_acc = 0 for the next forward.
__global__ void finalize_kernel(float *y_acc, __nv_bfloat16 *y, long long n4) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n4) return;
  float4 v = reinterpret_cast<float4 *>(y_acc)[i];
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 o;
  o.x = *reinterpret_cast<uint32_t *>(&a);
  o.y = *reinterpret_cast<uint32_t *>(&b);
  reinterpret_cast<uint2 *>(y)[i] = o;
  reinterpret_cast<float4 *>(y_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
}

}  // namespace ftmoe
