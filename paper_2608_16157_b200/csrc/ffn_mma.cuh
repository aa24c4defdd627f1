// Steps 5+6 for resident bf16 experts at decode-sized token counts: an HBM-streaming SwiGLU FFN.
//
// One persistent CTA per SM.  A producer warp streams the expert records through a 3-stage shared
// memory ring with bulk asynchronous copies (cp.async.bulk + mbarrier complete_tx), one 16-neuron
// tile of one matrix per stage, so ~190 KB per SM are in flight and HBM never waits for arithmetic.
// Eight consumer warps turn each tile into tensor-core MMAs (mma.sync m16n8k16, bf16 x bf16 -> fp32)
// with up to 8 tokens in the N dimension, so the arithmetic cost does not grow with the token count:
//   gate/up tile: warp w owns the k-slice [w*d/8, (w+1)*d/8); partial [16 neurons x 8 tokens] sums are
//                 reduced across warps through shared memory, then h = SiLU(g) * u.
//   down tile   : warp w owns the output columns [w*d/8, (w+1)*d/8); A = Wd^T through
//                 ldmatrix.trans, B = h; fp32 accumulators persist across the CTA's neuron range.
// The gate-weighted combine is a red.global.add into the fp32 [T][d] accumulator; the last CTA to
// finish rounds it once to bf16 and clears it.  Every mbarrier wait is bounded: on expiry the CTA
// latches a timeout status, stops waiting and runs to completion.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace ftmoe {

constexpr int kMmaStages = 6;     // one per (matrix, row half): a block of 16 neurons is 6 half tiles
constexpr int kMmaTileRows = 16;
constexpr int kMmaConsumers = 256;
constexpr int kMmaThreads = kMmaConsumers + 32;
constexpr int kMmaTokens = 8;  // tokens per weight pass

struct FfnMmaParams {
  const WorkItem *items;
  const int32_t *n_items;   // resident items (records in HBM slots): [hits][shared expert][fills]
  const int32_t *n_hit;     // how many of them lead the list and do not depend on this step's fills
  int part;                 // 0: everything; 1: hits + zero-copy items; 2: fills only
  const int32_t *n_zc;      // zero-copy items appended after them (records in the mapped host pool)
  const int32_t *pref;      // [n_items+1] exclusive prefix of the weight passes per item (from the plan)
  const __nv_bfloat16 *x;   // [T][d]
  const int32_t *perm;
  const float *topk_w;
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;         // [T][d], written by the last CTA when finalize != 0
  uint32_t *done;           // CTA completion counter, zero between launches
  uint32_t *status;
  int d, inter, top_k, T, finalize;
  int max_items;            // capacity of items / pref (entries beyond *n_items are ignored)
  long long *trace;         // optional [gridDim.x][4]: start and end of the CTA's streaming (global timer, ns), blocks
                            // streamed, segments (the finalizing CTA stores minus its finish time there); or nullptr
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait; returns false (after latching the abort flag) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag, uint32_t *status) {
  if (*abort_flag) return false;
  for (uint32_t i = 0; i < (1u << 22); ++i) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((i & 1023u) == 1023u && *abort_flag) return false;
  }
  *abort_flag = 1;
  atomicOr(status, kStatTimeout);
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 lds_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], uint32_t addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(addr));
}

// Dynamic shared memory layout (bytes): [stages][16 rows x (2d+64)] | red [8][2][16][8] f32 | hs [8][16] bf16
// | pref [2*kMaxExperts+2] i32 | mbarriers full[], empty[] | abort flag.
template <int KB>  // KB = d / 256: 32-wide k-blocks per warp in the gate/up phase
__global__ void __launch_bounds__(kMmaThreads, 1) ffn_mma_kernel(FfnMmaParams p) {
  constexpr int CTW = 2 * KB;  // 16-column tiles per warp in the down phase
  extern __shared__ __align__(128) unsigned char smem[];
  const int d = p.d;
  const uint32_t row_bytes = 2u * d;
  const uint32_t half_bytes = row_bytes / 2;   // a stage holds the lower or upper half of 16 rows
  const uint32_t stride_gu = half_bytes + 64;  // = 64 mod 128: conflict-free 16-byte fragment loads
  const uint32_t stride_d = half_bytes + 16;   // = 16 mod 128: conflict-free ldmatrix rows
  const uint32_t stage_bytes = kMmaTileRows * stride_gu;
  unsigned char *sp = smem + (size_t)kMmaStages * stage_bytes;
  float *s_red = reinterpret_cast<float *>(sp); sp += 8 * 2 * 16 * 8 * 4;
  __nv_bfloat16 *s_h = reinterpret_cast<__nv_bfloat16 *>(sp); sp += 8 * 16 * 2;
  int32_t *s_pref = reinterpret_cast<int32_t *>(sp); sp += (2 * kMaxExperts + 2) * 4;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(sp); sp += 2 * kMmaStages * 8;
  volatile int *s_abort = reinterpret_cast<volatile int *>(sp);
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  long long t_start;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_start));
  int trace_blocks = 0, trace_segments = 0;
  const int n_items = *p.n_items;
  const int NBLK = p.inter / kMmaTileRows;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kMmaStages + s); };

  if (tid == 0) {
    for (int s = 0; s < kMmaStages; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 4);   // the four warps that own this half
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // prefix sums of the weight passes per item (8 tokens per pass) and the record pointers, written by the
  // plan kernel; loaded up to the lists' capacity so that these loads do not wait for the item count
  const int n_zc = *p.n_zc;
  for (int i = tid; i <= p.max_items; i += blockDim.x) s_pref[i] = p.pref[i];
  __syncthreads();
  // two work ranges, each split evenly over the CTAs: HBM-resident blocks, then host-resident blocks (the
  // latter are bound by the host link, so every CTA takes an equal share of them).  `part` restricts the launch
  // to the items that do not depend on the fills (plus the zero-copy items) or to the filled items.
  const int n_hit = (p.part == 0) ? 0 : *p.n_hit;
  const int a0 = (p.part == 2) ? n_hit : 0, a1 = (p.part == 1) ? n_hit : n_items;
  const long long first_res = (long long)s_pref[a0] * NBLK;
  const long long total_res = (long long)s_pref[a1] * NBLK;
  const long long zc_begin = (long long)s_pref[n_items] * NBLK;
  const long long total_all = (p.part == 2) ? zc_begin : (long long)s_pref[n_items + n_zc] * NBLK;
  int item = 0;
  uint32_t tile = 0;  // 16-neuron blocks consumed / produced so far by this CTA

  if (warp == 8) {
    // ------------------------------ producer ------------------------------
    // lane 0 waits for the stage and posts the byte count; lanes 0..15 then issue one row copy each, so the
    // issue rate of a single thread never limits the stream
    for (int range = 0; range < 2; ++range) {
    const long long r0 = range ? zc_begin : first_res, rn = range ? total_all - zc_begin : total_res - first_res;
    long long u = r0 + rn * blockIdx.x / gridDim.x;
    const long long u1 = r0 + rn * (blockIdx.x + 1) / gridDim.x;
    while (u < u1) {
      const long long pu = u / NBLK;
      while (s_pref[item + 1] <= pu) ++item;
      const int b_begin = (int)(u - pu * NBLK);
      const long long left = u1 - u;
      const int b_end = (left < (long long)(NBLK - b_begin)) ? b_begin + (int)left : NBLK;
      const uint8_t *rec = p.items[item].w;
      const size_t mat_bytes = (size_t)row_bytes * p.inter;
      trace_blocks += b_end - b_begin;
      ++trace_segments;
      for (int b = b_begin; b < b_end; ++b, ++tile) {
        const uint32_t ph = tile & 1u;     // `tile` counts this CTA's blocks; stage = 2*matrix + half
#pragma unroll 1
        for (int s = 0; s < kMmaStages; ++s) {
          const int which = s >> 1, half = s & 1;
          if (lane == 0) {
            mbar_wait(empty_bar(s), ph ^ 1u, s_abort, p.status);
            mbar_expect_tx(full_bar(s), kMmaTileRows * half_bytes);
          }
          __syncwarp();
          if (lane < kMmaTileRows && !*s_abort) {
            const uint8_t *src = rec + which * mat_bytes + (size_t)(b * kMmaTileRows + lane) * row_bytes + half * half_bytes;
            const uint32_t stride = (which == 2) ? stride_d : stride_gu;
            bulk_g2s(smem_base + s * stage_bytes + lane * stride, src, half_bytes, full_bar(s));
          }
        }
      }
      u += (b_end - b_begin);
    }
    }
  } else {
    // ------------------------------ consumers ------------------------------
    const int g = lane >> 2, q = lane & 3;
    const int kslice = warp * (d / 8);      // first k of this warp's slice (gate/up) and first column (down)
    const int half = warp >> 2;             // which half of the rows' bytes this warp reads
    const int kl = (warp & 3) * (d / 8);    // the same offset inside that half
    for (int range = 0; range < 2; ++range) {
    const long long r0 = range ? zc_begin : first_res, rn = range ? total_all - zc_begin : total_res - first_res;
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
      // Resident records: one group of up to 8 tokens per weight pass, accumulators live across the CTA's
      // blocks of this pass.  Host-resident records cross the link once: every group of 8 tokens is served
      // from the staged block before its stages are released, and the accumulators are flushed per block.
      auto segment = [&](auto host_c) {   // instantiated twice so that the resident path carries no group loop
      constexpr bool host = decltype(host_c)::value;
      const int n_groups = host ? (it.n_tok + kMmaTokens - 1) / kMmaTokens : 1;
      int tok_g = -1;
      float gw_g = 0.f;
      uint32_t xf[KB][4];
      float dacc[CTW][4];
      auto load_group = [&](int grp) {   // token g of the group: row of x, gate weight, x fragments
        const int nt = min(kMmaTokens, it.n_tok - kMmaTokens * grp);
        tok_g = -1;
        gw_g = 0.f;
        if (g < nt) {
          if (it.expert >= 0) {
            const int pr = p.perm[it.off + kMmaTokens * grp + g];
            tok_g = pr / p.top_k;
            gw_g = p.topk_w[pr];
          } else {
            tok_g = kMmaTokens * grp + g;
            gw_g = 1.f;
          }
        }
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
          uint4 v = make_uint4(0u, 0u, 0u, 0u);
          if (tok_g >= 0) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok_g * d + kslice + 32 * kb + 8 * q);
          xf[kb][0] = v.x; xf[kb][1] = v.y; xf[kb][2] = v.z; xf[kb][3] = v.w;
        }
#pragma unroll
        for (int c = 0; c < CTW; ++c) { dacc[c][0] = dacc[c][1] = dacc[c][2] = dacc[c][3] = 0.f; }
      };
      auto flush = [&]() {   // gate-weighted combine: D fragment = [column g / g+8 of the tile][tokens 2q, 2q+1]
        const int tok_a = __shfl_sync(0xffffffffu, tok_g, (2 * q) * 4);
        const int tok_b = __shfl_sync(0xffffffffu, tok_g, (2 * q + 1) * 4);
        const float gw_a = __shfl_sync(0xffffffffu, gw_g, (2 * q) * 4);
        const float gw_b = __shfl_sync(0xffffffffu, gw_g, (2 * q + 1) * 4);
#pragma unroll
        for (int c = 0; c < CTW; ++c) {
          const int col = kslice + 16 * c + g;
          if (tok_a >= 0) {
            atomicAdd(p.y_acc + (size_t)tok_a * d + col, gw_a * dacc[c][0]);
            atomicAdd(p.y_acc + (size_t)tok_a * d + col + 8, gw_a * dacc[c][2]);
          }
          if (tok_b >= 0) {
            atomicAdd(p.y_acc + (size_t)tok_b * d + col, gw_b * dacc[c][1]);
            atomicAdd(p.y_acc + (size_t)tok_b * d + col + 8, gw_b * dacc[c][3]);
          }
        }
      };
      if (!host) load_group(pass);

      for (int b = b_begin; b < b_end; ++b, ++tile) {
        const uint32_t ph = tile & 1u;
        for (int grp = 0; grp < n_groups; ++grp) {
          const bool last = (grp == n_groups - 1);
          if (host) load_group(grp);
          float cgu[2][4];
#pragma unroll
          for (int which = 0; which < 2; ++which) {
            const int s = 2 * which + half;
            cgu[which][0] = cgu[which][1] = cgu[which][2] = cgu[which][3] = 0.f;
            float c2[4] = {0.f, 0.f, 0.f, 0.f};   // second accumulator: consecutive MMAs do not wait for each other
            const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
            if (ok) {
              const uint32_t base = smem_base + s * stage_bytes + (uint32_t)(kl + 8 * q) * 2u;
#pragma unroll
              for (int kb = 0; kb < KB; ++kb) {
                const uint4 lo = lds_v4(base + g * stride_gu + kb * 64);
                const uint4 hi = lds_v4(base + (g + 8) * stride_gu + kb * 64);
                mma_bf16(cgu[which], lo.x, hi.x, lo.y, hi.y, xf[kb][0], xf[kb][1]);
                mma_bf16(c2, lo.z, hi.z, lo.w, hi.w, xf[kb][2], xf[kb][3]);
              }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) cgu[which][i] += c2[i];
            __syncwarp();
            if (last && lane == 0) mbar_arrive(empty_bar(s));
          }
          // cross-warp reduction of the [16 neurons][8 tokens] partial sums
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
            s_h[t * 16 + n] = __float2bfloat16_rn(h);
          }
          asm volatile("bar.sync 1, 256;" ::: "memory");
          // down tile
          {
            const int s = 4 + half;
            const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
            if (ok) {
              const uint32_t *h32 = reinterpret_cast<const uint32_t *>(s_h);
              const uint32_t b0 = h32[g * 8 + q], b1 = h32[g * 8 + q + 4];
              // ldmatrix.x4.trans: lanes 0-7 / 8-15 / 16-23 / 24-31 address the four 8x8 blocks
              const int mat = lane >> 3, r = lane & 7;
              const uint32_t abase = smem_base + s * stage_bytes + (uint32_t)(r + 8 * (mat >> 1)) * stride_d +
                                     (uint32_t)(kl + 8 * (mat & 1)) * 2u;
#pragma unroll
              for (int c = 0; c < CTW; ++c) {
                uint32_t a[4];
                ldmatrix_x4_trans(a, abase + c * 32);
                mma_bf16(dacc[c], a[0], a[1], a[2], a[3], b0, b1);
              }
            }
            __syncwarp();
            if (last && lane == 0) mbar_arrive(empty_bar(s));
          }
          if (host) flush();
        }
      }
      if (!host) flush();
      };
      if (range == 0) segment(std::false_type{}); else segment(std::true_type{});
      u += (b_end - b_begin);
    }
    }
  }

  if (p.trace != nullptr && tid == 256) {   // lane 0 of the producer warp
    long long *tr = p.trace + 4 * blockIdx.x;
    long long t_end;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_end));
    tr[0] = t_start; tr[1] = t_end; tr[2] = trace_blocks; tr[3] = trace_segments;
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
  if (tid == 0) {
    *p.done = 0u;
    if (p.trace != nullptr) {   // the finalizing CTA also notes when the whole kernel was done
      long long t_fin;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_fin));
      p.trace[4 * blockIdx.x + 3] = -t_fin;
    }
  }
}

inline size_t ffn_mma_smem_bytes(int d) {
  return (size_t)kMmaStages * kMmaTileRows * ((size_t)d + 64) + 8 * 2 * 16 * 8 * 4 + 8 * 16 * 2 +
         (2 * kMaxExperts + 2) * 4 + 2 * kMmaStages * 8 + 16;
}

}  // namespace ftmoe
