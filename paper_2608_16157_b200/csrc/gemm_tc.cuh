// Step 5 for prefill-sized token counts: the gate/up half of the grouped SwiGLU expert FFN on the
// 5th-generation tensor cores, plus the helpers shared with the down-projection kernel (gemm_tc2.cuh), the row
// gather and the fused gather-combine.
//   H[P][I] = SiLU(Xs Wg^T) * (Xs Wu^T)   A = expert-sorted x rows (K-major, 128-byte swizzle), B = 128 gate rows +
//                                          the same 128 up rows of the record, N = 256, over the experts that hold
//                                          a slot and have at least `gemm_min_tokens` tokens.
// The record's tile order is already the tensor core's K-major layout with 64-byte swizzle (groups of 8 rows of
// 64 bytes): a weight tile is moved by plain TMA boxes of whole 1 KiB tiles and described to the MMA with a
// 512-byte step between 8-row groups; the two K = 16 slices of a tile are 32 bytes apart.
// One persistent CTA per SM: warp 0 feeds a 4-stage shared-memory ring with TMA tile loads (cp.async.bulk.tensor,
// each into this CTA's shared memory only), warp 1 issues tcgen05.mma (M=128, N=256, K=16, bf16 -> fp32) into one of two
// 256-column TMEM accumulators and signals stages free / tiles done with tcgen05.commit, warps 2-5 drain the other
// accumulator with tcgen05.ld, apply SwiGLU and store bf16, so the epilogue of tile i overlaps the main loop of
// tile i+1.  Every mbarrier wait is bounded; on expiry the CTA latches a timeout status, stops waiting, frees its
// TMEM and returns.  (Measured alternatives for this GEMM: two row tiles per CTA sharing B, 904 TFLOP/s, and CTA
// pairs, 961 unswapped / 815 swapped, against 956-973 for this form.)
#pragma once
#include <cuda.h>

#include "common.cuh"
#include "async.cuh"

namespace ftmoe {

constexpr int kGemmThreads = 192;
constexpr int kGemmBM = 128, kGemmBN = 256, kGemmBK = 64;
constexpr int kGemmATile = kGemmBM * kGemmBK * 2;   // 16 KiB
constexpr int kGemmBTile = kGemmBN * kGemmBK * 2;   // 32 KiB
constexpr int kGemmStages = 4, kGemmStageBytes = kGemmATile + kGemmBTile, kGemmBufs = 2;

struct GemmParams {
  const WorkItem *items;
  const int32_t *n_items;
  const int32_t *mt_pref;   // [n_items+1] exclusive prefix of 128-row tiles per item
  int K;                    // contraction length: d (gate/up) or I (down)
  int n_tiles;              // N tiles per row tile: I/128 (gate/up)
  int inter, d;
  long long layer_unit0;    // 16-neuron unit index of slot 0 of this layer in the weight tensor maps
  __nv_bfloat16 *out;       // H [P][I] (MODE 0) or O [P][d] (MODE 1)
  uint32_t *status;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar)
      : "memory");
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar)
      : "memory");
}

// 64-bit shared-memory matrix descriptor.  lbo/sbo in bytes (K-major: sbo = step between 8-row groups);
// swizzle: 2 = 128-byte, 4 = 64-byte, 6 = 32-byte rows.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo, uint32_t swizzle = 2) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3fffu);
  d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;   // descriptor version of this architecture
  d |= (uint64_t)swizzle << 61;
  return d;
}

__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// SiLU(g) * u with one MUFU: sigmoid(g) = 0.5 * tanh(0.5 g) + 0.5 (tanh.approx, rel. error ~2^-11, far below
// the bf16 rounding of the result).
__device__ __forceinline__ float swiglu_fast(float g, float u) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
  return g * fmaf(0.5f, t, 0.5f) * u;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 v = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t *>(&v);
}

// Dynamic shared memory (1024-byte aligned by the kernel): [stages][A 16 KiB | B 32 KiB] | barriers | tmem base |
// abort flag | tile prefix.
__global__ void __launch_bounds__(kGemmThreads, 1)
gateup_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmParams p) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  constexpr int MT = 1, kBufs = kGemmBufs;   // one 128-row tile per unit, two accumulator buffers
  unsigned char *sp = smem + kGemmStages * kGemmStageBytes;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(sp); sp += 16 * 8;
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(sp); sp += 8;
  volatile int *s_abort = reinterpret_cast<volatile int *>(sp); sp += 8;
  int32_t *s_pref = reinterpret_cast<int32_t *>(sp); sp += (kMaxExperts + 2) * 4;
  int32_t *s_upref = reinterpret_cast<int32_t *>(sp);   // exclusive prefix of the units (groups of MT row tiles)

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };
  auto empty_bar = [&](int s) { return bar_base + 8u * (kGemmStages + s); };
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kGemmStages + b); };
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kGemmStages + 2 + b); };

  const int n_items = *p.n_items;
  if (n_items == 0) return;
  if (tid == 0) {
    for (int s = 0; s < kGemmStages; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 4); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i <= n_items; i += blockDim.x) s_pref[i] = p.mt_pref[i];
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    int acc = 0;
    for (int i = 0; i < n_items; ++i) {
      s_upref[i] = acc;
      acc += (s_pref[i + 1] - s_pref[i] + MT - 1) / MT;
    }
    s_upref[n_items] = acc;
  }
  __syncthreads();
  const uint32_t tmem_base = *s_tmem;
  const int total_tiles = s_upref[n_items] * p.n_tiles;
  const int kblocks = p.K / kGemmBK;

  // work unit -> (item, first row tile inside the item, row tiles in the unit, n tile)
  auto locate = [&](int tile, int &item, int &mt_in, int &n_mt, int &nt) {
    const int un = tile / p.n_tiles;
    nt = tile - un * p.n_tiles;
    int lo = 0, hi = n_items;            // largest item with upref[item] <= un
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_upref[mid] <= un) lo = mid; else hi = mid;
    }
    item = lo;
    mt_in = (un - s_upref[lo]) * MT;
    n_mt = min(MT, s_pref[lo + 1] - s_pref[lo] - mt_in);
  };

  if (warp == 0) {
    // ------------------------------ TMA producer ------------------------------
    if (lane == 0) {
      uint32_t it_k = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x) {
        int item, mt_in, n_mt, nt;
        locate(tile, item, mt_in, n_mt, nt);
        const WorkItem it = p.items[item];
        const int a_row = it.off + mt_in * kGemmBM;
        const int unit0 = (int)(p.layer_unit0 + (long long)it.slot * (p.inter / 16)) + nt * 8;   // 128 neurons = 8 units
        for (int kb = 0; kb < kblocks; ++kb, ++it_k) {
          const int s = it_k % kGemmStages;
          const uint32_t ph = (it_k / kGemmStages) & 1u;
          mbar_wait(empty_bar(s), ph ^ 1u, s_abort, p.status);
          if (*s_abort) break;
          const uint32_t sa = smem_base + s * kGemmStageBytes;
          const uint32_t sb = sa + MT * kGemmATile;
          mbar_expect_tx(full_bar(s), n_mt * kGemmATile + kGemmBTile);
          if ((g_debug_withhold & kWithholdGemm) && it_k == 0) continue;   // test hook: stage never fills
          for (int m = 0; m < n_mt; ++m) tma_load_2d(sa + m * kGemmATile, &tmA, kb * kGemmBK, a_row + m * kGemmBM, full_bar(s));
          // per 32-wide hidden tile: 8 gate tiles (8 KiB: 16 groups of 8 neurons, 512 bytes apart) then the 8 up tiles
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            tma_load_3d(sb + j * 16384, &tmB, 0, 2 * kb + j, unit0, full_bar(s));
            tma_load_3d(sb + j * 16384 + 8192, &tmB, 0, p.d / 32 + 2 * kb + j, unit0, full_bar(s));
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer ------------------------------
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) |
                             ((uint32_t)(kGemmBN >> 3) << 17) | ((uint32_t)(kGemmBM >> 4) << 24);
      uint32_t it_k = 0, n_tile = 0;
      for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++n_tile) {
        int item, mt_in, n_mt, nt;
        locate(tile, item, mt_in, n_mt, nt);
        const int buf = n_tile % kBufs;
        mbar_wait(tempty_bar(buf), ((n_tile / kBufs) & 1u) ^ 1u, s_abort, p.status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * kGemmBN;   // (kBufs == 1: accumulator m at column m*256)
        for (int kb = 0; kb < kblocks; ++kb, ++it_k) {
          const int s = it_k % kGemmStages;
          const uint32_t ph = (it_k / kGemmStages) & 1u;
          const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
          tc_fence_after();
          if (ok) {
            const uint32_t sa = smem_base + s * kGemmStageBytes;
            const uint32_t sb = sa + MT * kGemmATile;
#pragma unroll
            for (int k16 = 0; k16 < kGemmBK / 16; ++k16) {
              const uint64_t bdesc = umma_desc(sb + (k16 >> 1) * 16384 + (k16 & 1) * 32, 16, 512, 4);
              for (int m = 0; m < n_mt; ++m) {
                const uint64_t adesc = umma_desc(sa + m * kGemmATile + k16 * 32, 16, 1024);
                umma_bf16(d_tmem + (uint32_t)m * kGemmBN, adesc, bdesc, idesc, (kb | k16) != 0 ? 1u : 0u);
              }
            }
          }
          umma_commit(empty_bar(s));   // the stage is free once these MMAs have read it
        }
        umma_commit(tfull_bar(buf));   // the accumulator is complete once all MMAs of the tile are done
      }
    }
  } else {
    // ------------------------------ epilogue (warps 2..5) ------------------------------
    const int quarter = warp & 3;      // TMEM lanes [32*quarter, 32*quarter+32) are visible to this warp
    uint32_t n_tile = 0;
    for (int tile = blockIdx.x; tile < total_tiles; tile += gridDim.x, ++n_tile) {
      int item, mt_in, n_mt, nt;
      locate(tile, item, mt_in, n_mt, nt);
      const WorkItem it = p.items[item];
      const int buf = n_tile % kBufs;
      const bool ok = mbar_wait(tfull_bar(buf), (n_tile / kBufs) & 1u, s_abort, p.status);
      tc_fence_after();
      for (int m = 0; m < n_mt; ++m) {
      const int row_in = (mt_in + m) * kGemmBM + quarter * 32 + lane;
      const bool valid = ok && row_in < it.n_tok;
      const size_t row = (size_t)it.off + row_in;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf + m) * kGemmBN;
      {
        __nv_bfloat16 *dst = p.out + row * p.inter + nt * 128;
#pragma unroll 1
        for (int c = 0; c < 128; c += 32) {
          uint32_t g[32], u[32];
          tmem_ld32(taddr + c, g);
          tmem_ld32(taddr + 128 + c, u);
          tmem_ld_wait();
          if (valid) {
            uint32_t o[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              o[j] = pack_bf16(swiglu_fast(__uint_as_float(g[2 * j]), __uint_as_float(u[2 * j])),
                               swiglu_fast(__uint_as_float(g[2 * j + 1]), __uint_as_float(u[2 * j + 1])));
            }
            uint4 *d4 = reinterpret_cast<uint4 *>(dst + c);
#pragma unroll
            for (int j = 0; j < 4; ++j) d4[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
          }
        }
      }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(buf));
    }
  }
  abort_drain(s_abort);   // (after a bounded wait gave up: let the copies in flight land before the CTA goes away)
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

inline size_t gateup_gemm_smem_bytes() {
  return 1024 + (size_t)kGemmStages * kGemmStageBytes + 16 * 8 + 16 + 2 * (kMaxExperts + 2) * 4;
}

// x rows into expert-sorted order: xs[pos] = x[perm[pos] / k]  (16 bytes per thread).
__global__ void __launch_bounds__(256) gather_rows_kernel(const __nv_bfloat16 *x, const int32_t *perm, int top_k, int d,
                                                          const int32_t *n_pairs, __nv_bfloat16 *xs) {
  const int P = *n_pairs;
  const int chunks = d / 8;
  const long long total = (long long)P * chunks;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int pos = (int)(i / chunks), c = (int)(i - (long long)pos * chunks);
    const int tok = perm[pos] / top_k;
    reinterpret_cast<uint4 *>(xs)[i] = *reinterpret_cast<const uint4 *>(x + (size_t)tok * d + c * 8);
  }
}

// Fused gather-combine: y[t] = bf16( y_acc[t] + sum_j w[t][j] * O[inv[t*k+j]] over the pairs whose expert went
// through the grouped GEMM ), ascending j, fp32; clears y_acc.
__global__ void __launch_bounds__(256) combine_kernel(const __nv_bfloat16 *o, const int32_t *ids, const float *w,
                                                      const int32_t *inv, const uint8_t *is_gemm, float *y_acc,
                                                      __nv_bfloat16 *y, int T, int top_k, int d) {
  const int chunks = d / 8;
  const long long total = (long long)T * chunks;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x) {
    const int t = (int)(i / chunks), c = (int)(i - (long long)t * chunks);
    float acc[8];
    float4 *ya = reinterpret_cast<float4 *>(y_acc + (size_t)t * d + c * 8);
    const float4 a0 = ya[0], a1 = ya[1];
    acc[0] = a0.x; acc[1] = a0.y; acc[2] = a0.z; acc[3] = a0.w;
    acc[4] = a1.x; acc[5] = a1.y; acc[6] = a1.z; acc[7] = a1.w;
    for (int j = 0; j < top_k; ++j) {
      const int pr = t * top_k + j;
      if (!is_gemm[ids[pr]]) continue;
      const float wj = w[pr];
      const uint4 v = *reinterpret_cast<const uint4 *>(o + (size_t)inv[pr] * d + c * 8);
      const uint32_t r[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        acc[2 * q] = fmaf(wj, __uint_as_float(r[q] << 16), acc[2 * q]);
        acc[2 * q + 1] = fmaf(wj, __uint_as_float(r[q] & 0xffff0000u), acc[2 * q + 1]);
      }
    }
    uint4 out = make_uint4(pack_bf16(acc[0], acc[1]), pack_bf16(acc[2], acc[3]), pack_bf16(acc[4], acc[5]),
                           pack_bf16(acc[6], acc[7]));
    *reinterpret_cast<uint4 *>(y + (size_t)t * d + c * 8) = out;
    ya[0] = make_float4(0.f, 0.f, 0.f, 0.f);
    ya[1] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

}  // namespace ftmoe
