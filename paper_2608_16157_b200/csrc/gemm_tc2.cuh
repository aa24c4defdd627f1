// Step 5 for prefill-sized token counts: the down-projection half of the grouped SwiGLU expert FFN on CTA pairs
// (gemm_tc.cuh holds the gate/up half and the shared helpers).
//
// Two CTAs of a cluster (two SMs) work on one tile with tcgen05.mma.cta_group::2 (M = 256 over the pair): each
// CTA stages its own 128 rows of A and one half of the rows of B, the leader CTA issues the MMAs for both, and
// each CTA's TMEM receives the accumulators of its own 128 rows, double-buffered against the epilogue.  Every
// CTA issues its own TMA loads, each for its own shared memory only (with .cta_group::2 so that they can signal the leader's mbarrier); stage
// release and accumulator hand-over go through one tcgen05.commit per CTA of the pair.
// Every mbarrier wait is bounded; on expiry the CTA latches a timeout status and runs to completion.
#pragma once
#include "gemm_tc.cuh"

namespace ftmoe {

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t mapa_u32(uint32_t addr, uint32_t rank) {
  uint32_t out;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(out) : "r"(addr), "r"(rank));
  return out;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive (optionally with a byte count) on an mbarrier given by its shared::cluster address
__device__ __forceinline__ void mbar_expect_tx_cluster(uint32_t bar_cluster, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;" ::"r"(bar_cluster), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const CUtensorMap *tm, int x, int y, int z, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(z), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap *tm, int x, int y, uint32_t bar_cluster) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(tm), "r"(x), "r"(y), "r"(bar_cluster)
      : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the mbarrier at this shared-memory offset in both CTAs of the pair once the MMAs issued so far are
// done: one commit per CTA (the leader's own barrier, then the peer's through its cluster address)
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mapa_u32(bar, 0)) : "memory");
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(mapa_u32(bar, 1)) : "memory");
}

// Swapped operands: the weights are the M side (always full 128-row tiles per CTA, 256 per pair), the tokens
// are the N side, so a ragged expert is padded to a multiple of 16 tokens instead of 128 rows.
//   O^T[column][token] : A = W_down^T, 128 columns per CTA x 64 neurons per stage, taken from the record's down
//   tiles as they are (K-major rows of 32 bytes with 32-byte swizzle, 256 bytes between 8-column groups); B = up
//   to 256 rows of H (each CTA stages half).  TMEM lane = output column,
//   TMEM column = token; the epilogue writes O[token][column].
struct Gemm2Cfg {
  static constexpr int kTokTile = 256;                                  // tokens per unit
  static constexpr int kStageBytes = kGemmATile + kGemmATile;           // Wd tile 16 KiB + 128 token rows 16 KiB
  static constexpr int kStages = 6;
};

// Dynamic shared memory (1024-byte aligned by the kernel): [stages][A | B half] | barriers | tmem base |
// abort flag | tile prefix | unit prefix.
__global__ void __launch_bounds__(kGemmThreads, 1)
down_gemm2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB, GemmParams p) {
  constexpr int MODE = 1;   // (the gate/up form of this kernel, MODE 0, measured slower than gemm_tc.cuh's; its
                            // constant-folded branches are gone)
  using Cfg = Gemm2Cfg;
  constexpr int kStages = Cfg::kStages, kStageBytes = Cfg::kStageBytes, kTok = Cfg::kTokTile;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *smem = reinterpret_cast<unsigned char *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  unsigned char *sp = smem + kStages * kStageBytes;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(sp); sp += 16 * 8;
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(sp); sp += 8;
  volatile int *s_abort = reinterpret_cast<volatile int *>(sp); sp += 8;
  int32_t *s_pref = reinterpret_cast<int32_t *>(sp); sp += (kMaxExperts + 2) * 4;
  int32_t *s_upref = reinterpret_cast<int32_t *>(sp); sp += (kMaxExperts + 2) * 4;   // prefix of the token tiles per item
  __nv_bfloat16 *s_trans = reinterpret_cast<__nv_bfloat16 *>(((uintptr_t)sp + 15) & ~(uintptr_t)15);   // 4 x [32][32]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = cluster_ctarank();           // 0 = leader (issues the MMAs)
  const uint32_t smem_base = smem_u32(smem);
  const uint32_t bar_base = smem_u32(s_bar);
  auto full_bar = [&](int s) { return bar_base + 8u * s; };                   // used in the leader only
  auto empty_bar = [&](int s) { return bar_base + 8u * (kStages + s); };      // local, released by the commit
  auto tfull_bar = [&](int b) { return bar_base + 8u * (2 * kStages + b); };  // local
  auto tempty_bar = [&](int b) { return bar_base + 8u * (2 * kStages + 2 + b); };  // used in the leader only

  const int n_items = *p.n_items;       // the same in both CTAs: either both leave here or none
  if (n_items == 0) return;
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(full_bar(s), 2); mbar_init(empty_bar(s), 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(tfull_bar(b), 1); mbar_init(tempty_bar(b), 8); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i <= n_items; i += blockDim.x) s_pref[i] = p.mt_pref[i];
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (tid == 0) {
    int acc = 0;
    for (int i = 0; i < n_items; ++i) {
      s_upref[i] = acc;
      const int t128 = s_pref[i + 1] - s_pref[i];             // 128-token tiles of the item
      acc += (MODE == 0) ? t128 : (t128 + 1) / 2;
    }
    s_upref[n_items] = acc;
  }
  __syncthreads();
  cluster_sync_all();                   // the peer's barriers are initialised before anything is signalled
  const uint32_t tmem_base = *s_tmem;
  const int m_pairs = ((MODE == 0) ? p.inter : p.d) / 256;   // 256 neurons / output columns per CTA pair
  const int total_units = s_upref[n_items] * m_pairs;
  const int kblocks = p.K / kGemmBK;
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  // unit -> item, first token of the tile (relative to the item), tokens in it, this CTA's first neuron / column
  auto locate = [&](int unit, int &item, int &tok0, int &n_valid, int &m_base) {
    const int tt = unit / m_pairs;
    const int mp = unit - tt * m_pairs;
    int lo = 0, hi = n_items;
    while (hi - lo > 1) {
      const int mid = (lo + hi) >> 1;
      if (s_upref[mid] <= tt) lo = mid; else hi = mid;
    }
    item = lo;
    tok0 = (tt - s_upref[lo]) * kTok;
    m_base = mp * 256 + (int)rank * 128;
    n_valid = 0;   // filled by the caller from the item's token count
  };

  if (warp == 0) {
    // ------------------------------ TMA producer (both CTAs) ------------------------------
    if (lane == 0) {
      uint32_t it_k = 0;
      for (int unit = pair; unit < total_units; unit += n_pairs) {
        int item, tok0, n_valid, m_base;
        locate(unit, item, tok0, n_valid, m_base);
        const WorkItem it = p.items[item];
        n_valid = min(kTok, it.n_tok - tok0);
        const int N = (n_valid + 15) & ~15;
        const int b_row = it.off + tok0 + (int)rank * (N / 2);       // this CTA stages the tokens [rank*N/2, +N/2)
        const int unit0 = (int)(p.layer_unit0 + (long long)it.slot * (p.inter / 16));
        for (int kb = 0; kb < kblocks; ++kb, ++it_k) {
          const int s = it_k % kStages;
          const uint32_t ph = (it_k / kStages) & 1u;
          mbar_wait(empty_bar(s), ph ^ 1u, s_abort, p.status);
          if (*s_abort) break;
          const uint32_t sa = smem_base + s * kStageBytes;
          const uint32_t lead_full = mapa_u32(full_bar(s), 0);
          mbar_expect_tx_cluster(lead_full, kStageBytes);
          // the down tiles of 128 columns (4 KiB) of the stage's 4 units (64 neurons): one box of 16 KiB
          tma_load_3d_pair(sa, &tmA, 0, p.d / 32 + m_base / 64, unit0 + 4 * kb, lead_full);
          tma_load_2d_pair(sa + kGemmATile, &tmB, kb * kGemmBK, b_row, lead_full);              // 128 token rows of H
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------ MMA issuer (leader CTA only) ------------------------------
    if (lane == 0 && rank == 0) {
      uint32_t it_k = 0, n_unit = 0;
      for (int unit = pair; unit < total_units; unit += n_pairs, ++n_unit) {
        int item, tok0, n_valid, m_base;
        locate(unit, item, tok0, n_valid, m_base);
        n_valid = min(kTok, p.items[item].n_tok - tok0);
        const uint32_t N = (uint32_t)((n_valid + 15) & ~15);
        // bf16 x bf16 -> fp32, M = 256 over the pair, N tokens, both operands K-major
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((uint32_t)(256 >> 4) << 24);
        const int buf = n_unit & 1;
        mbar_wait(tempty_bar(buf), ((n_unit >> 1) & 1u) ^ 1u, s_abort, p.status);
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)buf * 256;
        for (int kb = 0; kb < kblocks; ++kb, ++it_k) {
          const int s = it_k % kStages;
          const uint32_t ph = (it_k / kStages) & 1u;
          const bool ok = mbar_wait(full_bar(s), ph, s_abort, p.status);
          tc_fence_after();
          if (ok) {
            const uint32_t sa = smem_base + s * kStageBytes;
#pragma unroll
            for (int k16 = 0; k16 < kGemmBK / 16; ++k16) {
              const uint32_t acc = (kb | k16) != 0 ? 1u : 0u;
              umma2_bf16(d_tmem, umma_desc(sa + k16 * 4096, 16, 256, 6),
                         umma_desc(sa + kGemmATile + k16 * 32, 16, 1024), idesc, acc);
            }
          }
          umma2_commit_both(empty_bar(s));    // frees the stage in both CTAs once these MMAs have read it
        }
        umma2_commit_both(tfull_bar(buf));    // both CTAs' accumulators are complete
      }
    }
  } else {
    // ------------------------------ epilogue (warps 2..5 of both CTAs) ------------------------------
    const int quarter = warp & 3;
    uint32_t n_unit = 0;
    for (int unit = pair; unit < total_units; unit += n_pairs, ++n_unit) {
      int item, tok0, n_valid, m_base;
      locate(unit, item, tok0, n_valid, m_base);
      const WorkItem it = p.items[item];
      n_valid = min(kTok, it.n_tok - tok0);
      const int buf = n_unit & 1;
      const bool ok = mbar_wait(tfull_bar(buf), (n_unit >> 1) & 1u, s_abort, p.status);
      tc_fence_after();
      // this warp's 32 neurons / output columns start at m0; lane l holds row m0 + l of the accumulator, i.e. one
      // neuron for 32 tokens at a time.  The chunk is transposed through shared memory so that the global
      // stores are 16-byte vectors along the contiguous (neuron / column) dimension of H / O.
      const int m0 = m_base + quarter * 32;
      const size_t row0 = (size_t)it.off + tok0;                  // first expert-sorted row of the tile
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * 256;
      const size_t ld = (MODE == 0) ? (size_t)p.inter : (size_t)p.d;
      __nv_bfloat16 *s_t = s_trans + (warp - 2) * (32 * 32);      // [32 tokens][32 columns] bf16
#pragma unroll 1
      for (int c = 0; c < n_valid; c += 32) {                     // 32 tokens per TMEM load; warp-uniform bound
        uint32_t v[32];
        tmem_ld32(taddr + c, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) s_t[j * 32 + lane] = __float2bfloat16_rn(__uint_as_float(v[j]));
        __syncwarp();
        if (ok) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int idx = lane + 32 * i, r = idx >> 2, q4 = idx & 3;      // token r of the chunk, 8 columns
            if (c + r < n_valid)
              *reinterpret_cast<uint4 *>(p.out + (row0 + c + r) * ld + m0 + q4 * 8) =
                  *reinterpret_cast<const uint4 *>(s_t + r * 32 + q4 * 8);
          }
        }
        __syncwarp();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(mapa_u32(tempty_bar(buf), 0));   // the leader's MMA thread waits for both CTAs
    }
  }
  abort_drain(s_abort);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                   // neither CTA leaves while the other may still touch its memory or barriers
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem_base) : "memory");
  }
}

inline size_t down_gemm2_smem_bytes() {
  return 1024 + (size_t)Gemm2Cfg::kStages * Gemm2Cfg::kStageBytes + 16 * 8 + 16 + 2 * (kMaxExperts + 2) * 4 +
         16 + 4 * 32 * 32 * 2;
}

}  // namespace ftmoe
