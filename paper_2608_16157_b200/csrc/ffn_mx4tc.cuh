// Steps 5+6 for MXFP4 experts stored as tensor-core operand images (FT_W_MXFP4_TC), 8 tokens of an expert per pass:
// the block-scaled 5th-generation tensor-core instruction tcgen05.mma kind::mxf4 multiplies packed e2m1 weights by
// e2m1 activations, both with one power-of-two scale per 32 elements held in tensor memory, so the weights need no
// unpacking at all: a record's bytes go from HBM (or, for zero-copy experts, from the mapped host pool) to shared
// memory by bulk copies and are consumed there by the instruction (paper Sec. 5.1 expert representations; Sec. 3.2
// grouped evaluation of the resident and the zero-copy experts).
//   * Activations keep their precision by bit slicing along N: a (token, block of 32) is written as a sum of
//     kTcTerms block-scaled e2m1 vectors, term i being the e2m1 rounding of what the terms before it left over,
//     each with its own scale (the smallest power of two that brings the leftover's largest magnitude to <= 6).
//     Every term removes at least a factor 3 of the block's largest leftover, so 6 terms leave <= 2^-9.5 of the
//     block's largest magnitude; the terms of the 8 tokens are the N = 48 columns of the MMA (column 8 i + token),
//     and the epilogue adds a token's 6 columns.  The tensor pipe has room for this: the kernels are HBM-bound.
//     A call with at most 8 tokens has one activation image (its tokens, for every expert); a larger call one image
//     per pass (8 tokens of the pass's expert, gathered through the expert-sorted permutation), which a CTA brings
//     into shared memory when its tiles change pass.
//   * Gate/up kernel: M = 128 neurons of the gate and of the up matrix per tile, K split into four parts (a CTA
//     keeps the activation image of one part in shared memory: CTA i that of part i % 4, which leaves most of the
//     shared memory to the ring), each CTA an equal share of (tile, 128-index stage) steps of its part.  A producer
//     warp issues the bulk copies (17408 bytes per stage: gate image, up image, gate scales, up scales) into a
//     ring; two issuing threads, one for the gate and one for the up matrix, copy the stage's scale factors to
//     tensor memory (tcgen05.cp) and issue two MMAs each (an MMA of this shape occupies the tensor pipe for about
//     136 clocks whatever N is, so the pipe is busy most of the time and the scalar work of one issuer must hide
//     behind the MMAs of the other); four warps read the accumulators of a finished tile (tcgen05.ld), add a
//     token's terms and add the partial sums into the per-unit fp32 accumulators in global memory; the CTA whose
//     contribution completes a group of 128 neurons applies SiLU(gate) * up and writes the group's h as the
//     bit-sliced activation image of the down kernel.
//   * Down kernel: M = 128 output columns per tile, K = the neurons; same ring, the two issuers take the stages
//     alternately and accumulate separately; the epilogue adds the two, multiplies by the gate weight and adds into
//     the fp32 output accumulator; the last CTA rounds it to bf16.
// Every mbarrier wait is bounded (see async.cuh); a CTA whose wait runs out latches the timeout status, stops
// issuing work, lets its copies in flight land, frees its tensor memory and returns.
#pragma once
#include <cuda_fp4.h>

#include "async.cuh"
#include "ffn_w4.cuh"
#include "gemm_tc.cuh"

namespace ftmoe {

constexpr int kTcTerms = 6;                 // e2m1 terms per activation
constexpr int kTcN = 8 * kTcTerms;          // MMA columns: 8 tokens x terms
constexpr uint32_t kTcStepB = kTcN * 32u;   // bytes of the activation image of one K = 64 step
constexpr uint32_t kTcStageA = 17408u;      // gate/up stage: two images of 8192 bytes, two scale atoms of 512
constexpr uint32_t kTcStageD = 8704u;       // down stage: one image, one scale atom
constexpr int kTcLoaders = 128;             // the first kTcLW warps copy the records' stages into the ring, 16 bytes per cp.async
constexpr int kTcLW = kTcLoaders / 32;      // (a loader warp has one stage in flight; eight warps measured slower than four)
constexpr int kTcThreads = kTcLoaders + 64 + 128;   // then two warps: MMA issuers, four warps: epilogue
constexpr int kTcMaxStages = 16;
constexpr size_t kTcSmem = 232448 - 1024;   // dynamic shared memory the two kernels may use (1 KiB left for static data)

// Activation images in global memory (written by tc_quant_x_kernel / by the gate/up kernel's group conversion).
// Gate/up operand: for each of the kTcParts parts of the hidden dimension: [d/256 steps][kTcStepB] then
// [d/512 scale atoms][512].
constexpr int kTcParts = 4;
__host__ __device__ inline size_t tc_x_part_bytes(int d) {
  return (size_t)(d / (64 * kTcParts)) * kTcStepB + (size_t)(d / (128 * kTcParts)) * 512;
}
// Down operand of one pass: [inter/64 steps][kTcStepB] then [inter/128 scale atoms][512].
__host__ __device__ inline size_t tc_h_pass_bytes(int inter) { return (size_t)(inter / 64) * kTcStepB + (size_t)(inter / 128) * 512; }

// One bit-slicing term of 8 values held by each of the 4 lanes of a quad (the quad = one block of 32): returns the 8
// codes (nibble e = element e) and the scale byte, and subtracts the term from r[].  bad: a non-finite input.
// The e2m1 rounding (nearest, saturating at 6) and the way back are the hardware's conversions.
__device__ __forceinline__ void tc_term(float (&r)[8], bool bad, uint32_t &codes, uint32_t &scale_byte) {
  float m = 0.f;
#pragma unroll
  for (int e = 0; e < 8; ++e) m = fmaxf(m, fabsf(r[e]));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
  codes = 0u;
  if (bad) { scale_byte = 255u; return; }           // the scale format's NaN: the token's outputs become NaN
  if (m < 1e-37f) { scale_byte = 127u; return; }    // nothing left: zeros
  const uint32_t tb = __float_as_uint(m * (1.f / 6.f));
  uint32_t ex = (tb >> 23) + ((tb & 0x007FFFFFu) ? 1u : 0u);   // smallest power of two >= m / 6
  ex = min(max(ex, 1u), 253u);
  scale_byte = ex;
  const float scale = __uint_as_float(ex << 23), inv = __uint_as_float((254u - ex) << 23);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const __nv_fp4x2_storage_t c = __nv_cvt_float2_to_fp4x2(make_float2(r[2 * k] * inv, r[2 * k + 1] * inv), __NV_E2M1, cudaRoundNearest);
    const __half2_raw hb = __nv_cvt_fp4x2_to_halfraw2(c, __NV_E2M1);
    const float2 back = __half22float2(*reinterpret_cast<const __half2 *>(&hb));
    r[2 * k] -= back.x * scale;
    r[2 * k + 1] -= back.y * scale;
    codes |= (uint32_t)c << (8 * k);
  }
}

// Tokens of a pass: with at most 8 tokens in the call ("dense") the 8 columns are the call's tokens for every pass;
// otherwise a pass serves 8 tokens of its list entry (pass = the entry's first pass + k: tokens 8k .. 8k+7 of the
// entry, gathered through the expert-sorted permutation; the shared expert's entry holds the tokens themselves).
struct TcPassTokens {
  int nt;        // columns in use
  int tok[8];    // token of column j, or -1
  float w[8];    // its gate weight
};
__device__ __forceinline__ void tc_pass_tokens(const W4Params &p, bool dense, uint32_t pass, bool want_weights, TcPassTokens &o) {
#pragma unroll
  for (int j = 0; j < 8; ++j) { o.tok[j] = -1; o.w[j] = 0.f; }
  const int n_lists = *p.n_items + *p.n_zc;
  const int item = dense ? (int)pass : w4_find_item(p.pref, n_lists, pass);
  const WorkItem wi = p.items[item];
  const int tok0 = dense ? 0 : (int)(pass - (uint32_t)p.pref[item]) * 8;
  const int cnt = min(8, wi.n_tok - tok0);
  o.nt = dense ? p.T : cnt;
  if (wi.expert < 0) {
#pragma unroll
    for (int j = 0; j < 8; ++j)
      if (j < cnt) { o.tok[j] = tok0 + j; o.w[j] = 1.f; }
    return;
  }
  for (int j = 0; j < cnt; ++j) {
    const int pr = p.perm[wi.off + tok0 + j];
    const int tk = pr / p.top_k;
    const float wv = want_weights ? p.topk_w[pr] : 1.f;
    const int col = dense ? tk : j;       // dense: column = token
#pragma unroll
    for (int c = 0; c < 8; ++c)
      if (c == col) { o.tok[c] = tk; o.w[c] = wv; }
  }
}

// Completion counts of the launches of a handle (cumulative numbers of CTAs that have finished: [0] gate/up kernels,
// [1] down kernels).  A launch is given the counts all earlier launches add up to and waits for them, bounded, before
// it touches what those launches use; in stream order the waits are satisfied on arrival, and they are what makes
// launch overlap mode 2 (a call's first kernels start while the call before is still finishing) safe by construction.
__device__ __forceinline__ bool tc_wait_count(const int *addr, int expect, uint32_t *status) {
  const uint32_t limit = g_wait_polls;
  for (uint32_t polls = 0; polls < limit; ++polls) {
    int have;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(have) : "l"(addr) : "memory");
    if ((int)((uint32_t)have - (uint32_t)expect) >= 0) return true;
    __nanosleep(64);
  }
  atomicOr(status, kStatTimeout);
  return false;
}

// x [T][d] bf16 -> the gate/up kernel's activation images: image i (blockIdx.y) holds the 8 token columns of pass i
// (dense: one image, columns = the call's tokens), each as kTcParts parts of the hidden dimension.  One thread per 8
// consecutive hidden indices of a column (unused columns are written as zeros); a quad of lanes is one block of 32.
struct TcQuantParams {
  W4Params w;
  const __nv_bfloat16 *x;
  uint8_t *xq;      // [images][kTcParts][tc_x_part_bytes(d)]
  int d, dense;
  const int *gen;   // completion counts (see tc_wait_count)
  int expect_gu;    // gate/up CTAs of all earlier calls: they read the images this kernel overwrites
  int early;        // launch overlap mode 2: do not wait for the kernel before this one
};
__global__ void __launch_bounds__(256) tc_quant_x_kernel(TcQuantParams q) {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const W4Params &p = q.w;
  if (!q.early) {
    // (when launched as a programmatic dependent: the images are still being read until the kernels before have completed)
    asm volatile("griddepcontrol.wait;" ::: "memory");
  } else {
    // the caller's word: x, the plan and the slots are not produced by the kernel before; the images were last read
    // by the gate/up kernel of the call before
    if (threadIdx.x == 0) (void)tc_wait_count(q.gen, q.expect_gu, p.status);
    __syncthreads();
  }
  const uint32_t pass = blockIdx.y;
  if (!q.dense && pass >= (uint32_t)p.pref[*p.n_items + *p.n_zc]) return;
  const int per_tok = q.d / 8;
  const int i = blockIdx.x * 256 + threadIdx.x;
  if (i >= 8 * per_tok) return;
  const int col = i / per_tok, c8 = i - col * per_tok;   // hidden indices 8 c8 .. 8 c8 + 7 of column col
  int tok;
  if (q.dense) {
    tok = col < p.T ? col : -1;
  } else {
    __shared__ TcPassTokens s_pt;
    if (threadIdx.x == 0) tc_pass_tokens(p, false, pass, false, s_pt);
    __syncthreads();
    tok = s_pt.tok[col];
  }
  float r[8];
  bool bad = false;
  if (tok >= 0) {
    const uint4 v = *reinterpret_cast<const uint4 *>(q.x + (size_t)tok * q.d + 8 * c8);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      r[2 * e] = __uint_as_float(w[e] << 16);
      r[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) bad |= !(fabsf(r[e]) <= 3.0e38f);
  } else {
#pragma unroll
    for (int e = 0; e < 8; ++e) r[e] = 0.f;
  }
  bad = (__shfl_xor_sync(0xffffffffu, (int)bad, 1) | __shfl_xor_sync(0xffffffffu, (int)bad, 2) | (int)bad) != 0;
  const int part_k = q.d / kTcParts;
  const int k = 8 * c8, part = k / part_k, kk = k - part * part_k;
  uint8_t *img = q.xq + ((size_t)(q.dense ? 0u : pass) * kTcParts + part) * tc_x_part_bytes(q.d);
  uint8_t *sf = img + (size_t)(part_k / 64) * kTcStepB;
  const int step = kk >> 6, kcore = (kk >> 5) & 1, word = (kk & 31) >> 3;
#pragma unroll
  for (int t = 0; t < kTcTerms; ++t) {
    uint32_t codes, sb;
    tc_term(r, bad, codes, sb);
    *reinterpret_cast<uint32_t *>(img + (size_t)step * kTcStepB + kcore * (kTcN * 16) + t * 128 + col * 16 + word * 4) = codes;
    if ((threadIdx.x & 3) == 0) {
      const int n = 8 * t + col, blk = kk >> 5;   // scale of (column n, block blk of the part)
      sf[(size_t)(blk >> 2) * 512 + (n & 31) * 16 + (n >> 5) * 4 + (blk & 3)] = (uint8_t)sb;
    }
  }
}


struct TcParams {
  W4Params w;          // the work lists, the hand-over buffers (hraw, hcount, hq) and the output, as for the other 4-bit kernels
  const uint8_t *xq;   // activation images (tc_quant_x_kernel): one per pass, or one for all passes when dense
  int dense;           // at most 8 tokens in the call: the MMA's token columns are the call's tokens for every pass
  int d;
  int n_stages;        // ring stages (what fits in shared memory, at most kTcMaxStages)
  int *pass_done;      // per pass: groups of 128 neurons whose h the gate/up kernel has written (0 between calls)
  int *gen;            // completion counts (see tc_wait_count)
  int expect_gu, expect_dn;   // gate/up CTAs, down CTAs of all earlier calls
};

// ---- PTX wrappers of the block-scaled path ----
__device__ __forceinline__ uint64_t tc_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  return umma_desc(smem_addr, lbo, sbo, 0);   // K-major core matrices of 8 rows x 16 bytes, no swizzle
}
__device__ __forceinline__ void tc_cp_scales(uint32_t tmem_col, uint32_t smem_addr) {
  // 32 rows x 16 bytes -> lanes 0..31 x 4 columns, repeated for the four lane quarters
  asm volatile("tcgen05.cp.cta_group::1.32x128b.warpx4 [%0], %1;" ::"r"(tmem_col), "l"(tc_desc(smem_addr, 0, 128)) : "memory");
}
// D[128 x kTcN] (+)= A[128 x 64] * B[kTcN x 64]^T, e2m1 operands, one ue8m0 scale per 32 elements; sf_id = 0 or 2:
// which two of a scale word's four bytes belong to this K step.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t sf_id, uint32_t sfa,
                                       uint32_t sfb, uint32_t accumulate) {
  const uint32_t idesc = (sf_id << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcN >> 3) << 17) | (1u << 23) |
                         ((128u >> 4) << 24) | (sf_id << 29);
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::mxf4.block_scale.scale_vec::2X [%0], %1, %2, %3, [%5], [%6], p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(sfa | (sf_id << 30)), "r"(sfb | (sf_id << 30))
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
// The kTcN columns of this thread's accumulator row -> one sum per token, added to v[].
__device__ __forceinline__ void tc_row_sums(uint32_t taddr, float (&v)[8]) {
#pragma unroll
  for (int c = 0; c < kTcN; c += 16) {
    uint32_t r[16];
    tmem_ld16(taddr + c, r);
    tmem_ld_wait();
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j & 7] += __uint_as_float(r[j]);
  }
}
__device__ __forceinline__ void tc_cp16(uint32_t dst, const void *src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
// Shared memory written by the loaders' copies is read by the tensor core: order the two kinds of access.
__device__ __forceinline__ void tc_fence_copies() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// One stage is copied by one loader warp (the loader warps take the stages in turn): each lane copies its 16-byte
// pieces and posts an arrival that fires when its copies have landed.  The arrival orders a warp's later copies
// behind it, so a warp has one stage in flight; the stages in flight are those of the different loader warps.
template <uint32_t BYTES>
__device__ __forceinline__ void tc_load_stage(uint32_t dst, const uint8_t *src, int lane, uint32_t full_bar) {
  constexpr uint32_t kPieces = BYTES / 16u;
  static_assert(kPieces % 32u == 0, "whole warps");
#pragma unroll
  for (uint32_t c = 0; c < kPieces / 32u; ++c) tc_cp16(dst + (c * 32u + lane) * 16u, src + (c * 32u + lane) * 16u);
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(full_bar) : "memory");
}
__device__ __forceinline__ void tc_epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// Barriers of both kernels (8 bytes each): full[16] | empty[16] | tfull[2] | tempty[2] | four more.
struct TcBars {
  uint32_t base;
  __device__ uint32_t full(uint32_t s) const { return base + 8u * s; }
  __device__ uint32_t empty(uint32_t s) const { return base + 8u * (kTcMaxStages + s); }
  __device__ uint32_t tfull(uint32_t b) const { return base + 8u * (2 * kTcMaxStages + b); }
  __device__ uint32_t tempty(uint32_t b) const { return base + 8u * (2 * kTcMaxStages + 2 + b); }
  __device__ uint32_t extra(uint32_t i) const { return base + 8u * (2 * kTcMaxStages + 4 + i); }
};

// Shared memory of the gate/up kernel: activation image of the CTA's part of K | its scale atoms | ring | barriers |
// flags.
inline size_t tc_gateup_fixed_bytes(int d) { return tc_x_part_bytes(d) + 64 * 8 + 64 + 128; }

__global__ void __launch_bounds__(kTcThreads, 1) tc_gateup_kernel(TcParams q) {
  const W4Params &p = q.w;
  const int d = q.d;
  const uint32_t NS = (uint32_t)q.n_stages;
  const uint32_t KS = (uint32_t)d / 128u, SPH = KS / kTcParts;    // stages of a tile; of one part of the hidden dimension
  const uint32_t NG = (uint32_t)p.inter / 128u, NBLK = (uint32_t)p.inter / 16u;
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_b = smem;                                        // [2 SPH steps][kTcStepB]
  unsigned char *s_sfb = s_b + (size_t)2 * SPH * kTcStepB;          // [SPH][512]
  unsigned char *s_ring = s_sfb + (size_t)SPH * 512;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(s_ring + (size_t)NS * kTcStageA);
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(s_bar + 64);
  volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);
  volatile int *s_last = s_abort + 1, *s_stop = s_abort + 2;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const TcBars bar{smem_u32(s_bar)};
  const uint32_t x_bar = bar.extra(0), sfb_bar = bar.extra(1), xempty_bar = bar.extra(2);
  if (tid == 0) {
    for (uint32_t s = 0; s < NS; ++s) { mbar_init(bar.full(s), 32); mbar_init(bar.empty(s), 2); }
    for (uint32_t b = 0; b < 2; ++b) { mbar_init(bar.tfull(b), 2); mbar_init(bar.tempty(b), 4); }
    mbar_init(x_bar, 1);
    mbar_init(sfb_bar, 1);
    mbar_init(xempty_bar, 2);
    *s_abort = 0;
    *s_last = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  const bool dense = q.dense != 0;   // then every list entry is one pass: pass = index into the list
  if (warp == kTcLW) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // tensor memory columns: accumulators (buffer b: gate at 128 b, up at 128 b + 64) | weight scales of the ring
  // slots (gate 4 s, up 64 + 4 s) | activation scales of the part (4 per stage)
  const uint32_t t_sfa = tmem + 256u, t_sfb = tmem + 384u;

  // this CTA's share: CTA i works on part i % kTcParts of the hidden dimension; within a part and within each of the
  // two pass ranges (resident passes, then zero-copy passes) an equal number of stages per CTA
  const uint32_t part = blockIdx.x % kTcParts, ci = blockIdx.x / kTcParts, nc = gridDim.x / kTcParts;
  uint32_t pass0[2], s_begin[2], s_end[2];
  pass0[0] = 0u;
  pass0[1] = (uint32_t)p.pref[n_items];
  {
    const uint32_t t0 = pass0[1] * NG * SPH, t1 = ((uint32_t)p.pref[n_items + n_zc] - pass0[1]) * NG * SPH;
    s_begin[0] = w4_first(t0, nc, ci); s_end[0] = w4_first(t0, nc, ci + 1);
    s_begin[1] = w4_first(t1, nc, ci); s_end[1] = w4_first(t1, nc, ci + 1);
  }
  // body(pass, ng, st0, n): a run of n stages, starting at stage st0 of the part, of tile (pass, ng)
  auto walk = [&](auto body) {
    for (int r = 0; r < 2; ++r)
      for (uint32_t s = s_begin[r]; s < s_end[r];) {
        const uint32_t tile = s / SPH, st0 = s - tile * SPH, n = min(SPH - st0, s_end[r] - s);
        if (!body(pass0[r] + tile / NG, tile % NG, st0, n)) return;
        s += n;
      }
  };

  if (warp < kTcLW) {
    // ---- loaders: the weights do not depend on the preceding kernels; the activation images do ----
    // Thread 0 also brings the activation image (of the pass, or the one image of a dense call) into shared memory:
    // the first one after the first ring fill (so that the weights start to stream while the kernel before still
    // runs), a later one once the MMAs that read its predecessor have completed.
    uint32_t it = 0, n_x = 0, cur = 0xffffffffu, pending = 0xffffffffu;
    bool waited = false;
    auto send_x = [&](uint32_t img) {
      if (!waited) { asm volatile("griddepcontrol.wait;" ::: "memory"); waited = true; }
      // (a wait that gives up latches the abort flag: every loader then leaves at its next wait)
      if (!n_x || mbar_wait(xempty_bar, (n_x - 1u) & 1u, s_abort, p.status)) {
        const uint32_t bytes = (uint32_t)tc_x_part_bytes(d);
        mbar_expect_tx(x_bar, bytes);
        const uint8_t *src = q.xq + ((size_t)img * kTcParts + part) * bytes;
        for (uint32_t o = 0; o < bytes; o += 16384u) bulk_g2s(smem_u32(s_b) + o, src + o, min(16384u, bytes - o), x_bar);
        ++n_x;
      }
    };
    walk([&](uint32_t pass, uint32_t ng, uint32_t st0, uint32_t n) {
      const uint32_t img = dense ? 0u : pass;
      if (tid == 0 && img != cur) {
        if (pending != 0xffffffffu) { send_x(pending); pending = 0xffffffffu; }
        if (cur == 0xffffffffu) pending = img;   // the first image is sent below, after the first ring fill
        else send_x(img);
        cur = img;
      }
      const int item = dense ? (int)pass : w4_find_item(p.pref, n_items + n_zc, pass);
      const uint8_t *src = p.items[item].w + ((size_t)ng * KS + part * SPH + st0) * kTcStageA;
      for (uint32_t s = 0; s < n; ++s, ++it, src += kTcStageA) {
        const uint32_t slot = it % NS;
        if (it % (kTcLoaders / 32) == (uint32_t)warp) {
          bool ok = true;
          if (lane == 0) ok = mbar_wait(bar.empty(slot), ((it / NS) & 1u) ^ 1u, s_abort, p.status);
          if (!__shfl_sync(0xffffffffu, (int)ok, 0)) return false;
          if ((g_debug_withhold & kWithholdTc) && it == 0) continue;   // test hook: this stage never arrives
          tc_load_stage<kTcStageA>(smem_u32(s_ring) + slot * kTcStageA, src, lane, bar.full(slot));
        }
        if (tid == 0 && pending != 0xffffffffu && it + 1 == NS) { send_x(pending); pending = 0xffffffffu; }
      }
      return true;
    });
    if (tid == 0 && pending != 0xffffffffu) send_x(pending);
    // the copies issued must have landed before this CTA's shared memory is released
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (tid == 0) {
      if (n_x) (void)mbar_wait(x_bar, (n_x - 1u) & 1u, s_abort, p.status);
      abort_drain(s_abort);
    }
  } else if (warp <= kTcLW + 1) {
    if (lane == 0) {
      // ---- MMA issuers: the first of the two warps the gate matrix, the second the up matrix ----
      const uint32_t mat = (uint32_t)(warp - kTcLW);
      uint32_t it = 0, seg = 0, n_x = 0, cur = 0xffffffffu;
      const uint32_t b_base = smem_u32(s_b), ring = smem_u32(s_ring) + mat * 8192u, t_sf = t_sfa + mat * 64u;
      walk([&](uint32_t pass, uint32_t, uint32_t st0, uint32_t n) {
          const uint32_t img = dense ? 0u : pass;
          if (img != cur) {
            // a new activation image: its scales go to tensor memory once the MMAs on the old one are done
            if (n_x) umma_commit(xempty_bar);   // (count 2) arrives when every MMA this thread has issued so far has completed
            if (mat == 0) {
              if (!mbar_wait(x_bar, n_x & 1u, s_abort, p.status)) return false;
              tc_fence_after();
              for (uint32_t a = 0; a < SPH; ++a) tc_cp_scales(t_sfb + 4u * a, smem_u32(s_sfb) + a * 512u);
              umma_commit(sfb_bar);   // the other issuer's MMAs read these scales too
            } else {
              if (!mbar_wait(sfb_bar, n_x & 1u, s_abort, p.status)) return false;
              tc_fence_after();
            }
            cur = img;
            ++n_x;
          }
          const uint32_t buf = seg & 1u;
          if (!mbar_wait(bar.tempty(buf), ((seg >> 1) & 1u) ^ 1u, s_abort, p.status)) return false;
          tc_fence_after();
          const uint32_t dacc = tmem + buf * 128u + mat * 64u;
          for (uint32_t s = 0; s < n; ++s, ++it) {
            const uint32_t slot = it % NS;
            if (!mbar_wait(bar.full(slot), (it / NS) & 1u, s_abort, p.status)) return false;
            tc_fence_copies();
            tc_fence_after();
            const uint32_t st = ring + slot * kTcStageA;
            tc_cp_scales(t_sf + slot * 4u, smem_u32(s_ring) + slot * kTcStageA + 16384u + mat * 512u);
#pragma unroll
            for (uint32_t step = 0; step < 2; ++step)
              tc_mma(dacc, tc_desc(st + step * 4096u, 2048u, 128u),
                     tc_desc(b_base + ((st0 + s) * 2u + step) * kTcStepB, kTcN * 16u, 128u), 2u * step, t_sf + slot * 4u,
                     t_sfb + 4u * (st0 + s), (s | step) ? 1u : 0u);
            umma_commit(bar.empty(slot));   // (count 2) the stage may be refilled once both issuers' MMAs have read it
          }
          umma_commit(bar.tfull(buf));
          ++seg;
          return true;
      });
    }
  } else {
    // ---- epilogue: thread = accumulator row (neuron of the tile) ----
    const int ew = warp & 3, row = ew * 32 + lane, et = (warp - kTcLW - 2) * 32 + lane;
    uint32_t seg = 0, nt_pass = 0xffffffffu;
    int nt = p.T;   // token columns of the pass in use
    // the hand-over buffers (partial sums, arrival counters, h images, pass counters) are free once the gate/up and
    // down kernels of the earlier calls have completed
    if (et == 0 && !(tc_wait_count(q.gen, q.expect_gu, p.status) && tc_wait_count(q.gen + 1, q.expect_dn, p.status))) *s_abort = 1;
    tc_epi_barrier();
    walk([&](uint32_t pass, uint32_t ng, uint32_t, uint32_t n) {
      const uint32_t buf = seg & 1u;
      if (!dense && pass != nt_pass) {
        const int item = w4_find_item(p.pref, n_items + n_zc, pass);
        nt = min(8, p.items[item].n_tok - (int)(pass - (uint32_t)p.pref[item]) * 8);
        nt_pass = pass;
      }
      bool ok = true;
      if (lane == 0) ok = mbar_wait(bar.tfull(buf), (seg >> 1) & 1u, s_abort, p.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (ok) {
        tc_fence_after();
        const uint32_t trow = tmem + buf * 128u + ((uint32_t)(ew * 32) << 16);
        float gsum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f}, usum[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        tc_row_sums(trow, gsum);
        tc_row_sums(trow + 64u, usum);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar.tempty(buf));
        float *hacc = p.hraw + ((size_t)pass * NBLK + 8u * ng + (uint32_t)(row >> 4)) * 256 + (row & 15);
        for (int t = 0; t < nt; ++t) {
          red_add_f32(hacc + t * 16, gsum[t]);
          red_add_f32(hacc + 128 + t * 16, usum[t]);
        }
        __threadfence();
      }
      tc_epi_barrier();
      if (et == 0) {
        // (one thread decides for all whether to go on, so that the 128 threads leave together)
        *s_stop = *s_abort;
        *s_last = 0;
        if (!*s_stop) {
          const int old = atomicAdd(p.hcount + pass * NG + ng, (int)n);
          *s_last = (old + (int)n == (int)KS) ? 1 : 0;
        }
      }
      tc_epi_barrier();
      if (*s_stop) return false;
      if (*s_last) {
        // this CTA's stages completed the group: h = SiLU(gate) * up, bit-sliced into the down kernel's operand
        __threadfence();
        const int tok = et >> 4, sub = et & 15;   // 8 neurons 8 sub .. 8 sub + 7 of the group, one token
        float *src = p.hraw + ((size_t)pass * NBLK + 8u * ng + (uint32_t)(sub >> 1)) * 256 + tok * 16 + (sub & 1) * 8;
        float h[8];
#pragma unroll
        for (int k4 = 0; k4 < 2; ++k4) {
          float4 *pg = reinterpret_cast<float4 *>(src) + k4, *pu = reinterpret_cast<float4 *>(src + 128) + k4;
          const float4 a = __ldcg(pg), b = __ldcg(pu);
          __stcg(pg, make_float4(0.f, 0.f, 0.f, 0.f));   // the sums start from zero in the next call
          __stcg(pu, make_float4(0.f, 0.f, 0.f, 0.f));
          h[4 * k4] = __fdividef(a.x, 1.f + __expf(-a.x)) * b.x;
          h[4 * k4 + 1] = __fdividef(a.y, 1.f + __expf(-a.y)) * b.y;
          h[4 * k4 + 2] = __fdividef(a.z, 1.f + __expf(-a.z)) * b.z;
          h[4 * k4 + 3] = __fdividef(a.w, 1.f + __expf(-a.w)) * b.w;
        }
        bool bad = false;
#pragma unroll
        for (int e = 0; e < 8; ++e) bad |= !(fabsf(h[e]) <= 3.0e38f);
        bad = (__shfl_xor_sync(0xffffffffu, (int)bad, 1) | __shfl_xor_sync(0xffffffffu, (int)bad, 2) | (int)bad) != 0;
        uint8_t *img = p.hq + (size_t)pass * tc_h_pass_bytes(p.inter);
        uint8_t *sf = img + (size_t)(p.inter / 64) * kTcStepB + (size_t)ng * 512;
        uint8_t *dst = img + (size_t)(2u * ng + (uint32_t)(sub >> 3)) * kTcStepB + ((sub >> 2) & 1) * (kTcN * 16) + tok * 16 + (sub & 3) * 4;
#pragma unroll
        for (int t = 0; t < kTcTerms; ++t) {
          uint32_t codes, sb;
          tc_term(h, bad, codes, sb);
          *reinterpret_cast<uint32_t *>(dst + t * 128) = codes;
          // the scale bytes of the token's four blocks (held by the lanes sub = 0, 4, 8, 12) leave as one word
          const int base = lane & 16;
          const uint32_t w4 = __shfl_sync(0xffffffffu, sb, base) | (__shfl_sync(0xffffffffu, sb, base + 4) << 8) |
                              (__shfl_sync(0xffffffffu, sb, base + 8) << 16) | (__shfl_sync(0xffffffffu, sb, base + 12) << 24);
          if (sub == 0) {
            const int nn = 8 * t + tok;
            *reinterpret_cast<uint32_t *>(sf + (nn & 31) * 16 + (nn >> 5) * 4) = w4;
          }
        }
        // publish: the down kernel starts a pass when all its groups are there (it does not wait for this grid to end)
        __threadfence();
        tc_epi_barrier();
        if (et == 0) {
          p.hcount[pass * NG + ng] = 0;
          atomicAdd(q.pass_done + pass, 1);
        }
      }
      ++seg;
      return true;
    });
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kTcLW) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  if (tid == 0) {
    __threadfence();
    atomicAdd(q.gen, 1);
  }
}

// Shared memory of the down kernel: activation image of the current pass and its scale atoms | ring | barriers |
// flags.
inline size_t tc_down_fixed_bytes(int inter) { return tc_h_pass_bytes(inter) + 64 * 8 + 64 + 128; }

__global__ void __launch_bounds__(kTcThreads, 1) tc_down_kernel(TcParams q) {
  const W4Params &p = q.w;
  const int d = q.d;
  const uint32_t NS = (uint32_t)q.n_stages;
  const uint32_t DS = (uint32_t)p.inter / 128u;        // stages (and scale atoms) of a tile
  const uint32_t CG = (uint32_t)d / 128u, NG = (uint32_t)p.inter / 128u, KSA = (uint32_t)d / 128u;
  const uint32_t h_bytes = (uint32_t)tc_h_pass_bytes(p.inter);
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char *s_b = smem;                                        // [2 DS steps][kTcStepB] | [DS][512]
  unsigned char *s_ring = s_b + h_bytes;
  uint64_t *s_bar = reinterpret_cast<uint64_t *>(s_ring + (size_t)NS * kTcStageD);
  uint32_t *s_tmem = reinterpret_cast<uint32_t *>(s_bar + 64);
  volatile int *s_abort = reinterpret_cast<volatile int *>(s_tmem + 1);
  __shared__ int s_final;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const TcBars bar{smem_u32(s_bar)};
  const uint32_t hfull_bar = bar.extra(0), hempty_bar = bar.extra(1), sfb_bar = bar.extra(2);
  if (tid == 0) {
    for (uint32_t s = 0; s < NS; ++s) { mbar_init(bar.full(s), 32); mbar_init(bar.empty(s), 1); }
    for (uint32_t b = 0; b < 2; ++b) { mbar_init(bar.tfull(b), 2); mbar_init(bar.tempty(b), 4); }
    mbar_init(hfull_bar, 1);
    mbar_init(hempty_bar, 2);
    mbar_init(sfb_bar, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  const int n_items = *p.n_items, n_zc = *p.n_zc;
  const bool dense = q.dense != 0;   // then pass = index into the list, see the gate/up kernel
  if (warp == kTcLW) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  // tensor memory columns: accumulators (buffer b: the even stages' at 128 b, the odd stages' at 128 b + 64) | weight
  // scales of the ring slots (4 s) | activation scales of the pass (4 per stage)
  const uint32_t t_sfa = tmem + 256u, t_sfb = tmem + 320u;
  const size_t sec_b = (size_t)NG * KSA * kTcStageA;   // the down section follows the gate/up section

  uint32_t pass0[2], s_begin[2], s_end[2];
  pass0[0] = 0u;
  pass0[1] = (uint32_t)p.pref[n_items];
  {
    const uint32_t t0 = pass0[1] * CG * DS, t1 = ((uint32_t)p.pref[n_items + n_zc] - pass0[1]) * CG * DS;
    s_begin[0] = w4_first(t0, gridDim.x, blockIdx.x); s_end[0] = w4_first(t0, gridDim.x, blockIdx.x + 1);
    s_begin[1] = w4_first(t1, gridDim.x, blockIdx.x); s_end[1] = w4_first(t1, gridDim.x, blockIdx.x + 1);
  }
  // body(pass, cg, st0, n): a run of n stages of tile (pass, column group cg), starting at stage st0
  auto walk = [&](auto body) {
    for (int r = 0; r < 2; ++r)
      for (uint32_t s = s_begin[r]; s < s_end[r];) {
        const uint32_t tile = s / DS, st0 = s - tile * DS, n = min(DS - st0, s_end[r] - s);
        if (!body(pass0[r] + tile / CG, tile % CG, st0, n)) return;
        s += n;
      }
  };

  if (warp < kTcLW) {
    // ---- loaders ----
    uint32_t it = 0, n_h = 0, cur = 0xffffffffu;
    walk([&](uint32_t pass, uint32_t cg, uint32_t st0, uint32_t n) {
      if (pass != cur && tid == 0) {
        // the pass's h image replaces the previous one once the MMAs that read that have completed (a wait that
        // gives up latches the abort flag: every loader then leaves at its next wait)
        if (!n_h || mbar_wait(hempty_bar, (n_h - 1u) & 1u, s_abort, p.status)) {
          // h of this pass is written by the gate/up kernel, which precedes this kernel in the stream and is at least
          // running (this kernel is its programmatic dependent): wait, bounded, for the pass's groups
          {
            const uint32_t limit = g_wait_polls;
            uint32_t polls = 0;
            int have;
            do {
              asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(have) : "l"(q.pass_done + pass) : "memory");
              if (have >= (int)NG) break;
              __nanosleep(64);
            } while (++polls < limit && !*s_abort);
            if (have < (int)NG && !*s_abort) {
              *s_abort = 1;
              atomicOr(p.status, kStatTimeout);
            }
            asm volatile("fence.proxy.async;" ::: "memory");   // the copies below read what those generic stores wrote
          }
          mbar_expect_tx(hfull_bar, h_bytes);
          const uint8_t *hsrc = p.hq + (size_t)pass * h_bytes;
          for (uint32_t o = 0; o < h_bytes; o += 16384u) bulk_g2s(smem_u32(s_b) + o, hsrc + o, min(16384u, h_bytes - o), hfull_bar);
          ++n_h;
        }
      }
      cur = pass;
      const int item = dense ? (int)pass : w4_find_item(p.pref, n_items + n_zc, pass);
      const uint8_t *src = p.items[item].w + sec_b + ((size_t)cg * DS + st0) * kTcStageD;
      for (uint32_t s = 0; s < n; ++s, ++it, src += kTcStageD) {
        const uint32_t slot = it % NS;
        if (it % (kTcLoaders / 32) == (uint32_t)warp) {
          bool ok = true;
          if (lane == 0) ok = mbar_wait(bar.empty(slot), ((it / NS) & 1u) ^ 1u, s_abort, p.status);
          if (!__shfl_sync(0xffffffffu, (int)ok, 0)) return false;
          tc_load_stage<kTcStageD>(smem_u32(s_ring) + slot * kTcStageD, src, lane, bar.full(slot));
        }
      }
      return true;
    });
    asm volatile("cp.async.wait_all;" ::: "memory");
    if (tid == 0) {
      if (n_h) (void)mbar_wait(hfull_bar, (n_h - 1u) & 1u, s_abort, p.status);
      abort_drain(s_abort);
    }
  } else if (warp <= kTcLW + 1) {
    if (lane == 0) {
      // ---- MMA issuers: the first warp takes the stages of even ring index, the second the odd ones ----
      const uint32_t me = (uint32_t)(warp - kTcLW);
      uint32_t it = 0, seg = 0, n_h = 0, cur = 0xffffffffu;
      const uint32_t b_base = smem_u32(s_b);
      walk([&](uint32_t pass, uint32_t, uint32_t st0, uint32_t n) {
        if (pass != cur) {
          if (n_h) umma_commit(hempty_bar);   // (count 2) arrives when every MMA this thread has issued so far has completed
          if (me == 0) {
            if (!mbar_wait(hfull_bar, n_h & 1u, s_abort, p.status)) return false;
            tc_fence_after();
            for (uint32_t a = 0; a < DS; ++a) tc_cp_scales(t_sfb + 4u * a, b_base + 2u * DS * kTcStepB + a * 512u);
            umma_commit(sfb_bar);
          } else {
            if (!mbar_wait(sfb_bar, n_h & 1u, s_abort, p.status)) return false;
            tc_fence_after();
          }
          cur = pass;
          ++n_h;
        }
        const uint32_t buf = seg & 1u;
        if (!mbar_wait(bar.tempty(buf), ((seg >> 1) & 1u) ^ 1u, s_abort, p.status)) return false;
        tc_fence_after();
        const uint32_t dacc = tmem + buf * 128u + me * 64u;
        uint32_t mine = 0;
        for (uint32_t s = 0; s < n; ++s, ++it) {
          if ((it & 1u) != me) continue;
          const uint32_t slot = it % NS;
          if (!mbar_wait(bar.full(slot), (it / NS) & 1u, s_abort, p.status)) return false;
          tc_fence_copies();
          tc_fence_after();
          const uint32_t st = smem_u32(s_ring) + slot * kTcStageD;
          tc_cp_scales(t_sfa + slot * 4u, st + 8192u);
#pragma unroll
          for (uint32_t step = 0; step < 2; ++step)
            tc_mma(dacc, tc_desc(st + step * 4096u, 2048u, 128u), tc_desc(b_base + ((st0 + s) * 2u + step) * kTcStepB, kTcN * 16u, 128u),
                   2u * step, t_sfa + slot * 4u, t_sfb + 4u * (st0 + s), (mine | step) ? 1u : 0u);
          ++mine;
          umma_commit(bar.empty(slot));
        }
        umma_commit(bar.tfull(buf));   // (count 2; immediate for an issuer without a stage in this run)
        ++seg;
        return true;
      });
    }
  } else {
    // ---- epilogue: thread = output column of the tile ----
    const int ew = warp & 3, row = ew * 32 + lane;
    uint32_t seg = 0, it = 0, gw_pass = 0xffffffffu;
    TcPassTokens pt;
    // the output accumulator is free once the down kernels of the earlier calls (their last CTA rounds and clears it)
    // have completed
    if (warp == kTcLW + 2 && lane == 0 && !tc_wait_count(q.gen + 1, q.expect_dn, p.status)) *s_abort = 1;
    tc_epi_barrier();
    walk([&](uint32_t pass, uint32_t cg, uint32_t, uint32_t n) {
      const uint32_t buf = seg & 1u;
      if (pass != gw_pass) {
        // the tokens of the pass's columns and their gate weights; a CTA's tiles mostly belong to one pass, so these
        // dependent loads are rare
        gw_pass = pass;
        tc_pass_tokens(p, dense, pass, true, pt);
      }
      bool ok = true;
      if (lane == 0) ok = mbar_wait(bar.tfull(buf), (seg >> 1) & 1u, s_abort, p.status);
      ok = __shfl_sync(0xffffffffu, (int)ok, 0) != 0;
      if (!ok) return false;
      tc_fence_after();
      // the run's stages it .. it+n-1 went alternately to the two issuers: add the accumulators that were written
      const bool has_even = n >= 2u || (it & 1u) == 0u, has_odd = n >= 2u || (it & 1u) == 1u;
      float v[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      const uint32_t trow = tmem + buf * 128u + ((uint32_t)(ew * 32) << 16);
      if (has_even) tc_row_sums(trow, v);
      if (has_odd) tc_row_sums(trow + 64u, v);
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar.tempty(buf));
      float *yc = p.y_acc + 128u * cg + row;
#pragma unroll
      for (int t = 0; t < 8; ++t)
        if (pt.tok[t] >= 0) red_add_f32(yc + (size_t)pt.tok[t] * d, pt.w[t] * v[t]);
      it += n;
      ++seg;
      return true;
    });
  }
  tc_fence_before();
  __syncthreads();
  if (warp == kTcLW) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");

  // ---- the last CTA to finish clears the passes' hand-over counters and, unless a finalize launch follows (more
  // than 16 tokens), rounds the accumulator to bf16 and clears it ----
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const uint32_t prev = atomicAdd(p.done, 1u);
    s_final = (prev == gridDim.x - 1);
  }
  __syncthreads();
  if (!s_final) {
    if (tid == 0) atomicAdd(q.gen + 1, 1);   // (after the fence above: this CTA's adds are visible)
    return;
  }
  __threadfence();
  const int n4 = p.finalize ? p.T * (d / 4) : 0;
  for (int i = tid; i < n4; i += kTcThreads) {
    const float4 v = __ldcg(reinterpret_cast<const float4 *>(p.y_acc) + i);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b2 = __floats2bfloat162_rn(v.z, v.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t *>(&a);
    o.y = *reinterpret_cast<uint32_t *>(&b2);
    reinterpret_cast<uint2 *>(p.y)[i] = o;
    reinterpret_cast<float4 *>(p.y_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
  for (int i = tid; i < p.pref[n_items + n_zc]; i += kTcThreads) q.pass_done[i] = 0;
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    *p.done = 0u;
    __threadfence();
    atomicAdd(q.gen + 1, 1);
  }
}

}  // namespace ftmoe
