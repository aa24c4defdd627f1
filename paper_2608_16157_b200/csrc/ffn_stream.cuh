// Steps 5+6 for bf16 experts at decode-sized token counts: an HBM-streaming SwiGLU FFN whose weight loads go
// straight from global memory into tensor-core fragments.
//
// The record is stored in tile order (include/ftmoe.h): a warp's 16-byte (gate/up) or 8-byte (down) accesses of one
// tile cover 512 / 256 contiguous bytes, every quarter warp one whole 128-byte line, and the loaded words ARE the A
// fragments of mma.sync.m16n8k16, so there is no ldmatrix, no transposition and no producer warp.  One persistent
// CTA of 16 warps per SM walks a contiguous range of 16-neuron units (96*d bytes each: gate, up, down part):
//   gate/up : warp w owns the hidden slice [w*d/16, (w+1)*d/16); [16 neurons x 8 tokens] partial sums are reduced
//             across warps through shared memory, then h = SiLU(g) * u (rounded to bf16).
//   down    : warp w owns the output columns [w*d/16, (w+1)*d/16); A = the unit's 16 x 16 tiles of W_down^T,
//             B = h; fp32 accumulators persist across the CTA's units of one (expert, pass).
// Tokens sit in the N dimension of the MMA (8 per group), so the arithmetic does not grow with the token count.
// Every part has a buffer of its own that is refilled with the next unit's part as soon as it has been consumed:
// gate and up parts go straight into registers (two buffers of 16-byte loads), the down part is copied by
// cp.async into shared memory, each warp its own 16-column tiles.  So ~190 KB per SM are in flight and every load
// has about one unit's time to arrive, also across the barriers of the reduction.
// The gate-weighted combine is a red.global.add into the fp32 [T][d] accumulator; the last CTA to finish rounds
// it once to bf16 and clears it.  Records in the mapped host pool (zero-copy experts) stream through the same
// loads; since they must cross the host link only once, all token groups of such an expert are served from one
// pass (up to kFsMaxGroups groups) and the partial outputs are flushed per unit.
#pragma once
#include "async.cuh"
#include "common.cuh"

namespace ftmoe {

constexpr int kFsThreads = 512;
constexpr int kFsWarps = 16;
constexpr int kFsTokens = 8;       // tokens per group = N of the MMA
constexpr int kFsMaxGroups = 2;    // token groups one pass can serve
constexpr int kFsResTokensPerPass = kFsTokens;                 // HBM-resident records: accumulators stay in registers
constexpr int kFsZcTokensPerPass = kFsTokens * kFsMaxGroups;   // host-resident records: one link pass for 16 tokens

struct FfnStreamParams {
  const WorkItem *items;
  const int32_t *n_items;   // resident items (records in HBM slots): [hits][shared expert][fills]
  const int32_t *n_hit;     // how many of them lead the list and do not depend on this step's fills
  int part;                 // 0: everything; 1: hits + zero-copy items; 2: fills only
  const int32_t *n_zc;      // zero-copy items appended after them (records in the mapped host pool)
  const int32_t *pref;      // [n_items+n_zc+1] exclusive prefix of the weight passes per item (from the plan)
  const __nv_bfloat16 *x;   // [T][d]
  const int32_t *perm;
  const float *topk_w;
  float *y_acc;             // [T][d]
  __nv_bfloat16 *y;         // [T][d], written by the last CTA when finalize != 0
  uint32_t *done;           // CTA completion counter, zero between launches
  uint32_t *status;
  int inter, top_k, T, finalize;
  int max_items;            // capacity of items / pref (entries beyond the counts are ignored)
  int overlap;              // programmatic dependent launch: 0 = plain launch; 1 = the grid may be scheduled while the
                            // preceding kernel of the stream still runs and waits for it before reading anything;
                            // 2 = it waits only before its first write to y_acc (inputs must already be final)
  long long *trace;         // optional [gridDim.x][4]: start and end of the CTA's streaming (global timer, ns), 0, 0
                            // (the finalizing CTA stores minus its finish time in the last field); or nullptr
};

// Dynamic shared memory: red [groups][16 warps][2][16 x 8] f32 | h [groups][8][16] bf16 | tok, gw [16] |
// x [8][d + 32] bf16 | down part of the current unit [32 d bytes] | items [max_items] | pref [max_items + 1].
inline size_t ffn_stream_smem_bytes(int max_items, int d) {
  return (size_t)kFsMaxGroups * kFsWarps * 2 * 128 * 4 + kFsMaxGroups * 128 * 2 + kFsZcTokensPerPass * 8 +
         (size_t)kFsTokens * (2 * d + 64) + 32 * (size_t)d + (size_t)max_items * sizeof(WorkItem) +
         ((size_t)max_items + 1) * 4 + 16;
}

__device__ __forceinline__ void red_add_f32(float *addr, float v) {
  asm volatile("red.global.add.f32 [%0], %1;" ::"l"(addr), "f"(v) : "memory");
}

// y = bf16(y_acc), y_acc = 0 over the whole grid: the output rounding of calls with many tokens, where one CTA (the
// last one of the streaming kernel) would take longer than a launch of its own.
static __global__ void __launch_bounds__(256) finalize_kernel(float *y_acc, __nv_bfloat16 *y, int n4) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += gridDim.x * blockDim.x) {
    const float4 v = __ldcg(reinterpret_cast<const float4 *>(y_acc) + i);
    __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 o;
    o.x = *reinterpret_cast<uint32_t *>(&a);
    o.y = *reinterpret_cast<uint32_t *>(&b);
    reinterpret_cast<uint2 *>(y)[i] = o;
    reinterpret_cast<float4 *>(y_acc)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
  }
}

template <int DB>  // DB = d / 256
__global__ void __launch_bounds__(kFsThreads, 1) ffn_stream_kernel(FfnStreamParams p) {
  constexpr int KT = (DB >= 2) ? DB / 2 : 1;   // 16 x 32 gate/up tiles per active warp
  constexpr int NWK = (DB * 8) / KT;           // warps that take part in gate/up (all 16 unless d = 256)
  constexpr int CTW = DB;                      // 16-column down tiles per warp
  constexpr int d = 256 * DB;
  constexpr uint32_t kPart = 32u * d, kUnit = 96u * d;
  constexpr uint32_t kXStride = 2u * d + 64u;   // = 64 mod 128: conflict-free 16-byte fragment loads
  extern __shared__ __align__(128) unsigned char smem[];
  float *s_red = reinterpret_cast<float *>(smem);
  __nv_bfloat16 *s_h = reinterpret_cast<__nv_bfloat16 *>(smem + (size_t)kFsMaxGroups * kFsWarps * 2 * 128 * 4);
  int32_t *s_tok = reinterpret_cast<int32_t *>(s_h + kFsMaxGroups * 128);
  float *s_gw = reinterpret_cast<float *>(s_tok + kFsZcTokensPerPass);
  unsigned char *s_x = reinterpret_cast<unsigned char *>(s_gw + kFsZcTokensPerPass);
  unsigned char *s_d = s_x + kFsTokens * kXStride;   // the current unit's down part, byte for byte
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_d + kPart);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  if (p.trace != nullptr && tid == 0) {
    long long t_start;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_start));
    p.trace[4 * blockIdx.x] = t_start;
  }
  // The next kernel of the stream, if it was launched as a programmatic dependent, may be scheduled as soon as an SM
  // has room for one of its CTAs, i.e. when one of this grid's CTAs has finished (what it may touch before this
  // grid has completed is its own business: see `overlap`).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (p.overlap == 1) asm volatile("griddepcontrol.wait;" ::: "memory");
  bool dep_waited = p.overlap != 2;
  const int n_items = *p.n_items;
  const int n_zc = *p.n_zc;
  const int n_hit = (p.part == 0) ? 0 : *p.n_hit;
  const bool dense = p.T <= kFsTokens;   // MMA column j is token j: the x rows are staged once per CTA
  // x rows of the MMA columns into shared memory (16 bytes per thread and step); zeros for absent columns
  auto stage_x = [&](auto tok_of_column) {
    for (int i = tid; i < kFsTokens * (d / 8); i += kFsThreads) {
      const int j = i / (d / 8), c8 = i - j * (d / 8);
      const int tok = tok_of_column(j);
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (tok >= 0) v = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 8 * c8);
      *reinterpret_cast<uint4 *>(s_x + j * kXStride + 16 * c8) = v;
    }
  };
  // the work list and the prefix of its weight passes, up to the lists' capacity so that these loads do not wait
  // for the counts
  for (int i = tid; i <= p.max_items; i += kFsThreads) s_pref[i] = p.pref[i];
  {
    const uint4 *src = reinterpret_cast<const uint4 *>(p.items);
    uint4 *dst = reinterpret_cast<uint4 *>(s_items);
    static_assert(sizeof(WorkItem) == 32, "WorkItem is copied as two 16-byte words");
    for (int i = tid; i < 2 * p.max_items; i += kFsThreads) dst[i] = src[i];
  }
  __syncthreads();
  const uint32_t NBLK = (uint32_t)p.inter / 16u;

  // ---- per-lane constants of the loads ----
  // gate/up: tile kb = warp*KT + t; row g, chunk q of the 64-byte row (stored at position q ^ (g >> 1))
  const uint32_t gu_off = (uint32_t)(warp * KT) * 1024u + g * 64u + ((q ^ (g >> 1)) * 16u);
  // down: this warp's CTW tiles of 512 bytes are copied as they are into the same place of s_d ...
  const uint32_t d_off = (uint32_t)(warp * CTW) * 512u + lane * 16u;
  const uint32_t my_d = smem_u32(s_d) + d_off;
  // ... and read back as A fragments: column row g (and g + 8), neurons 4q..4q+3 = half (q & 1) of chunk (q >> 1)
  const uint32_t my_dfrag =
      smem_u32(s_d) + (uint32_t)(warp * CTW) * 512u + g * 32u + (((q >> 1) ^ (g >> 2)) * 16u) + (q & 1) * 8u;
  const uint32_t my_x = smem_u32(s_x) + g * kXStride + (uint32_t)(warp * KT) * 64u + 16u * q;
  const bool gu_warp = (NWK == kFsWarps) || warp < NWK;

  uint4 bufg[2 * KT], bufu[2 * KT];
  auto load_gu = [&](uint4 (&buf)[2 * KT], const uint8_t *part) {
    if (gu_warp) {
#pragma unroll
      for (int t = 0; t < KT; ++t) {
        buf[2 * t] = ld_stream_16(part + gu_off + t * 1024);
        buf[2 * t + 1] = ld_stream_16(part + gu_off + t * 1024 + 512);
      }
    }
  };
  auto load_d = [&](const uint8_t *part) {   // only this warp reads the region: warp-level synchronisation suffices
#pragma unroll
    for (int c = 0; c < CTW; ++c)
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(my_d + c * 512), "l"(part + d_off + c * 512) : "memory");
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  auto load_unit = [&](const uint8_t *unit) {
    load_gu(bufg, unit);
    load_gu(bufu, unit + kPart);
    load_d(unit + 2 * kPart);
  };

  // partial [16 neurons x 8 tokens] sums of one part over this warp's hidden slice -> shared memory
  // (x fragments of MMA column g: from the staged rows, or -- tok != -2 -- straight from global memory, zeros if tok < 0)
  auto gu_part = [&](const uint4 (&buf)[2 * KT], float *r, int tok) {
    if (gu_warp) {
      float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};   // two chains: consecutive MMAs do not wait
#pragma unroll
      for (int t = 0; t < KT; ++t) {
        uint4 xv = make_uint4(0u, 0u, 0u, 0u);
        if (tok == -2) xv = lds_v4(my_x + 64u * t);
        else if (tok >= 0) xv = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 32 * (warp * KT + t) + 8 * q);
        mma_bf16(c1, buf[2 * t].x, buf[2 * t + 1].x, buf[2 * t].y, buf[2 * t + 1].y, xv.x, xv.y);
        mma_bf16(c2, buf[2 * t].z, buf[2 * t + 1].z, buf[2 * t].w, buf[2 * t + 1].w, xv.z, xv.w);
      }
      *reinterpret_cast<float2 *>(r + g * 8 + 2 * q) = make_float2(c1[0] + c2[0], c1[1] + c2[1]);
      *reinterpret_cast<float2 *>(r + (g + 8) * 8 + 2 * q) = make_float2(c1[2] + c2[2], c1[3] + c2[3]);
    }
  };
  // h = SiLU(sum gate) * (sum up), bf16, [group][token][neuron]: four threads per value, each sums a quarter of the
  // warps' partial sums
  auto reduce_h = [&](int ngroups) {
    const int r = tid >> 2, qu = tid & 3;   // r = neuron * 8 + token
    for (int grp = 0; grp < ngroups; ++grp) {
      const float *base = s_red + (size_t)grp * kFsWarps * 2 * 128 + r;
      float a = 0.f, c = 0.f;
#pragma unroll
      for (int w = 0; w < NWK / 4; ++w) {
        a += base[((qu * (NWK / 4) + w) * 2 + 0) * 128];
        c += base[((qu * (NWK / 4) + w) * 2 + 1) * 128];
      }
      a += __shfl_xor_sync(0xffffffffu, a, 1);
      c += __shfl_xor_sync(0xffffffffu, c, 1);
      a += __shfl_xor_sync(0xffffffffu, a, 2);
      c += __shfl_xor_sync(0xffffffffu, c, 2);
      if (qu == 0) s_h[grp * 128 + (r & 7) * 16 + (r >> 3)] = __float2bfloat16_rn(__fdividef(a, 1.f + __expf(-a)) * c);
    }
  };
  float dacc[CTW][4];
  auto down_part = [&](int grp) {
    const uint2 hb = *reinterpret_cast<const uint2 *>(s_h + grp * 128 + g * 16 + 4 * q);
#pragma unroll
    for (int cc = 0; cc < CTW; ++cc) {
      uint2 lo, hi;
      asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(lo.x), "=r"(lo.y) : "r"(my_dfrag + cc * 512));
      asm volatile("ld.shared.v2.u32 {%0,%1}, [%2];" : "=r"(hi.x), "=r"(hi.y) : "r"(my_dfrag + cc * 512 + 256));
      mma_bf16(dacc[cc], lo.x, hi.x, lo.y, hi.y, hb.x, hb.y);
    }
  };
  // gate-weighted combine of the accumulators: D fragment = [column g / g+8 of the tile][MMA columns 2q, 2q+1]
  auto flush = [&](int tok_a, float gw_a, int tok_b, float gw_b) {
    if (!dep_waited) {   // the preceding kernel's last writes to y_acc (its finalize) are ordered before ours
      asm volatile("griddepcontrol.wait;" ::: "memory");
      dep_waited = true;
    }
    float *ya = p.y_acc + (size_t)(tok_a < 0 ? 0 : tok_a) * d + 16 * (warp * CTW) + g;
    float *yb = p.y_acc + (size_t)(tok_b < 0 ? 0 : tok_b) * d + 16 * (warp * CTW) + g;
#pragma unroll
    for (int cc = 0; cc < CTW; ++cc) {
      if (tok_a >= 0) {
        red_add_f32(ya + 16 * cc, gw_a * dacc[cc][0]);
        red_add_f32(ya + 16 * cc + 8, gw_a * dacc[cc][2]);
      }
      if (tok_b >= 0) {
        red_add_f32(yb + 16 * cc, gw_b * dacc[cc][1]);
        red_add_f32(yb + 16 * cc + 8, gw_b * dacc[cc][3]);
      }
    }
  };
  auto zero_dacc = [&]() {
#pragma unroll
    for (int cc = 0; cc < CTW; ++cc) { dacc[cc][0] = dacc[cc][1] = dacc[cc][2] = dacc[cc][3] = 0.f; }
  };

  // ---- this CTA's share of the two work ranges ----
  // HBM-resident units, then host-resident units (bound by the host link, so every CTA takes an equal share of
  // them), each split evenly over the CTAs.  `part` restricts the launch to the items that do not depend on the
  // fills (plus the zero-copy items) or to the filled items.
  auto share = [&](uint32_t total, uint32_t &first, uint32_t &count) {   // CTA i: total/grid units, the first total%grid CTAs one more
    const uint32_t per = total / gridDim.x, rem = total - per * gridDim.x;
    first = blockIdx.x * per + min((uint32_t)blockIdx.x, rem);
    count = per + (blockIdx.x < rem ? 1u : 0u);
  };
  const int a0 = (p.part == 2) ? n_hit : 0, a1 = (p.part == 1) ? n_hit : n_items;
  uint32_t rfirst0, rcount0, rfirst1, rcount1;
  share((uint32_t)(s_pref[a1] - s_pref[a0]) * NBLK, rfirst0, rcount0);
  rfirst0 += (uint32_t)s_pref[a0] * NBLK;
  share((p.part == 2) ? 0u : (uint32_t)(s_pref[n_items + n_zc] - s_pref[n_items]) * NBLK, rfirst1, rcount1);
  rfirst1 += (uint32_t)s_pref[n_items] * NBLK;

  // Segments (this CTA's units of one (item, pass)) in order; the loads of a segment's first unit are issued by
  // the previous segment's last step (or right here for the very first one).
  struct Seg { const uint8_t *unit0; int item, pass, n_units, zc; };
  int range = 0, item = 0;
  uint32_t pu = 0, b = 0, left = 0;
  auto next_segment = [&](Seg &s) -> bool {   // false when the CTA's work is exhausted
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
    s.unit0 = s_items[item].w + (size_t)b * kUnit;
    s.zc = range - 1;
    left -= s.n_units;
    ++pu;
    b = 0;
    return true;
  };

  Seg sg, nsg;
  bool more = next_segment(sg);
  if (more) load_unit(sg.unit0);
  if (dense) {   // staged while the first unit's loads are in flight
    stage_x([&](int j) { return j < p.T ? j : -1; });
    __syncthreads();
  }

  while (more) {
    more = next_segment(nsg);
    const uint8_t *after = more ? nsg.unit0 : nullptr;   // the unit that follows this segment's last one
    const WorkItem &it = s_items[sg.item];
    const int tpp = sg.zc ? kFsZcTokensPerPass : kFsResTokensPerPass;
    const int tok0 = sg.pass * tpp;
    const int ntok = min(tpp, it.n_tok - tok0);
    if (ntok <= kFsTokens) {
      // ---------------- one token group: accumulators persist over the segment ----------------
      int my_tok = -1;      // lane i < ntok: token and gate weight of the pass's i-th pair
      float my_w = 0.f;
      if (lane < ntok) {
        if (it.expert >= 0) {
          const int pr = p.perm[it.off + tok0 + lane];
          my_tok = pr / p.top_k;
          my_w = p.topk_w[pr];
        } else {
          my_tok = tok0 + lane;
          my_w = 1.f;
        }
      }
      if (!dense) {   // MMA column j is the pass's j-th pair: stage those tokens' rows
        // (the previous segment's readers of s_x are past the barriers of their last unit)
        const int off_ = it.off + tok0, expert_ = it.expert;
        stage_x([&](int j) {
          if (j >= ntok) return -1;
          return expert_ >= 0 ? p.perm[off_ + j] / p.top_k : tok0 + j;
        });
        __syncthreads();
      }
      zero_dacc();
      const uint8_t *unit = sg.unit0;
      for (int k = 0; k < sg.n_units; ++k, unit += kUnit) {
        const uint8_t *nunit = (k + 1 < sg.n_units) ? unit + kUnit : after;
        gu_part(bufg, s_red + (warp * 2 + 0) * 128, -2);
        if (nunit) load_gu(bufg, nunit);
        gu_part(bufu, s_red + (warp * 2 + 1) * 128, -2);
        if (nunit) load_gu(bufu, nunit + kPart);
        __syncthreads();
        reduce_h(1);
        asm volatile("cp.async.wait_group 0;" ::: "memory");   // this lane's copies of the down part have landed
        __syncthreads();                                        // h is complete (and so are the other lanes' copies)
        down_part(0);
        __syncwarp();   // every lane has read its fragments: the region may be overwritten
        if (nunit) load_d(nunit + 2 * kPart);
      }
      // combine
      int tok_a, tok_b;
      float gw_a, gw_b;
      if (dense) {   // MMA column j is token j: find the pairs (if any) of tokens 2q and 2q+1
        tok_a = tok_b = -1;
        gw_a = gw_b = 0.f;
        for (int i = 0; i < ntok; ++i) {
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
      flush(tok_a, gw_a, tok_b, gw_b);
    } else {
      // ---------------- several token groups from one pass over the record: flush per unit ----------------
      const int ngroups = (ntok + kFsTokens - 1) / kFsTokens;
      __syncthreads();   // the previous segment's readers of s_tok / s_gw are done
      if (tid < kFsZcTokensPerPass) {
        int tk = -1;
        float w = 0.f;
        if (tid < ntok) {
          if (it.expert >= 0) {
            const int pr = p.perm[it.off + tok0 + tid];
            tk = pr / p.top_k;
            w = p.topk_w[pr];
          } else {
            tk = tok0 + tid;
            w = 1.f;
          }
        }
        s_tok[tid] = tk;
        s_gw[tid] = w;
      }
      __syncthreads();
      const uint8_t *unit = sg.unit0;
      for (int k = 0; k < sg.n_units; ++k, unit += kUnit) {
        const uint8_t *nunit = (k + 1 < sg.n_units) ? unit + kUnit : after;
        for (int which = 0; which < 2; ++which) {
          for (int grp = 0; grp < ngroups; ++grp) {
            const int tok = s_tok[grp * kFsTokens + g];   // x fragments straight from global memory
            float *r = s_red + (((size_t)grp * kFsWarps + warp) * 2 + which) * 128;
            if (which == 0) gu_part(bufg, r, tok); else gu_part(bufu, r, tok);
          }
          if (nunit) { if (which == 0) load_gu(bufg, nunit); else load_gu(bufu, nunit + kPart); }
        }
        __syncthreads();
        reduce_h(ngroups);
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
        for (int grp = 0; grp < ngroups; ++grp) {
          zero_dacc();
          down_part(grp);
          const int ia = grp * kFsTokens + 2 * q;
          flush(s_tok[ia], s_gw[ia], s_tok[ia + 1], s_gw[ia + 1]);
        }
        __syncwarp();
        if (nunit) load_d(nunit + 2 * kPart);
      }
    }
    sg = nsg;
  }

  if (!dep_waited) asm volatile("griddepcontrol.wait;" ::: "memory");   // (a CTA without work still orders its exit)
  if (p.trace != nullptr && tid == 0) {
    long long *tr = p.trace + 4 * blockIdx.x;
    long long t_end;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_end));
    tr[1] = t_end; tr[2] = 0; tr[3] = 0;
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
  // several independent L2 loads in flight per thread: the round trips overlap instead of adding up
  for (int i0 = tid; i0 < n4; i0 += 8 * kFsThreads) {
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int i = i0 + j * kFsThreads;
      v[j] = (i < n4) ? __ldcg(reinterpret_cast<const float4 *>(p.y_acc) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int i = i0 + j * kFsThreads;
      if (i < n4) {
        __nv_bfloat162 a = __floats2bfloat162_rn(v[j].x, v[j].y), b2 = __floats2bfloat162_rn(v[j].z, v[j].w);
        uint2 o;
        o.x = *reinterpret_cast<uint32_t *>(&a);
        o.y = *reinterpret_cast<uint32_t *>(&b2);
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

}  // namespace ftmoe
