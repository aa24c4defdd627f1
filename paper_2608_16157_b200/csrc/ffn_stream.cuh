// Steps 5+6 for bf16 experts at decode-sized token counts: an HBM-streaming SwiGLU FFN whose weight loads go
// straight from global memory into tensor-core fragments.
//
// The record is stored in tile order (include/ftmoe.h): a warp's 16-byte (gate/up) or 8-byte (down) loads of one
// tile are contiguous 512 / 256 bytes and the loaded registers ARE the A fragments of mma.sync.m16n8k16, so there
// is no shared-memory staging, no ldmatrix and no producer warp.  One persistent CTA of 16 warps per SM walks a
// contiguous range of 16-neuron units (96*d bytes each: gate part, up part, down part):
//   gate/up : warp w owns the hidden slice [w*d/16, (w+1)*d/16); [16 neurons x 8 tokens] partial sums are reduced
//             across warps through shared memory, then h = SiLU(g) * u (rounded to bf16).
//   down    : warp w owns the output columns [w*d/16, (w+1)*d/16); A = the unit's 16 x 16 tiles of W_down^T,
//             B = h; fp32 accumulators persist across the CTA's units of one (expert, pass).
// Tokens sit in the N dimension of the MMA (8 per group), so the arithmetic does not grow with the token count.
// The loads are software-pipelined over two register buffers in the order gate, up, down: while one part is being
// consumed the next one (of this unit or the next) is in flight, also across the barriers of the reduction.
// The gate-weighted combine is a red.global.add into the fp32 [T][d] accumulator; the last CTA to finish rounds
// it once to bf16 and clears it.  Records in the mapped host pool (zero-copy experts) stream through the same
// loads; since they must cross the host link only once, all token groups of such an expert are served from the
// registers of one pass (up to kFsMaxGroups groups) and the partial outputs are flushed per unit.
#pragma once
#include <type_traits>

#include "async.cuh"
#include "common.cuh"

namespace ftmoe {

constexpr int kFsThreads = 512;
constexpr int kFsWarps = 16;
constexpr int kFsTokens = 8;       // tokens per group = N of the MMA
constexpr int kFsMaxGroups = 4;    // token groups one pass can serve from the registers
constexpr int kFsResTokensPerPass = kFsTokens;                 // HBM-resident records: accumulators stay in registers
constexpr int kFsZcTokensPerPass = kFsTokens * kFsMaxGroups;   // host-resident records: one link pass for 32 tokens

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
  long long *trace;         // optional [gridDim.x][4]: start and end of the CTA's streaming (global timer, ns), units
                            // streamed, 0 (the finalizing CTA stores minus its finish time there); or nullptr
};

// Dynamic shared memory: red [groups][16 warps][2][16 x 8] f32 | h [groups][8][16] bf16 | tok [32] | gw [32] |
// x [8][d + 32] bf16 | items [max_items] | pref [max_items + 1].
inline size_t ffn_stream_smem_bytes(int max_items, int d) {
  return (size_t)kFsMaxGroups * kFsWarps * 2 * 128 * 4 + kFsMaxGroups * 128 * 2 + kFsZcTokensPerPass * 8 +
         (size_t)kFsTokens * (2 * d + 64) + (size_t)max_items * sizeof(WorkItem) + ((size_t)max_items + 1) * 4 + 16;
}

template <int DB>  // DB = d / 256
__global__ void __launch_bounds__(kFsThreads, 1) ffn_stream_kernel(FfnStreamParams p) {
  constexpr int KT = (DB >= 2) ? DB / 2 : 1;   // 16 x 32 gate/up tiles per active warp
  constexpr int NWK = (DB * 8) / KT;           // warps that take part in gate/up (all 16 unless d = 256)
  constexpr int CTW = DB;                      // 16-column down tiles per warp
  constexpr int NB = (2 * KT > CTW) ? 2 * KT : CTW;   // 16-byte registers of one buffer
  constexpr int d = 256 * DB;
  constexpr uint32_t kPart = 32u * d, kUnit = 96u * d;
  constexpr uint32_t kXStride = 2u * d + 64u;   // = 64 mod 128: conflict-free 16-byte fragment loads
  extern __shared__ __align__(128) unsigned char smem[];
  float *s_red = reinterpret_cast<float *>(smem);
  __nv_bfloat16 *s_h = reinterpret_cast<__nv_bfloat16 *>(smem + (size_t)kFsMaxGroups * kFsWarps * 2 * 128 * 4);
  int32_t *s_tok = reinterpret_cast<int32_t *>(s_h + kFsMaxGroups * 128);
  float *s_gw = reinterpret_cast<float *>(s_tok + kFsZcTokensPerPass);
  unsigned char *s_x = reinterpret_cast<unsigned char *>(s_gw + kFsZcTokensPerPass);
  WorkItem *s_items = reinterpret_cast<WorkItem *>(s_x + kFsTokens * kXStride);
  int32_t *s_pref = reinterpret_cast<int32_t *>(s_items + p.max_items);
  __shared__ int s_last;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, q = lane & 3;
  if (p.trace != nullptr && tid == 0) {
    long long t_start;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_start));
    p.trace[4 * blockIdx.x] = t_start;
  }
  int trace_units = 0;
  const int n_items = *p.n_items;
  const int n_zc = *p.n_zc;
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
  if (dense) stage_x([&](int j) { return j < p.T ? j : -1; });
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
  const int NBLK = p.inter / 16;
  // two work ranges, each split evenly over the CTAs: HBM-resident units, then host-resident units (the latter
  // are bound by the host link, so every CTA takes an equal share of them).  `part` restricts the launch to the
  // items that do not depend on the fills (plus the zero-copy items) or to the filled items.
  const int n_hit = (p.part == 0) ? 0 : *p.n_hit;
  const int a0 = (p.part == 2) ? n_hit : 0, a1 = (p.part == 1) ? n_hit : n_items;
  long long rb0, rb1;   // first unit of this CTA in the two ranges
  int rn0, rn1;         // and how many
  {
    const long long first_res = (long long)s_pref[a0] * NBLK, total_res = (long long)s_pref[a1] * NBLK;
    const long long zc_begin = (long long)s_pref[n_items] * NBLK;
    const long long total_all = (p.part == 2) ? zc_begin : (long long)s_pref[n_items + n_zc] * NBLK;
    rb0 = first_res + (total_res - first_res) * blockIdx.x / gridDim.x;
    rn0 = (int)(first_res + (total_res - first_res) * (blockIdx.x + 1) / gridDim.x - rb0);
    rb1 = zc_begin + (total_all - zc_begin) * blockIdx.x / gridDim.x;
    rn1 = (int)(zc_begin + (total_all - zc_begin) * (blockIdx.x + 1) / gridDim.x - rb1);
  }
  // A cursor over this CTA's units: (range, flattened pass index, unit inside the pass, item).
  struct Cur { int range, b, item, pu, left; };
  auto cur_enter = [&](Cur &c) {   // positions at the start of range c.range, skipping empty ranges
    while (c.range < 2) {
      const long long u = c.range ? rb1 : rb0;
      c.left = c.range ? rn1 : rn0;
      if (c.left > 0) {
        c.pu = (int)(u / NBLK);
        c.b = (int)(u - (long long)c.pu * NBLK);
        while (s_pref[c.item + 1] <= c.pu) ++c.item;
        return;
      }
      ++c.range;
    }
  };
  auto cur_next = [&](Cur &c) {
    if (--c.left > 0) {
      if (++c.b == NBLK) {
        c.b = 0;
        ++c.pu;
        while (s_pref[c.item + 1] <= c.pu) ++c.item;
      }
    } else {
      ++c.range;
      cur_enter(c);
    }
  };
  auto unit_ptr = [&](const Cur &c) { return s_items[c.item].w + (size_t)c.b * kUnit; };

  // ---- loads: one part of a unit into one register buffer ----
  auto load_gu = [&](uint4 (&buf)[NB], const uint8_t *part) {
    if (NWK == kFsWarps || warp < NWK) {
      const uint8_t *a = part + (size_t)(warp * KT) * 1024 + q * 128 + g * 16;
#pragma unroll
      for (int t = 0; t < KT; ++t) {
        buf[2 * t] = ld_stream_16(a + t * 1024);
        buf[2 * t + 1] = ld_stream_16(a + t * 1024 + 512);
      }
    }
  };
  auto load_d = [&](uint4 (&buf)[NB], const uint8_t *part) {
    const uint8_t *a = part + (size_t)(warp * CTW) * 512 + (q >> 1) * 128 + g * 16 + (q & 1) * 8;
#pragma unroll
    for (int c = 0; c < CTW; ++c) {
      const uint2 lo = ld_stream_8(a + c * 512), hi = ld_stream_8(a + c * 512 + 256);
      buf[c] = make_uint4(lo.x, lo.y, hi.x, hi.y);
    }
  };

  // ---- per-segment state (a segment = this CTA's units of one (item, pass)) ----
  float dacc[CTW][4];
  int my_tok = -1;      // lane i < ntok: token and gate weight of the pass's i-th pair
  float my_w = 0.f;
  int ntok = 0, ngroups = 1;

  auto begin_segment = [&](const Cur &c) {
    const WorkItem &it = s_items[c.item];
    const int tpp = c.range ? kFsZcTokensPerPass : kFsResTokensPerPass;
    const int tok0 = (int)(c.pu - s_pref[c.item]) * tpp;
    ntok = min(tpp, it.n_tok - tok0);
    ngroups = (ntok + kFsTokens - 1) / kFsTokens;
    if (ngroups == 1) {
      my_tok = -1;
      my_w = 0.f;
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
      if (!dense) {
        // (the previous segment's readers of s_x are past the barriers of their last unit)
        const int tok0_ = tok0, off_ = it.off, expert_ = it.expert, ntok_ = ntok;
        stage_x([&](int j) {
          if (j >= ntok_) return -1;
          return expert_ >= 0 ? p.perm[off_ + tok0_ + j] / p.top_k : tok0_ + j;
        });
        __syncthreads();
      }
#pragma unroll
      for (int cc = 0; cc < CTW; ++cc) { dacc[cc][0] = dacc[cc][1] = dacc[cc][2] = dacc[cc][3] = 0.f; }
    } else {
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
    }
  };
  // gate-weighted combine of the accumulators: D fragment = [column g / g+8 of the tile][MMA columns 2q, 2q+1]
  auto flush = [&](int tok_a, float gw_a, int tok_b, float gw_b) {
#pragma unroll
    for (int cc = 0; cc < CTW; ++cc) {
      const int col = 16 * (warp * CTW + cc) + g;
      if (tok_a >= 0) {
        atomicAdd(p.y_acc + (size_t)tok_a * d + col, gw_a * dacc[cc][0]);
        atomicAdd(p.y_acc + (size_t)tok_a * d + col + 8, gw_a * dacc[cc][2]);
      }
      if (tok_b >= 0) {
        atomicAdd(p.y_acc + (size_t)tok_b * d + col, gw_b * dacc[cc][1]);
        atomicAdd(p.y_acc + (size_t)tok_b * d + col + 8, gw_b * dacc[cc][3]);
      }
    }
  };
  auto end_segment = [&]() {   // single-group segments only: the other kind flushes per unit
    int tok_a = -1, tok_b = -1;
    float gw_a = 0.f, gw_b = 0.f;
    if (dense) {   // MMA column j is token j: find the pairs (if any) of tokens 2q and 2q+1
      for (int i = 0; i < ntok; ++i) {
        const int ti = __shfl_sync(0xffffffffu, my_tok, i);
        const float wi = __shfl_sync(0xffffffffu, my_w, i);
        if (ti == 2 * q) { tok_a = ti; gw_a = wi; }
        if (ti == 2 * q + 1) { tok_b = ti; gw_b = wi; }
      }
    } else {       // MMA column j is the pass's j-th pair
      tok_a = __shfl_sync(0xffffffffu, my_tok, 2 * q);
      tok_b = __shfl_sync(0xffffffffu, my_tok, 2 * q + 1);
      gw_a = __shfl_sync(0xffffffffu, my_w, 2 * q);
      gw_b = __shfl_sync(0xffffffffu, my_w, 2 * q + 1);
    }
    flush(tok_a, gw_a, tok_b, gw_b);
  };
  // partial [16 neurons x 8 tokens] sums of one part over this warp's hidden slice -> shared memory
  // (x fragments: from the staged rows, or for multi-group passes straight from global memory, tok = the token of
  // MMA column g)
  auto gu_part = [&](const uint4 (&buf)[NB], int grp, int which, bool staged, int tok) {
    if (NWK == kFsWarps || warp < NWK) {
      float c1[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};   // two chains: consecutive MMAs do not wait
      const uint32_t xs = smem_u32(s_x) + g * kXStride + (uint32_t)(warp * KT) * 64u + 16u * q;
#pragma unroll
      for (int t = 0; t < KT; ++t) {
        uint4 xv = make_uint4(0u, 0u, 0u, 0u);
        if (staged) xv = lds_v4(xs + 64u * t);
        else if (tok >= 0) xv = *reinterpret_cast<const uint4 *>(p.x + (size_t)tok * d + 32 * (warp * KT + t) + 8 * q);
        mma_bf16(c1, buf[2 * t].x, buf[2 * t + 1].x, buf[2 * t].y, buf[2 * t + 1].y, xv.x, xv.y);
        mma_bf16(c2, buf[2 * t].z, buf[2 * t + 1].z, buf[2 * t].w, buf[2 * t + 1].w, xv.z, xv.w);
      }
      float *r = s_red + (((size_t)grp * kFsWarps + warp) * 2 + which) * 128;
      *reinterpret_cast<float2 *>(r + g * 8 + 2 * q) = make_float2(c1[0] + c2[0], c1[1] + c2[1]);
      *reinterpret_cast<float2 *>(r + (g + 8) * 8 + 2 * q) = make_float2(c1[2] + c2[2], c1[3] + c2[3]);
    }
  };
  auto consume_gu = [&](const uint4 (&buf)[NB], int which) {
    if (ngroups == 1) {
      gu_part(buf, 0, which, true, 0);
    } else {
      for (int grp = 0; grp < ngroups; ++grp) gu_part(buf, grp, which, false, s_tok[grp * kFsTokens + g]);
    }
  };
  auto reduce_h = [&]() {   // h = SiLU(sum gate) * (sum up), bf16, [group][token][neuron]
    for (int idx = tid; idx < 128 * ngroups; idx += kFsThreads) {
      const int grp = idx >> 7, r = idx & 127, n = r >> 3, t = r & 7;
      const float *base = s_red + (size_t)grp * kFsWarps * 2 * 128 + r;
      float a = 0.f, c = 0.f;
#pragma unroll
      for (int w = 0; w < NWK; ++w) {
        a += base[(w * 2 + 0) * 128];
        c += base[(w * 2 + 1) * 128];
      }
      s_h[grp * 128 + t * 16 + n] = __float2bfloat16_rn(a / (1.f + __expf(-a)) * c);
    }
  };
  auto down_part = [&](const uint4 (&buf)[NB], int grp) {
    const uint2 hb = *reinterpret_cast<const uint2 *>(s_h + grp * 128 + g * 16 + 4 * q);
#pragma unroll
    for (int cc = 0; cc < CTW; ++cc) mma_bf16(dacc[cc], buf[cc].x, buf[cc].z, buf[cc].y, buf[cc].w, hb.x, hb.y);
  };
  auto consume_d = [&](const uint4 (&buf)[NB]) {
    if (ngroups == 1) {
      down_part(buf, 0);
    } else {
      for (int grp = 0; grp < ngroups; ++grp) {
#pragma unroll
        for (int cc = 0; cc < CTW; ++cc) { dacc[cc][0] = dacc[cc][1] = dacc[cc][2] = dacc[cc][3] = 0.f; }
        down_part(buf, grp);
        const int ia = grp * kFsTokens + 2 * q;
        flush(s_tok[ia], s_gw[ia], s_tok[ia + 1], s_gw[ia + 1]);
      }
    }
  };

  // ---- the stream: gate -> buffer par, up -> buffer par^1, down -> buffer par; the next unit swaps the roles ----
  uint4 buf[2][NB];
  Cur cu;
  cu.range = 0; cu.item = 0; cu.b = 0; cu.pu = 0; cu.left = 0;
  cur_enter(cu);
  if (cu.range < 2) {
    Cur nx = cu;
    {
      const uint8_t *u0 = unit_ptr(cu);
      load_gu(buf[0], u0);
      load_gu(buf[1], u0 + kPart);
    }
    cur_next(nx);
    bool seg_first = true;
    auto step = [&](auto parc) -> bool {
      constexpr int par = decltype(parc)::value;
      if (seg_first) begin_segment(cu);
      const uint8_t *unit = unit_ptr(cu);
      const bool has_next = nx.range < 2;
      const uint8_t *nunit = has_next ? unit_ptr(nx) : unit;
      ++trace_units;
      consume_gu(buf[par], 0);
      load_d(buf[par], unit + 2 * kPart);
      consume_gu(buf[par ^ 1], 1);
      if (has_next) load_gu(buf[par ^ 1], nunit);
      __syncthreads();
      reduce_h();
      __syncthreads();
      consume_d(buf[par]);
      if (has_next) load_gu(buf[par], nunit + kPart);
      const bool seg_last = !(has_next && nx.pu == cu.pu && nx.range == cu.range);
      if (seg_last && ngroups == 1) end_segment();
      seg_first = seg_last;
      cu = nx;
      if (has_next) cur_next(nx);
      return has_next;
    };
    while (true) {
      if (!step(std::integral_constant<int, 0>{})) break;
      if (!step(std::integral_constant<int, 1>{})) break;
    }
  }

  if (p.trace != nullptr && tid == 0) {
    long long *tr = p.trace + 4 * blockIdx.x;
    long long t_end;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_end));
    tr[1] = t_end; tr[2] = trace_units; tr[3] = 0;
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
  // several independent L2 loads in flight per thread: the round trips overlap instead of adding up
  for (long long i0 = tid; i0 < n4; i0 += 8LL * kFsThreads) {
    float4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long i = i0 + (long long)j * kFsThreads;
      v[j] = (i < n4) ? __ldcg(reinterpret_cast<const float4 *>(p.y_acc) + i) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const long long i = i0 + (long long)j * kFsThreads;
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

}  // namespace ftmoe
