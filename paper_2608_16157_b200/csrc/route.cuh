// Step 1+2: top-k gating (softmax over the selected logits) and the stable expert-sorted
// permutation of the (token, choice) pairs, by warp-level scans.  No atomics decide an order, so
// ids, count, offset, perm and inv are bit-reproducible.
#pragma once
#include "common.cuh"

namespace ftmoe {

constexpr int kRouteSmallMaxTokens = 128;  // one CTA routes and permutes up to this many tokens

struct RouteParams {
  const float *logits;  // [T][E]
  int T, E, k;
  int32_t *ids;     // [T*k]
  float *w;         // [T*k]
  int32_t *count;   // [E]
  int32_t *offset;  // [E+1]
  int32_t *perm;    // [T*k]
  int32_t *inv;     // [T*k]
  uint32_t *status;
};

// (value descending, index ascending) total order; -0 == +0.
__device__ __forceinline__ bool route_better(float v, int i, float bv, int bi) {
  return v > bv || (v == bv && i < bi);
}

// One warp routes one token.  Lane l holds logits l, l+32, ...; k rounds of warp arg-max.
// On return lane j < k holds the j-th selected id and its gate weight.
template <int EPLANE>
__device__ __forceinline__ void route_token(const float *__restrict__ z, int E, int k, int lane,
                                            int &sel_id, float &sel_w, uint32_t *status) {
  float v[EPLANE];
  bool bad = false;
#pragma unroll
  for (int i = 0; i < EPLANE; ++i) {
    const int e = lane + 32 * i;
    float x = -INFINITY;
    if (e < E) {
      x = z[e];
      if (!isfinite(x)) bad = true;
    }
    v[i] = x;
  }
  if (__any_sync(0xffffffffu, bad) && lane == 0) atomicOr(status, kStatNonFinite);
  // order-preserving map float -> uint32 (-0 folded into +0), so that a warp maximum is one redux instruction
  auto ordered = [](float x) -> uint32_t {
    const uint32_t u = __float_as_uint(x + 0.f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
  };
  float my_v = 0.f;
  int my_i = 0;
  for (int r = 0; r < k; ++r) {
    float bv = -INFINITY;
    int bi = 0x7fffffff;
#pragma unroll
    for (int i = 0; i < EPLANE; ++i) {
      const int e = lane + 32 * i;
      if (e < E && route_better(v[i], e, bv, bi)) { bv = v[i]; bi = e; }
    }
    // warp arg-max in the total order (value descending, index ascending): maximum of the values, then the
    // smallest index among the lanes that hold it
    const uint32_t mx = __reduce_max_sync(0xffffffffu, ordered(bv));
    const uint32_t cand = (ordered(bv) == mx) ? (uint32_t)bi : 0xffffffffu;
    bi = (int)__reduce_min_sync(0xffffffffu, cand);
    bv = __shfl_sync(0xffffffffu, bv, bi & 31);
    if (bi == 0x7fffffff) bi = 0;  // only reachable with non-finite input (already latched)
    if (lane == r) { my_v = bv; my_i = bi; }
    if ((bi & 31) == lane) {
      const int wi = bi >> 5;
#pragma unroll
      for (int i = 0; i < EPLANE; ++i)
        if (i == wi) v[i] = -INFINITY;
    }
  }
  const float z0 = __shfl_sync(0xffffffffu, my_v, 0);
  const float ex = (lane < k) ? expf(my_v - z0) : 0.f;
  const float sum = warp_sum(ex);
  sel_id = my_i;
  sel_w = ex / sum;
}

template <int EPLANE>
__device__ __forceinline__ void route_token_dispatch(const RouteParams &p, int t, int lane, int &id, float &w) {
  route_token<EPLANE>(p.logits + (size_t)t * p.E, p.E, p.k, lane, id, w, p.status);
}

__device__ __forceinline__ void route_token_any(const RouteParams &p, int t, int lane, int &id, float &w) {
  if (p.E <= 128) route_token_dispatch<4>(p, t, lane, id, w);
  else if (p.E <= 256) route_token_dispatch<8>(p, t, lane, id, w);
  else route_token_dispatch<32>(p, t, lane, id, w);
}

// Shared memory of the single-CTA route + permute.
struct RouteSmem {
  int32_t cnt[kMaxExperts];
  int32_t off[kMaxExperts + 1];
  int16_t key[kRouteSmallMaxTokens * kMaxTopK];
  int32_t wsum[32];
};

// Decode-sized calls: one CTA (a warp multiple of at least E threads) routes all tokens, counts, scans and permutes.  On
// return (after a barrier) s.cnt / s.off hold count[] and offset[] for the caller.
__device__ __forceinline__ void route_small_body(const RouteParams &p, RouteSmem &s) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int P = p.T * p.k;
  for (int e = tid; e < p.E; e += blockDim.x) s.cnt[e] = 0;
  __syncthreads();
  const int nwarps = blockDim.x >> 5;
  for (int t = warp; t < p.T; t += nwarps) {
    int id;
    float w;
    route_token_any(p, t, lane, id, w);
    if (lane < p.k) {
      p.ids[t * p.k + lane] = id;
      p.w[t * p.k + lane] = w;
      s.key[t * p.k + lane] = (int16_t)id;
      atomicAdd(&s.cnt[id], 1);  // a count: the result does not depend on the order of the adds
    }
  }
  __syncthreads();
  // exclusive scan of the counts (one expert per thread)
  {
    const int c = (tid < p.E) ? s.cnt[tid] : 0;
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s.wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      int ws = (lane < nwarps) ? s.wsum[lane] : 0;
      int wincl = ws;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += n;
      }
      s.wsum[lane] = wincl - ws;
    }
    __syncthreads();
    const int excl = incl - c + s.wsum[warp];
    if (tid < p.E) {
      s.off[tid] = excl;
      p.count[tid] = c;
      p.offset[tid] = excl;
      if (tid == p.E - 1) { s.off[p.E] = excl + c; p.offset[p.E] = excl + c; }
    }
  }
  __syncthreads();
  // one warp per expert walks the pairs in index order: rank = number of earlier pairs with this key
  for (int e = warp; e < p.E; e += nwarps) {
    if (s.cnt[e] == 0) continue;
    int run = s.off[e];
    for (int base = 0; base < P; base += 32) {
      const int q = base + lane;
      const bool mine = (q < P) && (s.key[q] == e);
      const unsigned m = __ballot_sync(0xffffffffu, mine);
      if (mine) {
        const int pos = run + __popc(m & ((1u << lane) - 1u));
        p.perm[pos] = q;
        p.inv[q] = pos;
      }
      run += __popc(m);
    }
  }
}

__global__ void __launch_bounds__(1024) route_small_kernel(RouteParams p) {
  __shared__ RouteSmem s;
  route_small_body(p, s);
}

// ---- prefill-sized calls: two launches over blocks of kRouteBlockTokens tokens ----
constexpr int kRouteBlockTokens = 32;   // one token per warp of a 1024-thread block: 4096 tokens fill 128 SMs

// Kernel 1: block b routes its tokens (one warp per token), writes ids / w and the block's histogram hist[b][E]
// (integer atomics in shared memory: the counts do not depend on the order of the adds).
__global__ void __launch_bounds__(1024) route_block_kernel(RouteParams p, int32_t *hist) {
  __shared__ int32_t s_cnt[kMaxExperts];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int e = tid; e < p.E; e += blockDim.x) s_cnt[e] = 0;
  __syncthreads();
  const int t0 = blockIdx.x * kRouteBlockTokens;
  const int t1 = min(p.T, t0 + kRouteBlockTokens);
  for (int t = t0 + warp; t < t1; t += (blockDim.x >> 5)) {
    int id;
    float w;
    route_token_any(p, t, lane, id, w);
    if (lane < p.k) {
      p.ids[t * p.k + lane] = id;
      p.w[t * p.k + lane] = w;
      atomicAdd(&s_cnt[id], 1);
    }
  }
  __syncthreads();
  for (int e = tid; e < p.E; e += blockDim.x) hist[(size_t)blockIdx.x * p.E + e] = s_cnt[e];
}

// Kernel 2: block b ranks its pairs.  pos(p) = offset[e] + pairs of expert e in earlier blocks + pairs of e earlier
// in this block, which keeps the order stable in the pair index.  Every block sums the (small, L2-resident)
// histograms itself -- count[e] over all blocks, the part before block b -- and scans the counts into offset[];
// block 0 publishes count[] and offset[].  Each warp owns a contiguous part of the block's pairs and walks it 32
// pairs at a time; lanes with equal keys find each other with match.any.  blockDim.x = 1024 >= E.
__global__ void __launch_bounds__(1024) permute_block_kernel(RouteParams p, const int32_t *hist, int n_blocks) {
  __shared__ int32_t s_base[8][kMaxExperts];
  __shared__ int32_t s_start[kMaxExperts];   // offset[e] + pairs of e in earlier blocks
  __shared__ int32_t s_wsum[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const int P = p.T * p.k;
  {
    int c = 0, before = 0;
    if (tid < p.E) {
      for (int b = 0; b < n_blocks; ++b) {
        const int v = hist[(size_t)b * p.E + tid];
        if (b < (int)blockIdx.x) before += v;
        c += v;
      }
    }
    int incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    if (lane == 31) s_wsum[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const int ws = (lane < nwarps) ? s_wsum[lane] : 0;
      int wincl = ws;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, wincl, o);
        if (lane >= o) wincl += n;
      }
      s_wsum[lane] = wincl - ws;
    }
    __syncthreads();
    const int excl = incl - c + s_wsum[warp];
    if (tid < p.E) {
      s_start[tid] = excl + before;
      if (blockIdx.x == 0) {
        p.count[tid] = c;
        p.offset[tid] = excl;
        if (tid == p.E - 1) p.offset[p.E] = excl + c;
      }
    }
  }
  if (warp >= 8) {   // the ranking below is done by 8 warps
    __syncthreads();
    __syncthreads();
    return;
  }
  const int q0 = blockIdx.x * kRouteBlockTokens * p.k;
  const int q1 = min(P, q0 + kRouteBlockTokens * p.k);
  const int per_warp = (((q1 - q0 + 7) / 8) + 31) & ~31;    // a multiple of 32 pairs
  const int w0 = q0 + warp * per_warp, w1 = min(q1, w0 + per_warp);
  for (int e = tid; e < p.E; e += 256)
#pragma unroll
    for (int w = 0; w < 8; ++w) s_base[w][e] = 0;
  __syncthreads();
  const unsigned lt = (1u << lane) - 1u;
  for (int q = w0 + lane; q - lane < w1; q += 32) {         // this warp's histogram
    const int key = (q < w1) ? p.ids[q] : -1;
    const unsigned m = __match_any_sync(0xffffffffu, key);
    if (key >= 0 && (m & lt) == 0) s_base[warp][key] += __popc(m);   // one leader per key: no conflict
    __syncwarp();
  }
  __syncthreads();
  // (the barriers from here on are among the 8 ranking warps only)
  for (int e = tid; e < p.E; e += 256) {                    // where each warp's pairs of expert e begin
    int base = s_start[e];
#pragma unroll
    for (int w = 0; w < 8; ++w) {
      const int n = s_base[w][e];
      s_base[w][e] = base;
      base += n;
    }
  }
  asm volatile("bar.sync 1, 256;" ::: "memory");
  for (int q = w0 + lane; q - lane < w1; q += 32) {
    const int key = (q < w1) ? p.ids[q] : -1;
    const unsigned m = __match_any_sync(0xffffffffu, key);
    int pos = 0;
    if (key >= 0) pos = s_base[warp][key] + __popc(m & lt);
    __syncwarp();
    if (key >= 0 && (m & lt) == 0) s_base[warp][key] += __popc(m);
    __syncwarp();
    if (key >= 0) {
      p.perm[pos] = q;
      p.inv[q] = pos;
    }
  }
}

}  // namespace ftmoe
