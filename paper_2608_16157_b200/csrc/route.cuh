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

// Prefill-sized calls, kernel 1: one warp per token; counts by integer atomics (order-free result).
__global__ void __launch_bounds__(256) route_topk_kernel(RouteParams p) {
  const int lane = threadIdx.x & 31;
  const int t = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= p.T) return;
  int id;
  float w;
  route_token_any(p, t, lane, id, w);
  if (lane < p.k) {
    p.ids[t * p.k + lane] = id;
    p.w[t * p.k + lane] = w;
    atomicAdd(&p.count[id], 1);
  }
}

// Prefill-sized calls, kernel 2: one warp per expert; offset = sum of the counts before it, then a
// walk over all pair keys (four per lane and iteration) ranks this expert's pairs in index order.
__global__ void __launch_bounds__(256) permute_kernel(RouteParams p) {
  const int lane = threadIdx.x & 31;
  const int e = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (e >= p.E) return;
  int before = 0;
  for (int i = lane; i < e; i += 32) before += p.count[i];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) before += __shfl_xor_sync(0xffffffffu, before, o);
  const int c = p.count[e];
  if (lane == 0) {
    p.offset[e] = before;
    if (e == p.E - 1) p.offset[p.E] = before + c;
  }
  if (c == 0) return;
  const int P = p.T * p.k;
  int run = before;
  const int end = before + c;
  for (int base = 0; base < P && run < end; base += 128) {
    const int q0 = base + lane * 4;
    int4 kk = make_int4(-1, -1, -1, -1);
    if (q0 + 3 < P) {
      kk = *reinterpret_cast<const int4 *>(p.ids + q0);
    } else {
      if (q0 < P) kk.x = p.ids[q0];
      if (q0 + 1 < P) kk.y = p.ids[q0 + 1];
      if (q0 + 2 < P) kk.z = p.ids[q0 + 2];
    }
    const int n_mine = (kk.x == e) + (kk.y == e) + (kk.z == e) + (kk.w == e);
    // exclusive prefix of n_mine over the lanes (pairs of lower lanes come first)
    int incl = n_mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += n;
    }
    int pos = run + incl - n_mine;
    if (kk.x == e) { p.perm[pos] = q0; p.inv[q0] = pos; ++pos; }
    if (kk.y == e) { p.perm[pos] = q0 + 1; p.inv[q0 + 1] = pos; ++pos; }
    if (kk.z == e) { p.perm[pos] = q0 + 2; p.inv[q0 + 2] = pos; ++pos; }
    if (kk.w == e) { p.perm[pos] = q0 + 3; p.inv[q0 + 3] = pos; ++pos; }
    run += __shfl_sync(0xffffffffu, incl, 31);
  }
}

}  // namespace ftmoe
