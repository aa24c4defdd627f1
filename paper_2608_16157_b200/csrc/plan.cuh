// Step 3: device-side cache control (paper Sec. 4.1).  One CTA per call: deduplicate the routed
// experts, classify them against the slot table, refresh the stamps of the hits, order every
// evictable slot in one pass (free first, then least recently used; ties to the lower resident
// expert id), size the fill set from the bandwidths (Eq. 4, rounded half up, at least one), choose
// the fills (most tokens first), assign slots, and rewrite expert ids into slot ids or the
// zero-copy flag.  Integer arithmetic only, no atomics that could decide an order.
#pragma once
#include "common.cuh"

namespace ftmoe {

struct PlanParams {
  // inputs
  const int32_t *count;   // [E]
  const int32_t *offset;  // [E+1]
  int E, n_slots;        // experts of this layer; slots of the table (per layer, or the shared pool)
  int id_base;           // flattened id of this layer's expert 0 in the tables (layer*E with a shared pool, else 0)
  CostModelDev cm;
  // per-layer state
  int32_t *slot_expert;  // [n_slots]
  int64_t *slot_stamp;   // [n_slots]
  int32_t *expert_slot;  // [E]
  int64_t *step;         // [1] the LRU clock: stamps come from it and it advances by one per plan
  int64_t *layer_steps;  // [1] plan calls of this layer (the same counter unless the pool is shared)
  unsigned long long *stats;  // [FT_STAT_COUNT]
  // where records live
  const uint8_t *pool_layer_dev;  // device alias of the host pool, first record of this layer
  uint8_t *slots_layer;           // first slot of this layer
  const uint8_t *shared_rec;      // shared-expert record of this layer or nullptr
  size_t S;
  int T;
  int tokens_per_pass;   // tokens one weight pass of the resident streaming kernel serves
  int zc_tokens_per_pass;   // tokens one link pass of a zero-copy record serves
  // outputs
  PlanHeader *hdr_dev;   // device plan record (header + 8 arrays of E)
  PlanHeader *hdr_host;  // mapped host mirror, or nullptr when the host does not read the plan
  WorkItem *items_res;   // [2E+1] experts evaluated by the streaming kernel: from slots, then the shared
                         //        expert, then the zero-copy experts (records in the mapped host pool)
  int32_t *res_pref;     // [2E+2] exclusive prefix of the weight passes of items_res
  WorkItem *items_zc;    // [E]    experts evaluated from the mapped host pool
  WorkItem *items_gemm;  // [E]    experts evaluated from slots by the grouped GEMM
  int32_t *gemm_pref;    // [E+1]  exclusive prefix of the 128-row tiles of items_gemm
  uint8_t *is_gemm;      // [E]    1 if the expert goes through the grouped GEMM in this step
  uint32_t seq_value;    // sequence number of this plan (counted by the host)
  int prefetch;          // 1: admission of a whole layer ahead of its routing (no step of the layer is counted)
};

// Block-wide exclusive scan of one 64-bit value per thread (several small counters packed into it).
__device__ __forceinline__ unsigned long long block_excl_scan64(unsigned long long v, unsigned long long *s_w /*[33]*/,
                                                                unsigned long long &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
  unsigned long long incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned long long n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  __syncthreads();  // protects s_w against the previous use
  if (lane == 31) s_w[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const unsigned long long ws = (lane < nwarps) ? s_w[lane] : 0ull;
    unsigned long long wincl = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned long long n = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += n;
    }
    s_w[lane] = wincl - ws;
    if (lane == 31) s_w[32] = wincl;
  }
  __syncthreads();
  total = s_w[32];
  return incl - v + s_w[warp];
}

constexpr int64_t kSlotTaken = 0x7fffffffffffffffll;   // stamp marker of a slot already chosen as a victim
constexpr int kPlanField = 11;  // bits per packed counter (values <= 1024)
__device__ __forceinline__ unsigned long long pack4(int a, int b, int c, int d) {
  return (unsigned long long)a | ((unsigned long long)b << kPlanField) | ((unsigned long long)c << (2 * kPlanField)) |
         ((unsigned long long)d << (3 * kPlanField));
}
__device__ __forceinline__ int unpack(unsigned long long v, int i) {
  return (int)((v >> (i * kPlanField)) & ((1u << kPlanField) - 1u));
}

// Shared memory the plan needs besides the dynamic part (stamp/expert/victim per slot).
struct PlanSmem {
  unsigned long long w[33];
  int32_t cnt[kMaxExperts];
  uint8_t elig[kMaxExperts];
  uint8_t isfill[kMaxExperts];
  int32_t forder[kMaxExperts];
  int16_t miss[kMaxExperts];
  int pairs_res;
};

// Issues every global read of the layer's state up front (step counter, this thread's expert_slot, the slot
// table into shared memory) so their latencies overlap each other and whatever the caller does next.
// A barrier must separate this from plan_body.
__device__ __forceinline__ void plan_prefetch(const PlanParams &p, unsigned char *s_dyn, int64_t &t, int &slot) {
  int64_t *s_stamp = reinterpret_cast<int64_t *>(s_dyn);
  int32_t *s_sexp = reinterpret_cast<int32_t *>(s_stamp + p.n_slots);
  const int tid = threadIdx.x;
  t = *p.step;
  slot = (tid < p.E) ? p.expert_slot[p.id_base + tid] : -1;
  for (int s = tid; s < p.n_slots; s += blockDim.x) {
    s_stamp[s] = p.slot_stamp[s];
    s_sexp[s] = p.slot_expert[s];
  }
}

// One plan step.  Thread `tid` < E owns expert `tid`: `c` = its token count, `off` = its offset in the
// expert-sorted pair order, `n_pairs` = all pairs of the call.  blockDim.x >= E, a multiple of 32.
// s_dyn: int64 stamp[n_slots]; int32 sexp[n_slots]; int32 victim[n_slots] (filled by plan_prefetch).
__device__ __forceinline__ void plan_body(const PlanParams &p, PlanSmem &sm, unsigned char *s_dyn, int c, int off,
                                          int n_pairs, const int64_t t, const int slot_in) {
  int64_t *s_stamp = reinterpret_cast<int64_t *>(s_dyn);
  int32_t *s_sexp = reinterpret_cast<int32_t *>(s_stamp + p.n_slots);
  int32_t *s_victim = s_sexp + p.n_slots;
  const int tid = threadIdx.x;
  const int E = p.E;
  if (n_pairs == 0) return;  // nothing routed: the step does not advance

  int32_t *a_hit = reinterpret_cast<int32_t *>(p.hdr_dev + 1);
  int32_t *a_miss = a_hit + E, *a_fill = a_miss + E, *a_zc = a_fill + E, *a_forder = a_zc + E;
  int32_t *a_fslot = a_forder + E, *a_fevict = a_fslot + E, *a_loc = a_fevict + E;

  // ---- 1/2: classify, refresh recency of hits; 4: which misses are worth a fill
  int slot = slot_in, cls = 0, elig = 0;
  if (tid < E) {
    cls = (c > 0) ? (slot >= 0 ? 1 : 2) : 0;
    if (cls == 1) { p.slot_stamp[slot] = t; s_stamp[slot] = t; }
    if (cls == 2) {
      const int64_t pz = (c + p.cm.tz - 1) / p.cm.tz, pg = (c + p.cm.tg - 1) / p.cm.tg;
      const int64_t v = pz * p.cm.ns_zc - (p.cm.ns_fill + pg * p.cm.ns_hbm) +
                        (int64_t)p.cm.reuse_credit * (p.cm.ns_zc - p.cm.ns_hbm);
      elig = v > 0;
    }
    sm.cnt[tid] = c;
    sm.elig[tid] = (uint8_t)elig;
    sm.isfill[tid] = 0;
  }
  if (tid == 0) sm.pairs_res = 0;
  unsigned long long totA;
  const unsigned long long exA = block_excl_scan64(pack4(cls != 0, cls == 1, cls == 2, elig), sm.w, totA);
  const int n_routed = unpack(totA, 0), n_hit = unpack(totA, 1), n_miss = unpack(totA, 2), n_elig = unpack(totA, 3);
  if (cls == 1) a_hit[unpack(exA, 1)] = tid;
  if (cls == 2) {
    a_miss[unpack(exA, 2)] = tid;
    sm.miss[unpack(exA, 2)] = (int16_t)tid;
  }
  __syncthreads();   // sm.miss and the refreshed stamps are visible to the whole block from here on

  // ---- 3: victim candidates, ordered in one pass: each warp ranks a few candidates by counting, 32 slots per
  // ballot, how many candidates precede them (free slots first by index, then (stamp, resident expert id))
  // (the scan's barriers make the refreshed stamps in shared memory visible to the whole block)
  const int lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  int K = 0;
  int q = 0;
  if (n_miss > 0) {    // block-uniform: with no miss there is nothing to evict or fill
    for (int base = 0; base < p.n_slots; base += 32) {
      const int o = base + lane;
      const bool oc = (o < p.n_slots) && ((s_sexp[o] < 0) || (s_stamp[o] < t));
      K += __popc(__ballot_sync(0xffffffffu, oc));
    }
    // ---- 5: fill count
    const int64_t bt = p.cm.bw_fill + p.cm.bw_res;
    int64_t qbw = (2 * (int64_t)n_miss * p.cm.bw_fill + bt) / (2 * bt);
    if (qbw < 1) qbw = 1;
    q = (int)qbw;
    if (q > n_elig) q = n_elig;
    if (q > K) q = K;
    // The order key of a candidate slot: free slots by index, then occupied ones by (stamp, resident expert id);
    // keys are distinct, non-candidates get the largest value.
    auto slot_key = [&](int o) -> unsigned long long {
      if (o >= p.n_slots) return ~0ull;
      const int oex = s_sexp[o];
      const int64_t ost = s_stamp[o];
      if (ost == kSlotTaken) return ~0ull;
      if (oex < 0) return (unsigned long long)o;
      if (ost >= t) return ~0ull;
      return (1ull << 62) | ((unsigned long long)(ost + 1) << 20) | (unsigned long long)oex;
    };
    if (q <= 16 && p.n_slots > 256) {
      // few fills out of a large (shared) pool: q block-wide minima; a chosen slot is marked as touched
      unsigned long long *s_wmin = reinterpret_cast<unsigned long long *>(sm.forder);   // [32] keys (forder is free here)
      int *s_wslot = reinterpret_cast<int *>(s_wmin + 32);                               // [32] slots
      for (int r = 0; r < q; ++r) {
        unsigned long long best = ~0ull;
        int bslot = -1;
        for (int o = tid; o < p.n_slots; o += blockDim.x) {
          const unsigned long long ko = slot_key(o);
          if (ko < best) { best = ko; bslot = o; }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
          const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
          if (ob < best) { best = ob; bslot = os; }
        }
        if (lane == 0) { s_wmin[warp] = best; s_wslot[warp] = bslot; }
        __syncthreads();
        if (warp == 0) {
          best = (lane < nwarps) ? s_wmin[lane] : ~0ull;
          bslot = (lane < nwarps) ? s_wslot[lane] : -1;
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
            if (ob < best) { best = ob; bslot = os; }
          }
          if (lane == 0) {
            s_victim[r] = bslot;
            s_stamp[bslot] = kSlotTaken;   // no longer a candidate (the shared-memory copy is not used afterwards)
          }
        }
        __syncthreads();
      }
    } else if (q <= 8 && p.n_slots <= 256) {
      // few fills (decode): warp 0 extracts the q smallest keys one after the other (q warp-wide minima)
      if (warp == 0) {
        unsigned long long key[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) key[i] = slot_key(lane + 32 * i);
        for (int r = 0; r < q; ++r) {
          unsigned long long best = key[0];
          int bslot = lane;
#pragma unroll
          for (int i = 1; i < 8; ++i)
            if (key[i] < best) { best = key[i]; bslot = lane + 32 * i; }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long ob = __shfl_xor_sync(0xffffffffu, best, o);
            const int os = __shfl_xor_sync(0xffffffffu, bslot, o);
            if (ob < best) { best = ob; bslot = os; }
          }
          if (lane == 0) s_victim[r] = bslot;
          if ((bslot & 31) == lane) {
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (i == (bslot >> 5)) key[i] = ~0ull;
          }
        }
      }
    } else {
      // many fills (prefill): every candidate is ranked in one pass, 32 slots per ballot
      for (int s = warp; s < p.n_slots; s += nwarps) {
        const unsigned long long ks = slot_key(s);
        if (ks == ~0ull) continue;      // warp-uniform
        int rank = 0;
        for (int base = 0; base < p.n_slots; base += 32) {
          const int o = base + lane;
          rank += __popc(__ballot_sync(0xffffffffu, o != s && slot_key(o) < ks));
        }
        if (lane == 0) s_victim[rank] = s;
      }
    }
  }

  // ---- 6: priority of the eligible misses (tokens descending, id ascending): each warp ranks a few misses
  // by ballots over the experts; sm.miss was written before the scan's barriers
  for (int i = warp; i < n_miss; i += nwarps) {
    const int e = sm.miss[i];
    if (!sm.elig[e]) continue;                  // warp-uniform
    const int ce = sm.cnt[e];
    int rank = 0;
    for (int base = 0; base < E; base += 32) {
      const int o = base + lane;
      bool better = false;
      if (o < E && o != e && sm.elig[o]) {
        const int oc = sm.cnt[o];
        better = (oc > ce) || (oc == ce && o < e);
      }
      rank += __popc(__ballot_sync(0xffffffffu, better));
    }
    if (lane == 0 && rank < q) { sm.forder[rank] = e; sm.isfill[e] = 1; }
  }
  __syncthreads();
  const int is_fill = (tid < E) ? sm.isfill[tid] : 0;

  // ---- 7: the i-th fill takes the i-th candidate slot
  int loc = kLocNotRouted;
  if (cls == 1) loc = slot;
  if (tid < q) {
    const int e = sm.forder[tid];
    const int s = s_victim[tid];
    const int old = s_sexp[s];
    if (old >= 0) p.expert_slot[old] = -1;      // `old` is a flattened id: it may belong to another layer
    p.slot_expert[s] = p.id_base + e;
    p.expert_slot[p.id_base + e] = s;
    p.slot_stamp[s] = t;
    a_forder[tid] = e;
    a_fslot[tid] = s;
    a_fevict[tid] = old;
    sm.cnt[e] = -1 - s;   // hands the slot to the thread that owns expert e (negative marks "filled")
  }
  __syncthreads();
  if (is_fill) loc = -1 - sm.cnt[tid];

  // ---- 8: lists and locations
  const int is_zc = (cls == 2 && !is_fill);
  if (is_zc) loc = kLocZeroCopy;
  const int resident = (cls == 1 || is_fill);
  const int use_gemm = resident && p.cm.gemm_min_tokens > 0 && c >= p.cm.gemm_min_tokens;
  const int res_stream = resident && !use_gemm;
  if (resident) atomicAdd(&sm.pairs_res, c);   // a sum: order-free; read after the scans' barriers
  // The streaming kernel's list: [hits][shared expert][fills][zero-copy], so that the hits can be evaluated
  // while the fills are still in flight.
  const int hs = res_stream && cls == 1, fs = res_stream && is_fill;
  unsigned long long totB;
  const unsigned long long exB = block_excl_scan64(
      pack4(is_fill, is_zc, hs, use_gemm) | ((unsigned long long)fs << (4 * kPlanField)), sm.w, totB);
  const int n_fill = unpack(totB, 0), n_zc = unpack(totB, 1), n_hs = unpack(totB, 2), n_gemm = unpack(totB, 3);
  const int n_fs = unpack(totB, 4);
  // weight passes (tokens_per_pass tokens each) of the list entries, in list order
  const int passes = res_stream ? (c + p.tokens_per_pass - 1) / p.tokens_per_pass
                                : (is_zc ? (c + p.zc_tokens_per_pass - 1) / p.zc_tokens_per_pass : 0);
  unsigned long long totC, totZ;
  const unsigned long long exC = block_excl_scan64(
      ((unsigned long long)(fs ? passes : 0) << 32) | (unsigned long long)(hs ? passes : 0), sm.w, totC);
  const unsigned long long exZ = block_excl_scan64((unsigned long long)(is_zc ? passes : 0), sm.w, totZ);
  const int n_shared_items = (p.shared_rec != nullptr) ? 1 : 0;
  const int shared_passes = n_shared_items ? (p.T + p.tokens_per_pass - 1) / p.tokens_per_pass : 0;
  const int pass_hits = (int)(totC & 0xffffffffull) + shared_passes;   // passes before the first fill
  const int pass_res = pass_hits + (int)(totC >> 32);                   // passes before the first zero-copy item
  const int n_hit_items = n_hs + n_shared_items, n_res_items = n_hit_items + n_fs;
  if (p.cm.gemm_min_tokens > 0) {   // uniform branch: only prefill-capable handles pay for this scan
    unsigned long long totD;
    const unsigned long long exD = block_excl_scan64(
        use_gemm ? (((unsigned long long)c << 32) | (unsigned long long)((c + 127) / 128)) : 0ull, sm.w, totD);
    if (use_gemm) p.gemm_pref[unpack(exB, 3)] = (int32_t)(exD & 0xffffffffull);
    if (tid == 0) {
      p.gemm_pref[n_gemm] = (int32_t)(totD & 0xffffffffull);
      atomicAdd(&p.stats[9], (unsigned long long)(totD >> 32));   // pairs served by the grouped GEMM
    }
    if (tid < E) p.is_gemm[tid] = (uint8_t)use_gemm;
  }
  if (is_fill) a_fill[unpack(exB, 0)] = tid;
  if (is_zc) a_zc[unpack(exB, 1)] = tid;
  if (tid < E) a_loc[tid] = loc;
  if (resident) {
    WorkItem it;
    it.w = p.slots_layer + (size_t)loc * p.S;
    it.expert = tid;
    it.n_tok = c;
    it.off = off;
    it.slot = loc;
    if (use_gemm) {
      p.items_gemm[unpack(exB, 3)] = it;
    } else if (hs) {
      p.items_res[unpack(exB, 2)] = it;
      p.res_pref[unpack(exB, 2)] = (int32_t)(exC & 0xffffffffull);
    } else {
      p.items_res[n_hit_items + unpack(exB, 4)] = it;
      p.res_pref[n_hit_items + unpack(exB, 4)] = pass_hits + (int32_t)(exC >> 32);
    }
  }
  if (is_zc) {
    WorkItem it;
    it.w = p.pool_layer_dev + (size_t)tid * p.S;
    it.expert = tid;
    it.n_tok = c;
    it.off = off;
    it.slot = -1;
    p.items_zc[unpack(exB, 1)] = it;
    const int zi = n_res_items + unpack(exB, 1);   // appended after the resident items
    p.items_res[zi] = it;
    p.res_pref[zi] = pass_res + (int32_t)exZ;
  }

  if (tid == 0) {
    if (n_shared_items) {
      WorkItem it;
      it.w = p.shared_rec;
      it.expert = -1;
      it.n_tok = p.T;
      it.off = 0;
      it.slot = -1;
      p.items_res[n_hs] = it;
      p.res_pref[n_hs] = (int)(totC & 0xffffffffull);
    }
    if (n_fs == 0) p.res_pref[n_hit_items] = pass_hits;
    if (n_zc == 0) p.res_pref[n_res_items] = pass_res;
    p.res_pref[n_res_items + n_zc] = pass_res + (int)totZ;
    PlanHeader h;
    h.step = t;
    h.n_routed = n_routed; h.n_hit = n_hit; h.n_miss = n_miss; h.n_fill = n_fill; h.n_zc = n_zc;
    h.n_res_items = n_res_items; h.n_zc_items = n_zc; h.n_gemm_items = n_gemm;
    h.seq = p.seq_value;
    h.n_hit_items = n_hit_items;
    h.pad[0] = h.pad[1] = h.pad[2] = h.pad[3] = 0;
    *p.hdr_dev = h;
    *p.step = t + 1;
    if (p.layer_steps != p.step && !p.prefetch) *p.layer_steps += 1;
    int evictions = 0;
    for (int i = 0; i < n_fill; ++i) evictions += (s_sexp[s_victim[i]] >= 0);
    // fire-and-forget adds: nothing waits for the old values
    atomicAdd(&p.stats[4], (unsigned long long)n_fill);
    atomicAdd(&p.stats[6], (unsigned long long)evictions);
    if (!p.prefetch) {
      atomicAdd(&p.stats[0], 1ull);
      atomicAdd(&p.stats[1], (unsigned long long)n_routed);
      atomicAdd(&p.stats[2], (unsigned long long)n_hit);
      atomicAdd(&p.stats[3], (unsigned long long)n_miss);
      atomicAdd(&p.stats[5], (unsigned long long)n_zc);
      atomicAdd(&p.stats[7], (unsigned long long)n_pairs);
      atomicAdd(&p.stats[8], (unsigned long long)sm.pairs_res);
    }
  }
  // mirror the record into mapped host memory when the host reads the plan (copy-engine fills)
  if (p.hdr_host != nullptr) {
    __syncthreads();
    const int n_words = (int)(sizeof(PlanHeader) / 4) + 8 * E;
    const uint32_t *src = reinterpret_cast<const uint32_t *>(p.hdr_dev);
    volatile uint32_t *dst = reinterpret_cast<volatile uint32_t *>(p.hdr_host);
    for (int i = tid; i < n_words; i += blockDim.x) dst[i] = src[i];
  }
}

// Counts of a layer whose every expert is "routed" once: the input of a whole-layer admission.
__global__ void __launch_bounds__(1024) all_experts_kernel(int32_t *count, int32_t *offset, int E) {
  for (int e = threadIdx.x; e <= E; e += blockDim.x) {
    if (e < E) count[e] = 1;
    offset[e] = e;
  }
}

// Stand-alone plan kernel: blockDim.x = E rounded up to a warp multiple (at least 128).
__global__ void __launch_bounds__(1024) plan_kernel(PlanParams p) {
  extern __shared__ __align__(16) unsigned char s_dyn[];
  // a streaming kernel launched as a programmatic dependent may be scheduled now; it waits for this grid to
  // complete before it reads the plan
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  __shared__ PlanSmem sm;
  const int tid = threadIdx.x;
  int64_t t;
  int slot;
  plan_prefetch(p, s_dyn, t, slot);
  const int n_pairs = p.offset[p.E];
  int c = 0, off = 0;
  if (tid < p.E) { c = p.count[tid]; off = p.offset[tid]; }
  __syncthreads();
  plan_body(p, sm, s_dyn, c, off, n_pairs, t, slot);
}

}  // namespace ftmoe
