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
  int E, n_slots;
  CostModelDev cm;
  // per-layer state
  int32_t *slot_expert;  // [n_slots]
  int64_t *slot_stamp;   // [n_slots]
  int32_t *expert_slot;  // [E]
  int64_t *step;         // [1]
  unsigned long long *stats;  // [FT_STAT_COUNT]
  // where records live
  const uint8_t *pool_layer_dev;  // device alias of the host pool, first record of this layer
  uint8_t *slots_layer;           // first slot of this layer
  const uint8_t *shared_rec;      // shared-expert record of this layer or nullptr
  size_t S;
  int T;
  // outputs
  PlanHeader *hdr_dev;   // device plan record (header + 8 arrays of E)
  PlanHeader *hdr_host;  // mapped host mirror
  WorkItem *items_res;   // [E+1]  experts evaluated from slots by the streaming kernel
  WorkItem *items_zc;    // [E]    experts evaluated from the mapped host pool
  WorkItem *items_gemm;  // [E]    experts evaluated from slots by the grouped GEMM
  uint32_t *seq;         // [1] plan sequence number
};

// Block-wide exclusive scan of one int per thread (blockDim = 1024); returns the exclusive prefix and
// the total through `total`.
__device__ __forceinline__ int block_excl_scan(int v, int *s_w /*[33]*/, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  __syncthreads();  // protects s_w against the previous use
  if (lane == 31) s_w[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int ws = s_w[lane];
    int wincl = ws;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, wincl, o);
      if (lane >= o) wincl += n;
    }
    s_w[lane] = wincl - ws;
    if (lane == 31) s_w[32] = wincl;
  }
  __syncthreads();
  total = s_w[32];
  return incl - v + s_w[warp];
}

// Dynamic shared memory: int64 stamp[n_slots]; int32 sexp[n_slots]; int32 victim[n_slots].
__global__ void __launch_bounds__(1024) plan_kernel(PlanParams p) {
  extern __shared__ __align__(16) unsigned char s_raw[];
  int64_t *s_stamp = reinterpret_cast<int64_t *>(s_raw);
  int32_t *s_sexp = reinterpret_cast<int32_t *>(s_stamp + p.n_slots);
  int32_t *s_victim = s_sexp + p.n_slots;
  __shared__ int s_w[33];
  __shared__ int32_t s_cnt[kMaxExperts];
  __shared__ uint8_t s_elig[kMaxExperts];
  __shared__ int32_t s_forder[kMaxExperts];
  __shared__ int s_K;

  const int tid = threadIdx.x;
  const int E = p.E;
  if (p.offset[E] == 0) return;  // nothing routed: the step does not advance
  const int64_t t = *p.step;

  int32_t *a_hit = reinterpret_cast<int32_t *>(p.hdr_dev + 1);
  int32_t *a_miss = a_hit + E, *a_fill = a_miss + E, *a_zc = a_fill + E, *a_forder = a_zc + E;
  int32_t *a_fslot = a_forder + E, *a_fevict = a_fslot + E, *a_loc = a_fevict + E;

  // ---- 1/2: classify, refresh recency of hits
  int c = 0, slot = -1, cls = 0;
  if (tid < E) {
    c = p.count[tid];
    slot = p.expert_slot[tid];
    cls = (c > 0) ? (slot >= 0 ? 1 : 2) : 0;
    if (cls == 1) p.slot_stamp[slot] = t;
    s_cnt[tid] = c;
  }
  if (tid == 0) s_K = 0;
  __syncthreads();  // stamps of hits are visible to this block (global writes + barrier)

  int n_routed, n_hit, n_miss;
  block_excl_scan(cls != 0, s_w, n_routed);
  const int hpos = block_excl_scan(cls == 1, s_w, n_hit);
  if (cls == 1) a_hit[hpos] = tid;
  const int mpos = block_excl_scan(cls == 2, s_w, n_miss);
  if (cls == 2) a_miss[mpos] = tid;

  // ---- 3: victim candidates, ordered in one pass by counting how many candidates precede each
  for (int s = tid; s < p.n_slots; s += blockDim.x) {
    s_stamp[s] = p.slot_stamp[s];
    s_sexp[s] = p.slot_expert[s];
  }
  __syncthreads();
  for (int s = tid; s < p.n_slots; s += blockDim.x) {
    const int64_t st = s_stamp[s];
    const int ex = s_sexp[s];
    const bool cand = (ex < 0) || (st < t);
    if (!cand) continue;
    int rank = 0;
    for (int o = 0; o < p.n_slots; ++o) {
      const int oex = s_sexp[o];
      const int64_t ost = s_stamp[o];
      if (!((oex < 0) || (ost < t)) || o == s) continue;
      bool before;
      if (oex < 0) before = (ex >= 0) || (o < s);            // free slots first, by slot index
      else if (ex < 0) before = false;
      else before = (ost < st) || (ost == st && oex < ex);   // then (stamp, resident expert id)
      rank += before ? 1 : 0;
    }
    s_victim[rank] = s;
    atomicAdd(&s_K, 1);  // a count
  }
  __syncthreads();
  const int K = s_K;

  // ---- 4: which misses are worth a fill
  int elig = 0;
  if (cls == 2) {
    const int64_t pz = (c + p.cm.tz - 1) / p.cm.tz, pg = (c + p.cm.tg - 1) / p.cm.tg;
    const int64_t v = pz * p.cm.ns_zc - (p.cm.ns_fill + pg * p.cm.ns_hbm) +
                      (int64_t)p.cm.reuse_credit * (p.cm.ns_zc - p.cm.ns_hbm);
    elig = v > 0;
  }
  if (tid < E) s_elig[tid] = (uint8_t)elig;
  int n_elig;
  block_excl_scan(elig, s_w, n_elig);  // (also orders the s_elig writes before the reads below)

  // ---- 5: fill count
  int q = 0;
  if (n_miss > 0) {
    const int64_t bt = p.cm.bw_fill + p.cm.bw_res;
    int64_t qbw = (2 * (int64_t)n_miss * p.cm.bw_fill + bt) / (2 * bt);
    if (qbw < 1) qbw = 1;
    q = (int)qbw;
    if (q > n_elig) q = n_elig;
    if (q > K) q = K;
  }

  // ---- 6: priority of the eligible misses (tokens descending, id ascending)
  int is_fill = 0;
  if (elig) {
    int rank = 0;
    for (int o = 0; o < E; ++o) {
      if (!s_elig[o] || o == tid) continue;
      const int oc = s_cnt[o];
      rank += (oc > c || (oc == c && o < tid)) ? 1 : 0;
    }
    if (rank < q) { is_fill = 1; s_forder[rank] = tid; }
  }
  __syncthreads();

  // ---- 7: the i-th fill takes the i-th candidate slot
  if (tid < q) {
    const int e = s_forder[tid];
    const int s = s_victim[tid];
    const int old = s_sexp[s];
    if (old >= 0) p.expert_slot[old] = -1;
    p.slot_expert[s] = e;
    p.expert_slot[e] = s;
    p.slot_stamp[s] = t;
    a_forder[tid] = e;
    a_fslot[tid] = s;
    a_fevict[tid] = old;
  }
  __syncthreads();

  // ---- 8: lists and locations
  int n_fill, n_zc;
  const int fpos = block_excl_scan(is_fill, s_w, n_fill);
  if (is_fill) a_fill[fpos] = tid;
  const int is_zc = (cls == 2 && !is_fill);
  const int zpos = block_excl_scan(is_zc, s_w, n_zc);
  if (is_zc) a_zc[zpos] = tid;
  int loc = kLocNotRouted;
  if (cls == 1) loc = slot;
  else if (is_fill) loc = p.expert_slot[tid];  // written in step 7 by this block, barrier above
  else if (is_zc) loc = kLocZeroCopy;
  if (tid < E) a_loc[tid] = loc;

  // work lists for the execution step
  const int resident = (cls == 1 || is_fill);
  const int use_gemm = resident && p.cm.gemm_min_tokens > 0 && c >= p.cm.gemm_min_tokens;
  int n_res, n_gemm;
  const int rpos = block_excl_scan(resident && !use_gemm, s_w, n_res);
  const int gpos = block_excl_scan(use_gemm, s_w, n_gemm);
  if (resident) {
    WorkItem it;
    it.w = p.slots_layer + (size_t)loc * p.S;
    it.expert = tid;
    it.n_tok = c;
    it.off = p.offset[tid];
    it.slot = loc;
    if (use_gemm) p.items_gemm[gpos] = it; else p.items_res[rpos] = it;
  }
  if (is_zc) {
    WorkItem it;
    it.w = p.pool_layer_dev + (size_t)tid * p.S;
    it.expert = tid;
    it.n_tok = c;
    it.off = p.offset[tid];
    it.slot = -1;
    p.items_zc[zpos] = it;
  }
  int pairs_res;
  block_excl_scan(resident ? c : 0, s_w, pairs_res);

  if (tid == 0) {
    int n_res_items = n_res;
    if (p.shared_rec != nullptr) {
      WorkItem it;
      it.w = p.shared_rec;
      it.expert = -1;
      it.n_tok = p.T;
      it.off = 0;
      it.slot = -1;
      p.items_res[n_res_items++] = it;
    }
    PlanHeader h;
    h.step = t;
    h.n_routed = n_routed; h.n_hit = n_hit; h.n_miss = n_miss; h.n_fill = n_fill; h.n_zc = n_zc;
    h.n_res_items = n_res_items; h.n_zc_items = n_zc; h.n_gemm_items = n_gemm;
    h.seq = *p.seq + 1;
    h.pad[0] = h.pad[1] = h.pad[2] = h.pad[3] = h.pad[4] = 0;
    *p.hdr_dev = h;
    *p.seq = h.seq;
    *p.step = t + 1;
    int evictions = 0;
    for (int i = 0; i < n_fill; ++i) evictions += (a_fevict[i] >= 0);
    p.stats[0] += 1;
    p.stats[1] += n_routed;
    p.stats[2] += n_hit;
    p.stats[3] += n_miss;
    p.stats[4] += n_fill;
    p.stats[5] += n_zc;
    p.stats[6] += evictions;
    p.stats[7] += p.offset[E];
    p.stats[8] += pairs_res;
  }
  __syncthreads();
  // mirror the record into mapped host memory for the copy-engine fill path and for reports
  if (p.hdr_host != nullptr) {
    const int n_words = (int)(sizeof(PlanHeader) / 4) + 8 * E;
    const uint32_t *src = reinterpret_cast<const uint32_t *>(p.hdr_dev);
    volatile uint32_t *dst = reinterpret_cast<volatile uint32_t *>(p.hdr_host);
    // arrays first, header (with the sequence number) last
    for (int i = (int)(sizeof(PlanHeader) / 4) + tid; i < n_words; i += blockDim.x) dst[i] = src[i];
    __threadfence_system();
    __syncthreads();
    if (tid < (int)(sizeof(PlanHeader) / 4)) dst[tid] = src[tid];
    __threadfence_system();
  }
}

}  // namespace ftmoe
