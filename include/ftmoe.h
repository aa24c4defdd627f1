/*
 * ftmoe.h -- C ABI of the expert-cached Mixture-of-Experts layer for NVIDIA B200 (sm_100a).
 *
 * The library implements one thing: the MoE layer of an engine whose complete routed-expert
 * weights live in a pinned host pool (the source of truth) while a fixed pool of HBM slots caches
 * the experts in use (paper Sec. 3: two-level expert-memory hierarchy; each slot holds every tensor
 * of one (layer, expert) pair).  Per step and layer the caller runs
 *
 *     ft_moe_route -> ft_moe_plan -> ft_moe_fill -> ft_moe_forward
 *
 * route   : top-k gating with softmax over the selected logits, stable expert-sorted permutation.
 * plan    : slot-table lookup gives the hit set H; the m unique misses M are split into a fill set
 *           F (|F| = q, Eq. 1 and Eq. 4 of the paper) and an in-place set served by zero-copy reads
 *           of the mapped host pool (the paper's CPU branch, kept on the GPU here); LRU victims.
 * fill    : copies pool records of F into their slots over the host link.
 * forward : grouped SwiGLU expert FFN over H u F (from slots) and Z (from host), gate-weighted sum.
 *
 * Conventions
 *   - Every function returns an ft_status_t, never aborts, never throws, never traps on the device.
 *   - "dev" pointers are device pointers, "host" pointers are host pointers; streams are
 *     cudaStream_t passed as void*.  One host thread per handle.
 *   - Asynchronous device-detected conditions (non-finite logits) are latched in a device status
 *     word and reported by the next synchronising call (ft_moe_plan with a non-null out pointer,
 *     ft_moe_fill in copy-engine mode, the ft_moe_get_* calls, ft_moe_sync_status).
 *   - T = 0 is a no-op that does not advance the layer's step counter.
 *   - Device buffers of activations (x_dev, y_dev) and records must be 16-byte aligned (the kernels use vector
 *     accesses); a misaligned pointer is FT_ERR_INVALID_ARG, never a device fault.
 *
 * Expert record layout (pool records and slots are byte-identical, so a fill is one contiguous copy)
 *   record index in the pool: layer * n_experts + expert (the flattened id of paper Sec. 4.2).
 *   FT_W_BF16     : tensor-core tile order.  inter/16 units of 16 neurons, 96*hidden bytes each: a gate part, an
 *                   up part and a down part of 32*hidden bytes.  Gate/up part: 1 KiB tiles of 16 neurons x 32
 *                   hidden indices = two groups of 8 neuron rows of 64 bytes; down part: 512-byte tiles of 16 output
 *                   columns x the unit's 16 neurons = two groups of 8 column rows of 32 bytes.  The 16-byte chunks of
 *                   a row are stored swizzled (the tensor core's 64-byte / 32-byte swizzle of a K-major operand).
 *                   With n the neuron, i the hidden index, c the output column, offsets in 2-byte elements,
 *                   r = n%8 for gate/up and r = c%8 for down:
 *                     W_gate[i][n] at 48*hidden*(n/16) + 512*(i/32) + 256*((n%16)/8) + 32*r
 *                                     + 8*(((i%32)/8) ^ (r>>1)) + i%8
 *                     W_up[i][n]   at the same place + 16*hidden
 *                     W_down[n][c] at 48*hidden*(n/16) + 32*hidden + 256*(c/16) + 128*((c%16)/8) + 16*r
 *                                     + 8*(((n%16)/8) ^ (r>>2)) + n%8
 *                   A warp's 16-byte (gate/up) or 8-byte (down) loads of a tile cover whole 128-byte lines in lane
 *                   order and land directly in mma.sync fragments; a bulk copy of the same bytes into shared memory
 *                   is a valid swizzled K-major tcgen05 operand, so the prefill GEMMs consume the tiles as they are.
 *                   S = 3*inter*hidden*2 bytes.
 *   FT_W_INT4_G128: 4-bit two's-complement codes in [-8,7] and bf16 scales, weight = scale * code, groups of 128
 *                   along the contraction dimension (G = hidden/128 hidden groups for gate/up, NG = inter/128 neuron
 *                   groups for down), in tensor-core tile order.  Three sections:
 *                   A. inter/16 units of 16 neurons, 2112*G bytes each: G gate tiles, G up tiles (1 KiB each), gate
 *                      scales, up scales (32*G bytes each).  A tile is 16 neuron rows x 128 hidden indices = 16
 *                      rows of 64 bytes; in a row the code of hidden index 128*grp + 32*j + 8*q + e is nibble e
 *                      (bits 4e..4e+3) of the little-endian 32-bit word j of the 16-byte chunk q.  The scales of a
 *                      tile are 8 pairs (row r, row r+8) of bf16.
 *                   B. down codes: for each column block cb (CBW = 64*min(16, hidden/64) columns), neuron group ng
 *                      and 16-neuron step uu of the group: CBW/64 x 512 bytes; in each 512 bytes lane l = 4g + q
 *                      owns 16 bytes = 4 words, word j belongs to the 16-column tile 4w + j of the block; its nibble
 *                      e is the code of column g + 8*(e & 1) of the tile and neuron 4q + e/2 of the step.
 *                   C. down scales sd[ng][column] in the order (ng, cb, w, g, j, half): 8 pairs per tile again.
 *                   In both code sections (w & 0x0F0F0F0F) ^ 0x08080808 of a word w and of w >> 4 are operand
 *                   registers of the int8 tensor-core instruction as they are (bytes code + 8; the kernels subtract
 *                   8 x the activation sums).
 *                   S = 3*inter*hidden/2 + (2*inter*hidden/128 + (inter/128)*hidden)*2 bytes.
 *   FT_W_MXFP4    : microscaling FP4 (paper Sec. 5.1 serves MXFP4 experts): 4-bit e2m1 codes (bit 3 sign, bits 2..0
 *                   index the magnitudes 0, 0.5, 1, 1.5, 2, 3, 4, 6) and one scale byte b per 32 consecutive elements
 *                   of the contraction dimension, weight = (+-magnitude) * 2^(b-127).  The code sections are those of
 *                   FT_W_INT4_G128; a unit of section A is 2176*G bytes: its tiles, then per gate tile and per up
 *                   tile 64 scale bytes = for r in 0..7 the four block scales (j = 0..3) of row r, then those of row
 *                   r+8.  Section C: order (ng, cb, w, g, j, half, m), i.e. per lane g 32 bytes = for each tile j and
 *                   column half the scales of the four 32-neuron blocks m of the 128-neuron group.
 *                   S = 3*inter*hidden/2 + 3*inter*hidden/32 bytes.  Shapes as for int4.
 *   FT_W_MXFP4_TC : the numbers of FT_W_MXFP4 stored as operand images of the block-scaled tensor-core instruction
 *                   (tcgen05.mma kind::mxf4: packed e2m1 operands in K-major core matrices of 8 rows x 16 bytes, scale
 *                   factors in groups of 128 rows x 4 blocks), so that the decode kernels feed the record's bytes to
 *                   the instruction as they are.  Section A: for each group of 128 neurons ng and each 128 hidden
 *                   indices st (in that order) 17408 bytes = gate image (8192), up image (8192), gate scales (512), up
 *                   scales (512).  Section B: for each group of 128 output columns cg and each 128 neurons st 8704
 *                   bytes = image, scales.  In an image the code of (row r < 128, contraction index k < 128) is a
 *                   nibble (low when k is even) of byte 4096*(k/64) + 2048*((k%64)/32) + 128*(r/8) + 16*(r%8) +
 *                   (k%32)/2; the scale byte of (row r, block b < 4) is byte 16*(r%32) + 4*(r/32) + b.  Rows are
 *                   neurons (A) or output columns (B).  S as for FT_W_MXFP4.  The streaming kernels serve any token
 *                   count (8 tokens of an expert per weight pass; the bf16 activations are re-expressed as sums of
 *                   six block-scaled e2m1 vectors, error <= 3^-6 of a block's largest magnitude); on the tensor-core
 *                   prefill path the experts are expanded to bf16 records like the other 4-bit formats.
 *   FT_W_NVFP4    : two-level scaled FP4 (paper Sec. 5.1, expert representations): the same e2m1 codes with one
 *                   unsigned e4m3 scale byte b (exponent field E = b >> 3, mantissa M = b & 7: 2^(E-7) * (1 + M/8),
 *                   or 2^-6 * M/8 when E = 0; b <= 0x7E) per 16 consecutive elements of the contraction dimension and
 *                   one float32 scale per matrix: weight = (+-magnitude) * block scale * matrix scale.  Differences
 *                   from FT_W_MXFP4: in a gate/up tile row, nibble e of word j of chunk q is the code of hidden index
 *                   128*grp + 32*j + 16*(e & 1) + 4*q + e/2, so that the even nibbles of the row's words j are one
 *                   scale block and the odd nibbles the next (K = 16 tensor-core steps); a unit of section A is
 *                   2304*G bytes with 128 scale bytes per tile = for r in 0..7 the eight block scales of row r, then
 *                   those of row r+8.  Section B is unchanged (a 16-neuron unit is one scale block).  Section C:
 *                   order (ng, cb, w, g, j, half, unit), per lane g 64 bytes = for each tile j and column half the
 *                   scales of the eight 16-neuron blocks of the 128-neuron group.  Then the matrix scales of gate,
 *                   up and down as three little-endian float32, zero-padded to 256 bytes.
 *                   S = 3*inter*hidden/2 + 3*inter*hidden/16 + 256 bytes.  Shapes as for int4.
 *   Shape limits: bf16: hidden in {256, 512, 1024, 2048}, inter % 16 == 0; int4, mxfp4 and nvfp4: hidden in
 *   {512, 1024, 2048, 4096, 7168, 8192}, inter % 128 == 0; n_experts <= 1024;
 *   top_k <= min(n_experts, 32); slots per table (slots_per_layer, or n_layers*slots_per_layer with global_pool)
 *   <= 6144.  The tensor-core prefill path (gemm_min_tokens > 0) needs slots_per_layer > 0, hidden % 256 == 0 and
 *   inter % 256 == 0; 4-bit experts on that path are first expanded, once per call, to bf16 records in a
 *   scratch pool of slots_per_layer x 3*inter*hidden*2 bytes owned by the handle (not with global_pool).
 */
#ifndef FTMOE_H_
#define FTMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ft_moe ft_moe_t; /* opaque: owns the slot pool, the tables, scratch, events */

typedef enum {
  FT_OK = 0,
  FT_ERR_INVALID_ARG = 1,
  FT_ERR_NOT_PINNED = 2,   /* host_pool is not pinned + mapped host memory (no pageable fallback) */
  FT_ERR_OOM = 3,
  FT_ERR_CUDA = 4,
  FT_ERR_STATE = 5,        /* calls out of order for this layer */
  FT_ERR_TIMEOUT = 6,      /* a bounded device-side wait gave up */
  FT_ERR_NONFINITE = 7,    /* NaN/Inf in the router logits */
  FT_ERR_UNSUPPORTED = 8
} ft_status_t;

typedef enum { FT_W_BF16 = 0, FT_W_INT4_G128 = 1, FT_W_MXFP4 = 2, FT_W_NVFP4 = 3, FT_W_MXFP4_TC = 4 } ft_wdtype_t;

/* How ft_moe_fill moves records.  Both give byte-identical slots. */
typedef enum {
  FT_FILL_COPY_ENGINE = 0, /* host waits for the plan record, then one cudaMemcpyAsync per fill */
  FT_FILL_SM = 1           /* one fixed-shape copy kernel driven by the device-resident fill list
                              (paper Sec. 4.1: a work list plus a valid count); no host wait */
} ft_fill_mode_t;

typedef struct {
  uint32_t struct_size;     /* = sizeof(ft_moe_config_t) */
  int32_t device;           /* CUDA device ordinal */
  int32_t n_layers;
  int32_t hidden;           /* d */
  int32_t inter;            /* I */
  int32_t n_experts;        /* E routed experts per layer */
  int32_t top_k;
  int32_t n_shared;         /* 0 or 1 always-resident shared expert per layer */
  int32_t wdtype;           /* ft_wdtype_t */
  int32_t slots_per_layer;  /* N_s >= 0; 0 = every routed expert is served zero-copy */
  int32_t max_tokens;       /* largest T of any call */
  int32_t fill_mode;        /* ft_fill_mode_t */
  const void *host_pool;    /* HOST, caller-owned, pinned + mapped, n_layers*n_experts records;
                               must stay valid and unmodified for the life of the handle */
  size_t host_pool_bytes;
  const void *shared_weights; /* HOST, n_layers*n_shared records, copied to HBM at create; may be
                                 NULL when n_shared == 0 */
  /* Frozen integer constants of the plan's cost model, MB/s (1e6 bytes/s); all must be > 0 except
   * bw_zc_residual_MBps which may be 0 (then every miss that can get a slot is filled: the limit
   * of Eq. 4 in which the split degenerates to on-demand fills only, see the text after Eq. 4). */
  uint32_t bw_fill_MBps;        /* B_f: copy-engine fill rate            (the paper's B_PCIe)      */
  uint32_t bw_zc_MBps;          /* B_z: zero-copy read rate alone                                   */
  uint32_t bw_zc_residual_MBps; /* B_r: zero-copy rate while fills saturate the link (Eq. 2)        */
  uint32_t bw_hbm_MBps;         /* B_h: HBM streaming rate                                          */
  int32_t reuse_credit;         /* R >= 0: future link passes a fill is credited with saving        */
  int32_t zc_tokens_per_pass;   /* T_z >= 1: tokens one zero-copy weight pass serves                */
  int32_t hbm_tokens_per_pass;  /* T_g >= 1: tokens one resident weight pass serves                 */
  int32_t gemm_min_tokens;      /* experts with at least this many tokens and a slot use the
                                   tensor-core grouped GEMM; 0 = never                              */
  int32_t split_min_pairs;      /* calls with T*top_k at or above this evaluate the hit experts in a
                                   launch of their own while the fills are still in flight, the
                                   filled experts after the fill event; 0 = always one launch after
                                   the fills (cheaper for a few tokens)                             */
  int32_t global_pool;          /* 0: every layer owns slots_per_layer slots (an LRU per layer).
                                   1: one pool of n_layers*slots_per_layer slots and one LRU clock
                                   shared by all layers, keyed by the flattened id layer*n_experts +
                                   expert (paper Sec. 3: a single elastic cache shared by all MoE
                                   layers); slot indices, ft_moe_get_slot_table and fill_evicted then
                                   refer to the shared pool / flattened ids                         */
} ft_moe_config_t;

/* Host-visible plan of one (layer, step).  The caller provides arrays of n_experts int32 each. */
typedef struct {
  int64_t step;
  int32_t n_routed, n_hit, n_miss, n_fill, n_zc;
  int32_t *hit, *miss, *fill, *zc;  /* ascending expert ids */
  int32_t *fill_order;              /* F in priority order */
  int32_t *fill_slot;               /* slot of fill_order[i] */
  int32_t *fill_evicted;            /* expert evicted from that slot, -1 if it was free */
  int32_t *loc;                     /* [n_experts]: slot >= 0 | -1 not routed | -2 zero-copy */
} ft_moe_plan_t;

enum { FT_STAT_STEPS = 0, FT_STAT_ROUTED, FT_STAT_HITS, FT_STAT_MISSES, FT_STAT_FILLS, FT_STAT_ZC,
       FT_STAT_EVICTIONS, FT_STAT_PAIRS, FT_STAT_PAIRS_RESIDENT, FT_STAT_PAIRS_GEMM, FT_STAT_COUNT };

/* S, the bytes of one expert record for this configuration (0 if the shape is not supported). */
size_t ft_moe_expert_bytes(const ft_moe_config_t *cfg);

/* Pinned + mapped host memory for an expert pool (cudaHostAlloc, portable | mapped).  HOST pointer
 * out; free with ft_moe_host_free.  Contents are uninitialised. */
ft_status_t ft_moe_host_alloc(size_t bytes, void **out_host);
ft_status_t ft_moe_host_free(void *host);
/* Pins and maps memory the caller already owns (cudaHostRegister, portable | mapped), e.g. a file mapping
 * of the pool that several processes on the node share, or a pool that was read from disk into ordinary
 * memory first and is pinned only afterwards (paper Sec. 3.3: pin after the buffers are filled).  HOST
 * pointer, page aligned; undo with ft_moe_host_unregister before the memory goes away. */
ft_status_t ft_moe_host_register(void *host, size_t bytes);
ft_status_t ft_moe_host_unregister(void *host);

/* Validates the configuration, checks that host_pool is pinned and mapped (else FT_ERR_NOT_PINNED),
 * allocates n_layers*slots_per_layer slots (FT_ERR_OOM if HBM cannot hold them) and empty tables
 * (paper Sec. 3.3: the first request is served with a cold cache). */
ft_status_t ft_moe_create(const ft_moe_config_t *cfg, ft_moe_t **out);
ft_status_t ft_moe_destroy(ft_moe_t *h);

/* Bandwidth profiling at deployment (paper Sec. 3.2: the two bandwidths of Eq. 2 are measured on the machine that
 * serves): out_MBps = { fill (pinned H2D copy of records), zero-copy alone, zero-copy while the
 * copy engine is saturated, HBM streaming }.  Measures only; plans keep using the frozen constants
 * given at create.  Synchronises the device. */
ft_status_t ft_moe_calibrate(ft_moe_t *h, uint32_t out_MBps[4]);

/* Step 1+2 (paper Sec. 3.2: the router runs on the GPU).  logits_dev: DEVICE fp32 [T][n_experts]
 * row-major.  Produces, on the device: ids[T][k] (logit descending, id ascending), gate weights
 * w[T][k] = softmax over the selected logits, count[E], offset[E+1], and the stable expert-sorted
 * permutation perm[P] / inv[P] of the P = T*k pairs p = t*k + j. */
ft_status_t ft_moe_route(ft_moe_t *h, int layer, const float *logits_dev, int T, void *stream);

/* Step 3 (paper Sec. 3.2 Eq. 1-4; Sec. 4.1: the cache is controlled on the device): one device kernel
 * deduplicates the routed experts, classifies them against the slot table, refreshes the stamps of
 * hits, orders the evictable slots (free first, then least recently used, ties to the lower
 * resident expert id), sizes the fill set q = min(max(1, round(m*B_f/(B_f+B_r))), eligible, K),
 * picks F (most tokens first), assigns slots, and rewrites expert ids into slot ids or the
 * zero-copy flag.  out_host may be NULL (no synchronisation); otherwise the call waits for the
 * plan and fills *out_host (HOST arrays owned by the caller). */
ft_status_t ft_moe_plan(ft_moe_t *h, int layer, ft_moe_plan_t *out_host, void *stream);

/* Step 4 (paper Sec. 3.2: the fill set F is copied into the cache as one batch before the grouped
 * evaluation; Sec. 4.1: one fixed-shape transfer driven by a device-resident source/destination list with a
 * valid count): for every (expert, slot) of F copy the S-byte pool record into the slot on copy_stream and
 * record the handle's fill event there.  The copies are ordered after the plan. */
ft_status_t ft_moe_fill(ft_moe_t *h, int layer, void *copy_stream);

/* Full-layer prefetch for prefill (paper Sec. 3.1: while layer l is being computed, a transfer stream loads the
 * complete expert set of layer l+1, before its routing is known, into the second of two full-layer buffers taken
 * from the same slot pool; the survivors seed the decode cache).  Admits every expert of `layer` that is not yet
 * resident through the ordinary residency machinery -- one plan over "all experts routed once" on `stream`, then
 * the fills on copy_stream (NULL = the handle's own copy stream) -- so the victims are the least recently used
 * slots, i.e. those of layers already computed.  Nothing is evaluated and no step of the layer is counted; the
 * layer's later route/plan finds hits.  The handle's fill event is recorded: the next ft_moe_forward waits for
 * it.  Needs room for two full-layer buffers: with global_pool a shared pool of at least 2*n_experts slots,
 * otherwise slots_per_layer >= n_experts; else FT_ERR_UNSUPPORTED and the caller falls back to on-demand fills
 * (Sec. 3.1 names the same fallback for budgets without room for two full-layer buffers).  The layer must be idle (no route/plan/fill of it pending). */
ft_status_t ft_moe_prefetch_layer(ft_moe_t *h, int layer, void *stream, void *copy_stream);

/* Steps 5+6 (paper Sec. 3.2: grouped evaluation of H u F on the GPU, the in-place set beside it, and an exact
 * merge of the partial sums -- no approximation of the MoE output): x_dev DEVICE bf16 [T][hidden], y_dev DEVICE
 * bf16 [T][hidden] (written), both 16-byte aligned.  Waits (on the
 * stream, not the host) for the fill event, evaluates the SwiGLU expert FFN of every routed expert
 * from its slot or, for the zero-copy set, straight from the mapped host pool, and writes
 * y[t] = sum_j w[t][j] * FFN_{ids[t][j]}(x[t]) (+ the shared expert) rounded once to bf16. */
ft_status_t ft_moe_forward(ft_moe_t *h, int layer, const void *x_dev, void *y_dev, void *stream);

/* route + plan + fill + forward of one layer in one call (the per-layer control flow of paper Sec. 4.1, kept on
 * the device); fills go to the handle's own copy stream. */
ft_status_t ft_moe_layer(ft_moe_t *h, int layer, const float *logits_dev, const void *x_dev,
                         void *y_dev, int T, void *stream);

/* The same through HOST buffers (pinned or pageable): copies logits and x to the device, runs the
 * layer, copies y back and waits for it. */
ft_status_t ft_moe_layer_host(ft_moe_t *h, int layer, const float *logits_host, const void *x_host,
                              void *y_host, int T, void *stream);

/* ---- introspection (tests, reports); each synchronises the device ---- */
/* Results of the latest ft_moe_route of `layer` (every layer keeps its own routing arrays, plan record and work
 * lists, so route/plan/fill of several layers may be issued before their forward calls).  HOST arrays:
 * ids[T*k], w[T*k], count[E], offset[E+1], perm[T*k], inv[T*k]; any may be NULL. */
ft_status_t ft_moe_get_routing(ft_moe_t *h, int layer, int32_t *ids, float *w, int32_t *count,
                               int32_t *offset, int32_t *perm, int32_t *inv);
/* HOST arrays slot_expert[N_s] (-1 free), slot_stamp[N_s] (-1 never used), expert_slot[E]. */
ft_status_t ft_moe_get_slot_table(ft_moe_t *h, int layer, int32_t *slot_expert,
                                  int64_t *slot_stamp, int32_t *expert_slot);
ft_status_t ft_moe_read_slot(ft_moe_t *h, int layer, int slot, void *host_dst /* S bytes */);
/* counters[FT_STAT_*], accumulated since create/reset. */
ft_status_t ft_moe_get_stats(ft_moe_t *h, int layer, uint64_t *counters, int n);
/* Empties the slot table and zeroes step counter and statistics; layer = -1 for all layers.  (Paper Sec. 3.3: GPU
 * residency is disposable -- the host pool is the source of truth and a cold cache is served by the ordinary miss
 * path -- so a reset never loses anything but speed.) */
ft_status_t ft_moe_reset(ft_moe_t *h, int layer);
/* Runtime cache reconfiguration (paper Sec. 3.3): rebuilds the slot pool for a new budget of
 * slots_per_layer slots per layer (n_layers * slots_per_layer shared slots with global_pool) without touching
 * the host pool.  Call it at a safe point (no call of this handle in flight; it waits for the device).  The
 * cache restarts empty, step counters and statistics are kept.  FT_ERR_OOM leaves the handle with zero slots. */
ft_status_t ft_moe_resize(ft_moe_t *h, int slots_per_layer);
/* Waits for the device and returns (and clears) the latched device status. */
ft_status_t ft_moe_sync_status(ft_moe_t *h);
/* Duration of the most recent ft_moe_fill's copies in microseconds and their bytes (waits for them). */
ft_status_t ft_moe_last_fill(ft_moe_t *h, float *out_us, uint64_t *out_bytes);
/* Per-kernel device timing with CUDA events on the launching stream.  enable(1) clears the
 * accumulators and brackets every later launch with two events; read() waits for the device and
 * returns, per kind FT_TIME_*, the summed microseconds and the number of timed launches since
 * enable.  Timing adds two event records per launch, so throughput is measured with it off. */
enum { FT_TIME_ROUTE = 0, FT_TIME_PLAN, FT_TIME_FFN_ZC, FT_TIME_FFN_RES, FT_TIME_FINALIZE, FT_TIME_FILL,
       FT_TIME_GATHER, FT_TIME_GEMM1, FT_TIME_GEMM2, FT_TIME_COMBINE, FT_TIME_COUNT };
ft_status_t ft_moe_timing_enable(ft_moe_t *h, int on);
ft_status_t ft_moe_timing_read(ft_moe_t *h, double *out_us, uint64_t *out_launches, int n);
/* Per-CTA record of the latest bf16 streaming-kernel launch: out[4*i .. 4*i+3] = global timer (ns) at the
 * start and at the end of CTA i's streaming work, 16-neuron blocks it streamed, segments (expert, pass) it
 * touched (for the CTA that finalized y: minus the global timer when it finished).  n_ctas
 * entries at most (one CTA per SM).  Waits for the device. */
ft_status_t ft_moe_get_cta_trace(ft_moe_t *h, int64_t *out, int n_ctas);
/* Changes split_min_pairs of a live handle (see ft_moe_config_t); takes effect at the next ft_moe_forward.
 * Used to time the streaming kernel alone (0) or overlapped with the fills. */
ft_status_t ft_moe_set_split_min_pairs(ft_moe_t *h, int pairs);
/* How ft_moe_forward launches the bf16 streaming kernel.  0 (default): a plain launch.  1: a programmatic
 * dependent launch -- the grid may be scheduled while the preceding kernel of the stream is still running, and
 * waits for that kernel's completion before it reads anything; results are the same as with 0, only the launch
 * latency is hidden.  2: as 1, but the grid waits only before its first write to the output accumulator, so its
 * weight streaming overlaps the tail of the preceding kernel; the caller asserts that x_dev, the slots and the plan
 * of this layer are not produced by that preceding kernel (e.g. forward calls of several already planned layers
 * issued back to back).  For FT_W_MXFP4_TC handles mode 2 lets a call's first two kernels start while the call
 * before is in its last kernel (calls with at most 8 tokens; not meant for replay from a captured graph, where the
 * completion counts that order the calls are frozen).  Takes effect at the next ft_moe_forward. */
ft_status_t ft_moe_set_launch_overlap(ft_moe_t *h, int mode);
/* Test hook for the failure path of the bounded device-side waits (every wait of a kernel on an mbarrier gives up
 * after a limited number of polls, latches FT_ERR_TIMEOUT in the device status word, lets the copies already in
 * flight land and runs to completion: nothing traps, faults or hangs).  withhold_mask: FT_DEBUG_WITHHOLD_* bits;
 * the named kernel's producer then leaves out one copy of its first stage, so the consumer's wait can never be
 * satisfied.  wait_polls: the poll limit of every wait from now on (0 = the default, 2^22).  The setting is per
 * process and device and stays until changed; call with (0, 0) to restore normal operation.  The output of a
 * call that timed out is unspecified; ft_moe_sync_status reports FT_ERR_TIMEOUT once, and after ft_moe_reset
 * the handle works as before.  Waits for the device. */
enum { FT_DEBUG_WITHHOLD_FILL = 1,      /* device-driven fill kernel (FT_FILL_SM) */
       FT_DEBUG_WITHHOLD_GEMM = 4,      /* prefill gate/up grouped GEMM */
       FT_DEBUG_WITHHOLD_TC = 8 };      /* gate/up kernel of the FT_W_MXFP4_TC decode path (its down kernel then waits,
                                           bounded, for h that never comes) */
/* (The bf16 and int4 streaming kernels load weights straight into registers and contain no waits.) */
ft_status_t ft_moe_debug_inject(ft_moe_t *h, uint32_t withhold_mask, uint32_t wait_polls);
/* Number of kernels this handle has launched since create. */
ft_status_t ft_moe_launch_count(ft_moe_t *h, uint64_t *out);
const char *ft_moe_status_string(ft_status_t s);
/* Text of the CUDA runtime error behind the most recent FT_ERR_CUDA / FT_ERR_OOM of this process. */
const char *ft_moe_last_cuda_error(void);

/* An expert FFN for callers that are not allowed to allocate.  (The paper has no counterpart: this
 * is a convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a serving loop with a frozen memory
 * budget, a plug-in inside a process whose device memory pool belongs to the host application, a
 * component started after the application has already claimed all of HBM.  Such a caller cannot
 * create an ft_moe_t handle (ft_moe_create allocates slots, tables and scratch), but it can still
 * evaluate one expert on weights it already holds in device memory.
 *
 * What it does: y[t] = (SiLU(x[t] W_gate) * (x[t] W_up)) W_down for t < T, with the same streaming
 * tensor-core kernel ft_moe_forward uses for resident bf16 experts.
 *   record_dev : DEVICE, one FT_W_BF16 expert record (layout above), 16-byte aligned, caller-owned
 *   x_dev      : DEVICE bf16 [T][hidden], 16-byte aligned, caller-owned, read only
 *   y_dev      : DEVICE bf16 [T][hidden], 16-byte aligned, caller-owned, written
 *   stream     : cudaStream_t; the call only enqueues work
 * The kernel's scratch (an fp32 [T][hidden] accumulator and a few control words) lives in a fixed
 * array of FT_NOALLOC_MAX_TOKENS * FT_NOALLOC_MAX_HIDDEN * 4 + 256 bytes (512.25 KiB) in the library's
 * device data segment; every GPU that loads the library holds it until the process exits.  The
 * call makes no cudaMalloc / cudaFree and uses no allocating library routine.
 *
 * Limits and errors: T in [1, FT_NOALLOC_MAX_TOKENS] and hidden <= FT_NOALLOC_MAX_HIDDEN, otherwise
 * FT_ERR_INVALID_ARG (the scratch cannot be grown); hidden in {256, 512, 1024, 2048} and
 * inter % 16 == 0, otherwise FT_ERR_UNSUPPORTED; null or misaligned pointers FT_ERR_INVALID_ARG.
 * The calling thread's current device is the same after the call as before it.  The device must already have a
 * context (creating one allocates): make any other CUDA call on it first.
 *
 * First call on a device: looks up the device address of the scratch array and raises the kernel's
 * shared-memory limit for that device (no allocation, but not stream work either), so make the
 * first call on each device before any stream capture begins.
 *
 * Sharing: all calls on a device use the same array, which keeps whatever the last call left; each
 * call clears the part it needs on its own stream before use.  Two calls that can overlap on the GPU
 * (different streams without an ordering between them, or several host threads) race on the array
 * and give wrong results: order them. */
#define FT_NOALLOC_MAX_TOKENS 64
#define FT_NOALLOC_MAX_HIDDEN 2048
ft_status_t ft_moe_ffn_noalloc(int device, const void *record_dev, int hidden, int inter,
                               const void *x_dev, void *y_dev, int T, void *stream);
/* Waits for the device and returns (and clears) what the ft_moe_ffn_noalloc kernels latched there since the last
 * call of this function: FT_OK, or FT_ERR_TIMEOUT if a bounded device-side wait gave up (the y of that call is
 * then incomplete).  Allocates nothing. */
ft_status_t ft_moe_ffn_noalloc_status(int device);

#ifdef __cplusplus
}
#endif
#endif /* FTMOE_H_ */
