/* libra.h — C ABI of the B200 pool-attention library (liblibra.so).
 *
 * The library computes causal, sample-masked ("document-masked") attention forward and
 * backward over a pool of packed sequences on one GPU, with the work cut into
 * sequence-block x head-shard tiles (SH-Tiles) that are weighted by the causal
 * query-key pairs they cover and placed heaviest-first on persistent CTAs.
 *
 * Conventions for every entry point
 *   - returns 0 on success, a negative LIBRA_ERR_* code otherwise; never throws, aborts
 *     or prints;
 *   - pointers named *_dev are DEVICE pointers owned by the caller, pointers named
 *     *_host are HOST pointers owned by the caller; nothing is retained after the call
 *     returns except inside a libra_plan_t;
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream);
 *     work is enqueued on it and the call returns without synchronising unless stated;
 *   - tensors are contiguous bf16 in the packed "thd" layout: q, out, dout, dq are
 *     [T, Hq, d]; k, v, dk, dv are [T, Hkv, d]; lse is fp32 [Hq, T]; T = cu_seqlens[n];
 *     query head h reads kv head h / (Hq / Hkv);
 *   - cu_seqlens is int32 [n_samples + 1], starts at 0, non-decreasing (repeated offsets
 *     = empty samples are allowed), ends at T.
 *
 * Citations name the paper's section, equation or algorithm that defines the operation.
 */
#ifndef LIBRA_H_
#define LIBRA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define LIBRA_OK                 0
#define LIBRA_ERR_INVALID_ARG   (-1)  /* null pointer, non-positive size, H does not divide Hq, ... */
#define LIBRA_ERR_UNSUPPORTED   (-2)  /* head_dim not in {64,128,256}, tile size the kernels cannot run */
#define LIBRA_ERR_PLAN_MISMATCH (-3)  /* plan was built for another T / head count / direction      */
#define LIBRA_ERR_CUDA          (-4)  /* a CUDA runtime or driver call failed                        */
#define LIBRA_ERR_OVERFLOW      (-5)  /* tile ids or loads would not fit their integer types         */
#define LIBRA_ERR_TIMEOUT       (-6)  /* a bounded device-side wait gave up (see libra_busy_times)   */
#define LIBRA_ERR_BAD_SEQLENS   (-7)  /* cu_seqlens failed the device-side check                      */
#define LIBRA_ERR_NO_DEVICE     (-8)  /* no CUDA device / not an sm_100 device                        */
#define LIBRA_ERR_SCRATCH_TOO_SMALL (-9) /* problem needs more than the library's built-in scratch    */

/* Tile weight used by the placement.
 * PAIRS  : the paper's Eq. 6, the causal (query, key) pairs the tile covers.
 * BLOCKS : a time proxy the paper does not have (it notes in Section 3.2 that a FLOPs-balanced
 *          assignment need not be time-balanced): the kernels spend the same time on a
 *          cost_block x cost_block block of the score matrix whether all of it or only a corner is
 *          visible, so the weight counts blocks instead of pairs.  The token axis is cut into chunks
 *          at multiples of cost_block; a query-major tile weighs, summed over the row chunks it
 *          holds,  8 * (key chunks that hold a key some row of the chunk attends) + unit_cost_q;
 *          a key-major tile, summed over its key chunks,
 *          8 * (query chunks that hold a query attending some key of the chunk) + unit_cost_kv.
 *          Ordering, placement and tie-breaks are those of Algorithm 2 in both models. */
#define LIBRA_WEIGHT_PAIRS   0
#define LIBRA_WEIGHT_BLOCKS  1

#define LIBRA_DIR_Q   1   /* query-major tiles (forward)  */
#define LIBRA_DIR_KV  2   /* key-major tiles   (backward) */
#define LIBRA_DIR_PAIR 4  /* pair tiles: key block x query chunk x kv head (the fused backward); only on request */

/* kernels, for libra_busy_times / libra_kernel_time_ms */
#define LIBRA_KERNEL_FWD       1   /* forward kernel (walks the query-major lists)            */
#define LIBRA_KERNEL_BWD_DKDV  2   /* backward dK/dV kernel (walks the key-major lists)       */
#define LIBRA_KERNEL_BWD_DQ    3   /* backward dQ kernel (walks the query-major lists)        */
#define LIBRA_KERNEL_BWD_PREP  4   /* backward row statistics (timing only: it keeps no busy times) */
#define LIBRA_KERNEL_BWD_FUSED 5   /* fused backward kernel incl. clearing its accumulators (walks the pair tiles) */
#define LIBRA_KERNEL_BWD_POST  6   /* fused backward: scaling and rounding of the accumulators (timing only)   */

typedef struct libra_plan libra_plan_t;   /* opaque, library-owned */

typedef struct {
    int     n_workers;     /* persistent CTAs to place onto; 0 = one per SM of the current device */
    int     directions;    /* any of LIBRA_DIR_Q | LIBRA_DIR_KV | LIBRA_DIR_PAIR; 0 = Q and KV      */
    int     tile_kv;       /* key-major block size in tokens; 0 = 128                              */
    int     n_heads_kv;    /* key-major head shards; 0 = same as n_heads                           */
    int64_t total_tokens;  /* T if the caller knows it; 0 = read cu_seqlens[n] back (one 4-byte
                              synchronous copy on `stream`)                                         */
    int     weight_model;  /* LIBRA_WEIGHT_PAIRS (0, Eq. 6) or LIBRA_WEIGHT_BLOCKS                  */
    int     cost_block;    /* LIBRA_WEIGHT_BLOCKS: edge of the square blocks counted; 0 = 128      */
    int     unit_cost_q;   /* LIBRA_WEIGHT_BLOCKS: added per row chunk of a query-major tile, in
                              eighths of a block (>= 0)                                             */
    int     unit_cost_kv;  /* same per key chunk of a key-major tile                                */
    int     pair_chunk;    /* LIBRA_DIR_PAIR: tokens per query chunk, a multiple of the key block; 0 = 4096
                              (doubled by the planner while there are more than 262144 pair-blocks)    */
} libra_plan_opts;

typedef struct {
    int64_t total_tokens;  /* T */
    int     n_samples;     /* n */
    int     hq, hkv;       /* query / kv heads, hkv divides hq */
    int     head_dim;      /* 64, 128 or 256 */
    float   softmax_scale; /* 0 = 1/sqrt(head_dim) */
} libra_dims;

/* ---- planning ------------------------------------------------------------------------
 * SH-Tile construction (Section 4.3.1, Eq. 5), tile weights (Eq. 6) and heaviest-first
 * placement (Algorithm 2 with the communication term identically zero, which makes both
 * of its branches "least-loaded worker, lowest index on ties" and removes the soft cap).
 *
 *   blocks : the token axis [0, T) cut at multiples of the tile size (last block may be
 *            short; no cuts at sample boundaries); NB = ceil(T / tile)
 *   tiles  : id t = b * H + h for block b and head shard h (H = n_heads shards)
 *   weight : LIBRA_DIR_Q  - block b holds queries: sum over its tokens of (p + 1), p the
 *                           token's position inside its sample (= keys it attends)
 *            LIBRA_DIR_KV - block b holds keys: sum over its tokens of (len - p)
 *                           (= queries that attend the key); same for every h
 *   order  : tiles by decreasing weight, then increasing id
 *   place  : each tile in that order to the worker with the smallest load so far
 *   lists  : per-worker tile lists in placement order, CSR (cta_offsets, cta_tiles)
 *
 * All planning runs in device kernels on `stream`; results stay on the device inside the
 * plan and are reused by every forward and backward call on the same layout (the paper
 * builds one plan per pool and reuses it across layers and for the backward pass,
 * Sections 4.1 and 4.3.3).  cu_seqlens_dev is read during the call only.
 * With opts->weight_model = LIBRA_WEIGHT_BLOCKS the weight is the block count described at
 * LIBRA_WEIGHT_BLOCKS above; everything else is unchanged.
 * Errors: INVALID_ARG (null, n_samples <= 0, n_heads <= 0, tile_q <= 0, a negative option,
 * an unknown weight model), OVERFLOW (n_heads * T^2 >= 9e15, the bound under which loads fit the
 * placement's packed keys, or NB * H >= 2^31), CUDA.  A malformed cu_seqlens is detected on the
 * device and reported by libra_plan_status as BAD_SEQLENS; the per-token sample bounds of such a
 * plan are clamped into [0, T], and the attention kernels given it do no work: they leave their
 * outputs untouched and report BAD_SEQLENS through libra_busy_times.
 */
int libra_plan_tiles(const int32_t* cu_seqlens_dev, int n_samples, int n_heads, int tile_q,
                     const libra_plan_opts* opts /* nullable */, void* stream,
                     libra_plan_t** plan_out);

/* Sizes of a plan direction (host values, no synchronisation). */
int libra_plan_info(const libra_plan_t* plan, int direction, int64_t* n_tiles, int* n_workers,
                    int64_t* n_blocks, int* tile, int* n_heads);

/* Synchronises `stream` of the plan's creation and returns the device status word:
 * LIBRA_OK, LIBRA_ERR_BAD_SEQLENS or LIBRA_ERR_TIMEOUT. */
int libra_plan_status(const libra_plan_t* plan);

/* Copies one direction of the plan to caller-allocated HOST arrays (any may be NULL):
 * weight int64[n_tiles], order int32[n_tiles], cta_of_tile int32[n_tiles],
 * cta_offsets int32[n_workers+1], cta_tiles int32[n_tiles], loads int64[n_workers].
 * Synchronises the plan's stream. */
int libra_plan_export(const libra_plan_t* plan, int direction, int64_t* weight_host,
                      int32_t* order_host, int32_t* cta_of_tile_host, int32_t* cta_offsets_host,
                      int32_t* cta_tiles_host, int64_t* loads_host);

/* Pair tiles (directions & LIBRA_DIR_PAIR; the units of the fused backward; no counterpart in the paper beyond
 * the tile idea itself).  The paper's tile is a query block with all of its keys (Section 4.3.1); a pair tile
 * cuts that rectangle along the key axis as well.  The score matrix is cut into tile_kv x tile_kv cells at
 * global positions; a cell is live when a query of its row block attends a key of its key block.  Pair-block
 * (c, j) is key block j against the row blocks of query chunk c (pair_chunk tokens), present when one of those
 * cells is live; pair-blocks are numbered chunk by chunk, key blocks ascending inside a chunk; tile id =
 * h * n_blocks + pair-block (head-major).  The weight is the time proxy of LIBRA_WEIGHT_BLOCKS: the live cells
 * of the pair-block.  Placement uses Algorithm 2's greedy rule (least-loaded worker, lowest index on ties) but
 * takes the tiles in id order instead of heaviest first: the plan then equals the schedule of a first-in-first-
 * out work queue, the workers stay on neighbouring tiles, and the rows of Q, dO and the dQ accumulator that
 * those tiles share stay in L2 between their uses; since no tile is large, the loads still end up within one
 * tile weight of each other.  libra_plan_info / libra_plan_export take LIBRA_DIR_PAIR (n_blocks = pair-blocks,
 * order = identity).  libra_plan_export_pairs copies the key block and the query chunk of every pair-block
 * (int32[n_blocks] each, HOST, nullable) and the chunk size in tokens (the planner doubles pair_chunk while
 * there are more than 262144 pair-blocks). */
int libra_plan_export_pairs(const libra_plan_t* plan, int32_t* key_block_host, int32_t* query_chunk_host,
                            int* chunk_tokens_host);

/* Frees the plan's device and host memory (synchronises the device first). NULL is OK. */
int libra_plan_destroy(libra_plan_t* plan);

/* ---- attention -----------------------------------------------------------------------
 * Forward (Section 2.2, Eq. 1 applied inside each sample under the block-diagonal causal
 * mask of Section 2.3):  for row i of a sample starting at s, with keys s..i,
 *     out_i = sum_k softmax_k(scale * <q_i, k_k>) v_k,   lse_i = ln sum_k exp(scale * <q_i, k_k>)
 * bf16 inputs, fp32 accumulation and softmax, bf16 out (round to nearest even), fp32 lse
 * (natural log).  One persistent kernel walks the plan's query-major tile lists.  head_dim 256 (the
 * micro-benchmark head shape of Table 1) runs a kernel of its own: one 128-row slot at a time against
 * 64-key blocks, the 256-column output accumulator taking half of the tensor memory.
 * Requires a plan with LIBRA_DIR_Q, tile_q == 256 and n_heads dividing hq.
 * Errors: INVALID_ARG, UNSUPPORTED, PLAN_MISMATCH (plan T != dims->total_tokens), CUDA.
 */
int libra_attn_pool_fwd(const void* q_dev, const void* k_dev, const void* v_dev,
                        const int32_t* cu_seqlens_dev, const libra_plan_t* plan,
                        void* out_dev, float* lse_dev, const libra_dims* dims, void* stream);

/* Bytes of caller-owned device scratch libra_attn_pool_bwd needs; 0 on bad arguments.  Two-kernel form: the row
 * statistics D and LSE in log2 units, padded to a multiple of 128 rows (2 * hq * round_up(T, 128) floats).
 * Fused form (see below): in addition the fp32 accumulators of dQ (T * hq * 128 floats) and of dK and dV
 * (T * hkv * 128 floats each). */
size_t libra_attn_pool_bwd_workspace_bytes(const libra_plan_t* plan, const libra_dims* dims);

/* Backward: the gradient of <dout, out> with respect to q, k, v, given out and lse from the
 * forward call (Section 4.3.3 states that the backward pass reuses the forward plan's
 * structure; the arithmetic is the derivative of Eq. 1):
 *     P_ik = exp(scale <q_i,k_k> - lse_i), D_i = <dout_i, out_i>, dS_ik = P_ik (<dout_i,v_k> - D_i)
 *     dq_i = scale sum_k dS_ik k_k;  dk_k = scale sum_{h,i} dS_ik q_i;  dv_k = sum_{h,i} P_ik dout_i
 * (sums over the query heads h of the kv head's group and the rows i >= k of the sample).
 * The plan decides between two forms of the same computation.
 *   Two-kernel form (plan without pair tiles, or head_dim other than 128): three launches: row statistics, a dK/dV kernel
 *   that walks the plan's key-major lists, and a dQ kernel that walks its query-major lists (S and dP are computed
 *   by both, seven GEMMs per 128 x 128 cell); no atomics, so results are run-to-run identical.  Needs LIBRA_DIR_KV
 *   with tile_kv == 128 and n_heads_kv == hkv, and LIBRA_DIR_Q with tile_q == 256 and n_heads dividing hq.
 *   Fused form (plan with LIBRA_DIR_PAIR, tile_kv == 128, n_heads_kv == hkv, and head_dim 128): row statistics, one
 *   kernel that walks the pair-tile lists and computes S, dP, dV, dK and dQ of a cell together (five GEMMs per
 *   cell), and a conversion pass.  dK and dV of a pair tile accumulate on chip and are added to fp32 accumulators
 *   in the workspace when the tile ends; dQ of every cell is added to its fp32 accumulator; all by bulk reduce-adds.
 *   The accumulators are rounded to bf16 once, at the end, so the result is at least as accurate as the two-kernel
 *   form's, but the order of the floating-point additions varies from run to run: results agree to rounding, not
 *   bit for bit.  The other directions of the plan are not used by this form.
 *   At head_dim 256 the two-kernel form takes three passes of one kernel after the row statistics (dV and dK
 *   over the key-major lists, dQ over the query-major lists; S is recomputed by each: eight GEMMs per cell), because
 *   the accumulators of dK and dV together would fill the tensor memory.  Same plan, results and determinism.  With a
 *   pair-tile plan the dV and dK passes walk the pair tiles instead and add their partial sums to fp32 accumulators
 *   in the workspace (T * hkv * 256 floats each), rounded once at the end; like the fused form, those results agree
 *   to rounding from run to run, not bit for bit.
 * `workspace_dev` must hold libra_attn_pool_bwd_workspace_bytes bytes, 256-byte aligned; every byte the call reads
 * is written (or cleared) inside the call.  Errors: INVALID_ARG, UNSUPPORTED, PLAN_MISMATCH, CUDA.
 */
int libra_attn_pool_bwd(const void* q_dev, const void* k_dev, const void* v_dev,
                        const void* out_dev, const float* lse_dev, const void* dout_dev,
                        const int32_t* cu_seqlens_dev, const libra_plan_t* plan,
                        void* dq_dev, void* dk_dev, void* dv_dev, void* workspace_dev,
                        const libra_dims* dims, void* stream);

/* Backward without any allocation (no counterpart in the paper: this is a deployment aid).
 * Same computation, arguments and results as libra_attn_pool_bwd, but the caller passes no
 * workspace: the row-statistics scratch is a fixed 16 MiB array inside the library's device
 * image (libra_attn_pool_bwd_noalloc_max_bytes reports its size).  It is meant for callers that
 * cannot obtain device memory when they need the backward pass, for example while a stream is
 * being captured, inside an allocator callback, or in a process that fixes its device memory at
 * start-up.  The call performs no cudaMalloc / cudaFree and calls no allocating routine.
 *   - Limit: libra_attn_pool_bwd_workspace_bytes(plan, dims) must not exceed the built-in size
 *     (2 * hq * round_up(T, 128) floats <= 4 Mi floats); otherwise nothing is launched and
 *     LIBRA_ERR_SCRATCH_TOO_SMALL is returned.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents; the
 *     call overwrites every element it later reads, so nothing needs clearing.  Two calls whose
 *     GPU work overlaps (different streams, no dependency) race on it: serialise them.
 *   - Every GPU that loads the library holds the 16 MiB until the process exits.
 */
size_t libra_attn_pool_bwd_noalloc_max_bytes(void);
int libra_attn_pool_bwd_noalloc(const void* q_dev, const void* k_dev, const void* v_dev,
                                const void* out_dev, const float* lse_dev, const void* dout_dev,
                                const int32_t* cu_seqlens_dev, const libra_plan_t* plan,
                                void* dq_dev, void* dk_dev, void* dv_dev,
                                const libra_dims* dims, void* stream);

/* ---- Variance-Reduced Sequence Placement (Section 4.2, Algorithm 1) ----------------------
 * Groups the D packed sequences of one optimizer-step window into K = D / P pools of exactly P
 * sequences with even summed attention work.  The paper runs it on a CPU core in the data path;
 * these two calls run it in device kernels on `stream` (no allocation, no synchronisation).
 *
 * libra_vrsp_work: work_dev[i] = F_i = sum over the raw samples j of packed sequence i of
 *   len_ij^2 (Eq. 4).  sample_offsets_dev: int32[n_samples_total + 1], the sample start offsets of
 *   all sequences laid end to end (non-decreasing; only differences are used);
 *   seq_first_sample_dev: int32[D + 1], index of each sequence's first sample.
 * libra_vrsp_place: sequences in the order (F descending, index ascending) go one by one to the
 *   pool with the smallest load among those holding fewer than P sequences (lowest pool index on
 *   ties).  Outputs (device): order_dev int32[D], the reordered list S' as input indices, pools
 *   laid end to end in pool order, a pool's sequences in the order they were appended (pool k of
 *   the window is GA index k / (DP/P), pool k % (DP/P) of that index: GA-major, pool-minor);
 *   pool_of_seq_dev int32[D]; pool_load_dev int64[K].  scratch_dev: int32[D], overwritten.
 * Errors: INVALID_ARG (null, D <= 0, P <= 0, P does not divide D), UNSUPPORTED (K > 1024 or
 * D > 2^20), CUDA. */
int libra_vrsp_work(const int32_t* sample_offsets_dev, const int32_t* seq_first_sample_dev, int n_sequences,
                    int64_t* work_dev, void* stream);
int libra_vrsp_place(const int64_t* work_dev, int n_sequences, int pool_size, int32_t* order_dev,
                     int32_t* pool_of_seq_dev, int64_t* pool_load_dev, int32_t* scratch_dev, void* stream);

/* ---- Tiled Attention Pooling across workers (Section 4.3: Eq. 5-8, Algorithm 2, exchange plan) ----
 * Plans one sequence pool: P packed sequences, each held by its own group of CP workers, W = P * CP
 * workers in all.  Everything runs in device kernels on `stream`; the paper runs it on CPU cores.
 * libra_tap_plan places the tiles and sums the exchange volumes; libra_tap_schedule lists the transfers.
 * Executing them (peer copies into local memory, then the attention kernels per head chunk) is host code
 * above this library.
 *
 * Layout (a reading; the paper does not fix how a sequence is split over its CP group): sequence s
 * is tokens [seq_offsets[s], seq_offsets[s+1]) of the pool's sample list (a sequence boundary is
 * a sample boundary); worker s*CP + c holds the c-th run of ceil(L_s / CP) consecutive tokens.
 *   tiles   : every sequence is cut at multiples of `block` tokens from its own start; blocks are
 *             numbered sequence by sequence; tile id = block * n_shards + h            (Eq. 5)
 *   f       : causal pairs of the block                                               (Eq. 6)
 *   q(t)    : the worker holding the block's first token;
 *             V_Q = V_O = tokens * (hq / n_shards) * head_dim * 2 bytes
 *   K(t)    : the samples with a token in the block, on shard h                         (Eq. 7)
 *   V_g     : 2 * len * kv_heads_per_shard * head_dim * 2 bytes, kv_heads_per_shard = hkv / n_shards,
 *             or 1 when n_shards > hkv (shards then share a replicated kv head)
 *   C_r     : starts as the groups worker r holds in full (resident groups need no transfer)
 *   placement: Algorithm 2 with tau = tau_num / tau_den; "L_r + f <= C" is evaluated exactly as
 *             tau_den * W * (L_r + f) <= (tau_den + tau_num) * sum(f)
 * Outputs (device): sigma_dev int32[NT] destination worker of every tile; loads_dev int64[W];
 * fwd_bytes_dev / bwd_bytes_dev int64[W * W], bytes worker src sends to worker dst ([src * W + dst]) in
 * the forward / backward pass: each KV group selected for a destination and not resident there is
 * fetched once per destination, run by run from the workers that hold it (runs already there do
 * not move), a tile away from its Q-home has Q sent out and the output sent back; backward: dO along
 * the Q path, dQ along the output path, dK/dV back along the KV paths.  comm_total_dev int64[1]: the
 * summed Delta_comm (Eq. 8) of the choices taken.  status_dev int[1]: 0 or LIBRA_ERR_OVERFLOW.
 * seq_offsets_host is a HOST array of n_sequences + 1 entries (read before the call returns).
 * Scratch comes from the stream-ordered allocator and is released on `stream`.
 * When status_dev reports OVERFLOW (the integer soft-cap test could exceed 64 bits) sigma_dev holds
 * every tile's Q-home and the byte matrices are zero.
 * Errors: INVALID_ARG, UNSUPPORTED (W > 1024, more than 65536 blocks), OVERFLOW (the pool's work total
 * n_shards * T (T + 1) / 2 does not fit 64 bits), CUDA. */
typedef struct {
    int cp;                 /* workers per packed sequence */
    int block;              /* B, tokens per block */
    int n_shards;           /* H head shards; divides hq; divides or is a multiple of hkv */
    int hq, hkv, head_dim;
    int tau_num, tau_den;   /* soft cap slack, the paper uses 3 / 100 */
} libra_tap_opts;
int64_t libra_tap_num_tiles(const int32_t* seq_offsets_host, int n_sequences, int block, int n_shards);
int libra_tap_plan(const int32_t* cu_seqlens_dev, int n_samples, const int32_t* seq_offsets_host,
                   int n_sequences, const libra_tap_opts* opts, int32_t* sigma_dev, int64_t* loads_dev,
                   int64_t* fwd_bytes_dev, int64_t* bwd_bytes_dev, int64_t* comm_total_dev,
                   int* status_dev, void* stream);

/* Exchange schedule of an assignment (Section 4.3.3; the head pieces of Section 4.4 follow from it).
 * Turns sigma (as written by libra_tap_plan, or any assignment of the pool's tiles to its workers) into
 * transfer records of six int32 each, (kind, src, dst, tok0, ntok, shard), in device memory:
 *   kind 0 : a tile placed away from its Q-home.  Forward: the Q rows [tok0, tok0 + ntok) of head shard `shard`
 *            go src -> dst and the output rows come back dst -> src.  Backward: dO goes src -> dst, dQ comes
 *            back dst -> src.  (The rows are taken to live at the Q-home, the worker holding the block's first
 *            token; that is the case whenever the run length ceil(L / CP) is a multiple of B.)
 *   kind 1 : a KV group (sample, shard) some tile placed at dst refers to, not wholly resident there: one record
 *            per token run of the sample held by another worker.  Forward: K and V of the run go src -> dst,
 *            once per destination however many tiles use the group.  Backward: the dK / dV partial sums of the
 *            run go dst -> src and are added there.
 * Order: kind 0 records by tile id, then kind 1 records by (dst, sample, shard, src).
 * The Pipeliner moves every record in M equal head pieces (M divides hq / n_shards): chunk m carries the m-th
 * piece of the shard's query heads of every kind 0 record and, of every kind 1 record, the kv heads that this
 * piece is the first to read (query head q reads kv head q / (hq / hkv)); so one list serves all chunks and
 * both passes.
 * records_dev: int32[capacity * 6]; *n_records_dev receives the number of records the assignment implies
 * (records beyond `capacity` are not written).  Scratch comes from the stream-ordered allocator.
 * Errors: INVALID_ARG, UNSUPPORTED (W > 1024, n_samples * n_shards * W >= 2^31), CUDA. */
int libra_tap_schedule(const int32_t* cu_seqlens_dev, int n_samples, const int32_t* seq_offsets_host,
                       int n_sequences, const libra_tap_opts* opts, const int32_t* sigma_dev,
                       int32_t* records_dev, int64_t capacity, int64_t* n_records_dev, void* stream);

/* ---- instrumentation -------------------------------------------------------------------
 * Per-CTA busy time of the most recent launch of kernel `which` (LIBRA_KERNEL_*) that used this
 * plan: nanoseconds between the CTA starting and finishing its tile list, read with the GPU's
 * global timer.  Copies n_workers values to ns_host and synchronises the device.  Returns the
 * status of the most recent forward (LIBRA_KERNEL_FWD) or backward (the other two) launch:
 * LIBRA_OK, LIBRA_ERR_TIMEOUT if a bounded wait gave up, LIBRA_ERR_BAD_SEQLENS if the plan's
 * cu_seqlens was malformed and the kernels therefore did no work. */
int libra_busy_times(const libra_plan_t* plan, int which, uint64_t* ns_host);

/* Time each tile took in the most recent launch of the forward kernel (which = LIBRA_KERNEL_FWD, tiles of the
 * query-major direction) or of the fused backward kernel (LIBRA_KERNEL_BWD_FUSED, pair tiles): nanoseconds of the
 * global timer from the moment a compute thread of the CTA turns to the tile until it has finished the tile's
 * last output, indexed by tile id; 0 for a tile that was not run.  With the plan's weights (libra_plan_export)
 * this shows how well the tile weight predicts time: the paper notes that a FLOPs-balanced assignment need not
 * be time-balanced (Section 3.2).  Copies n_tiles values to ns_host (HOST) and synchronises the device.
 * Errors: INVALID_ARG (another kernel id), PLAN_MISMATCH (the plan lacks the direction), CUDA. */
int libra_tile_times(const libra_plan_t* plan, int which, uint32_t* ns_host);

/* Budget of one device-side wait of the attention kernels launched with this plan, in nanoseconds
 * (0 restores the default of 2 s, the maximum is 4 s).  Every wait on a barrier inside the kernels
 * is bounded: a wait that outlives the budget makes its CTA stop issuing work, let the copies and
 * MMAs it has in flight finish, free its tensor memory and return, and the launch reports
 * LIBRA_ERR_TIMEOUT through libra_busy_times.  A healthy run never comes near the default. */
int libra_plan_set_wait_limit_ns(libra_plan_t* plan, uint64_t ns);

/* Test aid (no counterpart in the paper): while enabled, the producer role of the attention kernels launched
 * with this plan issues no loads at all, so every consumer's first wait runs out of its budget on an
 * otherwise healthy GPU.  This is how the give-up path is exercised without a fault or an endless loop: set a
 * short budget with libra_plan_set_wait_limit_ns, launch, and libra_busy_times reports LIBRA_ERR_TIMEOUT; the
 * outputs of such a launch are undefined.  Off by default. */
int libra_plan_inject_stall(libra_plan_t* plan, int enabled);

/* Self-test of the bounded wait: launches one small CTA that waits, through the same routine as every
 * barrier wait of the attention kernels, on a barrier nothing ever arrives on, with a budget of limit_ns
 * (1 ns .. 0.1 s) and nothing else in flight.  *status_host receives LIBRA_ERR_TIMEOUT when the wait gave up
 * as designed (LIBRA_OK would mean it claimed completion), *waited_ns_host (nullable) how long it waited.
 * Synchronous; allocates and frees 8 bytes of device memory.  Errors: INVALID_ARG, CUDA. */
int libra_selftest_wait_timeout(uint32_t limit_ns, int* status_host, int* waited_ns_host);

/* Kernel timing: when enabled, every forward / backward call records CUDA events on its stream
 * around each of its kernels (LIBRA_KERNEL_*), keeping the 64 most recent launches of each;
 * enabling it again starts a fresh record.  libra_kernel_time_ms synchronises on the closing event
 * of the most recent launch of kernel `which` and returns its duration in milliseconds;
 * libra_kernel_times_ms returns the durations of up to `capacity` most recent recorded launches,
 * oldest first, and their number in *n_out.  Off by default.
 * Errors: INVALID_ARG, PLAN_MISMATCH (nothing recorded yet), CUDA. */
int libra_plan_set_timing(libra_plan_t* plan, int enabled);
int libra_kernel_time_ms(const libra_plan_t* plan, int which, float* ms_host);
int libra_kernel_times_ms(const libra_plan_t* plan, int which, float* ms_host, int capacity, int* n_out);

/* Number of kernels this library has launched in the calling process (for accounting). */
int64_t libra_launch_count(void);

const char* libra_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LIBRA_H_ */
