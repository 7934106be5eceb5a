/* CPU oracle for pool attention and for the SH-Tile plan.
 *
 * TEST INFRASTRUCTURE ONLY: a plain, slow, obviously correct restatement of the
 * definitions, used by the tests, the smoke check and the benchmark's CPU-baseline
 * leg.  The CUDA library never calls it and shares no code with it.
 *
 * Attention: see oracle_attn.inc (instantiated for float and double).
 * Plan: oracle_plan() below, following the paper's SH-Tile construction (Section
 * 4.3.1, Eq. 5), tile weight (Eq. 6) and heaviest-first placement (Algorithm 2) with
 * no communication term, step by step.
 *
 * Build: gcc -O3 -march=native -fopenmp -shared -fPIC oracle.c -o liboracle.so -lm
 * (no -ffast-math).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define CAT_(a, b) a##b
#define CAT(a, b) CAT_(a, b)

#define REAL float
#define REAL_EXP expf
#define REAL_LOG logf
#define FN(name) CAT(name, _f32)
#include "oracle_attn.inc"
#undef REAL
#undef REAL_EXP
#undef REAL_LOG
#undef FN

#define REAL double
#define REAL_EXP exp
#define REAL_LOG log
#define FN(name) CAT(name, _f64)
#include "oracle_attn.inc"
#undef REAL
#undef REAL_EXP
#undef REAL_LOG
#undef FN

/* ------------------------------------------------------------------------------------
 * Plan.
 *
 * Step 1 (Eq. 5): the pool's token axis [0, T) is cut at multiples of `tile` into
 *   NB = ceil(T / tile) blocks (the last may be short; no cut at sample boundaries);
 *   the heads are split in H shards; tile id t = b * H + h.
 * Step 2 (Eq. 6): weight of block b = number of causal (query, key) pairs it covers.
 *   Query-major (direction 0): block b holds queries; a query at sample-local position
 *   p attends p + 1 keys, so for every sample j the block intersects, with local range
 *   [a, e):  sum_{p=a}^{e-1} (p + 1).
 *   Key-major (direction 1): block b holds keys; a key at local position p of a sample
 *   of length len is attended by len - p queries:  sum_{p=a}^{e-1} (len - p).
 *   The sums are written out as loops (the closed forms are what the tests pin them to).
 *   All H shards of a block weigh the same (the common factor Hq/H is dropped).
 * Step 3 (Algorithm 2, ordering): tiles sorted by decreasing weight, then tile id.
 * Step 4 (Algorithm 2, placement with Delta_comm = 0): each tile in that order goes to
 *   the worker with the smallest load, lowest index on ties; its load grows by the weight.
 *   With no communication term both branches of the algorithm's choice reduce to this
 *   rule and the soft cap drops out.
 * Step 5: per-worker tile lists in assignment order, as CSR.
 * ------------------------------------------------------------------------------------ */

typedef struct { int64_t w; int32_t id; } tile_key;

static int cmp_tiles(const void* a, const void* b) {
    const tile_key* x = (const tile_key*)a;
    const tile_key* y = (const tile_key*)b;
    if (x->w != y->w) return x->w > y->w ? -1 : 1;
    return x->id < y->id ? -1 : (x->id > y->id ? 1 : 0);
}

/* Steps 3-5, common to both weight models: order, place, list. */
static int place_tiles(int64_t NT, int W, const int64_t* weight, int32_t* order, int32_t* cta_of_tile,
                       int32_t* cta_offsets, int32_t* cta_tiles, int64_t* loads) {
    if (W <= 0 || NT < 0) return -1;
    /* step 3 */
    tile_key* keys = (tile_key*)malloc(sizeof(tile_key) * (size_t)NT);
    if (!keys) return -2;
    for (int64_t t = 0; t < NT; ++t) { keys[t].w = weight[t]; keys[t].id = (int32_t)t; }
    qsort(keys, (size_t)NT, sizeof(tile_key), cmp_tiles);
    for (int64_t t = 0; t < NT; ++t) order[t] = keys[t].id;
    free(keys);

    /* step 4 */
    for (int r = 0; r < W; ++r) loads[r] = 0;
    for (int64_t x = 0; x < NT; ++x) {
        const int32_t t = order[x];
        int best = 0;
        for (int r = 1; r < W; ++r) if (loads[r] < loads[best]) best = r;
        cta_of_tile[t] = best;
        loads[best] += weight[t];
    }

    /* step 5 */
    for (int r = 0; r <= W; ++r) cta_offsets[r] = 0;
    for (int64_t t = 0; t < NT; ++t) cta_offsets[cta_of_tile[t] + 1] += 1;
    for (int r = 0; r < W; ++r) cta_offsets[r + 1] += cta_offsets[r];
    int32_t* fill = (int32_t*)calloc((size_t)W, sizeof(int32_t));
    if (!fill) return -2;
    for (int64_t x = 0; x < NT; ++x) {
        const int32_t t = order[x];
        const int r = cta_of_tile[t];
        cta_tiles[cta_offsets[r] + fill[r]++] = t;
    }
    free(fill);
    return 0;
}

int64_t oracle_plan_num_blocks(const int32_t* cu, int n, int tile) {
    if (!cu || n <= 0 || tile <= 0) return -1;
    const int64_t T = cu[n];
    return (T + tile - 1) / tile;
}

int oracle_plan(const int32_t* cu, int n, int H, int tile, int W, int direction,
                int64_t* weight /*[NB*H]*/, int32_t* order /*[NB*H]*/, int32_t* cta_of_tile /*[NB*H]*/,
                int32_t* cta_offsets /*[W+1]*/, int32_t* cta_tiles /*[NB*H]*/, int64_t* loads /*[W]*/) {
    if (!cu || n <= 0 || H <= 0 || tile <= 0 || W <= 0) return -1;
    if (cu[0] != 0) return -1;
    for (int j = 0; j < n; ++j) if (cu[j + 1] < cu[j]) return -1;
    const int64_t T = cu[n];
    const int64_t NB = (T + tile - 1) / tile;
    const int64_t NT = NB * H;

    /* steps 1-2 */
    for (int64_t b = 0; b < NB; ++b) {
        const int64_t q0 = b * tile, q1 = (b + 1) * tile < T ? (b + 1) * tile : T;
        int64_t w = 0;
        for (int j = 0; j < n; ++j) {
            const int64_t s = cu[j], t = cu[j + 1], len = t - s;
            const int64_t lo = q0 > s ? q0 : s, hi = q1 < t ? q1 : t;
            for (int64_t g = lo; g < hi; ++g) {
                const int64_t p = g - s;
                w += direction == 0 ? (p + 1) : (len - p);
            }
        }
        for (int h = 0; h < H; ++h) weight[b * H + h] = w;
    }

    return place_tiles(NT, W, weight, order, cta_of_tile, cta_offsets, cta_tiles, loads);
}

/* ------------------------------------------------------------------------------------
 * Plan over pair tiles (the fused backward's work units).  The paper's tile is a query block with all of its
 * keys (Section 4.3.1); a pair tile cuts that rectangle along the key axis too.  Not in the paper: the weight
 * is the time proxy of oracle_plan_blocks (cells of the score matrix that hold a visible pair), and the tiles
 * are placed in tile-id order instead of heaviest first, by the same greedy rule (least-loaded worker, lowest
 * index on ties).  Placing in id order makes the static plan the schedule a first-in-first-out work queue
 * would give, so the workers stay on neighbouring tiles, which share their query-side tensors.
 *
 * Cells: the score matrix cut into `tile` x `tile` cells at global positions; cell (i, j) is live if some
 * query of row block i attends some key of key block j (same sample, query not before the key).
 * Pair-block (c, j): key block j against query chunk c (`chunk` tokens, a multiple of `tile`), present when
 * one of the chunk's row blocks has a live cell with j.  Pair-blocks are numbered chunk by chunk, key blocks
 * ascending inside a chunk; tile id = h * NU + u (head-major); weight = live cells of the pair-block.
 * ------------------------------------------------------------------------------------ */
static int pair_cells(const int32_t* cu, int n, int tile, uint8_t** live_out, int64_t* nb_out) {
    const int64_t T = cu[n];
    const int64_t NB = (T + tile - 1) / tile;
    uint8_t* live = (uint8_t*)calloc((size_t)(NB * NB), 1);          /* [row block][key block] */
    if (!live) return -2;
    for (int j = 0; j < n; ++j)
        for (int64_t k = cu[j]; k < cu[j + 1]; ++k)                   /* key k is attended by queries k .. end - 1 */
            for (int64_t i = k / tile; i <= (cu[j + 1] - 1) / tile; ++i) live[i * NB + k / tile] = 1;
    *live_out = live;
    *nb_out = NB;
    return 0;
}

int64_t oracle_plan_pairs_num_blocks(const int32_t* cu, int n, int tile, int chunk) {
    if (!cu || n <= 0 || tile <= 0 || chunk <= 0 || chunk % tile) return -1;
    uint8_t* live; int64_t NB;
    if (pair_cells(cu, n, tile, &live, &NB)) return -2;
    const int64_t R = chunk / tile;
    int64_t nu = 0;
    for (int64_t c = 0; c * R < NB; ++c)
        for (int64_t j = 0; j < NB; ++j) {
            int any = 0;
            for (int64_t i = c * R; i < (c + 1) * R && i < NB; ++i) any |= live[i * NB + j];
            nu += any;
        }
    free(live);
    return nu;
}

int oracle_plan_pairs(const int32_t* cu, int n, int H, int tile, int chunk, int W, int64_t* weight /*[NU*H]*/,
                      int32_t* order, int32_t* cta_of_tile, int32_t* cta_offsets, int32_t* cta_tiles, int64_t* loads,
                      int32_t* key_block /*[NU]*/, int32_t* query_chunk /*[NU]*/) {
    if (!cu || n <= 0 || H <= 0 || tile <= 0 || chunk <= 0 || chunk % tile || W <= 0) return -1;
    if (cu[0] != 0) return -1;
    for (int j = 0; j < n; ++j) if (cu[j + 1] < cu[j]) return -1;
    uint8_t* live; int64_t NB;
    if (pair_cells(cu, n, tile, &live, &NB)) return -2;
    const int64_t R = chunk / tile;
    int64_t nu = 0;
    for (int64_t c = 0; c * R < NB; ++c)
        for (int64_t j = 0; j < NB; ++j) {
            int64_t cells = 0;
            for (int64_t i = c * R; i < (c + 1) * R && i < NB; ++i) cells += live[i * NB + j];
            if (!cells) continue;
            key_block[nu] = (int32_t)j;
            query_chunk[nu] = (int32_t)c;
            weight[nu] = cells;                                        /* head 0 for now, copied below */
            ++nu;
        }
    free(live);
    const int64_t NT = nu * H;
    for (int h = H - 1; h >= 0; --h)
        for (int64_t u = nu - 1; u >= 0; --u) weight[(int64_t)h * nu + u] = weight[u];
    /* placement in tile-id order: each tile to the least-loaded worker, lowest index on ties */
    for (int r = 0; r < W; ++r) loads[r] = 0;
    for (int r = 0; r <= W; ++r) cta_offsets[r] = 0;
    for (int64_t t = 0; t < NT; ++t) {
        int best = 0;
        for (int r = 1; r < W; ++r) if (loads[r] < loads[best]) best = r;
        order[t] = (int32_t)t;
        cta_of_tile[t] = best;
        loads[best] += weight[t];
        cta_offsets[best + 1] += 1;
    }
    for (int r = 0; r < W; ++r) cta_offsets[r + 1] += cta_offsets[r];
    int32_t* fill = (int32_t*)calloc((size_t)W, sizeof(int32_t));
    if (!fill) return -2;
    for (int64_t t = 0; t < NT; ++t) { const int r = cta_of_tile[t]; cta_tiles[cta_offsets[r] + fill[r]++] = (int32_t)t; }
    free(fill);
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Plan with the block-count weight (not in the paper; Section 3.2 only remarks that equal
 * FLOPs need not mean equal time).  A kernel spends the same time on a g x g block of the
 * score matrix whether one pair of it is visible or all, so this weight counts blocks.
 *
 * The token axis is cut into chunks at multiples of g.  A tile (block b of `tile` tokens,
 * any head shard) is the union of the chunk pieces it intersects.  For each piece:
 *   query-major: the piece holds query rows r0..r1.  The sample of r0 starts at s0.  Row r0
 *     attends keys s0..r0, rows after it attend keys no earlier than s0 and no later than
 *     r1, so the key chunks with a visible pair are floor(s0/g) .. floor(r1/g).
 *   key-major: the piece holds keys c0..c1.  The sample of c1 ends at e1 (exclusive).  Key
 *     c1 is attended by queries c1..e1-1, earlier keys of the piece by queries no earlier
 *     than c0 and no later than e1-1, so the query chunks are floor(c0/g) .. floor((e1-1)/g).
 * Weight of the tile = sum over its pieces of (8 * chunks + unit_cost).
 * Steps 3-5 are those of oracle_plan.
 * ------------------------------------------------------------------------------------ */
int oracle_plan_blocks(const int32_t* cu, int n, int H, int tile, int W, int direction, int g, int unit_cost,
                       int64_t* weight, int32_t* order, int32_t* cta_of_tile, int32_t* cta_offsets,
                       int32_t* cta_tiles, int64_t* loads) {
    if (!cu || n <= 0 || H <= 0 || tile <= 0 || W <= 0 || g <= 0 || unit_cost < 0) return -1;
    if (cu[0] != 0) return -1;
    for (int j = 0; j < n; ++j) if (cu[j + 1] < cu[j]) return -1;
    const int64_t T = cu[n];
    const int64_t NB = (T + tile - 1) / tile;
    const int64_t NT = NB * H;
    for (int64_t b = 0; b < NB; ++b) {
        const int64_t t0 = b * tile, t1 = (b + 1) * tile < T ? (b + 1) * tile : T;
        int64_t w = 0;
        int64_t first = t0;
        while (first < t1) {
            int64_t end = (first / g + 1) * g;  /* the piece ends at the next multiple of g or at the tile end */
            if (end > t1) end = t1;
            const int64_t last = end - 1;
            int64_t chunks;
            if (direction == 0) {
                int j = 0;
                while (!(cu[j] <= first && first < cu[j + 1])) ++j;  /* sample of the first row */
                chunks = last / g - cu[j] / g + 1;
            } else {
                int j = 0;
                while (!(cu[j] <= last && last < cu[j + 1])) ++j;    /* sample of the last key */
                chunks = (cu[j + 1] - 1) / g - first / g + 1;
            }
            w += 8 * chunks + unit_cost;
            first = end;
        }
        for (int h = 0; h < H; ++h) weight[b * H + h] = w;
    }
    return place_tiles(NT, W, weight, order, cta_of_tile, cta_offsets, cta_tiles, loads);
}

/* ------------------------------------------------------------------------------------
 * Variance-Reduced Sequence Placement (Section 4.2, Algorithm 1), in the algorithm's order:
 *   work      F_i = sum_j len_ij^2 over the raw samples of packed sequence i      (Eq. 4)
 *   pools     K = D / P, all empty
 *   order     sequences by decreasing F, then increasing index
 *   heap      min-heap of (load_k, k) over the pools that are not full
 *   loop      pop the minimum, append the sequence to that pool, add F to its load, push the
 *             pool back if it still holds fewer than P sequences
 *   output    the pools laid end to end in pool order (GA-major, pool-minor numbering of pools)
 * The heap is a plain array-based binary heap ordered lexicographically on (load, k).
 * ------------------------------------------------------------------------------------ */
int oracle_vrsp_work(const int32_t* sample_offsets, const int32_t* seq_first_sample, int D, int64_t* work) {
    if (!sample_offsets || !seq_first_sample || !work || D <= 0) return -1;
    for (int i = 0; i < D; ++i) {
        int64_t f = 0;
        for (int j = seq_first_sample[i]; j < seq_first_sample[i + 1]; ++j) {
            const int64_t len = (int64_t)sample_offsets[j + 1] - sample_offsets[j];
            f += len * len;
        }
        work[i] = f;
    }
    return 0;
}

typedef struct { int64_t load; int32_t k; } pool_key;

static int pool_less(pool_key a, pool_key b) { return a.load < b.load || (a.load == b.load && a.k < b.k); }

static void heap_push(pool_key* h, int* n, pool_key x) {
    int i = (*n)++;
    h[i] = x;
    while (i > 0 && pool_less(h[i], h[(i - 1) / 2])) {
        pool_key t = h[i]; h[i] = h[(i - 1) / 2]; h[(i - 1) / 2] = t;
        i = (i - 1) / 2;
    }
}

static pool_key heap_pop(pool_key* h, int* n) {
    pool_key top = h[0];
    h[0] = h[--(*n)];
    int i = 0;
    for (;;) {
        int l = 2 * i + 1, r = l + 1, m = i;
        if (l < *n && pool_less(h[l], h[m])) m = l;
        if (r < *n && pool_less(h[r], h[m])) m = r;
        if (m == i) break;
        pool_key t = h[i]; h[i] = h[m]; h[m] = t;
        i = m;
    }
    return top;
}

int oracle_vrsp_place(const int64_t* work, int D, int P, int32_t* order /*[D]*/, int32_t* pool_of_seq /*[D]*/,
                      int64_t* pool_load /*[D/P]*/) {
    if (!work || !order || !pool_of_seq || !pool_load || D <= 0 || P <= 0 || D % P != 0) return -1;
    const int K = D / P;
    tile_key* keys = (tile_key*)malloc(sizeof(tile_key) * (size_t)D);
    pool_key* heap = (pool_key*)malloc(sizeof(pool_key) * (size_t)K);
    int32_t* fill = (int32_t*)calloc((size_t)K, sizeof(int32_t));
    if (!keys || !heap || !fill) { free(keys); free(heap); free(fill); return -2; }
    for (int i = 0; i < D; ++i) { keys[i].w = work[i]; keys[i].id = i; }
    qsort(keys, (size_t)D, sizeof(tile_key), cmp_tiles);  /* decreasing F, then increasing index */
    int n = 0;
    for (int k = 0; k < K; ++k) { pool_load[k] = 0; pool_key x = {0, k}; heap_push(heap, &n, x); }
    for (int x = 0; x < D; ++x) {
        const int32_t i = keys[x].id;
        pool_key top = heap_pop(heap, &n);
        const int k = top.k;
        order[(int64_t)k * P + fill[k]] = i;
        fill[k] += 1;
        pool_of_seq[i] = k;
        pool_load[k] += work[i];
        if (fill[k] < P) { pool_key back = {pool_load[k], k}; heap_push(heap, &n, back); }
    }
    free(keys); free(heap); free(fill);
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Communication-aware SH-Tile placement (Section 4.3.2, Algorithm 2, Eq. 8) in the
 * algorithm's order and notation.
 *   tiles t with estimated work f_t, Q-home q(t), Q + output volume V_Q(t) + V_O(t) and the set
 *   K(t) of KV groups they reference (CSR lists); KV groups g with volume V_g; workers r with load
 *   L_r and the set C_r of KV groups already selected for them.
 *   C       = (1 + tau) * sum(f) / |W|.  tau = tau_num / tau_den, and "L_r + f_t <= C" is tested in
 *             integers as  tau_den * |W| * (L_r + f_t) <= (tau_den + tau_num) * sum(f).
 *   order   = tiles by decreasing f, then tile id.
 *   Delta_comm(t, r) = sum of V_g over g in K(t) \ C_r, plus V_Q(t) + V_O(t) if r != q(t).
 *   F       = workers with L_r + f_t <= C; if F is not empty the tile goes to
 *             argmin over F of (Delta_comm, L_r, r), else to argmin over W of (L_r, Delta_comm, r).
 *   then    L_r* += f_t and C_r* gains K(t).
 * C_r starts as the groups worker r already holds in full (resident[g] == r): the paper charges no
 * transfer for resident groups (Section 4.3.3) and does not say how C_r is initialised.
 * Outputs: sigma, L, the final C (W x NG bytes, 1 = selected or resident) and the summed
 * Delta_comm of the choices taken.
 * ------------------------------------------------------------------------------------ */
int oracle_tap_place(int64_t NT, int W, int64_t NG, const int64_t* f, const int32_t* q_home, const int64_t* v_qo,
                     const int32_t* kv_off, const int32_t* kv_grp, const int64_t* v_g, const int32_t* resident,
                     int tau_num, int tau_den, int32_t* sigma, int64_t* L, uint8_t* C, int64_t* comm_total) {
    if (NT < 0 || W <= 0 || NG < 0 || tau_num < 0 || tau_den <= 0) return -1;
    int64_t sum_f = 0;
    for (int64_t t = 0; t < NT; ++t) { if (f[t] < 0) return -1; sum_f += f[t]; }
    if (sum_f > (INT64_MAX / ((int64_t)(tau_den + tau_num) * 2)) / W) return -3;  /* the integer test would overflow */
    tile_key* keys = (tile_key*)malloc(sizeof(tile_key) * (size_t)(NT ? NT : 1));
    if (!keys) return -2;
    for (int64_t t = 0; t < NT; ++t) { keys[t].w = f[t]; keys[t].id = (int32_t)t; }
    qsort(keys, (size_t)NT, sizeof(tile_key), cmp_tiles);
    for (int r = 0; r < W; ++r) L[r] = 0;
    for (int r = 0; r < W; ++r)
        for (int64_t g = 0; g < NG; ++g) C[(int64_t)r * NG + g] = resident[g] == r ? 1 : 0;
    *comm_total = 0;
    for (int64_t x = 0; x < NT; ++x) {
        const int32_t t = keys[x].id;
        int best = -1;
        int64_t best_d = 0;
        int have_feasible = 0;
        for (int pass = 0; pass < 2 && best < 0; ++pass) {   /* pass 0: over F; pass 1: over W when F is empty */
            for (int r = 0; r < W; ++r) {
                const int feasible = (int64_t)tau_den * W * (L[r] + f[t]) <= (int64_t)(tau_den + tau_num) * sum_f;
                if (pass == 0 && !feasible) continue;
                int64_t delta = r != q_home[t] ? v_qo[t] : 0;
                for (int32_t e = kv_off[t]; e < kv_off[t + 1]; ++e)
                    if (!C[(int64_t)r * NG + kv_grp[e]]) delta += v_g[kv_grp[e]];
                int better;
                if (best < 0) better = 1;
                else if (pass == 0) better = delta < best_d || (delta == best_d && L[r] < L[best]);
                else better = L[r] < L[best] || (L[r] == L[best] && delta < best_d);
                if (better) { best = r; best_d = delta; }   /* equal keys keep the lower r */
            }
            if (pass == 0 && best >= 0) have_feasible = 1;
        }
        (void)have_feasible;
        sigma[t] = best;
        L[best] += f[t];
        for (int32_t e = kv_off[t]; e < kv_off[t + 1]; ++e) C[(int64_t)best * NG + kv_grp[e]] = 1;
        *comm_total += best_d;
    }
    free(keys);
    return 0;
}

/* ------------------------------------------------------------------------------------
 * Tables of a sequence pool for Algorithm 2 (Sections 4.1, 4.3.1) and the exchange volumes that an
 * assignment implies (Section 4.3.3).
 *
 * The pool holds P packed sequences; sequence s occupies tokens [seq_off[s], seq_off[s+1]) of the
 * pool's sample list cu[0..n] and belongs to the CP workers s*CP .. s*CP+CP-1.  The paper leaves the
 * split of a sequence over its CP group open; here worker c of the group holds the c-th run of
 * ceil(L_s / CP) consecutive tokens.
 *   blocks   every sequence is cut at multiples of B from its own start; tile id = block * H + h
 *            with blocks numbered sequence by sequence                                    (Eq. 5)
 *   f        causal pairs of the block, Eq. 6 without the common factor
 *   q(t)     the worker that holds the block's first token
 *   V_Q = V_O = tokens * (hq / H) * d * 2 bytes (bf16)
 *   K(t)     the samples with a token in the block, on head shard h; group id g = j * H + h (Eq. 7)
 *   V_g      K and V of the whole sample on the shard: 2 * len_j * kv_heads_per_shard * d * 2 bytes,
 *            kv_heads_per_shard = hkv / H if H <= hkv, else 1 (shards share a replicated kv head)
 *   resident the worker that holds every token of sample j, or -1
 * ------------------------------------------------------------------------------------ */
static int tap_owner(const int32_t* seq_off, int s, int CP, int64_t tok) {
    const int64_t len = seq_off[s + 1] - seq_off[s];
    const int64_t run = (len + CP - 1) / CP;
    return s * CP + (int)((tok - seq_off[s]) / (run > 0 ? run : 1));
}

int64_t oracle_tap_num_tiles(const int32_t* seq_off, int P, int B, int H) {
    int64_t nb = 0;
    for (int s = 0; s < P; ++s) nb += ((int64_t)seq_off[s + 1] - seq_off[s] + B - 1) / B;
    return nb * H;
}

int oracle_tap_layout(const int32_t* cu, int n, const int32_t* seq_off, int P, int CP, int B, int H, int hq, int hkv,
                      int d, int64_t* f, int32_t* q_home, int64_t* v_qo, int32_t* kv_off, int32_t* kv_grp /*[<= NB + n] * H*/,
                      int64_t* v_g /*[n*H]*/, int32_t* resident /*[n*H]*/) {
    if (!cu || !seq_off || n <= 0 || P <= 0 || CP <= 0 || B <= 0 || H <= 0 || hq % H != 0) return -1;
    if (!((H <= hkv && hkv % H == 0) || (H > hkv && H % hkv == 0))) return -1;
    const int kvps = H <= hkv ? hkv / H : 1;
    for (int j = 0; j < n; ++j) {
        const int64_t a = cu[j], e = cu[j + 1];
        int s = 0;
        while (s + 1 < P && seq_off[s + 1] <= a && !(a == e && seq_off[s + 1] > a)) ++s;  /* sequence of the sample */
        int res = -1;
        if (e > a) {
            const int first = tap_owner(seq_off, s, CP, a), last = tap_owner(seq_off, s, CP, e - 1);
            res = first == last ? first : -1;
        }
        for (int h = 0; h < H; ++h) {
            v_g[(int64_t)j * H + h] = 2 * (e - a) * kvps * d * 2;
            resident[(int64_t)j * H + h] = res;
        }
    }
    int64_t blk = 0;
    int32_t refs = 0;
    for (int s = 0; s < P; ++s) {
        for (int64_t q0 = seq_off[s]; q0 < seq_off[s + 1]; q0 += B, ++blk) {
            const int64_t q1 = q0 + B < seq_off[s + 1] ? q0 + B : seq_off[s + 1];
            int64_t w = 0;
            for (int j = 0; j < n; ++j) {
                const int64_t lo = q0 > cu[j] ? q0 : cu[j], hi = q1 < cu[j + 1] ? q1 : cu[j + 1];
                for (int64_t g = lo; g < hi; ++g) w += g - cu[j] + 1;
            }
            for (int h = 0; h < H; ++h) {
                const int64_t t = blk * H + h;
                f[t] = w;
                q_home[t] = tap_owner(seq_off, s, CP, q0);
                v_qo[t] = 2 * ((q1 - q0) * (hq / H) * d * 2);
                kv_off[t] = refs;
                for (int j = 0; j < n; ++j) {
                    const int64_t lo = q0 > cu[j] ? q0 : cu[j], hi = q1 < cu[j + 1] ? q1 : cu[j + 1];
                    if (lo < hi) kv_grp[refs++] = j * H + h;
                }
            }
        }
    }
    kv_off[blk * H] = refs;
    return 0;
}

/* Bytes every worker sends to every other in the forward pass under assignment sigma with final
 * residency C (from oracle_tap_place): a KV group selected for destination r and not resident there
 * is fetched once per destination, each token run from the worker that holds it (runs already at r
 * do not move); a tile away from its Q-home has its Q sent there and its output sent back.  The
 * backward pass moves dO along the Q path, dQ along the output path and dK/dV back along the KV
 * paths, so its matrix is the forward's KV part transposed plus the same Q / output part. */
int oracle_tap_exchange(const int32_t* cu, int n, const int32_t* seq_off, int P, int CP, int H, int hkv, int d,
                        int64_t NT, const int32_t* sigma, const int32_t* q_home, const int64_t* v_qo,
                        const uint8_t* C, const int32_t* resident, int64_t* fwd /*[W*W] src-major*/, int64_t* bwd) {
    const int W = P * CP;
    const int kvps = H <= hkv ? hkv / H : 1;
    for (int64_t i = 0; i < (int64_t)W * W; ++i) fwd[i] = bwd[i] = 0;
    for (int r = 0; r < W; ++r)
        for (int j = 0; j < n; ++j)
            for (int h = 0; h < H; ++h) {
                const int64_t g = (int64_t)j * H + h;
                if (!C[(int64_t)r * n * H + g] || resident[g] == r) continue;
                int s = 0;
                while (s + 1 < P && seq_off[s + 1] <= cu[j]) ++s;
                for (int64_t tok = cu[j]; tok < cu[j + 1]; ++tok) {
                    const int w = tap_owner(seq_off, s, CP, tok);
                    if (w == r) continue;
                    fwd[(int64_t)w * W + r] += 2 * (int64_t)kvps * d * 2;
                    bwd[(int64_t)r * W + w] += 2 * (int64_t)kvps * d * 2;
                }
            }
    for (int64_t t = 0; t < NT; ++t) {
        const int q = q_home[t], r = sigma[t];
        if (q == r) continue;
        fwd[(int64_t)q * W + r] += v_qo[t] / 2;   /* Q out */
        fwd[(int64_t)r * W + q] += v_qo[t] / 2;   /* output back */
        bwd[(int64_t)q * W + r] += v_qo[t] / 2;   /* dO along the Q path */
        bwd[(int64_t)r * W + q] += v_qo[t] / 2;   /* dQ along the output path */
    }
    return 0;
}
