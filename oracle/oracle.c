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
