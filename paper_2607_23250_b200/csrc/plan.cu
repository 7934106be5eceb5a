// Device tile planner: SH-Tile construction (Section 4.3.1, Eq. 5), tile weights (Eq. 6) and
// heaviest-first placement (Algorithm 2 with a zero communication term) as CUDA kernels.
//
// Integer work only; every result must equal the step-by-step definition bit for bit.
#include <stdio.h>

#include <new>

#include "common.h"

namespace libra {

std::atomic<int64_t> g_launches{0};

static std::atomic<int> g_cfg[kMaxDevices][kCfgSlots];
bool cfg_done(int slot) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return false;
    return g_cfg[dev][slot].load(std::memory_order_acquire) != 0;
}
void cfg_mark(int slot) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return;
    g_cfg[dev][slot].store(1, std::memory_order_release);
}
int check_plan_device(const libra_plan* plan) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return LIBRA_ERR_NO_DEVICE;
    return dev == plan->device ? LIBRA_OK : LIBRA_ERR_PLAN_MISMATCH;
}

// ---- kernels --------------------------------------------------------------------------------

// cu_seqlens checks: starts at 0, non-decreasing, ends at T.
__global__ void k_validate(const int32_t* __restrict__ cu, int n, int64_t T, int* status) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j > n) return;
    bool bad = false;
    if (j == 0 && cu[0] != 0) bad = true;
    if (j == n && cu[n] != T) bad = true;
    if (j < n && cu[j + 1] < cu[j]) bad = true;
    if (bad) atomicExch(status, LIBRA_ERR_BAD_SEQLENS);
}

// For every token: the bounds [start, end) of the sample that holds it.
// The search keeps every index inside [0, n] whatever cu contains, and the bounds are clamped to
// start <= t < end <= T, so that a malformed cu_seqlens (flagged by k_validate) can never make a
// later kernel form an address outside its tensors.
__global__ void k_token_bounds(const int32_t* __restrict__ cu, int n, int64_t T, int32_t* __restrict__ tok_start,
                               int32_t* __restrict__ tok_end) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= T) return;
    int lo = 0, hi = n;  // find the last j in [0, n) with cu[j] <= t
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (cu[mid] <= t) lo = mid; else hi = mid;
    }
    const int64_t a = cu[lo], e = cu[lo + 1];
    tok_start[t] = (int32_t)(a < 0 ? 0 : (a > t ? t : a));
    tok_end[t] = (int32_t)(e < t + 1 ? t + 1 : (e > T ? T : e));
}

// Weight of block b (Eq. 6): a token at position p of a sample of length len contributes
// p + 1 pairs as a query (keys 0..p) and len - p pairs as a key (queries p..len-1).
__global__ void k_block_weights(const int32_t* __restrict__ tok_start, const int32_t* __restrict__ tok_end,
                                int64_t T, int tile, int64_t NB, int key_major, int64_t* __restrict__ weight_blk) {
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= NB) return;
    const int64_t t0 = b * tile;
    const int64_t t1 = (t0 + tile < T) ? t0 + tile : T;
    int64_t w = 0;
    for (int64_t t = t0; t < t1; ++t) w += key_major ? (int64_t)tok_end[t] - t : t - (int64_t)tok_start[t] + 1;
    weight_blk[b] = w;
}

// Block-count weight (LIBRA_WEIGHT_BLOCKS): the token axis is cut into chunks at multiples of g.  For a
// chunk of query rows [r0, r1] the visible keys span the chunks from the one holding the first key of r0's
// sample to the one holding r1 (row r0 sees a key in every chunk of that range, later rows see no chunk
// outside it); for a chunk of keys [c0, c1] the attending queries span the chunks from the one holding c0
// to the one holding the last token of c1's sample.
__global__ void k_block_weights_blocks(const int32_t* __restrict__ tok_start, const int32_t* __restrict__ tok_end,
                                       int64_t T, int tile, int64_t NB, int key_major, int g, int unit_cost,
                                       int64_t* __restrict__ weight_blk) {
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= NB) return;
    const int64_t t0 = b * tile;
    const int64_t t1 = (t0 + tile < T) ? t0 + tile : T;
    int64_t w = 0;
    for (int64_t c = t0 / g; c * g < t1; ++c) {
        const int64_t first = c * g > t0 ? c * g : t0;
        const int64_t last = ((c + 1) * g < t1 ? (c + 1) * g : t1) - 1;
        const int64_t n = key_major ? ((int64_t)tok_end[last] - 1) / g - first / g + 1
                                    : last / g - (int64_t)tok_start[first] / g + 1;
        w += 8 * n + unit_cost;
    }
    weight_blk[b] = w;
}

// Order of Algorithm 2: decreasing weight, then increasing id.  All H shards of a block weigh
// the same and their ids b*H+h are consecutive, so ordering the blocks orders the tiles.
// rank(b) = number of blocks that precede b; one thread per block, O(NB) each.
__global__ void k_rank_blocks(const int64_t* __restrict__ weight_blk, int64_t NB, int32_t* __restrict__ blk_order) {
    __shared__ int64_t sw[256];
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t wb = b < NB ? weight_blk[b] : 0;
    int64_t rank = 0;
    for (int64_t base = 0; base < NB; base += 256) {
        const int64_t o = base + threadIdx.x;
        sw[threadIdx.x] = o < NB ? weight_blk[o] : -1;
        __syncthreads();
        const int lim = (int)((NB - base < 256) ? NB - base : 256);
        for (int i = 0; i < lim; ++i) {
            const int64_t w = sw[i];
            rank += (w > wb) || (w == wb && base + i < b);
        }
        __syncthreads();
    }
    if (b < NB) blk_order[rank] = (int32_t)b;
}

// Sequential placement by one warp (Algorithm 2's greedy rule: the next tile goes to the least-loaded worker, lowest
// index among equals).  The workers are kept as ONE sorted array of keys (load << 10 | worker) in shared memory; loads
// stay below 2^53 (checked on the host from the weight total) and there are at most 1024 workers, so a key fits 64 bits.
//   * Consecutive tiles are placed in waves.  Tile s of a batch goes to key[s], the s-th worker of the array, as long
//     as key[s] lies below every key put back by the tiles before it (key[s'] + w[s'], s' < s): nothing put back can
//     then overtake it.  The longest such prefix (at most 32 tiles) is placed at once, one tile per worker; the keys
//     put back are ranked among themselves and merged with the rest of the array (every key finds its place by a
//     binary search in the other sequence).  With equal weights (the H head shards of a block) the condition is
//     key[s] < key[0] + w.  The result is tile for tile what the one-by-one rule gives.
//   * When fewer than kWaveMin tiles can go at once, one tile takes the first key and re-inserts it: the warp counts
//     the keys below the new one and shifts that part of the array down by one.
constexpr int kPlaceMaxW = 1024;
constexpr int kWaveMin = 4;

struct PlaceJob {
    const int64_t* weight_blk;
    const int32_t* blk_order;   // null: tiles in id order, id = head * NB + block
    int64_t NB, NT;
    int H, W;
    int32_t* cta_of_tile;
    int32_t* pos;
    int32_t* cta_offsets;
    int64_t* loads;
};
struct PlaceJobs {
    PlaceJob job[3];            // the directions of a plan are independent: one block (one warp) each
};

template <int PER>   // PER * 32 >= W
__global__ void __launch_bounds__(32) k_place(const PlaceJobs jobs) {
    const PlaceJob& jb = jobs.job[blockIdx.x];
    const int64_t* __restrict__ weight_blk = jb.weight_blk;
    const int32_t* __restrict__ blk_order = jb.blk_order;
    const int64_t NB = jb.NB, NT = jb.NT;
    const int H = jb.H, W = jb.W;
    int32_t* __restrict__ cta_of_tile = jb.cta_of_tile;
    int32_t* __restrict__ pos = jb.pos;
    int32_t* __restrict__ cta_offsets = jb.cta_offsets;
    int64_t* __restrict__ loads = jb.loads;
    __shared__ uint64_t key_a[kPlaceMaxW], key_b[kPlaceMaxW];   // the sorted array and its next version
    __shared__ uint64_t back[32];                               // keys put back by a wave, in order
    __shared__ uint64_t put_raw[32];                            // the same in tile order
    __shared__ int32_t cnt[kPlaceMaxW];                         // tiles per worker so far
    const int lane = threadIdx.x;
    uint64_t* cur = key_a;
    uint64_t* nxt = key_b;
    for (int r = lane; r < W; r += 32) { cur[r] = (uint64_t)r; cnt[r] = 0; }
    __syncwarp();
    for (int64_t x0 = 0; x0 < NT; x0 += 32) {
        // each lane fetches one upcoming tile
        const int64_t xl = x0 + lane;
        int64_t w_l = -1;
        int32_t t_l = 0;
        if (xl < NT) {
            if (blk_order) {
                const int32_t blk = blk_order[xl / H];
                w_l = weight_blk[blk];
                t_l = (int32_t)((int64_t)blk * H + xl % H);
            } else {
                w_l = weight_blk[xl % NB];
                t_l = (int32_t)xl;
            }
        }
        const int lim = (int)((NT - x0 < 32) ? NT - x0 : 32);
        int i = 0;
        while (i < lim) {
            const int64_t w = __shfl_sync(0xffffffffu, w_l, i);
            if (w == 0) {
                // weightless tiles all go to the first worker and change nothing else
                const unsigned same = __ballot_sync(0xffffffffu, w_l == 0) >> i;
                int n = (~same == 0u) ? 32 : __ffs(~same) - 1;
                if (n > lim - i) n = lim - i;
                const int r0 = (int)(cur[0] & 1023u);
                const int base = cnt[r0];
                __syncwarp();
                if (lane >= i && lane < i + n) { cta_of_tile[t_l] = r0; pos[t_l] = base + (lane - i); }
                if (lane == 0) cnt[r0] = base + n;
                __syncwarp();
                i += n;
                continue;
            }
            // lane s looks at tile i + s of the batch and at key[s]
            const int64_t w_s = __shfl_sync(0xffffffffu, w_l, (i + lane) & 31);
            const bool live = i + lane < lim && lane < W && w_s > 0;
            const uint64_t first = cur[0];
            const uint64_t add = (uint64_t)w << 10;
            const uint64_t mine_k = lane < W ? cur[lane] : ~0ull;
            const uint64_t put = live ? mine_k + ((uint64_t)w_s << 10) : ~0ull;
            uint64_t before = put;                                // min of the keys put back by the lanes below this one
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint64_t other = __shfl_up_sync(0xffffffffu, before, o);
                if (lane >= o && other < before) before = other;
            }
            before = __shfl_up_sync(0xffffffffu, before, 1);
            if (lane == 0) before = ~0ull;
            const unsigned fits = __ballot_sync(0xffffffffu, live && mine_k < before);
            const int take = (~fits == 0u) ? 32 : __ffs(~fits) - 1;
            if (take < kWaveMin) {
                // one tile: the first key, put back w heavier at its new place
                const uint64_t k1 = first + add;
                const int r0 = (int)(first & 1023u);
                int below = 0;                                    // keys of cur[1..W) below the new key
                uint64_t mine[PER];
#pragma unroll
                for (int u = 0; u < PER; ++u) {
                    const int idx = 1 + lane + 32 * u;
                    mine[u] = idx < W ? cur[idx] : ~0ull;
                    below += (idx < W && mine[u] < k1) ? 1 : 0;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) below += __shfl_xor_sync(0xffffffffu, below, o);
                __syncwarp();
#pragma unroll
                for (int u = 0; u < PER; ++u) {
                    const int idx = 1 + lane + 32 * u;
                    if (idx <= below) cur[idx - 1] = mine[u];     // the keys below the new one move down by one
                }
                if (lane == 0) cur[below] = k1;
                const int32_t t = __shfl_sync(0xffffffffu, t_l, i);
                if (lane == 0) { cta_of_tile[t] = r0; pos[t] = cnt[r0]; cnt[r0] += 1; }
                __syncwarp();
                i += 1;
                continue;
            }
            // ---- a wave: tile i + s goes to the worker of key[s], s < take; the workers are distinct ----
            {
                const int32_t t = __shfl_sync(0xffffffffu, t_l, (i + lane) & 31);
                if (lane < take) {
                    const int r = (int)(mine_k & 1023u);
                    cta_of_tile[t] = r;
                    pos[t] = cnt[r];
                    cnt[r] += 1;
                    put_raw[lane] = put;
                }
                __syncwarp();
                if (lane < take) {   // the keys put back, ranked among themselves (all keys differ)
                    int rank = 0;
                    for (int j = 0; j < take; ++j) rank += put_raw[j] < put ? 1 : 0;
                    back[rank] = put;
                }
                __syncwarp();
                // the rest of the array and the keys put back, merged into the new sorted array
                const int na = W - take;
                for (int idx = lane; idx < na; idx += 32) {       // a key of the array: keys put back that are below it
                    const uint64_t k = cur[take + idx];
                    int lo = 0, hi = take;
                    while (lo < hi) { const int mid = (lo + hi) >> 1; if (back[mid] < k) lo = mid + 1; else hi = mid; }
                    nxt[idx + lo] = k;
                }
                if (lane < take) {                                 // a key put back: keys of the array below it
                    const uint64_t k = back[lane];
                    int lo = 0, hi = na;
                    while (lo < hi) { const int mid = (lo + hi) >> 1; if (cur[take + mid] < k) lo = mid + 1; else hi = mid; }
                    nxt[lane + lo] = k;
                }
                __syncwarp();
                uint64_t* tmp = cur; cur = nxt; nxt = tmp;
            }
            i += take;
        }
    }
    __syncwarp();
    for (int idx = lane; idx < W; idx += 32) {
        const uint64_t k = cur[idx];
        loads[k & 1023u] = (int64_t)(k >> 10);
    }
    for (int r = lane; r < W; r += 32) cta_offsets[r + 1] = cnt[r];
    __syncwarp();
    if (lane == 0) {  // counts -> offsets
        cta_offsets[0] = 0;
        int32_t run = 0;
        for (int r = 0; r < W; ++r) { run += cta_offsets[r + 1]; cta_offsets[r + 1] = run; }
    }
}

__global__ void k_scatter_lists(const int32_t* __restrict__ cta_of_tile, const int32_t* __restrict__ pos,
                                const int32_t* __restrict__ cta_offsets, int64_t NT, int32_t* __restrict__ cta_tiles) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= NT) return;
    cta_tiles[cta_offsets[cta_of_tile[t]] + pos[t]] = (int32_t)t;
}

// Execution order inside a worker's list.  The placement fixes WHICH tiles a worker runs; the order
// it runs them in is free.  Sorting every list by (head shard, block) makes all workers sweep
// the same head and neighbouring blocks at about the same time, so that the tiles several workers
// read (K/V in the forward and the dQ kernel, Q/dO in the dK/dV kernel) are more often found in L2.
// One thread block per worker, rank sort.
__global__ void k_exec_order(const int32_t* __restrict__ cta_offsets, const int32_t* __restrict__ cta_tiles, int H,
                             int64_t NB, int32_t* __restrict__ cta_exec) {
    const int r = blockIdx.x;
    const int beg = cta_offsets[r], n = cta_offsets[r + 1] - beg;
    if (n > 16384) {  // quadratic sort too slow: keep placement order
        for (int i = threadIdx.x; i < n; i += blockDim.x) cta_exec[beg + i] = cta_tiles[beg + i];
        return;
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int32_t t = cta_tiles[beg + i];
        const int64_t key = (int64_t)(t % H) * NB + t / H;
        int rank = 0;
        for (int j = 0; j < n; ++j) {
            const int32_t u = cta_tiles[beg + j];
            rank += ((int64_t)(u % H) * NB + u / H) < key;
        }
        cta_exec[beg + rank] = t;
    }
}

// ---- pair tiles: key block x query chunk x head (the fused backward's units) ---------------------------------
// The score matrix in tile x tile cells: cell (i, j) is live when a query of row block i attends a key of key
// block j; for a key block the live cells are the row blocks j .. last(j), last(j) = the block of the last token
// of the sample that holds the key block's last key.  Pair-block (c, j) = key block j against the R = chunk / tile
// row blocks of query chunk c, present when one of them is live; numbered chunk by chunk, key blocks ascending.
// last(j) never decreases with j, so the key blocks of a chunk are the range first(c) .. min(NKB, (c+1) R) - 1.
__device__ __forceinline__ int64_t pair_last_row_block(const int32_t* tok_end, int64_t T, int tile, int64_t j) {
    const int64_t last_key = ((j + 1) * tile < T ? (j + 1) * tile : T) - 1;
    return ((int64_t)tok_end[last_key] - 1) / tile;
}
__global__ void k_pair_chunks(const int32_t* __restrict__ tok_end, int64_t T, int tile, int R, int64_t NKB, int64_t NC,
                              int32_t* __restrict__ first_j, int32_t* __restrict__ count) {
    const int64_t c = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (c >= NC) return;
    int64_t lo = 0, hi = NKB;   // first j with last(j) / R >= c
    while (lo < hi) {
        const int64_t mid = (lo + hi) >> 1;
        if (pair_last_row_block(tok_end, T, tile, mid) / R >= c) hi = mid; else lo = mid + 1;
    }
    const int64_t last = (c + 1) * R - 1 < NKB - 1 ? (c + 1) * R - 1 : NKB - 1;
    first_j[c] = (int32_t)lo;
    count[c] = (int32_t)(last >= lo ? last - lo + 1 : 0);
}
// One block: exclusive prefix sum of count[0..n) into base, total into *total.
__global__ void __launch_bounds__(1024) k_scan_i32(const int32_t* __restrict__ count, int64_t n, int64_t* __restrict__ base,
                                                   int64_t* __restrict__ total) {
    __shared__ int64_t part[1024];
    const int64_t per = (n + blockDim.x - 1) / blockDim.x;
    const int64_t x0 = threadIdx.x * per, x1 = x0 + per < n ? x0 + per : n;
    int64_t sum = 0;
    for (int64_t x = x0; x < x1; ++x) sum += count[x];
    part[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t run = 0;
        for (int i = 0; i < (int)blockDim.x; ++i) { const int64_t v = part[i]; part[i] = run; run += v; }
        *total = run;
    }
    __syncthreads();
    int64_t run = part[threadIdx.x];
    for (int64_t x = x0; x < x1; ++x) { base[x] = run; run += count[x]; }
}
// Weight of pair-block (c, j): its live cells, min(last(j), c R + R - 1) - max(j, c R) + 1.
__global__ void k_pair_fill(const int32_t* __restrict__ tok_end, int64_t T, int tile, int R, int64_t NC,
                            const int32_t* __restrict__ first_j, const int32_t* __restrict__ count,
                            const int64_t* __restrict__ base, int32_t* __restrict__ u_blk,
                            int32_t* __restrict__ u_chunk, int64_t* __restrict__ weight_blk) {
    const int64_t c = blockIdx.x;
    if (c >= NC) return;
    for (int x = threadIdx.x; x < count[c]; x += blockDim.x) {
        const int64_t j = first_j[c] + x, u = base[c] + x;
        const int64_t last = pair_last_row_block(tok_end, T, tile, j);
        const int64_t i0 = j > c * R ? j : c * R, i1 = last < c * R + R - 1 ? last : c * R + R - 1;
        u_blk[u] = (int32_t)j;
        u_chunk[u] = (int32_t)c;
        weight_blk[u] = i1 - i0 + 1;
    }
}

// Expanders used by libra_plan_export.
__global__ void k_expand_weight(const int64_t* __restrict__ weight_blk, int64_t NT, int H, int64_t NB_headmajor,
                                int64_t* __restrict__ out) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t < NT) out[t] = NB_headmajor ? weight_blk[t % NB_headmajor] : weight_blk[t / H];
}
__global__ void k_expand_order(const int32_t* __restrict__ blk_order, int64_t NT, int H, int32_t* __restrict__ out) {
    const int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (x < NT) out[x] = blk_order ? (int32_t)((int64_t)blk_order[x / H] * H + x % H) : (int32_t)x;
}

// ---- host ---------------------------------------------------------------------------------

static inline unsigned grid_for(int64_t n, int block) { return (unsigned)((n + block - 1) / block); }

static void free_dir(PlanDir& d) {
    cudaFree(d.d_weight_blk); cudaFree(d.d_blk_order); cudaFree(d.d_cta_of_tile); cudaFree(d.d_pos);
    cudaFree(d.d_cta_offsets); cudaFree(d.d_cta_tiles); cudaFree(d.d_cta_exec); cudaFree(d.d_loads); cudaFree(d.d_busy); cudaFree(d.d_busy2); cudaFree(d.d_tile_ns);
    cudaFree(d.d_u_blk); cudaFree(d.d_u_chunk);
    d = PlanDir();
}

// The pair-blocks of a plan: counts per query chunk, their prefix sums, and the total read back (one synchronous
// 8-byte copy).  The query chunk is doubled while there are more than 262144 pair-blocks (the placement is
// sequential, about a third of a microsecond per tile).
struct PairTables { int32_t* first_j = nullptr; int32_t* count = nullptr; int64_t* base = nullptr; int64_t NC = 0; };
static void free_pair_tables(PairTables& t) { cudaFree(t.first_j); cudaFree(t.count); cudaFree(t.base); t = PairTables(); }
static int count_pair_blocks(libra_plan* p, PlanDir& d, PairTables& tb) {
    const int64_t T = p->T, NKB = (T + d.tile - 1) / d.tile;
    for (;;) {
        const int R = d.chunk / d.tile;
        tb.NC = (NKB + R - 1) / R;
        if (cudaMalloc((void**)&tb.first_j, sizeof(int32_t) * tb.NC) != cudaSuccess ||
            cudaMalloc((void**)&tb.count, sizeof(int32_t) * tb.NC) != cudaSuccess ||
            cudaMalloc((void**)&tb.base, sizeof(int64_t) * (tb.NC + 1)) != cudaSuccess)
            { free_pair_tables(tb); return LIBRA_ERR_CUDA; }
        k_pair_chunks<<<(unsigned)((tb.NC + 127) / 128), 128, 0, p->stream>>>(p->d_tok_end, T, d.tile, R, NKB, tb.NC,
                                                                             tb.first_j, tb.count);
        k_scan_i32<<<1, 1024, 0, p->stream>>>(tb.count, tb.NC, tb.base, tb.base + tb.NC);
        count_launch(2);
        int64_t nu = 0;
        if (cudaMemcpyAsync(&nu, tb.base + tb.NC, sizeof(int64_t), cudaMemcpyDeviceToHost, p->stream) != cudaSuccess ||
            cudaStreamSynchronize(p->stream) != cudaSuccess) { free_pair_tables(tb); return LIBRA_ERR_CUDA; }
        d.NB = nu;
        if (nu <= 262144) return LIBRA_OK;
        free_pair_tables(tb);
        if ((int64_t)d.chunk * 2 > (int64_t)1 << 30) return LIBRA_ERR_UNSUPPORTED;
        d.chunk *= 2;
    }
}

// First half of a direction: sizes, allocations, weights and block order; fills the placement job.
static int build_dir(libra_plan* p, PlanDir& d, int key_major, const libra_plan_opts& o, bool pairs, PlaceJob* job) {
    const int64_t T = p->T;
    PairTables tb;
    if (pairs) {
        const int rcp = count_pair_blocks(p, d, tb);
        if (rcp != LIBRA_OK) return rcp;
    } else {
        d.NB = (T + d.tile - 1) / d.tile;
    }
    if (d.NB * (int64_t)d.H >= (int64_t)INT32_MAX) { free_pair_tables(tb); return LIBRA_ERR_OVERFLOW; }
    // a worker's load is at most the weight total <= H * T^2 / 2 + ...; the placement packs load * 1024 + index
    if ((long double)d.H * (long double)T * (long double)T >= 9.0e15L) return LIBRA_ERR_OVERFLOW;
    if (!pairs && d.NB > 65536) return LIBRA_ERR_UNSUPPORTED;  // the rank sort is quadratic in blocks
    if (d.W > 1024) return LIBRA_ERR_UNSUPPORTED;
    d.NT = d.NB * d.H;
    cudaError_t e = cudaSuccess;
    auto A = [&](void** ptr, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(ptr, bytes ? bytes : 1); };
    A((void**)&d.d_weight_blk, sizeof(int64_t) * d.NB);
    A((void**)&d.d_blk_order, sizeof(int32_t) * d.NB);
    A((void**)&d.d_cta_of_tile, sizeof(int32_t) * d.NT);
    A((void**)&d.d_pos, sizeof(int32_t) * d.NT);
    A((void**)&d.d_cta_offsets, sizeof(int32_t) * (d.W + 1));
    A((void**)&d.d_cta_tiles, sizeof(int32_t) * d.NT);
    A((void**)&d.d_cta_exec, sizeof(int32_t) * d.NT);
    A((void**)&d.d_loads, sizeof(int64_t) * d.W);
    A((void**)&d.d_busy, sizeof(uint64_t) * 2 * d.W);
    A((void**)&d.d_busy2, sizeof(uint64_t) * 2 * d.W);
    A((void**)&d.d_tile_ns, sizeof(uint32_t) * d.NT);
    if (pairs) {
        A((void**)&d.d_u_blk, sizeof(int32_t) * d.NB);
        A((void**)&d.d_u_chunk, sizeof(int32_t) * d.NB);
    }
    if (e != cudaSuccess) { free_pair_tables(tb); return LIBRA_ERR_CUDA; }
    cudaStream_t s = p->stream;
    cudaMemsetAsync(d.d_busy, 0, sizeof(uint64_t) * 2 * d.W, s);
    cudaMemsetAsync(d.d_busy2, 0, sizeof(uint64_t) * 2 * d.W, s);
    cudaMemsetAsync(d.d_tile_ns, 0, sizeof(uint32_t) * d.NT, s);
    if (pairs) {
        k_pair_fill<<<(unsigned)tb.NC, 128, 0, s>>>(p->d_tok_end, T, d.tile, d.chunk / d.tile, tb.NC, tb.first_j, tb.count,
                                                    tb.base, d.d_u_blk, d.d_u_chunk, d.d_weight_blk);
        cudaStreamSynchronize(s);   // the tables are read by the kernel above
        free_pair_tables(tb);
    } else if (o.weight_model == LIBRA_WEIGHT_BLOCKS)
        k_block_weights_blocks<<<grid_for(d.NB, 128), 128, 0, s>>>(p->d_tok_start, p->d_tok_end, T, d.tile, d.NB,
                                                                   key_major, o.cost_block ? o.cost_block : 128,
                                                                   key_major ? o.unit_cost_kv : o.unit_cost_q,
                                                                   d.d_weight_blk);
    else
        k_block_weights<<<grid_for(d.NB, 128), 128, 0, s>>>(p->d_tok_start, p->d_tok_end, T, d.tile, d.NB, key_major,
                                                            d.d_weight_blk);
    if (!pairs) k_rank_blocks<<<grid_for(d.NB, 256), 256, 0, s>>>(d.d_weight_blk, d.NB, d.d_blk_order);
    job->weight_blk = d.d_weight_blk;
    job->blk_order = pairs ? nullptr : d.d_blk_order;   // pair tiles are placed in id order
    job->NB = d.NB; job->NT = d.NT; job->H = d.H; job->W = d.W;
    job->cta_of_tile = d.d_cta_of_tile; job->pos = d.d_pos; job->cta_offsets = d.d_cta_offsets; job->loads = d.d_loads;
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

// The placements of all directions in one launch (a block of one warp per direction).
static int place_all(const PlaceJobs& jobs, int n, int max_w, cudaStream_t s) {
    if (n == 0) return LIBRA_OK;
    if (max_w <= 160)
        k_place<5><<<n, 32, 0, s>>>(jobs);
    else if (max_w <= 320)
        k_place<10><<<n, 32, 0, s>>>(jobs);
    else
        k_place<32><<<n, 32, 0, s>>>(jobs);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

// Second half of a direction: the per-worker lists from the placement.
static int finish_dir(libra_plan* p, PlanDir& d, bool pairs) {
    cudaStream_t s = p->stream;
    k_scatter_lists<<<grid_for(d.NT, 256), 256, 0, s>>>(d.d_cta_of_tile, d.d_pos, d.d_cta_offsets, d.NT,
                                                        d.d_cta_tiles);
    if (pairs)   // placed in id order: the lists already are in execution order
        cudaMemcpyAsync(d.d_cta_exec, d.d_cta_tiles, sizeof(int32_t) * d.NT, cudaMemcpyDeviceToDevice, s);
    else
        k_exec_order<<<d.W, 256, 0, s>>>(d.d_cta_offsets, d.d_cta_tiles, d.H, d.NB, d.d_cta_exec);
    count_launch(2);
    d.enabled = 1;
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace libra

using namespace libra;

extern "C" int libra_plan_tiles(const int32_t* cu_seqlens_dev, int n_samples, int n_heads, int tile_q,
                                const libra_plan_opts* opts, void* stream, libra_plan_t** plan_out) {
    if (!cu_seqlens_dev || !plan_out || n_samples <= 0 || n_heads <= 0 || tile_q <= 0) return LIBRA_ERR_INVALID_ARG;
    *plan_out = nullptr;
    libra_plan_opts o = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0};
    if (opts) o = *opts;
    if (o.n_workers < 0 || o.tile_kv < 0 || o.n_heads_kv < 0 || o.total_tokens < 0) return LIBRA_ERR_INVALID_ARG;
    if (o.directions & ~(LIBRA_DIR_Q | LIBRA_DIR_KV | LIBRA_DIR_PAIR)) return LIBRA_ERR_INVALID_ARG;
    if (o.pair_chunk < 0) return LIBRA_ERR_INVALID_ARG;
    if (o.weight_model != LIBRA_WEIGHT_PAIRS && o.weight_model != LIBRA_WEIGHT_BLOCKS) return LIBRA_ERR_INVALID_ARG;
    if (o.cost_block < 0 || o.unit_cost_q < 0 || o.unit_cost_kv < 0) return LIBRA_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return LIBRA_ERR_NO_DEVICE;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return LIBRA_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)stream;
    int64_t T = o.total_tokens;
    if (T == 0) {
        int32_t last = 0;
        if (cudaMemcpyAsync(&last, cu_seqlens_dev + n_samples, sizeof(int32_t), cudaMemcpyDeviceToHost, s) !=
                cudaSuccess ||
            cudaStreamSynchronize(s) != cudaSuccess)
            return LIBRA_ERR_CUDA;
        T = last;
    }
    if (T <= 0 || T >= (int64_t)INT32_MAX) return LIBRA_ERR_INVALID_ARG;

    libra_plan* p = new (std::nothrow) libra_plan();
    if (!p) return LIBRA_ERR_CUDA;
    p->T = T; p->n = n_samples; p->device = dev; p->sm_count = sms; p->stream = s;
    int rc = LIBRA_OK;
    if (cudaMalloc((void**)&p->d_tok_start, sizeof(int32_t) * T) != cudaSuccess ||
        cudaMalloc((void**)&p->d_tok_end, sizeof(int32_t) * T) != cudaSuccess ||
        cudaMalloc((void**)&p->d_status, sizeof(int) * 4) != cudaSuccess)
        rc = LIBRA_ERR_CUDA;
    if (rc == LIBRA_OK) {
        cudaMemsetAsync(p->d_status, 0, sizeof(int) * 4, s);
        k_validate<<<grid_for(n_samples + 1, 128), 128, 0, s>>>(cu_seqlens_dev, n_samples, T, p->d_status);
        k_token_bounds<<<grid_for(T, 256), 256, 0, s>>>(cu_seqlens_dev, n_samples, T, p->d_tok_start, p->d_tok_end);
        count_launch(2);
        const int dirs = o.directions ? o.directions : (LIBRA_DIR_Q | LIBRA_DIR_KV);
        const int W = o.n_workers ? o.n_workers : sms;
        PlaceJobs jobs = {};
        int n_jobs = 0;
        bool built[3] = {false, false, false};
        if (dirs & LIBRA_DIR_Q) {
            PlanDir& d = p->dir[0];
            d.tile = tile_q; d.H = n_heads; d.W = W;
            rc = build_dir(p, d, 0, o, false, &jobs.job[n_jobs]);
            if (rc == LIBRA_OK) { built[0] = true; ++n_jobs; }
        }
        if (rc == LIBRA_OK && (dirs & LIBRA_DIR_KV)) {
            PlanDir& d = p->dir[1];
            d.tile = o.tile_kv ? o.tile_kv : 128; d.H = o.n_heads_kv ? o.n_heads_kv : n_heads; d.W = W;
            rc = build_dir(p, d, 1, o, false, &jobs.job[n_jobs]);
            if (rc == LIBRA_OK) { built[1] = true; ++n_jobs; }
        }
        if (rc == LIBRA_OK && (dirs & LIBRA_DIR_PAIR)) {
            PlanDir& d = p->dir[2];
            d.tile = o.tile_kv ? o.tile_kv : 128; d.H = o.n_heads_kv ? o.n_heads_kv : n_heads; d.W = W;
            d.chunk = o.pair_chunk ? o.pair_chunk : 4096;
            rc = d.chunk % d.tile ? LIBRA_ERR_INVALID_ARG : build_dir(p, d, 1, o, true, &jobs.job[n_jobs]);
            if (rc == LIBRA_OK) { built[2] = true; ++n_jobs; }
        }
        // the directions are independent: their placements run side by side, one warp each
        if (rc == LIBRA_OK) rc = place_all(jobs, n_jobs, W, s);
        for (int k = 0; k < 3 && rc == LIBRA_OK; ++k)
            if (built[k]) rc = finish_dir(p, p->dir[k], k == 2);
    }
    if (rc != LIBRA_OK) {
        libra_plan_destroy(p);
        return rc;
    }
    *plan_out = p;
    return LIBRA_OK;
}

static PlanDir* dir_of(const libra_plan_t* plan, int direction) {
    if (!plan) return nullptr;
    if (direction == LIBRA_DIR_Q) return plan->dir[0].enabled ? const_cast<PlanDir*>(&plan->dir[0]) : nullptr;
    if (direction == LIBRA_DIR_KV) return plan->dir[1].enabled ? const_cast<PlanDir*>(&plan->dir[1]) : nullptr;
    if (direction == LIBRA_DIR_PAIR) return plan->dir[2].enabled ? const_cast<PlanDir*>(&plan->dir[2]) : nullptr;
    return nullptr;
}

extern "C" int libra_plan_info(const libra_plan_t* plan, int direction, int64_t* n_tiles, int* n_workers,
                               int64_t* n_blocks, int* tile, int* n_heads) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    PlanDir* d = dir_of(plan, direction);
    if (!d) return LIBRA_ERR_PLAN_MISMATCH;
    if (n_tiles) *n_tiles = d->NT;
    if (n_workers) *n_workers = d->W;
    if (n_blocks) *n_blocks = d->NB;
    if (tile) *tile = d->tile;
    if (n_heads) *n_heads = d->H;
    return LIBRA_OK;
}

extern "C" int libra_plan_status(const libra_plan_t* plan) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    int st[4] = {0, 0, 0, 0};
    if (cudaStreamSynchronize(plan->stream) != cudaSuccess) return LIBRA_ERR_CUDA;
    if (cudaMemcpy(st, plan->d_status, sizeof(st), cudaMemcpyDeviceToHost) != cudaSuccess) return LIBRA_ERR_CUDA;
    return st[0];
}

extern "C" int libra_plan_export(const libra_plan_t* plan, int direction, int64_t* weight_host, int32_t* order_host,
                                 int32_t* cta_of_tile_host, int32_t* cta_offsets_host, int32_t* cta_tiles_host,
                                 int64_t* loads_host) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    PlanDir* d = dir_of(plan, direction);
    if (!d) return LIBRA_ERR_PLAN_MISMATCH;
    cudaStream_t s = plan->stream;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t x) { if (e == cudaSuccess) e = x; };
    void* tmp = nullptr;
    if (weight_host || order_host) ok(cudaMalloc(&tmp, sizeof(int64_t) * (d->NT ? d->NT : 1)));
    if (e != cudaSuccess) return LIBRA_ERR_CUDA;
    if (weight_host) {
        k_expand_weight<<<grid_for(d->NT, 256), 256, 0, s>>>(d->d_weight_blk, d->NT, d->H, d->d_u_blk ? d->NB : 0,
                                                             (int64_t*)tmp);
        count_launch();
        ok(cudaMemcpyAsync(weight_host, tmp, sizeof(int64_t) * d->NT, cudaMemcpyDeviceToHost, s));
        ok(cudaStreamSynchronize(s));
    }
    if (order_host) {
        k_expand_order<<<grid_for(d->NT, 256), 256, 0, s>>>(d->d_u_blk ? nullptr : d->d_blk_order, d->NT, d->H,
                                                            (int32_t*)tmp);
        count_launch();
        ok(cudaMemcpyAsync(order_host, tmp, sizeof(int32_t) * d->NT, cudaMemcpyDeviceToHost, s));
        ok(cudaStreamSynchronize(s));
    }
    if (cta_of_tile_host)
        ok(cudaMemcpyAsync(cta_of_tile_host, d->d_cta_of_tile, sizeof(int32_t) * d->NT, cudaMemcpyDeviceToHost, s));
    if (cta_offsets_host)
        ok(cudaMemcpyAsync(cta_offsets_host, d->d_cta_offsets, sizeof(int32_t) * (d->W + 1), cudaMemcpyDeviceToHost, s));
    if (cta_tiles_host)
        ok(cudaMemcpyAsync(cta_tiles_host, d->d_cta_tiles, sizeof(int32_t) * d->NT, cudaMemcpyDeviceToHost, s));
    if (loads_host) ok(cudaMemcpyAsync(loads_host, d->d_loads, sizeof(int64_t) * d->W, cudaMemcpyDeviceToHost, s));
    ok(cudaStreamSynchronize(s));
    cudaFree(tmp);
    return e == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_plan_export_pairs(const libra_plan_t* plan, int32_t* key_block_host, int32_t* query_chunk_host,
                                       int* chunk_tokens_host) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    PlanDir* d = dir_of(plan, LIBRA_DIR_PAIR);
    if (!d) return LIBRA_ERR_PLAN_MISMATCH;
    cudaError_t e = cudaStreamSynchronize(plan->stream);
    if (e == cudaSuccess && key_block_host)
        e = cudaMemcpy(key_block_host, d->d_u_blk, sizeof(int32_t) * d->NB, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && query_chunk_host)
        e = cudaMemcpy(query_chunk_host, d->d_u_chunk, sizeof(int32_t) * d->NB, cudaMemcpyDeviceToHost);
    if (chunk_tokens_host) *chunk_tokens_host = d->chunk;
    return e == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_plan_destroy(libra_plan_t* plan) {
    if (!plan) return LIBRA_OK;
    cudaDeviceSynchronize();
    free_dir(plan->dir[0]);
    free_dir(plan->dir[1]);
    free_dir(plan->dir[2]);
    cudaFree(plan->d_tok_start);
    cudaFree(plan->d_tok_end);
    cudaFree(plan->d_status);
    for (int a = 0; a < libra_plan::kTimedKernels; ++a)
        for (int r = 0; r < libra_plan::kTimeRing; ++r)
            for (int b = 0; b < 2; ++b)
                if (plan->ev[a][r][b]) cudaEventDestroy(plan->ev[a][r][b]);
    delete plan;
    return LIBRA_OK;
}

extern "C" int libra_busy_times(const libra_plan_t* plan, int which, uint64_t* ns_host) {
    if (!plan || !ns_host) return LIBRA_ERR_INVALID_ARG;
    if ((which < LIBRA_KERNEL_FWD || which > LIBRA_KERNEL_BWD_DQ) && which != LIBRA_KERNEL_BWD_FUSED) return LIBRA_ERR_INVALID_ARG;
    // the forward and the dQ kernel walk the query-major lists, the dK/dV kernel the key-major ones, the fused
    // backward the pair tiles
    PlanDir* d = dir_of(plan, which == LIBRA_KERNEL_BWD_FUSED ? LIBRA_DIR_PAIR
                                                              : (which == LIBRA_KERNEL_BWD_DKDV ? LIBRA_DIR_KV : LIBRA_DIR_Q));
    if (!d) return LIBRA_ERR_PLAN_MISMATCH;
    if (cudaDeviceSynchronize() != cudaSuccess) return LIBRA_ERR_CUDA;
    uint64_t* tmp = new (std::nothrow) uint64_t[2 * (size_t)d->W];
    if (!tmp) return LIBRA_ERR_CUDA;
    int st[4] = {0, 0, 0, 0};
    const uint64_t* src = which == LIBRA_KERNEL_BWD_DQ ? d->d_busy2 : d->d_busy;
    cudaError_t e = cudaMemcpy(tmp, src, sizeof(uint64_t) * 2 * d->W, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess) e = cudaMemcpy(st, plan->d_status, sizeof(st), cudaMemcpyDeviceToHost);
    for (int r = 0; r < d->W; ++r) ns_host[r] = tmp[2 * r + 1] >= tmp[2 * r] ? tmp[2 * r + 1] - tmp[2 * r] : 0;
    delete[] tmp;
    if (e != cudaSuccess) return LIBRA_ERR_CUDA;
    return st[which == LIBRA_KERNEL_FWD ? 1 : 2];
}

extern "C" int libra_tile_times(const libra_plan_t* plan, int which, uint32_t* ns_host) {
    if (!plan || !ns_host) return LIBRA_ERR_INVALID_ARG;
    if (which != LIBRA_KERNEL_FWD && which != LIBRA_KERNEL_BWD_FUSED) return LIBRA_ERR_INVALID_ARG;
    PlanDir* d = dir_of(plan, which == LIBRA_KERNEL_BWD_FUSED ? LIBRA_DIR_PAIR : LIBRA_DIR_Q);
    if (!d) return LIBRA_ERR_PLAN_MISMATCH;
    if (cudaDeviceSynchronize() != cudaSuccess) return LIBRA_ERR_CUDA;
    return cudaMemcpy(ns_host, d->d_tile_ns, sizeof(uint32_t) * d->NT, cudaMemcpyDeviceToHost) == cudaSuccess
               ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_plan_set_timing(libra_plan_t* plan, int enabled) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    if (enabled) {
        for (int a = 0; a < libra_plan::kTimedKernels; ++a)
            for (int r = 0; r < libra_plan::kTimeRing; ++r)
                for (int b = 0; b < 2; ++b)
                    if (!plan->ev[a][r][b] && cudaEventCreate(&plan->ev[a][r][b]) != cudaSuccess) return LIBRA_ERR_CUDA;
        for (int a = 0; a < libra_plan::kTimedKernels; ++a) plan->ev_count[a] = 0;   // a fresh record
    }
    plan->timing = enabled ? 1 : 0;
    return LIBRA_OK;
}

extern "C" int libra_plan_set_wait_limit_ns(libra_plan_t* plan, uint64_t ns) {
    if (!plan || ns > 4000000000ull) return LIBRA_ERR_INVALID_ARG;
    plan->wait_limit_ns = ns ? (uint32_t)ns : 2000000000u;
    return LIBRA_OK;
}

extern "C" int libra_plan_inject_stall(libra_plan_t* plan, int enabled) {
    if (!plan) return LIBRA_ERR_INVALID_ARG;
    plan->inject_stall = enabled ? 1 : 0;
    return LIBRA_OK;
}

static int kernel_time(const libra_plan_t* plan, int a, int64_t launch, float* ms) {
    cudaEvent_t e0 = plan->ev[a][launch % libra_plan::kTimeRing][0], e1 = plan->ev[a][launch % libra_plan::kTimeRing][1];
    if (cudaEventSynchronize(e1) != cudaSuccess) return LIBRA_ERR_CUDA;
    return cudaEventElapsedTime(ms, e0, e1) == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_kernel_time_ms(const libra_plan_t* plan, int which, float* ms_host) {
    if (!plan || !ms_host) return LIBRA_ERR_INVALID_ARG;
    const int a = which - 1;  // LIBRA_KERNEL_FWD / _BWD_DKDV / _BWD_DQ / _BWD_PREP
    if (a < 0 || a >= libra_plan::kTimedKernels) return LIBRA_ERR_INVALID_ARG;
    if (plan->ev_count[a] == 0) return LIBRA_ERR_PLAN_MISMATCH;
    return kernel_time(plan, a, plan->ev_count[a] - 1, ms_host);
}

extern "C" int libra_kernel_times_ms(const libra_plan_t* plan, int which, float* ms_host, int capacity, int* n_out) {
    if (!plan || !ms_host || !n_out || capacity < 0) return LIBRA_ERR_INVALID_ARG;
    const int a = which - 1;
    if (a < 0 || a >= libra_plan::kTimedKernels) return LIBRA_ERR_INVALID_ARG;
    int64_t n = plan->ev_count[a] < libra_plan::kTimeRing ? plan->ev_count[a] : libra_plan::kTimeRing;
    if (n > capacity) n = capacity;
    for (int64_t i = 0; i < n; ++i) {   // oldest first
        const int rc = kernel_time(plan, a, plan->ev_count[a] - n + i, ms_host + i);
        if (rc != LIBRA_OK) return rc;
    }
    *n_out = (int)n;
    return LIBRA_OK;
}

extern "C" int64_t libra_launch_count(void) { return g_launches.load(); }

extern "C" const char* libra_strerror(int code) {
    switch (code) {
        case LIBRA_OK: return "ok";
        case LIBRA_ERR_INVALID_ARG: return "invalid argument";
        case LIBRA_ERR_UNSUPPORTED: return "unsupported configuration";
        case LIBRA_ERR_PLAN_MISMATCH: return "plan does not match the call";
        case LIBRA_ERR_CUDA: return "CUDA call failed";
        case LIBRA_ERR_OVERFLOW: return "integer overflow in plan sizes";
        case LIBRA_ERR_TIMEOUT: return "a bounded device-side wait timed out";
        case LIBRA_ERR_BAD_SEQLENS: return "cu_seqlens is malformed";
        case LIBRA_ERR_NO_DEVICE: return "no usable CUDA device";
        case LIBRA_ERR_SCRATCH_TOO_SMALL: return "problem exceeds the library's built-in scratch (use libra_attn_pool_bwd with a caller workspace)";
        default: return "unknown error";
    }
}
