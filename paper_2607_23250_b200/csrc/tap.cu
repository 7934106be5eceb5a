// Communication-aware SH-Tile placement for a sequence pool spread over several workers
// (Section 4.3: tiles and KV groups, Algorithm 2, exchange planning), as device kernels.
//
// The pool holds P packed sequences; sequence s belongs to the CP workers s*CP .. s*CP+CP-1, worker c of
// the group holding the c-th run of ceil(L_s / CP) consecutive tokens (the paper leaves this split open).
// A block's KV groups are the samples with a token in it, which is a contiguous range of sample indices,
// so K(t) is kept as (first sample, last sample, head shard) instead of a list; samples of length zero
// inside the range weigh nothing and change no decision.
//
// Placement is sequential by nature (every choice depends on the loads and residency left by the previous
// ones).  One CTA runs it with one thread per worker: each thread scores its own worker for the current
// tile, a block-wide lexicographic arg-min picks the destination, the winner updates its load and its
// residency bits.  The residency sets C_r are bit rows in global memory.
#include <cstdint>
#include <new>
#include <cuda_runtime.h>

#include "../../include/libra.h"
#include "common.h"

namespace libra {

struct TapGeom {
    const int32_t* cu;        // [n+1] sample offsets of the pool
    const int32_t* seq_off;   // [P+1] token offsets of the packed sequences
    const int32_t* blk_off;   // [P+1] first block of each sequence
    int n, P, CP, B, H, hq, hkv, d;
};

__device__ __forceinline__ int tap_seq_of_token(const TapGeom& g, int64_t tok) {
    int s = 0;
    while (s + 1 < g.P && g.seq_off[s + 1] <= tok) ++s;
    return s;
}
__device__ __forceinline__ int tap_owner(const TapGeom& g, int s, int64_t tok) {
    const int64_t len = g.seq_off[s + 1] - g.seq_off[s];
    const int64_t run = (len + g.CP - 1) / g.CP;
    return s * g.CP + (int)((tok - g.seq_off[s]) / (run > 0 ? run : 1));
}
// index of the sample that holds token tok (the last j with cu[j] <= tok; it is never empty)
__device__ __forceinline__ int tap_sample_of_token(const TapGeom& g, int64_t tok) {
    int lo = 0, hi = g.n;  // invariant: cu[lo] <= tok < cu[hi]
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (g.cu[mid] <= tok) lo = mid; else hi = mid;
    }
    return lo;
}

// Per block: work (Eq. 6 in closed form), Q-home, Q + output bytes, first and last sample.
__global__ void k_tap_blocks(TapGeom g, int64_t NB, int64_t* __restrict__ f_blk, int32_t* __restrict__ q_home,
                             int64_t* __restrict__ v_qo, int32_t* __restrict__ j_first, int32_t* __restrict__ j_last) {
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (b >= NB) return;
    int s = 0;
    while (s + 1 < g.P && g.blk_off[s + 1] <= b) ++s;
    const int64_t q0 = g.seq_off[s] + (b - g.blk_off[s]) * g.B;
    const int64_t q1 = q0 + g.B < g.seq_off[s + 1] ? q0 + g.B : g.seq_off[s + 1];
    const int j0 = tap_sample_of_token(g, q0), j1 = tap_sample_of_token(g, q1 - 1);
    int64_t w = 0;
    for (int j = j0; j <= j1; ++j) {
        const int64_t lo = q0 > g.cu[j] ? q0 : g.cu[j], hi = q1 < g.cu[j + 1] ? q1 : g.cu[j + 1];
        if (lo < hi) {
            const int64_t a = lo - g.cu[j], e = hi - g.cu[j];
            w += (e * (e + 1) - a * (a + 1)) / 2;
        }
    }
    f_blk[b] = w;
    q_home[b] = tap_owner(g, s, q0);
    v_qo[b] = 2 * ((q1 - q0) * (g.hq / g.H) * g.d * 2);
    j_first[b] = j0;
    j_last[b] = j1;
}

// Per sample: bytes of its K and V on one head shard, and the worker that holds all of it (or -1).
__global__ void k_tap_samples(TapGeom g, int64_t* __restrict__ v_smp, int32_t* __restrict__ res_smp) {
    const int j = blockIdx.x * blockDim.x + threadIdx.x;
    if (j >= g.n) return;
    const int64_t a = g.cu[j], e = g.cu[j + 1];
    const int kvps = g.H <= g.hkv ? g.hkv / g.H : 1;
    v_smp[j] = 2 * (e - a) * kvps * g.d * 2;
    int res = -1;
    if (e > a) {
        const int s = tap_seq_of_token(g, a);
        const int first = tap_owner(g, s, a), last = tap_owner(g, s, e - 1);
        res = first == last ? first : -1;
    }
    res_smp[j] = res;
}

__global__ void k_tap_rank(const int64_t* __restrict__ f_blk, int64_t NB, int32_t* __restrict__ blk_order) {
    __shared__ int64_t sw[256];
    const int64_t b = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t wb = b < NB ? f_blk[b] : 0;
    int64_t rank = 0;
    for (int64_t base = 0; base < NB; base += 256) {
        const int64_t o = base + threadIdx.x;
        sw[threadIdx.x] = o < NB ? f_blk[o] : -1;
        __syncthreads();
        const int lim = (int)((NB - base < 256) ? NB - base : 256);
        for (int i = 0; i < lim; ++i) rank += (sw[i] > wb) || (sw[i] == wb && base + i < b);
        __syncthreads();
    }
    if (b < NB) blk_order[rank] = (int32_t)b;
}

struct TapKey {
    int64_t a, b;
    int32_t r;   // -1: no candidate
};
__device__ __forceinline__ bool tap_less(const TapKey& x, const TapKey& y) {
    if (y.r < 0) return x.r >= 0;
    if (x.r < 0) return false;
    if (x.a != y.a) return x.a < y.a;
    if (x.b != y.b) return x.b < y.b;
    return x.r < y.r;
}
__device__ __forceinline__ TapKey tap_shfl_xor(const TapKey& k, int off) {
    TapKey o;
    o.a = __shfl_xor_sync(0xffffffffu, k.a, off);
    o.b = __shfl_xor_sync(0xffffffffu, k.b, off);
    o.r = __shfl_xor_sync(0xffffffffu, k.r, off);
    return o;
}

// Algorithm 2.  blockDim.x = W rounded up to a warp; thread r is worker r.
__global__ void __launch_bounds__(1024) k_tap_place(
    const int64_t* __restrict__ f_blk, const int32_t* __restrict__ blk_order, const int32_t* __restrict__ q_home,
    const int64_t* __restrict__ v_qo, const int32_t* __restrict__ j_first, const int32_t* __restrict__ j_last,
    const int64_t* __restrict__ v_smp, const int32_t* __restrict__ res_smp, int64_t NB, int H, int W, int n,
    int tau_num, int tau_den, uint32_t* __restrict__ Cbits /*[W][words]*/, int words, int32_t* __restrict__ sigma,
    int64_t* __restrict__ loads, int64_t* __restrict__ comm_total, int* __restrict__ status) {
    __shared__ TapKey sk_f[32], sk_w[32];
    __shared__ int64_t s_sum[32];
    __shared__ int s_pick;
    __shared__ int64_t s_pick_delta;
    const int r = threadIdx.x, lane = r & 31, warp = r >> 5, nwarps = blockDim.x >> 5;
    const bool live = r < W;
    // residency rows start with the groups the worker already holds in full
    if (live) {
        uint32_t* row = Cbits + (size_t)r * words;
        for (int w = 0; w < words; ++w) row[w] = 0;
        for (int j = 0; j < n; ++j)
            if (res_smp[j] == r)
                for (int h = 0; h < H; ++h) { const int g = j * H + h; row[g >> 5] |= 1u << (g & 31); }
    }
    // sum of f over all tiles
    int64_t part = 0;
    for (int64_t b = r; b < NB; b += blockDim.x) part += f_blk[b] * H;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) part += __shfl_xor_sync(0xffffffffu, part, off);
    if (lane == 0) s_sum[warp] = part;
    __syncthreads();
    int64_t sum_f = 0;
    for (int w = 0; w < nwarps; ++w) sum_f += s_sum[w];
    if (sum_f > (INT64_MAX / ((int64_t)(tau_den + tau_num) * 2)) / W) {  // the integer cap test would overflow
        if (r == 0) *status = LIBRA_ERR_OVERFLOW;   // the exchange kernels see the flag and add nothing
        for (int64_t t = r; t < NB * H; t += blockDim.x) sigma[t] = q_home[t / H];   // defined output: every tile stays home
        return;
    }
    const int64_t cap_rhs = (int64_t)(tau_den + tau_num) * sum_f;
    int64_t L = 0, comm = 0;
    uint32_t* my_row = Cbits + (size_t)(live ? r : 0) * words;
    const int64_t NT = NB * H;
    for (int64_t x = 0; x < NT; ++x) {
        const int32_t blk = blk_order[x / H];
        const int h = (int)(x % H);
        const int64_t f = f_blk[blk];
        const int j0 = j_first[blk], j1 = j_last[blk];
        TapKey kf, kw;
        kf.r = kw.r = -1; kf.a = kf.b = kw.a = kw.b = 0;
        int64_t delta = 0;
        if (live) {
            delta = r != q_home[blk] ? v_qo[blk] : 0;
            for (int j = j0; j <= j1; ++j) {
                const int g = j * H + h;
                if (!((my_row[g >> 5] >> (g & 31)) & 1u)) delta += v_smp[j];
            }
            if ((int64_t)tau_den * W * (L + f) <= cap_rhs) { kf.a = delta; kf.b = L; kf.r = r; }
            kw.a = L; kw.b = delta; kw.r = r;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const TapKey of = tap_shfl_xor(kf, off), ow = tap_shfl_xor(kw, off);
            if (tap_less(of, kf)) kf = of;
            if (tap_less(ow, kw)) kw = ow;
        }
        if (lane == 0) { sk_f[warp] = kf; sk_w[warp] = kw; }
        __syncthreads();
        if (r == 0) {
            TapKey bf = sk_f[0], bw = sk_w[0];
            for (int w = 1; w < nwarps; ++w) {
                if (tap_less(sk_f[w], bf)) bf = sk_f[w];
                if (tap_less(sk_w[w], bw)) bw = sk_w[w];
            }
            if (bf.r >= 0) { s_pick = bf.r; s_pick_delta = bf.a; }   // some worker stays under the soft cap
            else           { s_pick = bw.r; s_pick_delta = bw.b; }   // nobody does: least loaded
            sigma[(int64_t)blk * H + h] = s_pick;
        }
        __syncthreads();
        if (r == s_pick) {
            L += f;
            for (int j = j0; j <= j1; ++j) { const int g = j * H + h; my_row[g >> 5] |= 1u << (g & 31); }
        }
        if (r == 0) comm += s_pick_delta;
        // the next iteration's first barrier orders these reads of s_pick before its rewrite
    }
    if (live) loads[r] = L;
    if (r == 0) *comm_total = comm;
}

// Forward / backward send-byte matrices [src][dst].
__global__ void k_tap_exchange_qo(const int32_t* __restrict__ sigma, const int32_t* __restrict__ q_home,
                                  const int64_t* __restrict__ v_qo, int64_t NT, int H, int W,
                                  const int* __restrict__ status, unsigned long long* __restrict__ fwd,
                                  unsigned long long* __restrict__ bwd) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= NT || *status != 0) return;   // a placement that gave up left sigma unwritten
    const int q = q_home[t / H], r = sigma[t];
    if (q == r || r < 0 || r >= W || q < 0 || q >= W) return;
    const unsigned long long v = (unsigned long long)(v_qo[t / H] / 2);
    atomicAdd(&fwd[(size_t)q * W + r], v);   // Q out
    atomicAdd(&fwd[(size_t)r * W + q], v);   // output back
    atomicAdd(&bwd[(size_t)q * W + r], v);   // dO along the Q path
    atomicAdd(&bwd[(size_t)r * W + q], v);   // dQ along the output path
}
__global__ void k_tap_exchange_kv(TapGeom g, const uint32_t* __restrict__ Cbits, int words,
                                  const int32_t* __restrict__ res_smp, int W, const int* __restrict__ status,
                                  unsigned long long* __restrict__ fwd, unsigned long long* __restrict__ bwd) {
    const int64_t idx = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t NG = (int64_t)g.n * g.H;
    if (idx >= NG * W || *status != 0) return;
    const int r = (int)(idx / NG);
    const int grp = (int)(idx % NG), j = grp / g.H;
    if (!((Cbits[(size_t)r * words + (grp >> 5)] >> (grp & 31)) & 1u) || res_smp[j] == r) return;
    const int64_t a = g.cu[j], e = g.cu[j + 1];
    if (e <= a) return;
    const int kvps = g.H <= g.hkv ? g.hkv / g.H : 1;
    const int s = tap_seq_of_token(g, a);
    const int64_t len = g.seq_off[s + 1] - g.seq_off[s];
    const int64_t run = (len + g.CP - 1) / g.CP;
    for (int w = tap_owner(g, s, a); w <= tap_owner(g, s, e - 1); ++w) {   // the sample's token runs, owner by owner
        if (w == r) continue;
        const int64_t w0 = g.seq_off[s] + (int64_t)(w - s * g.CP) * run, w1 = w0 + run;
        const int64_t lo = a > w0 ? a : w0, hi = e < w1 ? e : w1;
        const unsigned long long bytes = (unsigned long long)((hi - lo) * 2 * kvps * g.d * 2);
        atomicAdd(&fwd[(size_t)w * W + r], bytes);
        atomicAdd(&bwd[(size_t)r * W + w], bytes);
    }
}


// ---- exchange schedule (Section 4.3.3): the transfer records implied by an assignment ----------------------
// Record = 6 x int32 (kind, src, dst, tok0, ntok, shard); kind 0: Q rows of a tile placed away from its Q-home
// (output back the same way, dO / dQ in the backward pass), kind 1: the K / V rows of a selected KV group held by
// another worker (dK / dV back the same way).  Order: kind 0 by tile id, then kind 1 by (dst, sample, shard, src).

// The KV groups some tile placed at r refers to, as bit rows [W][words].
__global__ void k_tap_mark(const int32_t* __restrict__ sigma, const int32_t* __restrict__ j_first,
                           const int32_t* __restrict__ j_last, int64_t NT, int H, int W, int words,
                           uint32_t* __restrict__ marks) {
    const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (t >= NT) return;
    const int r = sigma[t], h = (int)(t % H);
    if (r < 0 || r >= W) return;
    for (int j = j_first[t / H]; j <= j_last[t / H]; ++j) {
        const int g = j * H + h;
        atomicOr(&marks[(size_t)r * words + (g >> 5)], 1u << (g & 31));
    }
}

// Records slot x of the enumeration produces: slot x < NT is tile x (0 or 1), slot NT + r * NG + g is group g
// at destination r (one per token run of the sample on another worker).
__device__ __forceinline__ int tap_slot_count(const TapGeom& g, int64_t x, int64_t NT, int64_t NG, int W,
                                              const int32_t* sigma, const int32_t* q_home, const uint32_t* marks,
                                              int words, const int32_t* res_smp) {
    if (x < NT) {
        const int r = sigma[x];
        return (r >= 0 && r < W && r != q_home[x / g.H]) ? 1 : 0;
    }
    const int64_t y = x - NT;
    const int r = (int)(y / NG);
    const int grp = (int)(y % NG), j = grp / g.H;
    if (!((marks[(size_t)r * words + (grp >> 5)] >> (grp & 31)) & 1u) || res_smp[j] == r) return 0;
    const int64_t a = g.cu[j], e = g.cu[j + 1];
    if (e <= a) return 0;
    const int s = tap_seq_of_token(g, a);
    int c = 0;
    for (int w = tap_owner(g, s, a); w <= tap_owner(g, s, e - 1); ++w) c += (w != r);
    return c;
}

// One block: exclusive prefix sum of the slot counts (each thread takes a contiguous piece), total to n_out.
__global__ void __launch_bounds__(1024) k_tap_sched_scan(TapGeom g, int64_t NT, int64_t NG, int W,
                                                         const int32_t* __restrict__ sigma,
                                                         const int32_t* __restrict__ q_home,
                                                         const uint32_t* __restrict__ marks, int words,
                                                         const int32_t* __restrict__ res_smp,
                                                         int64_t* __restrict__ offs /*[slots]*/, int64_t* n_out) {
    __shared__ int64_t part[1024];
    const int64_t slots = NT + NG * W;
    const int64_t per = (slots + blockDim.x - 1) / blockDim.x;
    const int64_t x0 = threadIdx.x * per, x1 = x0 + per < slots ? x0 + per : slots;
    int64_t sum = 0;
    for (int64_t x = x0; x < x1; ++x) sum += tap_slot_count(g, x, NT, NG, W, sigma, q_home, marks, words, res_smp);
    part[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        int64_t run = 0;
        for (int i = 0; i < (int)blockDim.x; ++i) { const int64_t v = part[i]; part[i] = run; run += v; }
        *n_out = run;
    }
    __syncthreads();
    int64_t run = part[threadIdx.x];
    for (int64_t x = x0; x < x1; ++x) {
        offs[x] = run;
        run += tap_slot_count(g, x, NT, NG, W, sigma, q_home, marks, words, res_smp);
    }
}

__global__ void k_tap_sched_fill(TapGeom g, int64_t NT, int64_t NG, int W, const int32_t* __restrict__ sigma,
                                 const int32_t* __restrict__ q_home, const uint32_t* __restrict__ marks, int words,
                                 const int32_t* __restrict__ res_smp, const int64_t* __restrict__ offs,
                                 int64_t capacity, int32_t* __restrict__ rec) {
    const int64_t x = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (x >= NT + NG * W) return;
    int64_t at = offs[x];
    if (x < NT) {
        const int r = sigma[x];
        const int64_t b = x / g.H;
        if (!(r >= 0 && r < W && r != q_home[b]) || at >= capacity) return;
        int s = 0;
        while (s + 1 < g.P && g.blk_off[s + 1] <= b) ++s;
        const int64_t q0 = g.seq_off[s] + (b - g.blk_off[s]) * g.B;
        const int64_t q1 = q0 + g.B < g.seq_off[s + 1] ? q0 + g.B : g.seq_off[s + 1];
        int32_t* o = rec + at * 6;
        o[0] = 0; o[1] = q_home[b]; o[2] = r; o[3] = (int32_t)q0; o[4] = (int32_t)(q1 - q0); o[5] = (int32_t)(x % g.H);
        return;
    }
    const int64_t y = x - NT;
    const int r = (int)(y / NG);
    const int grp = (int)(y % NG), j = grp / g.H;
    if (!((marks[(size_t)r * words + (grp >> 5)] >> (grp & 31)) & 1u) || res_smp[j] == r) return;
    const int64_t a = g.cu[j], e = g.cu[j + 1];
    if (e <= a) return;
    const int s = tap_seq_of_token(g, a);
    const int64_t len = g.seq_off[s + 1] - g.seq_off[s];
    const int64_t run = (len + g.CP - 1) / g.CP;
    for (int w = tap_owner(g, s, a); w <= tap_owner(g, s, e - 1); ++w) {
        if (w == r) continue;
        if (at >= capacity) return;
        const int64_t w0 = g.seq_off[s] + (int64_t)(w - s * g.CP) * run, w1 = w0 + run;
        const int64_t lo = a > w0 ? a : w0, hi = e < w1 ? e : w1;
        int32_t* o = rec + at * 6;
        o[0] = 1; o[1] = w; o[2] = r; o[3] = (int32_t)lo; o[4] = (int32_t)(hi - lo); o[5] = grp % g.H;
        ++at;
    }
}

}  // namespace libra

using namespace libra;

extern "C" int64_t libra_tap_num_tiles(const int32_t* seq_offsets_host, int n_sequences, int block, int n_shards) {
    if (!seq_offsets_host || n_sequences <= 0 || block <= 0 || n_shards <= 0) return LIBRA_ERR_INVALID_ARG;
    int64_t nb = 0;
    for (int s = 0; s < n_sequences; ++s) {
        if (seq_offsets_host[s + 1] < seq_offsets_host[s]) return LIBRA_ERR_INVALID_ARG;
        nb += ((int64_t)seq_offsets_host[s + 1] - seq_offsets_host[s] + block - 1) / block;
    }
    return nb * n_shards;
}

extern "C" int libra_tap_plan(const int32_t* cu_seqlens_dev, int n_samples, const int32_t* seq_offsets_host,
                              int n_sequences, const libra_tap_opts* o, int32_t* sigma_dev, int64_t* loads_dev,
                              int64_t* fwd_bytes_dev, int64_t* bwd_bytes_dev, int64_t* comm_total_dev,
                              int* status_dev, void* stream) {
    if (!cu_seqlens_dev || !seq_offsets_host || !o || !sigma_dev || !loads_dev || !fwd_bytes_dev || !bwd_bytes_dev ||
        !comm_total_dev || !status_dev)
        return LIBRA_ERR_INVALID_ARG;
    if (n_samples <= 0 || n_sequences <= 0 || o->cp <= 0 || o->block <= 0 || o->n_shards <= 0 || o->hq <= 0 ||
        o->hkv <= 0 || o->head_dim <= 0 || o->tau_num < 0 || o->tau_den <= 0 || o->hq % o->n_shards != 0)
        return LIBRA_ERR_INVALID_ARG;
    if (!((o->n_shards <= o->hkv && o->hkv % o->n_shards == 0) || (o->n_shards > o->hkv && o->n_shards % o->hkv == 0)))
        return LIBRA_ERR_INVALID_ARG;
    const int P = n_sequences, W = P * o->cp, H = o->n_shards;
    if (W > 1024 || P > 4096) return LIBRA_ERR_UNSUPPORTED;
    const int64_t NT = libra_tap_num_tiles(seq_offsets_host, P, o->block, H);
    if (NT <= 0) return LIBRA_ERR_INVALID_ARG;
    const int64_t NB = NT / H;
    if (NT >= INT32_MAX || NB > 65536) return LIBRA_ERR_UNSUPPORTED;  // the rank sort is quadratic in blocks
    {   // the work total (at most H * T (T + 1) / 2) must itself fit 64 bits before the device can test the cap
        const long double Tl = (long double)seq_offsets_host[P] - (long double)seq_offsets_host[0];
        if ((long double)H * Tl * (Tl + 1) / 2 > 4.0e18L) return LIBRA_ERR_OVERFLOW;
    }
    cudaStream_t s = (cudaStream_t)stream;
    const int words = (int)(((int64_t)n_samples * H + 31) / 32);

    // small host tables -> device (stream-ordered scratch; nothing outlives the call's work on `stream`)
    int32_t* h_tab = new (std::nothrow) int32_t[2 * (P + 1)];
    if (!h_tab) return LIBRA_ERR_CUDA;
    int64_t nb = 0;
    for (int q = 0; q <= P; ++q) {
        h_tab[q] = seq_offsets_host[q];
        h_tab[P + 1 + q] = (int32_t)nb;
        if (q < P) nb += ((int64_t)seq_offsets_host[q + 1] - seq_offsets_host[q] + o->block - 1) / o->block;
    }
    uint8_t* scratch = nullptr;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off += (bytes + 255) & ~size_t(255); return at; };
    const size_t o_tab = take(sizeof(int32_t) * 2 * (P + 1));
    const size_t o_f = take(sizeof(int64_t) * NB), o_vqo = take(sizeof(int64_t) * NB);
    const size_t o_q = take(sizeof(int32_t) * NB), o_j0 = take(sizeof(int32_t) * NB), o_j1 = take(sizeof(int32_t) * NB);
    const size_t o_ord = take(sizeof(int32_t) * NB);
    const size_t o_vs = take(sizeof(int64_t) * n_samples), o_rs = take(sizeof(int32_t) * n_samples);
    const size_t o_c = take(sizeof(uint32_t) * (size_t)words * W);
    if (cudaMallocAsync((void**)&scratch, off, s) != cudaSuccess) { delete[] h_tab; return LIBRA_ERR_CUDA; }
    int rc = LIBRA_OK;
    // the table is copied from pageable memory, so the copy has left h_tab when the call returns
    if (cudaMemcpyAsync(scratch + o_tab, h_tab, sizeof(int32_t) * 2 * (P + 1), cudaMemcpyHostToDevice, s) != cudaSuccess)
        rc = LIBRA_ERR_CUDA;
    delete[] h_tab;
    TapGeom g;
    g.cu = cu_seqlens_dev;
    g.seq_off = (const int32_t*)(scratch + o_tab);
    g.blk_off = g.seq_off + (P + 1);
    g.n = n_samples; g.P = P; g.CP = o->cp; g.B = o->block; g.H = H; g.hq = o->hq; g.hkv = o->hkv; g.d = o->head_dim;
    int64_t* f_blk = (int64_t*)(scratch + o_f);
    int64_t* v_qo = (int64_t*)(scratch + o_vqo);
    int32_t* q_home = (int32_t*)(scratch + o_q);
    int32_t* j0 = (int32_t*)(scratch + o_j0);
    int32_t* j1 = (int32_t*)(scratch + o_j1);
    int32_t* ord = (int32_t*)(scratch + o_ord);
    int64_t* v_smp = (int64_t*)(scratch + o_vs);
    int32_t* res_smp = (int32_t*)(scratch + o_rs);
    uint32_t* cbits = (uint32_t*)(scratch + o_c);
    if (rc == LIBRA_OK) {
        cudaMemsetAsync(status_dev, 0, sizeof(int), s);
        cudaMemsetAsync(fwd_bytes_dev, 0, sizeof(int64_t) * W * W, s);
        cudaMemsetAsync(bwd_bytes_dev, 0, sizeof(int64_t) * W * W, s);
        cudaMemsetAsync(comm_total_dev, 0, sizeof(int64_t), s);
        cudaMemsetAsync(loads_dev, 0, sizeof(int64_t) * W, s);
        k_tap_blocks<<<(unsigned)((NB + 127) / 128), 128, 0, s>>>(g, NB, f_blk, q_home, v_qo, j0, j1);
        k_tap_samples<<<(n_samples + 127) / 128, 128, 0, s>>>(g, v_smp, res_smp);
        k_tap_rank<<<(unsigned)((NB + 255) / 256), 256, 0, s>>>(f_blk, NB, ord);
        k_tap_place<<<1, ((W + 31) / 32) * 32, 0, s>>>(f_blk, ord, q_home, v_qo, j0, j1, v_smp, res_smp, NB, H, W,
                                                        n_samples, o->tau_num, o->tau_den, cbits, words, sigma_dev,
                                                        loads_dev, comm_total_dev, status_dev);
        k_tap_exchange_qo<<<(unsigned)((NT + 255) / 256), 256, 0, s>>>(sigma_dev, q_home, v_qo, NT, H, W, status_dev,
                                                                       (unsigned long long*)fwd_bytes_dev,
                                                                       (unsigned long long*)bwd_bytes_dev);
        const int64_t pairs = (int64_t)n_samples * H * W;
        k_tap_exchange_kv<<<(unsigned)((pairs + 255) / 256), 256, 0, s>>>(g, cbits, words, res_smp, W, status_dev,
                                                                          (unsigned long long*)fwd_bytes_dev,
                                                                          (unsigned long long*)bwd_bytes_dev);
        count_launch(6);
        if (cudaGetLastError() != cudaSuccess) rc = LIBRA_ERR_CUDA;
    }
    cudaFreeAsync(scratch, s);
    return rc;
}

extern "C" int libra_tap_schedule(const int32_t* cu_seqlens_dev, int n_samples, const int32_t* seq_offsets_host,
                                  int n_sequences, const libra_tap_opts* o, const int32_t* sigma_dev,
                                  int32_t* records_dev, int64_t capacity, int64_t* n_records_dev, void* stream) {
    if (!cu_seqlens_dev || !seq_offsets_host || !o || !sigma_dev || !records_dev || !n_records_dev || capacity < 0)
        return LIBRA_ERR_INVALID_ARG;
    if (n_samples <= 0 || n_sequences <= 0 || o->cp <= 0 || o->block <= 0 || o->n_shards <= 0 || o->hq <= 0 ||
        o->hkv <= 0 || o->head_dim <= 0 || o->hq % o->n_shards != 0)
        return LIBRA_ERR_INVALID_ARG;
    const int P = n_sequences, W = P * o->cp, H = o->n_shards;
    if (W > 1024 || P > 4096) return LIBRA_ERR_UNSUPPORTED;
    const int64_t NT = libra_tap_num_tiles(seq_offsets_host, P, o->block, H);
    if (NT <= 0) return LIBRA_ERR_INVALID_ARG;
    const int64_t NB = NT / H, NG = (int64_t)n_samples * H;
    if (NT >= INT32_MAX || NG * W >= INT32_MAX) return LIBRA_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    const int words = (int)((NG + 31) / 32);
    int32_t* h_tab = new (std::nothrow) int32_t[2 * (P + 1)];
    if (!h_tab) return LIBRA_ERR_CUDA;
    int64_t nb = 0;
    for (int q = 0; q <= P; ++q) {
        h_tab[q] = seq_offsets_host[q];
        h_tab[P + 1 + q] = (int32_t)nb;
        if (q < P) nb += ((int64_t)seq_offsets_host[q + 1] - seq_offsets_host[q] + o->block - 1) / o->block;
    }
    uint8_t* scratch = nullptr;
    size_t off = 0;
    auto take = [&](size_t bytes) { const size_t at = off; off += (bytes + 255) & ~size_t(255); return at; };
    const size_t o_tab = take(sizeof(int32_t) * 2 * (P + 1));
    const size_t o_f = take(sizeof(int64_t) * NB), o_vqo = take(sizeof(int64_t) * NB);
    const size_t o_q = take(sizeof(int32_t) * NB), o_j0 = take(sizeof(int32_t) * NB), o_j1 = take(sizeof(int32_t) * NB);
    const size_t o_vs = take(sizeof(int64_t) * n_samples), o_rs = take(sizeof(int32_t) * n_samples);
    const size_t o_m = take(sizeof(uint32_t) * (size_t)words * W);
    const size_t o_offs = take(sizeof(int64_t) * (size_t)(NT + NG * W));
    if (cudaMallocAsync((void**)&scratch, off, s) != cudaSuccess) { delete[] h_tab; return LIBRA_ERR_CUDA; }
    int rc = LIBRA_OK;
    if (cudaMemcpyAsync(scratch + o_tab, h_tab, sizeof(int32_t) * 2 * (P + 1), cudaMemcpyHostToDevice, s) != cudaSuccess)
        rc = LIBRA_ERR_CUDA;
    delete[] h_tab;
    TapGeom g;
    g.cu = cu_seqlens_dev;
    g.seq_off = (const int32_t*)(scratch + o_tab);
    g.blk_off = g.seq_off + (P + 1);
    g.n = n_samples; g.P = P; g.CP = o->cp; g.B = o->block; g.H = H; g.hq = o->hq; g.hkv = o->hkv; g.d = o->head_dim;
    int32_t* q_home = (int32_t*)(scratch + o_q);
    int32_t* j0 = (int32_t*)(scratch + o_j0);
    int32_t* j1 = (int32_t*)(scratch + o_j1);
    int32_t* res_smp = (int32_t*)(scratch + o_rs);
    uint32_t* marks = (uint32_t*)(scratch + o_m);
    int64_t* offs = (int64_t*)(scratch + o_offs);
    if (rc == LIBRA_OK) {
        cudaMemsetAsync(marks, 0, sizeof(uint32_t) * (size_t)words * W, s);
        k_tap_blocks<<<(unsigned)((NB + 127) / 128), 128, 0, s>>>(g, NB, (int64_t*)(scratch + o_f), q_home,
                                                                  (int64_t*)(scratch + o_vqo), j0, j1);
        k_tap_samples<<<(n_samples + 127) / 128, 128, 0, s>>>(g, (int64_t*)(scratch + o_vs), res_smp);
        k_tap_mark<<<(unsigned)((NT + 255) / 256), 256, 0, s>>>(sigma_dev, j0, j1, NT, H, W, words, marks);
        k_tap_sched_scan<<<1, 1024, 0, s>>>(g, NT, NG, W, sigma_dev, q_home, marks, words, res_smp, offs, n_records_dev);
        const int64_t slots = NT + NG * W;
        k_tap_sched_fill<<<(unsigned)((slots + 255) / 256), 256, 0, s>>>(g, NT, NG, W, sigma_dev, q_home, marks, words,
                                                                        res_smp, offs, capacity, records_dev);
        count_launch(5);
        if (cudaGetLastError() != cudaSuccess) rc = LIBRA_ERR_CUDA;
    }
    cudaFreeAsync(scratch, s);
    return rc;
}
