// Pool attention at head_dim 256 (the micro-benchmark head shape Hq 128 / Hkv 4 / d 256 of the paper's Table 1).
//
// A 128 x 256 bf16 operand tile is 64 KB and an accumulator of 128 rows x 256 head-dim columns takes half of
// TMEM, so the 128-wide kernels do not stretch to this width.  One kernel template covers the four passes; every
// pass keeps one side of the score matrix stationary (128 rows: its operand tile(s) stay in shared memory, its
// accumulator in TMEM) and streams the other side in blocks of 64 rows (32 KB tiles):
//
//   FWD  queries stationary   S  = Q K^T          P = softmax (online, lazy rescale)      O  += P V
//   DV   keys stationary      S^T = K Q^T         P^T = exp2(S^T c - LSE)                 dV += P^T dO
//   DK   keys stationary      S^T, dP^T = V dO^T  dS^T = P^T o (dP^T - D)                 dK += dS^T Q
//   DQ   queries stationary   S, dP = dO V^T      dS = P o (dP - D)                       dQ += dS K
//
// dK and dV cannot share TMEM with S^T and dP^T at this width (2 x 256 accumulator columns), so the gradient takes
// three passes and recomputes S (eight GEMMs per cell for the five of the definition).
// TMEM: X1 (2 x 64, double-buffered) | X2 (64) | W (32: the bf16 result of the element-wise step, A operand of the
// last GEMM) | acc (256).
// Roles (320 threads): warps 0-7 compute, warp 8 one TMA thread, warp 9 one MMA thread.  In the gradient passes two
// threads share a stationary row (32 of the block's 64 columns each; warps w and w + 4 reach the same TMEM lanes); the
// forward keeps one thread per row, because the running maximum and sum of a row live in its registers (warps 4-7
// idle there).  Per streamed block: X1 (and X2) are issued, the compute warps turn them into W, the accumulating GEMM
// is issued; X1 of the next block is issued ahead, so it runs under the element-wise step of the current one.
// Tiles are prefetched through a ring of 32 KB slots.  Masks follow the sample bounds per element.
#include <math.h>

#include "common.h"
#include "ptx.cuh"

namespace libra {
namespace d256 {

constexpr int kThreads = 320;
constexpr int kTmaWarp = 8, kMmaWarp = 9;
constexpr int kRows = 128;       // stationary rows per unit
constexpr int kBlk = 64;         // streamed rows per block
constexpr int kD = 256;
constexpr uint32_t kColX1 = 0 /* and 64 */, kColX2 = 128, kColW = 192, kColAcc = 256;
constexpr uint64_t kDrainNs = 2000000;
constexpr int kSmemMax = 232448;
enum Mode { FWD = 0, DV = 1, DK = 2, DQ = 3 };

template <int MODE>
struct Cfg {
    static constexpr bool kKeyStationary = (MODE == DV || MODE == DK);
    static constexpr bool kHasX2 = (MODE == DK || MODE == DQ);
    static constexpr int kGroups = MODE == FWD ? 1 : 2;      // compute threads per stationary row
    static constexpr int kCols = 64 / kGroups;               // columns of a streamed block per compute thread
    static constexpr int kStationary = kHasX2 ? 2 : 1;       // resident 64 KB tiles
    static constexpr int kSlots = kHasX2 ? 3 : 4;            // ring of 32 KB tiles
    static constexpr int kBig = 65536, kBigHalf = 16384;     // 128 x 256 bf16: four column halves of 128 rows x 128 B
    static constexpr int kSmall = 32768, kSmallHalf = 8192;  // 64 x 256 bf16: four column halves of 64 rows x 128 B
    static constexpr int kStatBytes = MODE == DV ? 256 : (MODE == DK ? 512 : 0);   // per streamed block: lse2[64], dvec[64]
    static constexpr int kSaOff = 0;
    static constexpr int kSbOff = kBig;
    static constexpr int kRingOff = kStationary * kBig;
    static constexpr int kStatOff = kRingOff + kSlots * kSmall;
    static constexpr int kBarOff = kStatOff + kSlots * 512;
    // full[kSlots], empty[kSlots], st_full, st_empty, x1_full[2], x2_full, w_ready, acc_done, acc_free, drain, acc_step
    static constexpr int kNumBars = 2 * kSlots + 10;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static_assert(kBytes <= kSmemMax, "exceeds the shared memory of an sm_100 CTA");
    // Ring slots by stream and iteration i (counted over the whole kernel): the first streamed tile alternates
    // between slots 0 and 1; the second has slot 2 to itself when it only feeds X2 (it is free again as soon as X2 has
    // run, so its successor loads early), else it alternates between slots 2 and 3.
    __host__ __device__ static constexpr uint32_t slot1(uint32_t i) { return i & 1; }
    __host__ __device__ static constexpr uint32_t phase1(uint32_t i) { return (i >> 1) & 1; }
    __host__ __device__ static constexpr uint32_t slot2(uint32_t i) { return kHasX2 ? 2 : 2 + (i & 1); }
    __host__ __device__ static constexpr uint32_t phase2(uint32_t i) { return kHasX2 ? (i & 1) : ((i >> 1) & 1); }
};

struct Params {
    __nv_bfloat16* out;     // FWD: out [T, Hq, 256]; DV: dv, DK: dk [T, Hkv, 256]; DQ: dq [T, Hq, 256]
    float* lse;             // FWD: [Hq, T]
    const float* lse2;      // backward passes: [Hq, Tpad]  LSE * log2(e)
    const float* dvec;      // backward passes: [Hq, Tpad]  D_i
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* tok_start;
    const int32_t* tok_end;
    int64_t T, Tpad;
    int hq, hkv, H;         // H: head shards of the query-major lists (FWD, DQ)
    // key-stationary passes over pair tiles (key block x query chunk x kv head) instead of key-major tiles: the
    // accumulator of a unit is added to acc32 [T, Hkv, 256] (fp32) and rounded by a later kernel
    float* acc32;           // null: key-major tiles, results stored as bf16 by the pass itself
    const int32_t* u_blk;   // [NU] key block of pair-block u
    const int32_t* u_chunk; // [NU] query chunk of pair-block u
    int64_t NU;
    int R;                  // 128-row blocks per query chunk
    float scale, scale_log2;
    int* status;
    const int* plan_status;
    uint32_t wait_limit_ns;
    int inject_stall;
    uint64_t* busy;
};

// Walks the units of a CTA's tile list in the order every role uses.
//   key-stationary passes: one unit per key-major tile (128 keys x one kv head); its iterations are the query heads of
//   the group times the 64-row query blocks from the diagonal to the end of the last key's sample;
//   query-stationary passes: a query-major tile (256 rows x head shard) gives one unit per head and 128-row half; its
//   iterations are the 64-key blocks from the start of the first row's sample to the diagonal.
template <int MODE>
struct Units {
    const Params& p;
    int idx, end, hh, g, hps, G;
    int64_t r0;                  // first stationary row
    int h, kvh, b_lo, n_blk, n_it;
    __device__ Units(const Params& p_, int cta) : p(p_) {
        idx = p.cta_offsets[cta];
        end = p.cta_offsets[cta + 1];
        G = p.hq / p.hkv;
        hps = Cfg<MODE>::kKeyStationary ? 1 : p.hq / p.H;
        hh = 0;
        g = -1;
        if (Cfg<MODE>::kKeyStationary) --idx;
    }
    __device__ bool next() {
        if constexpr (Cfg<MODE>::kKeyStationary) {
            if (++idx >= end) return false;
            const int t = p.cta_tiles[idx];
            if (p.acc32) {   // pair tile: the query blocks of one chunk only
                const int pb = (int)(t % p.NU);
                kvh = (int)(t / p.NU);
                const int j = p.u_blk[pb], c = p.u_chunk[pb];
                r0 = (int64_t)j * kRows;
                const int64_t last_key = r0 + kRows - 1 < p.T ? r0 + kRows - 1 : p.T - 1;
                const int last64 = (p.tok_end[last_key] - 1) / kBlk;
                const int lo128 = c * p.R > j ? c * p.R : j;
                const int hi64 = 2 * (c * p.R + p.R - 1) + 1;
                b_lo = 2 * lo128;
                n_blk = (hi64 < last64 ? hi64 : last64) - b_lo + 1;
            } else {
                kvh = t % p.hkv;
                r0 = (int64_t)(t / p.hkv) * kRows;
                const int64_t last_key = r0 + kRows - 1 < p.T ? r0 + kRows - 1 : p.T - 1;
                b_lo = (int)(r0 / kBlk);
                n_blk = (p.tok_end[last_key] - 1) / kBlk - b_lo + 1;
            }
            h = kvh * G;
            n_it = G * n_blk;
            return true;
        } else {
        for (;;) {
            if (++g == 2) { g = 0; if (++hh == hps) { hh = 0; ++idx; } }
            if (idx >= end) return false;
            const int t = p.cta_tiles[idx];
            r0 = (int64_t)(t / p.H) * (2 * kRows) + g * kRows;
            if (r0 >= p.T) continue;   // the second half of the pool's last tile may lie past its end
            h = (t % p.H) * hps + hh;
            kvh = h / G;
            const int64_t last_row = r0 + kRows - 1 < p.T ? r0 + kRows - 1 : p.T - 1;
            b_lo = p.tok_start[r0] / kBlk;
            n_blk = (int)(last_row / kBlk) - b_lo + 1;
            n_it = n_blk;
            return true;
        }
        }
    }
    // head and first row of the streamed block of iteration it
    __device__ int stream_head(int it) const { return Cfg<MODE>::kKeyStationary ? h + it / n_blk : kvh; }
    __device__ int stream_row(int it) const { return (b_lo + (Cfg<MODE>::kKeyStationary ? it % n_blk : it)) * kBlk; }
};

template <int MODE>
__global__ void __launch_bounds__(kThreads, 1)
k_attn_d256(const __grid_constant__ CUtensorMap tm_sa, const __grid_constant__ CUtensorMap tm_sb,
            const __grid_constant__ CUtensorMap tm_t1, const __grid_constant__ CUtensorMap tm_t2, const Params p) {
    using L = Cfg<MODE>;
    constexpr int S = L::kSlots;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_full = bars;
    uint64_t* bar_empty = bars + S;
    uint64_t* b2 = bars + 2 * S;
    uint64_t* bar_stfull = b2 + 0;
    uint64_t* bar_stempty = b2 + 1;
    uint64_t* bar_x2full = b2 + 3;
    uint64_t* bar_wready = b2 + 4;
    uint64_t* bar_accdone = b2 + 5;
    uint64_t* bar_accfree = b2 + 6;
    uint64_t* bar_drain = b2 + 7;
    uint64_t* bar_accstep = b2 + 8;    // the accumulating GEMM of an iteration has run: W may be rewritten, acc rescaled
    uint64_t* bar_x1full = b2 + 9;     // [2] one per X1 buffer: X1 of the next block is committed a block ahead
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicExch(p.status, LIBRA_ERR_CUDA);
        return;
    }
    if (const int ps = *p.plan_status; ps != 0) {  // malformed cu_seqlens: report and leave
        if (threadIdx.x == 0) { atomicExch(p.status, ps); p.busy[2 * cta] = p.busy[2 * cta + 1] = 0; }
        return;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < S; ++s) { mbar_init(&bar_full[s], 1); mbar_init(&bar_empty[s], 1); }
        mbar_init(bar_stfull, 1);
        mbar_init(bar_stempty, 1);
        mbar_init(&bar_x1full[0], 1);
        mbar_init(&bar_x1full[1], 1);
        mbar_init(bar_x2full, 1);
        mbar_init(bar_wready, kRows * L::kGroups);
        mbar_init(bar_accdone, 1);
        mbar_init(bar_accfree, kRows * L::kGroups);
        mbar_init(bar_drain, 1);
        mbar_init(bar_accstep, 1);
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit_ns;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == kMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kTmaWarp && lane == 0) {
        prefetch_tmap(&tm_sa);
        if (L::kStationary == 2) prefetch_tmap(&tm_sb);
        prefetch_tmap(&tm_t1);
        prefetch_tmap(&tm_t2);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == kTmaWarp) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            Units<MODE> u(p, cta);
            uint32_t n = 0, uc = 0;          // n: iterations so far (over all units)
            uint32_t armed[S] = {};          // per slot: 1 + parity of the phase last armed (0: never)
            bool ok = true;
            while (ok && !p.inject_stall && u.next()) {
                ok = mbar_wait(bar_stempty, (uc & 1) ^ 1, abort_flag);
                if (!ok) break;
                mbar_arrive_expect_tx(bar_stfull, L::kStationary * L::kBig);
                const int st_head = L::kKeyStationary ? u.kvh : u.h;
                for (int half = 0; half < 4; ++half) {
                    tma_load_3d(smem + L::kSaOff + half * L::kBigHalf, &tm_sa, bar_stfull, half * 64, st_head, (int)u.r0);
                    if (L::kStationary == 2)
                        tma_load_3d(smem + L::kSbOff + half * L::kBigHalf, &tm_sb, bar_stfull, half * 64, st_head, (int)u.r0);
                }
                ++uc;
                for (int it = 0; it < u.n_it && ok; ++it, ++n) {
                    const int sh = u.stream_head(it), row = u.stream_row(it);
                    for (int which = 0; which < 2 && ok; ++which) {
                        const uint32_t s = which == 0 ? L::slot1(n) : L::slot2(n);
                        const uint32_t ph = which == 0 ? L::phase1(n) : L::phase2(n);
                        ok = mbar_wait(&bar_empty[s], ph ^ 1, abort_flag);
                        if (!ok) break;
                        mbar_arrive_expect_tx(&bar_full[s], L::kSmall + (which == 0 ? L::kStatBytes : 0));
                        armed[s] = 1 + ph;
                        for (int half = 0; half < 4; ++half)
                            tma_load_3d(smem + L::kRingOff + s * L::kSmall + half * L::kSmallHalf, which == 0 ? &tm_t1 : &tm_t2,
                                        &bar_full[s], half * 64, sh, row);
                        if (which == 0 && L::kStatBytes >= 256)
                            bulk_load_1d(smem + L::kStatOff + s * 512, p.lse2 + (size_t)sh * p.Tpad + row, 256, &bar_full[s]);
                        if (which == 0 && L::kStatBytes == 512)
                            bulk_load_1d(smem + L::kStatOff + s * 512 + 256, p.dvec + (size_t)sh * p.Tpad + row, 256, &bar_full[s]);
                    }
                }
            }
            if (!ok || abort_flag[0]) {   // give-up path: the copies already issued land before shared memory is released
                if (uc > 0) mbar_wait_drain(bar_stfull, (uc - 1) & 1, kDrainNs);
                for (int b = 0; b < S; ++b)
                    if (armed[b]) mbar_wait_drain(&bar_full[b], armed[b] - 1, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            constexpr uint32_t idesc_x = make_idesc(kRows, kBlk, 0, 0);    // X = stationary x streamed^T, both K-major
            constexpr uint32_t idesc_acc = make_idesc(kRows, kD, 0, 1);    // acc += W (TMEM) x streamed tile, MN-major
            const uint32_t sb = smem_u32(smem);
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);              // K-major view at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kSmallHalf, 1024);   // MN-major view of a 64-row tile
            auto issue_x = [&](uint32_t d_col, uint32_t a_off, uint32_t b_off) {
                const uint64_t da = sdesc_advance(kdesc0, a_off), db = sdesc_advance(kdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < kD / 16; ++kk)
                    mma_ss(tmem_base + d_col, sdesc_advance(da, (kk / 4) * L::kBigHalf + (kk % 4) * 32),
                           sdesc_advance(db, (kk / 4) * L::kSmallHalf + (kk % 4) * 32), idesc_x, kk > 0);
            };
            Units<MODE> u(p, cta);
            uint32_t uc = 0, itc = 0;
            bool ok = true;
            while (ok && u.next()) {
                ok = mbar_wait(bar_stfull, uc & 1, abort_flag);
                if (ok) ok = mbar_wait(&bar_full[L::slot1(itc)], L::phase1(itc), abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_x(kColX1 + (itc & 1) * 64, L::kSaOff, L::kRingOff + L::slot1(itc) * L::kSmall);
                tc_commit(&bar_x1full[itc & 1]);
                for (int it = 0; it < u.n_it && ok; ++it, ++itc) {
                    const uint32_t s1 = L::slot1(itc), s2 = L::slot2(itc);
                    ok = mbar_wait(&bar_full[s2], L::phase2(itc), abort_flag);
                    if (!ok) break;
                    if (L::kHasX2) {
                        tc_fence_after();
                        issue_x(kColX2, L::kSbOff, L::kRingOff + s2 * L::kSmall);
                        tc_commit(bar_x2full);
                        tc_commit(&bar_empty[s2]);   // the second streamed tile only feeds X2
                    }
                    if (it + 1 < u.n_it) {
                        // X1 of the next block into the other buffer (read out two iterations ago): it runs while the
                        // compute warps work on this block
                        ok = mbar_wait(&bar_full[L::slot1(itc + 1)], L::phase1(itc + 1), abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_x(kColX1 + ((itc + 1) & 1) * 64, L::kSaOff, L::kRingOff + L::slot1(itc + 1) * L::kSmall);
                        tc_commit(&bar_x1full[(itc + 1) & 1]);
                    }
                    ok = mbar_wait(bar_wready, itc & 1, abort_flag);
                    if (ok && it == 0 && uc > 0) ok = mbar_wait(bar_accfree, (uc - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    {
                        const uint32_t sbt = L::kHasX2 ? s1 : s2;   // FWD: V, DV: dO; DK: Q, DQ: K
                        const uint64_t db = sdesc_advance(mdesc0, L::kRingOff + sbt * L::kSmall);
#pragma unroll
                        for (int kk = 0; kk < kBlk / 16; ++kk)
                            mma_ts(tmem_base + kColAcc, tmem_base + kColW + kk * 8, sdesc_advance(db, kk * 2048), idesc_acc,
                                   (it > 0 || kk > 0) ? 1u : 0u);
                    }
                    tc_commit(bar_accstep);
                    tc_commit(&bar_empty[s1]);
                    if (!L::kHasX2) tc_commit(&bar_empty[s2]);
                    if (it == u.n_it - 1) { tc_commit(bar_accdone); tc_commit(bar_stempty); }
                }
                ++uc;
            }
            if (!ok || abort_flag[0]) {
                tc_commit(bar_drain);
                mbar_wait_drain(bar_drain, 0, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp < 4 * L::kGroups) {
        // ---------------- compute warps: thread (r, grp) owns stationary row r (TMEM lane r) and the columns
        // [col0, col0 + kCols) of every streamed block ----------------
        constexpr int NC = L::kCols;
        const int grp = warp >> 2;
        const int col0 = grp * NC;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_x1 = tmem_base + lane_addr + kColX1 + col0;
        const uint32_t t_x2 = tmem_base + lane_addr + kColX2 + col0;
        const uint32_t t_w = tmem_base + lane_addr + kColW + col0 / 2;
        const uint32_t t_acc = tmem_base + lane_addr + kColAcc + grp * (kD / L::kGroups);
        Units<MODE> u(p, cta);
        uint32_t uc = 0, itc = 0;
        bool ok = true;
        while (ok && u.next()) {
            const int64_t row = u.r0 + r;            // this thread's query row (FWD, DQ) or key (DV, DK)
            const bool row_ok = row < p.T;
            // visible columns of streamed block starting at b0: [lo_abs - b0, hi_abs - b0]
            //   query-stationary: keys from the start of the row's sample to the row itself
            //   key-stationary:   queries from the key itself to the end of its sample
            int64_t lo_abs, hi_abs;
            if (L::kKeyStationary) {
                lo_abs = row;
                hi_abs = row_ok ? (int64_t)p.tok_end[row] - 1 : -1;
            } else {
                lo_abs = row_ok ? (int64_t)p.tok_start[row] : 0;
                hi_abs = row_ok ? row : -1;
            }
            float m_ref = -INFINITY, l_sum = 0.f;    // FWD
            float lse2r = 0.f, dvecr = 0.f;          // DQ
            if (MODE == DQ) {
                lse2r = p.lse2[(size_t)u.h * p.Tpad + row];   // row < Tpad always
                dvecr = p.dvec[(size_t)u.h * p.Tpad + row];
            }
            for (int it = 0; it < u.n_it && ok; ++it, ++itc) {
                const int64_t b0 = u.stream_row(it);
                // first and last visible column, counted from this thread's first column
                const int c_lo = (int)(lo_abs - b0 > kBlk ? kBlk : lo_abs - b0) - col0;
                const int c_hi = (int)(hi_abs - b0 < -1 ? -1 : hi_abs - b0) - col0;
                const uint32_t s1 = L::slot1(itc);
                const float* st = reinterpret_cast<const float*>(smem + L::kStatOff + s1 * 512) + col0;
                if (L::kStatBytes > 0) {   // the streamed rows' statistics arrive with their first tile
                    ok = warp_wait(&bar_full[s1], L::phase1(itc), abort_flag);
                    if (!ok) break;
                }
                ok = warp_wait(&bar_x1full[itc & 1], (itc >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t sr[NC];
#pragma unroll
                for (int c = 0; c < NC; c += 32) tmem_ld32(t_x1 + (itc & 1) * 64 + c, sr + c);
                tmem_ld_wait();
                uint32_t pk[NC / 2];
                if constexpr (MODE == FWD) {
#pragma unroll
                    for (int i = 0; i < kBlk; ++i)
                        if (i < c_lo || i > c_hi) sr[i] = 0xff800000u;  // -inf
                    float mx = -INFINITY;
                    {
                        float pm[8];
#pragma unroll
                        for (int q = 0; q < 8; ++q) pm[q] = fmaxf(__uint_as_float(sr[2 * q]), __uint_as_float(sr[2 * q + 1]));
#pragma unroll
                        for (int i = 16; i < kBlk; i += 16)
#pragma unroll
                            for (int q = 0; q < 8; ++q)
                                pm[q] = max3(pm[q], __uint_as_float(sr[i + 2 * q]), __uint_as_float(sr[i + 2 * q + 1]));
                        mx = fmaxf(max3(pm[0], pm[1], pm[2]), max3(pm[3], pm[4], pm[5]));
                        mx = max3(mx, pm[6], pm[7]);
                    }
                    mx *= p.scale_log2;
                    // lazy rescale: the reference only moves when the maximum grew by more than 2^8
                    float m_new = m_ref;
                    bool grow = false;
                    if (mx > m_ref + 8.0f || (m_ref == -INFINITY && mx > -INFINITY)) { m_new = mx; grow = true; }
                    const float factor = grow ? ex2_approx(m_ref - m_new) : 1.0f;
                    l_sum *= factor;
                    m_ref = m_new;
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    float ps0 = 0.f, ps1 = 0.f;
#pragma unroll
                    for (int i = 0; i < kBlk; i += 2) {
                        const float p0 = ex2_approx(fmaf(__uint_as_float(sr[i]), p.scale_log2, -m_use));
                        const float p1 = ex2_approx(fmaf(__uint_as_float(sr[i + 1]), p.scale_log2, -m_use));
                        ps0 += p0;
                        ps1 += p1;
                        pk[i >> 1] = pack_bf16x2(p0, p1);
                    }
                    if (it > 0 && __any_sync(0xffffffffu, grow)) {
                        // O is rescaled once the previous block's accumulation has landed (its W is spent then, too)
                        ok = warp_wait(bar_accstep, (itc - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < kD; c += 32) {
                            uint32_t orow[32];
                            tmem_ld32(t_acc + c, orow);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * factor);
                            tmem_st32(t_acc + c, orow);
                        }
                    }
                    l_sum += ps0 + ps1;
                } else {
                    // P = exp2(S c - LSE) on the visible elements, 0 elsewhere
                    float pf[NC];
#pragma unroll
                    for (int i = 0; i < NC; ++i) {
                        const float l2 = L::kKeyStationary ? st[i] : lse2r;
                        const float e = ex2_approx(fmaf(__uint_as_float(sr[i]), p.scale_log2, -l2));
                        pf[i] = (i < c_lo || i > c_hi) ? 0.f : e;
                    }
                    if (MODE == DV) {
#pragma unroll
                        for (int i = 0; i < NC; i += 2) pk[i >> 1] = pack_bf16x2(pf[i], pf[i + 1]);
                    } else {
                        ok = warp_wait(bar_x2full, itc & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        uint32_t dp[NC];
#pragma unroll
                        for (int c = 0; c < NC; c += 32) tmem_ld32(t_x2 + c, dp + c);
                        tmem_ld_wait();
#pragma unroll
                        for (int i = 0; i < NC; i += 2) {
                            const float d0 = L::kKeyStationary ? st[64 + i] : dvecr;
                            const float d1 = L::kKeyStationary ? st[64 + i + 1] : dvecr;
                            pk[i >> 1] = pack_bf16x2(pf[i] * (__uint_as_float(dp[i]) - d0), pf[i + 1] * (__uint_as_float(dp[i + 1]) - d1));
                        }
                    }
                }
                if (itc > 0) {   // the previous accumulating GEMM has consumed W
                    ok = warp_wait(bar_accstep, (itc - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll
                for (int c = 0; c < NC / 2; c += 16) tmem_st16(t_w + c, pk + c);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_wready);
            }
            if (!ok) break;
            // ---- unit epilogue: the accumulator leaves TMEM ----
            ok = warp_wait(bar_accdone, uc & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            float mul = 1.0f;
            if (MODE == FWD) mul = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
            if (MODE == DK || MODE == DQ) mul = p.scale;
            const int n_heads = L::kKeyStationary ? p.hkv : p.hq;
            const int head = L::kKeyStationary ? u.kvh : u.h;
            __nv_bfloat16* dst_row = p.out + ((size_t)row * n_heads + head) * kD + grp * (kD / L::kGroups);
            float* acc_row = L::kKeyStationary && p.acc32
                                 ? p.acc32 + ((size_t)row * n_heads + head) * kD + grp * (kD / L::kGroups) : nullptr;
#pragma unroll
            for (int c = 0; c < kD / L::kGroups; c += 32) {
                uint32_t v[32];
                tmem_ld32(t_acc + c, v);
                tmem_ld_wait();
                if (acc_row) {   // a key block meets several query chunks: its partial sums are added up in fp32
                    if (row_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(acc_row + c + i),
                                         "f"(__uint_as_float(v[i])), "f"(__uint_as_float(v[i + 1])),
                                         "f"(__uint_as_float(v[i + 2])), "f"(__uint_as_float(v[i + 3]))
                                         : "memory");
                    }
                } else if (row_ok) {
                    uint4* dst = reinterpret_cast<uint4*>(dst_row + c);
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 w;
                        w.x = pack_bf16x2(__uint_as_float(v[i]) * mul, __uint_as_float(v[i + 1]) * mul);
                        w.y = pack_bf16x2(__uint_as_float(v[i + 2]) * mul, __uint_as_float(v[i + 3]) * mul);
                        w.z = pack_bf16x2(__uint_as_float(v[i + 4]) * mul, __uint_as_float(v[i + 5]) * mul);
                        w.w = pack_bf16x2(__uint_as_float(v[i + 6]) * mul, __uint_as_float(v[i + 7]) * mul);
                        dst[i >> 3] = w;
                    }
                }
            }
            if (MODE == FWD && row_ok) p.lse[(size_t)u.h * p.T + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
            tc_fence_before();
            mbar_arrive(bar_accfree);
            ++uc;
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (abort_flag[0]) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

template <int MODE>
static int launch(const CUtensorMap& sa, const CUtensorMap& sb, const CUtensorMap& t1, const CUtensorMap& t2,
                  const Params& prm, int W, cudaStream_t s) {
    using L = Cfg<MODE>;
    if (!cfg_done(8 + MODE)) {   // per device
        if (cudaFuncSetAttribute(k_attn_d256<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kBytes) != cudaSuccess)
            return LIBRA_ERR_CUDA;
        cfg_mark(8 + MODE);
    }
    k_attn_d256<MODE><<<W, kThreads, L::kBytes, s>>>(sa, sb, t1, t2, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace d256

// Forward at head_dim 256 over the plan's query-major lists.
int launch_fwd_d256(const void* q, const void* k, const void* v, void* out, float* lse, const libra_plan* plan,
                    const libra_dims* dims, float scale, cudaStream_t s) {
    using namespace d256;
    const PlanDir& d = plan->dir[0];
    CUtensorMap tq, tk, tv;
    int rc = make_thd_map(&tq, q, plan->T, dims->hq, kD, kRows);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k, plan->T, dims->hkv, kD, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v, plan->T, dims->hkv, kD, kBlk);
    if (rc != LIBRA_OK) return rc;
    Params prm = {};
    prm.out = reinterpret_cast<__nv_bfloat16*>(out);
    prm.lse = lse;
    prm.cta_offsets = d.d_cta_offsets;
    prm.cta_tiles = d.d_cta_exec;
    prm.tok_start = plan->d_tok_start;
    prm.tok_end = plan->d_tok_end;
    prm.T = plan->T;
    prm.Tpad = (plan->T + 127) / 128 * 128;
    prm.hq = dims->hq; prm.hkv = dims->hkv; prm.H = d.H;
    prm.scale = scale; prm.scale_log2 = scale * 1.4426950408889634f;
    prm.status = plan->d_status + 1; prm.plan_status = plan->d_status;
    prm.wait_limit_ns = plan->wait_limit_ns; prm.inject_stall = plan->inject_stall;
    prm.busy = d.d_busy;
    return launch<FWD>(tq, tq, tk, tv, prm, d.W, s);
}

// Backward at head_dim 256: the dV and dK passes over the key-major lists, the dQ pass over the query-major lists.
// lse2 / dvec are the row statistics [Hq, Tpad] the caller has computed on the same stream.
int launch_bwd_d256(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                    const float* lse2, const float* dvec, int64_t Tpad, float* dk_acc, float* dv_acc,
                    const libra_plan* plan, const libra_dims* dims, float scale, cudaStream_t s) {
    using namespace d256;
    const PlanDir& dq_dir = plan->dir[0];
    const bool pairs = dk_acc != nullptr;            // key-stationary passes over pair tiles, fp32 accumulators
    const PlanDir& kv_dir = plan->dir[pairs ? 2 : 1];
    CUtensorMap q128, do128, k128, v128, q64, do64, k64, v64;
    int rc = make_thd_map(&q128, q, plan->T, dims->hq, kD, kRows);
    if (rc == LIBRA_OK) rc = make_thd_map(&do128, dout, plan->T, dims->hq, kD, kRows);
    if (rc == LIBRA_OK) rc = make_thd_map(&k128, k, plan->T, dims->hkv, kD, kRows);
    if (rc == LIBRA_OK) rc = make_thd_map(&v128, v, plan->T, dims->hkv, kD, kRows);
    if (rc == LIBRA_OK) rc = make_thd_map(&q64, q, plan->T, dims->hq, kD, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&do64, dout, plan->T, dims->hq, kD, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&k64, k, plan->T, dims->hkv, kD, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&v64, v, plan->T, dims->hkv, kD, kBlk);
    if (rc != LIBRA_OK) return rc;
    Params prm = {};
    prm.lse2 = lse2; prm.dvec = dvec;
    prm.tok_start = plan->d_tok_start;
    prm.tok_end = plan->d_tok_end;
    prm.T = plan->T;
    prm.Tpad = Tpad;
    prm.hq = dims->hq; prm.hkv = dims->hkv; prm.H = dq_dir.H;
    prm.scale = scale; prm.scale_log2 = scale * 1.4426950408889634f;
    prm.status = plan->d_status + 2; prm.plan_status = plan->d_status;
    prm.wait_limit_ns = plan->wait_limit_ns; prm.inject_stall = plan->inject_stall;
    libra_plan* mp = const_cast<libra_plan*>(plan);
    // dV and dK: key-major lists
    prm.cta_offsets = kv_dir.d_cta_offsets; prm.cta_tiles = kv_dir.d_cta_exec; prm.busy = kv_dir.d_busy;
    if (pairs) { prm.u_blk = kv_dir.d_u_blk; prm.u_chunk = kv_dir.d_u_chunk; prm.NU = kv_dir.NB; prm.R = kv_dir.chunk / kv_dir.tile; }
    time_begin(mp, 1, s);
    prm.out = reinterpret_cast<__nv_bfloat16*>(dv);
    prm.acc32 = dv_acc;
    rc = launch<DV>(k128, k128, q64, do64, prm, kv_dir.W, s);
    prm.out = reinterpret_cast<__nv_bfloat16*>(dk);
    prm.acc32 = dk_acc;
    if (rc == LIBRA_OK) rc = launch<DK>(k128, v128, q64, do64, prm, kv_dir.W, s);
    time_end(mp, 1, s);
    prm.acc32 = nullptr;
    if (rc != LIBRA_OK) return rc;
    // dQ: query-major lists
    prm.cta_offsets = dq_dir.d_cta_offsets; prm.cta_tiles = dq_dir.d_cta_exec; prm.busy = dq_dir.d_busy2;
    prm.out = reinterpret_cast<__nv_bfloat16*>(dq);
    time_begin(mp, 2, s);
    rc = launch<DQ>(q128, do128, k64, v64, prm, dq_dir.W, s);
    time_end(mp, 2, s);
    return rc;
}

}  // namespace libra
