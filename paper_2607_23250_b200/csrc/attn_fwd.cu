// Forward pool attention for sm_100a: one persistent, warp-specialised kernel.
//
// Each CTA walks the query-major tile list the planner gave it.  A tile is 256 query rows
// (two 128-row sub-tiles, "slots") of one head shard; for every head of the shard the CTA
// streams the key/value blocks the rows can see, from the block that holds the start of the
// first row's sample up to the diagonal block.  Blocks are cut at multiples of 128 on the
// pool's token axis, so the diagonal block of a sub-tile is aligned with it and every other
// visible block is either dense or needs the per-row sample-start mask.
//
// Roles (384 threads): warps 0-3 and 4-7 are the softmax groups of slot 0 and 1 (one row per
// thread, S read from TMEM, P written back to TMEM as bf16 over S), warp 8 issues TMA loads,
// warp 9 issues tcgen05.mma, warps 10-11 only hand their registers to the softmax groups.
// TMEM: S0 | S1 | O0 | O1, 128 fp32 columns each.
// Pipeline per key block j:   PV0(j) S0(j+1) PV1(j) S1(j+1)   on the tensor pipe, while the
// softmax group of one slot works during the other slot's MMAs.  P is handed over in two halves
// (keys 0-63, then 64-127), so the first four key steps of PV run under the second half's exponentials.
#include <math.h>

#include "common.h"
#include "ptx.cuh"

#ifndef LIBRA_FWD_REG_DEC
#define LIBRA_FWD_REG_DEC 56
#define LIBRA_FWD_REG_INC 216
#endif

namespace libra {

constexpr int kBM = 128;            // rows per slot
constexpr int kBN = 128;            // keys per block
constexpr int kFwdThreads = 384;  // warps 10-11 only donate registers
constexpr float kRescaleThreshold = 8.0f;  // log2 units: O is rescaled only when the max grows by more
constexpr uint64_t kFwdDrainNs = 2000000;  // teardown after a give-up: budget for work already in flight to land

template <int D>
struct FwdSmem {
    static constexpr int kHalfBytes = 128 * 128;              // 128 rows x 64 bf16 (one swizzle column)
    static constexpr int kTileBytes = kHalfBytes * (D / 64);  // one 128 x D operand tile
    static constexpr int kStages = (D == 128) ? 5 : 8;
    static constexpr int kQOff = 0;
    static constexpr int kRingOff = 2 * kTileBytes;
    static constexpr int kBarOff = kRingOff + kStages * kTileBytes;
    // barriers: full[kStages], empty[kStages], q_full, q_empty, s_full[2], p_ready[2], o_done[2], p_half[2], drain
    static constexpr int kNumBars = 2 * kStages + 11;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static constexpr int kAlloc = kBytes + 1024;  // slack to align the base to 1024 B
};

struct FwdParams {
    __nv_bfloat16* out;
    float* lse;
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* tok_start;
    int64_t T;
    int hq, hkv, H;
    float scale_log2;  // softmax scale * log2(e)
    int* status;       // word to flag LIBRA_ERR_TIMEOUT in
    const int* plan_status;  // the planner's verdict on cu_seqlens: non-zero = do not run
    uint32_t wait_limit_ns;  // budget of one device-side wait
    int inject_stall;        // test aid: the producer issues no loads, so the consumers' waits run out
    uint64_t* busy;    // [2 * gridDim.x]
    uint32_t* tile_ns; // [tiles] time spent on each tile (slot 0's first softmax thread), ns
};

// Range of key blocks slot g of a tile sees; empty (lo > hi) if the slot lies past T.
struct SlotRange {
    int lo, hi;
};
__device__ __forceinline__ SlotRange slot_range(const int32_t* tok_start, int64_t T, int64_t qs) {
    SlotRange r;
    if (qs >= T) { r.lo = 1; r.hi = 0; return r; }
    r.lo = tok_start[qs] / kBN;
    r.hi = (int)(qs / kBN);
    return r;
}



template <int D>
__global__ void __launch_bounds__(kFwdThreads, 1)
k_attn_fwd(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const FwdParams p) {
    using L = FwdSmem<D>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_full = bars;
    uint64_t* bar_empty = bars + L::kStages;
    uint64_t* bar_qfull = bars + 2 * L::kStages;
    uint64_t* bar_qempty = bar_qfull + 1;
    uint64_t* bar_sfull = bar_qfull + 2;   // [2]
    uint64_t* bar_pready = bar_qfull + 4;  // [2]
    uint64_t* bar_odone = bar_qfull + 6;   // [2]
    uint64_t* bar_phalf = bar_qfull + 8;   // [2] P of the first 64 keys is in TMEM
    uint64_t* bar_drain = bar_qfull + 10;  // teardown after a give-up: every MMA issued so far has completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    // A plan whose cu_seqlens failed the planner's check is never executed: report and leave.
    if (const int ps = *p.plan_status; ps != 0) {
        if (threadIdx.x == 0) { atomicExch(p.status, ps); p.busy[2 * cta] = p.busy[2 * cta + 1] = 0; }
        return;
    }
    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kStages; ++i) { mbar_init(&bar_full[i], 1); mbar_init(&bar_empty[i], 1); }
        mbar_init(bar_qfull, 1);
        mbar_init(bar_qempty, 1);
        for (int g = 0; g < 2; ++g) {
            mbar_init(&bar_sfull[g], 1);
            mbar_init(&bar_pready[g], kBM);
            mbar_init(&bar_odone[g], 1);
            mbar_init(&bar_phalf[g], kBM);
        }
        mbar_init(bar_drain, 1);
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit_ns;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == 9) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int tile_begin = p.cta_offsets[cta];
    const int tile_end = p.cta_offsets[cta + 1];
    const int heads_per_shard = p.hq / p.H;
    const int G = p.hq / p.hkv;

    // The softmax groups hold a whole 128-column row of S in registers; the producer / MMA
    // warpgroup needs few registers and hands the rest over.
    if (warp >= 10) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(LIBRA_FWD_REG_DEC));
    } else if (warp == 8) {
        // ---------------- TMA producer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(LIBRA_FWD_REG_DEC));
        const bool leader = elect_one();
        uint32_t ring = 0, qcnt = 0;
        bool ok = true;
        for (int idx = tile_begin; idx < tile_end && ok && !p.inject_stall; ++idx) {
            const int t = p.cta_tiles[idx];
            const int64_t q0 = (int64_t)(t / p.H) * (2 * kBM);
            const SlotRange r0 = slot_range(p.tok_start, p.T, q0);
            const SlotRange r1 = slot_range(p.tok_start, p.T, q0 + kBM);
            const bool act1 = r1.lo <= r1.hi;
            const int lo = r0.lo, hi = act1 ? r1.hi : r0.hi;
            for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                const int h = (t % p.H) * heads_per_shard + hh;
                const int kvh = h / G;
                ok = warp_wait(bar_qempty, (qcnt & 1) ^ 1, abort_flag);
                if (!ok) break;
                if (leader) {
                    mbar_arrive_expect_tx(bar_qfull, (act1 ? 2 : 1) * L::kTileBytes);
                    for (int g = 0; g < (act1 ? 2 : 1); ++g)
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_3d(smem + L::kQOff + g * L::kTileBytes + half * L::kHalfBytes, &tm_q, bar_qfull,
                                        half * 64, h, (int)(q0 + g * kBM));
                }
                ++qcnt;
                for (int j = lo; j <= hi && ok; ++j) {
                    for (int kv = 0; kv < 2 && ok; ++kv) {  // K_j then V_j
                        const uint32_t st = ring % L::kStages;
                        ok = warp_wait(&bar_empty[st], ((ring / L::kStages) & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        if (leader) {
                            mbar_arrive_expect_tx(&bar_full[st], L::kTileBytes);
                            for (int half = 0; half < D / 64; ++half)
                                tma_load_3d(smem + L::kRingOff + st * L::kTileBytes + half * L::kHalfBytes,
                                            kv == 0 ? &tm_k : &tm_v, &bar_full[st], half * 64, kvh, j * kBN);
                        }
                        ++ring;
                    }
                }
            }
        }
        if (leader && (!ok || abort_flag[0])) {
            // Give-up path: nothing new is issued; the copies already issued land before shared memory is released.
            if (qcnt > 0) mbar_wait_drain(bar_qfull, (qcnt - 1) & 1, kFwdDrainNs);
            for (uint32_t b = 1; b <= (uint32_t)L::kStages && b <= ring; ++b)
                mbar_wait_drain(&bar_full[(ring - b) % L::kStages], ((ring - b) / L::kStages) & 1, kFwdDrainNs);
        }
        __syncwarp();
    } else if (warp == 9) {
        // ---------------- MMA issuer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(LIBRA_FWD_REG_DEC));
        const bool leader = elect_one();
        constexpr uint32_t idesc_s = make_idesc(kBM, kBN, 0, 0);
        constexpr uint32_t idesc_pv = make_idesc(kBM, D, 0, 1);
        const uint32_t smem_base = smem_u32(smem);
        uint32_t ring = 0, qcnt = 0;
        uint32_t pcnt[2] = {0, 0};
        bool ok = true;
        // Base descriptors are built once; every MMA only adds a constant to them.
        const uint64_t desc_q = make_sdesc(smem_base + L::kQOff, 16, 1024);                  // K-major Q slot 0
        const uint64_t desc_k = make_sdesc(smem_base + L::kRingOff, 16, 1024);               // K-major ring stage 0
        const uint64_t desc_v = make_sdesc(smem_base + L::kRingOff, L::kHalfBytes, 1024);    // MN-major ring stage 0
        auto issue_s = [&](int g, uint32_t stage) {
            const uint64_t qa = sdesc_advance(desc_q, g * L::kTileBytes);
            const uint64_t ka = sdesc_advance(desc_k, stage * L::kTileBytes);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk / 4) * L::kHalfBytes + (kk % 4) * 32;
                mma_ss(tmem_base + g * kBN, sdesc_advance(qa, off), sdesc_advance(ka, off), idesc_s, kk > 0);
            }
            tc_commit(&bar_sfull[g]);
        };
        // O[g] (+)= P[g] V over the key steps [kk0, kk1) of 16 keys; the softmax group hands P over in two halves
        auto issue_pv = [&](int g, uint32_t stage, bool accumulate, int kk0, int kk1) {
            const uint64_t va = sdesc_advance(desc_v, stage * L::kTileBytes);
#pragma unroll
            for (int kk = kk0; kk < kk1; ++kk) {
                mma_ts(tmem_base + 2 * kBN + g * D, tmem_base + g * kBN + kk * 8, sdesc_advance(va, kk * 2048), idesc_pv,
                       (accumulate || kk > 0) ? 1u : 0u);
            }
            if (kk1 == kBN / 16) tc_commit(&bar_odone[g]);
        };
        for (int idx = tile_begin; idx < tile_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int64_t q0 = (int64_t)(t / p.H) * (2 * kBM);
            const SlotRange r[2] = {slot_range(p.tok_start, p.T, q0), slot_range(p.tok_start, p.T, q0 + kBM)};
            const bool act1 = r[1].lo <= r[1].hi;
            const int lo = r[0].lo, hi = act1 ? r[1].hi : r[0].hi;
            for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                ok = warp_wait(bar_qfull, qcnt & 1, abort_flag);
                if (!ok) break;
                ++qcnt;
                // prologue: S(lo)
                uint32_t st = ring % L::kStages;
                ok = warp_wait(&bar_full[st], (ring / L::kStages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                if (leader) {
                    for (int g = 0; g < 2; ++g)
                        if (lo >= r[g].lo && lo <= r[g].hi) issue_s(g, st);
                    tc_commit(&bar_empty[st]);
                    if (lo == hi) tc_commit(bar_qempty);  // no later MMA of this tile reads Q
                }
                ++ring;
                for (int j = lo; j <= hi && ok; ++j) {
                    const uint32_t st_v = ring % L::kStages;
                    ok = warp_wait(&bar_full[st_v], (ring / L::kStages) & 1, abort_flag);
                    if (!ok) break;
                    ++ring;
                    uint32_t st_k = 0;
                    if (j + 1 <= hi) {
                        st_k = ring % L::kStages;
                        ok = warp_wait(&bar_full[st_k], (ring / L::kStages) & 1, abort_flag);
                        if (!ok) break;
                        ++ring;
                    }
                    for (int g = 0; g < 2 && ok; ++g) {
                        if (j >= r[g].lo && j <= r[g].hi) {
                            ok = warp_wait(&bar_phalf[g], pcnt[g] & 1, abort_flag);   // P of keys 0..63
                            if (!ok) break;
                            tc_fence_after();
                            if (leader) issue_pv(g, st_v, j != r[g].lo, 0, kBN / 32);
                            ok = warp_wait(&bar_pready[g], pcnt[g] & 1, abort_flag);  // the rest, while those MMAs run
                            if (!ok) break;
                            ++pcnt[g];
                            tc_fence_after();
                            if (leader) issue_pv(g, st_v, j != r[g].lo, kBN / 32, kBN / 16);
                        }
                        if (j + 1 <= hi && j + 1 >= r[g].lo && j + 1 <= r[g].hi) {
                            if (leader) issue_s(g, st_k);
                        }
                    }
                    if (!ok) break;
                    if (leader) {
                        tc_commit(&bar_empty[st_v]);
                        if (j + 1 <= hi) tc_commit(&bar_empty[st_k]);
                        if (j + 1 == hi) tc_commit(bar_qempty);  // S(hi) was the last reader of Q: the next
                    }                                            // tile's Q load overlaps the last block
                    __syncwarp();
                }
                __syncwarp();
            }
        }
        if (leader && (!ok || abort_flag[0])) {   // give-up path: the MMAs already issued finish before TMEM is freed
            tc_commit(bar_drain);
            mbar_wait_drain(bar_drain, 0, kFwdDrainNs);
        }
        __syncwarp();
    } else {
        // ---------------- softmax groups ----------------
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(LIBRA_FWD_REG_INC));
        const int g = warp >> 2;
        const int row_in_tile = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem_base + lane_addr + g * kBN;
        const uint32_t t_o = tmem_base + lane_addr + 2 * kBN + g * D;
        uint32_t scnt = 0, ocnt = 0;
        bool ok = true;
        for (int idx = tile_begin; idx < tile_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int64_t qs = (int64_t)(t / p.H) * (2 * kBM) + g * kBM;
            const SlotRange rg = slot_range(p.tok_start, p.T, qs);
            if (rg.lo > rg.hi) continue;  // slot past the end of the pool
            const uint64_t tile_t0 = threadIdx.x == 0 ? globaltimer_ns() : 0;
            const int64_t row = qs + row_in_tile;
            const bool row_ok = row < p.T;
            const int kstart = row_ok ? p.tok_start[row] : 0;
            // last valid row of the slot decides which blocks need the sample-start mask
            const int64_t last_row = (qs + kBM <= p.T ? qs + kBM : p.T) - 1;
            const int max_kstart = p.tok_start[last_row];
            for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                const int h = (t % p.H) * heads_per_shard + hh;
                float m_ref = -INFINITY, l_sum = 0.f;
                for (int j = rg.lo; j <= rg.hi && ok; ++j) {
                    ok = warp_wait(&bar_sfull[g], scnt & 1, abort_flag);
                    if (!ok) break;
                    ++scnt;
                    tc_fence_after();
                    uint32_t sr[kBN];
                    tmem_ld32(t_s, sr);
                    tmem_ld32(t_s + 32, sr + 32);
                    tmem_ld32(t_s + 64, sr + 64);
                    tmem_ld32(t_s + 96, sr + 96);
                    tmem_ld_wait();
                    const int k0 = j * kBN;
                    const bool need_mask = (k0 + kBN - 1 > qs) || (k0 < max_kstart) || !row_ok;
                    if (need_mask) {
                        const int c_lo = row_ok ? kstart - k0 : kBN;        // first visible column
                        const int c_hi = row_ok ? (int)(row - k0) : -1;      // last visible column
#pragma unroll
                        for (int i = 0; i < kBN; ++i)
                            if (i < c_lo || i > c_hi) sr[i] = 0xff800000u;  // -inf
                    }
                    float mx;
                    {   // eight independent chains keep the 3-input max off the latency-bound path
                        float pm[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) pm[u] = fmaxf(__uint_as_float(sr[2 * u]), __uint_as_float(sr[2 * u + 1]));
#pragma unroll
                        for (int i = 16; i < kBN; i += 16)
#pragma unroll
                            for (int u = 0; u < 8; ++u)
                                pm[u] = max3(pm[u], __uint_as_float(sr[i + 2 * u]), __uint_as_float(sr[i + 2 * u + 1]));
                        mx = fmaxf(max3(pm[0], pm[1], pm[2]), max3(pm[3], pm[4], pm[5]));
                        mx = max3(mx, pm[6], pm[7]);
                    }
                    mx *= p.scale_log2;  // scale > 0, so the max commutes with it
                    // lazy rescale: keep the old reference unless the max grew by > threshold
                    float m_new = m_ref;
                    bool grow = false;
                    if (mx > m_ref + kRescaleThreshold || (m_ref == -INFINITY && mx > -INFINITY)) {
                        m_new = mx;
                        grow = true;
                    }
                    const float factor = grow ? ex2_approx(m_ref - m_new) : 1.0f;  // m_ref=-inf gives 0
                    const bool first = (j == rg.lo);
                    if (!first && __any_sync(0xffffffffu, grow)) {
                        // PV(j-1) must have landed in O before it is rescaled
                        ok = warp_wait(&bar_odone[g], (ocnt - 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
#pragma unroll
                        for (int c = 0; c < D; c += 32) {
                            uint32_t orow[32];
                            tmem_ld32(t_o + c, orow);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) orow[i] = __float_as_uint(__uint_as_float(orow[i]) * factor);
                            tmem_st32(t_o + c, orow);
                        }
                    }
                    l_sum *= factor;
                    m_ref = m_new;
                    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
                    const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
                    const uint64_t negm2 = f2_pack(-m_use, -m_use);
                    uint64_t psum2[4] = {f2_pack(0.f, 0.f), f2_pack(0.f, 0.f), f2_pack(0.f, 0.f), f2_pack(0.f, 0.f)};
#pragma unroll
                    for (int c = 0; c < kBN; c += 32) {
                        uint32_t pk[16];
#pragma unroll
                        for (int i = 0; i < 32; i += 2) {
                            float x0, x1;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(sr[c + i]), __uint_as_float(sr[c + i + 1])), scale2, negm2),
                                      x0, x1);
                            const float p0 = ex2_sel(x0, i), p1 = ex2_sel(x1, i + 1);
                            psum2[(i >> 1) & 3] = f2_add(psum2[(i >> 1) & 3], f2_pack(p0, p1));
                            pk[i >> 1] = pack_bf16x2(p0, p1);
                        }
                        tmem_st16(t_s + (c >> 1), pk);
                        if (c == kBN / 2 - 32) {  // P of the first 64 keys is complete: its PV steps can start
                            tmem_st_wait();
                            tc_fence_before();
                            mbar_arrive(&bar_phalf[g]);
                        }
                    }
                    {
                        float a, b;
                        f2_unpack(f2_add(f2_add(psum2[0], psum2[1]), f2_add(psum2[2], psum2[3])), a, b);
                        l_sum += a + b;
                    }
                    tmem_st_wait();
                    tc_fence_before();
                    mbar_arrive(&bar_pready[g]);
                    ++ocnt;
                }
                if (!ok) break;
                // epilogue: wait for the last PV, normalise, store
                ok = warp_wait(&bar_odone[g], (ocnt - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                const float inv_l = (l_sum > 0.f) ? 1.0f / l_sum : 0.f;
                __nv_bfloat16* orow_ptr = p.out + ((size_t)row * p.hq + h) * D;
#pragma unroll
                for (int c = 0; c < D; c += 32) {
                    uint32_t orow[32];
                    tmem_ld32(t_o + c, orow);
                    tmem_ld_wait();
                    if (row_ok) {
                        uint4* dst = reinterpret_cast<uint4*>(orow_ptr + c);
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(orow[i]) * inv_l, __uint_as_float(orow[i + 1]) * inv_l);
                            v.y = pack_bf16x2(__uint_as_float(orow[i + 2]) * inv_l, __uint_as_float(orow[i + 3]) * inv_l);
                            v.z = pack_bf16x2(__uint_as_float(orow[i + 4]) * inv_l, __uint_as_float(orow[i + 5]) * inv_l);
                            v.w = pack_bf16x2(__uint_as_float(orow[i + 6]) * inv_l, __uint_as_float(orow[i + 7]) * inv_l);
                            dst[i >> 3] = v;
                        }
                    }
                }
                if (row_ok) p.lse[(size_t)h * p.T + row] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
                // the next PV into this slot's O may only start after these reads: it is issued
                // after this group's next p_ready arrival, which follows in program order
                tc_fence_before();
            }
            if (threadIdx.x == 0 && ok) p.tile_ns[t] = (uint32_t)(globaltimer_ns() - tile_t0);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 9) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (*abort_flag) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

// ---- host ---------------------------------------------------------------------------------

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    }
    return fn;
}

// bf16 tensor [T, H, d] viewed as (d, H, T); box = 64 x 1 x 128 rows, 128-byte swizzle, zero fill.
int make_thd_map(CUtensorMap* m, const void* base, int64_t T, int H, int d, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return LIBRA_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)H * d * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LIBRA_OK : LIBRA_ERR_CUDA;
}

int make_f32_2d_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int box_cols, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return LIBRA_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 4};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LIBRA_OK : LIBRA_ERR_CUDA;
}

int make_f32_3d_map(CUtensorMap* m, const void* base, int64_t T, int H, int d, int box_cols, int box_rows) {
    EncodeTiledFn enc = get_encode();
    if (!enc) return LIBRA_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)H, (cuuint64_t)T};
    cuuint64_t strides[2] = {(cuuint64_t)d * 4, (cuuint64_t)H * d * 4};
    cuuint32_t box[3] = {(cuuint32_t)box_cols, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = enc(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? LIBRA_OK : LIBRA_ERR_CUDA;
}

template <int D>
static int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const FwdParams& prm, int W,
                      cudaStream_t s) {
    using L = FwdSmem<D>;
    constexpr int kSlot = D == 128 ? 0 : 1;
    if (!cfg_done(kSlot)) {   // per device: the attribute belongs to the device's copy of the kernel
        if (cudaFuncSetAttribute(k_attn_fwd<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kAlloc) != cudaSuccess)
            return LIBRA_ERR_CUDA;
        if (!regs_pool_ok(k_attn_fwd<D>, 256, LIBRA_FWD_REG_INC, 128, LIBRA_FWD_REG_DEC)) return LIBRA_ERR_UNSUPPORTED;
        cfg_mark(kSlot);
    }
    k_attn_fwd<D><<<W, kFwdThreads, L::kAlloc, s>>>(tq, tk, tv, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace libra

using namespace libra;


extern "C" int libra_attn_pool_fwd(const void* q_dev, const void* k_dev, const void* v_dev,
                                   const int32_t* cu_seqlens_dev, const libra_plan_t* plan, void* out_dev,
                                   float* lse_dev, const libra_dims* dims, void* stream) {
    if (!q_dev || !k_dev || !v_dev || !cu_seqlens_dev || !plan || !out_dev || !lse_dev || !dims)
        return LIBRA_ERR_INVALID_ARG;
    if (dims->hq <= 0 || dims->hkv <= 0 || dims->hq % dims->hkv) return LIBRA_ERR_INVALID_ARG;
    if (dims->head_dim != 64 && dims->head_dim != 128 && dims->head_dim != 256) return LIBRA_ERR_UNSUPPORTED;
    const PlanDir& d = plan->dir[0];
    if (!d.enabled || plan->T != dims->total_tokens) return LIBRA_ERR_PLAN_MISMATCH;
    if (d.tile != 2 * kBM) return LIBRA_ERR_UNSUPPORTED;
    if (dims->hq % d.H) return LIBRA_ERR_INVALID_ARG;
    if (d.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;  // one CTA per SM owns all 512 TMEM columns
    if (((uintptr_t)q_dev | (uintptr_t)k_dev | (uintptr_t)v_dev | (uintptr_t)out_dev) & 15) return LIBRA_ERR_INVALID_ARG;
    if (int rcd = check_plan_device(plan); rcd != LIBRA_OK) return rcd;

    const float scale = dims->softmax_scale > 0.f ? dims->softmax_scale : 1.0f / sqrtf((float)dims->head_dim);
    cudaStream_t s = (cudaStream_t)stream;
    libra_plan_t* mp = const_cast<libra_plan_t*>(plan);
    if (dims->head_dim == 256) {
        cudaMemsetAsync(plan->d_status + 1, 0, sizeof(int), s);
        time_begin(mp, 0, s);
        const int rc256 = launch_fwd_d256(q_dev, k_dev, v_dev, out_dev, lse_dev, plan, dims, scale, s);
        time_end(mp, 0, s);
        return rc256;
    }
    CUtensorMap tq, tk, tv;
    int rc = make_thd_map(&tq, q_dev, plan->T, dims->hq, dims->head_dim, kBM);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k_dev, plan->T, dims->hkv, dims->head_dim, kBN);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v_dev, plan->T, dims->hkv, dims->head_dim, kBN);
    if (rc != LIBRA_OK) return rc;

    FwdParams prm;
    prm.out = reinterpret_cast<__nv_bfloat16*>(out_dev);
    prm.lse = lse_dev;
    prm.cta_offsets = d.d_cta_offsets;
    prm.cta_tiles = d.d_cta_exec;
    prm.tok_start = plan->d_tok_start;
    prm.T = plan->T;
    prm.hq = dims->hq;
    prm.hkv = dims->hkv;
    prm.H = d.H;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.status = plan->d_status + 1;
    prm.plan_status = plan->d_status;
    prm.wait_limit_ns = plan->wait_limit_ns;
    prm.inject_stall = plan->inject_stall;
    prm.busy = d.d_busy;
    prm.tile_ns = d.d_tile_ns;
    cudaMemsetAsync(plan->d_status + 1, 0, sizeof(int), s);   // the word reports the most recent launch
    time_begin(mp, 0, s);
    rc = dims->head_dim == 128 ? launch_fwd<128>(tq, tk, tv, prm, d.W, s) : launch_fwd<64>(tq, tk, tv, prm, d.W, s);
    time_end(mp, 0, s);
    return rc;
}

