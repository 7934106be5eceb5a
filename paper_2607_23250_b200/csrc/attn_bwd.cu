// Backward pool attention for sm_100a.
//
// Two forms of the same computation; the plan decides (see libra_attn_pool_bwd in the public header).
// Fused form (attn_bwd_fused.cuh, plans with pair tiles, head_dim 128): row statistics, ONE kernel that computes
// S, dP, dV, dK and dQ of every 128 x 128 cell together (five GEMMs) with fp32 accumulators in global memory,
// and a conversion pass.
// Two-kernel form (this file and attn_bwd_dq.cuh): (1) prep: D_i = <dO_i, O_i> and LSE in log2 units, padded
// to a multiple of 128 rows; (2) the dK/dV kernel over key-major tiles; (3) the dQ kernel over query-major
// tiles.  Splitting dQ off costs two extra GEMMs per cell (S and dP are recomputed) but needs no cross-CTA
// reduction at all: no fp32 accumulator, no atomics, and the result is deterministic.  All kernels are persistent
// and warp-specialised (compute warpgroups, one TMA thread, one MMA-issuing thread; the dQ kernel also has a
// store thread) and keep their accumulators in TMEM.
//
// dK/dV kernel: a unit is 128 keys x one kv head; K and V stay in shared memory, dK and dV in
// TMEM, while the CTA streams every (query head of the group, 128-row query block) that sees the
// keys.  Keys sit in TMEM lanes:
//   S^T  = K Q^T   (SS)   P^T  = exp2(S^T c - LSE)   -> bf16, own columns     dV += P^T dO   (A in TMEM)
//   dP^T = V dO^T  (SS)   dS^T = P^T o (dP^T - D)    -> bf16, own columns     dK += dS^T Q   (A in TMEM)
// TMEM: X | P^T | dS^T | dK | dV = 128 + 64 + 64 + D + D columns.  S^T and dP^T take turns in the one fp32
// region X: it is free again as soon as the compute groups have READ it, not when the MMA that consumes the
// bf16 result has run, so dP^T(it) is issued right after S^T(it) has been read and S^T(it+1) right after
// dP^T(it) has been read, while dV(it) and dK(it) read P^T / dS^T from their own columns.
// P^T is handed to the dV MMA in two halves, so half of dV(it) runs under the second half's exponentials.
// dQ kernel (attn_bwd_dq.cuh): a unit is 128 query rows x one head; Q and dO are copied once per unit from
// shared memory into TMEM, dQ accumulates in TMEM, the CTA streams the key blocks the rows see (as the
// forward does).  Queries sit in TMEM lanes:
//   S  = Q K^T   dP = dO V^T   dS = P o (dP - D) -> bf16 over dP   dQ += dS K     (every A operand in TMEM)
#include <math.h>

#include "common.h"
#include "ptx.cuh"

namespace libra {


// warps 0-3, 4-7: exp groups (64 query columns each), 8-11: dS group, 12: TMA thread, 13: MMA thread,
// 14-15 only hand their registers over
constexpr int kBwdThreads = 512;
constexpr int kDkvTmaWarp = 12, kDkvMmaWarp = 13;
constexpr int kDkvRegsDs = 200, kDkvRegsOther = 56;   // setmaxnreg: the dS group keeps a whole row of dP^T in registers
constexpr int kBlk = 128;
constexpr int kSmemMax = 232448;  // 227 KB per CTA on sm_100
constexpr uint64_t kDrainNs = 2000000;  // teardown after a give-up: budget for work already in flight to land

// =================================================================================================
// dK / dV kernel
// =================================================================================================

template <int D>
struct DkvSmem {
    static constexpr int kHalfBytes = 128 * 128;
    static constexpr int kTileBytes = kHalfBytes * (D / 64);  // 128 x D bf16
    static constexpr int kQStages = 3;   // Q(it) lives from S(it) to dK(it), which runs behind dP(it+1)
    static constexpr int kDoStages = 2;  // dO(it) lives from dP(it) to dV(it)
    static constexpr int kKOff = 0;
    static constexpr int kVOff = kTileBytes;
    static constexpr int kQOff = 2 * kTileBytes;
    static constexpr int kDoOff = kQOff + kQStages * kTileBytes;
    static constexpr int kLseOff = kDoOff + kDoStages * kTileBytes;  // per Q stage:  lse2[128]
    static constexpr int kDvecOff = kLseOff + kQStages * 512;        // per dO stage: dvec[128]
    static constexpr int kBarOff = kDvecOff + kDoStages * 512;
    // kv_full, kv_empty, q_full[3], q_empty[3], do_full[2], do_empty[2], s_full, x_free1, dp_full, x_free2,
    // p_half, p_ready, p_free, ds_ready, dkv_full, dkv_empty, drain
    static constexpr int kNumBars = 2 + 2 * kQStages + 2 * kDoStages + 11;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static_assert(kBytes <= kSmemMax, "exceeds the shared memory of an sm_100 CTA");
};

struct DkvParams {
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    const float* lse2;  // [Hq, Tpad]  LSE * log2(e)
    const float* dvec;  // [Hq, Tpad]  D_i
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* tok_end;
    int64_t T, Tpad;
    int hq, hkv;
    float scale, scale_log2;
    int* status;
    const int* plan_status;  // the planner's verdict on cu_seqlens: non-zero = do not run
    uint32_t wait_limit_ns;
    int inject_stall;        // test aid: the producer issues no loads, so the consumers' waits run out
    uint64_t* busy;
};

// Query blocks a key block [k0, k0+128) is seen by: diagonal .. block of (end of last key's sample - 1).
__device__ __forceinline__ int last_q_block(const int32_t* tok_end, int64_t T, int64_t k0) {
    const int64_t last_key = (k0 + kBlk <= T ? k0 + kBlk : T) - 1;
    return (tok_end[last_key] - 1) / kBlk;
}

__device__ __forceinline__ void tmem_ld128(uint32_t taddr, uint32_t* r) {
    tmem_ld32(taddr, r);
    tmem_ld32(taddr + 32, r + 32);
    tmem_ld32(taddr + 64, r + 64);
    tmem_ld32(taddr + 96, r + 96);
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
k_attn_bwd_dkdv(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const DkvParams p) {
    using L = DkvSmem<D>;
    constexpr int QS = L::kQStages, DS = L::kDoStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_kvfull = bars + 0;
    uint64_t* bar_kvempty = bars + 1;
    uint64_t* bar_qfull = bars + 2;               // [QS]
    uint64_t* bar_qempty = bar_qfull + QS;        // [QS] dK(it) has run: Q stage free, dS^T columns free
    uint64_t* bar_dofull = bar_qempty + QS;       // [DS]
    uint64_t* bar_doempty = bar_dofull + DS;      // [DS] dV(it) has run: dO stage free
    uint64_t* bar_sfull = bar_doempty + DS;
    uint64_t* bar_xfree1 = bar_sfull + 1;   // S^T(it) has been read out of region X: dP^T(it) may overwrite it
    uint64_t* bar_dpfull = bar_sfull + 2;
    uint64_t* bar_xfree2 = bar_sfull + 3;   // dP^T(it) has been read out: S^T(it+1) may overwrite it
    uint64_t* bar_phalf = bar_sfull + 4;    // P^T of the first 32 queries of each exp group is in TMEM
    uint64_t* bar_pready = bar_sfull + 5;   // all of P^T(it) is in TMEM
    uint64_t* bar_pfree = bar_sfull + 6;    // dV(it) has run and the dS group has read P^T(it): columns free
    uint64_t* bar_dsready = bar_sfull + 7;
    uint64_t* bar_dkvfull = bar_sfull + 8;
    uint64_t* bar_dkvempty = bar_sfull + 9;
    uint64_t* bar_drain = bar_sfull + 10;   // teardown after a give-up: every MMA issued so far has completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicExch(p.status, LIBRA_ERR_CUDA);
        return;
    }
    if (const int ps = *p.plan_status; ps != 0) {  // malformed cu_seqlens: report and leave
        if (threadIdx.x == 0) { atomicExch(p.status, ps); p.busy[2 * cta] = p.busy[2 * cta + 1] = 0; }
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(bar_kvfull, 1);
        mbar_init(bar_kvempty, 1);
        for (int s = 0; s < QS; ++s) { mbar_init(&bar_qfull[s], 1); mbar_init(&bar_qempty[s], 1); }
        for (int s = 0; s < DS; ++s) { mbar_init(&bar_dofull[s], 1); mbar_init(&bar_doempty[s], 1); }
        mbar_init(bar_sfull, 1);
        mbar_init(bar_xfree1, 256);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_xfree2, 128);
        mbar_init(bar_phalf, 256);
        mbar_init(bar_pready, 256);
        mbar_init(bar_pfree, 129);       // the dS group's 128 threads + the commit behind dV(it)
        mbar_init(bar_dsready, 128);
        mbar_init(bar_dkvfull, 1);
        mbar_init(bar_dkvempty, 256);
        mbar_init(bar_drain, 1);
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit_ns;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == kDkvMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kDkvTmaWarp && lane == 0) {
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    constexpr uint32_t kColX = 0, kColP = 128, kColDS = 192, kColDK = 256, kColDV = 256 + D;

    const int unit_begin = p.cta_offsets[cta];
    const int unit_end = p.cta_offsets[cta + 1];
    const int G = p.hq / p.hkv;

    if (warp > kDkvMmaWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));
    } else if (warp == kDkvTmaWarp) {
        // ---------------- TMA producer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            uint32_t ucnt = 0, it_all = 0;
            bool ok = true;
            for (int idx = unit_begin; idx < unit_end && ok && !p.inject_stall; ++idx) {
                const int t = p.cta_tiles[idx];
                const int kvh = t % p.hkv;
                const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
                const int i_lo = (int)(k0 / kBlk);
                const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
                ok = mbar_wait(bar_kvempty, (ucnt & 1) ^ 1, abort_flag);
                if (!ok) break;
                mbar_arrive_expect_tx(bar_kvfull, 2 * L::kTileBytes);
                for (int half = 0; half < D / 64; ++half) {
                    tma_load_3d(smem + L::kKOff + half * L::kHalfBytes, &tm_k, bar_kvfull, half * 64, kvh, (int)k0);
                    tma_load_3d(smem + L::kVOff + half * L::kHalfBytes, &tm_v, bar_kvfull, half * 64, kvh, (int)k0);
                }
                ++ucnt;
                const int n_it = G * nblk;
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    const int h = kvh * G + it / nblk;
                    const int qb = (i_lo + it % nblk) * kBlk;
                    const uint32_t qs = it_all % QS, ds = it_all % DS;
                    ok = mbar_wait(&bar_qempty[qs], ((it_all / QS) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&bar_qfull[qs], L::kTileBytes + 512);
                    for (int half = 0; half < D / 64; ++half)
                        tma_load_3d(smem + L::kQOff + qs * L::kTileBytes + half * L::kHalfBytes, &tm_q, &bar_qfull[qs],
                                    half * 64, h, qb);
                    bulk_load_1d(smem + L::kLseOff + qs * 512, p.lse2 + (size_t)h * p.Tpad + qb, 512, &bar_qfull[qs]);
                    ok = mbar_wait(&bar_doempty[ds], ((it_all / DS) & 1) ^ 1, abort_flag);
                    if (!ok) {   // the Q load just issued is still in flight
                        mbar_wait_drain(&bar_qfull[qs], (it_all / QS) & 1, kDrainNs);
                        break;
                    }
                    mbar_arrive_expect_tx(&bar_dofull[ds], L::kTileBytes + 512);
                    for (int half = 0; half < D / 64; ++half)
                        tma_load_3d(smem + L::kDoOff + ds * L::kTileBytes + half * L::kHalfBytes, &tm_do,
                                    &bar_dofull[ds], half * 64, h, qb);
                    bulk_load_1d(smem + L::kDvecOff + ds * 512, p.dvec + (size_t)h * p.Tpad + qb, 512, &bar_dofull[ds]);
                }
            }
            if (!ok || abort_flag[0]) {
                // Give-up path: nothing new is issued; let the copies already issued land before the CTA's
                // shared memory is released (each armed phase completes when its bytes have arrived).
                if (ucnt > 0) mbar_wait_drain(bar_kvfull, (ucnt - 1) & 1, kDrainNs);
                for (uint32_t b = 1; b <= (uint32_t)QS && b <= it_all; ++b)
                    mbar_wait_drain(&bar_qfull[(it_all - b) % QS], ((it_all - b) / QS) & 1, kDrainNs);
                for (uint32_t b = 1; b <= (uint32_t)DS && b <= it_all; ++b)
                    mbar_wait_drain(&bar_dofull[(it_all - b) % DS], ((it_all - b) / DS) & 1, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp == kDkvMmaWarp) {
        // ---------------- MMA issuer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);  // S^T, dP^T: both operands K-major
            constexpr uint32_t idesc_acc = make_idesc(128, D, 0, 1);  // dV, dK: A from TMEM, B MN-major
            const uint32_t sb = smem_u32(smem);
            uint32_t ucnt = 0, it_all = 0;
            bool ok = true;
            // Base descriptors are built once; every MMA only adds a constant to them.
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);             // K-major view of a tile at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kHalfBytes, 1024);  // MN-major view
            // X[tmem] = A(K-major tile) * B(K-major tile)^T over the head dimension; offsets from smem base
            auto issue_kmajor = [&](uint32_t a_off, uint32_t b_off) {
                const uint64_t da = sdesc_advance(kdesc0, a_off), db = sdesc_advance(kdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * L::kHalfBytes + (kk % 4) * 32;
                    mma_ss(tmem_base + kColX, sdesc_advance(da, off), sdesc_advance(db, off), idesc_s, kk > 0);
                }
            };
            // C[tmem] (+)= A(TMEM, bf16 packed: queries 2 c and 2 c + 1 in column a_col + c) * B(MN-major tile)
            auto issue_acc = [&](uint32_t d_col, uint32_t a_col, uint32_t b_off, bool accumulate) {
                const uint64_t db = sdesc_advance(mdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem_base + d_col, tmem_base + a_col + kk * 8, sdesc_advance(db, kk * 2048), idesc_acc,
                           (accumulate || kk > 0) ? 1u : 0u);
            };
            // dK(i) += dS^T(i) Q(i), i a CTA-wide iteration index
            auto issue_dk = [&](uint32_t i, bool accumulate) -> bool {
                if (!mbar_wait(bar_dsready, i & 1, abort_flag)) return false;
                tc_fence_after();
                issue_acc(kColDK, kColDS, L::kQOff + (i % QS) * L::kTileBytes, accumulate);
                tc_commit(&bar_qempty[i % QS]);   // also tells the dS group that dS^T may be rewritten
                return true;
            };
            for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
                const int t = p.cta_tiles[idx];
                const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
                const int i_lo = (int)(k0 / kBlk);
                const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
                const int n_it = G * nblk;
                ok = mbar_wait(bar_kvfull, ucnt & 1, abort_flag);
                if (!ok) break;
                // S(0): region X is free once dP of the previous unit's last iteration has been read
                ok = mbar_wait(&bar_qfull[it_all % QS], (it_all / QS) & 1, abort_flag);
                if (ok && it_all > 0) ok = mbar_wait(bar_xfree2, (it_all - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_kmajor(L::kKOff, L::kQOff + (it_all % QS) * L::kTileBytes);
                tc_commit(bar_sfull);
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    const uint32_t ds = it_all % DS;
                    const uint32_t nx = it_all + 1;
                    const bool more = it + 1 < n_it;
                    // dP(it) over S(it), as soon as the exp group holds S(it) in registers
                    ok = mbar_wait(&bar_dofull[ds], (it_all / DS) & 1, abort_flag);
                    if (ok) ok = mbar_wait(bar_xfree1, it_all & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_kmajor(L::kVOff, L::kDoOff + ds * L::kTileBytes);
                    tc_commit(bar_dpfull);
                    if (!more) tc_commit(bar_kvempty);   // the unit's last readers of K and V: the next unit's K / V
                                                         // load overlaps the rest of this iteration
                    // dK(it-1): its dS^T was finished while S(it) ran
                    if (it > 0) { ok = issue_dk(it_all - 1, it > 1); if (!ok) break; }
                    // S(it+1) over dP(it), as soon as the dS group holds dP(it) in registers
                    if (more) {
                        ok = mbar_wait(&bar_qfull[nx % QS], (nx / QS) & 1, abort_flag);
                        if (ok) ok = mbar_wait(bar_xfree2, it_all & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_kmajor(L::kKOff, L::kQOff + (nx % QS) * L::kTileBytes);
                        tc_commit(bar_sfull);
                    }
                    // dV(it) += P^T dO
                    ok = mbar_wait(bar_pready, it_all & 1, abort_flag);
                    if (ok && it == 0 && ucnt > 0)   // the previous unit's dK / dV must have been read out
                        ok = mbar_wait(bar_dkvempty, (ucnt - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_acc(kColDV, kColP, L::kDoOff + ds * L::kTileBytes, it > 0);
                    tc_commit(&bar_doempty[ds]);
                    tc_commit(bar_pfree);
                }
                if (ok) ok = issue_dk(it_all - 1, n_it > 1);   // the unit's last dK
                if (ok) tc_commit(bar_dkvfull);
                ++ucnt;
            }
            if (!ok || abort_flag[0]) {   // give-up path: wait for the MMAs already issued before TMEM is freed
                tc_commit(bar_drain);
                mbar_wait_drain(bar_drain, 0, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ---------------- dS group ----------------
        // Thread r owns key row r (TMEM lane r) and all 128 query columns of dP^T; it turns dP^T and P^T (read back
        // as bf16) into dS^T.  The reads of region X are made by different warps for S^T and dP^T, so each happens
        // as soon as its MMA has landed.
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kDkvRegsDs));
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_x = tmem_base + lane_addr + kColX;
        const uint32_t t_p = tmem_base + lane_addr + kColP;
        const uint32_t t_ds = tmem_base + lane_addr + kColDS;
        uint32_t it_all = 0;
        bool ok = true;
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            const int n_it = G * nblk;
            // ---- dS group: dS^T = P^T o (dP^T - D) ----
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const uint32_t ds = it_all % DS;
                const float* dvec = reinterpret_cast<const float*>(smem + L::kDvecOff + ds * 512);
                ok = warp_wait(&bar_dofull[ds], (it_all / DS) & 1, abort_flag) &&
                     warp_wait(bar_dpfull, it_all & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t xs[64];   // (dP^T - D) as packed bf16 pairs
                {
                    uint32_t dpv[128];
                    tmem_ld128(t_x, dpv);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(bar_xfree2);   // dP^T(it) is in registers: S^T(it+1) may take the columns
                    const uint64_t neg1 = f2_pack(-1.f, -1.f);
#pragma unroll
                    for (int j = 0; j < 128; j += 4) {   // packed pairs: dP - D = fma(D, -1, dP)
                        const ulonglong2 d4 = *reinterpret_cast<const ulonglong2*>(dvec + j);
                        float a0, a1, b0, b1;
                        f2_unpack(f2_fma(d4.x, neg1, f2_pack(__uint_as_float(dpv[j]), __uint_as_float(dpv[j + 1]))), a0, a1);
                        f2_unpack(f2_fma(d4.y, neg1, f2_pack(__uint_as_float(dpv[j + 2]), __uint_as_float(dpv[j + 3]))), b0, b1);
                        xs[j >> 1] = pack_bf16x2(a0, a1);
                        xs[(j >> 1) + 1] = pack_bf16x2(b0, b1);
                    }
                }
                // dS^T(it-1) must have been consumed by dK(it-1) before its columns are rewritten
                if (it_all > 0) {
                    ok = warp_wait(&bar_qempty[(it_all - 1) % QS], ((it_all - 1) / QS) & 1, abort_flag);
                    if (!ok) break;
                }
                // P^T arrives in the order the exp groups finish it: the first 32 queries of each group's 64
                // (columns 0..15 and 32..47 of the packed P^T), then the rest.  dS^T = P^T o (dP^T - D) in bf16 pairs.
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    ok = warp_wait(half == 0 ? bar_phalf : bar_pready, it_all & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t pa[16], pb[16];
                    tmem_ld16(t_p + half * 16, pa);
                    tmem_ld16(t_p + 32 + half * 16, pb);
                    tmem_ld_wait();
                    if (half == 1) {           // all of P^T(it) is in registers
                        tc_fence_before();
                        mbar_arrive(bar_pfree);
                    }
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        pa[j] = mul_bf16x2(pa[j], xs[half * 16 + j]);
                        pb[j] = mul_bf16x2(pb[j], xs[32 + half * 16 + j]);
                    }
                    tmem_st16(t_ds + half * 16, pa);
                    tmem_st16(t_ds + 32 + half * 16, pb);
                }
                if (!ok) break;
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_dsready);
            }
        }
    } else {
        // ---------------- exp groups ----------------
        // Thread r of group grp owns key row r and the query columns [64 grp, 64 grp + 64) of S^T.
        const int grp = warp >> 2;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_x = tmem_base + lane_addr + kColX;
        const uint32_t t_p = tmem_base + lane_addr + kColP;
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int kvh = t % p.hkv;
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            const int n_it = G * nblk;
            const int64_t key = k0 + r;
            const bool key_ok = key < p.T;
            // ---- exp groups: P^T = exp2(S^T * c - LSE), zero where the query does not see the key ----
            const int c0 = 64 * grp;   // this group's query columns
            const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), neg1 = f2_pack(-1.f, -1.f);
            const int kend = key_ok ? p.tok_end[key] : 0;
            const int min_kend = p.tok_end[k0];
            const bool partial = k0 + kBlk > p.T;
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const int qb = (i_lo + it % nblk) * kBlk;
                const uint32_t qs = it_all % QS;
                const float* lse2 = reinterpret_cast<const float*>(smem + L::kLseOff + qs * 512) + c0;
                const bool need_mask = (qb == k0) || (qb + kBlk - 1 >= min_kend) || partial;
                const int j_lo = (int)(key - qb) - c0;   // first visible column of this group's range
                const int j_hi = kend - 1 - qb - c0;     // last visible column
                ok = warp_wait(&bar_qfull[qs], (it_all / QS) & 1, abort_flag) &&
                     warp_wait(bar_sfull, it_all & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t sv[64];
                tmem_ld32(t_x + c0, sv);
                tmem_ld32(t_x + c0 + 32, sv + 32);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_xfree1);   // S^T(it) is in registers: dP^T(it) may take the columns
                // P^T(it-1) must have been consumed (dV(it-1), the dS group) before its columns are rewritten
                if (it_all > 0) {
                    ok = warp_wait(bar_pfree, (it_all - 1) & 1, abort_flag);
                    if (!ok) break;
                }
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    float pf[32];
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {   // packed pairs: S * c - LSE
                        const int jj = half * 32 + j;
                        const ulonglong2 l4 = *reinterpret_cast<const ulonglong2*>(lse2 + jj);
                        float x0, x1, x2, x3;
                        f2_unpack(f2_fma(f2_pack(__uint_as_float(sv[jj]), __uint_as_float(sv[jj + 1])), scale2,
                                         f2_mul(l4.x, neg1)), x0, x1);
                        f2_unpack(f2_fma(f2_pack(__uint_as_float(sv[jj + 2]), __uint_as_float(sv[jj + 3])), scale2,
                                         f2_mul(l4.y, neg1)), x2, x3);
                        pf[j] = ex2_sel(x0, jj);
                        pf[j + 1] = ex2_sel(x1, jj + 1);
                        pf[j + 2] = ex2_sel(x2, jj + 2);
                        pf[j + 3] = ex2_sel(x3, jj + 3);
                    }
                    if (need_mask) {   // one uniform branch per half: the exponentials above stay one straight run
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (half * 32 + j < j_lo || half * 32 + j > j_hi) pf[j] = 0.f;
                    }
                    uint32_t pk[16];
#pragma unroll
                    for (int j = 0; j < 32; j += 2) pk[j >> 1] = pack_bf16x2(pf[j], pf[j + 1]);
                    tmem_st16(t_p + c0 / 2 + half * 16, pk);
                    tmem_st_wait();
                    tc_fence_before();
                    mbar_arrive(half == 0 ? bar_phalf : bar_pready);
                }
            }
            if (!ok) break;
            ++ucnt;
            // ---- unit epilogue: dK * scale and dV to global (each exp group stores half of the columns) ----
            ok = warp_wait(bar_dkvfull, (ucnt - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            constexpr int kCols = D / 2;
            const uint32_t t_dk = tmem_base + lane_addr + kColDK + grp * kCols;
            const uint32_t t_dv = tmem_base + lane_addr + kColDV + grp * kCols;
            const size_t gofs = ((size_t)key * p.hkv + kvh) * D + grp * kCols;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const float mul = which == 0 ? p.scale : 1.0f;
                __nv_bfloat16* gdst = (which == 0 ? p.dk : p.dv) + gofs;
#pragma unroll
                for (int cc = 0; cc < kCols; cc += 32) {
                    uint32_t v[32];
                    tmem_ld32((which == 0 ? t_dk : t_dv) + cc, v);
                    tmem_ld_wait();
                    if (key_ok) {
#pragma unroll
                        for (int i = 0; i < 32; i += 8) {
                            uint4 w;
                            w.x = pack_bf16x2(__uint_as_float(v[i]) * mul, __uint_as_float(v[i + 1]) * mul);
                            w.y = pack_bf16x2(__uint_as_float(v[i + 2]) * mul, __uint_as_float(v[i + 3]) * mul);
                            w.z = pack_bf16x2(__uint_as_float(v[i + 4]) * mul, __uint_as_float(v[i + 5]) * mul);
                            w.w = pack_bf16x2(__uint_as_float(v[i + 6]) * mul, __uint_as_float(v[i + 7]) * mul);
                            *reinterpret_cast<uint4*>(gdst + cc + i) = w;
                        }
                    }
                }
            }
            tc_fence_before();
            mbar_arrive(bar_dkvempty);
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == kDkvMmaWarp) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (abort_flag[0]) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

}  // namespace libra

#include "attn_bwd_dq.cuh"
#include "attn_bwd_fused.cuh"

namespace libra {

// ---- prep kernel ------------------------------------------------------------------------------

// D = <dO, O> per (token, head) and LSE in log2 units; rows in [T, Tpad) get zeros.
// One warp per (head, 32 consecutive tokens): D / 8 lanes read a row with 16-byte loads, lane i ends up with the sum
// of row i, so the two statistics leave as one coalesced 128-byte store each.  Eight steps' loads are issued at a time.
template <int D>
__global__ void k_bwd_prep(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                           const float* __restrict__ lse, int64_t T, int64_t Tpad, int hq, float* __restrict__ dvec,
                           float* __restrict__ lse2) {
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int64_t groups = Tpad / 32;  // Tpad is a multiple of 128
    if (w >= groups * hq) return;
    const int h = (int)(w / groups);
    const int64_t t0 = (w % groups) * 32;
    // 16-byte loads: D / 8 lanes cover a row, so a warp reads 32 / (D / 8) rows per step; eight steps' loads are
    // issued before the first is used
    constexpr int LPR = D / 8, RPS = 32 / LPR, STEPS = 32 / RPS, UNR = STEPS < 8 ? STEPS : 8;
    const int sub = lane / LPR, part = lane % LPR;
    float mine = 0.f;
    for (int s0 = 0; s0 < STEPS; s0 += UNR) {
        uint4 a[UNR], b[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const int64_t t = t0 + (s0 + u) * RPS + sub;
            a[u] = b[u] = make_uint4(0, 0, 0, 0);
            if (t < T) {
                a[u] = __ldg(reinterpret_cast<const uint4*>(out + ((size_t)t * hq + h) * D) + part);
                b[u] = __ldg(reinterpret_cast<const uint4*>(dout + ((size_t)t * hq + h) * D) + part);
            }
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            const uint32_t* x = reinterpret_cast<const uint32_t*>(&a[u]);
            const uint32_t* y = reinterpret_cast<const uint32_t*>(&b[u]);
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&x[i]));
                const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&y[i]));
                acc += fa.x * fb.x + fa.y * fb.y;
            }
#pragma unroll
            for (int off = LPR / 2; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
            // row (s0 + u) * RPS + sub of the warp's 32 goes to the lane of that number
            const float got = __shfl_sync(0xffffffffu, acc, (lane % RPS) * LPR);
            if (lane / RPS == s0 + u) mine = got;
        }
    }
    const int64_t t = t0 + lane;
    dvec[(size_t)h * Tpad + t] = mine;
    lse2[(size_t)h * Tpad + t] = t < T ? lse[(size_t)h * T + t] * 1.4426950408889634f : 0.f;
}

struct BwdWorkspace {
    size_t stat_bytes, total;
    size_t dq_acc_bytes, dkv_acc_bytes;   // fused form only: fp32 accumulators of dQ and of dK, dV (each)
    int64_t Tpad;
};
static BwdWorkspace bwd_workspace(int64_t T, int hq, int hkv = 0, int d = 0, bool fused = false) {
    BwdWorkspace w;
    w.Tpad = (T + 127) / 128 * 128;
    w.stat_bytes = ((size_t)hq * w.Tpad * sizeof(float) + 255) & ~(size_t)255;
    w.total = 2 * w.stat_bytes;
    w.dq_acc_bytes = w.dkv_acc_bytes = 0;
    if (fused) {
        if (d == 128) w.dq_acc_bytes = ((size_t)T * hq * d * sizeof(float) + 255) & ~(size_t)255;
        w.dkv_acc_bytes = ((size_t)T * hkv * d * sizeof(float) + 255) & ~(size_t)255;
        w.total += w.dq_acc_bytes + 2 * w.dkv_acc_bytes;
    }
    return w;
}
// A plan with pair tiles selects the accumulating forms: at head_dim 128 the fused kernel (dQ, dK, dV accumulated in
// fp32), at head_dim 256 the dV and dK passes over pair tiles (dK, dV accumulated in fp32; the dQ pass is unchanged).
static bool use_fused(const libra_plan_t* plan, const libra_dims* dims) {
    return plan->dir[2].enabled && (dims->head_dim == 128 || dims->head_dim == 256);
}

template <typename Kernel>
static int set_smem(Kernel k, int bytes) {
    return cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess ? LIBRA_OK
                                                                                                      : LIBRA_ERR_CUDA;
}

template <int D>
static int launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                      const CUtensorMap& tdq,
                      const DkvParams& pa, int Wa, const DqParams& pb, int Wb, libra_plan_t* mp, cudaStream_t s) {
    constexpr int kSlot = D == 128 ? 2 : 3;
    if (!cfg_done(kSlot)) {   // per device
        if (set_smem(k_attn_bwd_dkdv<D>, DkvSmem<D>::kBytes) != LIBRA_OK) return LIBRA_ERR_CUDA;
        if (set_smem(k_attn_bwd_dq<D>, DqSmem<D>::kBytes) != LIBRA_OK) return LIBRA_ERR_CUDA;
        if (!regs_pool_ok(k_attn_bwd_dkdv<D>, 128, kDkvRegsDs, 128, kDkvRegsOther)) return LIBRA_ERR_UNSUPPORTED;
        if (!regs_pool_ok(k_attn_bwd_dq<D>, 128 * kDqGroups, kDqRegsCompute, 128, kDqRegsOther)) return LIBRA_ERR_UNSUPPORTED;
        cfg_mark(kSlot);
    }
    time_begin(mp, 1, s);
    k_attn_bwd_dkdv<D><<<Wa, kBwdThreads, DkvSmem<D>::kBytes, s>>>(tq, tk, tv, tdo, pa);
    time_end(mp, 1, s);
    time_begin(mp, 2, s);
    k_attn_bwd_dq<D><<<Wb, kDqThreads, DqSmem<D>::kBytes, s>>>(tq, tk, tv, tdo, tdq, pb);
    time_end(mp, 2, s);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace libra

using namespace libra;


extern "C" size_t libra_attn_pool_bwd_workspace_bytes(const libra_plan_t* plan, const libra_dims* dims) {
    if (!plan || !dims || dims->hq <= 0 || dims->hkv <= 0 ||
        (dims->head_dim != 64 && dims->head_dim != 128 && dims->head_dim != 256))
        return 0;
    return bwd_workspace(plan->T, dims->hq, dims->hkv, dims->head_dim, use_fused(plan, dims)).total;
}

// fp32 tensor [T, H, 128] viewed as (128, H, T); box = 32 floats x 1 head x 32 rows, 128-byte swizzle.
static int make_f32_thd_map(CUtensorMap* m, const void* base, int64_t T, int H) {
    // three dimensions through the same driver entry point as the bf16 maps
    return libra::make_f32_3d_map(m, base, T, H, 128, 32, 32);
}

static int launch_fused(const void* q_dev, const void* k_dev, const void* v_dev, const void* dout_dev, void* dq_dev,
                        void* dk_dev, void* dv_dev, uint8_t* ws_dev, const BwdWorkspace& ws, const libra_plan_t* plan,
                        const libra_dims* dims, float scale, cudaStream_t s) {
    const PlanDir& d = plan->dir[2];
    const int64_t T = plan->T;
    if (d.tile != kBlk || d.H != dims->hkv) return LIBRA_ERR_PLAN_MISMATCH;
    if (d.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;
    float* dvec = reinterpret_cast<float*>(ws_dev);
    float* lse2 = reinterpret_cast<float*>(ws_dev + ws.stat_bytes);
    float* dq_acc = reinterpret_cast<float*>(ws_dev + 2 * ws.stat_bytes);
    float* dk_acc = reinterpret_cast<float*>(ws_dev + 2 * ws.stat_bytes + ws.dq_acc_bytes);
    float* dv_acc = reinterpret_cast<float*>(ws_dev + 2 * ws.stat_bytes + ws.dq_acc_bytes + ws.dkv_acc_bytes);
    CUtensorMap tq, tk, tv, tdo, tacc, tdkacc, tdvacc;
    int rc = make_thd_map(&tq, q_dev, T, dims->hq, 128, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k_dev, T, dims->hkv, 128, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v_dev, T, dims->hkv, 128, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdo, dout_dev, T, dims->hq, 128, kBlk);
    if (rc == LIBRA_OK) rc = make_f32_thd_map(&tacc, dq_acc, T, dims->hq);
    if (rc == LIBRA_OK) rc = make_f32_thd_map(&tdkacc, dk_acc, T, dims->hkv);
    if (rc == LIBRA_OK) rc = make_f32_thd_map(&tdvacc, dv_acc, T, dims->hkv);
    if (rc != LIBRA_OK) return rc;
    if (!cfg_done(4)) {
        if (set_smem(k_attn_bwd_fused, FusedSmem::kBytes) != LIBRA_OK) return LIBRA_ERR_CUDA;
        {   // the register pool: what warps 12-15 release must cover what the exp and dS groups ask for
            cudaFuncAttributes a;
            if (cudaFuncGetAttributes(&a, k_attn_bwd_fused) != cudaSuccess) return LIBRA_ERR_CUDA;
            const long long wanted = 256LL * (kFuRegsExp - a.numRegs) + 128LL * (kFuRegsDs - a.numRegs);
            if (a.numRegs < kFuRegsOther || wanted > 128LL * (a.numRegs - kFuRegsOther)) return LIBRA_ERR_UNSUPPORTED;
        }
        cfg_mark(4);
    }
    libra_plan_t* mp = const_cast<libra_plan_t*>(plan);
    FusedParams fp;
    fp.dq_acc = dq_acc; fp.dk_acc = dk_acc; fp.dv_acc = dv_acc;
    fp.lse2 = lse2; fp.dvec = dvec;
    fp.cta_offsets = d.d_cta_offsets; fp.cta_tiles = d.d_cta_exec;
    fp.u_blk = d.d_u_blk; fp.u_chunk = d.d_u_chunk; fp.tok_end = plan->d_tok_end;
    fp.T = T; fp.Tpad = ws.Tpad; fp.NU = d.NB;
    fp.hq = dims->hq; fp.hkv = dims->hkv; fp.R = d.chunk / d.tile;
    fp.scale_log2 = scale * 1.4426950408889634f;
    fp.status = plan->d_status + 2; fp.plan_status = plan->d_status;
    fp.wait_limit_ns = plan->wait_limit_ns; fp.inject_stall = plan->inject_stall;
    fp.busy = d.d_busy;
    fp.tile_ns = d.d_tile_ns;
    time_begin(mp, 4, s);
    cudaMemsetAsync(dq_acc, 0, ws.dq_acc_bytes + 2 * ws.dkv_acc_bytes, s);   // the three accumulators are contiguous
    k_attn_bwd_fused<<<d.W, kFusedThreads, FusedSmem::kBytes, s>>>(tq, tk, tv, tdo, tacc, tdkacc, tdvacc, fp);
    time_end(mp, 4, s);
    time_begin(mp, 5, s);
    const int64_t nq8 = T * dims->hq * 128 / 8, nk8 = T * dims->hkv * 128 / 8;
    k_bwd_fused_finish<<<(unsigned)((nq8 + 255) / 256), 256, 0, s>>>(dq_acc, (__nv_bfloat16*)dq_dev, nq8, scale);
    k_bwd_fused_finish<<<(unsigned)((nk8 + 255) / 256), 256, 0, s>>>(dk_acc, (__nv_bfloat16*)dk_dev, nk8, scale);
    k_bwd_fused_finish<<<(unsigned)((nk8 + 255) / 256), 256, 0, s>>>(dv_acc, (__nv_bfloat16*)dv_dev, nk8, 1.0f);
    time_end(mp, 5, s);
    count_launch(4);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_attn_pool_bwd(const void* q_dev, const void* k_dev, const void* v_dev, const void* out_dev,
                                   const float* lse_dev, const void* dout_dev, const int32_t* cu_seqlens_dev,
                                   const libra_plan_t* plan, void* dq_dev, void* dk_dev, void* dv_dev,
                                   void* workspace_dev, const libra_dims* dims, void* stream) {
    if (!q_dev || !k_dev || !v_dev || !out_dev || !lse_dev || !dout_dev || !cu_seqlens_dev || !plan || !dq_dev ||
        !dk_dev || !dv_dev || !workspace_dev || !dims)
        return LIBRA_ERR_INVALID_ARG;
    if (dims->hq <= 0 || dims->hkv <= 0 || dims->hq % dims->hkv) return LIBRA_ERR_INVALID_ARG;
    if (dims->head_dim != 64 && dims->head_dim != 128 && dims->head_dim != 256) return LIBRA_ERR_UNSUPPORTED;
    const PlanDir& dq_dir = plan->dir[0];
    const PlanDir& dkv_dir = plan->dir[1];
    const bool fused = use_fused(plan, dims);
    if (plan->T != dims->total_tokens) return LIBRA_ERR_PLAN_MISMATCH;
    if (fused && dims->head_dim == 256) {   // the dQ pass walks the query-major lists
        const PlanDir& pd = plan->dir[2];
        if (!dq_dir.enabled || dq_dir.tile != 2 * kBlk || dims->hq % dq_dir.H) return LIBRA_ERR_PLAN_MISMATCH;
        if (pd.tile != kBlk || pd.H != dims->hkv) return LIBRA_ERR_PLAN_MISMATCH;
        if (pd.W > plan->sm_count || dq_dir.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;
    }
    if (!fused) {
        if (!dq_dir.enabled || !dkv_dir.enabled) return LIBRA_ERR_PLAN_MISMATCH;
        if (dkv_dir.tile != kBlk || dq_dir.tile != 2 * kBlk) return LIBRA_ERR_UNSUPPORTED;
        if (dkv_dir.H != dims->hkv) return LIBRA_ERR_PLAN_MISMATCH;
        if (dims->hq % dq_dir.H) return LIBRA_ERR_INVALID_ARG;
        if (dkv_dir.W > plan->sm_count || dq_dir.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;
    }
    if (((uintptr_t)q_dev | (uintptr_t)k_dev | (uintptr_t)v_dev | (uintptr_t)out_dev | (uintptr_t)dout_dev |
         (uintptr_t)dq_dev | (uintptr_t)dk_dev | (uintptr_t)dv_dev) & 15)
        return LIBRA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev & 255) return LIBRA_ERR_INVALID_ARG;
    if (int rcd = check_plan_device(plan); rcd != LIBRA_OK) return rcd;

    const int D = dims->head_dim;
    const int64_t T = plan->T;
    const BwdWorkspace ws = bwd_workspace(T, dims->hq, dims->hkv, D, fused);
    float* dvec = reinterpret_cast<float*>(workspace_dev);
    float* lse2 = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + ws.stat_bytes);
    cudaStream_t s = (cudaStream_t)stream;
    cudaMemsetAsync(plan->d_status + 2, 0, sizeof(int), s);   // the word reports the most recent launch

    const float scale = dims->softmax_scale > 0.f ? dims->softmax_scale : 1.0f / sqrtf((float)D);
    if (D == 256) {   // row statistics, then the three passes of the 256-wide kernel
        libra_plan_t* mp256 = const_cast<libra_plan_t*>(plan);
        time_begin(mp256, 3, s);
        const int64_t warps = ws.Tpad / 32 * dims->hq;
        k_bwd_prep<256><<<(unsigned)((warps * 32 + 255) / 256), 256, 0, s>>>(
            (const __nv_bfloat16*)out_dev, (const __nv_bfloat16*)dout_dev, lse_dev, T, ws.Tpad, dims->hq, dvec, lse2);
        count_launch();
        time_end(mp256, 3, s);
        float* dk_acc = nullptr;
        float* dv_acc = nullptr;
        if (fused) {
            dk_acc = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + 2 * ws.stat_bytes);
            dv_acc = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + 2 * ws.stat_bytes + ws.dkv_acc_bytes);
            cudaMemsetAsync(dk_acc, 0, 2 * ws.dkv_acc_bytes, s);
        }
        int rc256 = launch_bwd_d256(q_dev, k_dev, v_dev, dout_dev, dq_dev, dk_dev, dv_dev, lse2, dvec, ws.Tpad, dk_acc,
                                    dv_acc, plan, dims, scale, s);
        if (rc256 == LIBRA_OK && fused) {
            time_begin(mp256, 5, s);
            const int64_t nk8 = T * dims->hkv * 256 / 8;
            k_bwd_fused_finish<<<(unsigned)((nk8 + 255) / 256), 256, 0, s>>>(dk_acc, (__nv_bfloat16*)dk_dev, nk8, scale);
            k_bwd_fused_finish<<<(unsigned)((nk8 + 255) / 256), 256, 0, s>>>(dv_acc, (__nv_bfloat16*)dv_dev, nk8, 1.0f);
            time_end(mp256, 5, s);
            count_launch(2);
            if (cudaGetLastError() != cudaSuccess) rc256 = LIBRA_ERR_CUDA;
        }
        return rc256;
    }
    CUtensorMap tq, tk, tv, tdo, tdq;
    int rc = make_thd_map(&tq, q_dev, T, dims->hq, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdo, dout_dev, T, dims->hq, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdq, dq_dev, T, dims->hq, D, kBlk);
    if (rc != LIBRA_OK) return rc;

    libra_plan_t* mp0 = const_cast<libra_plan_t*>(plan);
    time_begin(mp0, 3, s);
    {
        const int64_t warps = ws.Tpad / 32 * dims->hq;
        const unsigned grid = (unsigned)((warps * 32 + 255) / 256);
        if (D == 128)
            k_bwd_prep<128><<<grid, 256, 0, s>>>((const __nv_bfloat16*)out_dev, (const __nv_bfloat16*)dout_dev, lse_dev,
                                                 T, ws.Tpad, dims->hq, dvec, lse2);
        else
            k_bwd_prep<64><<<grid, 256, 0, s>>>((const __nv_bfloat16*)out_dev, (const __nv_bfloat16*)dout_dev, lse_dev,
                                                T, ws.Tpad, dims->hq, dvec, lse2);
        count_launch();
    }
    time_end(mp0, 3, s);
    if (fused)
        return launch_fused(q_dev, k_dev, v_dev, dout_dev, dq_dev, dk_dev, dv_dev, reinterpret_cast<uint8_t*>(workspace_dev),
                            ws, plan, dims, scale, s);
    DkvParams pa;
    pa.dk = reinterpret_cast<__nv_bfloat16*>(dk_dev);
    pa.dv = reinterpret_cast<__nv_bfloat16*>(dv_dev);
    pa.lse2 = lse2;
    pa.dvec = dvec;
    pa.cta_offsets = dkv_dir.d_cta_offsets;
    pa.cta_tiles = dkv_dir.d_cta_exec;
    pa.tok_end = plan->d_tok_end;
    pa.T = T;
    pa.Tpad = ws.Tpad;
    pa.hq = dims->hq;
    pa.hkv = dims->hkv;
    pa.scale = scale;
    pa.scale_log2 = scale * 1.4426950408889634f;
    pa.status = plan->d_status + 2;
    pa.plan_status = plan->d_status;
    pa.wait_limit_ns = plan->wait_limit_ns;
    pa.inject_stall = plan->inject_stall;
    pa.busy = dkv_dir.d_busy;
    DqParams pb;
    pb.dq = reinterpret_cast<__nv_bfloat16*>(dq_dev);
    pb.lse2 = lse2;
    pb.dvec = dvec;
    pb.cta_offsets = dq_dir.d_cta_offsets;
    pb.cta_tiles = dq_dir.d_cta_exec;
    pb.tok_start = plan->d_tok_start;
    pb.T = T;
    pb.Tpad = ws.Tpad;
    pb.hq = dims->hq;
    pb.hkv = dims->hkv;
    pb.H = dq_dir.H;
    pb.scale = scale;
    pb.scale_log2 = scale * 1.4426950408889634f;
    pb.status = plan->d_status + 2;
    pb.plan_status = plan->d_status;
    pb.wait_limit_ns = plan->wait_limit_ns;
    pb.inject_stall = plan->inject_stall;
    pb.busy = dq_dir.d_busy2;
    libra_plan_t* mp = const_cast<libra_plan_t*>(plan);
    return D == 128 ? launch_bwd<128>(tq, tk, tv, tdo, tdq, pa, dkv_dir.W, pb, dq_dir.W, mp, s)
                    : launch_bwd<64>(tq, tk, tv, tdo, tdq, pa, dkv_dir.W, pb, dq_dir.W, mp, s);
}
