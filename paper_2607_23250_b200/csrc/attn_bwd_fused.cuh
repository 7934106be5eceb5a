// Fused backward kernel (included by attn_bwd.cu): dQ, dK and dV of a pair tile in one pass, five GEMMs per
// 128 x 128 cell instead of the seven of the two-kernel form (S and dP are computed once).
//
// A unit is a pair tile: 128 keys of one kv head against the query row blocks of one query chunk, for every
// query head of the kv head's group.  K and V stay in shared memory, dK and dV accumulate in TMEM over the
// unit; every iteration (one query head, one 128-row query block) also yields that block's dQ contribution,
// which leaves through shared memory as a bulk tensor reduce-add into an fp32 accumulator in global memory.
// dK and dV of the unit are added to fp32 accumulators as well (a key block meets several query chunks); a
// last kernel scales and rounds the three accumulators to bf16.  The plan runs the pair tiles in id order
// (head, query chunk, key block) on all CTAs in step, so the accumulator rows and the Q / dO tiles of a query
// chunk are shared by the CTAs while they are in L2.
//
// Keys sit in TMEM lanes:
//   S^T  = K Q^T   (SS) -> X     P^T  = exp2(S^T c - LSE)      -> bf16, own TMEM columns    dV += P^T dO  (A in TMEM)
//   dP^T = V dO^T  (SS) -> X     dS^T = P^T o (dP^T - D)       -> bf16, own TMEM columns    dK += dS^T Q  (A in TMEM)
//                                                               and the same tile in shared memory:
//   dQ   = dS K    (SS, A = the shared-memory dS^T read along its contiguous query axis) -> Y
// TMEM: X | Y | dK | dV = 128 + 128 + 128 + 128 columns.  X holds S^T, then dP^T (fp32), and is free again as soon
// as it has been READ, so S^T(it+1) and dP^T(it+1) run ahead.  Y holds P^T and dS^T (bf16, 64 columns each) and,
// once dV(it) and dK(it) have consumed them, receives dQ(it) (fp32, 128 columns: the MMAs run in issue order, so
// the overwrite needs no extra barrier); P^T(it+1), already computed in registers, is written as soon as dQ(it) has
// been read out.
// Roles (512 threads): warps 0-3 and 4-7 exp groups (64 query columns of S^T each; 64 head-dim columns of dQ
// each), 8-11 dS group, 12 TMA thread, 13 MMA thread, 14-15 only hand their registers over.
#pragma once

namespace libra {

constexpr int kFusedThreads = 512;
constexpr int kFuTmaWarp = 12, kFuMmaWarp = 13;
// setmaxnreg budgets: 512 threads x 128 compiled registers = 256 x 144 (exp groups: P^T(it) and dQ(it-1) held
// together) + 128 x 144 (dS group) + 128 x 80
constexpr int kFuRegsExp = 144, kFuRegsDs = 144, kFuRegsOther = 80;

struct FusedSmem {
    static constexpr int kTile = 32768;        // 128 x 128 bf16
    static constexpr int kHalf = 16384;
    static constexpr int kQStages = 2;         // Q(it) lives from S(it) to dK(it), which runs behind dP(it+1)
    static constexpr int kKOff = 0;
    static constexpr int kVOff = kTile;
    static constexpr int kQOff = 2 * kTile;
    static constexpr int kDoOff = kQOff + kQStages * kTile;
    static constexpr int kDsOff = kDoOff + kTile;          // dS^T tile (bf16, the operand layout of K / V tiles)
    static constexpr int kStageOff = kDsOff + kTile;       // dQ staging: per exp warp a tile of 32 rows x 32 floats, swizzled
    static constexpr int kLseOff = kStageOff + 2 * kHalf;  // per Q stage: lse2[128]
    static constexpr int kDvecOff = kLseOff + kQStages * 512;   // two buffers: dvec(it+1) lands while dvec(it) is read
    static constexpr int kBarOff = kDvecOff + 2 * 512;
    // kv_full, kv_empty, q_full[2], q_empty[2], do_full, do_empty, s_full, x_free1, dp_full, x_free2, dq_full,
    // y_free, p_half, p_ready, ds_ready, dkv_full, dkv_empty, drain
    static constexpr int kNumBars = 2 + 2 * kQStages + 16;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static_assert(kBytes <= kSmemMax, "exceeds the shared memory of an sm_100 CTA");
};

struct FusedParams {
    float* dq_acc;      // [T, Hq, 128]   fp32, zero on entry
    float* dk_acc;      // [T, Hkv, 128]  fp32, zero on entry
    float* dv_acc;
    const float* lse2;  // [Hq, Tpad]  LSE * log2(e)
    const float* dvec;  // [Hq, Tpad]  D_i
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* u_blk;     // key block of pair-block u
    const int32_t* u_chunk;   // query chunk of pair-block u
    const int32_t* tok_end;
    int64_t T, Tpad, NU;
    int hq, hkv, R;           // R = row blocks per query chunk
    float scale_log2;
    int* status;
    const int* plan_status;
    uint32_t wait_limit_ns;
    int inject_stall;
    uint64_t* busy;
    uint32_t* tile_ns;        // [tiles] time spent on each pair tile (first exp thread), ns
};

// The row blocks [i0, i1] a pair tile walks for every head of its group.
struct FusedUnit {
    int kvh, i0, n_blk;
    int64_t k0;
};
__device__ __forceinline__ FusedUnit fused_unit(const FusedParams& p, int t) {
    FusedUnit u;
    const int pb = (int)(t % p.NU);
    u.kvh = (int)(t / p.NU);
    const int j = p.u_blk[pb], c = p.u_chunk[pb];
    u.k0 = (int64_t)j * kBlk;
    const int last = last_q_block(p.tok_end, p.T, u.k0);
    const int lo = c * p.R > j ? c * p.R : j;
    const int hi = c * p.R + p.R - 1 < last ? c * p.R + p.R - 1 : last;
    u.i0 = lo;
    u.n_blk = hi - lo + 1;
    return u;
}

// Bulk tensor reduce-add of a shared-memory tile into global memory (fp32 elements, given by the tensor map).
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* m, const void* smem_src, int c0, int c1, int c2) {
    asm volatile("cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%2, %3, %4}], [%1];" ::"l"(
                     reinterpret_cast<uint64_t>(m)),
                 "r"(smem_u32(smem_src)), "r"(c0), "r"(c1), "r"(c2)
                 : "memory");
}

// dQ of one iteration: out of Y (query rows in lanes; this thread's 64 head-dim columns at `taddr`) into registers,
// after which Y is released.
__device__ __forceinline__ bool fused_read_dq(uint64_t* bar_dqfull, uint64_t* bar_yfree, uint32_t i, volatile int* ctl,
                                              uint32_t taddr, uint32_t (&dqv)[64]) {
    if (!warp_wait(bar_dqfull, i & 1, ctl)) return false;
    tc_fence_after();
    tmem_ld32(taddr, dqv);
    tmem_ld32(taddr + 32, dqv + 32);
    tmem_ld_wait();
    tc_fence_before();
    mbar_arrive(bar_yfree);
    return true;
}
// ... and from the registers through the warp's staging tile (32 rows of 128 bytes, 128-byte swizzle) into the fp32
// accumulator: one bulk tensor reduce-add of 32 head-dim columns (from column col0), rows row0 .. row0 + 31 of head h.
// The reduce that last used the tile must have finished reading it.
__device__ __forceinline__ void fused_stage_dq(const CUtensorMap* tm, uint8_t* stage, const uint32_t* dq, int lane,
                                               int col0, int h, int row0) {
    if (lane == 0) tma_store_wait_read();
    __syncwarp();
#pragma unroll
    for (int ch = 0; ch < 8; ++ch) {
        const int at = lane * 128 + ((ch ^ (lane & 7)) << 4);
        *reinterpret_cast<uint4*>(stage + at) = make_uint4(dq[4 * ch], dq[4 * ch + 1], dq[4 * ch + 2], dq[4 * ch + 3]);
    }
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        tma_reduce_add_3d(tm, stage, col0, h, row0);
        tma_store_commit();
    }
}

__global__ void __launch_bounds__(kFusedThreads, 1)
k_attn_bwd_fused(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                 const __grid_constant__ CUtensorMap tm_dqacc, const __grid_constant__ CUtensorMap tm_dkacc,
                 const __grid_constant__ CUtensorMap tm_dvacc, const FusedParams p) {
    using L = FusedSmem;
    constexpr int D = 128, QS = L::kQStages;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_kvfull = bars + 0;
    uint64_t* bar_kvempty = bars + 1;
    uint64_t* bar_qfull = bars + 2;             // [QS]
    uint64_t* bar_qempty = bar_qfull + QS;      // [QS] dK(it) has run: Q stage free, TMEM dS^T columns free
    uint64_t* b2 = bar_qempty + QS;
    uint64_t* bar_dofull = b2 + 0;
    uint64_t* bar_doempty = b2 + 1;    // dV(it) has run: the dO tile is free
    uint64_t* bar_sfull = b2 + 2;
    uint64_t* bar_xfree1 = b2 + 3;     // S^T(it) has been read out of X: dP^T(it) may overwrite it
    uint64_t* bar_dpfull = b2 + 4;
    uint64_t* bar_xfree2 = b2 + 5;     // dP^T(it) has been read out: S^T(it+1) may overwrite it
    uint64_t* bar_dqfull = b2 + 6;     // dQ(it) is in Y (so dV(it), dK(it) and dQ(it) have all run)
    uint64_t* bar_yfree = b2 + 7;      // dQ(it) has been read out of Y: P^T(it+1), then dS^T(it+1), may be written
    uint64_t* bar_phalf = b2 + 8;
    uint64_t* bar_pready = b2 + 9;
    uint64_t* bar_dsready = b2 + 10;   // dS^T(it) is in TMEM and in shared memory
    uint64_t* bar_dkvfull = b2 + 11;
    uint64_t* bar_dkvempty = b2 + 12;
    uint64_t* bar_drain = b2 + 13;
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
        mbar_init(bar_kvfull, 1);
        mbar_init(bar_kvempty, 1);
        for (int s = 0; s < QS; ++s) { mbar_init(&bar_qfull[s], 1); mbar_init(&bar_qempty[s], 1); }
        mbar_init(bar_dofull, 1);
        mbar_init(bar_doempty, 1);
        mbar_init(bar_sfull, 1);
        mbar_init(bar_xfree1, 256);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_xfree2, 128);
        mbar_init(bar_dqfull, 1);
        mbar_init(bar_yfree, 256);
        mbar_init(bar_phalf, 256);
        mbar_init(bar_pready, 256);
        mbar_init(bar_dsready, 128);
        mbar_init(bar_dkvfull, 1);
        mbar_init(bar_dkvempty, 256);
        mbar_init(bar_drain, 1);
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit_ns;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == kFuMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kFuTmaWarp && lane == 0) {
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
        prefetch_tmap(&tm_dqacc);
        prefetch_tmap(&tm_dkacc);
        prefetch_tmap(&tm_dvacc);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    constexpr uint32_t kColX = 0, kColY = 128, kColP = 128, kColDS = 192, kColDK = 256, kColDV = 384;

    const int unit_begin = p.cta_offsets[cta];
    const int unit_end = p.cta_offsets[cta + 1];
    const int G = p.hq / p.hkv;

    if (warp > kFuMmaWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFuRegsOther));
    } else if (warp == kFuTmaWarp) {
        // ---------------- TMA producer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFuRegsOther));
        if (elect_one()) {
            uint32_t ucnt = 0, it_all = 0, n_do = 0;
            bool ok = true;
            for (int idx = unit_begin; idx < unit_end && ok && !p.inject_stall; ++idx) {
                const FusedUnit u = fused_unit(p, p.cta_tiles[idx]);
                ok = mbar_wait(bar_kvempty, (ucnt & 1) ^ 1, abort_flag);
                if (!ok) break;
                mbar_arrive_expect_tx(bar_kvfull, 2 * L::kTile);
                for (int half = 0; half < 2; ++half) {
                    tma_load_3d(smem + L::kKOff + half * L::kHalf, &tm_k, bar_kvfull, half * 64, u.kvh, (int)u.k0);
                    tma_load_3d(smem + L::kVOff + half * L::kHalf, &tm_v, bar_kvfull, half * 64, u.kvh, (int)u.k0);
                }
                ++ucnt;
                const int n_it = G * u.n_blk;
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    const int h = u.kvh * G + it / u.n_blk;
                    const int qb = (u.i0 + it % u.n_blk) * kBlk;
                    const uint32_t qs = it_all % QS;
                    ok = mbar_wait(&bar_qempty[qs], ((it_all / QS) & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(&bar_qfull[qs], L::kTile + 512);
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(smem + L::kQOff + qs * L::kTile + half * L::kHalf, &tm_q, &bar_qfull[qs], half * 64, h, qb);
                    bulk_load_1d(smem + L::kLseOff + qs * 512, p.lse2 + (size_t)h * p.Tpad + qb, 512, &bar_qfull[qs]);
                    ok = mbar_wait(bar_doempty, (it_all & 1) ^ 1, abort_flag);
                    if (!ok) { mbar_wait_drain(&bar_qfull[qs], (it_all / QS) & 1, kDrainNs); break; }
                    mbar_arrive_expect_tx(bar_dofull, L::kTile + 512);
                    ++n_do;
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(smem + L::kDoOff + half * L::kHalf, &tm_do, bar_dofull, half * 64, h, qb);
                    bulk_load_1d(smem + L::kDvecOff + (it_all & 1) * 512, p.dvec + (size_t)h * p.Tpad + qb, 512, bar_dofull);
                }
            }
            if (!ok || abort_flag[0]) {   // give-up path: the copies already issued land before shared memory is released
                if (ucnt > 0) mbar_wait_drain(bar_kvfull, (ucnt - 1) & 1, kDrainNs);
                for (uint32_t b = 1; b <= (uint32_t)QS && b <= it_all; ++b)
                    mbar_wait_drain(&bar_qfull[(it_all - b) % QS], ((it_all - b) / QS) & 1, kDrainNs);
                if (n_do > 0) mbar_wait_drain(bar_dofull, (n_do - 1) & 1, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp == kFuMmaWarp) {
        // ---------------- MMA issuer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFuRegsOther));
        if (elect_one()) {
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // S^T, dP^T: both operands K-major
            constexpr uint32_t idesc_acc = make_idesc(128, D, 0, 1);   // dV, dK: A from TMEM, B MN-major
            constexpr uint32_t idesc_dq = make_idesc(128, D, 1, 1);    // dQ: A = dS^T read along queries, B = K, both MN-major
            const uint32_t sb = smem_u32(smem);
            uint32_t ucnt = 0, it_all = 0;
            bool ok = true;
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);          // K-major view of a tile at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kHalf, 1024);    // MN-major view
            auto issue_kmajor = [&](uint32_t a_off, uint32_t b_off) {
                const uint64_t da = sdesc_advance(kdesc0, a_off), db = sdesc_advance(kdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * L::kHalf + (kk % 4) * 32;
                    mma_ss(tmem_base + kColX, sdesc_advance(da, off), sdesc_advance(db, off), idesc_s, kk > 0);
                }
            };
            auto issue_acc = [&](uint32_t d_col, uint32_t a_col, uint32_t b_off, bool accumulate) {
                const uint64_t db = sdesc_advance(mdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < 8; ++kk)
                    mma_ts(tmem_base + d_col, tmem_base + a_col + kk * 8, sdesc_advance(db, kk * 2048), idesc_acc,
                           (accumulate || kk > 0) ? 1u : 0u);
            };
            for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
                const FusedUnit u = fused_unit(p, p.cta_tiles[idx]);
                const int n_it = G * u.n_blk;
                ok = mbar_wait(bar_kvfull, ucnt & 1, abort_flag);
                if (!ok) break;
                // S(0): X is free once dP of the previous unit's last iteration has been read
                ok = mbar_wait(&bar_qfull[it_all % QS], (it_all / QS) & 1, abort_flag);
                if (ok && it_all > 0) ok = mbar_wait(bar_xfree2, (it_all - 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                issue_kmajor(L::kKOff, L::kQOff + (it_all % QS) * L::kTile);
                tc_commit(bar_sfull);
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    const uint32_t nx = it_all + 1;
                    const bool more = it + 1 < n_it;
                    // dP(it) over S(it), as soon as the exp groups hold S(it) in registers
                    ok = mbar_wait(bar_dofull, it_all & 1, abort_flag);
                    if (ok) ok = mbar_wait(bar_xfree1, it_all & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_kmajor(L::kVOff, L::kDoOff);
                    tc_commit(bar_dpfull);
                    // S(it+1) over dP(it), as soon as the dS group holds dP(it) in registers
                    if (more) {
                        ok = mbar_wait(&bar_qfull[nx % QS], (nx / QS) & 1, abort_flag);
                        if (ok) ok = mbar_wait(bar_xfree2, it_all & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        issue_kmajor(L::kKOff, L::kQOff + (nx % QS) * L::kTile);
                        tc_commit(bar_sfull);
                    }
                    // dV(it) += P^T dO
                    ok = mbar_wait(bar_pready, it_all & 1, abort_flag);
                    if (ok && it == 0 && ucnt > 0) ok = mbar_wait(bar_dkvempty, (ucnt - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_acc(kColDV, kColP, L::kDoOff, it > 0);
                    tc_commit(bar_doempty);
                    // dK(it) += dS^T Q from the TMEM copy of dS^T, then dQ(it) = dS K from the shared-memory copy,
                    // into Y over P^T and dS^T: dV(it) and dK(it) precede it in issue order
                    ok = mbar_wait(bar_dsready, it_all & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_acc(kColDK, kColDS, L::kQOff + (it_all % QS) * L::kTile, it > 0);
                    tc_commit(&bar_qempty[it_all % QS]);
                    {
                        const uint64_t da = sdesc_advance(mdesc0, L::kDsOff), db = sdesc_advance(mdesc0, L::kKOff);
#pragma unroll
                        for (int kk = 0; kk < 8; ++kk)   // 16 keys per step
                            mma_ss(tmem_base + kColY, sdesc_advance(da, kk * 2048), sdesc_advance(db, kk * 2048), idesc_dq, kk > 0);
                        tc_commit(bar_dqfull);
                        if (!more) { tc_commit(bar_kvempty); tc_commit(bar_dkvfull); }   // the unit's last MMAs
                    }
                }
                ++ucnt;
            }
            if (!ok || abort_flag[0]) {
                tc_commit(bar_drain);
                mbar_wait_drain(bar_drain, 0, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp >= 8) {
        // ---------------- dS group ----------------
        // Thread r owns key row r: it turns dP^T and P^T (read back as bf16) into dS^T, which goes to TMEM (the A
        // operand of dK) and to shared memory (the A operand of dQ).
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kFuRegsDs));
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_x = tmem_base + lane_addr + kColX;
        const uint32_t t_p = tmem_base + lane_addr + kColP;
        const uint32_t t_ds = tmem_base + lane_addr + kColDS;
        uint8_t* ds_row = smem + L::kDsOff + r * 128;
        uint32_t it_all = 0;
        bool ok = true;
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const FusedUnit u = fused_unit(p, p.cta_tiles[idx]);
            const int n_it = G * u.n_blk;
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const float* dvec = reinterpret_cast<const float*>(smem + L::kDvecOff + (it_all & 1) * 512);
                ok = warp_wait(bar_dofull, it_all & 1, abort_flag) && warp_wait(bar_dpfull, it_all & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t xs[64];   // (dP^T - D) as packed bf16 pairs
                {
                    const uint64_t neg1 = f2_pack(-1.f, -1.f);
#pragma unroll
                    for (int part = 0; part < 2; ++part) {   // 64 columns at a time keeps the live registers down
                        uint32_t dpv[64];
                        tmem_ld32(t_x + part * 64, dpv);
                        tmem_ld32(t_x + part * 64 + 32, dpv + 32);
                        tmem_ld_wait();
                        if (part == 1) {
                            tc_fence_before();
                            mbar_arrive(bar_xfree2);   // dP^T(it) is in registers: S^T(it+1) may take the columns
                        }
#pragma unroll
                        for (int j = 0; j < 64; j += 4) {
                            const ulonglong2 d4 = *reinterpret_cast<const ulonglong2*>(dvec + part * 64 + j);
                            float a0, a1, b0, b1;
                            f2_unpack(f2_fma(d4.x, neg1, f2_pack(__uint_as_float(dpv[j]), __uint_as_float(dpv[j + 1]))), a0, a1);
                            f2_unpack(f2_fma(d4.y, neg1, f2_pack(__uint_as_float(dpv[j + 2]), __uint_as_float(dpv[j + 3]))), b0, b1);
                            xs[part * 32 + (j >> 1)] = pack_bf16x2(a0, a1);
                            xs[part * 32 + (j >> 1) + 1] = pack_bf16x2(b0, b1);
                        }
                    }
                }
                // P^T(it) only appears in Y after dQ(it-1) has been read out of it, and dQ(it-1) ran behind dK(it-1): by
                // the time P^T(it) is seen, both copies of dS^T(it-1) have been consumed
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    ok = warp_wait(half == 0 ? bar_phalf : bar_pready, it_all & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    uint32_t pa[16], pb[16];   // queries 32 half .. and 64 + 32 half ..
                    tmem_ld16(t_p + half * 16, pa);
                    tmem_ld16(t_p + 32 + half * 16, pb);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        pa[j] = mul_bf16x2(pa[j], xs[half * 16 + j]);
                        pb[j] = mul_bf16x2(pb[j], xs[32 + half * 16 + j]);
                    }
                    tmem_st16(t_ds + half * 16, pa);
                    tmem_st16(t_ds + 32 + half * 16, pb);
                    // the same values into the shared-memory tile: row r, 16-byte chunks of 8 queries, 128-byte swizzle;
                    // queries 0..63 in the first 16 KB half of the tile, 64..127 in the second
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const int chunk_a = half * 4 + ch;            // queries 32 half + 8 ch ..
                        *reinterpret_cast<uint4*>(ds_row + ((chunk_a ^ (r & 7)) << 4)) =
                            make_uint4(pa[4 * ch], pa[4 * ch + 1], pa[4 * ch + 2], pa[4 * ch + 3]);
                        *reinterpret_cast<uint4*>(ds_row + L::kHalf + ((chunk_a ^ (r & 7)) << 4)) =
                            make_uint4(pb[4 * ch], pb[4 * ch + 1], pb[4 * ch + 2], pb[4 * ch + 3]);
                    }
                }
                if (!ok) break;
                tmem_st_wait();
                fence_proxy_async_smem();     // the MMA reads the shared-memory tile through the async proxy
                tc_fence_before();
                mbar_arrive(bar_dsready);
            }
        }
    } else {
        // ---------------- exp groups ----------------
        // Thread r of group grp owns key row r and the query columns [64 grp, 64 grp + 64) of S^T; when dQ comes
        // back in Y (query rows in lanes) it owns query row r and the head-dim columns [64 grp, 64 grp + 64).
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kFuRegsExp));
        const int grp = warp >> 2;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_x = tmem_base + lane_addr + kColX;
        const uint32_t t_p = tmem_base + lane_addr + kColP;
        const uint32_t t_y = tmem_base + lane_addr + kColY;
        const int c0 = 64 * grp;
        const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2), neg1 = f2_pack(-1.f, -1.f);
        uint8_t* stage = smem + L::kStageOff + warp * 4096;   // this warp's staging tile: 32 rows x 32 floats
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const uint64_t tile_t0 = threadIdx.x == 0 ? globaltimer_ns() : 0;
            const FusedUnit u = fused_unit(p, p.cta_tiles[idx]);
            const int n_it = G * u.n_blk;
            const int64_t key = u.k0 + r;
            const bool key_ok = key < p.T;
            const int kend = key_ok ? p.tok_end[key] : 0;
            const int min_kend = p.tok_end[u.k0];
            const bool partial = u.k0 + kBlk > p.T;
            int prev_h = 0, prev_qb = 0;
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const int h = u.kvh * G + it / u.n_blk;
                const int qb = (u.i0 + it % u.n_blk) * kBlk;
                const uint32_t qs = it_all % QS;
                const float* lse2 = reinterpret_cast<const float*>(smem + L::kLseOff + qs * 512) + c0;
                const bool need_mask = (qb == u.k0) || (qb + kBlk - 1 >= min_kend) || partial;
                const int j_lo = (int)(key - qb) - c0;
                const int j_hi = kend - 1 - qb - c0;
                ok = warp_wait(&bar_qfull[qs], (it_all / QS) & 1, abort_flag) && warp_wait(bar_sfull, it_all & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t pk[32];   // P^T(it) of this thread's 64 queries, packed, kept until Y is free
                {
                    uint32_t sv[64];
                    tmem_ld32(t_x + c0, sv);
                    tmem_ld32(t_x + c0 + 32, sv + 32);
                    tmem_ld_wait();
                    tc_fence_before();
                    mbar_arrive(bar_xfree1);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        float pf[32];
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            const int jj = half * 32 + j;
                            const ulonglong2 l4 = *reinterpret_cast<const ulonglong2*>(lse2 + jj);
                            float x0, x1, x2, x3;
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(sv[jj]), __uint_as_float(sv[jj + 1])), scale2,
                                             f2_mul(l4.x, neg1)), x0, x1);
                            f2_unpack(f2_fma(f2_pack(__uint_as_float(sv[jj + 2]), __uint_as_float(sv[jj + 3])), scale2,
                                             f2_mul(l4.y, neg1)), x2, x3);
                            pf[j] = ex2_approx(x0);
                            pf[j + 1] = ex2_approx(x1);
                            pf[j + 2] = ex2_approx(x2);
                            pf[j + 3] = ex2_approx(x3);
                        }
                        if (need_mask) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (half * 32 + j < j_lo || half * 32 + j > j_hi) pf[j] = 0.f;
                        }
#pragma unroll
                        for (int j = 0; j < 32; j += 2) pk[half * 16 + (j >> 1)] = pack_bf16x2(pf[j], pf[j + 1]);
                    }
                }
                // dQ(it-1) leaves Y (its MMA ran behind dV(it-1) and dK(it-1), so P^T(it-1) and dS^T(it-1) are spent)
                uint32_t dqv[64];   // this thread's share of dQ(it-1): head-dim columns c0 .. c0 + 63 of query row r
                if (it > 0) {
                    ok = fused_read_dq(bar_dqfull, bar_yfree, it_all - 1, abort_flag, t_y + c0, dqv);
                    if (!ok) break;
                }
                if (it_all > 0) {   // every exp thread has read its part of the last dQ: Y is free
                    ok = warp_wait(bar_yfree, (it_all - 1) & 1, abort_flag);
                    if (!ok) break;
                }
                tc_fence_after();
                tmem_st16(t_p + c0 / 2, pk);
                tmem_st16(t_p + c0 / 2 + 16, pk + 16);
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_phalf);
                mbar_arrive(bar_pready);
                if (it > 0) {
                    fused_stage_dq(&tm_dqacc, stage, dqv, lane, c0, prev_h, prev_qb + (warp & 3) * 32);
                    fused_stage_dq(&tm_dqacc, stage, dqv + 32, lane, c0 + 32, prev_h, prev_qb + (warp & 3) * 32);
                }
                prev_h = h;
                prev_qb = qb;
            }
            if (!ok) break;
            // the unit's last dQ, then its dK and dV
            {
                uint32_t dqv[64];
                ok = fused_read_dq(bar_dqfull, bar_yfree, it_all - 1, abort_flag, t_y + c0, dqv);
                if (!ok) break;
                fused_stage_dq(&tm_dqacc, stage, dqv, lane, c0, prev_h, prev_qb + (warp & 3) * 32);
                fused_stage_dq(&tm_dqacc, stage, dqv + 32, lane, c0 + 32, prev_h, prev_qb + (warp & 3) * 32);
            }
            ++ucnt;
            // ---- unit epilogue: dK and dV of the pair tile are added to the fp32 accumulators ----
            ok = warp_wait(bar_dkvfull, (ucnt - 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t t_dk = tmem_base + lane_addr + kColDK + c0;
            const uint32_t t_dv = tmem_base + lane_addr + kColDV + c0;
            // through the warp's staging tile, like dQ: bulk reduce-adds of 32 key rows x 32 head-dim columns (rows
            // past the end of the pool are dropped by the hardware)
#pragma unroll
            for (int which = 0; which < 2; ++which) {
#pragma unroll
                for (int cc = 0; cc < 64; cc += 32) {
                    uint32_t v[32];
                    tmem_ld32((which == 0 ? t_dk : t_dv) + cc, v);
                    tmem_ld_wait();
                    fused_stage_dq(which == 0 ? &tm_dkacc : &tm_dvacc, stage, v, lane, c0 + cc, u.kvh,
                                   (int)u.k0 + (warp & 3) * 32);
                }
            }
            tc_fence_before();
            mbar_arrive(bar_dkvempty);
            if (threadIdx.x == 0) p.tile_ns[p.cta_tiles[idx]] = (uint32_t)(globaltimer_ns() - tile_t0);
        }
        // every bulk reduce this warp issued has completed before the CTA leaves
        if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == kFuMmaWarp) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (abort_flag[0]) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

// dq = scale * dq_acc, dk = scale * dk_acc, dv = dv_acc, rounded to bf16 (8 elements per thread).
__global__ void k_bwd_fused_finish(const float* __restrict__ acc, __nv_bfloat16* __restrict__ out, int64_t n8, float mul) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= n8) return;
    const float4 a = reinterpret_cast<const float4*>(acc)[2 * i], b = reinterpret_cast<const float4*>(acc)[2 * i + 1];
    uint4 w;
    w.x = pack_bf16x2(a.x * mul, a.y * mul);
    w.y = pack_bf16x2(a.z * mul, a.w * mul);
    w.z = pack_bf16x2(b.x * mul, b.y * mul);
    w.w = pack_bf16x2(b.z * mul, b.w * mul);
    reinterpret_cast<uint4*>(out)[i] = w;
}

}  // namespace libra
