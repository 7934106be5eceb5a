// Backward pool attention for sm_100a.
//
// Three launches: (1) prep: D_i = <dO_i, O_i> and LSE in log2 units, padded to a multiple of 128
// rows; (2) the dK/dV kernel over key-major tiles; (3) the dQ kernel over query-major tiles.
// Splitting dQ off costs two extra GEMMs per block pair (S and dP are recomputed) but needs no
// cross-CTA reduction at all: no fp32 dQ accumulator, no atomics, no shared-memory staging, and
// the result is deterministic.  Both kernels are persistent and warp-specialised (compute warpgroups,
// one TMA thread, one MMA-issuing thread; the dQ kernel also has a store thread) and keep their
// accumulators in TMEM.
//
// dK/dV kernel: a unit is 128 keys x one kv head; K and V stay in shared memory, dK and dV in
// TMEM, while the CTA streams every (query head of the group, 128-row query block) that sees the
// keys.  Keys sit in TMEM lanes:
//   S^T  = K Q^T   (SS)   P^T  = exp2(S^T c - LSE)   -> bf16 over S^T     dV += P^T dO   (A in TMEM)
//   dP^T = V dO^T  (SS)   dS^T = P^T o (dP^T - D)    -> bf16 over dP^T    dK += dS^T Q   (A in TMEM)
// P^T is handed to the dV MMA in two halves, so half of dV(it) runs under the second half's exponentials.
// dQ kernel (attn_bwd_dq.cuh): a unit is 128 query rows x one head; Q and dO are copied once per unit from
// shared memory into TMEM, dQ accumulates in TMEM, the CTA streams the key blocks the rows see (as the
// forward does).  Queries sit in TMEM lanes:
//   S  = Q K^T   dP = dO V^T   dS = P o (dP - D) -> bf16 over dP   dQ += dS K     (every A operand in TMEM)
#include <math.h>

#include "common.h"
#include "ptx.cuh"

namespace libra {

#ifndef LIBRA_DKV_GROUPS
#define LIBRA_DKV_GROUPS 2
#endif
constexpr int kDkvGroups = LIBRA_DKV_GROUPS;            // compute warpgroups: each owns 128 / kDkvGroups query columns
constexpr int kDkvCW = 128 / kDkvGroups;                // S^T / dP^T columns per compute thread
constexpr int kDkvTmaWarp = 4 * kDkvGroups, kDkvMmaWarp = 4 * kDkvGroups + 1;
// two groups: 10 warps at 168 registers; four groups: the producer / MMA warps get a warpgroup of their own
// (two of its warps idle) and hand registers to the compute groups, as in the dQ kernel
constexpr int kBwdThreads = kDkvGroups == 2 ? 320 : (4 * kDkvGroups + 4) * 32;
constexpr int kDkvRegsCompute = 104, kDkvRegsOther = 40;
constexpr int kBlk = 128;
constexpr int kSmemMax = 232448;  // 227 KB per CTA on sm_100

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

#ifdef LIBRA_PROF
// Profiling build only: per-CTA cycle sums of the phases of one thread per role.
__device__ unsigned long long g_bwd_prof[1024 * 24];
struct Prof {
    long long last;
    unsigned long long acc[8];
    __device__ void start() { last = clock64(); for (int i = 0; i < 8; ++i) acc[i] = 0; }
    __device__ void mark(int k) { const long long now = clock64(); acc[k] += now - last; last = now; }
    __device__ void flush(int cta, int base) { for (int i = 0; i < 8; ++i) g_bwd_prof[cta * 24 + base + i] = acc[i]; }
};
#define PROF_DECL Prof prof; prof.start();
#define PROF(k) prof.mark(k);
#define PROF_FLUSH(cond, base) if (cond) prof.flush(cta, base);
#else
#define PROF_DECL
#define PROF(k)
#define PROF_FLUSH(cond, base)
#endif

// =================================================================================================
// dK / dV kernel
// =================================================================================================

template <int D>
struct DkvSmem {
    static constexpr int kHalfBytes = 128 * 128;
    static constexpr int kTileBytes = kHalfBytes * (D / 64);  // 128 x D bf16
    static constexpr int kKOff = 0;
    static constexpr int kVOff = kTileBytes;
    static constexpr int kQOff = 2 * kTileBytes;   // 2 stages
    static constexpr int kDoOff = 4 * kTileBytes;  // 2 stages
    static constexpr int kStatOff = 6 * kTileBytes;  // per Q stage: lse2[128], dvec[128]
    static constexpr int kBarOff = kStatOff + 2 * 1024;
    // kv_full, kv_empty, q_full[2], q_empty[2], do_full[2], do_empty[2], s_full, p_ready, dp_full,
    // ds_ready, dkv_full, dkv_empty, p_half
    static constexpr int kNumBars = 17;
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
    uint64_t* busy;
};

// Query blocks a key block [k0, k0+128) is seen by: diagonal .. block of (end of last key's sample - 1).
__device__ __forceinline__ int last_q_block(const int32_t* tok_end, int64_t T, int64_t k0) {
    const int64_t last_key = (k0 + kBlk <= T ? k0 + kBlk : T) - 1;
    return (tok_end[last_key] - 1) / kBlk;
}

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
k_attn_bwd_dkdv(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
                const DkvParams p) {
    using L = DkvSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_kvfull = bars + 0;
    uint64_t* bar_kvempty = bars + 1;
    uint64_t* bar_qfull = bars + 2;    // [2]
    uint64_t* bar_qempty = bars + 4;   // [2]
    uint64_t* bar_dofull = bars + 6;   // [2]
    uint64_t* bar_doempty = bars + 8;  // [2]
    uint64_t* bar_sfull = bars + 10;
    uint64_t* bar_pready = bars + 11;
    uint64_t* bar_dpfull = bars + 12;
    uint64_t* bar_dsready = bars + 13;
    uint64_t* bar_dkvfull = bars + 14;
    uint64_t* bar_dkvempty = bars + 15;
    uint64_t* bar_phalf = bars + 16;   // the first half of every group's P^T columns is in TMEM
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
        for (int s = 0; s < 2; ++s) {
            mbar_init(&bar_qfull[s], 1);
            mbar_init(&bar_qempty[s], 1);
            mbar_init(&bar_dofull[s], 1);
            mbar_init(&bar_doempty[s], 1);
        }
        mbar_init(bar_sfull, 1);
        mbar_init(bar_pready, 128 * kDkvGroups);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_dsready, 128 * kDkvGroups);
        mbar_init(bar_dkvfull, 1);
        mbar_init(bar_dkvempty, 128 * kDkvGroups);
        mbar_init(bar_phalf, 128 * kDkvGroups);
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
    constexpr uint32_t kColS = 0, kColDP = 128, kColDK = 256, kColDV = 256 + D;

    const int unit_begin = p.cta_offsets[cta];
    const int unit_end = p.cta_offsets[cta + 1];
    const int G = p.hq / p.hkv;

    if (warp > kDkvMmaWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));  // only with four groups
    } else if (warp == kDkvTmaWarp) {
        // ---------------- TMA producer ----------------
        if constexpr (kDkvGroups > 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            uint32_t ucnt = 0, it_all = 0;
            bool ok = true;
            for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
                const int t = p.cta_tiles[idx];
                const int kvh = t % p.hkv;
                const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
                const int i_lo = (int)(k0 / kBlk);
                const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
                ok = mbar_wait(bar_kvempty, (ucnt & 1) ^ 1, abort_flag);
                if (!ok) break;
                {
                    mbar_arrive_expect_tx(bar_kvfull, 2 * L::kTileBytes);
                    for (int half = 0; half < D / 64; ++half) {
                        tma_load_3d(smem + L::kKOff + half * L::kHalfBytes, &tm_k, bar_kvfull, half * 64, kvh, (int)k0);
                        tma_load_3d(smem + L::kVOff + half * L::kHalfBytes, &tm_v, bar_kvfull, half * 64, kvh, (int)k0);
                    }
                }
                ++ucnt;
                const int n_it = G * nblk;
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    const int h = kvh * G + it / nblk;
                    const int qb = (i_lo + it % nblk) * kBlk;
                    const uint32_t st = it_all & 1, par = ((it_all >> 1) & 1) ^ 1;
                    ok = mbar_wait(&bar_qempty[st], par, abort_flag);
                    if (!ok) break;
                    {
                        mbar_arrive_expect_tx(&bar_qfull[st], L::kTileBytes + 1024);
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_3d(smem + L::kQOff + st * L::kTileBytes + half * L::kHalfBytes, &tm_q, &bar_qfull[st],
                                        half * 64, h, qb);
                        bulk_load_1d(smem + L::kStatOff + st * 1024, p.lse2 + (size_t)h * p.Tpad + qb, 512, &bar_qfull[st]);
                        bulk_load_1d(smem + L::kStatOff + st * 1024 + 512, p.dvec + (size_t)h * p.Tpad + qb, 512,
                                     &bar_qfull[st]);
                    }
                    ok = mbar_wait(&bar_doempty[st], par, abort_flag);
                    if (!ok) break;
                    {
                        mbar_arrive_expect_tx(&bar_dofull[st], L::kTileBytes);
                        for (int half = 0; half < D / 64; ++half)
                            tma_load_3d(smem + L::kDoOff + st * L::kTileBytes + half * L::kHalfBytes, &tm_do,
                                        &bar_dofull[st], half * 64, h, qb);
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == kDkvMmaWarp) {
        // ---------------- MMA issuer ----------------
        if constexpr (kDkvGroups > 2) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDkvRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);  // S^T, dP^T: both operands K-major
            constexpr uint32_t idesc_acc = make_idesc(128, D, 0, 1);  // dV, dK: A from TMEM, B MN-major
            const uint32_t sb = smem_u32(smem);
            uint32_t ucnt = 0, it_all = 0;
            bool ok = true;
            PROF_DECL
            TRACE_DECL(17, cta == 0)
            // Base descriptors are built once; every MMA only adds a constant to them.
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);             // K-major view of a tile at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kHalfBytes, 1024);  // MN-major view
            // C[tmem] = A(K-major tile) * B(K-major tile)^T over the head dimension; offsets from smem base
            auto issue_kmajor = [&](uint32_t d_col, uint32_t a_off, uint32_t b_off) {
                const uint64_t da = sdesc_advance(kdesc0, a_off), db = sdesc_advance(kdesc0, b_off);
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * L::kHalfBytes + (kk % 4) * 32;
                    mma_ss(tmem_base + d_col, sdesc_advance(da, off), sdesc_advance(db, off), idesc_s, kk > 0);
                }
            };
            // C[tmem] (+)= A(TMEM, bf16 packed: group c's queries at columns a_col + CW c ..) * B(MN-major tile).
            // `half` 0 / 1 issues the key steps that read the first / second half of every group's columns
            // (the compute groups hand P^T over in two halves), 2 issues all of them.
            auto issue_acc = [&](uint32_t d_col, uint32_t a_col, uint32_t b_off, bool accumulate, int half) {
                const uint64_t db = sdesc_advance(mdesc0, b_off);
                constexpr int kPerGroup = kDkvCW / 16;  // key steps of 16 queries per group
#pragma unroll
                for (int kk = 0; kk < 8; ++kk) {
                    const int within = kk % kPerGroup;
                    if (half != 2 && (within >= kPerGroup / 2) != (half == 1)) continue;
                    mma_ts(tmem_base + d_col, tmem_base + a_col + (kk / kPerGroup) * kDkvCW + within * 8,
                           sdesc_advance(db, kk * 2048), idesc_acc, (accumulate || kk > 0) ? 1u : 0u);
                }
            };
            for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
                const int t = p.cta_tiles[idx];
                const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
                const int i_lo = (int)(k0 / kBlk);
                const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
                const int n_it = G * nblk;
                ok = mbar_wait(bar_kvfull, ucnt & 1, abort_flag);
                if (!ok) break;
                // S(0), dP(0)
                ok = mbar_wait(&bar_qfull[it_all & 1], (it_all >> 1) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                {
                    issue_kmajor(kColS, L::kKOff, L::kQOff + (it_all & 1) * L::kTileBytes);
                    tc_commit(bar_sfull);
                }
                ok = mbar_wait(&bar_dofull[it_all & 1], (it_all >> 1) & 1, abort_flag);
                if (!ok) break;
                {
                    issue_kmajor(kColDP, L::kVOff, L::kDoOff + (it_all & 1) * L::kTileBytes);
                    tc_commit(bar_dpfull);
                }
                for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                    TRACE(20)
                    const uint32_t st = it_all & 1;
                    const uint32_t nx = it_all + 1;
                    const bool more = it + 1 < n_it;
                    // dV(it) += P^T dO
                    PROF(7)
                    ok = mbar_wait(bar_phalf, it_all & 1, abort_flag);   // first half of P^T
                    if (ok && it == 0 && ucnt > 0)                        // previous unit's dK/dV must have been read out
                        ok = mbar_wait(bar_dkvempty, (ucnt - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    issue_acc(kColDV, kColS, L::kDoOff + st * L::kTileBytes, it > 0, 0);
                    ok = mbar_wait(bar_pready, it_all & 1, abort_flag);  // second half, while those MMAs run
                    if (!ok) break;
                    PROF(0)
                    tc_fence_after();
                    {
                        TRACE(10)
                        issue_acc(kColDV, kColS, L::kDoOff + st * L::kTileBytes, it > 0, 1);
                        tc_commit(&bar_doempty[st]);
                        TRACE(11)
                    }
                    // S(it+1)
                    if (more) {
                        PROF(7)
                        ok = mbar_wait(&bar_qfull[nx & 1], (nx >> 1) & 1, abort_flag);
                        if (!ok) break;
                        PROF(1)
                        {
                            issue_kmajor(kColS, L::kKOff, L::kQOff + (nx & 1) * L::kTileBytes);
                            tc_commit(bar_sfull);
                            TRACE(12)
                        }
                    }
                    // dK(it) += dS^T Q
                    PROF(7)
                    ok = mbar_wait(bar_dsready, it_all & 1, abort_flag);
                    if (!ok) break;
                    PROF(2)
                    tc_fence_after();
                    {
                        TRACE(13)
                        issue_acc(kColDK, kColDP, L::kQOff + st * L::kTileBytes, it > 0, 2);
                        tc_commit(&bar_qempty[st]);
                        TRACE(14)
                    }
                    // dP(it+1)
                    if (more) {
                        PROF(7)
                        ok = mbar_wait(&bar_dofull[nx & 1], (nx >> 1) & 1, abort_flag);
                        if (!ok) break;
                        PROF(3)
                        {
                            issue_kmajor(kColDP, L::kVOff, L::kDoOff + (nx & 1) * L::kTileBytes);
                            tc_commit(bar_dpfull);
                            TRACE(15)
                        }
                    }
                }
                if (ok) {
                    tc_commit(bar_dkvfull);
                    tc_commit(bar_kvempty);
                }
                ++ucnt;
            }
            PROF_FLUSH(true, 8)
        }
        __syncwarp();
    } else {
        // ---------------- compute groups ----------------
        if constexpr (kDkvGroups > 2) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kDkvRegsCompute));
        constexpr int CW = kDkvCW;
        const int c = warp >> 2;  // which CW query columns of each key row this group owns
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem_base + lane_addr + kColS + CW * c;
        const uint32_t t_dp = tmem_base + lane_addr + kColDP + CW * c;
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        PROF_DECL
        TRACE_DECL(1 + warp, cta == 0 && lane == 0)
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int kvh = t % p.hkv;
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            const int n_it = G * nblk;
            const int64_t key = k0 + r;
            const bool key_ok = key < p.T;
            const int kend = key_ok ? p.tok_end[key] : 0;
            const int min_kend = p.tok_end[k0];
            const bool partial = k0 + kBlk > p.T;
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const int qb = (i_lo + it % nblk) * kBlk;
                const uint32_t st = it_all & 1, par = (it_all >> 1) & 1;
                const float* lse2 = reinterpret_cast<const float*>(smem + L::kStatOff + st * 1024) + CW * c;
                const float* dvec = lse2 + 128;
                const bool need_mask = (qb == k0) || (qb + kBlk - 1 >= min_kend) || partial;
                const int j_lo = (int)(key - qb) - CW * c;  // first visible column of this group's range
                const int j_hi = kend - 1 - qb - CW * c;    // last visible column
                // ---- exp phase: P^T = exp2(S^T * c - LSE) ----
                ok = mbar_wait(&bar_qfull[st], par, abort_flag) && mbar_wait(bar_sfull, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(0)
                TRACE(2)
                tc_fence_after();
                uint32_t sv[CW];
#pragma unroll
                for (int j = 0; j < CW; j += 32) tmem_ld32(t_s + j, sv + j);
                tmem_ld_wait();
                float pf[CW];
                // two halves: the dV key steps over the first half of this group's queries start while the second
                // half's exponentials are computed (S(it+1) has to wait for all of dV(it), which overwrites nothing
                // but reads P^T from the columns S(it+1) goes to)
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    constexpr int HW = CW / 2;
                    const int b0 = half * HW;
#pragma unroll
                    for (int j = b0; j < b0 + HW; j += 4) {
                        const float4 l4 = *reinterpret_cast<const float4*>(lse2 + j);
                        pf[j] = ex2_sel(fmaf(__uint_as_float(sv[j]), p.scale_log2, -l4.x), j);
                        pf[j + 1] = ex2_sel(fmaf(__uint_as_float(sv[j + 1]), p.scale_log2, -l4.y), j + 1);
                        pf[j + 2] = ex2_sel(fmaf(__uint_as_float(sv[j + 2]), p.scale_log2, -l4.z), j + 2);
                        pf[j + 3] = ex2_sel(fmaf(__uint_as_float(sv[j + 3]), p.scale_log2, -l4.w), j + 3);
                    }
                    if (need_mask) {
#pragma unroll
                        for (int j = b0; j < b0 + HW; ++j)
                            if (j < j_lo || j > j_hi) pf[j] = 0.f;
                    }
                    uint32_t pk[HW / 2];
#pragma unroll
                    for (int j = 0; j < HW; j += 2) pk[j >> 1] = pack_bf16x2(pf[b0 + j], pf[b0 + j + 1]);
                    // packed P^T of this group sits in the first CW / 2 columns of its own S^T range
                    if constexpr (HW == 32) tmem_st16(t_s + b0 / 2, pk); else tmem_st8(t_s + b0 / 2, pk);
                    if (half == 0) {
                        tmem_st_wait();
                        tc_fence_before();
                        mbar_arrive(bar_phalf);
                    }
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_pready);
                PROF(1)
                TRACE(3)
                // ---- dS phase: dS^T = P^T o (dP^T - D), packed over this half's own dP^T columns ----
                ok = mbar_wait(bar_dpfull, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(2)
                TRACE(4)
                tc_fence_after();
                uint32_t dpv[CW];
#pragma unroll
                for (int j = 0; j < CW; j += 32) tmem_ld32(t_dp + j, dpv + j);
                tmem_ld_wait();
                {
                    uint32_t pk[CW / 2];
#pragma unroll
                    for (int j = 0; j < CW; j += 4) {
                        const float4 d4 = *reinterpret_cast<const float4*>(dvec + j);
                        pk[j >> 1] = pack_bf16x2(pf[j] * (__uint_as_float(dpv[j]) - d4.x),
                                                 pf[j + 1] * (__uint_as_float(dpv[j + 1]) - d4.y));
                        pk[(j >> 1) + 1] = pack_bf16x2(pf[j + 2] * (__uint_as_float(dpv[j + 2]) - d4.z),
                                                       pf[j + 3] * (__uint_as_float(dpv[j + 3]) - d4.w));
                    }
                    if constexpr (CW == 64) tmem_st32(t_dp, pk); else tmem_st16(t_dp, pk);
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_dsready);
                PROF(3)
                TRACE(5)
            }
            if (!ok) break;
            // ---- unit epilogue: dK * scale and dV to global ----
            ok = mbar_wait(bar_dkvfull, ucnt & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            constexpr int kCols = D / kDkvGroups;  // columns of dK and dV this group stores
            const uint32_t t_dk = tmem_base + lane_addr + kColDK + c * kCols;
            const uint32_t t_dv = tmem_base + lane_addr + kColDV + c * kCols;
            const size_t gofs = ((size_t)key * p.hkv + kvh) * D + c * kCols;
#pragma unroll
            for (int which = 0; which < 2; ++which) {
                const float mul = which == 0 ? p.scale : 1.0f;
                __nv_bfloat16* gdst = (which == 0 ? p.dk : p.dv) + gofs;
                constexpr int kChunk = kCols < 32 ? kCols : 32;
#pragma unroll
                for (int cc = 0; cc < kCols; cc += kChunk) {
                    uint32_t v[kChunk];
                    if constexpr (kChunk == 32) tmem_ld32((which == 0 ? t_dk : t_dv) + cc, v);
                    else tmem_ld16((which == 0 ? t_dk : t_dv) + cc, v);
                    tmem_ld_wait();
                    if (key_ok) {
#pragma unroll
                        for (int i = 0; i < kChunk; i += 8) {
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
            ++ucnt;
            PROF(4)
        }
        PROF_FLUSH(threadIdx.x == 0, 0)
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == kDkvMmaWarp) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (*abort_flag) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

}  // namespace libra

#include "attn_bwd_dq.cuh"

namespace libra {

// ---- prep kernel ------------------------------------------------------------------------------

// D = <dO, O> per (token, head) and LSE in log2 units; rows in [T, Tpad) get zeros.
// One warp per (head, 32 consecutive tokens): a row is read by the whole warp (one contiguous 2 D bytes), lane i
// keeps the sum of row i, so the two statistics leave as one coalesced 128-byte store each.  Rows are taken
// four at a time to keep several loads in flight.
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
    constexpr int kPer = D / 32;  // 2 or 4 elements per lane
    float mine = 0.f;
#pragma unroll 2
    for (int i0 = 0; i0 < 32; i0 += 4) {
        float acc[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t t = t0 + i0 + u;
            acc[u] = 0.f;
            if (t < T) {
                const __nv_bfloat16* o = out + ((size_t)t * hq + h) * D + lane * kPer;
                const __nv_bfloat16* g = dout + ((size_t)t * hq + h) * D + lane * kPer;
#pragma unroll
                for (int i = 0; i < kPer; i += 2) {
                    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(o + i));
                    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(g + i));
                    acc[u] += a.x * b.x + a.y * b.y;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) acc[u] += __shfl_xor_sync(0xffffffffu, acc[u], off);
            if (lane == i0 + u) mine = acc[u];
        }
    }
    const int64_t t = t0 + lane;
    dvec[(size_t)h * Tpad + t] = mine;
    lse2[(size_t)h * Tpad + t] = t < T ? lse[(size_t)h * T + t] * 1.4426950408889634f : 0.f;
}

struct BwdWorkspace {
    size_t stat_bytes, total;
    int64_t Tpad;
};
static BwdWorkspace bwd_workspace(int64_t T, int hq) {
    BwdWorkspace w;
    w.Tpad = (T + 127) / 128 * 128;
    w.stat_bytes = ((size_t)hq * w.Tpad * sizeof(float) + 255) & ~(size_t)255;
    w.total = 2 * w.stat_bytes;
    return w;
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
        if (kDkvGroups > 2 && !regs_pool_ok(k_attn_bwd_dkdv<D>, 128 * kDkvGroups, kDkvRegsCompute, 128, kDkvRegsOther))
            return LIBRA_ERR_UNSUPPORTED;
        if (!regs_pool_ok(k_attn_bwd_dq<D>, 128 * kDqGroups, kDqRegsCompute, 128, kDqRegsOther)) return LIBRA_ERR_UNSUPPORTED;
        cfg_mark(kSlot);
    }
    if (mp->timing) cudaEventRecord(mp->ev[1][0], s);
    k_attn_bwd_dkdv<D><<<Wa, kBwdThreads, DkvSmem<D>::kBytes, s>>>(tq, tk, tv, tdo, pa);
    if (mp->timing) { cudaEventRecord(mp->ev[1][1], s); mp->ev_valid[1] = 1; cudaEventRecord(mp->ev[2][0], s); }
    k_attn_bwd_dq<D><<<Wb, kDqThreads, DqSmem<D>::kBytes, s>>>(tq, tk, tv, tdo, tdq, pb);
    if (mp->timing) { cudaEventRecord(mp->ev[2][1], s); mp->ev_valid[2] = 1; }
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace libra

using namespace libra;

#ifdef LIBRA_TRACE
extern "C" int libra_debug_trace(long long* host, int n) {
    return cudaMemcpyFromSymbol(host, libra::g_trace, sizeof(long long) * n) == cudaSuccess ? 0 : -4;
}
#endif

#ifdef LIBRA_PROF
extern "C" int libra_debug_bwd_prof(unsigned long long* host, int n) {
    return cudaMemcpyFromSymbol(host, libra::g_bwd_prof, sizeof(unsigned long long) * n) == cudaSuccess ? 0 : -4;
}
#endif

extern "C" size_t libra_attn_pool_bwd_workspace_bytes(const libra_plan_t* plan, const libra_dims* dims) {
    if (!plan || !dims || dims->hq <= 0 || (dims->head_dim != 64 && dims->head_dim != 128)) return 0;
    return bwd_workspace(plan->T, dims->hq).total;
}

extern "C" int libra_attn_pool_bwd(const void* q_dev, const void* k_dev, const void* v_dev, const void* out_dev,
                                   const float* lse_dev, const void* dout_dev, const int32_t* cu_seqlens_dev,
                                   const libra_plan_t* plan, void* dq_dev, void* dk_dev, void* dv_dev,
                                   void* workspace_dev, const libra_dims* dims, void* stream) {
    if (!q_dev || !k_dev || !v_dev || !out_dev || !lse_dev || !dout_dev || !cu_seqlens_dev || !plan || !dq_dev ||
        !dk_dev || !dv_dev || !workspace_dev || !dims)
        return LIBRA_ERR_INVALID_ARG;
    if (dims->hq <= 0 || dims->hkv <= 0 || dims->hq % dims->hkv) return LIBRA_ERR_INVALID_ARG;
    if (dims->head_dim != 64 && dims->head_dim != 128) return LIBRA_ERR_UNSUPPORTED;
    const PlanDir& dq_dir = plan->dir[0];
    const PlanDir& dkv_dir = plan->dir[1];
    if (!dq_dir.enabled || !dkv_dir.enabled || plan->T != dims->total_tokens) return LIBRA_ERR_PLAN_MISMATCH;
    if (dkv_dir.tile != kBlk || dq_dir.tile != 2 * kBlk) return LIBRA_ERR_UNSUPPORTED;
    if (dkv_dir.H != dims->hkv) return LIBRA_ERR_PLAN_MISMATCH;
    if (dims->hq % dq_dir.H) return LIBRA_ERR_INVALID_ARG;
    if (dkv_dir.W > plan->sm_count || dq_dir.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;
    if (((uintptr_t)q_dev | (uintptr_t)k_dev | (uintptr_t)v_dev | (uintptr_t)out_dev | (uintptr_t)dout_dev |
         (uintptr_t)dq_dev | (uintptr_t)dk_dev | (uintptr_t)dv_dev) & 15)
        return LIBRA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev & 255) return LIBRA_ERR_INVALID_ARG;
    if (int rcd = check_plan_device(plan); rcd != LIBRA_OK) return rcd;

    const int D = dims->head_dim;
    const int64_t T = plan->T;
    const BwdWorkspace ws = bwd_workspace(T, dims->hq);
    float* dvec = reinterpret_cast<float*>(workspace_dev);
    float* lse2 = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + ws.stat_bytes);
    cudaStream_t s = (cudaStream_t)stream;
    cudaMemsetAsync(plan->d_status + 2, 0, sizeof(int), s);   // the word reports the most recent launch

    CUtensorMap tq, tk, tv, tdo, tdq;
    int rc = make_thd_map(&tq, q_dev, T, dims->hq, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdo, dout_dev, T, dims->hq, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdq, dq_dev, T, dims->hq, D, kBlk);
    if (rc != LIBRA_OK) return rc;

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
    const float scale = dims->softmax_scale > 0.f ? dims->softmax_scale : 1.0f / sqrtf((float)D);
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
    pb.busy = dq_dir.d_busy2;
    libra_plan_t* mp = const_cast<libra_plan_t*>(plan);
    return D == 128 ? launch_bwd<128>(tq, tk, tv, tdo, tdq, pa, dkv_dir.W, pb, dq_dir.W, mp, s)
                    : launch_bwd<64>(tq, tk, tv, tdo, tdq, pa, dkv_dir.W, pb, dq_dir.W, mp, s);
}
