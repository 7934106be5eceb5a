// Backward pool attention for sm_100a.
//
// Three kernels: (1) prep: D_i = <dO_i, O_i> and LSE in log2 units, both padded to a multiple
// of 128 rows; (2) the persistent main kernel; (3) dQ fp32 -> bf16 with the softmax scale.
//
// Main kernel.  A work unit is a key-major tile: 128 keys x one kv head.  K and V of the unit
// stay in shared memory; dK and dV stay in TMEM for the whole unit while the CTA streams every
// (query head of the group, 128-row query block) that can see the keys, from the diagonal
// block up to the block holding the end of the last key's sample.  Keys sit in TMEM lanes:
//   S^T  = K Q^T          (SS)      P^T = exp2(S^T * c - LSE)   written over S^T as bf16
//   dP^T = V dO^T         (SS)      dS^T = P^T o (dP^T - D)     written to shared memory
//   dV  += P^T dO         (A from TMEM)
//   dK  += dS^T Q         (SS, A K-major)
//   dQ   = dS K           (SS, A and B MN-major; dQ reuses dP^T's TMEM columns)
// dQ tiles are drained by a reduce group and added to an fp32 accumulator with vector atomics.
// Roles (448 threads): warps 0-3 / 4-7 compute groups (query columns 0-63 / 64-127 of each key
// row), warps 8-11 dQ reduce, warp 12 TMA, warp 13 MMA.
// Tensor-pipe order per iteration i:  dP(i) | dV(i) S(i+1) | dK(i) dQ(i), so the exp phase of
// iteration i+1 overlaps dK/dQ/dP and the dS phase overlaps dV/S.
#include <math.h>

#include "common.h"
#include "ptx.cuh"

namespace libra {

constexpr int kBwdThreads = 448;
constexpr int kBlk = 128;

template <int D>
struct BwdSmem {
    static constexpr int kHalfBytes = 128 * 128;
    static constexpr int kTileBytes = kHalfBytes * (D / 64);  // 128 x D bf16
    static constexpr int kDoStages = (D == 128) ? 1 : 2;      // shared memory is full at D = 128
    static constexpr int kKOff = 0;
    static constexpr int kVOff = kTileBytes;
    static constexpr int kQOff = 2 * kTileBytes;                    // 2 stages
    static constexpr int kDoOff = 4 * kTileBytes;                   // kDoStages stages
    static constexpr int kDsOff = kDoOff + kDoStages * kTileBytes;  // 128 keys x 128 queries bf16
    static constexpr int kStageOff = kDsOff + 2 * kHalfBytes;       // 2 x (128 rows x 32 fp32) dQ staging
    static constexpr int kStatOff = kStageOff + 2 * kHalfBytes;     // per Q stage: lse2[128], dvec[128]
    static constexpr int kBarOff = kStatOff + 2 * 1024;
    // kv_full, kv_empty, q_full[2], q_empty[2], do_full[2], do_empty[2], s_full, p_ready, dp_full,
    // ds_ready, dq_full, dq_empty, dkv_full, dkv_empty
    static constexpr int kNumBars = 18;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static_assert(kBytes <= 232448, "exceeds the 227 KB shared memory of an sm_100 CTA");
};

struct BwdParams {
    float* dq_acc;            // [T, Hq, D] fp32, zeroed before the launch
    __nv_bfloat16* dk;
    __nv_bfloat16* dv;
    const float* lse2;        // [Hq, Tpad]  LSE * log2(e)
    const float* dvec;        // [Hq, Tpad]  D_i
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* tok_end;
    int64_t T, Tpad;
    int hq, hkv;
    float scale, scale_log2;
    int* status;
    uint64_t* busy;
};

__device__ __forceinline__ void bulk_load_1d(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(reinterpret_cast<uint64_t>(gsrc)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void red_add_v4(float* gptr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(gptr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}
__device__ __forceinline__ bool warp_wait_b(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
    int ok = 1;
    if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag) ? 1 : 0;
    return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// Query blocks a key block [k0, k0+128) is seen by: diagonal .. block of (end of last key's sample - 1).
__device__ __forceinline__ int last_q_block(const int32_t* tok_end, int64_t T, int64_t k0) {
    const int64_t last_key = (k0 + kBlk <= T ? k0 + kBlk : T) - 1;
    return (tok_end[last_key] - 1) / kBlk;
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

template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
k_attn_bwd(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const __grid_constant__ CUtensorMap tm_dq,
           const BwdParams p) {
    using L = BwdSmem<D>;
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
    uint64_t* bar_dqfull = bars + 14;
    uint64_t* bar_dqempty = bars + 15;
    uint64_t* bar_dkvfull = bars + 16;
    uint64_t* bar_dkvempty = bars + 17;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if ((smem_u32(smem) & 1023u) != 0) {  // the swizzled tiles need a 1024-byte aligned base
        if (threadIdx.x == 0) atomicExch(p.status, LIBRA_ERR_CUDA);
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
        mbar_init(bar_pready, 256);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_dsready, 256);
        mbar_init(bar_dqfull, 1);
        mbar_init(bar_dqempty, 128);
        mbar_init(bar_dkvfull, 1);
        mbar_init(bar_dkvempty, 256);
        *abort_flag = 0;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == 13) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == 12 && lane == 0) {
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
        prefetch_tmap(&tm_dq);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    constexpr uint32_t kColS = 0, kColDP = 128, kColDK = 256, kColDV = 256 + D;

    const int unit_begin = p.cta_offsets[cta];
    const int unit_end = p.cta_offsets[cta + 1];
    const int G = p.hq / p.hkv;

    if (warp == 12) {
        // ---------------- TMA producer ----------------
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int kvh = t % p.hkv;
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            ok = warp_wait_b(bar_kvempty, (ucnt & 1) ^ 1, abort_flag);
            if (!ok) break;
            if (lane == 0) {
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
                ok = warp_wait_b(&bar_qempty[st], par, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bar_qfull[st], L::kTileBytes + 1024);
                    for (int half = 0; half < D / 64; ++half)
                        tma_load_3d(smem + L::kQOff + st * L::kTileBytes + half * L::kHalfBytes, &tm_q, &bar_qfull[st],
                                    half * 64, h, qb);
                    bulk_load_1d(smem + L::kStatOff + st * 1024, p.lse2 + (size_t)h * p.Tpad + qb, 512, &bar_qfull[st]);
                    bulk_load_1d(smem + L::kStatOff + st * 1024 + 512, p.dvec + (size_t)h * p.Tpad + qb, 512,
                                 &bar_qfull[st]);
                }
                const uint32_t dst = it_all % L::kDoStages, dpar = ((it_all / L::kDoStages) & 1) ^ 1;
                ok = warp_wait_b(&bar_doempty[dst], dpar, abort_flag);
                if (!ok) break;
                if (lane == 0) {
                    mbar_arrive_expect_tx(&bar_dofull[dst], L::kTileBytes);
                    for (int half = 0; half < D / 64; ++half)
                        tma_load_3d(smem + L::kDoOff + dst * L::kTileBytes + half * L::kHalfBytes, &tm_do,
                                    &bar_dofull[dst], half * 64, h, qb);
                }
            }
        }
    } else if (warp == 13) {
        // ---------------- MMA issuer ----------------
        constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);   // S^T, dP^T: both operands K-major
        constexpr uint32_t idesc_dv = make_idesc(128, D, 0, 1);    // A from TMEM, B = dO MN-major
        constexpr uint32_t idesc_dk = make_idesc(128, D, 0, 1);    // A = dS^T K-major, B = Q MN-major
        constexpr uint32_t idesc_dq = make_idesc(128, D, 1, 1);    // A = dS MN-major, B = K MN-major
        const uint32_t sb = smem_u32(smem);
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        PROF_DECL
        // C[tmem] = A(K-major tile) * B(K-major tile)^T over the head dimension
        auto issue_kmajor = [&](uint32_t d_col, uint32_t a_addr, uint32_t b_addr) {
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk / 4) * L::kHalfBytes + (kk % 4) * 32;
                mma_ss(tmem_base + d_col, make_sdesc(a_addr + off, 16, 1024), make_sdesc(b_addr + off, 16, 1024),
                       idesc_s, kk > 0);
            }
        };
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            const int n_it = G * nblk;
            ok = warp_wait_b(bar_kvfull, ucnt & 1, abort_flag);
            if (!ok) break;
            // S(0)
            ok = warp_wait_b(&bar_qfull[it_all & 1], (it_all >> 1) & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) {
                issue_kmajor(kColS, sb + L::kKOff, sb + L::kQOff + (it_all & 1) * L::kTileBytes);
                tc_commit(bar_sfull);
            }
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const uint32_t st = it_all & 1, par = (it_all >> 1) & 1;
                // dP(it): needs dO and the dP/dQ columns drained of dQ(it-1)
                const uint32_t dst = it_all % L::kDoStages, dpar = (it_all / L::kDoStages) & 1;
                PROF(7)
                ok = warp_wait_b(&bar_dofull[dst], dpar, abort_flag);
                if (!ok) break;
                PROF(0)
                if (it_all > 0) {
                    ok = warp_wait_b(bar_dqempty, (it_all - 1) & 1, abort_flag);
                    if (!ok) break;
                }
                PROF(1)
                tc_fence_after();
                if (lane == 0) {
                    issue_kmajor(kColDP, sb + L::kVOff, sb + L::kDoOff + dst * L::kTileBytes);
                    tc_commit(bar_dpfull);
                }
                // dV(it) += P^T dO
                PROF(7)
                ok = warp_wait_b(bar_pready, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(2)
                if (it == 0 && ucnt > 0) {  // previous unit's dK/dV must have been read out
                    ok = warp_wait_b(bar_dkvempty, (ucnt - 1) & 1, abort_flag);
                    if (!ok) break;
                }
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t doa = sb + L::kDoOff + dst * L::kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)  // 16 queries per step; P^T of columns 64c.. lives at 64c + ..
                        mma_ts(tmem_base + kColDV, tmem_base + kColS + (kk / 4) * 64 + (kk % 4) * 8,
                               make_sdesc(doa + kk * 2048, L::kHalfBytes, 1024), idesc_dv, (it > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(&bar_doempty[dst]);
                }
                // S(it+1)
                if (it + 1 < n_it) {
                    const uint32_t nx = it_all + 1;
                    PROF(7)
                    ok = warp_wait_b(&bar_qfull[nx & 1], (nx >> 1) & 1, abort_flag);
                    if (!ok) break;
                    PROF(3)
                    if (lane == 0) {
                        issue_kmajor(kColS, sb + L::kKOff, sb + L::kQOff + (nx & 1) * L::kTileBytes);
                        tc_commit(bar_sfull);
                    }
                }
                // dK(it) += dS^T Q ; dQ(it) = dS K
                PROF(7)
                ok = warp_wait_b(bar_dsready, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(4)
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t dsa = sb + L::kDsOff;
                    const uint32_t qa = sb + L::kQOff + st * L::kTileBytes;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)  // over 16 queries
                        mma_ss(tmem_base + kColDK, make_sdesc(dsa + (kk / 4) * L::kHalfBytes + (kk % 4) * 32, 16, 1024),
                               make_sdesc(qa + kk * 2048, L::kHalfBytes, 1024), idesc_dk, (it > 0 || kk > 0) ? 1u : 0u);
                    tc_commit(&bar_qempty[st]);
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)  // over 16 keys
                        mma_ss(tmem_base + kColDP, make_sdesc(dsa + kk * 2048, L::kHalfBytes, 1024),
                               make_sdesc(sb + L::kKOff + kk * 2048, L::kHalfBytes, 1024), idesc_dq, kk > 0);
                    tc_commit(bar_dqfull);
                }
                __syncwarp();
            }
            if (ok && lane == 0) {
                tc_commit(bar_dkvfull);
                tc_commit(bar_kvempty);
            }
            __syncwarp();
            ++ucnt;
        }
        PROF_FLUSH(lane == 0, 8)
    } else if (warp >= 12) {
        // warps 14-15: nothing to do
    } else if (warp >= 8) {
        // ---------------- dQ reduce group ----------------
        // TMEM -> registers (whole tile, frees the columns at once) -> 32-column chunks through two
        // staging buffers -> TMA reduce-add into the fp32 accumulator (full 128-byte lines).
        const int r = (warp & 3) * 32 + lane;
        const bool leader = (threadIdx.x == 8 * 32);
        const uint32_t t_dq = tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + kColDP;
        uint8_t* stage_row = smem + L::kStageOff + r * 128;
        uint32_t it_all = 0;
        bool ok = true;
        PROF_DECL
        for (int idx = unit_begin; idx < unit_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            const int kvh = t % p.hkv;
            const int64_t k0 = (int64_t)(t / p.hkv) * kBlk;
            const int i_lo = (int)(k0 / kBlk);
            const int nblk = last_q_block(p.tok_end, p.T, k0) - i_lo + 1;
            const int n_it = G * nblk;
            for (int it = 0; it < n_it && ok; ++it, ++it_all) {
                const int h = kvh * G + it / nblk;
                const int qb = (i_lo + it % nblk) * kBlk;
                ok = mbar_wait(bar_dqfull, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(0)
                tc_fence_after();
                uint32_t v[D];
#pragma unroll
                for (int c = 0; c < D; c += 32) tmem_ld32(t_dq + c, v + c);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_dqempty);  // the dP/dQ columns may be overwritten now
                PROF(1)
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint8_t* dst = stage_row + (c & 1) * L::kHalfBytes;
                    // the buffer may still be read by the reduce issued two chunks ago
                    if (leader) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                    asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        uint4 w;
                        w.x = v[c * 32 + k * 4]; w.y = v[c * 32 + k * 4 + 1];
                        w.z = v[c * 32 + k * 4 + 2]; w.w = v[c * 32 + k * 4 + 3];
                        *reinterpret_cast<uint4*>(dst + ((k ^ (r & 7)) << 4)) = w;
                    }
                    fence_proxy_async_smem();
                    asm volatile("bar.sync 1, 128;" ::: "memory");
                    if (leader) {
#ifndef LIBRA_DBG_NO_RED
                        asm volatile(
                            "cp.reduce.async.bulk.tensor.2d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2}], [%3];"
                            ::"l"(reinterpret_cast<uint64_t>(&tm_dq)), "r"(h * D + c * 32), "r"(qb),
                            "r"(smem_u32(smem + L::kStageOff + (c & 1) * L::kHalfBytes))
                            : "memory");
#endif
                        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                    }
                }
                PROF(2)
            }
        }
        if (leader) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // all reduce-adds done before exit
        PROF_FLUSH(leader, 16)
    } else {
        // ---------------- compute groups ----------------
        const int c = warp >> 2;  // query-column half of each key row
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem_base + lane_addr + kColS + 64 * c;
        const uint32_t t_dp = tmem_base + lane_addr + kColDP + 64 * c;
        uint8_t* ds_row = smem + L::kDsOff + c * L::kHalfBytes + r * 128;
        uint32_t ucnt = 0, it_all = 0;
        bool ok = true;
        PROF_DECL
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
                const float* lse2 = reinterpret_cast<const float*>(smem + L::kStatOff + st * 1024) + 64 * c;
                const float* dvec = lse2 + 128;
                const bool need_mask = (qb == k0) || (qb + kBlk - 1 >= min_kend) || partial;
                const int j_lo = (int)(key - qb) - 64 * c;       // first visible column of this half
                const int j_hi = kend - 1 - qb - 64 * c;         // last visible column
                // ---- exp phase: P^T = exp2(S^T * c - LSE) ----
                ok = mbar_wait(&bar_qfull[st], par, abort_flag) && mbar_wait(bar_sfull, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(0)
                tc_fence_after();
                uint32_t sv[64];
                tmem_ld32(t_s, sv);
                tmem_ld32(t_s + 32, sv + 32);
                tmem_ld_wait();
                float pf[64];
#pragma unroll
                for (int j = 0; j < 64; j += 4) {
                    const float4 l4 = *reinterpret_cast<const float4*>(lse2 + j);
                    pf[j] = ex2_approx(fmaf(__uint_as_float(sv[j]), p.scale_log2, -l4.x));
                    pf[j + 1] = ex2_approx(fmaf(__uint_as_float(sv[j + 1]), p.scale_log2, -l4.y));
                    pf[j + 2] = ex2_approx(fmaf(__uint_as_float(sv[j + 2]), p.scale_log2, -l4.z));
                    pf[j + 3] = ex2_approx(fmaf(__uint_as_float(sv[j + 3]), p.scale_log2, -l4.w));
                }
                if (need_mask) {
#pragma unroll
                    for (int j = 0; j < 64; ++j)
                        if (j < j_lo || j > j_hi) pf[j] = 0.f;
                }
                {
                    uint32_t pk[32];
#pragma unroll
                    for (int j = 0; j < 64; j += 2) pk[j >> 1] = pack_bf16x2(pf[j], pf[j + 1]);
                    tmem_st32(t_s, pk);  // packed P^T of this half sits in the first 32 columns of its own S^T half
                }
                tmem_st_wait();
                tc_fence_before();
                mbar_arrive(bar_pready);
                PROF(1)
                // ---- dS phase: dS^T = P^T o (dP^T - D) ----
                ok = mbar_wait(bar_dpfull, it_all & 1, abort_flag);
                if (!ok) break;
                PROF(2)
                tc_fence_after();
                uint32_t dpv[64];
                tmem_ld32(t_dp, dpv);
                tmem_ld32(t_dp + 32, dpv + 32);
                tmem_ld_wait();
                PROF(3)
                PROF(4)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const float4 d0 = *reinterpret_cast<const float4*>(dvec + ch * 8);
                    const float4 d1 = *reinterpret_cast<const float4*>(dvec + ch * 8 + 4);
                    const int j = ch * 8;
                    uint4 w;
                    w.x = pack_bf16x2(pf[j] * (__uint_as_float(dpv[j]) - d0.x), pf[j + 1] * (__uint_as_float(dpv[j + 1]) - d0.y));
                    w.y = pack_bf16x2(pf[j + 2] * (__uint_as_float(dpv[j + 2]) - d0.z), pf[j + 3] * (__uint_as_float(dpv[j + 3]) - d0.w));
                    w.z = pack_bf16x2(pf[j + 4] * (__uint_as_float(dpv[j + 4]) - d1.x), pf[j + 5] * (__uint_as_float(dpv[j + 5]) - d1.y));
                    w.w = pack_bf16x2(pf[j + 6] * (__uint_as_float(dpv[j + 6]) - d1.z), pf[j + 7] * (__uint_as_float(dpv[j + 7]) - d1.w));
                    *reinterpret_cast<uint4*>(ds_row + ((ch ^ (r & 7)) << 4)) = w;
                }
                PROF(5)
                fence_proxy_async_smem();
                tc_fence_before();
                mbar_arrive(bar_dsready);
                PROF(7)
            }
            if (!ok) break;
            // ---- unit epilogue: dK * scale and dV to global ----
            ok = mbar_wait(bar_dkvfull, ucnt & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            constexpr int kCols = D / 2;  // columns of dK and dV this group stores
            const uint32_t t_dk = tmem_base + lane_addr + kColDK + c * kCols;
            const uint32_t t_dv = tmem_base + lane_addr + kColDV + c * kCols;
            const size_t gofs = ((size_t)key * p.hkv + kvh) * D + c * kCols;
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
            ++ucnt;
            PROF(6)
        }
        PROF_FLUSH(threadIdx.x == 0, 0)
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == 13) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (*abort_flag) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

// ---- prep and post kernels --------------------------------------------------------------------

// One warp per (token, head): D = <dO, O>; LSE to log2 units; rows in [T, Tpad) get zeros.
template <int D>
__global__ void k_bwd_prep(const __nv_bfloat16* __restrict__ out, const __nv_bfloat16* __restrict__ dout,
                           const float* __restrict__ lse, int64_t T, int64_t Tpad, int hq, float* __restrict__ dvec,
                           float* __restrict__ lse2) {
    const int64_t w = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= Tpad * hq) return;
    const int64_t t = w / hq;
    const int h = (int)(w % hq);
    float acc = 0.f;
    if (t < T) {
        constexpr int kPer = D / 32;  // 2 or 4 elements per lane
        const __nv_bfloat16* o = out + ((size_t)t * hq + h) * D + lane * kPer;
        const __nv_bfloat16* g = dout + ((size_t)t * hq + h) * D + lane * kPer;
#pragma unroll
        for (int i = 0; i < kPer; i += 2) {
            const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(o + i));
            const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(g + i));
            acc += a.x * b.x + a.y * b.y;
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    }
    if (lane == 0) {
        dvec[(size_t)h * Tpad + t] = acc;
        lse2[(size_t)h * Tpad + t] = t < T ? lse[(size_t)h * T + t] * 1.4426950408889634f : 0.f;
    }
}

__global__ void k_bwd_dq_convert(const float* __restrict__ acc, int64_t n4, float scale, __nv_bfloat16* __restrict__ dq) {
    const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 v = reinterpret_cast<const float4*>(acc)[i];
    uint2 w;
    w.x = pack_bf16x2(v.x * scale, v.y * scale);
    w.y = pack_bf16x2(v.z * scale, v.w * scale);
    reinterpret_cast<uint2*>(dq)[i] = w;
}

struct BwdWorkspace {
    size_t dq_acc_bytes, stat_bytes, total;
    int64_t Tpad;
};
static BwdWorkspace bwd_workspace(int64_t T, int hq, int d) {
    BwdWorkspace w;
    w.Tpad = (T + 127) / 128 * 128;
    w.dq_acc_bytes = ((size_t)T * hq * d * sizeof(float) + 255) & ~(size_t)255;
    w.stat_bytes = ((size_t)hq * w.Tpad * sizeof(float) + 255) & ~(size_t)255;
    w.total = w.dq_acc_bytes + 2 * w.stat_bytes;
    return w;
}

template <int D>
static int launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                      const CUtensorMap& tdq, const BwdParams& prm, int W, cudaStream_t s) {
    using L = BwdSmem<D>;
    static bool configured = false;
    if (!configured) {
        if (cudaFuncSetAttribute(k_attn_bwd<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kBytes) != cudaSuccess)
            return LIBRA_ERR_CUDA;
        configured = true;
    }
    k_attn_bwd<D><<<W, kBwdThreads, L::kBytes, s>>>(tq, tk, tv, tdo, tdq, prm);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

}  // namespace libra

using namespace libra;

#ifdef LIBRA_PROF
extern "C" int libra_debug_bwd_prof(unsigned long long* host, int n) {
    return cudaMemcpyFromSymbol(host, libra::g_bwd_prof, sizeof(unsigned long long) * n) == cudaSuccess ? 0 : -4;
}
#endif

extern "C" size_t libra_attn_pool_bwd_workspace_bytes(const libra_plan_t* plan, const libra_dims* dims) {
    if (!plan || !dims || dims->hq <= 0 || (dims->head_dim != 64 && dims->head_dim != 128)) return 0;
    return bwd_workspace(plan->T, dims->hq, dims->head_dim).total;
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
    const PlanDir& d = plan->dir[1];
    if (!d.enabled || plan->T != dims->total_tokens) return LIBRA_ERR_PLAN_MISMATCH;
    if (d.tile != kBlk) return LIBRA_ERR_UNSUPPORTED;
    if (d.H != dims->hkv) return LIBRA_ERR_PLAN_MISMATCH;
    if (d.W > plan->sm_count) return LIBRA_ERR_UNSUPPORTED;
    if (((uintptr_t)q_dev | (uintptr_t)k_dev | (uintptr_t)v_dev | (uintptr_t)out_dev | (uintptr_t)dout_dev |
         (uintptr_t)dq_dev | (uintptr_t)dk_dev | (uintptr_t)dv_dev) & 15)
        return LIBRA_ERR_INVALID_ARG;
    if ((uintptr_t)workspace_dev & 255) return LIBRA_ERR_INVALID_ARG;

    const int D = dims->head_dim;
    const int64_t T = plan->T;
    const BwdWorkspace ws = bwd_workspace(T, dims->hq, D);
    float* dq_acc = reinterpret_cast<float*>(workspace_dev);
    float* dvec = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + ws.dq_acc_bytes);
    float* lse2 = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(workspace_dev) + ws.dq_acc_bytes + ws.stat_bytes);
    cudaStream_t s = (cudaStream_t)stream;

    CUtensorMap tq, tk, tv, tdo, tdq;
    int rc = make_f32_2d_map(&tdq, dq_acc, T, (int64_t)dims->hq * D, 32, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tq, q_dev, T, dims->hq, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tk, k_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tv, v_dev, T, dims->hkv, D, kBlk);
    if (rc == LIBRA_OK) rc = make_thd_map(&tdo, dout_dev, T, dims->hq, D, kBlk);
    if (rc != LIBRA_OK) return rc;

    if (cudaMemsetAsync(dq_acc, 0, (size_t)T * dims->hq * D * sizeof(float), s) != cudaSuccess) return LIBRA_ERR_CUDA;
    {
        const int64_t warps = ws.Tpad * dims->hq;
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
    BwdParams prm;
    prm.dq_acc = dq_acc;
    prm.dk = reinterpret_cast<__nv_bfloat16*>(dk_dev);
    prm.dv = reinterpret_cast<__nv_bfloat16*>(dv_dev);
    prm.lse2 = lse2;
    prm.dvec = dvec;
    prm.cta_offsets = d.d_cta_offsets;
    prm.cta_tiles = d.d_cta_exec;
    prm.tok_end = plan->d_tok_end;
    prm.T = T;
    prm.Tpad = ws.Tpad;
    prm.hq = dims->hq;
    prm.hkv = dims->hkv;
    prm.scale = scale;
    prm.scale_log2 = scale * 1.4426950408889634f;
    prm.status = plan->d_status + 2;
    prm.busy = d.d_busy;
    libra_plan_t* mp = const_cast<libra_plan_t*>(plan);
    if (mp->timing) cudaEventRecord(mp->ev[1][0], s);
    rc = D == 128 ? launch_bwd<128>(tq, tk, tv, tdo, tdq, prm, d.W, s) : launch_bwd<64>(tq, tk, tv, tdo, tdq, prm, d.W, s);
    if (mp->timing) { cudaEventRecord(mp->ev[1][1], s); mp->ev_valid[1] = 1; }
    if (rc != LIBRA_OK) return rc;
    {
        const int64_t n4 = T * dims->hq * D / 4;
        k_bwd_dq_convert<<<(unsigned)((n4 + 255) / 256), 256, 0, s>>>(dq_acc, n4, scale, (__nv_bfloat16*)dq_dev);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}
