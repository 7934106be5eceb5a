// dQ kernel of the backward pass (included by attn_bwd.cu).
//
// A unit is 128 query rows x one head.  Q and dO of the unit are copied once from shared memory
// into TMEM (bf16, packed two per column), so all three GEMMs of a key block take their A operand
// from TMEM and only stream K_j / V_j through shared memory:
//   S  = Q K_j^T     (A = Q  in TMEM, B = K_j K-major)
//   dP = dO V_j^T    (A = dO in TMEM, B = V_j K-major)
//   dS = P o (dP - D), P = exp2(S c - LSE)   -> bf16 over this thread's own dP columns
//   dQ += dS K_j     (A = dS in TMEM, B = K_j MN-major)
// TMEM: S | dP (dS) | dQ | Q^ | dO^ = 128 + 128 + D + D/2 + D/2 columns.
// Queries sit in TMEM lanes, so LSE and D are per-thread scalars and the masks are the forward's.
// Pipeline per key block j on the tensor pipe:  S(j+1) | dQ(j) dP(j+1); the exp phase of block
// j+1 overlaps dQ(j) and dP(j+1), the dS phase overlaps S(j+2).
#pragma once

namespace libra {

constexpr int kDqGroups = 4;                      // compute warpgroups: each owns 128 / kDqGroups key columns
constexpr int kDqCW = 128 / kDqGroups;            // S / dP columns per compute thread
constexpr int kDqThreads = (4 * kDqGroups + 2) * 32;
constexpr int kDqTmaWarp = 4 * kDqGroups, kDqMmaWarp = 4 * kDqGroups + 1;

template <int D>
struct DqSmem {
    static constexpr int kHalfBytes = 128 * 128;
    static constexpr int kTileBytes = kHalfBytes * (D / 64);
    static constexpr int kKStages = 3;  // K_j lives from S(j) to dQ(j); S(j+1) is issued in between
    static constexpr int kVStages = 2;
    static constexpr int kQOff = 0;
    static constexpr int kDoOff = kTileBytes;
    static constexpr int kKOff = 2 * kTileBytes;
    static constexpr int kVOff = kKOff + kKStages * kTileBytes;
    static constexpr int kBarOff = kVOff + kVStages * kTileBytes;
    // q_full, q_empty, do_full, do_empty, k_full[3], k_empty[3], v_full[2], v_empty[2], qt_ready,
    // s_full, s_free, dp_full, ds_ready, dq_full
    static constexpr int kNumBars = 20;
    static constexpr int kMiscOff = kBarOff + kNumBars * 8;
    static constexpr int kBytes = kMiscOff + 16;
    static_assert(kBytes <= kSmemMax, "exceeds the shared memory of an sm_100 CTA");
};

struct DqParams {
    __nv_bfloat16* dq;
    const float* lse2;
    const float* dvec;
    const int32_t* cta_offsets;
    const int32_t* cta_tiles;
    const int32_t* tok_start;
    int64_t T, Tpad;
    int hq, hkv, H;
    float scale, scale_log2;
    int* status;
    uint64_t* busy;
};

template <int D>
__global__ void __launch_bounds__(kDqThreads, 1)
k_attn_bwd_dq(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, const DqParams p) {
    using L = DqSmem<D>;
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + L::kBarOff);
    uint64_t* bar_qfull = bars + 0;
    uint64_t* bar_qempty = bars + 1;
    uint64_t* bar_dofull = bars + 2;
    uint64_t* bar_doempty = bars + 3;
    uint64_t* bar_kfull = bars + 4;    // [3]
    uint64_t* bar_kempty = bars + 7;   // [3]
    uint64_t* bar_vfull = bars + 10;   // [2]
    uint64_t* bar_vempty = bars + 12;  // [2]
    uint64_t* bar_qtready = bars + 14;
    uint64_t* bar_sfull = bars + 15;
    uint64_t* bar_sfree = bars + 16;
    uint64_t* bar_dpfull = bars + 17;
    uint64_t* bar_dsready = bars + 18;
    uint64_t* bar_dqfull = bars + 19;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(smem + L::kMiscOff);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + L::kMiscOff + 4);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    if ((smem_u32(smem) & 1023u) != 0) {
        if (threadIdx.x == 0) atomicExch(p.status, LIBRA_ERR_CUDA);
        return;
    }
    if (threadIdx.x == 0) {
        mbar_init(bar_qfull, 1);
        mbar_init(bar_qempty, 64 * kDqGroups);   // the groups that stage Q
        mbar_init(bar_dofull, 1);
        mbar_init(bar_doempty, 64 * kDqGroups);  // the groups that stage dO
        for (int s = 0; s < L::kKStages; ++s) { mbar_init(&bar_kfull[s], 1); mbar_init(&bar_kempty[s], 1); }
        for (int s = 0; s < L::kVStages; ++s) { mbar_init(&bar_vfull[s], 1); mbar_init(&bar_vempty[s], 1); }
        mbar_init(bar_qtready, 128 * kDqGroups);
        mbar_init(bar_sfull, 1);
        mbar_init(bar_sfree, 128 * kDqGroups);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_dsready, 128 * kDqGroups);
        mbar_init(bar_dqfull, 1);
        *abort_flag = 0;
        fence_mbar_init();
        p.busy[2 * cta] = globaltimer_ns();
    }
    if (warp == kDqMmaWarp) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }
    if (warp == kDqTmaWarp && lane == 0) {
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    constexpr uint32_t kColS = 0, kColDP = 128, kColDQ = 256, kColQ = 256 + D, kColDO = 256 + D + D / 2;
    static_assert(kColDO + D / 2 <= 512, "TMEM columns");

    const int tile_begin = p.cta_offsets[cta];
    const int tile_end = p.cta_offsets[cta + 1];
    const int heads_per_shard = p.hq / p.H;
    const int G = p.hq / p.hkv;

    // All roles walk the same sequence of sub-blocks: (tile, sub-block of 128 rows, head of the shard).
    // A sub-block past the end of the pool is skipped by every role.
    if (warp == kDqTmaWarp) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {  // one elected thread runs the whole role
            uint32_t bcnt = 0, kcnt = 0, vcnt = 0;
            bool ok = true;
            for (int idx = tile_begin; idx < tile_end && ok; ++idx) {
                const int t = p.cta_tiles[idx];
                for (int sub = 0; sub < 2 && ok; ++sub) {
                    const int64_t q0 = (int64_t)(t / p.H) * (2 * kBlk) + sub * kBlk;
                    if (q0 >= p.T) continue;
                    const int lo = p.tok_start[q0] / kBlk, hi = (int)(q0 / kBlk);
                    for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                        const int h = (t % p.H) * heads_per_shard + hh;
                        const int kvh = h / G;
                        ok = mbar_wait(bar_qempty, (bcnt & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        {
                            mbar_arrive_expect_tx(bar_qfull, L::kTileBytes);
                            for (int half = 0; half < D / 64; ++half)
                                tma_load_3d(smem + L::kQOff + half * L::kHalfBytes, &tm_q, bar_qfull, half * 64, h, (int)q0);
                        }
                        ok = mbar_wait(bar_doempty, (bcnt & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        {
                            mbar_arrive_expect_tx(bar_dofull, L::kTileBytes);
                            for (int half = 0; half < D / 64; ++half)
                                tma_load_3d(smem + L::kDoOff + half * L::kHalfBytes, &tm_do, bar_dofull, half * 64, h, (int)q0);
                        }
                        ++bcnt;
                        for (int j = lo; j <= hi && ok; ++j) {
                            const uint32_t ks = kcnt % L::kKStages;
                            ok = mbar_wait(&bar_kempty[ks], ((kcnt / L::kKStages) & 1) ^ 1, abort_flag);
                            if (!ok) break;
                            {
                                mbar_arrive_expect_tx(&bar_kfull[ks], L::kTileBytes);
                                for (int half = 0; half < D / 64; ++half)
                                    tma_load_3d(smem + L::kKOff + ks * L::kTileBytes + half * L::kHalfBytes, &tm_k,
                                                &bar_kfull[ks], half * 64, kvh, j * kBlk);
                            }
                            ++kcnt;
                            const uint32_t vs = vcnt % L::kVStages;
                            ok = mbar_wait(&bar_vempty[vs], ((vcnt / L::kVStages) & 1) ^ 1, abort_flag);
                            if (!ok) break;
                            {
                                mbar_arrive_expect_tx(&bar_vfull[vs], L::kTileBytes);
                                for (int half = 0; half < D / 64; ++half)
                                    tma_load_3d(smem + L::kVOff + vs * L::kTileBytes + half * L::kHalfBytes, &tm_v,
                                                &bar_vfull[vs], half * 64, kvh, j * kBlk);
                            }
                            ++vcnt;
                        }
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp == kDqMmaWarp) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {  // one elected thread runs the whole role
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);  // S, dP: A in TMEM, B K-major
            constexpr uint32_t idesc_dq = make_idesc(128, D, 0, 1);   // dQ: A in TMEM, B = K MN-major
            const uint32_t sb = smem_u32(smem);
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);             // K-major view of a tile at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kHalfBytes, 1024);  // MN-major view
            uint32_t bcnt = 0, kcnt = 0, vcnt = 0, blk = 0;
            bool ok = true;
            PROF_DECL
            TRACE_DECL(0, cta == 0)
            // C[tmem d_col] = A[tmem a_col, bf16 packed over the head dimension] * B(K-major tile at b_off)^T
            auto issue_qk = [&](uint32_t d_col, uint32_t a_col, uint32_t b_off) {
                const uint64_t db = sdesc_advance(kdesc0, b_off);
    #pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk / 4) * L::kHalfBytes + (kk % 4) * 32;
                    mma_ts(tmem_base + d_col, tmem_base + a_col + kk * 8, sdesc_advance(db, off), idesc_s, kk > 0);
                }
            };
            // S(j) from K ring entry kidx
            auto do_s = [&](uint32_t kidx) -> bool {
                PROF(7)
                if (!mbar_wait(&bar_kfull[kidx % L::kKStages], (kidx / L::kKStages) & 1, abort_flag)) return false;
                PROF(0)
                TRACE(1)
                {
                    issue_qk(kColS, kColQ, L::kKOff + (kidx % L::kKStages) * L::kTileBytes);
                    tc_commit(bar_sfull);
                }
                TRACE(2)
                return true;
            };
            auto do_dp = [&]() -> bool {
                const uint32_t vs = vcnt % L::kVStages;
                PROF(7)
                if (!mbar_wait(&bar_vfull[vs], (vcnt / L::kVStages) & 1, abort_flag)) return false;
                PROF(1)
                TRACE(3)
                {
                    issue_qk(kColDP, kColDO, L::kVOff + vs * L::kTileBytes);
                    tc_commit(bar_dpfull);
                    tc_commit(&bar_vempty[vs]);
                }
                TRACE(4)
                ++vcnt;
                return true;
            };
            for (int idx = tile_begin; idx < tile_end && ok; ++idx) {
                const int t = p.cta_tiles[idx];
                for (int sub = 0; sub < 2 && ok; ++sub) {
                    const int64_t q0 = (int64_t)(t / p.H) * (2 * kBlk) + sub * kBlk;
                    if (q0 >= p.T) continue;
                    const int lo = p.tok_start[q0] / kBlk, hi = (int)(q0 / kBlk);
                    for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                        PROF(7)
                        ok = mbar_wait(bar_qtready, bcnt & 1, abort_flag);  // Q and dO are in TMEM
                        if (!ok) break;
                        PROF(2)
                        ++bcnt;
                        tc_fence_after();
                        const uint32_t kbase = kcnt;  // ring index of K_lo
                        ok = do_s(kbase);             // S(lo)
                        if (ok) ok = do_dp();         // dP(lo)
                        if (!ok) break;
                        for (int j = lo; j <= hi && ok; ++j, ++blk) {
                            // S(j+1) as soon as the compute groups have read S(j)
                            if (j + 1 <= hi) {
                                PROF(7)
                                TRACE(8)
                                ok = mbar_wait(bar_sfree, blk & 1, abort_flag);
                                if (!ok) break;
                                PROF(3)
                                TRACE(5)
                                tc_fence_after();
                                ok = do_s(kbase + (j + 1 - lo));
                                if (!ok) break;
                            }
                            // dQ += dS(j) K_j
                            PROF(7)
                            ok = mbar_wait(bar_dsready, blk & 1, abort_flag);
                            if (!ok) break;
                            PROF(4)
                            TRACE(6)
                            tc_fence_after();
                            const uint32_t kidx = kbase + (j - lo);
                            {
                                const uint64_t ka = sdesc_advance(mdesc0, L::kKOff + (kidx % L::kKStages) * L::kTileBytes);
    #pragma unroll
                                for (int kk = 0; kk < 8; ++kk)  // 16 keys per step; group c left dS of its keys at columns CW c ..
                                    mma_ts(tmem_base + kColDQ,
                                           tmem_base + kColDP + (kk / (kDqCW / 16)) * kDqCW + (kk % (kDqCW / 16)) * 8,
                                           sdesc_advance(ka, kk * 2048), idesc_dq, (j > lo || kk > 0) ? 1u : 0u);
                                tc_commit(&bar_kempty[kidx % L::kKStages]);
                            }
                            TRACE(7)
                            if (j + 1 <= hi) ok = do_dp();  // dP(j+1) over dS(j), after dQ(j) in pipe order
                            TRACE(15)
                            TRACE(16)
                        }
                        if (!ok) break;
                        kcnt = kbase + (hi - lo + 1);
                        tc_commit(bar_dqfull);
                    }
                }
            }
            PROF_FLUSH(true, 512 * 24 + 8)
        }
        __syncwarp();
    } else {
        // ---------------- compute groups ----------------
        constexpr int CW = kDqCW;
        const int c = warp >> 2;  // which CW key columns of each query row this group owns
        // staging duty: even groups copy Q, odd groups dO; group pair c >> 1 takes that 64-column half
        const int st_op = c & 1, st_half = c >> 1;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem_base + lane_addr + kColS + CW * c;
        const uint32_t t_dp = tmem_base + lane_addr + kColDP + CW * c;
        uint32_t bcnt = 0, blk = 0;
        bool ok = true;
        PROF_DECL
        TRACE_DECL(1 + warp, cta == 0 && lane == 0)
        for (int idx = tile_begin; idx < tile_end && ok; ++idx) {
            const int t = p.cta_tiles[idx];
            for (int sub = 0; sub < 2 && ok; ++sub) {
                const int64_t q0 = (int64_t)(t / p.H) * (2 * kBlk) + sub * kBlk;
                if (q0 >= p.T) continue;
                const int lo = p.tok_start[q0] / kBlk, hi = (int)(q0 / kBlk);
                const int64_t row = q0 + r;
                const bool row_ok = row < p.T;
                const int kstart = row_ok ? p.tok_start[row] : 0;
                const int64_t last_row = (q0 + kBlk <= p.T ? q0 + kBlk : p.T) - 1;
                const int max_kstart = p.tok_start[last_row];
                for (int hh = 0; hh < heads_per_shard && ok; ++hh) {
                    const int h = (t % p.H) * heads_per_shard + hh;
                    const float lse2 = p.lse2[(size_t)h * p.Tpad + row];  // padded rows hold zeros
                    const float dsum = p.dvec[(size_t)h * p.Tpad + row];
                    // ---- stage this group's operand (Q or dO) row from shared memory into TMEM ----
                    // The MMAs that read the previous unit's copy have completed: their s_full / dp_full
                    // completions were waited for above in program order.
                    ok = mbar_wait(st_op == 0 ? bar_qfull : bar_dofull, bcnt & 1, abort_flag);
                    if (!ok) break;
                    {
                        if (st_half < D / 64) {
                            const uint8_t* src = smem + (st_op == 0 ? L::kQOff : L::kDoOff) + st_half * L::kHalfBytes + r * 128;
                            const uint32_t t_dst = tmem_base + lane_addr + (st_op == 0 ? kColQ : kColDO) + 32 * st_half;
                            uint32_t w[32];
#pragma unroll
                            for (int ch = 0; ch < 8; ++ch) {
                                const uint4 v = *reinterpret_cast<const uint4*>(src + ((ch ^ (r & 7)) << 4));
                                w[4 * ch] = v.x; w[4 * ch + 1] = v.y; w[4 * ch + 2] = v.z; w[4 * ch + 3] = v.w;
                            }
                            tmem_st32(t_dst, w);
                            tmem_st_wait();
                        }
                        mbar_arrive(st_op == 0 ? bar_qempty : bar_doempty);  // the smem tile may be reloaded
                        tc_fence_before();
                        mbar_arrive(bar_qtready);
                    }
                    ++bcnt;
                    for (int j = lo; j <= hi && ok; ++j, ++blk) {
                        const int k0 = j * kBlk;
                        const bool need_mask = (j == hi) || (k0 < max_kstart) || !row_ok;
                        const int c_lo = (row_ok ? kstart - k0 : kBlk) - CW * c;    // first visible column of this group's range
                        const int c_hi = (row_ok ? (int)(row - k0) : -1) - CW * c;  // last visible column
                        // ---- P = exp2(S c - LSE) ----
                        PROF(4)
                        ok = mbar_wait(bar_sfull, blk & 1, abort_flag);
                        if (!ok) break;
                        PROF(0)
                        TRACE(10)
                        tc_fence_after();
                        uint32_t sv[CW];
#pragma unroll
                        for (int i = 0; i < CW; i += 32) tmem_ld32(t_s + i, sv + i);
                        tmem_ld_wait();
                        tc_fence_before();
                        mbar_arrive(bar_sfree);  // S(j+1) may overwrite the columns
                        TRACE(14)
                        float pf[CW];
#pragma unroll
                        for (int i = 0; i < CW; i += 2) {
                            pf[i] = ex2_sel(fmaf(__uint_as_float(sv[i]), p.scale_log2, -lse2), i);
                            pf[i + 1] = ex2_sel(fmaf(__uint_as_float(sv[i + 1]), p.scale_log2, -lse2), i + 1);
                        }
                        if (need_mask) {
#pragma unroll
                            for (int i = 0; i < CW; ++i)
                                if (i < c_lo || i > c_hi) pf[i] = 0.f;
                        }
                        // ---- dS = P o (dP - D), packed over this half's own dP columns ----
                        PROF(1)
                        TRACE(11)
                        ok = mbar_wait(bar_dpfull, blk & 1, abort_flag);
                        if (!ok) break;
                        PROF(2)
                        TRACE(12)
                        tc_fence_after();
                        uint32_t dpv[CW];
#pragma unroll
                        for (int i = 0; i < CW; i += 32) tmem_ld32(t_dp + i, dpv + i);
                        tmem_ld_wait();
                        {
                            uint32_t pk[CW / 2];
#pragma unroll
                            for (int i = 0; i < CW; i += 2)
                                pk[i >> 1] = pack_bf16x2(pf[i] * (__uint_as_float(dpv[i]) - dsum),
                                                         pf[i + 1] * (__uint_as_float(dpv[i + 1]) - dsum));
                            if constexpr (CW == 64) tmem_st32(t_dp, pk); else tmem_st16(t_dp, pk);
                        }
                        tmem_st_wait();
                        tc_fence_before();
                        mbar_arrive(bar_dsready);
                        PROF(3)
                        TRACE(13)
                    }
                    if (!ok) break;
                    // ---- epilogue: dQ * scale to global ----
                    ok = mbar_wait(bar_dqfull, (bcnt - 1) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    constexpr int kCols = D / kDqGroups;
                    constexpr int kChunk = kCols < 32 ? kCols : 32;
                    const uint32_t t_dq = tmem_base + lane_addr + kColDQ + c * kCols;
                    __nv_bfloat16* gdst = p.dq + ((size_t)row * p.hq + h) * D + c * kCols;
#pragma unroll
                    for (int cc = 0; cc < kCols; cc += kChunk) {
                        uint32_t v[kChunk];
                        if constexpr (kChunk == 32) tmem_ld32(t_dq + cc, v); else tmem_ld16(t_dq + cc, v);
                        tmem_ld_wait();
                        if (row_ok) {
#pragma unroll
                            for (int i = 0; i < kChunk; i += 8) {
                                uint4 w;
                                w.x = pack_bf16x2(__uint_as_float(v[i]) * p.scale, __uint_as_float(v[i + 1]) * p.scale);
                                w.y = pack_bf16x2(__uint_as_float(v[i + 2]) * p.scale, __uint_as_float(v[i + 3]) * p.scale);
                                w.z = pack_bf16x2(__uint_as_float(v[i + 4]) * p.scale, __uint_as_float(v[i + 5]) * p.scale);
                                w.w = pack_bf16x2(__uint_as_float(v[i + 6]) * p.scale, __uint_as_float(v[i + 7]) * p.scale);
                                *reinterpret_cast<uint4*>(gdst + cc + i) = w;
                            }
                        }
                    }
                    tc_fence_before();  // the next dQ MMA follows this group's next ds_ready arrival
                }
            }
        }
        PROF_FLUSH(threadIdx.x == 0, 512 * 24)
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    if (warp == kDqMmaWarp) tmem_dealloc(tmem_base, 512);
    if (threadIdx.x == 0) {
        if (*abort_flag) atomicExch(p.status, LIBRA_ERR_TIMEOUT);
        p.busy[2 * cta + 1] = globaltimer_ns();
    }
}

}  // namespace libra
