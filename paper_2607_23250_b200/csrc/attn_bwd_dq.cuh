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
// Units are chained the same way: once a thread has seen the last S and dP of a unit complete it copies
// the next unit's Q / dO row over the old one, so S and dP of the next unit's first block are issued right
// behind the last dQ of this one, and the dQ read-out overlaps them.
#pragma once

namespace libra {

#ifndef LIBRA_DQ_PREFETCH
#define LIBRA_DQ_PREFETCH 0
#endif
constexpr int kDqGroups = 4;                      // compute warpgroups: each owns 128 / kDqGroups key columns
constexpr int kDqCW = 128 / kDqGroups;            // S / dP columns per compute thread
// The producer / MMA warps sit in a warpgroup of their own (two of its warps idle) so that it can hand
// registers to the compute groups with setmaxnreg.
constexpr int kDqThreads = (4 * kDqGroups + 4) * 32;
constexpr int kDqRegsCompute = 104, kDqRegsOther = 40;  // from 96 at launch: 4 x 128 x 8 asked, 128 x 56 released
constexpr int kDqTmaWarp = 4 * kDqGroups, kDqMmaWarp = 4 * kDqGroups + 1, kDqStoreWarp = 4 * kDqGroups + 2;

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
    // s_full, s_free, dp_full, ds_ready, dq_full, dot_ready, dq_empty, dq_staged, drain
    static constexpr int kNumBars = 24;
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
    const int* plan_status;
    uint32_t wait_limit_ns;
    int inject_stall;
    uint64_t* busy;
};

// Walks the units of one CTA in the order every role uses: tiles of the CTA's list x the two 128-row
// sub-blocks of a tile x the heads of the shard.  A sub-block past the end of the pool is skipped.
struct DqUnit {
    int64_t q0;
    int lo, hi, h;  // key blocks lo..hi, query head h
    bool valid;
};
struct DqUnitIter {
    const DqParams& p;
    int idx, end, sub, hh, hps;
    int t;  // cta_tiles[idx], fetched when idx moves so that the load has a unit's time to land
    __device__ DqUnitIter(const DqParams& p_, int begin, int end_, int heads_per_shard)
        : p(p_), idx(begin), end(end_), sub(0), hh(0), hps(heads_per_shard) {
        t = idx < end ? p.cta_tiles[idx] : 0;
    }
    __device__ DqUnit next() {
        DqUnit u;
        u.valid = false;
        while (idx < end) {
            const int64_t q0 = (int64_t)(t / p.H) * (2 * kBlk) + sub * kBlk;
            const bool live = q0 < p.T;
            if (live) {
                u.q0 = q0;
                u.lo = p.tok_start[q0] / kBlk;
                u.hi = (int)(q0 / kBlk);
                u.h = (t % p.H) * hps + hh;
                u.valid = true;
            }
            if (!live || ++hh == hps) {
                hh = 0;
                if (++sub == 2) {
                    sub = 0;
                    ++idx;
                    t = idx < end ? p.cta_tiles[idx] : 0;
                }
            }
            if (live) return u;
        }
        return u;
    }
};

template <int D>
__global__ void __launch_bounds__(kDqThreads, 1)
k_attn_bwd_dq(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
              const __grid_constant__ CUtensorMap tm_dq, const DqParams p) {
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
    uint64_t* bar_dotready = bars + 20;
    uint64_t* bar_dqempty = bars + 21;
    uint64_t* bar_dqstaged = bars + 22;
    uint64_t* bar_drain = bars + 23;   // teardown after a give-up: every MMA issued so far has completed
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
        mbar_init(bar_qfull, 1);
        mbar_init(bar_qempty, 1);                // the thread that stores dQ through the Q tile
        mbar_init(bar_dofull, 1);
        mbar_init(bar_doempty, 64 * kDqGroups);  // the groups that stage dO
        for (int s = 0; s < L::kKStages; ++s) { mbar_init(&bar_kfull[s], 1); mbar_init(&bar_kempty[s], 1); }
        for (int s = 0; s < L::kVStages; ++s) { mbar_init(&bar_vfull[s], 1); mbar_init(&bar_vempty[s], 1); }
        mbar_init(bar_qtready, 64 * kDqGroups);   // the groups that stage Q
        mbar_init(bar_dotready, 64 * kDqGroups);  // the groups that stage dO
        mbar_init(bar_dqempty, 128 * kDqGroups);
        mbar_init(bar_dqstaged, 128 * kDqGroups);
        mbar_init(bar_sfull, 1);
        mbar_init(bar_sfree, 128 * kDqGroups);
        mbar_init(bar_dpfull, 1);
        mbar_init(bar_dsready, 128 * kDqGroups);
        mbar_init(bar_dqfull, 1);
        mbar_init(bar_drain, 1);
        abort_flag[0] = 0;
        abort_flag[1] = (int)p.wait_limit_ns;
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
        prefetch_tmap(&tm_dq);
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
    if (warp > kDqStoreWarp) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDqRegsOther));
    } else if (warp == kDqStoreWarp) {
        // ---------------- dQ store ----------------
        // The compute groups leave a unit's dQ tile (bf16, the swizzled layout of the tensor map) in the Q tile
        // of shared memory, which is idle between the copy of the next unit's Q into TMEM and the load of the
        // one after; one thread writes it out with bulk tensor stores.  Rows stored straight from registers
        // (one row per thread, rows 2*hq*D bytes apart) touch 32 cache lines per instruction and took ~3000
        // cycles per unit.
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDqRegsOther));
        if (elect_one()) {
            DqUnitIter units(p, tile_begin, tile_end, heads_per_shard);
            DqUnit u = units.next();
            uint32_t cnt = 0;
            bool ok = true;
            if (u.valid) {  // first unit: its Q rows have been copied to TMEM, the tile may be reloaded
                ok = mbar_wait(bar_dqstaged, 0, abort_flag);
                cnt = 1;
                if (ok) mbar_arrive(bar_qempty);
            }
            while (u.valid && ok) {
                ok = mbar_wait(bar_dqstaged, cnt & 1, abort_flag);
                ++cnt;
                if (!ok) break;
                for (int half = 0; half < D / 64; ++half)
                    tma_store_3d(&tm_dq, smem + L::kQOff + half * L::kHalfBytes, half * 64, u.h, (int)u.q0);
                tma_store_commit();
                tma_store_wait_read();
                mbar_arrive(bar_qempty);
                u = units.next();
            }
            asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // all of this thread's stores have landed
        }
        __syncwarp();
    } else if (warp == kDqTmaWarp) {
        // ---------------- TMA producer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDqRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            uint32_t ucnt = 0, kcnt = 0, vcnt = 0;
            uint32_t n_q = 0, n_do = 0;   // Q / dO loads armed so far (for the give-up path)
            bool ok = true;
            // Tiles a unit will need are pulled into L2 this many key blocks ahead: the shared-memory rings
            // hold one block of lead, which covers an L2 hit but not a first touch in DRAM.
            constexpr int kAhead = LIBRA_DQ_PREFETCH;
            auto prefetch_kv = [&](int kvh, int j) {
                for (int half = 0; half < D / 64; ++half) {
                    tma_prefetch_3d(&tm_k, half * 64, kvh, j * kBlk);
                    tma_prefetch_3d(&tm_v, half * 64, kvh, j * kBlk);
                }
            };
            DqUnitIter units(p, tile_begin, tile_end, heads_per_shard);
            DqUnit u = units.next();
            // Q and dO of unit `un`, whose tiles go through phase `cnt` of their barriers.  The shared-memory
            // copies are free again as soon as the compute groups have moved the previous unit's rows into
            // TMEM, which happens at the end of the unit before it: the next unit's Q and dO (first touches,
            // DRAM latency) can therefore be requested a whole unit ahead.
            auto load_q_do = [&](const DqUnit& un, uint32_t cnt) -> bool {
                if (!mbar_wait(bar_qempty, (cnt & 1) ^ 1, abort_flag)) return false;
                mbar_arrive_expect_tx(bar_qfull, L::kTileBytes);
                ++n_q;
                for (int half = 0; half < D / 64; ++half)
                    tma_load_3d(smem + L::kQOff + half * L::kHalfBytes, &tm_q, bar_qfull, half * 64, un.h, (int)un.q0);
                if (!mbar_wait(bar_doempty, (cnt & 1) ^ 1, abort_flag)) return false;
                mbar_arrive_expect_tx(bar_dofull, L::kTileBytes);
                ++n_do;
                for (int half = 0; half < D / 64; ++half)
                    tma_load_3d(smem + L::kDoOff + half * L::kHalfBytes, &tm_do, bar_dofull, half * 64, un.h, (int)un.q0);
                return true;
            };
            if (p.inject_stall) u.valid = false;   // test aid: no loads at all
            if (u.valid) ok = load_q_do(u, 0);
            while (u.valid && ok) {
                const DqUnit nx = units.next();
                const int h = u.h, kvh = h / G, lo = u.lo, hi = u.hi;
                const int j_q = lo + 1 < hi ? lo + 1 : hi;  // after this block's K/V the next unit's Q / dO are requested
                ++ucnt;
                const int j_next = hi - kAhead > lo ? hi - kAhead : lo;  // where the next unit's first tiles are requested
                for (int j = lo; j <= hi && ok; ++j) {
                    if (kAhead > 0) {
                        if (j + kAhead <= hi) prefetch_kv(kvh, j + kAhead);
                        if (j == j_next && nx.valid) {
                            for (int half = 0; half < D / 64; ++half) {
                                tma_prefetch_3d(&tm_q, half * 64, nx.h, (int)nx.q0);
                                tma_prefetch_3d(&tm_do, half * 64, nx.h, (int)nx.q0);
                            }
                            for (int jj = nx.lo; jj <= nx.hi && jj < nx.lo + kAhead; ++jj) prefetch_kv(nx.h / G, jj);
                        }
                    }
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
                    if (j == j_q && nx.valid) {
                        ok = load_q_do(nx, ucnt);
                        if (!ok) break;
                        if (kAhead == 0)   // pull the next unit's first K / V blocks into L2 meanwhile
                            for (int jj = nx.lo; jj <= nx.hi && jj < nx.lo + 2; ++jj) prefetch_kv(nx.h / G, jj);
                    }
                }
                u = nx;
            }
            if (!ok || abort_flag[0]) {
                // Give-up path: nothing new is issued; the copies already issued land before shared memory is released.
                if (n_q > 0) mbar_wait_drain(bar_qfull, (n_q - 1) & 1, kDrainNs);
                if (n_do > 0) mbar_wait_drain(bar_dofull, (n_do - 1) & 1, kDrainNs);
                for (uint32_t b = 1; b <= (uint32_t)L::kKStages && b <= kcnt; ++b)
                    mbar_wait_drain(&bar_kfull[(kcnt - b) % L::kKStages], ((kcnt - b) / L::kKStages) & 1, kDrainNs);
                for (uint32_t b = 1; b <= (uint32_t)L::kVStages && b <= vcnt; ++b)
                    mbar_wait_drain(&bar_vfull[(vcnt - b) % L::kVStages], ((vcnt - b) / L::kVStages) & 1, kDrainNs);
            }
        }
        __syncwarp();
    } else if (warp == kDqMmaWarp) {
        // ---------------- MMA issuer ----------------
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kDqRegsOther));
        if (elect_one()) {  // one elected thread runs the whole role
            constexpr uint32_t idesc_s = make_idesc(128, 128, 0, 0);  // S, dP: A in TMEM, B K-major
            constexpr uint32_t idesc_dq = make_idesc(128, D, 0, 1);   // dQ: A in TMEM, B = K MN-major
            const uint32_t sb = smem_u32(smem);
            const uint64_t kdesc0 = make_sdesc(sb, 16, 1024);             // K-major view of a tile at offset 0
            const uint64_t mdesc0 = make_sdesc(sb, L::kHalfBytes, 1024);  // MN-major view
            uint32_t kcnt = 0, vcnt = 0, blk = 0;
            bool ok = true;
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
                if (!mbar_wait(&bar_kfull[kidx % L::kKStages], (kidx / L::kKStages) & 1, abort_flag)) return false;
                {
                    issue_qk(kColS, kColQ, L::kKOff + (kidx % L::kKStages) * L::kTileBytes);
                    tc_commit(bar_sfull);
                }
                return true;
            };
            auto do_dp = [&]() -> bool {
                const uint32_t vs = vcnt % L::kVStages;
                if (!mbar_wait(&bar_vfull[vs], (vcnt / L::kVStages) & 1, abort_flag)) return false;
                {
                    issue_qk(kColDP, kColDO, L::kVOff + vs * L::kTileBytes);
                    tc_commit(bar_dpfull);
                    tc_commit(&bar_vempty[vs]);
                }
                ++vcnt;
                return true;
            };
            DqUnitIter units(p, tile_begin, tile_end, heads_per_shard);
            DqUnit u = units.next();
            uint32_t ucnt = 0;
            if (u.valid) {  // first unit: nothing to overlap its first S and dP with
                ok = mbar_wait(bar_qtready, 0, abort_flag);
                if (ok) { tc_fence_after(); ok = do_s(kcnt); }
                if (ok) ok = mbar_wait(bar_dotready, 0, abort_flag);
                if (ok) { tc_fence_after(); ok = do_dp(); }
            }
            while (u.valid && ok) {
                const DqUnit nx = units.next();
                const int lo = u.lo, hi = u.hi;
                const uint32_t kbase = kcnt;  // ring index of K_lo
                for (int j = lo; j <= hi && ok; ++j, ++blk) {
                    const bool last = j == hi;
                    // S(j+1) as soon as the compute groups have read S(j)
                    if (!last) {
                        ok = mbar_wait(bar_sfree, blk & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        ok = do_s(kbase + (j + 1 - lo));
                        if (!ok) break;
                    }
                    // dQ += dS(j) K_j
                    ok = mbar_wait(bar_dsready, blk & 1, abort_flag);
                    if (ok && j == lo && ucnt > 0) ok = mbar_wait(bar_dqempty, (ucnt - 1) & 1, abort_flag);  // dQ read out
                    if (!ok) break;
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
                        if (last) tc_commit(bar_dqfull);
                    }
                    if (!last) {
                        ok = do_dp();  // dP(j+1) over dS(j), after dQ(j) in pipe order
                    } else if (nx.valid) {
                        // first block of the next unit, behind the last dQ of this one: its Q and dO rows
                        // were copied into TMEM while that dQ ran
                        ok = mbar_wait(bar_sfree, blk & 1, abort_flag);
                        if (ok) ok = mbar_wait(bar_qtready, (ucnt + 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        ok = do_s(kbase + (hi - lo + 1));
                        if (ok) ok = mbar_wait(bar_dotready, (ucnt + 1) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after();
                        ok = do_dp();
                    }
                }
                kcnt = kbase + (hi - lo + 1);
                ++ucnt;
                u = nx;
            }
            if (!ok || abort_flag[0]) {   // give-up path: the MMAs already issued finish before TMEM is freed
                tc_commit(bar_drain);
                mbar_wait_drain(bar_drain, 0, kDrainNs);
            }
        }
        __syncwarp();
    } else {
        // ---------------- compute groups ----------------
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kDqRegsCompute));
        constexpr int CW = kDqCW;
        const int c = warp >> 2;  // which CW key columns of each query row this group owns
        // staging duty: even groups copy Q, odd groups dO; group pair c >> 1 takes that 64-column half
        const int st_op = c & 1, st_half = c >> 1;
        const int r = (warp & 3) * 32 + lane;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem_base + lane_addr + kColS + CW * c;
        const uint32_t t_dp = tmem_base + lane_addr + kColDP + CW * c;
        uint32_t ucnt = 0, blk = 0;
        bool ok = true;
        // Copies this thread's row of Q or dO (its group's duty) of the unit whose tile has landed into TMEM.
        // The caller has seen every MMA that read the previous copy complete (s_full for Q, dp_full for dO).
        auto stage = [&](uint32_t parity) -> bool {
            if (!warp_wait(st_op == 0 ? bar_qfull : bar_dofull, parity, abort_flag)) return false;
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
            if (st_op == 1) mbar_arrive(bar_doempty);  // the dO tile may be reloaded (the Q tile: see the dQ store)
            tc_fence_before();
            mbar_arrive(st_op == 0 ? bar_qtready : bar_dotready);
            return true;
        };
        // Per-row values of a unit, fetched one unit ahead so the loads are off the path between units.
        struct RowCtx {
            float lse2, dsum;
            int kstart, max_kstart;
            bool row_ok;
        };
        auto load_ctx = [&](const DqUnit& un) {
            RowCtx x;
            const int64_t row = un.q0 + r;
            x.row_ok = row < p.T;
            x.kstart = x.row_ok ? p.tok_start[row] : 0;
            const int64_t last_row = (un.q0 + kBlk <= p.T ? un.q0 + kBlk : p.T) - 1;
            x.max_kstart = p.tok_start[last_row];
            x.lse2 = p.lse2[(size_t)un.h * p.Tpad + row];  // padded rows hold zeros
            x.dsum = p.dvec[(size_t)un.h * p.Tpad + row];
            return x;
        };
        DqUnitIter units(p, tile_begin, tile_end, heads_per_shard);
        DqUnit u = units.next();
        RowCtx cx{};
        if (u.valid) {
            cx = load_ctx(u);
            ok = stage(0);
            mbar_arrive(bar_dqstaged);   // phase 0: the store thread frees the Q tile once every row has been read
        }
        while (u.valid && ok) {
            const DqUnit nx = units.next();
            RowCtx cx_next{};
            if (nx.valid) cx_next = load_ctx(nx);
            const int lo = u.lo, hi = u.hi;
            const int64_t row = u.q0 + r;
            const bool row_ok = cx.row_ok;
            const int kstart = cx.kstart, max_kstart = cx.max_kstart;
            const float lse2 = cx.lse2, dsum = cx.dsum;
            for (int j = lo; j <= hi && ok; ++j, ++blk) {
                const int k0 = j * kBlk;
                const bool need_mask = (j == hi) || (k0 < max_kstart) || !row_ok;
                const int c_lo = (row_ok ? kstart - k0 : kBlk) - CW * c;    // first visible column of this group's range
                const int c_hi = (row_ok ? (int)(row - k0) : -1) - CW * c;  // last visible column
                // ---- P = exp2(S c - LSE) ----
                ok = warp_wait(bar_sfull, blk & 1, abort_flag);
                if (!ok) break;
                tc_fence_after();
                uint32_t sv[CW];
#pragma unroll
                for (int i = 0; i < CW; i += 32) tmem_ld32(t_s + i, sv + i);
                tmem_ld_wait();
                tc_fence_before();
                mbar_arrive(bar_sfree);  // S(j+1) may overwrite the columns
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
                ok = warp_wait(bar_dpfull, blk & 1, abort_flag);
                if (!ok) break;
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
                // Last block of the unit: every S and dP MMA that read this unit's Q / dO copy has completed, so
                // the next unit's row goes into TMEM now, while the tensor pipe runs the last dQ.
                if (j == hi && nx.valid) {
                    ok = stage((ucnt + 1) & 1);
                }
            }
            if (!ok) break;
            // ---- epilogue: dQ * scale to global ----
            ok = warp_wait(bar_dqfull, ucnt & 1, abort_flag);
            if (!ok) break;
            tc_fence_after();
            constexpr int kCols = D / kDqGroups;   // this group's dQ columns: kCols * 2 bytes of every row
            const uint32_t t_dq = tmem_base + lane_addr + kColDQ + c * kCols;
            uint32_t v[kCols];
            if constexpr (kCols == 32) tmem_ld32(t_dq, v); else tmem_ld16(t_dq, v);
            tmem_ld_wait();
            // The Q tile still holds the next unit's Q until every row of it has been copied to TMEM.
            if (nx.valid) ok = warp_wait(bar_qtready, (ucnt + 1) & 1, abort_flag);
            if (!ok) break;
            {
                uint8_t* dst = smem + L::kQOff + ((c * kCols) / 64) * L::kHalfBytes + r * 128;
                const int chunk0 = ((c * kCols) % 64) / 8;  // first 16-byte chunk of this group's columns
#pragma unroll
                for (int i = 0; i < kCols; i += 8) {
                    uint4 w;
                    w.x = pack_bf16x2(__uint_as_float(v[i]) * p.scale, __uint_as_float(v[i + 1]) * p.scale);
                    w.y = pack_bf16x2(__uint_as_float(v[i + 2]) * p.scale, __uint_as_float(v[i + 3]) * p.scale);
                    w.z = pack_bf16x2(__uint_as_float(v[i + 4]) * p.scale, __uint_as_float(v[i + 5]) * p.scale);
                    w.w = pack_bf16x2(__uint_as_float(v[i + 6]) * p.scale, __uint_as_float(v[i + 7]) * p.scale);
                    *reinterpret_cast<uint4*>(dst + (((chunk0 + i / 8) ^ (r & 7)) << 4)) = w;
                }
            }
            fence_proxy_async_smem();     // the bulk store reads these writes through the async proxy
            mbar_arrive(bar_dqstaged);
            tc_fence_before();
            mbar_arrive(bar_dqempty);  // the next unit's first dQ MMA may overwrite the accumulator
            ++ucnt;
            u = nx;
            cx = cx_next;
        }
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
