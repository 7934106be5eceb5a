// Host-side structures shared by the library's translation units.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/libra.h"

namespace libra {

// One direction (query-major or key-major) of a plan.  All d_* pointers are device memory.
struct PlanDir {
    int enabled = 0;
    int tile = 0;        // tokens per block
    int H = 0;           // head shards
    int W = 0;           // workers (persistent CTAs)
    int64_t NB = 0;      // blocks
    int64_t NT = 0;      // tiles = NB * H
    int64_t* d_weight_blk = nullptr;   // [NB]  weight of block b (every shard of it)
    int32_t* d_blk_order = nullptr;    // [NB]  blocks by (weight desc, index asc)
    int32_t* d_cta_of_tile = nullptr;  // [NT]
    int32_t* d_pos = nullptr;          // [NT]  position of the tile in its worker's list
    int32_t* d_cta_offsets = nullptr;  // [W+1]
    int32_t* d_cta_tiles = nullptr;    // [NT]  per-worker lists in placement order (the plan proper)
    int32_t* d_cta_exec = nullptr;     // [NT]  the same lists, each re-ordered for execution (head-major)
    int64_t* d_loads = nullptr;        // [W]
    uint64_t* d_busy = nullptr;        // [2*W] (start, end) global-timer stamps of the last run
    uint64_t* d_busy2 = nullptr;       // [2*W] same, for the second kernel that walks this direction (dQ)
    uint32_t* d_tile_ns = nullptr;     // [NT] time the last run spent on each tile (forward / fused backward), ns
    // pair tiles only (key block x query chunk x head): the "blocks" above are pair-blocks
    int chunk = 0;                     // tokens per query chunk
    int32_t* d_u_blk = nullptr;        // [NB] key block of pair-block u
    int32_t* d_u_chunk = nullptr;      // [NB] query chunk of pair-block u
};

}  // namespace libra

struct libra_plan {
    int64_t T = 0;
    int n = 0;
    int device = 0;
    int sm_count = 0;
    cudaStream_t stream = nullptr;
    int32_t* d_tok_start = nullptr;  // [T] first token of the sample that holds token t
    int32_t* d_tok_end = nullptr;    // [T] one past the last token of that sample
    int* d_status = nullptr;         // [4] word 0: plan status; word 1: fwd; word 2: bwd
    libra::PlanDir dir[3];           // 0 = query-major, 1 = key-major, 2 = pair tiles (key block x query chunk)
    uint32_t wait_limit_ns = 2000000000u;  // budget of one device-side wait (libra_plan_set_wait_limit_ns)
    int inject_stall = 0;            // test aid: the producer role issues no loads (libra_plan_inject_stall)
    int timing = 0;                  // record events around the main kernels
    // [kernel][slot][begin, end]: a ring of the most recent launches of each kernel (LIBRA_KERNEL_* - 1)
    static constexpr int kTimedKernels = 6, kTimeRing = 64;
    cudaEvent_t ev[kTimedKernels][kTimeRing][2] = {};
    int64_t ev_count[kTimedKernels] = {0, 0, 0, 0, 0, 0};   // launches recorded since timing was switched on
};

namespace libra {
// Per-device one-time kernel configuration (dynamic shared memory size, register-pool check).  The
// attributes are per device, so the flag is kept per device ordinal; `slot` is a small integer the
// caller picks per kernel family.  Returns true when this (device, slot) has been configured.
constexpr int kMaxDevices = 64;
constexpr int kCfgSlots = 16;
bool cfg_done(int slot);
void cfg_mark(int slot);
// LIBRA_ERR_PLAN_MISMATCH when the current device is not the one the plan was built on.
int check_plan_device(const libra_plan* plan);
// Kernel timing (libra_plan_set_timing): events on the launch stream around kernel k (LIBRA_KERNEL_* - 1).
inline void time_begin(libra_plan* p, int k, cudaStream_t s) {
    if (p->timing) cudaEventRecord(p->ev[k][p->ev_count[k] % libra_plan::kTimeRing][0], s);
}
inline void time_end(libra_plan* p, int k, cudaStream_t s) {
    if (p->timing) { cudaEventRecord(p->ev[k][p->ev_count[k] % libra_plan::kTimeRing][1], s); ++p->ev_count[k]; }
}
extern std::atomic<int64_t> g_launches;
inline void count_launch(int n = 1) { g_launches.fetch_add(n, std::memory_order_relaxed); }
}  // namespace libra

namespace libra {
// bf16 [T, H, d] tensor viewed as (d, H, T); TMA box = 64 columns x 1 head x box_rows tokens,
// 128-byte swizzle, out-of-range rows read as zero.  Defined in attn_fwd.cu.
int make_thd_map(CUtensorMap* m, const void* base, int64_t T, int H, int d, int box_rows);
// fp32 matrix [rows, cols] (cols contiguous); box = box_cols x box_rows, 128-byte swizzle.
int make_f32_2d_map(CUtensorMap* m, const void* base, int64_t rows, int64_t cols, int box_cols, int box_rows);
// fp32 tensor [T, H, d] viewed as (d, H, T); box = box_cols x 1 x box_rows, 128-byte swizzle.
int make_f32_3d_map(CUtensorMap* m, const void* base, int64_t T, int H, int d, int box_cols, int box_rows);
// head_dim 256 (attn_d256.cu): the forward over the plan's query-major lists; the three gradient passes over
// its key-major (dV, dK) and query-major (dQ) lists, given the row statistics lse2 / dvec [Hq, Tpad].
int launch_fwd_d256(const void* q, const void* k, const void* v, void* out, float* lse, const libra_plan* plan,
                    const libra_dims* dims, float scale, cudaStream_t s);
// dk_acc / dv_acc: fp32 accumulators [T, Hkv, 256], zero on entry, when the dV and dK passes are to walk the plan's
// pair tiles (the caller rounds them afterwards); null: key-major tiles, dk / dv written directly.
int launch_bwd_d256(const void* q, const void* k, const void* v, const void* dout, void* dq, void* dk, void* dv,
                    const float* lse2, const float* dvec, int64_t Tpad, float* dk_acc, float* dv_acc,
                    const libra_plan* plan, const libra_dims* dims, float scale, cudaStream_t s);
}  // namespace libra

// setmaxnreg moves registers inside the pool the CTA got at launch (registers per thread as compiled x
// threads): what the shrinking warps release must cover what the growing warps ask for, or the last
// warpgroup to grow waits for ever.  Checked on the host against the compiled register count before the
// first launch, so that a build with other flags fails with an error instead.
template <typename Kernel>
static inline bool regs_pool_ok(Kernel k, int threads_grow, int regs_grow, int threads_shrink, int regs_shrink) {
    cudaFuncAttributes a;
    if (cudaFuncGetAttributes(&a, k) != cudaSuccess) return false;
    const long long released = (long long)(a.numRegs - regs_shrink) * threads_shrink;
    const long long wanted = (long long)(regs_grow - a.numRegs) * threads_grow;
    return a.numRegs >= regs_shrink && wanted <= released;
}
