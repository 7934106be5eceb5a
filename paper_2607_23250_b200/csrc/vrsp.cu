// Variance-Reduced Sequence Placement (Algorithm 1) on the device.
//
// Packed sequences of one optimizer-step window are grouped into K = D / P pools of exactly P
// sequences so that the pools' summed attention work is even: sequences in decreasing work order
// (ties: lower index first) each go to the least-loaded pool that still has room (ties: lower pool
// index).  The paper runs this on a CPU core per step (48-106 us for D = 128-256); here it is three
// small kernels on the caller's stream so that a data path that already lives on the GPU does not
// have to come back to the host.  Integer only; results are bit-identical to the sequential rule.
#include <cstdint>
#include <cuda_runtime.h>

#include "../../include/libra.h"
#include "common.h"

namespace libra {

// F_i = sum over the samples of sequence i of len^2 (the work proxy of Section 4.2).
__global__ void k_vrsp_work(const int32_t* __restrict__ sample_offsets, const int32_t* __restrict__ seq_first_sample,
                            int D, int64_t* __restrict__ work) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= D) return;
    int64_t f = 0;
    for (int j = seq_first_sample[i]; j < seq_first_sample[i + 1]; ++j) {
        const int64_t len = (int64_t)sample_offsets[j + 1] - sample_offsets[j];
        f += len * len;
    }
    work[i] = f;
}

// rank of sequence i in the order (work descending, index ascending); one thread per sequence.
__global__ void k_vrsp_rank(const int64_t* __restrict__ work, int D, int32_t* __restrict__ sorted) {
    __shared__ int64_t sw[256];
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t wi = i < D ? work[i] : 0;
    int rank = 0;
    for (int base = 0; base < D; base += 256) {
        const int o = base + threadIdx.x;
        sw[threadIdx.x] = o < D ? work[o] : -1;
        __syncthreads();
        const int lim = D - base < 256 ? D - base : 256;
        for (int k = 0; k < lim; ++k) {
            const int64_t w = sw[k];
            rank += (w > wi) || (w == wi && base + k < i);
        }
        __syncthreads();
    }
    if (i < D) sorted[rank] = i;
}

// One warp places the sequences one after the other.  Pool k's load and fill count live in lane
// k % 32, register k / 32; a full pool's load is replaced by INT64_MAX in the comparison, which is
// what removing it from the algorithm's heap does.  Popping the heap's minimum (load, k) is the
// lexicographic arg-min taken here.
template <int PER>
__global__ void __launch_bounds__(32) k_vrsp_place(const int64_t* __restrict__ work, const int32_t* __restrict__ sorted,
                                                   int D, int P, int K, int32_t* __restrict__ order,
                                                   int32_t* __restrict__ pool_of_seq, int64_t* __restrict__ pool_load) {
    const int lane = threadIdx.x;
    int64_t load[PER];
    int32_t cnt[PER];
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        load[i] = 0;
        cnt[i] = (lane + 32 * i < K) ? 0 : P;  // pools that do not exist count as full
    }
    for (int x0 = 0; x0 < D; x0 += 32) {
        const int xl = x0 + lane;
        int32_t s_l = 0;
        int64_t w_l = 0;
        if (xl < D) { s_l = sorted[xl]; w_l = work[s_l]; }
        const int lim = D - x0 < 32 ? D - x0 : 32;
        for (int i = 0; i < lim; ++i) {
            const int64_t w = __shfl_sync(0xffffffffu, w_l, i);
            const int32_t sq = __shfl_sync(0xffffffffu, s_l, i);
            int64_t best = INT64_MAX;
            int32_t bidx = INT32_MAX;
#pragma unroll
            for (int k = 0; k < PER; ++k) {
                if (cnt[k] < P && (load[k] < best || bidx == INT32_MAX)) { best = load[k]; bidx = lane + 32 * k; }
            }
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) {
                const int64_t ob = __shfl_xor_sync(0xffffffffu, best, off);
                const int32_t oi = __shfl_xor_sync(0xffffffffu, bidx, off);
                // a lane without a candidate carries bidx = INT32_MAX and never wins
                if (oi != INT32_MAX && (bidx == INT32_MAX || ob < best || (ob == best && oi < bidx))) { best = ob; bidx = oi; }
            }
            if (bidx != INT32_MAX && (bidx & 31) == lane) {
#pragma unroll
                for (int k = 0; k < PER; ++k) {
                    if (k == (bidx >> 5)) {
                        order[(int64_t)bidx * P + cnt[k]] = sq;  // pools are concatenated in pool order
                        load[k] += w;
                        cnt[k] += 1;
                    }
                }
                pool_of_seq[sq] = bidx;
            }
        }
    }
#pragma unroll
    for (int i = 0; i < PER; ++i) {
        const int k = lane + 32 * i;
        if (k < K) pool_load[k] = load[i];
    }
}

}  // namespace libra

using namespace libra;

extern "C" int libra_vrsp_work(const int32_t* sample_offsets_dev, const int32_t* seq_first_sample_dev, int n_sequences,
                               int64_t* work_dev, void* stream) {
    if (!sample_offsets_dev || !seq_first_sample_dev || !work_dev || n_sequences <= 0) return LIBRA_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    k_vrsp_work<<<(n_sequences + 127) / 128, 128, 0, s>>>(sample_offsets_dev, seq_first_sample_dev, n_sequences, work_dev);
    count_launch(1);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}

extern "C" int libra_vrsp_place(const int64_t* work_dev, int n_sequences, int pool_size, int32_t* order_dev,
                                int32_t* pool_of_seq_dev, int64_t* pool_load_dev, int32_t* scratch_dev, void* stream) {
    if (!work_dev || !order_dev || !pool_of_seq_dev || !pool_load_dev || !scratch_dev) return LIBRA_ERR_INVALID_ARG;
    if (n_sequences <= 0 || pool_size <= 0 || n_sequences % pool_size != 0) return LIBRA_ERR_INVALID_ARG;
    const int D = n_sequences, P = pool_size, K = D / P;
    if (K > 1024 || D > (1 << 20)) return LIBRA_ERR_UNSUPPORTED;
    cudaStream_t s = (cudaStream_t)stream;
    k_vrsp_rank<<<(D + 255) / 256, 256, 0, s>>>(work_dev, D, scratch_dev);
    if (K <= 32)
        k_vrsp_place<1><<<1, 32, 0, s>>>(work_dev, scratch_dev, D, P, K, order_dev, pool_of_seq_dev, pool_load_dev);
    else if (K <= 128)
        k_vrsp_place<4><<<1, 32, 0, s>>>(work_dev, scratch_dev, D, P, K, order_dev, pool_of_seq_dev, pool_load_dev);
    else
        k_vrsp_place<32><<<1, 32, 0, s>>>(work_dev, scratch_dev, D, P, K, order_dev, pool_of_seq_dev, pool_load_dev);
    count_launch(2);
    return cudaGetLastError() == cudaSuccess ? LIBRA_OK : LIBRA_ERR_CUDA;
}
