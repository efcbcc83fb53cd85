// Parallel unmask selection on the int32 token state, in place.  One CTA per row.
// The rule is decided by rank: position i's rank is the number of masked block positions that beat it
// (higher fp32 confidence, or equal confidence and lower index).  TOPK commits ranks < k; THRESHOLD
// commits conf > tau, and rank 0 when nothing passes.  Integer/bit-exact; a few KB of traffic.
#include <math.h>

#include "internal.h"

namespace dare {
namespace {

constexpr int SEL_THREADS = 128;
constexpr int SEL_MAX_L = 4096;

__global__ void __launch_bounds__(SEL_THREADS)
unmask_select_kernel(int32_t* __restrict__ tokens, int64_t row_stride, int block_start, int L,
                     const int32_t* __restrict__ pred, const float* __restrict__ conf, int32_t mask_id, int mode,
                     float threshold, int k, int32_t* __restrict__ n_committed, int32_t* __restrict__ n_remaining) {
    extern __shared__ float s_conf[];   // [L]; -inf for NaN; positions that are not masked hold NaN as "absent"
    __shared__ int s_masked, s_above, s_commit;
    const int r = blockIdx.x;
    int32_t* row = tokens + static_cast<int64_t>(r) * row_stride + block_start;
    if (threadIdx.x == 0) { s_masked = 0; s_above = 0; s_commit = 0; }
    __syncthreads();
    int local_masked = 0, local_above = 0;
    for (int i = threadIdx.x; i < L; i += SEL_THREADS) {
        const bool masked = row[i] == mask_id;
        float c = conf[static_cast<int64_t>(r) * L + i];
        if (c != c) c = -INFINITY;
        s_conf[i] = masked ? c : __int_as_float(0x7fc00000);
        if (masked) {
            ++local_masked;
            if (c > threshold) ++local_above;
        }
    }
    if (local_masked) atomicAdd(&s_masked, local_masked);
    if (local_above) atomicAdd(&s_above, local_above);
    __syncthreads();
    const int n_masked = s_masked;
    const int n_above = s_above;
    int local_commit = 0;
    for (int i = threadIdx.x; i < L; i += SEL_THREADS) {
        const float c = s_conf[i];
        if (c != c) continue;   // not masked: committed tokens are never touched
        bool commit;
        if (mode == DARE_SELECT_THRESHOLD && n_above > 0) {
            commit = c > threshold;
        } else {
            const int want = (mode == DARE_SELECT_TOPK) ? k : 1;
            int rank = 0;
            for (int j = 0; j < L; ++j) {
                const float cj = s_conf[j];
                rank += (cj > c || (cj == c && j < i)) ? 1 : 0;   // NaN (absent) compares false
            }
            commit = rank < want;
        }
        if (commit) {
            row[i] = pred[static_cast<int64_t>(r) * L + i];
            ++local_commit;
        }
    }
    if (local_commit) atomicAdd(&s_commit, local_commit);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (n_committed) n_committed[r] = s_commit;
        if (n_remaining) n_remaining[r] = n_masked - s_commit;
    }
}

}  // namespace

int launch_unmask_select(int32_t* tokens, int B, int64_t row_stride, int block_start, int L, const int32_t* pred,
                         const float* conf, int32_t mask_id, int mode, float threshold, int k, int32_t* n_committed,
                         int32_t* n_remaining, cudaStream_t stream) {
    if (L > SEL_MAX_L) return DARE_ERR_SHAPE;
    unmask_select_kernel<<<B, SEL_THREADS, L * sizeof(float), stream>>>(tokens, row_stride, block_start, L, pred, conf,
                                                                        mask_id, mode, threshold, k, n_committed,
                                                                        n_remaining); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

}  // namespace dare
