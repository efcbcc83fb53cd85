// Forward (corruption) process of masked diffusion and the Monte-Carlo likelihood bound built on it.
//   forward_mask_kernel  Eq. 1: every token of a row's window independently becomes <MASK> with probability
//                        1 - alpha_t, decided by a counter-based uniform (Philox4x32-10 keyed by the seed, counter =
//                        (position / 4, row, Monte-Carlo sample, tag)), so any draw can be reproduced anywhere.
//   masked_nelbo_kernel  Eq. 2: -(1 / t) * sum of log p(x_0 | x_t) over the window positions that are masked in x_t.
// Both are a few KB to a few MB of traffic: one pass, no shared state.
#include <math.h>

#include "internal.h"

namespace dare {
namespace {

constexpr uint32_t MASK_TAG = 0x4D41534Bu;

__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c.x), lo0 = 0xD2511F53u * c.x;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c.z), lo1 = 0xCD9E8D57u * c.z;
        c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return c;
}

// One thread per group of 4 window positions (one generator call).  xt may alias x0.
__global__ void forward_mask_kernel(const int32_t* x0, int32_t* xt, int64_t row_stride, int start, int length,
                                    const float* __restrict__ p_mask, int32_t mask_id, uint32_t seed_lo,
                                    uint32_t seed_hi, uint32_t sample) {
    const int b = blockIdx.y;
    const int q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q * 4 >= length) return;
    const uint4 w4 = philox4x32_10(make_uint4(static_cast<uint32_t>(q), static_cast<uint32_t>(b), sample, MASK_TAG),
                                   seed_lo, seed_hi);
    const uint32_t ww[4] = {w4.x, w4.y, w4.z, w4.w};
    const float p = p_mask[b];
    const int64_t base = static_cast<int64_t>(b) * row_stride + start;
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int i = q * 4 + e;
        if (i < length) {
            const float u = static_cast<float>(((ww[e] >> 9) << 1) | 1u) * 5.9604644775390625e-08f;   // (2 k + 1) / 2^24
            xt[base + i] = u < p ? mask_id : x0[base + i];
        }
    }
}

// One warp per row.
__global__ void masked_nelbo_kernel(const float* __restrict__ logprob, const int32_t* __restrict__ xt, int B,
                                    int64_t row_stride, int start, int length, int32_t mask_id,
                                    const float* __restrict__ t, float* __restrict__ nelbo,
                                    int32_t* __restrict__ n_masked) {
    const int b = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (b >= B) return;
    const int32_t* row = xt + static_cast<int64_t>(b) * row_stride + start;
    const float* lp = logprob + static_cast<int64_t>(b) * length;
    float s = 0.f;
    int n = 0;
    for (int i = lane; i < length; i += 32)
        if (row[i] == mask_id) { s += lp[i]; ++n; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        s += __shfl_xor_sync(0xffffffffu, s, off);
        n += __shfl_xor_sync(0xffffffffu, n, off);
    }
    if (lane == 0) {
        nelbo[b] = -s / t[b];
        if (n_masked) n_masked[b] = n;
    }
}

}  // namespace

int launch_forward_mask(const int32_t* x0, int32_t* xt, int B, int64_t row_stride, int start, int length,
                        const float* p_mask, int32_t mask_id, uint64_t seed, uint32_t sample, cudaStream_t stream) {
    const int groups = (length + 3) / 4;
    dim3 grid((groups + 127) / 128, B, 1);
    forward_mask_kernel<<<grid, 128, 0, stream>>>(x0, xt, row_stride, start, length, p_mask, mask_id,
                                                  static_cast<uint32_t>(seed & 0xffffffffu),
                                                  static_cast<uint32_t>(seed >> 32), sample); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int launch_masked_nelbo(const float* logprob, const int32_t* xt, int B, int64_t row_stride, int start, int length,
                        int32_t mask_id, const float* t, float* nelbo, int32_t* n_masked, cudaStream_t stream) {
    masked_nelbo_kernel<<<(B + 3) / 4, 128, 0, stream>>>(logprob, xt, B, row_stride, start, length, mask_id, t, nelbo,
                                                         n_masked); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

}  // namespace dare

extern "C" {

int dare_forward_mask(dare_ctx* ctx, const int32_t* x0, int32_t* xt, int B, int64_t row_stride, int start, int length,
                      const float* p_mask, int32_t mask_id, uint64_t seed, uint32_t sample, void* stream) {
    if (!ctx || !x0 || !xt || !p_mask) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (B < 1 || B > 65535 || length < 1) return DARE_ERR_SHAPE;
    if (start < 0 || row_stride < 1 || static_cast<int64_t>(start) + length > row_stride) return DARE_ERR_RANGE;
    return dare::launch_forward_mask(x0, xt, B, row_stride, start, length, p_mask, mask_id, seed, sample,
                                     static_cast<cudaStream_t>(stream));
}

int dare_masked_nelbo(dare_ctx* ctx, const float* logprob, const int32_t* xt, int B, int64_t row_stride, int start,
                      int length, int32_t mask_id, const float* t, float* nelbo, int32_t* n_masked, void* stream) {
    if (!ctx || !logprob || !xt || !t || !nelbo) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (B < 1 || length < 1) return DARE_ERR_SHAPE;
    if (start < 0 || row_stride < 1 || static_cast<int64_t>(start) + length > row_stride) return DARE_ERR_RANGE;
    return dare::launch_masked_nelbo(logprob, xt, B, row_stride, start, length, mask_id, t, nelbo, n_masked,
                                     static_cast<cudaStream_t>(stream));
}

}  // extern "C"
