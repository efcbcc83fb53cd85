// Backward of the log-probability head (the actor update differentiates the per-token log-probabilities of
// Section 3.4): host-side sequencing of three kernels plus a small transpose.
//   1. the LM-head main loop again, with the gradient epilogue: dz = g * (onehot(target) - softmax(z)) from the
//      recomputed logits and the forward pass's logsumexp, written as bf16 in both orientations;
//   2. d_hidden [M, D] = dz [M, V] . w        (projection kernel, K = V, with the caller's transposed weights)
//   3. d_w      [V, D] = dz^T [V, M] . hidden (projection kernel, K = M, with hidden transposed into the workspace)
// Logits are never stored; dz (bf16, both orientations) is the only M x V intermediate and lives in buffers the
// caller provides, so the caller bounds it by the number of rows it passes per call.
#include <cuda_bf16.h>

#include "internal.h"

namespace dare {
int launch_lmhead_grad(const dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V,
                       const int32_t* targets, int32_t mask_id, int exclude_mask_column, const float* lse,
                       const float* grad, void* dz, void* dzt, int ldm, cudaStream_t stream);

namespace {

// out[c, r] = in[r, c] for a bf16 matrix [rows, cols]; 32 x 32 tiles through shared memory (padded: no bank
// conflicts), both sides coalesced.
__global__ void __launch_bounds__(256)
transpose_bf16_kernel(const unsigned short* __restrict__ in, int rows, int cols, unsigned short* __restrict__ out) {
    __shared__ unsigned short tile[32][34];
    const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;      // 32 x 8 threads
    for (int i = ty; i < 32; i += 8) {
        const int r = r0 + i, c = c0 + tx;
        tile[i][tx] = (r < rows && c < cols) ? in[static_cast<size_t>(r) * cols + c] : static_cast<unsigned short>(0);
    }
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int c = c0 + i, r = r0 + tx;
        if (c < cols && r < rows) out[static_cast<size_t>(c) * rows + r] = tile[tx][i];
    }
}

int launch_transpose(const void* in, int rows, int cols, void* out, cudaStream_t stream) {
    dim3 grid((cols + 31) / 32, (rows + 31) / 32, 1);
    if (grid.y > 65535u) return DARE_ERR_SHAPE;
    transpose_bf16_kernel<<<grid, 256, 0, stream>>>(static_cast<const unsigned short*>(in), rows, cols,
                                                    static_cast<unsigned short*>(out)); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace dare

extern "C" {

int dare_transpose_bf16(dare_ctx* ctx, const void* in, int rows, int cols, void* out, void* stream) {
    if (!ctx || !in || !out) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (rows < 1 || cols < 1) return DARE_ERR_SHAPE;
    if (in == out) return DARE_ERR_RANGE;
    // the tile grid puts the row tiles on the y axis (65 535 at most): transpose the longer side along x
    if ((rows + 31) / 32 > 65535) return DARE_ERR_SHAPE;
    return dare::launch_transpose(in, rows, cols, out, static_cast<cudaStream_t>(stream));
}

int dare_lmhead_logprob_backward(dare_ctx* ctx, const void* hidden, int M, int D, const void* w, const void* w_t, int V,
                                 const int32_t* targets, int32_t mask_id, int exclude_mask_column, const float* lse,
                                 const float* grad_logprob, void* dz, void* dzt, void* d_hidden, void* d_w, void* stream) {
    if (!ctx || !hidden || !w || !w_t || !targets || !lse || !grad_logprob || !dz || !dzt || !d_hidden || !d_w)
        return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (M < 8 || D < 8 || V < 8 || (M % 8) || (D % 8) || (V % 8)) return DARE_ERR_SHAPE;
    if (!dare::aligned16(hidden) || !dare::aligned16(w) || !dare::aligned16(w_t) || !dare::aligned16(dz) ||
        !dare::aligned16(dzt) || !dare::aligned16(d_hidden) || !dare::aligned16(d_w))
        return DARE_ERR_ALIGN;
    const size_t xt_bytes = static_cast<size_t>(M) * D * 2;
    if (xt_bytes > ctx->workspace_bytes) return DARE_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int rc = dare::launch_lmhead_grad(ctx, hidden, M, D, w, V, targets, mask_id, exclude_mask_column, lse, grad_logprob,
                                      dz, dzt, M, s);
    if (rc != DARE_OK) return rc;
    rc = dare::launch_transpose(hidden, M, D, ctx->workspace, s);                      // hidden^T [D, M]
    if (rc != DARE_OK) return rc;
    rc = dare::launch_gemm(ctx, dare::GEMM_EPI_STORE, dz, M, V, w_t, nullptr, D, d_hidden, nullptr, D, s);
    if (rc != DARE_OK) return rc;
    return dare::launch_gemm(ctx, dare::GEMM_EPI_STORE, dzt, V, M, ctx->workspace, nullptr, D, d_w, nullptr, D, s);
}

}  // extern "C"
