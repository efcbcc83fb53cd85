// The bandwidth-bound pieces of the layer stack: embedding gather, RMSNorm, and RoPE with the in-place
// K/V cache write.  Each is one pass over its rows with 128-bit accesses; fp32 inside, bf16 in memory.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace dare {
namespace {

constexpr int ROWS_PER_BLOCK = 8;   // one warp per row

__device__ __forceinline__ float lo_f(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float hi_f(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// x[m, :] = E[tokens[b, start + i], :] for row m = b * length + i.
__global__ void __launch_bounds__(ROWS_PER_BLOCK * 32)
embed_gather_kernel(const uint4* __restrict__ emb, int D8, int V, const int32_t* __restrict__ tokens, int64_t row_stride,
                    int start, int length, int n_rows, uint4* __restrict__ x) {
    const int m = blockIdx.x * ROWS_PER_BLOCK + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= n_rows) return;
    int tok = tokens[static_cast<int64_t>(m / length) * row_stride + start + m % length];
    tok = min(max(tok, 0), V - 1);
    const uint4* src = emb + static_cast<size_t>(tok) * D8;
    uint4* dst = x + static_cast<size_t>(m) * D8;
    for (int i = lane; i < D8; i += 32) dst[i] = src[i];
}

// y = x / sqrt(mean(x^2) + eps), weight 1.  Two passes over the row (the second one hits L1/L2).
__global__ void __launch_bounds__(ROWS_PER_BLOCK * 32)
rmsnorm_kernel(const uint4* __restrict__ x, int D8, int n_rows, float eps, uint4* __restrict__ y) {
    const int m = blockIdx.x * ROWS_PER_BLOCK + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (m >= n_rows) return;
    const uint4* src = x + static_cast<size_t>(m) * D8;
    float ss = 0.f;
    for (int i = lane; i < D8; i += 32) {
        const uint4 v = src[i];
        const float a0 = lo_f(v.x), a1 = hi_f(v.x), a2 = lo_f(v.y), a3 = hi_f(v.y);
        const float a4 = lo_f(v.z), a5 = hi_f(v.z), a6 = lo_f(v.w), a7 = hi_f(v.w);
        ss += a0 * a0 + a1 * a1 + a2 * a2 + a3 * a3 + a4 * a4 + a5 * a5 + a6 * a6 + a7 * a7;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
    const float inv = rsqrtf(ss / static_cast<float>(D8 * 8) + eps);
    uint4* dst = y + static_cast<size_t>(m) * D8;
    for (int i = lane; i < D8; i += 32) {
        const uint4 v = src[i];
        uint4 o;
        o.x = pack_bf16(lo_f(v.x) * inv, hi_f(v.x) * inv);
        o.y = pack_bf16(lo_f(v.y) * inv, hi_f(v.y) * inv);
        o.z = pack_bf16(lo_f(v.z) * inv, hi_f(v.z) * inv);
        o.w = pack_bf16(lo_f(v.w) * inv, hi_f(v.w) * inv);
        dst[i] = o;
    }
}

// cs[p, c] = (cos, sin)(p * base^(-2c/d)), c < d/2, evaluated in double precision.
__global__ void rope_table_kernel(float2* __restrict__ cs, int n_pos, int half, double base) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_pos * half) return;
    const int p = i / half, c = i % half;
    const double ang = static_cast<double>(p) * pow(base, -static_cast<double>(c) / static_cast<double>(half));
    double s, co;
    sincos(ang, &s, &co);
    cs[i] = make_float2(static_cast<float>(co), static_cast<float>(s));
}

// Row m = (b, i) of the fused QKV projection [n_rows, (Hq + 2 Hkv) d], position p = start + i:
//   q heads  -> q_out[m, h, :] rotated;  k heads -> k_cache[b, h, p, :] rotated;  v heads -> v_cache[b, h, p, :].
// Half-split pairing: channel c turns together with channel c + d/2.  A work item is 8 channels c..c+7 of one
// head (and their partners), or one 8-channel chunk of a v head.
__global__ void __launch_bounds__(128)
rope_kv_write_kernel(const __nv_bfloat16* __restrict__ qkv, int Hq, int Hkv, int d, int start, int length,
                     const float2* __restrict__ cs, __nv_bfloat16* __restrict__ q_out,
                     __nv_bfloat16* __restrict__ k_cache, __nv_bfloat16* __restrict__ v_cache, int cap) {
    const int m = blockIdx.x;
    const int b = m / length, i = m % length, p = start + i;
    const int half = d / 2, cpb = half / 8;                 // 8-channel chunks per half head
    const int n_rot = (Hq + Hkv) * cpb;
    const int n_items = n_rot + Hkv * (d / 8);
    const size_t ld = static_cast<size_t>(Hq + 2 * Hkv) * d;
    const __nv_bfloat16* row = qkv + static_cast<size_t>(m) * ld;
    for (int it = threadIdx.x; it < n_items; it += blockDim.x) {
        if (it < n_rot) {
            const int h = it / cpb, c0 = (it % cpb) * 8;
            const uint4 a = *reinterpret_cast<const uint4*>(row + static_cast<size_t>(h) * d + c0);
            const uint4 bb = *reinterpret_cast<const uint4*>(row + static_cast<size_t>(h) * d + half + c0);
            const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {bb.x, bb.y, bb.z, bb.w};
            uint32_t o1[4], o2[4];
            const float2* t = cs + static_cast<size_t>(p) * half + c0;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 t0 = t[2 * j], t1 = t[2 * j + 1];
                const float x10 = lo_f(aw[j]), x11 = hi_f(aw[j]), x20 = lo_f(bw[j]), x21 = hi_f(bw[j]);
                o1[j] = pack_bf16(x10 * t0.x - x20 * t0.y, x11 * t1.x - x21 * t1.y);
                o2[j] = pack_bf16(x20 * t0.x + x10 * t0.y, x21 * t1.x + x11 * t1.y);
            }
            __nv_bfloat16* dst = h < Hq ? q_out + (static_cast<size_t>(m) * Hq + h) * d
                                        : k_cache + ((static_cast<size_t>(b) * Hkv + (h - Hq)) * cap + p) * d;
            *reinterpret_cast<uint4*>(dst + c0) = make_uint4(o1[0], o1[1], o1[2], o1[3]);
            *reinterpret_cast<uint4*>(dst + half + c0) = make_uint4(o2[0], o2[1], o2[2], o2[3]);
        } else {
            const int j = it - n_rot, h = j / (d / 8), c0 = (j % (d / 8)) * 8;
            const uint4 v = *reinterpret_cast<const uint4*>(row + static_cast<size_t>(Hq + Hkv + h) * d + c0);
            *reinterpret_cast<uint4*>(v_cache + ((static_cast<size_t>(b) * Hkv + h) * cap + p) * d + c0) = v;
        }
    }
}

}  // namespace

int launch_embed(const void* emb, int D, int V, const int32_t* tokens, int64_t row_stride, int start, int length,
                 int n_rows, void* x, cudaStream_t stream) {
    embed_gather_kernel<<<(n_rows + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK, ROWS_PER_BLOCK * 32, 0, stream>>>(
        static_cast<const uint4*>(emb), D / 8, V, tokens, row_stride, start, length, n_rows, static_cast<uint4*>(x)); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int launch_rmsnorm(const void* x, int D, int n_rows, float eps, void* y, cudaStream_t stream) {
    rmsnorm_kernel<<<(n_rows + ROWS_PER_BLOCK - 1) / ROWS_PER_BLOCK, ROWS_PER_BLOCK * 32, 0, stream>>>(
        static_cast<const uint4*>(x), D / 8, n_rows, eps, static_cast<uint4*>(y)); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int launch_rope_table(float* cs, int n_pos, int half, double base, cudaStream_t stream) {
    const int n = n_pos * half;
    rope_table_kernel<<<(n + 255) / 256, 256, 0, stream>>>(reinterpret_cast<float2*>(cs), n_pos, half, base); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int launch_rope_kv_write(const void* qkv, int n_rows, int Hq, int Hkv, int d, int start, int length, const float* cs,
                         void* q_out, void* k_cache, void* v_cache, int cap, cudaStream_t stream) {
    rope_kv_write_kernel<<<n_rows, 128, 0, stream>>>(static_cast<const __nv_bfloat16*>(qkv), Hq, Hkv, d, start, length,
                                                     reinterpret_cast<const float2*>(cs),
                                                     static_cast<__nv_bfloat16*>(q_out),
                                                     static_cast<__nv_bfloat16*>(k_cache),
                                                     static_cast<__nv_bfloat16*>(v_cache), cap); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

}  // namespace dare
