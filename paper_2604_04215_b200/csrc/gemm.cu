// Dense bf16 projections of the layer stack on the tcgen05 tensor cores: out = epilogue(A W^T).
//
// A [M, K] activations and W [N, K] weights are both K-major bf16, so one pipeline serves every projection:
//   warp 0      TMA producer: A tile [128 x 64] and W tile [BN x 64] per stage (128-byte swizzle)
//   warp 1      UMMA issuer: 128 x BN x 16 MMAs into one of two fp32 accumulators in TMEM
//   warps 2..5  epilogue: one TMEM lane = one output row per thread, 32 columns at a time
// Two accumulators let the epilogue of one tile overlap the MMAs of the next.  CTAs are persistent and walk
// the tiles with the row-tile index fastest, so the CTAs that share a weight tile run at the same time and the
// weights leave HBM once.
// Epilogues: plain bf16 store (QKV projection); residual add, rounded once after the add (attention output
// and feed-forward down projections, in place on the residual stream); SwiGLU, where a 256-column tile holds
// 128 gate columns and the matching 128 up columns (two TMA loads, one per matrix) and silu(g) * u is formed
// in registers, so the 2F-wide intermediate never reaches memory.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace dare {
namespace {

constexpr int GM = 128;
constexpr int GK = 64;
constexpr int GEMM_THREADS = 192;
constexpr int A_TILE_BYTES = GM * GK * 2;

template <int BN>
struct GemmShape {
    static constexpr int STAGES = BN == 256 ? 4 : 6;
    static constexpr int B_TILE_BYTES = BN * GK * 2;
    static constexpr int STAGE_BYTES = A_TILE_BYTES + B_TILE_BYTES;
    static constexpr uint32_t TMEM_COLS = 2 * BN;
};

template <int STAGES>
struct GemmBarriers {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int BN>
constexpr int gemm_smem_bytes() {
    return GemmShape<BN>::STAGES * GemmShape<BN>::STAGE_BYTES +
           static_cast<int>(sizeof(GemmBarriers<GemmShape<BN>::STAGES>)) + 1024;
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// N = rows of W covered by the output (EPI_SWIGLU: rows of each of the two matrices); n_cols_per_tile is BN,
// or 128 for EPI_SWIGLU.  `res` may alias `out` (every element is read and written by the same thread).
template <int BN, int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_b2, int M, int N, int K, __nv_bfloat16* out,
                 const __nv_bfloat16* res, int ldo, uint32_t* __restrict__ dev_status) {
    using S = GemmShape<BN>;
    constexpr int STAGES = S::STAGES;
    constexpr int OUT_COLS = EPI == GEMM_EPI_SWIGLU ? BN / 2 : BN;   // output columns per tile
    static_assert(EPI != GEMM_EPI_SWIGLU || BN == 256, "the SwiGLU tile pairs 128 gate with 128 up columns");

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GemmBarriers<STAGES>* bars = reinterpret_cast<GemmBarriers<STAGES>*>(tiles + STAGES * S::STAGE_BYTES);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int m_tiles = (M + GM - 1) / GM;
    const int n_tiles = (N + OUT_COLS - 1) / OUT_COLS;
    const int n_work = m_tiles * n_tiles;
    const int num_k = (K + GK - 1) / GK;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->tmem_full[a], 1);
            mbar_init(&bars->tmem_empty[a], 128);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, S::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_a);
            prefetch_tensormap(&tmap_b);
            if (EPI == GEMM_EPI_SWIGLU) prefetch_tensormap(&tmap_b2);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_work && ok; t += gridDim.x) {
                const int m_tile = t % m_tiles, n_tile = t / m_tiles;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                    uint8_t* a_dst = tiles + stage * S::STAGE_BYTES;
                    uint8_t* b_dst = a_dst + A_TILE_BYTES;
                    mbar_arrive_expect_tx(&bars->full[stage], S::STAGE_BYTES);
                    tma_load_2d(a_dst, &tmap_a, &bars->full[stage], kb * GK, m_tile * GM);
                    if (EPI == GEMM_EPI_SWIGLU) {
                        tma_load_2d(b_dst, &tmap_b, &bars->full[stage], kb * GK, n_tile * 128);
                        tma_load_2d(b_dst + 128 * GK * 2, &tmap_b2, &bars->full[stage], kb * GK, n_tile * 128);
                    } else {
                        tma_load_2d(b_dst, &tmap_b, &bars->full[stage], kb * GK, n_tile * BN);
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = umma_idesc_bf16(GM, BN);
            int stage = 0;
            uint32_t phase = 0;
            int it = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < n_work && ok; t += gridDim.x, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_k; ++kb) {
                    if (!mbar_wait(&bars->full[stage], phase, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(tiles + stage * S::STAGE_BYTES);
                    const uint64_t a_desc = umma_desc_sw128_kmajor(a_addr);
                    const uint64_t b_desc = umma_desc_sw128_kmajor(a_addr + A_TILE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < GK / 16; ++kk)   // +32 bytes along K per step = +2 descriptor units
                        umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
                    umma_commit(&bars->empty[stage]);
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
                if (ok) umma_commit(&bars->tmem_full[acc]);
            }
        }
    } else {
        const int lq = warp & 3;   // warp w may touch TMEM lanes [32 * (w % 4), +32)
        int it = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < n_work && ok; t += gridDim.x, ++it) {
            const int m_tile = t % m_tiles, n_tile = t / m_tiles;
            const int acc = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!mbar_wait(&bars->tmem_full[acc], acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lq * 32) << 16) + acc * BN;
            const int row = m_tile * GM + lq * 32 + lane;
            const size_t row_off = static_cast<size_t>(row) * ldo;
#pragma unroll 1
            for (int c = 0; c < OUT_COLS / 32; ++c) {
                uint32_t v[32];
                const int col0 = n_tile * OUT_COLS + c * 32;
                if (EPI == GEMM_EPI_SWIGLU) {
                    uint32_t u[32];
                    tmem_ld_32cols(taddr + c * 32, v);
                    tmem_ld_32cols(taddr + 128 + c * 32, u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float g = __uint_as_float(v[j]);
                        const float s = __fdividef(g, 1.0f + __expf(-g));      // silu(g)
                        v[j] = __float_as_uint(s * __uint_as_float(u[j]));
                    }
                } else {
                    tmem_ld_32cols(taddr + c * 32, v);
                    tmem_ld_wait();
                }
                if (row < M) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int col = col0 + q * 8;
                        if (col < N) {    // N is a multiple of 8: a group of 8 columns is inside or outside
                            float f[8];
#pragma unroll
                            for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[q * 8 + j]);
                            if (EPI == GEMM_EPI_RESIDUAL) {
                                const uint4 r = *reinterpret_cast<const uint4*>(res + row_off + col);
                                f[0] += bf16_lo(r.x); f[1] += bf16_hi(r.x); f[2] += bf16_lo(r.y); f[3] += bf16_hi(r.y);
                                f[4] += bf16_lo(r.z); f[5] += bf16_hi(r.z); f[6] += bf16_lo(r.w); f[7] += bf16_hi(r.w);
                            }
                            uint4 o;
                            o.x = pack_bf16(f[0], f[1]); o.y = pack_bf16(f[2], f[3]);
                            o.z = pack_bf16(f[4], f[5]); o.w = pack_bf16(f[6], f[7]);
                            *reinterpret_cast<uint4*>(out + row_off + col) = o;
                        }
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(&bars->tmem_empty[acc]);
        }
    }

    // teardown
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}   // let copies in flight land before the shared memory goes away
        if (threadIdx.x == 0) atomicOr(dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, S::TMEM_COLS);
    }
}

template <int BN, int EPI>
int launch_one(const dare_ctx* ctx, const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, int M, int N,
               int K, void* out, const void* res, int ldo, int tiles, cudaStream_t stream) {
    constexpr int SMEM = gemm_smem_bytes<BN>();
    if (cudaFuncSetAttribute(gemm_bf16_kernel<BN, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
        return DARE_ERR_CUDA;
    const int grid = tiles < ctx->sm_count ? tiles : ctx->sm_count;
    gemm_bf16_kernel<BN, EPI><<<grid, GEMM_THREADS, SMEM, stream>>>(ta, tb, tb2, M, N, K, static_cast<__nv_bfloat16*>(out),
                                                                    static_cast<const __nv_bfloat16*>(res), ldo,
                                                                    ctx->dev_status);
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

}  // namespace

int launch_gemm(const dare_ctx* ctx, int epi, const void* a, int M, int K, const void* w, const void* w2, int N,
                void* out, const void* res, int ldo, cudaStream_t stream) {
    if (M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8) || (ldo % 8)) return DARE_ERR_SHAPE;
    const int m_tiles = (M + GM - 1) / GM;
    CUtensorMap ta, tb, tb2;
    int rc = make_tmap_bf16_2d(ctx, &ta, a, static_cast<uint64_t>(M), static_cast<uint64_t>(K), GM, GK);
    if (rc != DARE_OK) return rc;
    if (epi == GEMM_EPI_SWIGLU) {
        rc = make_tmap_bf16_2d(ctx, &tb, w, static_cast<uint64_t>(N), static_cast<uint64_t>(K), 128, GK);
        if (rc == DARE_OK) rc = make_tmap_bf16_2d(ctx, &tb2, w2, static_cast<uint64_t>(N), static_cast<uint64_t>(K), 128, GK);
        if (rc != DARE_OK) return rc;
        return launch_one<256, GEMM_EPI_SWIGLU>(ctx, ta, tb, tb2, M, N, K, out, res, ldo, m_tiles * ((N + 127) / 128), stream);
    }
    // tile width by the number of waves it takes: a 256-wide tile costs two 128-wide ones
    const long long t256 = static_cast<long long>(m_tiles) * ((N + 255) / 256);
    const long long t128 = static_cast<long long>(m_tiles) * ((N + 127) / 128);
    const long long sms = ctx->sm_count;
    const bool wide = 2 * ((t256 + sms - 1) / sms) <= (t128 + sms - 1) / sms;
    rc = make_tmap_bf16_2d(ctx, &tb, w, static_cast<uint64_t>(N), static_cast<uint64_t>(K), wide ? 256 : 128, GK);
    if (rc != DARE_OK) return rc;
    if (epi == GEMM_EPI_STORE)
        return wide ? launch_one<256, GEMM_EPI_STORE>(ctx, ta, tb, tb, M, N, K, out, res, ldo, static_cast<int>(t256), stream)
                    : launch_one<128, GEMM_EPI_STORE>(ctx, ta, tb, tb, M, N, K, out, res, ldo, static_cast<int>(t128), stream);
    if (epi == GEMM_EPI_RESIDUAL)
        return wide ? launch_one<256, GEMM_EPI_RESIDUAL>(ctx, ta, tb, tb, M, N, K, out, res, ldo, static_cast<int>(t256), stream)
                    : launch_one<128, GEMM_EPI_RESIDUAL>(ctx, ta, tb, tb, M, N, K, out, res, ldo, static_cast<int>(t128), stream);
    return DARE_ERR_RANGE;
}

}  // namespace dare
