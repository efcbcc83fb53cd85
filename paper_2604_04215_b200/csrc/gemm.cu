// Dense bf16 projections of the layer stack on the tcgen05 tensor cores: out = epilogue(A W^T).
//
// A [M, K] activations and W [N, K] weights are both K-major bf16.  Problems with two or more row tiles run on
// CTA pairs (gemm_pair_kernel, further down); the single-CTA kernel described here serves the rest and is the
// shape the pair kernel is derived from.  One CTA computes one output tile of up to
// two 128-row tiles by `bn` columns over a range of K:
//   warp 0      TMA producer: one or two A tiles [128 x 64] and a W tile [bn x 64] per stage (128-byte swizzle)
//   warp 1      UMMA issuer: 128 x bn x 16 MMAs, one fp32 accumulator in TMEM per row tile
//   warps 2..9  epilogue: one TMEM lane = one output row per thread, 8 columns at a time
// The tile shape is chosen per problem on the host (gemm_plan): at the few hundred rows of a denoising step a
// projection has too few 128 x 256 tiles to fill the SMs evenly, so the column width bn (any multiple of 16)
// and, for long K, a split of K are picked so that the CTAs make whole waves; two row tiles per CTA share
// each W tile, which keeps the shared-memory and L2 traffic per flop low.  CTAs are numbered with the row index
// fastest, so the CTAs that share a weight tile run at the same time and the weights leave HBM once.
// Epilogues: plain bf16 store (QKV projection); residual add, rounded once after the add (attention output
// and feed-forward down projections, in place on the residual stream); SwiGLU, where a tile holds w gate
// columns and the matching w up columns (two TMA loads, one per matrix) and silu(g) * u is formed in
// registers, so the 2F-wide intermediate never reaches memory.
// Split K: the CTAs that share an output tile form a thread-block cluster.  After the main loop each CTA
// sends, through distributed shared memory, the accumulator column groups it does not own into the idle
// operand ring of the CTA that owns them; every CTA then adds the partials of its own groups in split order
// and applies the epilogue, so all CTAs of the cluster share the output work and nothing goes through HBM.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace dare {
namespace {

constexpr int GM = 128;
constexpr int GK = 64;
constexpr int GEMM_THREADS = 320;
constexpr int A_TILE_BYTES = GM * GK * 2;
constexpr int MAX_STAGES = 8;
constexpr int RING_BYTES = 226 * 1024;      // shared memory for the operand ring (the CTA has 227 KB)
constexpr int MAX_SPLITS = 2;                // CTAs along K per output tile (pairs are always co-resident)
constexpr int L2_AHEAD = 8;                 // pipeline steps between the L2 prefetch of a W tile and its load

struct GemmBarriers {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t tmem_full;
    uint32_t tmem_base;
    uint32_t abort_flag;
};
constexpr int GEMM_SMEM_BYTES = RING_BYTES - 1024;   // dynamic request; the ring starts at the next 1 KB boundary

struct GemmPlan {
    int nsub;        // row tiles per CTA (1 or 2)
    int bn;          // MMA N: columns of W per tile (SwiGLU: w gate rows + w up rows)
    int wcols;       // output columns per tile (bn, or bn / 2 for SwiGLU)
    int splits;      // CTAs along K per output tile
    int stages;
    int m_items, n_tiles;
    uint32_t tmem_cols;
};

struct GemmArgs {
    int M, N, K, ldo;
    GemmPlan p;
    __nv_bfloat16* out;
    const __nv_bfloat16* res;
    uint32_t* dev_status;
};

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Applies the epilogue to 8 accumulated columns of one row and stores them.  `res` may alias `out`.
template <int EPI>
__device__ __forceinline__ void store_group(const float (&f)[8], const float (&u)[8], __nv_bfloat16* out,
                                            const __nv_bfloat16* res, size_t off) {
    float r[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) r[j] = f[j];
    if (EPI == GEMM_EPI_RESIDUAL) {
        const uint4 x = *reinterpret_cast<const uint4*>(res + off);
        r[0] += bf16_lo(x.x); r[1] += bf16_hi(x.x); r[2] += bf16_lo(x.y); r[3] += bf16_hi(x.y);
        r[4] += bf16_lo(x.z); r[5] += bf16_hi(x.z); r[6] += bf16_lo(x.w); r[7] += bf16_hi(x.w);
    } else if (EPI == GEMM_EPI_SWIGLU) {
#pragma unroll
        for (int j = 0; j < 8; ++j) r[j] = __fdividef(f[j], 1.0f + __expf(-f[j])) * u[j];   // silu(g) * u
    }
    uint4 o;
    o.x = pack_bf16(r[0], r[1]); o.y = pack_bf16(r[2], r[3]);
    o.z = pack_bf16(r[4], r[5]); o.w = pack_bf16(r[6], r[7]);
    *reinterpret_cast<uint4*>(out + off) = o;
}

template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_bf16_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_b2, const GemmArgs g) {
    const GemmPlan& p = g.p;
    const int stage_bytes = p.nsub * A_TILE_BYTES + p.bn * (GK * 2);

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(tiles + p.stages * stage_bytes);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = warp_index_uniform();
    const int lane = threadIdx.x & 31;
    // CTA -> (K split, row item, column tile): the splits of one output tile form a cluster, row items next
    const int split = p.splits > 1 ? static_cast<int>(cluster_cta_rank()) : 0;
    const int m_item = (blockIdx.x / p.splits) % p.m_items;
    const int n_tile = blockIdx.x / (p.m_items * p.splits);
    const int nk = (g.K + GK - 1) / GK;
    const int kb_begin = static_cast<int>(static_cast<long long>(nk) * split / p.splits);
    const int kb_end = static_cast<int>(static_cast<long long>(nk) * (split + 1) / p.splits);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        mbar_init(&bars->tmem_full, 1);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, p.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const int acc_stride = p.nsub == 2 ? 256 : 0;   // accumulator of row tile s starts at column s * 256

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_a);
            prefetch_tensormap(&tmap_b);
            if (EPI == GEMM_EPI_SWIGLU) prefetch_tensormap(&tmap_b2);
            int stage = 0;
            uint32_t phase = 0;
            // the weights come from HBM: ask L2 for them L2_AHEAD steps before the load that needs them
            for (int kb = kb_begin; kb < kb_end && kb < kb_begin + L2_AHEAD; ++kb) {
                tma_prefetch_l2_2d(&tmap_b, kb * GK, n_tile * (EPI == GEMM_EPI_SWIGLU ? p.wcols : p.bn));
                if (EPI == GEMM_EPI_SWIGLU) tma_prefetch_l2_2d(&tmap_b2, kb * GK, n_tile * p.wcols);
            }
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                if (kb + L2_AHEAD < kb_end) {
                    tma_prefetch_l2_2d(&tmap_b, (kb + L2_AHEAD) * GK, n_tile * (EPI == GEMM_EPI_SWIGLU ? p.wcols : p.bn));
                    if (EPI == GEMM_EPI_SWIGLU) tma_prefetch_l2_2d(&tmap_b2, (kb + L2_AHEAD) * GK, n_tile * p.wcols);
                }
                if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) break;
                uint8_t* a_dst = tiles + stage * stage_bytes;
                uint8_t* b_dst = a_dst + p.nsub * A_TILE_BYTES;
                mbar_arrive_expect_tx(&bars->full[stage], stage_bytes);
                for (int s = 0; s < p.nsub; ++s)
                    tma_load_2d(a_dst + s * A_TILE_BYTES, &tmap_a, &bars->full[stage], kb * GK, (m_item * p.nsub + s) * GM);
                if (EPI == GEMM_EPI_SWIGLU) {
                    tma_load_2d(b_dst, &tmap_b, &bars->full[stage], kb * GK, n_tile * p.wcols);
                    tma_load_2d(b_dst + p.wcols * (GK * 2), &tmap_b2, &bars->full[stage], kb * GK, n_tile * p.wcols);
                } else {
                    tma_load_2d(b_dst, &tmap_b, &bars->full[stage], kb * GK, n_tile * p.bn);
                }
                if (++stage == p.stages) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // all lanes run the loop, one elected lane issues the MMAs and their commits
        const bool leader = elect_one_sync();
        const uint32_t idesc = umma_idesc_bf16(GM, p.bn);
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        for (int kb = kb_begin; kb < kb_end; ++kb) {
            ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[stage], phase, abort_flag));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t a_addr = smem_u32(tiles + stage * stage_bytes);
            const uint64_t b_desc = umma_desc_sw128_kmajor(a_addr + p.nsub * A_TILE_BYTES);
            const uint32_t accumulate = kb > kb_begin;
            if (leader) {
                for (int s = 0; s < p.nsub; ++s) {
                    const uint64_t a_desc = umma_desc_sw128_kmajor(a_addr + s * A_TILE_BYTES);
#pragma unroll
                    for (int kk = 0; kk < GK / 16; ++kk)   // +32 bytes along K per step = +2 descriptor units
                        umma_bf16(tmem_base + s * acc_stride, a_desc + 2 * kk, b_desc + 2 * kk, idesc,
                                  accumulate | (kk != 0));
                }
                umma_commit(&bars->empty[stage]);
            }
            __syncwarp();
            if (++stage == p.stages) { stage = 0; phase ^= 1; }
        }
        if (ok && leader) umma_commit(&bars->tmem_full);
        __syncwarp();
    }

    // ---- epilogue (warps 2..9).  Warp w may touch TMEM lanes [32 * (w % 4), +32); warps 2..5 are set 0, warps
    // 6..9 set 1.  Two row tiles: set s owns row tile s.  One row tile: the sets share it, alternating 8-column
    // groups.  With a K split the CTAs of the cluster first hand each other the column groups they do not own.
    const bool epi_warp = warp >= 2;
    const int lq = warp & 3;
    const int set = epi_warp ? (warp - 2) >> 2 : 0;
    const int rt = p.nsub == 2 ? set : 0;
    const int g_first = p.nsub == 2 ? 0 : set, g_step = p.nsub == 2 ? 1 : 2;
    const int n_groups = p.wcols / 8;
    const int tile_rows = p.nsub * GM;
    const int row_local = rt * GM + lq * 32 + lane;
    const int row = m_item * tile_rows + row_local;
    const bool row_ok = row < g.M;
    const size_t row_off = static_cast<size_t>(row) * g.ldo;
    const int col_base = n_tile * p.wcols;
    const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lq * 32) << 16) + rt * acc_stride;
    if (epi_warp) {
        mbar_wait(&bars->tmem_full, 0, abort_flag);     // (a wait that gave up leaves the abort flag set)
        tc_fence_after_sync();
    }
    __syncwarp();
    if (p.splits > 1) {
        // Group gi belongs to the CTA of rank gi % splits.  Receiver layout in the (now idle) operand ring:
        // [slot of the sending split, ascending, own split left out][gi / splits][row][8 floats].
        const int per_owner = (n_groups + p.splits - 1) / p.splits;
        cluster_sync_all();                              // every CTA of the cluster is done with its ring
        if (epi_warp) {
            const uint32_t ring = smem_u32(tiles);
            for (int gi = g_first; gi < n_groups; gi += g_step) {
                const int owner = gi % p.splits;
                if (owner == split) continue;
                uint32_t v[8];
                tmem_ld_8cols(taddr + gi * 8, v);
                tmem_ld_wait();
                const int slot = split < owner ? split : split - 1;
                const uint32_t local = ring + ((static_cast<uint32_t>(slot * per_owner + gi / p.splits) * tile_rows + row_local) << 5);
                const uint32_t remote = cluster_map_shared(local, static_cast<uint32_t>(owner));
                st_shared_cluster_v4(remote, v[0], v[1], v[2], v[3]);
                st_shared_cluster_v4(remote + 16, v[4], v[5], v[6], v[7]);
            }
        }
        cluster_sync_all();                              // the partials of the groups this CTA owns have arrived
    }
    if (epi_warp && !*abort_flag) {
        for (int gi = g_first; gi < n_groups; gi += g_step) {
            if (p.splits > 1 && gi % p.splits != split) continue;
            uint32_t v[8];
            float f[8], u[8];
            tmem_ld_8cols(taddr + gi * 8, v);
            if (EPI == GEMM_EPI_SWIGLU) {
                uint32_t w[8];
                tmem_ld_8cols(taddr + p.wcols + gi * 8, w);
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = __uint_as_float(w[j]);
            } else {
                tmem_ld_wait();
#pragma unroll
                for (int j = 0; j < 8; ++j) u[j] = 0.f;
            }
            if (p.splits > 1) {
                // add the partials in split order; this CTA's own values take their place in it
                const int per_owner = (n_groups + p.splits - 1) / p.splits;
                const float* base = reinterpret_cast<const float*>(tiles) +
                                    (static_cast<size_t>(gi / p.splits) * tile_rows + row_local) * 8;
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = 0.f;
                for (int s = 0; s < p.splits; ++s) {
                    if (s == split) {
#pragma unroll
                        for (int j = 0; j < 8; ++j) f[j] += __uint_as_float(v[j]);
                    } else {
                        const int slot = s < split ? s : s - 1;
                        const float4* q = reinterpret_cast<const float4*>(base + static_cast<size_t>(slot) * per_owner * tile_rows * 8);
                        const float4 a = q[0], c = q[1];
                        f[0] += a.x; f[1] += a.y; f[2] += a.z; f[3] += a.w;
                        f[4] += c.x; f[5] += c.y; f[6] += c.z; f[7] += c.w;
                    }
                }
            } else {
#pragma unroll
                for (int j = 0; j < 8; ++j) f[j] = __uint_as_float(v[j]);
            }
            const int col = col_base + gi * 8;
            if (row_ok && col < g.N)          // N is a multiple of 8: a group of 8 columns is inside or outside
                store_group<EPI>(f, u, g.out, g.res, row_off + col);
        }
    }

    // teardown
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}   // let copies in flight land before the shared memory goes away
        if (threadIdx.x == 0) atomicOr(g.dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, p.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------------------------
// CTA-pair variant (cta_group::2), used when the problem has at least two row tiles.  The two CTAs of a cluster
// compute one 256-row x bn-column tile with MMAs of M = 256: each CTA loads its own 128 rows of A and only HALF
// of the W rows of every MMA (the tensor cores exchange the halves), and holds 128 rows x bn columns of the
// accumulator.  Per flop a CTA writes and reads a third less shared memory than a single CTA computing a
// 128-row tile, which is what limits the single-CTA kernel.  bn may exceed 256: the tile is then made of two
// MMAs of bn / 2 columns per K step.  SwiGLU: the even CTA loads the gate rows, the odd CTA the matching up rows,
// so that every accumulator row holds [gate | up] column pairs.
// K split (long K, few output tiles): two pairs form a cluster of four CTAs (ranks 0, 1 = first half of K, ranks 2,
// 3 = second half).  After the main loop each CTA hands the accumulator column groups it does not own to the CTA
// with the same rows in the other pair, through distributed shared memory into that CTA's idle operand ring; both
// add in the same order (first half + second half) and each applies the epilogue to the groups it owns.
struct PairPlan {
    int bn;          // accumulator columns per tile = W rows per tile and K block (both CTAs together)
    int wcols;       // output columns per tile (bn, or bn / 2 for SwiGLU)
    int nmma;        // MMAs per K step (1 or 2), each nchunk columns wide
    int nchunk;
    int splits;      // pairs along K per output tile (1 or 2); two pairs form a cluster of four CTAs
    int resident;    // clusters of this shape the device holds at once
    int stages;
    int m_pairs, n_tiles;
    uint32_t tmem_cols;
};

struct PairArgs {
    int M, N, K, ldo;
    PairPlan p;
    __nv_bfloat16* out;
    const __nv_bfloat16* res;
    uint32_t* dev_status;
};

// 4 x 4 transpose of 16-byte pieces inside every group of four lanes.  In: v[q] = piece q of this lane's row.
// Out: v[i] = piece (lane % 4) of the row of lane (lane & ~3) + i.  Its own inverse.  All lanes take part.
__device__ __forceinline__ void quad_transpose(uint4 (&v)[4], int lane) {
#pragma unroll
    for (int m = 1; m <= 2; m <<= 1) {
        const bool hi = (lane & m) != 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (q & m) continue;
            const uint4 send = hi ? v[q] : v[q ^ m];
            uint4 recv;
            recv.x = __shfl_xor_sync(0xffffffffu, send.x, m);
            recv.y = __shfl_xor_sync(0xffffffffu, send.y, m);
            recv.z = __shfl_xor_sync(0xffffffffu, send.z, m);
            recv.w = __shfl_xor_sync(0xffffffffu, send.w, m);
            if (hi) v[q] = recv; else v[q ^ m] = recv;
        }
    }
}

// Stores 32 consecutive output columns of the 32 rows a warp owns (lane = row, f = this row's values; SwiGLU
// already applied).  The values are rounded to bf16, transposed among each four lanes and written so that one
// store instruction covers 8 rows x 64 contiguous bytes instead of 32 rows x 16 bytes; the residual, if any, is
// read the same way and transposed back before the add.  row0 = the warp's first row; all lanes must call.
template <int EPI>
__device__ __forceinline__ void store_chunk32(float (&f)[32], int lane, int row0, int n_rows_total, int col0, int n_cols_total,
                                              int ldo, __nv_bfloat16* out, const __nv_bfloat16* res) {
    const int my_col = col0 + (lane & 3) * 8;             // after the transpose: this lane's 8 columns ...
    const int my_row0 = row0 + (lane & ~3);               // ... of rows my_row0 + i, i = 0..3
    const bool col_ok = my_col < n_cols_total;            // (columns come in whole groups of 8)
    if (EPI == GEMM_EPI_RESIDUAL) {
        uint4 r[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int row = my_row0 + i;
            r[i] = (col_ok && row < n_rows_total)
                       ? *reinterpret_cast<const uint4*>(res + static_cast<size_t>(row) * ldo + my_col)
                       : make_uint4(0u, 0u, 0u, 0u);
        }
        quad_transpose(r, lane);                           // back to lane = row: r[q] = columns 8q .. 8q+7 of my row
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            f[q * 8 + 0] += bf16_lo(r[q].x); f[q * 8 + 1] += bf16_hi(r[q].x);
            f[q * 8 + 2] += bf16_lo(r[q].y); f[q * 8 + 3] += bf16_hi(r[q].y);
            f[q * 8 + 4] += bf16_lo(r[q].z); f[q * 8 + 5] += bf16_hi(r[q].z);
            f[q * 8 + 6] += bf16_lo(r[q].w); f[q * 8 + 7] += bf16_hi(r[q].w);
        }
    }
    uint4 o[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        o[q].x = pack_bf16(f[q * 8 + 0], f[q * 8 + 1]);
        o[q].y = pack_bf16(f[q * 8 + 2], f[q * 8 + 3]);
        o[q].z = pack_bf16(f[q * 8 + 4], f[q * 8 + 5]);
        o[q].w = pack_bf16(f[q * 8 + 6], f[q * 8 + 7]);
    }
    quad_transpose(o, lane);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = my_row0 + i;
        if (col_ok && row < n_rows_total)
            *reinterpret_cast<uint4*>(out + static_cast<size_t>(row) * ldo + my_col) = o[i];
    }
}

struct PairBarriers {
    uint64_t full[MAX_STAGES];
    uint64_t empty[MAX_STAGES];
    uint64_t tmem_full[2];       // accumulator buffer ready (arrives in both CTAs)
    uint64_t tmem_empty[2];      // accumulator buffer drained by the epilogue warps of both CTAs (even CTA's is used)
    uint32_t tmem_base;
    uint32_t abort_flag;
};
constexpr int PAIR_EPI_WARPS = 8;

// Persistent: cluster c computes tiles c, c + #clusters, ... (row index fastest).  The copies run ahead into the
// next tile, and with bn <= 256 two accumulator buffers alternate, so a tile's epilogue overlaps the next tile's
// main loop.  With a K split every cluster has exactly one tile (the exchange needs the idle ring).
template <int EPI>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                 const __grid_constant__ CUtensorMap tmap_b2, const PairArgs g) {
    const PairPlan& p = g.p;
    const int half_rows = p.nchunk / 2;                      // W rows this CTA holds per MMA
    const int chunk_bytes = half_rows * (GK * 2);
    const int stage_bytes = A_TILE_BYTES + p.nmma * chunk_bytes;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    PairBarriers* bars = reinterpret_cast<PairBarriers*>(tiles + p.stages * stage_bytes);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = warp_index_uniform();
    const int lane = threadIdx.x & 31;
    const int rank4 = static_cast<int>(cluster_cta_rank());
    const int rank = rank4 & 1;                               // 0: issues the MMAs and owns the "full" barriers
    const int split = rank4 >> 1;                             // which part of K this pair computes
    const int cluster_size = 2 * p.splits;
    const int cluster_id = blockIdx.x / cluster_size;
    const int n_clusters = gridDim.x / cluster_size;
    const int total_tiles = p.m_pairs * p.n_tiles;
    const int nk = (g.K + GK - 1) / GK;
    const int kb_begin = static_cast<int>(static_cast<long long>(nk) * split / p.splits);
    const int kb_end = static_cast<int>(static_cast<long long>(nk) * (split + 1) / p.splits);
    const int n_acc = p.bn <= 256 ? 2 : 1;                   // accumulator buffers (256 columns apart)

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->tmem_full[a], 1);
            mbar_init(&bars->tmem_empty[a], 2 * PAIR_EPI_WARPS);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(&bars->tmem_base, p.tmem_cols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    cluster_sync_all();              // every CTA's barriers exist before another CTA signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_a);
            prefetch_tensormap(&tmap_b);
            if (EPI == GEMM_EPI_SWIGLU) prefetch_tensormap(&tmap_b2);
            const CUtensorMap* tmap_w = (EPI == GEMM_EPI_SWIGLU && rank == 1) ? &tmap_b2 : &tmap_b;
            const int w_step = EPI == GEMM_EPI_SWIGLU ? half_rows : p.nchunk;   // rows from one chunk to the next
            const uint32_t full0 = cluster_map_shared(smem_u32(&bars->full[0]), rank4 & ~1);   // the even CTA's barriers
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters) {
                const int m_pair = tile % p.m_pairs, n_tile = tile / p.m_pairs;
                const int w_row0 = EPI == GEMM_EPI_SWIGLU ? n_tile * p.wcols : n_tile * p.bn + rank * half_rows;
                for (int kb = kb_begin; kb < kb_end; ++kb) {
                    if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                    uint8_t* a_dst = tiles + stage * stage_bytes;
                    uint8_t* b_dst = a_dst + A_TILE_BYTES;
                    const uint32_t full = full0 + stage * static_cast<uint32_t>(sizeof(uint64_t));
                    if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], 2 * stage_bytes);   // both CTAs' bytes
                    tma_load_2d_pair(a_dst, &tmap_a, full, kb * GK, m_pair * 2 * GM + rank * GM);
                    for (int c = 0; c < p.nmma; ++c)
                        tma_load_2d_pair(b_dst + c * chunk_bytes, tmap_w, full, kb * GK, w_row0 + c * w_step);
                    if (++stage == p.stages) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1 && rank == 0) {
        // all lanes run the loops, one elected lane issues the MMAs and their commits (which arrive in both CTAs)
        const bool leader = elect_one_sync();
        const uint32_t idesc = umma_idesc_bf16(2 * GM, p.nchunk);
        const uint16_t pair_mask = static_cast<uint16_t>(3u << rank4);     // this CTA (even rank) and the next
        int stage = 0;
        uint32_t phase = 0;
        int it = 0;
        bool ok = true;
        for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters, ++it) {
            const int acc = it % n_acc;
            const uint32_t acc_phase = (it / n_acc) & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, abort_flag));
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t d_tmem = tmem_base + acc * 256;
            for (int kb = kb_begin; kb < kb_end; ++kb) {
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[stage], phase, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a_addr = smem_u32(tiles + stage * stage_bytes);
                const uint64_t a_desc = umma_desc_sw128_kmajor(a_addr);
                const uint32_t accumulate = kb > kb_begin;
                if (leader) {
                    for (int c = 0; c < p.nmma; ++c) {
                        const uint64_t b_desc = umma_desc_sw128_kmajor(a_addr + A_TILE_BYTES + c * chunk_bytes);
#pragma unroll
                        for (int kk = 0; kk < GK / 16; ++kk)   // +32 bytes along K per step = +2 descriptor units
                            umma_bf16_pair(d_tmem + c * p.nchunk, a_desc + 2 * kk, b_desc + 2 * kk, idesc,
                                           accumulate | (kk != 0));
                    }
                    umma_commit_pair(&bars->empty[stage], pair_mask);
                }
                __syncwarp();
                if (++stage == p.stages) { stage = 0; phase ^= 1; }
            }
            if (ok && leader) umma_commit_pair(&bars->tmem_full[acc], pair_mask);
            __syncwarp();
        }
    }
    __syncwarp();      // (the lanes of the producer and MMA warps walk the tile loop below together)

    // ---- epilogue (warps 2..9 of every CTA): warp w may touch TMEM lanes [32 * (w % 4), +32); the two sets of
    // four warps alternate over the column groups of the CTA's 128 rows.  With a K split, 8-column group gi belongs
    // to the pair (gi / 2) % 2; the other pair's CTA with the same rows sends its partial into slot gi of this
    // CTA's idle ring ([group][row][8 floats]).
    const bool epi_warp = warp >= 2;
    const int lq = warp & 3;
    const int set = epi_warp ? (warp - 2) >> 2 : 0;
    const int n_groups = p.wcols / 8;
    const int row_local = lq * 32 + lane;
    int it = 0;
    bool epi_ok = true;
    for (int tile = cluster_id; tile < total_tiles; tile += n_clusters, ++it) {
        const int m_pair = tile % p.m_pairs, n_tile = tile / p.m_pairs;
        const int acc = it % n_acc;
        const uint32_t acc_phase = (it / n_acc) & 1;
        const int row = m_pair * 2 * GM + rank * GM + row_local;
        const bool row_ok = row < g.M;
        const size_t row_off = static_cast<size_t>(row) * g.ldo;
        const int col_base = n_tile * p.wcols;
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lq * 32) << 16) + acc * 256;
        if (epi_warp && epi_ok) {
            epi_ok = mbar_wait(&bars->tmem_full[acc], acc_phase, abort_flag);   // (a wait that gave up leaves the abort flag set)
            tc_fence_after_sync();
        }
        __syncwarp();
        if (p.splits > 1) {              // (one tile per cluster in this case)
            cluster_sync_all();                              // every CTA of the cluster is done with its ring
            if (epi_warp) {
                const uint32_t ring = smem_u32(tiles);
                for (int gi = set; gi < n_groups; gi += 2) {
                    if (((gi >> 1) & 1) == split) continue;  // mine: stays here
                    uint32_t v[8];
                    tmem_ld_8cols(taddr + gi * 8, v);
                    tmem_ld_wait();
                    const uint32_t local = ring + ((static_cast<uint32_t>(gi) * GM + row_local) << 5);
                    const uint32_t remote = cluster_map_shared(local, static_cast<uint32_t>(rank4 ^ 2));
                    st_shared_cluster_v4(remote, v[0], v[1], v[2], v[3]);
                    st_shared_cluster_v4(remote + 16, v[4], v[5], v[6], v[7]);
                }
            }
            cluster_sync_all();                              // the partials of the groups this CTA owns have arrived
        }
        if (!epi_warp) continue;
        const bool live = epi_ok && !*abort_flag;
        // Without a K split the output goes 32 columns at a time through store_chunk32 (coalesced stores); the
        // last n_groups % 4 groups, and the K-split case, go 8 columns at a time with one 16-byte store per lane.
        int g_begin = set;
        if (p.splits == 1) {             // (warp-uniform: store_chunk32 shuffles)
            const int n_chunks = n_groups / 4;
            const int warp_row0 = m_pair * 2 * GM + rank * GM + lq * 32;
            for (int ci = set; ci < n_chunks; ci += 2) {
                float f[32];
                if (EPI == GEMM_EPI_SWIGLU) {
                    uint32_t vg[32], vu[32];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {          // each group of 8 output columns has its gate and up columns
                        const int j = (ci * 4 + q) * 8, c = j / half_rows;
                        const int gcol = c * p.nchunk + (j - c * half_rows);
                        uint32_t a8[8], b8[8];
                        tmem_ld_8cols(taddr + gcol, a8);
                        tmem_ld_8cols(taddr + gcol + half_rows, b8);
#pragma unroll
                        for (int k = 0; k < 8; ++k) { vg[q * 8 + k] = a8[k]; vu[q * 8 + k] = b8[k]; }
                    }
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) {
                        const float gte = __uint_as_float(vg[k]);
                        f[k] = __fdividef(gte, 1.0f + __expf(-gte)) * __uint_as_float(vu[k]);   // silu(g) * u
                    }
                } else {
                    uint32_t v[32];
                    tmem_ld_32cols(taddr + ci * 32, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 32; ++k) f[k] = __uint_as_float(v[k]);
                }
                if (live) store_chunk32<EPI>(f, lane, warp_row0, g.M, col_base + ci * 32, g.N, g.ldo, g.out, g.res);
            }
            g_begin = n_chunks * 4 + set;
        }
        if (live) {
            for (int gi = g_begin; gi < n_groups; gi += 2) {
                if (p.splits > 1 && ((gi >> 1) & 1) != split) continue;
                uint32_t v[8];
                float f[8], u[8];
                if (EPI == GEMM_EPI_SWIGLU) {
                    const int j = gi * 8, c = j / half_rows;
                    const int gcol = c * p.nchunk + (j - c * half_rows);
                    uint32_t w[8];
                    tmem_ld_8cols(taddr + gcol, v);
                    tmem_ld_8cols(taddr + gcol + half_rows, w);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 8; ++k) u[k] = __uint_as_float(w[k]);
                } else {
                    tmem_ld_8cols(taddr + gi * 8, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int k = 0; k < 8; ++k) u[k] = 0.f;
                }
#pragma unroll
                for (int k = 0; k < 8; ++k) f[k] = __uint_as_float(v[k]);
                if (p.splits > 1) {
                    // first half of K + second half of K, in that order in both pairs
                    const float4* q = reinterpret_cast<const float4*>(tiles + ((static_cast<size_t>(gi) * GM + row_local) << 5));
                    const float4 a = q[0], c = q[1];
                    const float o[8] = {a.x, a.y, a.z, a.w, c.x, c.y, c.z, c.w};
#pragma unroll
                    for (int k = 0; k < 8; ++k) f[k] = split == 0 ? f[k] + o[k] : o[k] + f[k];
                }
                const int col = col_base + gi * 8;
                if (row_ok && col < g.N) store_group<EPI>(f, u, g.out, g.res, row_off + col);
            }
        }
        // this warp has read its part of the buffer: tell the even CTA's MMA warp
        tc_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(&bars->tmem_empty[acc], static_cast<uint32_t>(rank4 & ~1));
    }

    // teardown: no CTA may leave while a partner can still signal its barriers or read its tiles
    tc_fence_before_sync();
    cluster_sync_all();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}   // let copies in flight land before the shared memory goes away
        if (threadIdx.x == 0) atomicOr(g.dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, p.tmem_cols);
    }
}

template <int EPI>
int launch_pair(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, const PairArgs& g,
                cudaStream_t stream, int* max_clusters_query) {
    static std::atomic<uint64_t> smem_set{0};
    if (ensure_dynamic_smem(smem_set, gemm_pair_kernel<EPI>, GEMM_SMEM_BYTES) != DARE_OK) return DARE_ERR_CUDA;
    // one cluster per tile with a K split; otherwise as many clusters as the device holds, each walking the tiles
    long long clusters = static_cast<long long>(g.p.m_pairs) * g.p.n_tiles;
    if (g.p.splits == 1 && !max_clusters_query && clusters > g.p.resident) clusters = g.p.resident;
    const long long ctas = 2LL * g.p.splits * clusters;
    if (ctas > 0x7fffffffLL) return DARE_ERR_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas), 1, 1);
    cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = GEMM_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = static_cast<unsigned>(2 * g.p.splits);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (max_clusters_query) {
        cfg.gridDim = dim3(4096u, 1, 1);
        return cudaOccupancyMaxActiveClusters(max_clusters_query, gemm_pair_kernel<EPI>, &cfg) == cudaSuccess
                   ? DARE_OK : DARE_ERR_CUDA;
    }
    note_launch();
    return cudaLaunchKernelEx(&cfg, gemm_pair_kernel<EPI>, ta, tb, tb2, g) == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

// Clusters of `splits` CTA pairs of the pair kernel that can be resident at once (cached; 0 = they cannot run).
int max_active_pairs(int splits = 1) {
    static int cache[3] = {-1, -1, -1};
    if (cache[splits] < 0) {
        PairArgs g{};
        g.p.m_pairs = g.p.n_tiles = 1;
        g.p.splits = splits;
        g.p.resident = 1;
        CUtensorMap dummy{};
        int n = 0;
        if (launch_pair<GEMM_EPI_STORE>(dummy, dummy, dummy, g, nullptr, &n) != DARE_OK) n = 0;
        cache[splits] = n;
    }
    return cache[splits];
}

// Tile shape for the pair kernel.  Per K block a CTA's time is the largest of: its MMA time (nchunk / 2 cycles
// per MMA plus the ~45 measured on top of that), its shared-memory traffic (the stage written by the copies plus, per MMA, 4 KB of
// A and its half of W read by the tensor core) at 128 bytes per cycle, and the operand delivery at ~55 bytes
// per cycle; a launch takes as many rounds as the pairs need on the device.  cost_out: the model's cycles.
PairPlan pair_plan(int epi, int M, int N, int K, double* cost_out) {
    PairPlan best{};
    double best_cost = 1e300;
    const int nk = (K + GK - 1) / GK;
    const int m_pairs = (M + 2 * GM - 1) / (2 * GM);
    const int ring = GEMM_SMEM_BYTES - 1024 - 256;
    for (int splits = 1; splits <= 2; ++splits) {
        if (splits > 1 && (epi == GEMM_EPI_SWIGLU || nk < 32)) break;
        const int resident = max_active_pairs(splits);
        if (resident < 1) continue;
        for (int nmma = 1; nmma <= 2; ++nmma) {
            for (int nchunk = 256; nchunk >= 32; nchunk -= 16) {
                const int bn = nmma * nchunk;
                const int wcols = epi == GEMM_EPI_SWIGLU ? bn / 2 : bn;
                if (wcols > ((N + 7) / 8) * 8 + 15 && bn > 32) continue;      // wider than the whole output
                const int half_rows = nchunk / 2;
                const int stage_bytes = A_TILE_BYTES + nmma * half_rows * GK * 2;
                int stages = ring / stage_bytes;
                if (stages > MAX_STAGES) stages = MAX_STAGES;
                if (stages < 3) continue;
                if (splits > 1 && (wcols / 8) * GM * 32 > stages * stage_bytes) continue;   // partials must fit the ring
                const int n_tiles = (N + wcols - 1) / wcols;
                const long long tiles = static_cast<long long>(m_pairs) * n_tiles;
                const long long rounds = (tiles + resident - 1) / resident;
                const double kb = static_cast<double>((nk + splits - 1) / splits);
                const double mma = nmma * 4 * (nchunk / 2.0 + 45.0);
                const double smem = (stage_bytes + nmma * 4 * (4096.0 + half_rows * 32.0)) / 128.0;
                const double ld = stage_bytes / 55.0;
                double per_kb = mma > smem ? mma : smem;
                if (ld > per_kb) per_kb = ld;
                const double epilogue = wcols * 14.0 / splits + (splits > 1 ? 6000.0 : 0.0);   // two cluster barriers, exchange
                const double cost = rounds * (kb * per_kb + 2500.0 + epilogue);
                if (cost < best_cost) {
                    best_cost = cost;
                    best.bn = bn; best.wcols = wcols; best.nmma = nmma; best.nchunk = nchunk; best.stages = stages;
                    best.splits = splits; best.m_pairs = m_pairs; best.n_tiles = n_tiles;
                    best.resident = resident;
                    best.tmem_cols = 512;       // two buffers of up to 256 columns, or one of up to 512
                }
            }
        }
    }
    if (cost_out) *cost_out = best_cost;
    return best;
}

template <int EPI>
int launch_one(const CUtensorMap& ta, const CUtensorMap& tb, const CUtensorMap& tb2, const GemmArgs& g,
               cudaStream_t stream, int* max_clusters_query) {
    static std::atomic<uint64_t> smem_set{0};
    if (ensure_dynamic_smem(smem_set, gemm_bf16_kernel<EPI>, GEMM_SMEM_BYTES) != DARE_OK) return DARE_ERR_CUDA;
    const long long ctas = static_cast<long long>(g.p.m_items) * g.p.n_tiles * g.p.splits;
    if (ctas > 0x7fffffffLL) return DARE_ERR_SHAPE;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(ctas), 1, 1);
    cfg.blockDim = dim3(GEMM_THREADS, 1, 1);
    cfg.dynamicSmemBytes = GEMM_SMEM_BYTES;
    cfg.stream = stream;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = static_cast<unsigned>(g.p.splits);
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    if (max_clusters_query) {     // how many clusters of this size the device runs at once (plan input)
        cfg.gridDim = dim3(static_cast<unsigned>(g.p.splits) * 1024u, 1, 1);
        return cudaOccupancyMaxActiveClusters(max_clusters_query, gemm_bf16_kernel<EPI>, &cfg) == cudaSuccess
                   ? DARE_OK : DARE_ERR_CUDA;
    }
    note_launch();
    return cudaLaunchKernelEx(&cfg, gemm_bf16_kernel<EPI>, ta, tb, tb2, g) == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

// Clusters of `splits` CTAs of this kernel that can be resident at once (cached; 0 = such clusters cannot run).
int max_active_clusters(int splits) {
    static int cache[MAX_SPLITS + 1] = {-1, -1, -1};
    if (cache[splits] < 0) {
        GemmArgs g{};
        g.p.m_items = g.p.n_tiles = 1;
        g.p.splits = splits;
        CUtensorMap dummy{};
        int n = 0;
        if (launch_one<GEMM_EPI_STORE>(dummy, dummy, dummy, g, nullptr, &n) != DARE_OK) n = 0;
        cache[splits] = n;
    }
    return cache[splits];
}

// Picks the tile shape by a small cost model: a CTA's time is the longer of its MMA issue time (bn / 2 cycles
// per 128 x bn x 16 MMA) and its operand traffic at ~55 bytes per cycle (what L2 delivers per SM when every SM streams), plus prologue and epilogue; the launch
// takes as many rounds of it as the CTAs (or clusters, with a K split) need on the device.
GemmPlan gemm_plan(int epi, int M, int N, int K, int sm_count) {
    const int nk = (K + GK - 1) / GK;
    const int m_tiles = (M + GM - 1) / GM;
    const int ring = GEMM_SMEM_BYTES - 1024 - 256;
    GemmPlan best{};
    double best_cost = 1e300;
    for (int nsub = 1; nsub <= (m_tiles >= 2 ? 2 : 1); ++nsub) {
        const int m_items = (m_tiles + nsub - 1) / nsub;
        for (int bn = 256; bn >= 32; bn -= 16) {
            const int wcols = epi == GEMM_EPI_SWIGLU ? bn / 2 : bn;
            if (wcols > ((N + 7) / 8) * 8 + 15 && bn > 32) continue;          // wider than the whole output
            const int n_tiles = (N + wcols - 1) / wcols;
            const int stage_bytes = nsub * A_TILE_BYTES + bn * GK * 2;
            int stages = ring / stage_bytes;
            if (stages > MAX_STAGES) stages = MAX_STAGES;
            if (stages < 2) continue;
            for (int splits = 1; splits <= MAX_SPLITS; ++splits) {
                const long long tiles = static_cast<long long>(m_items) * n_tiles;
                long long rounds;
                if (splits > 1) {
                    if (epi == GEMM_EPI_SWIGLU || nk < 8 * splits) break;
                    const int per_owner = (wcols / 8 + splits - 1) / splits;
                    if (static_cast<long long>(splits - 1) * per_owner * nsub * GM * 32 > static_cast<long long>(stages) * stage_bytes)
                        continue;                                              // partials must fit the idle ring
                    const int resident = max_active_clusters(splits);
                    if (resident < 1) continue;
                    rounds = (tiles + resident - 1) / resident;
                } else {
                    rounds = (tiles + sm_count - 1) / sm_count;
                }
                const double kb = static_cast<double>((nk + splits - 1) / splits);
                const double mma = kb * nsub * 4 * (bn / 2.0);
                const double ld = kb * stage_bytes / 55.0;
                const double epilogue = wcols * 14.0 + (splits > 1 ? 9000.0 : 0.0);   // two cluster barriers and the exchange
                const double cost = rounds * ((mma > ld ? mma : ld) + 2500.0 + epilogue);
                if (cost < best_cost) {
                    best_cost = cost;
                    best.nsub = nsub; best.bn = bn; best.wcols = wcols; best.splits = splits; best.stages = stages;
                    best.m_items = m_items; best.n_tiles = n_tiles;
                    uint32_t cols = 32;
                    while (cols < static_cast<uint32_t>(nsub == 2 ? 256 + bn : bn)) cols <<= 1;
                    best.tmem_cols = cols;
                }
            }
        }
    }
    return best;
}

}  // namespace

// The pair kernel serves every problem with more than one row tile.
bool use_pair_kernel(int M, const PairPlan& pp) { return M > GM && pp.bn != 0; }

int gemm_plan_describe(const dare_ctx* ctx, int epi, int M, int N, int K, int* out) {
    const PairPlan pp = pair_plan(epi, M, N, K, nullptr);
    if (use_pair_kernel(M, pp)) {
        out[0] = 2; out[1] = pp.bn; out[2] = pp.wcols; out[3] = pp.splits; out[4] = pp.stages;
        out[5] = pp.m_pairs; out[6] = pp.n_tiles; out[7] = max_active_pairs(pp.splits);
        return DARE_OK;
    }
    const GemmPlan p = gemm_plan(epi, M, N, K, ctx->sm_count);
    out[0] = p.nsub; out[1] = p.bn; out[2] = p.wcols; out[3] = p.splits; out[4] = p.stages;
    out[5] = p.m_items; out[6] = p.n_tiles; out[7] = p.splits > 1 ? max_active_clusters(p.splits) : 0;
    return p.bn ? DARE_OK : DARE_ERR_SHAPE;
}

int launch_gemm(const dare_ctx* ctx, int epi, const void* a, int M, int K, const void* w, const void* w2, int N,
                void* out, const void* res, int ldo, cudaStream_t stream) {
    if (M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8) || (ldo % 8)) return DARE_ERR_SHAPE;
    if (epi < GEMM_EPI_STORE || epi > GEMM_EPI_SWIGLU) return DARE_ERR_RANGE;
    const PairPlan pp = pair_plan(epi, M, N, K, nullptr);
    if (use_pair_kernel(M, pp)) {
        PairArgs pg;
        pg.M = M; pg.N = N; pg.K = K; pg.ldo = ldo;
        pg.p = pp;
        pg.out = static_cast<__nv_bfloat16*>(out);
        pg.res = static_cast<const __nv_bfloat16*>(res);
        pg.dev_status = ctx->dev_status;
        CUtensorMap pa, pb, pb2;
        int prc = make_tmap_bf16_2d(ctx, &pa, a, static_cast<uint64_t>(M), static_cast<uint64_t>(K), GM, GK);
        if (prc != DARE_OK) return prc;
        const uint32_t half_rows = static_cast<uint32_t>(pp.nchunk / 2);
        prc = make_tmap_bf16_2d(ctx, &pb, w, static_cast<uint64_t>(N), static_cast<uint64_t>(K), half_rows, GK);
        if (prc != DARE_OK) return prc;
        if (epi == GEMM_EPI_SWIGLU) {
            prc = make_tmap_bf16_2d(ctx, &pb2, w2, static_cast<uint64_t>(N), static_cast<uint64_t>(K), half_rows, GK);
            if (prc != DARE_OK) return prc;
            return launch_pair<GEMM_EPI_SWIGLU>(pa, pb, pb2, pg, stream, nullptr);
        }
        return epi == GEMM_EPI_STORE ? launch_pair<GEMM_EPI_STORE>(pa, pb, pb, pg, stream, nullptr)
                                     : launch_pair<GEMM_EPI_RESIDUAL>(pa, pb, pb, pg, stream, nullptr);
    }
    GemmArgs g;
    g.M = M; g.N = N; g.K = K; g.ldo = ldo;
    g.p = gemm_plan(epi, M, N, K, ctx->sm_count);
    if (g.p.bn == 0) return DARE_ERR_SHAPE;
    g.out = static_cast<__nv_bfloat16*>(out);
    g.res = static_cast<const __nv_bfloat16*>(res);
    g.dev_status = ctx->dev_status;
    CUtensorMap ta, tb, tb2;
    int rc = make_tmap_bf16_2d(ctx, &ta, a, static_cast<uint64_t>(M), static_cast<uint64_t>(K), GM, GK);
    if (rc != DARE_OK) return rc;
    const uint32_t box_rows = static_cast<uint32_t>(epi == GEMM_EPI_SWIGLU ? g.p.wcols : g.p.bn);
    rc = make_tmap_bf16_2d(ctx, &tb, w, static_cast<uint64_t>(N), static_cast<uint64_t>(K), box_rows, GK);
    if (rc != DARE_OK) return rc;
    if (epi == GEMM_EPI_SWIGLU) {
        rc = make_tmap_bf16_2d(ctx, &tb2, w2, static_cast<uint64_t>(N), static_cast<uint64_t>(K), box_rows, GK);
        if (rc != DARE_OK) return rc;
        return launch_one<GEMM_EPI_SWIGLU>(ta, tb, tb2, g, stream, nullptr);
    }
    return epi == GEMM_EPI_STORE ? launch_one<GEMM_EPI_STORE>(ta, tb, tb, g, stream, nullptr)
                                 : launch_one<GEMM_EPI_RESIDUAL>(ta, tb, tb, g, stream, nullptr);
}

}  // namespace dare
