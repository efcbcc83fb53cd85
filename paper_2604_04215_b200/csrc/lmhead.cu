// Fused LM head + vocabulary softmax: per row the argmax token and its probability, logits kept on chip.
//
// z = X W^T is a dense bf16 contraction (M x V x D), so it runs on the tcgen05 tensor cores:
//   warp 0      TMA producer: X tile [128 x 64] and W tile [256 x 64] per pipeline stage (128-byte swizzle)
//   warp 1      UMMA issuer: 128 x 256 x 16 MMAs into one of two 128 x 256 fp32 accumulators in TMEM
//   warps 2..5  epilogue: each thread owns one row (one TMEM lane), streams the 256 logits of the tile
//               through registers and keeps (running max, sum of exp, argmax); no cross-thread traffic
// The two accumulators let the epilogue of tile i overlap the MMAs of tile i+1.
// A second instantiation runs the same roles on CTA pairs (cta_group::2, MMAs of 256 rows, half a W tile per CTA);
// see lm_pair_mode below for when it is the one that works.
//
// Only rows that are still masked need logits.  A first small kernel compacts those rows of X into a dense
// buffer (and answers the committed rows directly); the GEMM reads the number of live rows from device
// memory, so the host never synchronises.  Work is cut into items (row tile, vocabulary group): a CTA keeps
// one row tile for all vocabulary tiles of its group, so every epilogue thread carries its row's running
// triple in registers across tiles and writes ONE partial per item.  The CTAs of the row tiles of one group
// walk the same W tiles at the same time, so W leaves HBM once.  A last small kernel merges the (few)
// partials of a row into (token, confidence) and scatters them to the row's original position.
#include <math.h>
#include <mutex>
#include <type_traits>

#include "internal.h"
#include "ptx.cuh"

namespace dare {
namespace {

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES = BN * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int LM_THREADS = 192;
// The sampling epilogue does several times the arithmetic of the greedy one per logit (a generator block and two
// logarithms): it gets two sets of four epilogue warps that take alternate 32-column chunks of every tile.
constexpr int LM_SAMPLE_THREADS = 320;
__host__ __device__ constexpr int lm_threads(int mode) { return mode == 1 ? LM_SAMPLE_THREADS : LM_THREADS; }
constexpr uint32_t TMEM_COLS = 512;
constexpr float LOG2E = 1.4426950408889634f;
constexpr int ARG_NONE = 0x7fffffff;

struct LmBarriers {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t exch_full, exch_empty;      // two epilogue sets: hand-over of the second set's running values
    uint32_t tmem_base;
    uint32_t abort_flag;
};
constexpr int LM_SMEM_BYTES = STAGES * STAGE_BYTES + static_cast<int>(sizeof(LmBarriers)) + 1024;
// CTA-pair mode (cta_group::2): two CTAs of a cluster take two row tiles against the same W tiles with MMAs of
// M = 256; each CTA loads its own X tile and only half of the W tile, which takes a third off the shared-memory
// traffic per flop that limits the single-CTA mode (tensor pipe 83 % -> 93 % busy in the projections).
constexpr int PSTAGES = 6;
constexpr int PB_BYTES = (BN / 2) * BK * 2;
constexpr int PSTAGE_BYTES = A_BYTES + PB_BYTES;
struct LmPairBarriers {
    uint64_t full[PSTAGES];
    uint64_t empty[PSTAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t exch_full, exch_empty;
    uint32_t tmem_base;
    uint32_t abort_flag;
};
constexpr int LM_PAIR_SMEM_BYTES = PSTAGES * PSTAGE_BYTES + static_cast<int>(sizeof(LmPairBarriers)) + 1024;

// Number of vocabulary groups for a grid of `grid` CTAs and `m_tiles` row tiles (same formula on the host,
// in the GEMM and in the merge kernel).
__host__ __device__ inline int lm_groups(int grid, int m_tiles, int n_tiles) {
    int g = m_tiles > 0 ? grid / m_tiles : 1;
    if (g < 1) g = 1;
    if (g > n_tiles) g = n_tiles;
    return g;
}

// Pairs pay when the row tiles come in twos (an odd tile would drag an empty partner along: measured at 3584 x
// 152064, five tiles take 544 us on single CTAs and 600 to 660 us on pairs with the sixth tile empty).  The row
// count is only known on the device, so both kernels are launched and the one whose mode does not apply returns
// at once.
__host__ __device__ inline bool lm_pair_mode(int m_tiles, int allow_pair) {
    return allow_pair && m_tiles >= 2 && (m_tiles & 1) == 0;
}
// Vocabulary groups in the mode that applies: pairs count as one CTA and two row tiles as one.
__host__ __device__ inline int lm_groups_mode(int grid, int m_tiles, int n_tiles, int allow_pair) {
    return lm_pair_mode(m_tiles, allow_pair) ? lm_groups(grid / 2, (m_tiles + 1) / 2, n_tiles) : lm_groups(grid, m_tiles, n_tiles);
}

__device__ __forceinline__ int32_t row_token(const int32_t* row_tokens, int tok_L, int64_t tok_row_stride, int m) {
    return row_tokens[static_cast<int64_t>(m / tok_L) * tok_row_stride + m % tok_L];
}

// Compacts the still-masked rows of X into xc (order preserved), records their original indices, counts
// them, and answers committed rows (pred = their token, conf = -inf).  One warp per row.
constexpr int CP_ROWS = 8;
__global__ void __launch_bounds__(CP_ROWS * 32)
lmhead_compact_kernel(const uint4* __restrict__ x, int M, int D8, const int32_t* __restrict__ row_tokens, int tok_L,
                      int64_t tok_row_stride, int32_t mask_id, uint4* __restrict__ xc, int32_t* __restrict__ idx,
                      int32_t* __restrict__ count, int32_t* __restrict__ pred, float* __restrict__ conf) {
    __shared__ int s_base;
    __shared__ int s_flag[CP_ROWS];
    const int row0 = blockIdx.x * CP_ROWS;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) s_base = 0;
    __syncthreads();
    int local = 0;
    for (int m = threadIdx.x; m < row0; m += blockDim.x) local += row_token(row_tokens, tok_L, tok_row_stride, m) == mask_id;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
    if (lane == 0 && local) atomicAdd(&s_base, local);
    const int row = row0 + warp;
    int32_t tok = 0;
    bool masked = false;
    if (row < M) {
        tok = row_token(row_tokens, tok_L, tok_row_stride, row);
        masked = tok == mask_id;
    }
    if (lane == 0) s_flag[warp] = masked ? 1 : 0;
    __syncthreads();
    int before = s_base, total = s_base;
    for (int i = 0; i < CP_ROWS; ++i) {
        if (i < warp) before += s_flag[i];
        total += s_flag[i];
    }
    if (blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) *count = total;
    if (row >= M) return;
    if (!masked) {
        if (lane == 0) { pred[row] = tok; conf[row] = -INFINITY; }
        return;
    }
    if (lane == 0) idx[before] = row;
    const uint4* src = x + static_cast<size_t>(row) * D8;
    uint4* dst = xc + static_cast<size_t>(before) * D8;
    // eight loads in flight per lane before the first store: the copy of a row is a chain of latencies otherwise
    int i = lane;
    for (; i + 7 * 32 < D8; i += 8 * 32) {
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = src[i + u * 32];
#pragma unroll
        for (int u = 0; u < 8; ++u) dst[i + u * 32] = v[u];
    }
    for (; i < D8; i += 32) dst[i] = src[i];
}

// Sampling epilogue (temperature + Gumbel-max): token = argmax_v (z_v / T + g_v), g_v = -ln(-ln u_v), with u_v from
// the counter-based generator Philox4x32-10 (Salmon et al., SC 2011) keyed by the seed, counter = (v / 4, row,
// step, tag); element v takes output word v % 4, whose top 23 bits k give u = (2 k + 1) / 2^24 (exact in fp32).
struct LmSampling {
    float inv_temperature;
    uint32_t seed_lo, seed_hi, step;
    const uint32_t* step_dev;      // optional device word added to `step`
    const int32_t* row_index;      // original row of compacted row c (NULL: identity): keys the generator
    const int32_t* targets;        // LM_LOGPROB: target token per row
    float* part_y;                 // per partial: best perturbed score and the raw logit there
    float* part_zb;
    // LM_GRAD: per-row logsumexp of the forward pass and upstream gradient; outputs dz [M, V] and its transpose
    // [V, ldm] (bf16)
    const float* lse;
    const float* grad;
    __nv_bfloat16* dz;
    __nv_bfloat16* dzt;
    int ldm;
};

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
__device__ __forceinline__ float gumbel_from_word(uint32_t w) {
    const float u = static_cast<float>(((w >> 9) << 1) | 1u) * 5.9604644775390625e-08f;   // (2 k + 1) / 2^24, exact
    return -logf(-logf(u));
}

// MODE 0: greedy (argmax token, its probability); 1: sampling epilogue; 2: log-probability of a given target
// token per row (the partial's third slot then carries the target's logit instead of an argmax).
// MODE 3: gradient of the log-probability with respect to the logits, g * (onehot(target) - softmax), written as
// bf16 in both orientations (the two products of the backward pass take it from there); no partials.
constexpr int LM_GREEDY = 0, LM_SAMPLE = 1, LM_LOGPROB = 2, LM_GRAD = 3;

// The work of one launch, or of the part of a launch that runs this body: `n_units` units (CTAs, or CTA pairs with
// PAIR), of which this CTA belongs to unit `unit`, walk the row tiles [tile0, tile0 + m_tiles) against all
// vocabulary tiles; a row's partials start at row * parts_stride (parts_stride < 0: at row * groups, the packed
// layout of the stand-alone kernels).  W_HALF_BOX: the W tensor map's box is 128 rows (half a tile), so a single
// CTA fetches its 256-row tile as two boxes.
struct LmUnits { int unit, n_units, tile0, m_tiles, parts_stride; };
template <int MODE, bool PAIR, bool W_HALF_BOX = false>
__device__ __forceinline__ void
lm_rowmajor_body(const CUtensorMap& tmap_x, const CUtensorMap& tmap_w,
                 int Mc, int D, int V, int mask_col, int n_tiles,
                 float* __restrict__ part_max, float* __restrict__ part_sum, int32_t* __restrict__ part_arg,
                 uint32_t* __restrict__ dev_status, const LmSampling& smp, const LmUnits u) {
    constexpr int NSTAGES = PAIR ? PSTAGES : STAGES;
    constexpr int STAGE_SZ = PAIR ? PSTAGE_BYTES : STAGE_BYTES;
    using Barriers = typename std::conditional<PAIR, LmPairBarriers, LmBarriers>::type;
    constexpr bool SAMPLE = MODE == LM_SAMPLE;
    constexpr bool LOGPROB = MODE == LM_LOGPROB;
    constexpr bool GRAD = MODE == LM_GRAD;
    constexpr int EPI_SETS = SAMPLE ? 2 : 1;                 // sets of four epilogue warps
    __shared__ float s_exch[5][BM];                          // (max, sum, best y, its logit, its column) per row
    if (u.m_tiles <= 0) return;
    // PAIR: a work unit is a cluster of two CTAs, an item two row tiles (one per CTA) and a vocabulary group
    const int rank = PAIR ? static_cast<int>(cluster_cta_rank()) : 0;
    const int unit = u.unit;
    const int n_units = u.n_units;
    const int item_rows = PAIR ? (u.m_tiles + 1) >> 1 : u.m_tiles;   // row tiles (pairs of them) to walk
    const int groups = lm_groups(n_units, item_rows, n_tiles);
    const int n_items = item_rows * groups;
    if (unit >= n_items) return;                                    // (both CTAs of a pair alike)
    const int parts_stride = u.parts_stride < 0 ? groups : u.parts_stride;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    Barriers* bars = reinterpret_cast<Barriers*>(tiles + NSTAGES * STAGE_SZ);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = warp_index_uniform();
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < NSTAGES; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->tmem_full[a], 1);
            // every epilogue thread arrives (PAIR: one arrival per epilogue warp of both CTAs)
            mbar_init(&bars->tmem_empty[a], (PAIR ? 8 : 128) * EPI_SETS);
        }
        mbar_init(&bars->exch_full, 128);
        mbar_init(&bars->exch_empty, 128);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(&bars->tmem_base, TMEM_COLS); tmem_relinquish_pair(); }
        else { tmem_alloc(&bars->tmem_base, TMEM_COLS); tmem_relinquish(); }
    }
    tc_fence_before_sync();
    if (PAIR) cluster_sync_all();     // both CTAs' barriers exist before either signals the other's
    else __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const int num_k = (D + BK - 1) / BK;

    // item w -> row tile w % m_tiles, vocabulary group w / m_tiles; the group's tiles are g, g + groups, ...
    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_x);
            prefetch_tensormap(&tmap_w);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            // PAIR: the even CTA's "full" barriers count the bytes of both CTAs' copies
            const uint32_t full0 = PAIR ? cluster_map_shared(smem_u32(&bars->full[0]), 0) : 0u;
            for (int item = unit; item < n_items && ok; item += n_units) {
                const int m_tile = u.tile0 + (PAIR ? 2 * (item % item_rows) + rank : item % item_rows);
                for (int n_tile = item / item_rows; n_tile < n_tiles && ok; n_tile += groups) {
                    for (int kb = 0; kb < num_k; ++kb) {
                        if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                        uint8_t* a_dst = tiles + stage * STAGE_SZ;
                        uint8_t* b_dst = a_dst + A_BYTES;
                        if (PAIR) {
                            const uint32_t full = full0 + stage * static_cast<uint32_t>(sizeof(uint64_t));
                            if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], 2 * STAGE_SZ);
                            tma_load_2d_pair(a_dst, &tmap_x, full, kb * BK, m_tile * BM);
                            tma_load_2d_pair(b_dst, &tmap_w, full, kb * BK, n_tile * BN + rank * (BN / 2));
                        } else {
                            mbar_arrive_expect_tx(&bars->full[stage], STAGE_SZ);
                            tma_load_2d(a_dst, &tmap_x, &bars->full[stage], kb * BK, m_tile * BM);
                            tma_load_2d(b_dst, &tmap_w, &bars->full[stage], kb * BK, n_tile * BN);
                            if (W_HALF_BOX)
                                tma_load_2d(b_dst + (BN / 2) * BK * 2, &tmap_w, &bars->full[stage], kb * BK, n_tile * BN + BN / 2);
                        }
                        if (++stage == NSTAGES) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1 && rank == 0) {
        // all lanes run the loops, one elected lane issues the MMAs and their commits (PAIR: the even CTA issues
        // for both, and the commits arrive on both CTAs' barriers)
        const bool leader = elect_one_sync();
        constexpr uint32_t idesc = umma_idesc_bf16(PAIR ? 2 * BM : BM, BN);
        int stage = 0;
        uint32_t phase = 0;
        int it = 0;
        bool ok = true;
        for (int item = unit; item < n_items && ok; item += n_units) {
            for (int n_tile = item / item_rows; n_tile < n_tiles && ok; n_tile += groups, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * BN;
                for (int kb = 0; kb < num_k; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[stage], phase, abort_flag));
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_u32(tiles + stage * STAGE_SZ);
                    const uint64_t a_desc = umma_desc_sw128_kmajor(a_addr);
                    const uint64_t b_desc = umma_desc_sw128_kmajor(a_addr + A_BYTES);
                    if (leader) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk) {
                            // 16 bf16 = 32 bytes further along K inside the 128-byte swizzled row: +2 in the
                            // descriptor's 16-byte address units
                            if (PAIR) umma_bf16_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
                            else umma_bf16(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
                        }
                        // frees the stage when these MMAs have read it
                        if (PAIR) umma_commit_pair(&bars->empty[stage], 3);
                        else umma_commit(&bars->empty[stage]);
                    }
                    __syncwarp();
                    if (++stage == NSTAGES) { stage = 0; phase ^= 1; }
                }
                if (ok && leader) {
                    if (PAIR) umma_commit_pair(&bars->tmem_full[acc], 3);
                    else umma_commit(&bars->tmem_full[acc]);
                }
                __syncwarp();
            }
        }
    } else if (warp >= 2) {
        // epilogue: warp w may touch TMEM lanes [32 * (w % 4), +32)
        const int lq = warp & 3;
        const int set = (warp - 2) >> 2;
        const int row_in_tile = lq * 32 + lane;
        int it = 0;
        int items_done = 0;
        bool ok = true;
        for (int item = unit; item < n_items && ok; item += n_units, ++items_done) {
            const int m_tile = u.tile0 + (PAIR ? 2 * (item % item_rows) + rank : item % item_rows);
            const int group = item / item_rows;
            float run_max = -INFINITY;
            float run_sum = 0.f;
            int run_arg = ARG_NONE;
            float best_y = -INFINITY, best_z = -INFINITY;       // SAMPLE: best perturbed score, raw logit there
            uint32_t rng_row = 0, rng_step = 0;
            if (SAMPLE) {
                rng_step = smp.step + (smp.step_dev ? *smp.step_dev : 0u);
                const int row_c = m_tile * BM + row_in_tile;
                rng_row = static_cast<uint32_t>(row_c < Mc && smp.row_index ? smp.row_index[row_c] : row_c);
            }
            int target = -1;                                     // LOGPROB: this row's target column, its logit
            float target_z = -INFINITY;
            if (LOGPROB) {
                const int row_c = m_tile * BM + row_in_tile;
                if (row_c < Mc) target = smp.targets[row_c];
            }
            float g_row = 0.f, lse2 = 0.f;                       // GRAD: upstream gradient, logsumexp * log2(e)
            const int row_g = m_tile * BM + row_in_tile;
            if (GRAD && row_g < Mc) {
                target = smp.targets[row_g];
                // a target outside the vocabulary or in the excluded column has log-probability -inf: no gradient
                if (target >= 0 && target < V && target != mask_col) g_row = smp.grad[row_g];
                lse2 = smp.lse[row_g] * LOG2E;
            }
            for (int n_tile = group; n_tile < n_tiles && ok; n_tile += groups, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                ok = mbar_wait(&bars->tmem_full[acc], acc_phase, abort_flag);
                if (PAIR) ok = __all_sync(0xffffffffu, ok);      // the warp arrives as one further down
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lq * 32) << 16) + acc * BN;
                const int col0 = n_tile * BN;
                const bool edge = (col0 + BN > V) || (mask_col >= col0 && mask_col < col0 + BN);
#pragma unroll 1
                for (int c = set; c < BN / 32; c += EPI_SETS) {
                    uint32_t v[32];
                    tmem_ld_32cols(taddr + c * 32, v);
                    tmem_ld_wait();
                    const int cbase = col0 + c * 32;
                    if (GRAD) {
                        // dz = g * (1[col = target] - exp(z - lse)); 0 beyond the vocabulary and in the excluded column
                        if (row_g < Mc) {
                            uint32_t packed[16];
#pragma unroll
                            for (int j = 0; j < 32; j += 2) {
                                float d2[2];
#pragma unroll
                                for (int e = 0; e < 2; ++e) {
                                    const int col = cbase + j + e;
                                    const float pr = fast_exp2(fmaf(__uint_as_float(v[j + e]), LOG2E, -lse2));
                                    float d = g_row * ((col == target ? 1.0f : 0.0f) - pr);
                                    if (col >= V || col == mask_col) d = 0.f;
                                    d2[e] = d;
                                }
                                packed[j >> 1] = pack_bf16(d2[0], d2[1]);
                            }
                            __nv_bfloat16* dz_row = smp.dz + static_cast<size_t>(row_g) * V + cbase;
#pragma unroll
                            for (int q = 0; q < 4; ++q)       // V is a multiple of 8: a group of 8 columns is inside or outside
                                if (cbase + q * 8 < V)
                                    *reinterpret_cast<uint4*>(dz_row + q * 8) =
                                        make_uint4(packed[q * 4], packed[q * 4 + 1], packed[q * 4 + 2], packed[q * 4 + 3]);
                            // transposed copy: the lanes of a warp are consecutive rows, so each column is one 64-byte run
                            unsigned short* dzt_col = reinterpret_cast<unsigned short*>(smp.dzt) +
                                                      static_cast<size_t>(cbase) * smp.ldm + row_g;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (cbase + j < V)
                                    dzt_col[static_cast<size_t>(j) * smp.ldm] =
                                        static_cast<unsigned short>(j & 1 ? packed[j >> 1] >> 16 : packed[j >> 1] & 0xffffu);
                        }
                        continue;
                    }
                    float cmax = -INFINITY;
                    int carg = ARG_NONE;
                    if (edge) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const int col = cbase + j;
                            if (col >= V || col == mask_col) v[j] = __float_as_uint(-INFINITY);
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float z = __uint_as_float(v[j]);
                        if (z > cmax) { cmax = z; carg = cbase + j; }   // strict '>' keeps the lowest index
                    }
                    if (LOGPROB && target >= cbase && target < cbase + 32) {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (cbase + j == target) target_z = __uint_as_float(v[j]);   // (-inf if it is the excluded column)
                    }
                    if (SAMPLE) {
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const uint4 w4 = philox4x32_10(make_uint4(static_cast<uint32_t>(cbase >> 2) + q, rng_row, rng_step,
                                                                      0x44415245u), smp.seed_lo, smp.seed_hi);
                            const uint32_t ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float z = __uint_as_float(v[q * 4 + e]);
                                const float y = fmaf(z, smp.inv_temperature, gumbel_from_word(ww[e]));
                                if (y > best_y) { best_y = y; best_z = z; run_arg = cbase + q * 4 + e; }   // ascending columns
                            }
                        }
                    }
                    if (cmax > -INFINITY) {
                        if (cmax > run_max) {   // tiles of a group come in ascending order: '>' keeps the lowest id
                            run_sum *= fast_exp2((run_max - cmax) * LOG2E);   // exp2(-inf) = 0 the first time
                            run_max = cmax;
                            if (MODE == LM_GREEDY) run_arg = carg;
                        }
                        const float mb = run_max * LOG2E;
                        float s = 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) s += fast_exp2(fmaf(__uint_as_float(v[j]), LOG2E, -mb));
                        run_sum += s;
                    }
                }
                tc_fence_before_sync();
                if (PAIR) {           // one arrival per warp, on the even CTA's barrier
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(&bars->tmem_empty[acc], 0);
                } else {
                    mbar_arrive(&bars->tmem_empty[acc]);
                }
            }
            if (EPI_SETS == 2 && ok) {
                // the second set hands its running values to the first, which folds them into its own: the larger
                // perturbed score wins, the lower column on a tie (each set saw its columns in ascending order)
                const uint32_t par = items_done & 1;
                if (set == 1) {
                    ok = mbar_wait(&bars->exch_empty, par ^ 1, abort_flag);
                    s_exch[0][row_in_tile] = run_max; s_exch[1][row_in_tile] = run_sum;
                    s_exch[2][row_in_tile] = best_y; s_exch[3][row_in_tile] = best_z;
                    s_exch[4][row_in_tile] = __int_as_float(run_arg);
                    mbar_arrive(&bars->exch_full);          // (release: the values above are visible to the waiter)
                } else {
                    ok = mbar_wait(&bars->exch_full, par, abort_flag);
                    if (ok) {
                        const float m2 = s_exch[0][row_in_tile], s2 = s_exch[1][row_in_tile];
                        const float y2 = s_exch[2][row_in_tile], z2 = s_exch[3][row_in_tile];
                        const int a2 = __float_as_int(s_exch[4][row_in_tile]);
                        mbar_arrive(&bars->exch_empty);
                        if (m2 > -INFINITY) {
                            if (m2 > run_max) { run_sum = run_sum * fast_exp2((run_max - m2) * LOG2E) + s2; run_max = m2; }
                            else run_sum += s2 * fast_exp2((m2 - run_max) * LOG2E);
                        }
                        if (y2 > best_y || (y2 == best_y && a2 < run_arg)) { best_y = y2; best_z = z2; run_arg = a2; }
                    }
                }
            }
            const int row = m_tile * BM + row_in_tile;
            if (!GRAD && ok && row < Mc && set == 0) {
                const size_t o = static_cast<size_t>(row) * parts_stride + group;
                part_max[o] = run_max;
                part_sum[o] = run_sum;
                part_arg[o] = LOGPROB ? __float_as_int(target_z) : run_arg;
                if (SAMPLE) { smp.part_y[o] = best_y; smp.part_zb[o] = best_z; }
            }
        }
    }

    // teardown (PAIR: neither CTA leaves while its partner can still signal its barriers or read its tiles)
    tc_fence_before_sync();
    if (PAIR) cluster_sync_all();
    else __syncthreads();
    if (*abort_flag) {
        // give copies still in flight time to land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
        if (threadIdx.x == 0) atomicOr(dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        if (PAIR) tmem_dealloc_pair(tmem_base, TMEM_COLS);
        else tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

template <int MODE, bool PAIR>
__global__ void __launch_bounds__(lm_threads(MODE), 1)
lmhead_partial_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                      int M, const int32_t* __restrict__ live_rows, int D, int V, int mask_col, int n_tiles,
                      float* __restrict__ part_max, float* __restrict__ part_sum, int32_t* __restrict__ part_arg,
                      uint32_t* __restrict__ dev_status, const LmSampling smp, int allow_pair) {
    const int Mc = live_rows ? *live_rows : M;          // rows that need logits (uniform over the grid)
    const int m_tiles = (Mc + BM - 1) / BM;
    if (lm_pair_mode(m_tiles, allow_pair) != PAIR) return;        // the other kernel does this launch's work
    const LmUnits u = {static_cast<int>(PAIR ? blockIdx.x >> 1 : blockIdx.x),
                       static_cast<int>(PAIR ? gridDim.x >> 1 : gridDim.x), 0, m_tiles, -1};
    lm_rowmajor_body<MODE, PAIR>(tmap_x, tmap_w, Mc, D, V, mask_col, n_tiles, part_max, part_sum, part_arg, dev_status,
                                 smp, u);
}

// ---------------------------------------------------------------------------------------------------------
// Greedy head with the operands swapped: the VOCABULARY sits on the accumulator's lanes (W is the MMA's A operand,
// 128 rows per CTA, 256 per CTA pair) and the live ROWS are its columns (the compacted X is the B operand,
// N = the number of rows, any multiple of 16 up to 256).  What that buys over the row-major kernel above:
//   * no padding to 128-row tiles: a step with 96 masked rows issues MMAs of N = 96, not of 128 padded rows;
//   * every work item is a CTA pair whatever the row count, and the 128-row vocabulary tiles per CTA spread evenly
//     over the SMs: with few rows left the W stream is the bound and the kernel reads it at the copy bandwidth.
// More rows than SW_NMAX are cut into equal chunks (items = chunk x vocabulary group); lm_greedy_swapped says for
// which counts that beats the row-major tiles.  An MMA alone takes max(N / 2, ~45) cycles whether M is 64 or 128 and
// wherever A sits (timed in isolation), but here every MMA takes a fresh 128 x 16 slab of W as its A operand, so a
// chunk streams all of W from L2 into the SMs whatever its N: two chunks of N = 144 cost nearly what two chunks of
// N = 256 cost (319 us for 288 rows, 350 us for 512), and only chunks close to 256 rows are worth it.
// The price is the epilogue: a thread's TMEM lane is now a vocabulary entry and the softmax runs ACROSS lanes.
// Each epilogue warp turns its 32 x 32 block of logits through shared memory (padded rows, conflict-free) so that
// a thread again holds 32 consecutive vocabulary entries of ONE row, and keeps that row's running
// (max, sum, argmax) in registers across the group's tiles: 8 column blocks x 3 values per thread.  At the end of
// an item the four epilogue warps fold their values through the same shared memory, and one partial per (row,
// vocabulary group, CTA of the pair) goes to the merge kernel.
constexpr int SW_BV = 128;                               // vocabulary rows per CTA and tile
constexpr int SW_NMAX = 256;                             // rows (accumulator columns) per chunk
// Row counts for which the greedy head takes this path: up to one chunk, where W is streamed once and the launch is
// bound by HBM; and, up to 1024 rows, counts that cut into chunks of 208 to 240 rows, i.e. whose row-major tiles
// would carry 64 or more padded rows per pair (measured in one process, us, swapped against row-major: D = 4096,
// V = 126464: 416 rows 333 / 380, 448 rows 415 / 462, 480 rows 410 / 428, 512 rows 425 / 421; D = 3584, V = 152064:
// 704 rows 625 / 650, 832 rows 784 / 840, 960 rows 851 / 895).  With shorter chunks the path loses (288 to 384 rows:
// 339 to 372 against 329 to 343): every MMA of this path takes a fresh 128 x 16 slab of W as its A operand, so a
// chunk streams all of W from L2 into the SMs whatever its N, and at N = 144 to 192 that stream (~12 TB/s over the
// GPU), not the tensor pipe, sets the pace.
__host__ __device__ inline bool lm_greedy_swapped(int rows) {
    if (rows <= SW_NMAX) return true;
    if (rows > 1024) return false;
    const int n_chunks = (rows + SW_NMAX - 1) / SW_NMAX;
    const int nc = ((rows + n_chunks - 1) / n_chunks + 15) & ~15;      // as in sw_plan below
    return nc >= 208 && nc < SW_NMAX;
}
constexpr int SW_STAGES = 6;                             // ring slots when a CTA's X tile has its full 128 rows
constexpr int SW_MAX_STAGES = 11;                        // ... and when it is small: the ring's bytes are cut into more slots
constexpr int SW_W_BYTES = SW_BV * BK * 2;               // 16 KB
constexpr int SW_X_BYTES = (SW_NMAX / 2) * BK * 2;       // each CTA loads half of the chunk's rows: up to 16 KB
constexpr int SW_STAGE_BYTES = SW_W_BYTES + SW_X_BYTES;
constexpr int SW_XP_FLOATS = 32 * 33;                    // per epilogue warp: one 32 x 32 block, rows padded to 33
constexpr int SW_PARTS_PER_GROUP = 2;                    // one per CTA of the pair
struct SwBarriers {
    uint64_t full[SW_MAX_STAGES];
    uint64_t empty[SW_MAX_STAGES];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint64_t fold_full, fold_empty;                      // the epilogue warps' exchange at the end of an item
    uint32_t tmem_base;
    uint32_t abort_flag;
};
constexpr int SW_SMEM_BYTES = SW_STAGES * SW_STAGE_BYTES + 4 * SW_XP_FLOATS * 4 + static_cast<int>(sizeof(SwBarriers)) + 1024;
// X tiles of 128, 64, 32, 16 and 8 rows: a CTA's share of a chunk (a multiple of 8 rows) is covered by one or two
// of them, stacked in shared memory (each a whole number of 1 KB swizzle atoms); a few rows too many may be loaded,
// the MMA reads only its own.  (Exact covers of up to four boxes were measured slower: 432 us for 480 rows, where
// each CTA loaded 64 + 32 + 16 + 8 rows per stage, against 350 us for 512 rows with one box.)
struct SwXMaps { CUtensorMap m[5]; };
struct SwBoxes { int i1, i2, rows; };      // indices into SwXMaps::m (i2 < 0: one box), rows loaded in all
__device__ __forceinline__ SwBoxes sw_boxes(int rows_half) {
    int single = 0;                        // smallest box that holds the rows
    while ((128 >> single) >= 2 * rows_half && single < 4) ++single;
    int first = single + 1;                // largest box below that, plus the smallest box for the remainder
    SwBoxes b = {single, -1, 128 >> single};
    if (first <= 4) {
        const int rem = rows_half - (128 >> first);
        if (rem > 0) {
            int second = 4;
            while ((128 >> second) < rem) --second;
            if ((128 >> first) + (128 >> second) < (128 >> single)) { b.i1 = first; b.i2 = second; b.rows = (128 >> first) + (128 >> second); }
        }
    }
    return b;
}

// How `rows` live rows are cut up for a grid of n_units CTA pairs and n_vt vocabulary tiles of 256 (the same
// formula on the host, in the GEMM and in the merge kernels).
struct SwPlan { int n_chunks, nc, groups, parts; };
__host__ __device__ inline SwPlan sw_plan(int rows, int n_units, int n_vt) {
    SwPlan p;
    p.n_chunks = (rows + SW_NMAX - 1) / SW_NMAX;
    if (p.n_chunks < 1) p.n_chunks = 1;
    const int per = (rows + p.n_chunks - 1) / p.n_chunks;
    p.nc = (per + 15) & ~15;                             // rows per chunk: N of the pair's MMA
    if (p.nc < 16) p.nc = 16;
    p.groups = lm_groups(n_units, p.n_chunks, n_vt);
    p.parts = SW_PARTS_PER_GROUP * p.groups;
    return p;
}

__device__ __forceinline__ void
lm_swapped_body(const CUtensorMap& tmap_w, const SwXMaps& xmaps, int Mc, int D, int V, int mask_col, int n_vt,
                float* __restrict__ part_max, float* __restrict__ part_sum, int32_t* __restrict__ part_arg,
                uint32_t* __restrict__ dev_status, int parts_stride) {
    if (Mc <= 0) return;
    const int rank = static_cast<int>(cluster_cta_rank());
    const int unit = blockIdx.x >> 1;
    const int n_units = gridDim.x >> 1;
    const SwPlan plan = sw_plan(Mc, n_units, n_vt);
    const int n_items = plan.n_chunks * plan.groups;
    if (unit >= n_items) return;                         // (both CTAs of a pair alike)
    const int nc = plan.nc, groups = plan.groups;
    const int rows_half = nc >> 1;                       // this CTA's share of a chunk's rows (multiple of 8)

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    float* xpose = reinterpret_cast<float*>(tiles + SW_STAGES * SW_STAGE_BYTES);
    SwBarriers* bars = reinterpret_cast<SwBarriers*>(xpose + 4 * SW_XP_FLOATS);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = warp_index_uniform();
    const int lane = threadIdx.x & 31;

    // A ring slot holds a 16 KB W tile and the X rows this CTA loads.  With few live rows the X part is small and the
    // ring's bytes make more slots: while W streams from HBM, what a CTA has in flight is what bounds its share of the
    // bandwidth (6 slots per CTA, 14 MB over the GPU, covered ~2 us of HBM latency at 6.3 TB/s and no more).
    const SwBoxes xbox = sw_boxes(rows_half);
    const int stage_bytes = SW_W_BYTES + ((xbox.rows * 128 + 1023) & ~1023);
    const int n_stages = min(SW_MAX_STAGES, SW_STAGES * SW_STAGE_BYTES / stage_bytes);
    if (threadIdx.x == 0) {
        for (int s = 0; s < n_stages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(&bars->tmem_full[a], 1);
            mbar_init(&bars->tmem_empty[a], 8);          // one arrival per epilogue warp of both CTAs
        }
        mbar_init(&bars->fold_full, 128);
        mbar_init(&bars->fold_empty, 128);
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    if (warp == 1) { tmem_alloc_pair(&bars->tmem_base, TMEM_COLS); tmem_relinquish_pair(); }
    tc_fence_before_sync();
    cluster_sync_all();                                  // both CTAs' barriers exist before either signals the other's
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;
    const int num_k = (D + BK - 1) / BK;

    // item w -> chunk w % n_chunks, vocabulary group w / n_chunks; the group's tiles are g, g + groups, ...
    if (warp == 0) {
        if (lane == 0) {
            prefetch_tensormap(&tmap_w);
#pragma unroll
            for (int i = 0; i < 5; ++i) prefetch_tensormap(&xmaps.m[i]);
            int stage = 0;
            uint32_t phase = 0;
            bool ok = true;
            const uint32_t full0 = cluster_map_shared(smem_u32(&bars->full[0]), 0);   // the even CTA's barriers count both CTAs' bytes
            const SwBoxes box = xbox;
            const uint32_t stage_tx = 2u * static_cast<uint32_t>(SW_W_BYTES + box.rows * 128);
            for (int item = unit; item < n_items && ok; item += n_units) {
                const int x_row0 = (item % plan.n_chunks) * nc + rank * rows_half;
                for (int vt = item / plan.n_chunks; vt < n_vt && ok; vt += groups) {
                    const int w_row0 = vt * (2 * SW_BV) + rank * SW_BV;
                    for (int kb = 0; kb < num_k; ++kb) {
                        if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) { ok = false; break; }
                        uint8_t* w_dst = tiles + stage * stage_bytes;
                        uint8_t* x_dst = w_dst + SW_W_BYTES;
                        const uint32_t full = full0 + stage * static_cast<uint32_t>(sizeof(uint64_t));
                        if (rank == 0) mbar_arrive_expect_tx(&bars->full[stage], stage_tx);
                        tma_load_2d_pair(w_dst, &tmap_w, full, kb * BK, w_row0);
                        tma_load_2d_pair(x_dst, &xmaps.m[box.i1], full, kb * BK, x_row0);
                        if (box.i2 >= 0)
                            tma_load_2d_pair(x_dst + (128 >> box.i1) * 128, &xmaps.m[box.i2], full, kb * BK,
                                             x_row0 + (128 >> box.i1));
                        if (++stage == n_stages) { stage = 0; phase ^= 1; }
                    }
                }
            }
        }
    } else if (warp == 1 && rank == 0) {
        // all lanes run the loops, one elected lane issues the MMAs of the pair and their commits
        const bool leader = elect_one_sync();
        const uint32_t idesc = umma_idesc_bf16(2 * SW_BV, nc);
        int stage = 0;
        uint32_t phase = 0;
        int it = 0;
        bool ok = true;
        for (int item = unit; item < n_items && ok; item += n_units) {
            for (int vt = item / plan.n_chunks; vt < n_vt && ok; vt += groups, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->tmem_empty[acc], acc_phase ^ 1, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * SW_NMAX;
                for (int kb = 0; kb < num_k; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->full[stage], phase, abort_flag));
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t w_addr = smem_u32(tiles + stage * stage_bytes);
                    const uint64_t a_desc = umma_desc_sw128_kmajor(w_addr);
                    const uint64_t b_desc = umma_desc_sw128_kmajor(w_addr + SW_W_BYTES);
                    if (leader) {
#pragma unroll
                        for (int kk = 0; kk < BK / 16; ++kk)
                            umma_bf16_pair(d_tmem, a_desc + 2 * kk, b_desc + 2 * kk, idesc, (kb | kk) != 0);
                        umma_commit_pair(&bars->empty[stage], 3);      // frees the stage in both CTAs
                    }
                    __syncwarp();
                    if (++stage == n_stages) { stage = 0; phase ^= 1; }
                }
                if (ok && leader) umma_commit_pair(&bars->tmem_full[acc], 3);
                __syncwarp();
            }
        }
    } else if (warp >= 2) {
        // epilogue: warp w may touch TMEM lanes [32 * (w % 4), +32) = 32 consecutive vocabulary entries of the tile
        const int lq = warp & 3;
        float* xp = xpose + lq * SW_XP_FLOATS;
        int it = 0;
        uint32_t items_done = 0;
        bool ok = true;
        for (int item = unit; item < n_items && ok; item += n_units, ++items_done) {
            const int chunk = item % plan.n_chunks;
            const int group = item / plan.n_chunks;
            float run_max[SW_NMAX / 32], run_sum[SW_NMAX / 32];
            int run_arg[SW_NMAX / 32];
#pragma unroll
            for (int cb = 0; cb < SW_NMAX / 32; ++cb) { run_max[cb] = -INFINITY; run_sum[cb] = 0.f; run_arg[cb] = ARG_NONE; }
            for (int vt = group; vt < n_vt && ok; vt += groups, ++it) {
                const int acc = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->tmem_full[acc], acc_phase, abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t taddr = tmem_base + (static_cast<uint32_t>(lq * 32) << 16) + acc * SW_NMAX;
                const int vbase = vt * (2 * SW_BV) + rank * SW_BV + lq * 32;     // first vocabulary entry of this warp's lanes
                const bool edge = (vbase + 32 > V) || (mask_col >= vbase && mask_col < vbase + 32);
                if (vbase < V) {
#pragma unroll
                    for (int cb = 0; cb < SW_NMAX / 32; ++cb) {
                        if (cb * 32 < nc) {
                            uint32_t v[32];
                            tmem_ld_32cols(taddr + cb * 32, v);
                            tmem_ld_wait();
                            // turn the block: in, thread = vocabulary entry with 32 rows; out, thread = row with 32 entries
#pragma unroll
                            for (int c = 0; c < 32; ++c) xp[lane * 33 + c] = __uint_as_float(v[c]);
                            __syncwarp();
                            float z[32];
#pragma unroll
                            for (int l = 0; l < 32; ++l) z[l] = xp[l * 33 + lane];
                            __syncwarp();
                            if (edge) {
#pragma unroll
                                for (int l = 0; l < 32; ++l)
                                    if (vbase + l >= V || vbase + l == mask_col) z[l] = -INFINITY;
                            }
                            float cmax = -INFINITY;
                            int carg = ARG_NONE;
#pragma unroll
                            for (int l = 0; l < 32; ++l)
                                if (z[l] > cmax) { cmax = z[l]; carg = vbase + l; }       // strict '>' keeps the lowest id
                            if (cmax > -INFINITY) {
                                if (cmax > run_max[cb]) {     // tiles of a group come in ascending order: '>' keeps the lowest id
                                    run_sum[cb] *= fast_exp2((run_max[cb] - cmax) * LOG2E);   // exp2(-inf) = 0 the first time
                                    run_max[cb] = cmax;
                                    run_arg[cb] = carg;
                                }
                                const float mb = run_max[cb] * LOG2E;
                                float sum = 0.f;
#pragma unroll
                                for (int l = 0; l < 32; ++l) sum += fast_exp2(fmaf(z[l], LOG2E, -mb));
                                run_sum[cb] += sum;
                            }
                        }
                    }
                }
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(&bars->tmem_empty[acc], 0);   // one arrival per warp, on the even CTA's barrier
            }
            if (ok) {
                // fold the four warps' values (each saw a quarter of every tile's vocabulary entries): every warp
                // leaves its own in its block of shared memory, then warp q folds column blocks 2 q and 2 q + 1
#pragma unroll
                for (int cb = 0; cb < SW_NMAX / 32; ++cb) {
                    xp[(cb * 3 + 0) * 32 + lane] = run_max[cb];
                    xp[(cb * 3 + 1) * 32 + lane] = run_sum[cb];
                    xp[(cb * 3 + 2) * 32 + lane] = __int_as_float(run_arg[cb]);
                }
                mbar_arrive(&bars->fold_full);            // (release: the values above are visible to the waiters)
                ok = __all_sync(0xffffffffu, mbar_wait(&bars->fold_full, items_done & 1, abort_flag));
                if (ok) {
                    for (int cb = 2 * lq; cb < 2 * lq + 2; ++cb) {
                        const int col = cb * 32 + lane;
                        const int row = chunk * nc + col;
                        if (col < nc && row < Mc) {
                            float m = -INFINITY, sum = 0.f;
                            int a = ARG_NONE;
                            for (int q = 0; q < 4; ++q) {
                                const float* src = xpose + q * SW_XP_FLOATS + cb * 96 + lane;
                                const float m2 = src[0], s2 = src[32];
                                const int a2 = __float_as_int(src[64]);
                                if (m2 > -INFINITY) {
                                    if (m2 > m) { sum = sum * fast_exp2((m - m2) * LOG2E) + s2; m = m2; a = a2; }
                                    else { sum += s2 * fast_exp2((m2 - m) * LOG2E); if (m2 == m && a2 < a) a = a2; }
                                }
                            }
                            const size_t o = static_cast<size_t>(row) * parts_stride + group * 2 + rank;
                            part_max[o] = m;
                            part_sum[o] = sum;
                            part_arg[o] = a;
                        }
                    }
                    mbar_arrive(&bars->fold_empty);       // the blocks may be written again once all have read
                    ok = __all_sync(0xffffffffu, mbar_wait(&bars->fold_empty, items_done & 1, abort_flag));
                }
            }
        }
    }

    // teardown: neither CTA leaves while its partner can still signal its barriers or read its tiles
    tc_fence_before_sync();
    cluster_sync_all();
    if (*abort_flag) {
        // give copies still in flight time to land before the shared memory is released
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
        if (threadIdx.x == 0) atomicOr(dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc_pair(tmem_base, TMEM_COLS);
    }
}

// An odd number of row tiles, 2 p + 1, on n_clusters CTA pairs: the first lm_mixed_pair_clusters() clusters run the
// row-major pair path on the tiles [0, 2 p), and the CTAs of the remaining clusters each run the single-CTA path on
// the last tile.  The split balances the two parts: an item of two row tiles costs a pair one unit of time, an item
// of one row tile costs a single CTA about 1.2 (its tensor pipe is busy 83 % of the time against 97 %), i.e. a
// cluster of two such CTAs 0.6 per item.  (Same formula on the host, in the GEMM and in the merge kernels.)
__host__ __device__ inline int lm_mixed_pair_clusters(int n_clusters, int p) {
    int up = (n_clusters * 10 * p + 5 * p + 3) / (10 * p + 6);      // round(n_clusters * p / (p + 0.6))
    if (up > n_clusters - 1) up = n_clusters - 1;
    if (up < 1) up = 1;
    return up;
}

// The greedy head, one launch on CTA pairs whatever the number of live rows (known only on the device when rows are
// skipped): the swapped-operand path for the counts lm_greedy_swapped names (up to SW_NMAX rows, and counts that
// cut into long chunks); otherwise row-major tiles of 128 rows, on CTA pairs when the tiles come in twos, and for
// an odd count on pairs plus single CTAs for the last tile (see above).  The W
// tile box is 128 rows for all of them.  A row's partials start at row * parts_stride; how many there are follows
// from the same rules in lm_row_partials.
__global__ void __launch_bounds__(LM_THREADS, 1)
lmhead_greedy_kernel(const __grid_constant__ CUtensorMap tmap_w, const __grid_constant__ SwXMaps xmaps, int M,
                     const int32_t* __restrict__ live_rows, int D, int V, int mask_col, int n_tiles,
                     float* __restrict__ part_max, float* __restrict__ part_sum, int32_t* __restrict__ part_arg,
                     uint32_t* __restrict__ dev_status, int parts_stride) {
    const int Mc = live_rows ? *live_rows : M;          // rows that need logits (uniform over the grid)
    if (lm_greedy_swapped(Mc)) {
        lm_swapped_body(tmap_w, xmaps, Mc, D, V, mask_col, n_tiles, part_max, part_sum, part_arg, dev_status, parts_stride);
        return;
    }
    const LmSampling none = {};
    const int m_tiles = (Mc + BM - 1) / BM;
    const int cluster = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    if ((m_tiles & 1) == 0) {
        const LmUnits u = {cluster, n_clusters, 0, m_tiles, parts_stride};
        lm_rowmajor_body<LM_GREEDY, true>(xmaps.m[0], tmap_w, Mc, D, V, mask_col, n_tiles, part_max, part_sum, part_arg,
                                          dev_status, none, u);
    } else if (n_clusters < 2) {
        const LmUnits u = {static_cast<int>(blockIdx.x), static_cast<int>(gridDim.x), 0, m_tiles, parts_stride};
        lm_rowmajor_body<LM_GREEDY, false, true>(xmaps.m[0], tmap_w, Mc, D, V, mask_col, n_tiles, part_max, part_sum,
                                                 part_arg, dev_status, none, u);
    } else {
        const int p = m_tiles >> 1;
        const int up = lm_mixed_pair_clusters(n_clusters, p);
        if (cluster < up) {
            const LmUnits u = {cluster, up, 0, 2 * p, parts_stride};
            lm_rowmajor_body<LM_GREEDY, true>(xmaps.m[0], tmap_w, Mc, D, V, mask_col, n_tiles, part_max, part_sum,
                                              part_arg, dev_status, none, u);
        } else {
            const LmUnits u = {static_cast<int>(blockIdx.x) - 2 * up, static_cast<int>(gridDim.x) - 2 * up, 2 * p, 1,
                               parts_stride};
            lm_rowmajor_body<LM_GREEDY, false, true>(xmaps.m[0], tmap_w, Mc, D, V, mask_col, n_tiles, part_max, part_sum,
                                                     part_arg, dev_status, none, u);
        }
    }
}

// Partials of live row `row`, as the GEMM that ran wrote them (they start at row * stride).  layout 0 / 1: the
// stand-alone row-major kernels (single CTAs only / CTA pairs where they apply), one partial per vocabulary group,
// packed (stride = count).  layout 2: lmhead_greedy_kernel's rules.  `grid` = CTAs of the GEMM launch, n_tiles =
// vocabulary tiles of 256.
constexpr int LM_LAYOUT_GREEDY = 2;
__host__ __device__ inline int lm_row_partials(int layout, int grid, int rows, int n_tiles, int row) {
    const int m_tiles = (rows + BM - 1) / BM;
    if (layout != LM_LAYOUT_GREEDY) return lm_groups_mode(grid, m_tiles, n_tiles, layout);
    const int n_clusters = grid >> 1;
    if (lm_greedy_swapped(rows)) return sw_plan(rows, n_clusters, n_tiles).parts;
    if ((m_tiles & 1) == 0) return lm_groups(n_clusters, m_tiles >> 1, n_tiles);
    if (n_clusters < 2) return lm_groups(grid, m_tiles, n_tiles);
    const int p = m_tiles >> 1;
    const int up = lm_mixed_pair_clusters(n_clusters, p);
    return row < 2 * p * BM ? lm_groups(up, p, n_tiles) : lm_groups(grid - 2 * up, 1, n_tiles);
}

// Fold of one row's partial triples by a warp: returns (argmax token, sum of exp relative to the maximum) in all
// lanes.  Ties of the maximum go to the lowest token id.
__device__ __forceinline__ void merge_row_partials(const float* __restrict__ part_max, const float* __restrict__ part_sum,
                                                   const int32_t* __restrict__ part_arg, size_t base, int groups, int lane,
                                                   int& a_out, float& s_out) {
    float m = -INFINITY, s = 0.f;
    int a = ARG_NONE;
    // the loads of a batch are issued together (five per lane cover 160 partials: one round trip to memory for the
    // usual case), then folded
    constexpr int BATCH = 5;
    for (int t0 = lane; t0 < groups; t0 += 32 * BATCH) {
        float bm[BATCH], bs[BATCH];
        int ba[BATCH];
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const int t = t0 + 32 * u;
            const bool in = t < groups;
            bm[u] = in ? part_max[base + t] : -INFINITY;
            bs[u] = in ? part_sum[base + t] : 0.f;
            ba[u] = in ? part_arg[base + t] : ARG_NONE;
        }
#pragma unroll
        for (int u = 0; u < BATCH; ++u) {
            const float m2 = bm[u], s2 = bs[u];
            const int a2 = ba[u];
            if (m2 > -INFINITY) {
                if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; a = a2; }
                else { s += s2 * exp2f((m2 - m) * LOG2E); if (m2 == m && a2 < a) a = a2; }
            }
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
        const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
        const int a2 = __shfl_xor_sync(0xffffffffu, a, off);
        if (m2 > -INFINITY) {
            if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; a = a2; }
            else { s += s2 * exp2f((m2 - m) * LOG2E); if (m2 == m && a2 < a) a = a2; }
        }
    }
    a_out = a;
    s_out = s;
}

// One warp per live row: fold the row's partial triples (one per vocabulary group) into (token, confidence)
// and write them at the row's original position.
__global__ void lmhead_merge_kernel(const float* __restrict__ part_max, const float* __restrict__ part_sum,
                                    const int32_t* __restrict__ part_arg, int grid_gemm, int n_tiles, int M,
                                    const int32_t* __restrict__ live_rows, const int32_t* __restrict__ idx,
                                    int32_t* __restrict__ pred, float* __restrict__ conf, int allow_pair,
                                    int parts_stride) {
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int Mc = live_rows ? *live_rows : M;
    if (c >= Mc) return;
    const int groups = lm_row_partials(allow_pair, grid_gemm, Mc, n_tiles, c);
    int a;
    float s;
    merge_row_partials(part_max, part_sum, part_arg, static_cast<size_t>(c) * (parts_stride < 0 ? groups : parts_stride),
                       groups, lane, a, s);
    if (lane == 0) {
        const int row = idx ? idx[c] : c;
        pred[row] = a;
        conf[row] = 1.0f / s;   // exp(max - logsumexp) with the sum taken relative to the max
    }
}

// Merge and unmask selection in one kernel, for blocks of at most 32 positions: one CTA per rollout, one warp per
// block position.  A warp whose position is still masked finds its row's place among the compacted rows (from the
// compaction kernel's sorted row list: other CTAs change the token state meanwhile), folds the row's partials and writes
// (pred, conf); then the CTA applies the selection rule of select.cu to the block: rank by counting, bit for bit
// the same decisions as the separate kernel takes from the same (pred, conf).
struct LmSelect {
    int32_t* tokens_block;      // tokens + block_start (row b at + b * row_stride)
    int64_t row_stride;
    int mode;
    float threshold;
    int k;
    int32_t* n_committed;
    int32_t* n_remaining;
};
__global__ void __launch_bounds__(1024)
lmhead_merge_select_kernel(const float* __restrict__ part_max, const float* __restrict__ part_sum,
                           const int32_t* __restrict__ part_arg, int grid_gemm, int n_tiles, int L,
                           const int32_t* __restrict__ live_rows, const int32_t* __restrict__ idx, int32_t mask_id,
                           int32_t* __restrict__ pred, float* __restrict__ conf, int allow_pair, int parts_stride,
                           const LmSelect sel) {
    __shared__ int s_before;
    __shared__ int s_flag[32];
    __shared__ float s_conf[32];
    __shared__ int32_t s_pred[32];
    const int b = blockIdx.x;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;      // warp = block position (blockDim = 32 L)
    const int Mc = *live_rows;
    if (threadIdx.x == 0) {
        // compacted rows that belong to earlier rollouts = first entry of the ascending row list that is >= b * L
        int lo = 0, hi = Mc;
        while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (idx[mid] < b * L) lo = mid + 1; else hi = mid;
        }
        s_before = lo;
    }
    int32_t* row = sel.tokens_block + static_cast<int64_t>(b) * sel.row_stride;
    const bool masked = row[warp] == mask_id;
    if (lane == 0) s_flag[warp] = masked ? 1 : 0;
    __syncthreads();
    if (masked) {
        int c = s_before;
        for (int i = 0; i < warp; ++i) c += s_flag[i];
        const int groups = lm_row_partials(allow_pair, grid_gemm, Mc, n_tiles, c);
        int a;
        float s;
        merge_row_partials(part_max, part_sum, part_arg, static_cast<size_t>(c) * (parts_stride < 0 ? groups : parts_stride),
                           groups, lane, a, s);
        if (lane == 0) {
            float cf = 1.0f / s;
            pred[b * L + warp] = a;
            conf[b * L + warp] = cf;
            if (cf != cf) cf = -INFINITY;
            s_conf[warp] = cf;
            s_pred[warp] = a;
        }
    } else if (lane == 0) {
        s_conf[warp] = __int_as_float(0x7fc00000);      // absent
    }
    __syncthreads();
    if (warp != 0) return;
    // selection (warp 0, lane = block position)
    const float cf = lane < L ? s_conf[lane] : __int_as_float(0x7fc00000);
    const bool is_masked = cf == cf;
    const unsigned masked_set = __ballot_sync(0xffffffffu, is_masked);
    const unsigned above_set = __ballot_sync(0xffffffffu, is_masked && cf > sel.threshold);
    bool commit = false;
    if (is_masked) {
        if (sel.mode == DARE_SELECT_THRESHOLD && above_set != 0u) {
            commit = cf > sel.threshold;
        } else {
            const int want = sel.mode == DARE_SELECT_TOPK ? sel.k : 1;
            int rank = 0;
            for (int j = 0; j < L; ++j) {
                const float cj = s_conf[j];
                rank += (cj > cf || (cj == cf && j < lane)) ? 1 : 0;   // NaN (absent) compares false
            }
            commit = rank < want;
        }
    }
    if (commit) row[lane] = s_pred[lane];
    const unsigned commit_set = __ballot_sync(0xffffffffu, commit);
    if (lane == 0) {
        if (sel.n_committed) sel.n_committed[b] = __popc(commit_set);
        if (sel.n_remaining) sel.n_remaining[b] = __popc(masked_set) - __popc(commit_set);
    }
}

// The same fold for the sampling epilogue: log-sum-exp of the raw logits from (max, sum); the sampled token is the
// partial with the best perturbed score (lowest token id on ties); confidence = exp(z_token - logsumexp z).
__global__ void lmhead_merge_sample_kernel(const float* __restrict__ part_max, const float* __restrict__ part_sum,
                                           const int32_t* __restrict__ part_arg, const float* __restrict__ part_y,
                                           const float* __restrict__ part_zb, int grid_gemm, int n_tiles, int M,
                                           const int32_t* __restrict__ live_rows, const int32_t* __restrict__ idx,
                                           int32_t* __restrict__ pred, float* __restrict__ conf, int allow_pair,
                                           uint32_t* __restrict__ step_dev) {
    if (step_dev && blockIdx.x == 0 && threadIdx.x == 0) *step_dev += 1;   // the GEMM kernels before this one read it
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int Mc = live_rows ? *live_rows : M;
    if (c >= Mc) return;
    const int groups = lm_groups_mode(grid_gemm, (Mc + BM - 1) / BM, n_tiles, allow_pair);
    float m = -INFINITY, s = 0.f, y = -INFINITY, zb = -INFINITY;
    int a = ARG_NONE;
    const size_t base = static_cast<size_t>(c) * groups;
    for (int t = lane; t < groups; t += 32) {
        const float m2 = part_max[base + t], s2 = part_sum[base + t];
        if (m2 > -INFINITY) {
            if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; }
            else s += s2 * exp2f((m2 - m) * LOG2E);
        }
        const float y2 = part_y[base + t];
        const int a2 = part_arg[base + t];
        if (y2 > y || (y2 == y && a2 < a)) { y = y2; a = a2; zb = part_zb[base + t]; }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
        const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
        const float y2 = __shfl_xor_sync(0xffffffffu, y, off);
        const float z2 = __shfl_xor_sync(0xffffffffu, zb, off);
        const int a2 = __shfl_xor_sync(0xffffffffu, a, off);
        if (m2 > -INFINITY) {
            if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; }
            else s += s2 * exp2f((m2 - m) * LOG2E);
        }
        if (y2 > y || (y2 == y && a2 < a)) { y = y2; a = a2; zb = z2; }
    }
    if (lane == 0) {
        const int row = idx ? idx[c] : c;
        pred[row] = a;
        conf[row] = exp2f((zb - m) * LOG2E) / s;
    }
}

// Log-probability of the target: (z_target - max) - ln(sum of exp(z - max)); the target's logit sits in exactly one
// partial (the others carry -inf).  Optionally also writes logsumexp z.
__global__ void lmhead_merge_logprob_kernel(const float* __restrict__ part_max, const float* __restrict__ part_sum,
                                            const int32_t* __restrict__ part_zt, int grid_gemm, int n_tiles, int M,
                                            float* __restrict__ logprob, float* __restrict__ lse_out, int allow_pair) {
    const int c = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (c >= M) return;
    const int groups = lm_groups_mode(grid_gemm, (M + BM - 1) / BM, n_tiles, allow_pair);
    float m = -INFINITY, s = 0.f, zt = -INFINITY;
    const size_t base = static_cast<size_t>(c) * groups;
    for (int t = lane; t < groups; t += 32) {
        const float m2 = part_max[base + t], s2 = part_sum[base + t];
        if (m2 > -INFINITY) {
            if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; }
            else s += s2 * exp2f((m2 - m) * LOG2E);
        }
        zt = fmaxf(zt, __int_as_float(part_zt[base + t]));
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
        const float s2 = __shfl_xor_sync(0xffffffffu, s, off);
        zt = fmaxf(zt, __shfl_xor_sync(0xffffffffu, zt, off));
        if (m2 > -INFINITY) {
            if (m2 > m) { s = s * exp2f((m - m2) * LOG2E) + s2; m = m2; }
            else s += s2 * exp2f((m2 - m) * LOG2E);
        }
    }
    if (lane == 0) {
        logprob[c] = (zt - m) - logf(s);
        if (lse_out) lse_out[c] = m + logf(s);
    }
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Whether clusters of two CTAs of the pair-mode kernel can run on this device (asked once).
int lm_pair_available() {
    static int cache = -1;
    if (cache < 0) {
        int n = 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2048, 1, 1);
        cfg.blockDim = dim3(LM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = LM_PAIR_SMEM_BYTES;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaFuncSetAttribute(lmhead_partial_kernel<LM_GREEDY, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 LM_PAIR_SMEM_BYTES) != cudaSuccess ||
            cudaOccupancyMaxActiveClusters(&n, lmhead_partial_kernel<LM_GREEDY, true>, &cfg) != cudaSuccess)
            n = 0;
        cache = n > 0 ? 1 : 0;
    }
    return cache;
}

// The GEMM part of a head: the single-CTA kernel, the CTA-pair kernel, or (when the row count is only known on
// the device) both, of which the one whose mode does not apply returns at once.  *allow_pair_out tells the
// merge kernel which rule was in force.
template <int MODE>
int launch_partial(const dare_ctx* ctx, int grid, const CUtensorMap& tmap_x, const void* w, int M,
                   const int32_t* live_rows, int D, int V, int mask_col, int n_tiles, float* part_max, float* part_sum,
                   int32_t* part_arg, const LmSampling& smp, cudaStream_t stream, int* allow_pair_out) {
    const int allow_pair = (grid >= 2 && lm_pair_available()) ? 1 : 0;
    *allow_pair_out = allow_pair;
    const int m_tiles_host = (M + BM - 1) / BM;
    const bool pair_known = live_rows == nullptr && lm_pair_mode(m_tiles_host, allow_pair);
    const bool run_single = !allow_pair || live_rows != nullptr || !pair_known;
    const bool run_pair = allow_pair && (live_rows != nullptr || pair_known);
    if (run_single) {
        CUtensorMap tmap_w;
        int rc = make_tmap_bf16_2d(ctx, &tmap_w, w, static_cast<uint64_t>(V), static_cast<uint64_t>(D), BN, BK);
        if (rc != DARE_OK) return rc;
        static std::atomic<uint64_t> smem_set{0};
        if (ensure_dynamic_smem(smem_set, lmhead_partial_kernel<MODE, false>, LM_SMEM_BYTES) != DARE_OK) return DARE_ERR_CUDA;
        lmhead_partial_kernel<MODE, false><<<grid, lm_threads(MODE), LM_SMEM_BYTES, stream>>>(
            tmap_x, tmap_w, M, live_rows, D, V, mask_col, n_tiles, part_max, part_sum, part_arg, ctx->dev_status, smp,
            allow_pair); note_launch();
        if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
    }
    if (run_pair) {
        CUtensorMap tmap_wh;      // half a W tile per CTA
        int rc = make_tmap_bf16_2d(ctx, &tmap_wh, w, static_cast<uint64_t>(V), static_cast<uint64_t>(D), BN / 2, BK);
        if (rc != DARE_OK) return rc;
        static std::atomic<uint64_t> smem_set_pair{0};
        if (ensure_dynamic_smem(smem_set_pair, lmhead_partial_kernel<MODE, true>, LM_PAIR_SMEM_BYTES) != DARE_OK)
            return DARE_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(grid & ~1), 1, 1);
        cfg.blockDim = dim3(lm_threads(MODE), 1, 1);
        cfg.dynamicSmemBytes = LM_PAIR_SMEM_BYTES;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, lmhead_partial_kernel<MODE, true>, tmap_x, tmap_wh, M, live_rows, D, V, mask_col,
                               n_tiles, part_max, part_sum, part_arg, ctx->dev_status, smp, allow_pair) != cudaSuccess)
            return DARE_ERR_CUDA;
        note_launch();
    }
    return DARE_OK;
}

}  // namespace

// Scratch layout: [compacted X: M*D bf16][row indices: M int32][live-row count][partials: 3 x M x groups]
size_t lmhead_workspace_bytes(int M, int D, int V, int sm_count, bool with_row_tokens, bool sampling) {
    const size_t n_tiles = (static_cast<size_t>(V) + BN - 1) / BN;
    size_t groups = static_cast<size_t>(sm_count);
    if (groups > n_tiles) groups = n_tiles;
    if (!sampling) {      // the greedy head's swapped path: two partials per vocabulary group of a CTA pair
        groups = static_cast<size_t>(sm_count);
        if (groups > 2 * n_tiles) groups = 2 * n_tiles;
    }
    size_t bytes = (sampling ? 5 : 3) * sizeof(float) * groups * static_cast<size_t>(M);
    if (with_row_tokens)
        bytes += round_up(static_cast<size_t>(M) * D * 2, 1024) + round_up(static_cast<size_t>(M) * 4 + 4, 1024);
    return bytes;
}

int launch_lmhead(const dare_ctx* ctx, void* scratch, const void* hidden, int M, int D, const void* w, int V,
                  const int32_t* row_tokens, int tok_L, int64_t tok_row_stride, int32_t mask_id,
                  int exclude_mask_column, int32_t* pred, float* conf, cudaStream_t stream, const LmSampleArgs* sample,
                  const LmSelectArgs* select, cudaEvent_t after_compaction) {
    if (select && (sample || !row_tokens || tok_L > LMHEAD_SELECT_MAX_L || tok_L < 1 || M != select->B * tok_L))
        return DARE_ERR_SHAPE;
    const int n_tiles = (V + BN - 1) / BN;
    const int m_tiles_max = (M + BM - 1) / BM;
    int grid = ctx->sm_count;
    if (grid > m_tiles_max * n_tiles) grid = m_tiles_max * n_tiles;

    uint8_t* cur = static_cast<uint8_t*>(scratch);
    const void* x_gemm = hidden;
    int32_t* idx = nullptr;
    int32_t* live_rows = nullptr;
    if (row_tokens != nullptr) {
        void* xc = cur;
        cur += round_up(static_cast<size_t>(M) * D * 2, 1024);
        idx = reinterpret_cast<int32_t*>(cur);
        live_rows = idx + M;
        cur += round_up(static_cast<size_t>(M) * 4 + 4, 1024);
        x_gemm = xc;
        lmhead_compact_kernel<<<(M + CP_ROWS - 1) / CP_ROWS, CP_ROWS * 32, 0, stream>>>(
            static_cast<const uint4*>(hidden), M, D / 8, row_tokens, tok_L, tok_row_stride, mask_id,
            static_cast<uint4*>(xc), idx, live_rows, pred, conf); note_launch();
        if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
    }
    if (after_compaction && cudaEventRecord(after_compaction, stream) != cudaSuccess) return DARE_ERR_CUDA;
    size_t groups_max = static_cast<size_t>(ctx->sm_count);
    if (groups_max > static_cast<size_t>(n_tiles)) groups_max = n_tiles;
    const bool greedy_pairs = sample == nullptr && grid >= 2 && lm_pair_available();
    if (greedy_pairs) {      // lmhead_greedy_kernel: a fixed stride, at most min(#CTAs, 2 per vocabulary tile) partials
        groups_max = static_cast<size_t>(grid & ~1);
        if (groups_max > static_cast<size_t>(2 * n_tiles)) groups_max = 2 * n_tiles;
    }
    const size_t n_part = static_cast<size_t>(M) * groups_max;
    float* part_max = reinterpret_cast<float*>(cur);
    float* part_sum = part_max + n_part;
    int32_t* part_arg = reinterpret_cast<int32_t*>(part_sum + n_part);

    const int mask_col = (exclude_mask_column && mask_id >= 0 && mask_id < V) ? mask_id : -1;
    const int rows_per_block = 8;
    int rc = DARE_OK;
    if (greedy_pairs) {
        CUtensorMap tmap_w;
        SwXMaps xm;
        rc = make_tmap_bf16_2d(ctx, &tmap_w, w, static_cast<uint64_t>(V), static_cast<uint64_t>(D), SW_BV, BK);
        for (int i = 0; i < 5 && rc == DARE_OK; ++i)
            rc = make_tmap_bf16_2d(ctx, &xm.m[i], x_gemm, static_cast<uint64_t>(M), static_cast<uint64_t>(D), 128u >> i, BK);
        if (rc != DARE_OK) return rc;
        const int grid_pair = grid & ~1;
        const int parts_stride = static_cast<int>(groups_max);
        constexpr int SMEM_A = SW_SMEM_BYTES > LM_PAIR_SMEM_BYTES ? SW_SMEM_BYTES : LM_PAIR_SMEM_BYTES;
        constexpr int SMEM = SMEM_A > LM_SMEM_BYTES ? SMEM_A : LM_SMEM_BYTES;
        static std::atomic<uint64_t> smem_set_greedy{0};
        if (ensure_dynamic_smem(smem_set_greedy, lmhead_greedy_kernel, SMEM) != DARE_OK) return DARE_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(static_cast<unsigned>(grid_pair), 1, 1);
        cfg.blockDim = dim3(LM_THREADS, 1, 1);
        cfg.dynamicSmemBytes = SMEM;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, lmhead_greedy_kernel, tmap_w, xm, M, static_cast<const int32_t*>(live_rows), D, V,
                               mask_col, n_tiles, part_max, part_sum, part_arg, ctx->dev_status, parts_stride) != cudaSuccess)
            return DARE_ERR_CUDA;
        note_launch();
        if (select) {
            LmSelect sel;
            sel.tokens_block = select->tokens_block; sel.row_stride = tok_row_stride; sel.mode = select->mode;
            sel.threshold = select->threshold; sel.k = select->k;
            sel.n_committed = select->n_committed; sel.n_remaining = select->n_remaining;
            lmhead_merge_select_kernel<<<select->B, 32 * tok_L, 0, stream>>>(part_max, part_sum, part_arg, grid_pair, n_tiles,
                                                                             tok_L, live_rows, idx, mask_id, pred, conf,
                                                                             LM_LAYOUT_GREEDY, parts_stride, sel);
        } else {
            lmhead_merge_kernel<<<(M + rows_per_block - 1) / rows_per_block, rows_per_block * 32, 0, stream>>>(
                part_max, part_sum, part_arg, grid_pair, n_tiles, M, live_rows, idx, pred, conf, LM_LAYOUT_GREEDY,
                parts_stride);
        }
        note_launch();
        return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
    }

    CUtensorMap tmap_x;
    rc = make_tmap_bf16_2d(ctx, &tmap_x, x_gemm, static_cast<uint64_t>(M), static_cast<uint64_t>(D), BM, BK);
    if (rc != DARE_OK) return rc;

    LmSampling smp = {};
    int allow_pair = 0;
    if (sample == nullptr) {
        rc = launch_partial<LM_GREEDY>(ctx, grid, tmap_x, w, M, live_rows, D, V, mask_col, n_tiles, part_max, part_sum,
                                       part_arg, smp, stream, &allow_pair);
        if (rc != DARE_OK) return rc;
        if (select) {
            LmSelect sel;
            sel.tokens_block = select->tokens_block; sel.row_stride = tok_row_stride; sel.mode = select->mode;
            sel.threshold = select->threshold; sel.k = select->k;
            sel.n_committed = select->n_committed; sel.n_remaining = select->n_remaining;
            lmhead_merge_select_kernel<<<select->B, 32 * tok_L, 0, stream>>>(part_max, part_sum, part_arg, grid, n_tiles,
                                                                             tok_L, live_rows, idx, mask_id, pred, conf,
                                                                             allow_pair, -1, sel); note_launch();
        } else {
            lmhead_merge_kernel<<<(M + rows_per_block - 1) / rows_per_block, rows_per_block * 32, 0, stream>>>(
                part_max, part_sum, part_arg, grid, n_tiles, M, live_rows, idx, pred, conf, allow_pair, -1); note_launch();
        }
    } else {
        smp.inv_temperature = 1.0f / sample->temperature;
        smp.seed_lo = static_cast<uint32_t>(sample->seed & 0xffffffffu);
        smp.seed_hi = static_cast<uint32_t>(sample->seed >> 32);
        smp.step = sample->step;
        smp.step_dev = sample->step_dev;
        smp.row_index = idx;
        smp.part_y = reinterpret_cast<float*>(part_arg + n_part);
        smp.part_zb = smp.part_y + n_part;
        rc = launch_partial<LM_SAMPLE>(ctx, grid, tmap_x, w, M, live_rows, D, V, mask_col, n_tiles, part_max, part_sum,
                                       part_arg, smp, stream, &allow_pair);
        if (rc != DARE_OK) return rc;
        lmhead_merge_sample_kernel<<<(M + rows_per_block - 1) / rows_per_block, rows_per_block * 32, 0, stream>>>(
            part_max, part_sum, part_arg, smp.part_y, smp.part_zb, grid, n_tiles, M, live_rows, idx, pred, conf,
            allow_pair, sample->step_dev); note_launch();
    }
    if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
    return DARE_OK;
}

int launch_lmhead_logprob(const dare_ctx* ctx, void* scratch, const void* hidden, int M, int D, const void* w, int V,
                          const int32_t* targets, int32_t mask_id, int exclude_mask_column, float* logprob, float* lse_out,
                          cudaStream_t stream) {
    const int n_tiles = (V + BN - 1) / BN;
    const int m_tiles_max = (M + BM - 1) / BM;
    int grid = ctx->sm_count;
    if (grid > m_tiles_max * n_tiles) grid = m_tiles_max * n_tiles;
    size_t groups_max = static_cast<size_t>(ctx->sm_count);
    if (groups_max > static_cast<size_t>(n_tiles)) groups_max = n_tiles;
    const size_t n_part = static_cast<size_t>(M) * groups_max;
    float* part_max = static_cast<float*>(scratch);
    float* part_sum = part_max + n_part;
    int32_t* part_zt = reinterpret_cast<int32_t*>(part_sum + n_part);
    CUtensorMap tmap_x;
    int rc = make_tmap_bf16_2d(ctx, &tmap_x, hidden, static_cast<uint64_t>(M), static_cast<uint64_t>(D), BM, BK);
    if (rc != DARE_OK) return rc;
    const int mask_col = (exclude_mask_column && mask_id >= 0 && mask_id < V) ? mask_id : -1;
    LmSampling smp = {};
    smp.targets = targets;
    int allow_pair = 0;
    rc = launch_partial<LM_LOGPROB>(ctx, grid, tmap_x, w, M, nullptr, D, V, mask_col, n_tiles, part_max, part_sum, part_zt,
                                    smp, stream, &allow_pair);
    if (rc != DARE_OK) return rc;
    const int rows_per_block = 8;
    lmhead_merge_logprob_kernel<<<(M + rows_per_block - 1) / rows_per_block, rows_per_block * 32, 0, stream>>>(
        part_max, part_sum, part_zt, grid, n_tiles, M, logprob, lse_out, allow_pair); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

// dz[m, v] = grad[m] * (1[v = targets[m]] - exp(z[m, v] - lse[m])) as bf16 [M, V] and transposed [V, ldm]
// (ldm >= M; columns [M, ldm) of the transpose are not written).
int launch_lmhead_grad(const dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V,
                       const int32_t* targets, int32_t mask_id, int exclude_mask_column, const float* lse,
                       const float* grad, void* dz, void* dzt, int ldm, cudaStream_t stream) {
    const int n_tiles = (V + BN - 1) / BN;
    const int m_tiles_max = (M + BM - 1) / BM;
    int grid = ctx->sm_count;
    if (grid > m_tiles_max * n_tiles) grid = m_tiles_max * n_tiles;
    CUtensorMap tmap_x;
    int rc = make_tmap_bf16_2d(ctx, &tmap_x, hidden, static_cast<uint64_t>(M), static_cast<uint64_t>(D), BM, BK);
    if (rc != DARE_OK) return rc;
    const int mask_col = (exclude_mask_column && mask_id >= 0 && mask_id < V) ? mask_id : -1;
    LmSampling smp = {};
    smp.targets = targets;
    smp.lse = lse;
    smp.grad = grad;
    smp.dz = static_cast<__nv_bfloat16*>(dz);
    smp.dzt = static_cast<__nv_bfloat16*>(dzt);
    smp.ldm = ldm;
    int allow_pair = 0;
    return launch_partial<LM_GRAD>(ctx, grid, tmap_x, w, M, nullptr, D, V, mask_col, n_tiles, nullptr, nullptr, nullptr, smp,
                                   stream, &allow_pair);
}

}  // namespace dare

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the LM-head entry point.
//
// Some callers must not allocate device memory at all: code inside a framework's allocator callback or
// under a memory budget that forbids cudaMalloc, and plug-ins loaded into a process whose allocator they
// do not own.  dare_create allocates its workspace,
// so those callers cannot have a context.  For them the per-tile (max, sum, argmax) triples of the LM
// head live in a fixed array inside the library's device image.
namespace dare {
namespace {

// Scratch shared by every call of dare_lmhead_confidence_static on a device (8 MiB, resident on every GPU
// that loads the library until the process exits).
static __device__ __align__(256) unsigned char g_lm_static_scratch[DARE_LMHEAD_STATIC_SCRATCH_BYTES];
// Status bits of these calls (only ever OR-ed into; starts at zero when the module is loaded).
static __device__ uint32_t g_lm_static_status;

struct StaticDeviceState {
    bool ready = false;
    int device = -1;
    void* scratch = nullptr;        // device address of g_lm_static_scratch on this device
    uint32_t* status = nullptr;     // device address of g_lm_static_status on this device
    int sm_count = 0;
    dare_encode_tiled_fn encode = nullptr;
};
constexpr int MAX_DEVICES = 64;
StaticDeviceState g_static_state[MAX_DEVICES];
std::mutex g_static_mutex;

// One-time set-up for the current device.  In host code the array's name is only a handle; the address a
// kernel can use has to be asked for, with this device current.
int static_state_for_current_device(StaticDeviceState** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return DARE_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState& st = g_static_state[dev];
    if (!st.ready) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return DARE_ERR_CUDA;
        if (major != 10) return DARE_ERR_UNSUPPORTED;
        if (cudaDeviceGetAttribute(&st.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return DARE_ERR_CUDA;
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_lm_static_scratch) != cudaSuccess || p == nullptr) return DARE_ERR_CUDA;
        st.scratch = p;
        void* ps = nullptr;
        if (cudaGetSymbolAddress(&ps, g_lm_static_status) != cudaSuccess || ps == nullptr) return DARE_ERR_CUDA;
        st.status = static_cast<uint32_t*>(ps);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || fn == nullptr)
            return DARE_ERR_CUDA;
        st.encode = reinterpret_cast<dare_encode_tiled_fn>(fn);
        st.device = dev;
        st.ready = true;
    }
    *out = &st;
    return DARE_OK;
}

}  // namespace
}  // namespace dare

extern "C" int dare_lmhead_confidence_static(const void* hidden, int M, int D, const void* w, int V,
                                             const int32_t* row_tokens, int32_t mask_id, int exclude_mask_column,
                                             int32_t* pred, float* conf, void* stream) {
    if (!hidden || !w || !pred || !conf) return DARE_ERR_NULL;
    if (M < 1 || D < 8 || D % 8 != 0 || V < 2) return DARE_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(hidden) & 15u) || (reinterpret_cast<uintptr_t>(w) & 15u)) return DARE_ERR_ALIGN;
    dare::StaticDeviceState* st = nullptr;
    int rc = dare::static_state_for_current_device(&st);
    if (rc != DARE_OK) return rc;
    if (dare::lmhead_workspace_bytes(M, D, V, st->sm_count, row_tokens != nullptr, false) >
        static_cast<size_t>(DARE_LMHEAD_STATIC_SCRATCH_BYTES))
        return DARE_ERR_WORKSPACE;   // beyond the fixed scratch: use dare_lmhead_confidence with a context
    // The kernels run on the current device with that device's scratch: a buffer that lives on another GPU would be
    // read or written through the wrong address space.  Asking where a pointer lives allocates nothing.
    const void* bufs[5] = {hidden, w, row_tokens, pred, conf};
    for (const void* p : bufs) {
        if (!p) continue;
        cudaPointerAttributes attr;
        if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) return DARE_ERR_CUDA;
        if ((attr.type == cudaMemoryTypeDevice || attr.type == cudaMemoryTypeManaged) && attr.device != st->device)
            return DARE_ERR_DEVICE;
    }
    // a context-shaped view of the static state for the shared launcher; nothing here is allocated
    dare_ctx view;
    view.tmaps = nullptr;
    view.aux = nullptr; view.ev_fork = nullptr; view.ev_mid = nullptr; view.ev_join = nullptr;
    view.device = st->device;
    view.sm_count = st->sm_count;
    view.workspace = st->scratch;
    view.workspace_bytes = DARE_LMHEAD_STATIC_SCRATCH_BYTES;
    view.dev_status = st->status;
    view.encode_tiled = st->encode;
    return dare::launch_lmhead(&view, st->scratch, hidden, M, D, w, V, row_tokens, M, 0, mask_id, exclude_mask_column,
                               pred, conf, static_cast<cudaStream_t>(stream), nullptr);
}


// Reads and clears the status word of the allocation-free calls on the current device (bits DARE_DEV_*), after
// everything enqueued on `stream` so far has run.  Allocates nothing.
extern "C" int dare_lmhead_static_status(void* stream, uint32_t* host_out) {
    if (!host_out) return DARE_ERR_NULL;
    dare::StaticDeviceState* st = nullptr;
    int rc = dare::static_state_for_current_device(&st);
    if (rc != DARE_OK) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host_out, st->status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess ||
        cudaMemsetAsync(st->status, 0, sizeof(uint32_t), s) != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess)
        return DARE_ERR_CUDA;
    return DARE_OK;
}
