// Block-bidirectional attention of the current block's queries against the prefix cache, the block's own
// K/V and the optional suffix cache, with GQA.
//
// In every workload of this path the step is bound by reading K/V from HBM (L * Hq/Hkv flops per cache
// byte, at or below the machine's ridge), so the kernel is organised around the K/V stream:
//   * one CTA per (query chunk, batch row x KV head, KV split); the query rows of all Hq/Hkv heads that
//     share a KV head are packed into the same tile so each K/V byte is read once per unit;
//   * a producer warp streams 64-key K and V tiles through a 3-stage shared-memory ring with TMA
//     (128-byte swizzle, full/empty mbarriers); a consumer warp owns 16 query rows and, when few rows
//     share a KV head, a slice of each tile's keys (its running softmax is merged with its peers' at the end);
//   * QK^T and PV run on warp-level tensor-core MMAs (m16n8k16, bf16 -> fp32) straight from the swizzled
//     tiles via ldmatrix; the online softmax lives in registers (quad shuffles for the row max).
// The 128-row tcgen05 tile does not fit these shapes (32 or 4 query rows per KV head in the MHA workloads).
// With KV splits each CTA writes a normalised partial and its log-sum-exp; a small kernel combines them.
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace dare {
namespace {

constexpr int KT_MAX = 64;       // keys per tile of the widest variant (sizes the launch plan)
constexpr int ATT_MAX_STAGES = 4;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;

struct AttnParams {
    int B, L, Hq, Hkv, g, R;      // R = L * g packed query rows per (row, kv head)
    int prefix_cap, suffix_cap;
    int inplace, has_suffix, splits;
    int uniform_P;                // >= 0: every row's prefix length (used when prefix_len is NULL)
    const int32_t* cu_seqlens;    // packed variable-length mode (tcgen05 kernel): sequence b owns tokens [cu[b], cu[b+1])
    int total_tokens;             // packed mode: rows of q / k / v
    float scale_log2;
    const __nv_bfloat16* q;
    const int32_t* prefix_len;
    const int32_t* suffix_len;
    __nv_bfloat16* out;
    float* lse;
    float* part_o;                // [splits][B*L*Hq][D] fp32, used when splits > 1
    float* part_lse;              // [splits][B*L*Hq]
    uint32_t* dev_status;
};

struct AttBarriers {
    uint64_t full[ATT_MAX_STAGES];
    uint64_t empty[ATT_MAX_STAGES];
    uint32_t abort_flag;
};

template <int D, int KT>
__host__ __device__ constexpr int att_stage_bytes() { return 2 * KT * D * 2; }
template <int D, int KT, int STAGES>
__host__ __device__ constexpr int att_smem_bytes() { return STAGES * att_stage_bytes<D, KT>() + static_cast<int>(sizeof(AttBarriers)) + 1024; }

// Segment bookkeeping of one (row, kv head) unit: tiles of the prefix, then the block, then the suffix.
struct TileInfo {
    int seg;      // 0 prefix buffer, 1 block buffer, 2 suffix buffer
    int row0;     // first row of the tile in that buffer's 2-D [rows, D] view
    int valid;    // keys of the tile that exist (1..KT)
};

template <int KT>
__device__ __forceinline__ TileInfo tile_info(int t, int n_pre, int n_blk, int len_pre, int len_blk, int len_suf,
                                              int base_pre, int base_blk, int base_suf) {
    TileInfo ti;
    if (t < n_pre) {
        ti.seg = 0; ti.row0 = base_pre + t * KT; ti.valid = min(KT, len_pre - t * KT);
    } else if (t < n_pre + n_blk) {
        t -= n_pre;
        ti.seg = 1; ti.row0 = base_blk + t * KT; ti.valid = min(KT, len_blk - t * KT);
    } else {
        t -= n_pre + n_blk;
        ti.seg = 2; ti.row0 = base_suf + t * KT; ti.valid = min(KT, len_suf - t * KT);
    }
    return ti;
}

// NW row groups of 16 packed query rows; KS warps share a row group and split every 64-key tile between
// them (KT / KS keys each), keeping separate running (max, sum, O) that are merged through shared memory at
// the end.  More warps per SM hide the latency of the ldmatrix -> MMA -> softmax chain.
// KT keys per tile and ATT_STAGES ring slots set the shared memory of a CTA and so how many CTAs an SM holds (CPS).
template <int D, int NW, int KS, int KT, int ATT_STAGES, int CPS>
__global__ void __launch_bounds__((NW * KS + 1) * 32, CPS)
attn_block_kernel(const __grid_constant__ CUtensorMap tm_kpre, const __grid_constant__ CUtensorMap tm_vpre,
                  const __grid_constant__ CUtensorMap tm_kblk, const __grid_constant__ CUtensorMap tm_vblk,
                  const __grid_constant__ CUtensorMap tm_ksuf, const __grid_constant__ CUtensorMap tm_vsuf,
                  const AttnParams p) {
    constexpr int STAGE = att_stage_bytes<D, KT>();
    constexpr int HALF = KT * 128;           // one 64-column half of a tile: KT rows x 128 bytes
    constexpr int NHALF = D / 64;
    constexpr int KV_BYTES = KT * D * 2;
    constexpr int NCW = NW * KS;             // consumer warps
    constexpr int KPW = KT / KS;             // keys per warp per tile
    constexpr int NREG = (D / 8) * 4 + 4;    // floats a thread hands over in the final merge

    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    AttBarriers* bars = reinterpret_cast<AttBarriers*>(tiles + ATT_STAGES * STAGE);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int chunk = blockIdx.x;
    const int unit = blockIdx.y;
    const int split = blockIdx.z;
    const int b = unit / p.Hkv;
    const int kvh = unit % p.Hkv;

    // A CTA lives for a handful of tiles, so what it does before its first tile arrives counts.  Nothing below waits
    // for anything else: the row's lengths are requested first (needed only after the barrier below), the producer
    // lane sets up the barriers itself and, where the first tile's place does not depend on the lengths (in-place
    // cache: the prefix segment holds at least the block's L >= 1 keys and starts at the unit's base), sends for that
    // tile at once; the consumers' Q rows are requested beside it.
    int P = p.prefix_len ? p.prefix_len[b]
                         : (p.uniform_P >= 0 ? p.uniform_P : (p.inplace ? p.prefix_cap - p.L : p.prefix_cap));
    int S = p.has_suffix ? (p.suffix_len ? p.suffix_len[b] : p.suffix_cap) : 0;
    // (only without a K/V split: a CTA of a split launch may own no tile at all, and a tile sent for must be waited for)
    const bool early_tile = p.inplace && p.splits == 1;     // tile 0 of this CTA is tile 0 of the prefix segment
    if (threadIdx.x == NCW * 32) {
        for (int s = 0; s < ATT_STAGES; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], NCW);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_kpre);
        prefetch_tensormap(&tm_vpre);
        if (early_tile) {
            mbar_arrive_expect_tx(&bars->full[0], 2 * KV_BYTES);
#pragma unroll
            for (int h = 0; h < NHALF; ++h) {
                tma_load_2d(tiles + h * HALF, &tm_kpre, &bars->full[0], h * 64, unit * p.prefix_cap);
                tma_load_2d(tiles + KV_BYTES + h * HALF, &tm_vpre, &bars->full[0], h * 64, unit * p.prefix_cap);
            }
        }
    }

    // per-thread state of the consumers (declared here so that the final merge can see it)
    const int rg = warp % NW;              // row group
    const int ks = warp / NW;              // key slice (NW*KS == producer warp: unused there)
    const int quad = lane >> 2;            // row inside the 16-row tile (and +8)
    const int tq = lane & 3;
    const int rho0 = chunk * (NW * 16) + rg * 16 + quad;
    const int rho1 = rho0 + 8;
    const bool live0 = rho0 < p.R, live1 = rho1 < p.R;
    const int i0 = live0 ? rho0 / p.g : 0, h0 = kvh * p.g + (live0 ? rho0 % p.g : 0);
    const int i1 = live1 ? rho1 / p.g : 0, h1 = kvh * p.g + (live1 ? rho1 % p.g : 0);
    uint32_t qf[D / 16][4];
    if (warp < NCW) {
        const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((static_cast<size_t>(b) * p.L + i0) * p.Hq + h0) * D);
        const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + ((static_cast<size_t>(b) * p.L + i1) * p.Hq + h1) * D);
#pragma unroll
        for (int kk = 0; kk < D / 16; ++kk) {
            qf[kk][0] = live0 ? q0[kk * 8 + tq] : 0u;
            qf[kk][1] = live1 ? q1[kk * 8 + tq] : 0u;
            qf[kk][2] = live0 ? q0[kk * 8 + 4 + tq] : 0u;
            qf[kk][3] = live1 ? q1[kk * 8 + 4 + tq] : 0u;
        }
    }
    __syncthreads();

    // lengths (clamped to capacity; a clamp is reported, never trapped on)
    const int p_max = p.inplace ? p.prefix_cap - p.L : p.prefix_cap;
    if (P < 0 || P > p_max || S < 0 || S > p.suffix_cap) {
        P = max(0, min(P, p_max));
        S = max(0, min(S, p.suffix_cap));
        if (threadIdx.x == 0) atomicOr(p.dev_status, DEV_LEN_CLAMPED);
    }
    const int len_pre = p.inplace ? P + p.L : P;
    const int len_blk = p.inplace ? 0 : p.L;
    const int n_pre = (len_pre + KT - 1) / KT;
    const int n_blk = (len_blk + KT - 1) / KT;
    const int n_suf = (S + KT - 1) / KT;
    const int n_tiles = n_pre + n_blk + n_suf;
    const int t_begin = static_cast<int>(static_cast<long long>(n_tiles) * split / p.splits);
    const int t_end = static_cast<int>(static_cast<long long>(n_tiles) * (split + 1) / p.splits);
    const int base_pre = unit * p.prefix_cap;
    const int base_blk = unit * p.L;
    const int base_suf = unit * p.suffix_cap;

    float oacc[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) { oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    bool ok = true;

    if (warp == NCW) {
        // ---------------- producer
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int t = t_begin;
            if (early_tile) {                         // tile 0 is on its way already (no split: t_begin = 0, t_end = n_tiles >= 1)
                ++t;
                if (++stage == ATT_STAGES) { stage = 0; phase ^= 1; }
            }
            for (; t < t_end; ++t) {
                const TileInfo ti = tile_info<KT>(t, n_pre, n_blk, len_pre, len_blk, S, base_pre, base_blk, base_suf);
                const CUtensorMap* mk = ti.seg == 0 ? &tm_kpre : (ti.seg == 1 ? &tm_kblk : &tm_ksuf);
                const CUtensorMap* mv = ti.seg == 0 ? &tm_vpre : (ti.seg == 1 ? &tm_vblk : &tm_vsuf);
                if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) break;
                uint8_t* kdst = tiles + stage * STAGE;
                uint8_t* vdst = kdst + KV_BYTES;
                mbar_arrive_expect_tx(&bars->full[stage], 2 * KV_BYTES);
#pragma unroll
                for (int h = 0; h < NHALF; ++h) {
                    tma_load_2d(kdst + h * HALF, mk, &bars->full[stage], h * 64, ti.row0);
                    tma_load_2d(vdst + h * HALF, mv, &bars->full[stage], h * 64, ti.row0);
                }
                if (++stage == ATT_STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else {
        // ---------------- consumers
        int stage = 0;
        uint32_t phase = 0;
        const int mi = lane >> 3, rin = lane & 7;
        const int koff = ks * KPW;           // this warp's keys inside a tile: [koff, koff + KPW)
        for (int t = t_begin; t < t_end; ++t) {
            const TileInfo ti = tile_info<KT>(t, n_pre, n_blk, len_pre, len_blk, S, base_pre, base_blk, base_suf);
            if (!mbar_wait(&bars->full[stage], phase, abort_flag)) { ok = false; break; }
            uint8_t* kt = tiles + stage * STAGE;
            uint8_t* vt = kt + KV_BYTES;
            const uint32_t kbase = smem_u32(kt), vbase = smem_u32(vt);

            if (ti.valid < koff + KPW && ti.valid > koff) {
                // rows past the segment's end hold whatever lies behind it in memory: zero this warp's V rows
                // there so that probability 0 times garbage cannot make a NaN (rows are contiguous in a half)
                const int first = ti.valid * 128, count = (koff + KPW - ti.valid) * 128;
#pragma unroll
                for (int h = 0; h < NHALF; ++h)
                    for (int o = lane * 16; o < count; o += 32 * 16)
                        *reinterpret_cast<uint4*>(vt + h * HALF + first + o) = make_uint4(0, 0, 0, 0);
                fence_proxy_async_smem();
                __syncwarp();
            }
            if (ti.valid > koff) {   // (a warp whose key slice lies wholly past the end has nothing to add)
                // S = Q K^T for this warp's keys
                float sacc[KPW / 8][4];
#pragma unroll
                for (int nb = 0; nb < KPW / 8; ++nb) {
                    sacc[nb][0] = sacc[nb][1] = sacc[nb][2] = sacc[nb][3] = 0.f;
                    const int key = koff + nb * 8 + rin;
#pragma unroll
                    for (int kq = 0; kq < D / 32; ++kq) {
                        const int ch = 4 * kq + mi;
                        const uint32_t addr = kbase + (ch >> 3) * HALF + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                        uint32_t r0, r1, r2, r3;
                        ldmatrix_x4(addr, r0, r1, r2, r3);
                        mma_bf16_16816(sacc[nb], qf[2 * kq], r0, r1);
                        mma_bf16_16816(sacc[nb], qf[2 * kq + 1], r2, r3);
                    }
                }
                // mask keys that do not exist (only a segment's last tile has any), row max.  The scores stay
                // unscaled: the softmax scale (times log2 e) goes into the exponent's multiply-add below, and
                // the running max m0 / m1 is kept in score units until the tiles are done.
                if (ti.valid < koff + KPW) {
#pragma unroll
                    for (int nb = 0; nb < KPW / 8; ++nb) {
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (koff + nb * 8 + tq * 2 + (e & 1) >= ti.valid) sacc[nb][e] = -INFINITY;
                    }
                }
                float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
                for (int nb = 0; nb < KPW / 8; ++nb) {
                    tmax0 = fmaxf(tmax0, fmaxf(sacc[nb][0], sacc[nb][1]));
                    tmax1 = fmaxf(tmax1, fmaxf(sacc[nb][2], sacc[nb][3]));
                }
                tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 1));
                tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 2));
                tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 1));
                tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 2));
                const float mn0 = fmaxf(m0, tmax0), mn1 = fmaxf(m1, tmax1);   // finite: the slice has >= 1 key
                const bool moved = __any_sync(0xffffffffu, mn0 != m0 || mn1 != m1);
                const float c = p.scale_log2;
                const float nb0 = -mn0 * c, nb1 = -mn1 * c;
                float ps0 = 0.f, ps1 = 0.f;
                uint32_t pa[KPW / 16][4];
#pragma unroll
                for (int nb = 0; nb < KPW / 8; ++nb) {
                    const float e0 = fast_exp2(fmaf(sacc[nb][0], c, nb0)), e1 = fast_exp2(fmaf(sacc[nb][1], c, nb0));
                    const float e2 = fast_exp2(fmaf(sacc[nb][2], c, nb1)), e3 = fast_exp2(fmaf(sacc[nb][3], c, nb1));
                    ps0 += e0 + e1;
                    ps1 += e2 + e3;
                    pa[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(e0, e1);
                    pa[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(e2, e3);
                }
                if (moved) {   // (rare after the first tiles: a row's max over hundreds of keys settles early)
                    const float a0 = fast_exp2((m0 - mn0) * c), a1 = fast_exp2((m1 - mn1) * c);
                    m0 = mn0; m1 = mn1;
                    l0 *= a0;
                    l1 *= a1;
#pragma unroll
                    for (int n = 0; n < D / 8; ++n) {
                        oacc[n][0] *= a0; oacc[n][1] *= a0;
                        oacc[n][2] *= a1; oacc[n][3] *= a1;
                    }
                }
                l0 += ps0;
                l1 += ps1;
                // O += P V
#pragma unroll
                for (int kk = 0; kk < KPW / 16; ++kk) {
                    const int key = koff + kk * 16 + (mi & 1) * 8 + rin;
#pragma unroll
                    for (int nbp = 0; nbp < D / 16; ++nbp) {
                        const int ch = 2 * nbp + (mi >> 1);
                        const uint32_t addr = vbase + (ch >> 3) * HALF + key * 128 + (((ch & 7) ^ (key & 7)) << 4);
                        uint32_t r0, r1, r2, r3;
                        ldmatrix_x4_trans(addr, r0, r1, r2, r3);
                        mma_bf16_16816(oacc[2 * nbp], pa[kk], r0, r1);
                        mma_bf16_16816(oacc[2 * nbp + 1], pa[kk], r2, r3);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->empty[stage]);
            if (++stage == ATT_STAGES) { stage = 0; phase ^= 1; }
        }
        l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
        l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
        l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
        m0 *= p.scale_log2;      // from here on the max is in the log2 domain (-inf stays -inf: the scale is > 0)
        m1 *= p.scale_log2;
    }

    // ---------------- merge the key slices of a row group (through the now idle tile ring), then write out
    __syncthreads();   // every tile has been consumed (or the CTA is aborting): the ring may be reused
    const bool aborted = *abort_flag != 0;
    float* xch = reinterpret_cast<float*>(tiles);
    if (KS > 1 && !aborted && warp < NCW && ks > 0) {
        float* dst = xch + static_cast<size_t>((ks - 1) * NW + rg) * NREG * 32 + lane;
#pragma unroll
        for (int n = 0; n < D / 8; ++n) {
#pragma unroll
            for (int e = 0; e < 4; ++e) dst[(n * 4 + e) * 32] = oacc[n][e];
        }
        dst[(NREG - 4) * 32] = m0; dst[(NREG - 3) * 32] = m1; dst[(NREG - 2) * 32] = l0; dst[(NREG - 1) * 32] = l1;
    }
    if (KS > 1) __syncthreads();
    if (!aborted && warp < NCW && ks == 0) {
#pragma unroll
        for (int o = 1; o < KS; ++o) {
            const float* src = xch + static_cast<size_t>((o - 1) * NW + rg) * NREG * 32 + lane;
            const float om0 = src[(NREG - 4) * 32], om1 = src[(NREG - 3) * 32];
            const float ol0 = src[(NREG - 2) * 32], ol1 = src[(NREG - 1) * 32];
            const float mn0 = fmaxf(m0, om0), mn1 = fmaxf(m1, om1);
            const float sa0 = mn0 == -INFINITY ? 0.f : fast_exp2(m0 - mn0), sb0 = mn0 == -INFINITY ? 0.f : fast_exp2(om0 - mn0);
            const float sa1 = mn1 == -INFINITY ? 0.f : fast_exp2(m1 - mn1), sb1 = mn1 == -INFINITY ? 0.f : fast_exp2(om1 - mn1);
            l0 = l0 * sa0 + ol0 * sb0;
            l1 = l1 * sa1 + ol1 * sb1;
            m0 = mn0; m1 = mn1;
#pragma unroll
            for (int n = 0; n < D / 8; ++n) {
                oacc[n][0] = oacc[n][0] * sa0 + src[(n * 4 + 0) * 32] * sb0;
                oacc[n][1] = oacc[n][1] * sa0 + src[(n * 4 + 1) * 32] * sb0;
                oacc[n][2] = oacc[n][2] * sa1 + src[(n * 4 + 2) * 32] * sb1;
                oacc[n][3] = oacc[n][3] * sa1 + src[(n * 4 + 3) * 32] * sb1;
            }
        }
        const float inv0 = l0 > 0.f ? 1.f / l0 : 0.f, inv1 = l1 > 0.f ? 1.f / l1 : 0.f;
        const float lse0 = l0 > 0.f ? (m0 + log2f(l0)) * LN2_F : -INFINITY;
        const float lse1 = l1 > 0.f ? (m1 + log2f(l1)) * LN2_F : -INFINITY;
        const size_t orow0 = (static_cast<size_t>(b) * p.L + i0) * p.Hq + h0;
        const size_t orow1 = (static_cast<size_t>(b) * p.L + i1) * p.Hq + h1;
        if (p.splits == 1) {
#pragma unroll
            for (int n = 0; n < D / 8; ++n) {
                const int col = n * 8 + tq * 2;
                if (live0)
                    *reinterpret_cast<uint32_t*>(p.out + orow0 * D + col) = pack_bf16(oacc[n][0] * inv0, oacc[n][1] * inv0);
                if (live1)
                    *reinterpret_cast<uint32_t*>(p.out + orow1 * D + col) = pack_bf16(oacc[n][2] * inv1, oacc[n][3] * inv1);
            }
            if (p.lse != nullptr && tq == 0) {
                if (live0) p.lse[(static_cast<size_t>(b) * p.Hq + h0) * p.L + i0] = lse0;
                if (live1) p.lse[(static_cast<size_t>(b) * p.Hq + h1) * p.L + i1] = lse1;
            }
        } else {
            const size_t n_rows = static_cast<size_t>(p.B) * p.L * p.Hq;
            float* po = p.part_o + static_cast<size_t>(split) * n_rows * D;
            float* pl = p.part_lse + static_cast<size_t>(split) * n_rows;
#pragma unroll
            for (int n = 0; n < D / 8; ++n) {
                const int col = n * 8 + tq * 2;
                if (live0) *reinterpret_cast<float2*>(po + orow0 * D + col) = make_float2(oacc[n][0] * inv0, oacc[n][1] * inv0);
                if (live1) *reinterpret_cast<float2*>(po + orow1 * D + col) = make_float2(oacc[n][2] * inv1, oacc[n][3] * inv1);
            }
            if (tq == 0) {
                if (live0) pl[orow0] = lse0;
                if (live1) pl[orow1] = lse1;
            }
        }
    }
    (void)ok;
    if (aborted) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
        if (threadIdx.x == 0) atomicOr(p.dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
}

// ---------------------------------------------------------------------------------------------------------
// tcgen05 path: used when the query rows that share a KV head fill 128-row tensor-core tiles well (GQA
// groups, long blocks such as the prefill).  One CTA per (one or two tiles of packed query rows, rollout x
// KV head); the two query tiles share every K/V tile:
//   warp 0        TMA producer: 128-key K and V tiles through a shared-memory ring (as above)
//   warp 1        UMMA issuer (one thread, so that the order of its MMAs is the order they run in):
//                 S = Q K^T (128 x 128, K-major operands from shared memory) into tensor memory, then
//                 O += P V (128 x D) with P, the A operand, read from TENSOR memory and V, the MN-major B operand,
//                 straight from the TMA tile; O stays in tensor memory over the whole key range
//   warps 2..5    softmax of query tile 0 (warps 6..9: tile 1): one TMEM lane = one query row per thread;
//                 reads S twice (tile max, then exponentials), keeps the row's reference max and sum, and writes
//                 P as packed bf16 over the columns S came from: P never touches shared memory
// An MMA whose A operand sits in shared memory costs ~80 to 120 cycles whatever its N (the 128 x 16 A slab is
// read at ~32 bytes per cycle); with P in tensor memory the second product runs at its N / 2 cycles, and with
// 128-key tiles the first product's MMAs have N = 128 instead of 64: per 64 keys and query tile ~740 cycles of
// tensor pipe instead of ~1120.
// With two query tiles each has ONE S/P buffer and the issuer interleaves them: while the softmax warps of one
// tile work, the pipe runs the other tile's products (S_a(t), S_b(t), then per tile P V(t) and S(t + 1), which may
// overwrite P(t) because the pipe runs the issuer's MMAs in order).  With one query tile there are two S/P buffers.
// O stays in TMEM, so it cannot be rescaled for free when a row's max grows.  The exponentials are therefore
// taken relative to a reference max that is only moved when the true max has run more than 2^8 ahead of it;
// then (rarely, mostly in the first tiles) the warp waits for the MMAs in flight, multiplies its rows of O by
// the correction factor in place and moves the reference.  The sum uses the same reference, so O / l is exact.
// A tile holds floor(128 / g) block positions x g heads so that a position's heads never straddle two tiles.
constexpr int TC_KT = 128;                // keys per tile
constexpr float TC_RESCALE_GAP = 8.0f;    // log2 units the true max may run ahead of the reference

template <int D, int QT>
struct TcShape {
    static constexpr int Q_BYTES = 128 * D * 2;                        // per query tile
    static constexpr int KV_STAGE = 2 * TC_KT * D * 2;                 // K tile + V tile
    static constexpr int NBUF = QT == 2 ? 1 : 2;                       // S / P buffers per query tile
    static constexpr int FIXED = QT * Q_BYTES;
    static constexpr int FIT = (226 * 1024 - 2048 - FIXED) / KV_STAGE;
    static constexpr int STAGES = FIT > 4 ? 4 : FIT;
    static constexpr int SMEM = FIXED + STAGES * KV_STAGE + 1024 + 512;
    static constexpr int THREADS = (2 + 4 * QT) * 32;                  // TMA warp, MMA warp, softmax warps
    static constexpr uint32_t TMEM_COLS = 512;
    // tensor-memory columns: two query tiles: tile j has S/P at j * 256 and O at j * 256 + 128;
    // one query tile: S/P buffers at 0 and 128, O at 256
    __host__ __device__ static constexpr uint32_t s_col(int j, int b) { return QT == 2 ? j * 256 : b * 128; }
    __host__ __device__ static constexpr uint32_t o_col(int j) { return QT == 2 ? j * 256 + 128 : 256; }
    static_assert(STAGES >= NBUF + 1, "K/V ring too small");
};

template <int STAGES, int QT>
struct TcBarriers {
    uint64_t full[STAGES];
    uint64_t empty[STAGES];
    uint64_t q_ready;
    uint64_t s_full[QT][2], p_full[QT][2], pv_done[QT][2];     // indexed by the key tile's parity
    uint32_t tmem_base;
    uint32_t abort_flag;
};

template <int D, int QT>
__global__ void __launch_bounds__(TcShape<D, QT>::THREADS, 1)
attn_block_tc_kernel(const __grid_constant__ CUtensorMap tm_kpre, const __grid_constant__ CUtensorMap tm_vpre,
                     const __grid_constant__ CUtensorMap tm_kblk, const __grid_constant__ CUtensorMap tm_vblk,
                     const __grid_constant__ CUtensorMap tm_ksuf, const __grid_constant__ CUtensorMap tm_vsuf,
                     const AttnParams p) {
    using S = TcShape<D, QT>;
    constexpr int STAGES = S::STAGES;
    constexpr int NBUF = S::NBUF;
    constexpr int NHALF = D / 64;
    constexpr int HALF_K = TC_KT * 128;            // one 64-column half of a K or V tile: 128 rows x 128 bytes
    constexpr int KV_BYTES = TC_KT * D * 2;
    constexpr int HALF_Q = 128 * 128;              // one 64-column half of a Q tile: 128 rows x 128 bytes

    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* q_s = base;                                   // [QT][Q_BYTES]
    uint8_t* kv_s = q_s + QT * S::Q_BYTES;                 // [STAGES][KV_STAGE]
    TcBarriers<STAGES, QT>* bars = reinterpret_cast<TcBarriers<STAGES, QT>*>(kv_s + STAGES * S::KV_STAGE);
    volatile uint32_t* abort_flag = &bars->abort_flag;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int unit = blockIdx.y;
    const int b = unit / p.Hkv;
    const int kvh = unit % p.Hkv;
    const int pos_per_tile = 128 / p.g;            // block positions per query tile
    // Packed variable-length mode: "rollout" b is sequence b of the packed token list; its tokens are both the
    // queries (a block of L_eff positions, no prefix) and, in place, the keys.  K and V are [tokens, Hkv * D].
    const bool packed = p.cu_seqlens != nullptr;
    const int seq_base = packed ? p.cu_seqlens[b] : 0;
    const int L_eff = packed ? p.cu_seqlens[b + 1] - seq_base : p.L;
    if (static_cast<int>(blockIdx.x) * QT * pos_per_tile >= L_eff) return;   // (whole CTA, before anything is set up)
    const int kv_col0 = packed ? kvh * D : 0;      // first column of this KV head in the 2-D view of K / V

    // Set-up, with nothing waiting for anything else (a launch is a single wave of CTAs that live for about ten key
    // tiles, so the time to the first product counts): the lengths are requested first; thread 0, which is also the
    // TMA producer, sets up the barriers and sends for key tile 0 at once where its place does not depend on the
    // lengths (packed sequences and the in-place cache: the first segment is not empty and starts at the unit's
    // base); warp 1 allocates tensor memory; the softmax threads stage their Q rows.
    int P = p.prefix_len ? p.prefix_len[b]
                         : (p.uniform_P >= 0 ? p.uniform_P : (p.inplace ? p.prefix_cap - p.L : p.prefix_cap));
    int Sx = p.has_suffix ? (p.suffix_len ? p.suffix_len[b] : p.suffix_cap) : 0;
    const bool early_tile = packed || p.inplace;
    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], 1);                 // released by the issuer once both query tiles are done with it
        }
        mbar_init(&bars->q_ready, 128 * QT);
        for (int j = 0; j < QT; ++j)
            for (int i = 0; i < 2; ++i) {
                mbar_init(&bars->s_full[j][i], 1);
                mbar_init(&bars->p_full[j][i], 128);
                mbar_init(&bars->pv_done[j][i], 1);
            }
        bars->abort_flag = 0;
        fence_barrier_init();
        prefetch_tensormap(&tm_kpre);
        prefetch_tensormap(&tm_vpre);
        if (early_tile) {
            const int row0 = packed ? seq_base : unit * p.prefix_cap;
            mbar_arrive_expect_tx(&bars->full[0], 2 * KV_BYTES);
#pragma unroll
            for (int h = 0; h < NHALF; ++h) {
                tma_load_2d(kv_s + h * HALF_K, &tm_kpre, &bars->full[0], kv_col0 + h * 64, row0);
                tma_load_2d(kv_s + KV_BYTES + h * HALF_K, &tm_vpre, &bars->full[0], kv_col0 + h * 64, row0);
            }
        }
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, S::TMEM_COLS);
        tmem_relinquish();
    }
    if (warp >= 2) {
        // Q rows -> shared memory, K-major with the 128-byte swizzle (16-byte chunk c of row r sits at c ^ (r & 7)).
        // A warp copies the 32 rows whose softmax it runs, coalesced: one instruction reads 32 / CPR whole rows
        // (a lane per 16-byte chunk), so that a request touches 2 to 4 cache lines, not one per lane.
        constexpr int CPR = D / 8;                     // 16-byte chunks per row
        const int j = (warp - 2) >> 2;
        const int c = lane % CPR;
        const size_t q_token = packed ? static_cast<size_t>(seq_base) : static_cast<size_t>(b) * p.L;
        uint8_t* qt = q_s + j * S::Q_BYTES;
        uint4 v[CPR];
#pragma unroll
        for (int k = 0; k < CPR; ++k) {
            const int r = (warp & 3) * 32 + k * (32 / CPR) + lane / CPR;
            const int i = (blockIdx.x * QT + j) * pos_per_tile + r / p.g;
            const int h = kvh * p.g + r % p.g;
            const bool live = r < pos_per_tile * p.g && i < L_eff;
            v[k] = live ? reinterpret_cast<const uint4*>(p.q + ((q_token + i) * p.Hq + h) * D)[c] : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < CPR; ++k) {
            const int r = (warp & 3) * 32 + k * (32 / CPR) + lane / CPR;
            *reinterpret_cast<uint4*>(qt + (c >> 3) * HALF_Q + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = v[k];
        }
        fence_proxy_async_smem();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = bars->tmem_base;

    // lengths and tiles of this unit (same bookkeeping as the warp-level kernel)
    const int p_max = p.inplace ? p.prefix_cap - p.L : p.prefix_cap;
    if (!packed && (P < 0 || P > p_max || Sx < 0 || Sx > p.suffix_cap)) {
        P = max(0, min(P, p_max));
        Sx = max(0, min(Sx, p.suffix_cap));
        if (threadIdx.x == 0) atomicOr(p.dev_status, DEV_LEN_CLAMPED);
    }
    const int len_pre = packed ? L_eff : (p.inplace ? P + p.L : P);
    const int len_blk = (packed || p.inplace) ? 0 : p.L;
    const int n_pre = (len_pre + TC_KT - 1) / TC_KT;
    const int n_blk = (len_blk + TC_KT - 1) / TC_KT;
    const int n_suf = (Sx + TC_KT - 1) / TC_KT;
    const int n_tiles = n_pre + n_blk + n_suf;
    const int base_pre = packed ? seq_base : unit * p.prefix_cap;
    const int base_blk = unit * p.L;
    const int base_suf = unit * p.suffix_cap;

    if (warp == 0) {
        if (lane == 0) {
            int stage = 0;
            uint32_t phase = 0;
            int t = 0;
            if (early_tile) {                               // key tile 0 is on its way already (n_tiles >= 1 here)
                ++t;
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            for (; t < n_tiles; ++t) {
                const TileInfo ti = tile_info<TC_KT>(t, n_pre, n_blk, len_pre, len_blk, Sx, base_pre, base_blk, base_suf);
                const CUtensorMap* mk = ti.seg == 0 ? &tm_kpre : (ti.seg == 1 ? &tm_kblk : &tm_ksuf);
                const CUtensorMap* mv = ti.seg == 0 ? &tm_vpre : (ti.seg == 1 ? &tm_vblk : &tm_vsuf);
                if (!mbar_wait(&bars->empty[stage], phase ^ 1, abort_flag)) break;
                uint8_t* kdst = kv_s + stage * S::KV_STAGE;
                uint8_t* vdst = kdst + KV_BYTES;
                mbar_arrive_expect_tx(&bars->full[stage], 2 * KV_BYTES);
#pragma unroll
                for (int h = 0; h < NHALF; ++h) {
                    tma_load_2d(kdst + h * HALF_K, mk, &bars->full[stage], kv_col0 + h * 64, ti.row0);
                    tma_load_2d(vdst + h * HALF_K, mv, &bars->full[stage], kv_col0 + h * 64, ti.row0);
                }
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    } else if (warp == 1) {
        // All 32 lanes run the loops (waits, counters and descriptors stay warp-uniform, in the registers the MMA
        // instruction takes its operands from); one elected lane issues the MMAs and their commits.
        const bool leader = elect_one_sync();
        constexpr uint32_t idesc_s = umma_idesc_bf16(128, TC_KT);
        constexpr uint32_t idesc_o = umma_idesc_bf16(128, D) | UMMA_B_MN_MAJOR;
        // descriptor lower words (address >> 4 [| leading byte offset]); the upper word is a constant
        const uint32_t q_lo = smem_u32(q_s) >> 4, kv_lo = smem_u32(kv_s) >> 4;
        const uint32_t v_lbo = static_cast<uint32_t>(HALF_K >> 4) << 16;   // second 64 head-dim columns: one half tile on
        bool ok = __all_sync(0xffffffffu, mbar_wait(&bars->q_ready, 0, abort_flag));
        // S_j(t) = Q_j K_t^T into tile j's buffer t % NBUF (whatever that buffer held has been consumed: the P V
        // product that read it was issued before this, and the pipe keeps the issue order)
        auto issue_s = [&](int j, int t) -> bool {
            const int stage = t % STAGES;
            if (!__all_sync(0xffffffffu, mbar_wait(&bars->full[stage], (t / STAGES) & 1, abort_flag))) return false;
            tc_fence_after_sync();
            const uint32_t k_lo = kv_lo + stage * (S::KV_STAGE >> 4), qj = q_lo + j * (S::Q_BYTES >> 4);
            const uint32_t sd = tmem_base + S::s_col(j, t % NBUF);
            if (leader) {
                umma_bf16_lo<false>(sd, qj, k_lo, idesc_s);
#pragma unroll
                for (int kk = 1; kk < D / 16; ++kk)     // 16 channels = 32 bytes along the swizzled row: +2
                    umma_bf16_lo<true>(sd, qj + (kk >> 2) * (HALF_Q >> 4) + 2 * (kk & 3),
                                       k_lo + (kk >> 2) * (HALF_K >> 4) + 2 * (kk & 3), idesc_s);
                umma_commit(&bars->s_full[j][t & 1]);
            }
            __syncwarp();
            return true;
        };
        for (int t = 0; t < NBUF && t < n_tiles && ok; ++t)
            for (int j = 0; j < QT && ok; ++j) ok = issue_s(j, t);
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int stage = t % STAGES;
            const uint32_t v_lo = (kv_lo + stage * (S::KV_STAGE >> 4) + (KV_BYTES >> 4)) | v_lbo;
            for (int j = 0; j < QT && ok; ++j) {
                if (!__all_sync(0xffffffffu, mbar_wait(&bars->p_full[j][t & 1], (t >> 1) & 1, abort_flag))) { ok = false; break; }
                tc_fence_after_sync();
                // A: P in tensor memory, 16 keys = 8 columns per MMA; B: 16 key rows (2 KB) further down V
                const uint32_t pa = tmem_base + S::s_col(j, t % NBUF), od = tmem_base + S::o_col(j);
                if (leader) {
                    if (t == 0) umma_bf16_ts_lo<false>(od, pa, v_lo, idesc_o);
                    else umma_bf16_ts_lo<true>(od, pa, v_lo, idesc_o);
#pragma unroll
                    for (int kk = 1; kk < TC_KT / 16; ++kk)
                        umma_bf16_ts_lo<true>(od, pa + 8 * kk, v_lo + kk * (2048 >> 4), idesc_o);
                    umma_commit(&bars->pv_done[j][t & 1]);     // O holds tiles 0..t
                }
                __syncwarp();
                if (t + NBUF < n_tiles) ok = issue_s(j, t + NBUF);
            }
            if (ok && leader) umma_commit(&bars->empty[stage]);      // every product that reads this K/V tile has been issued
            __syncwarp();
        }
    } else {
        // ---------------- softmax warps: set j = query tile, thread = packed query row r of that tile = TMEM lane r
        const int j = (warp - 2) >> 2;
        const int r = (warp & 3) * 32 + lane;          // warp w may touch TMEM lanes [32 * (w % 4), +32)
        const int rows_in_tile = pos_per_tile * p.g;
        const int i = (blockIdx.x * QT + j) * pos_per_tile + r / p.g;   // block position
        const int h = kvh * p.g + r % p.g;                              // query head
        const bool live = r < rows_in_tile && i < L_eff;
        const size_t q_token = packed ? static_cast<size_t>(seq_base) : static_cast<size_t>(b) * p.L;   // first token of b
        mbar_arrive(&bars->q_ready);                   // (the warp's Q rows were staged before the barrier above)
        float m_ref = -INFINITY, l = 0.f;              // reference max (log2 domain) and sum of exp2(s - m_ref)
        const uint32_t lane_off = static_cast<uint32_t>((warp & 3) * 32) << 16;
        const uint32_t tm_o = tmem_base + S::o_col(j) + lane_off;
        const float c2 = p.scale_log2;
        bool ok = true;
        for (int t = 0; t < n_tiles; ++t) {
            const TileInfo ti = tile_info<TC_KT>(t, n_pre, n_blk, len_pre, len_blk, Sx, base_pre, base_blk, base_suf);
            const int buf = t & 1, stage = t % STAGES;
            if (!mbar_wait(&bars->s_full[j][buf], (t >> 1) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after_sync();
            const uint32_t tm_s = tmem_base + S::s_col(j, t % NBUF) + lane_off;
            // first pass over S: the tile's largest score (keys past the segment's end do not count).  The load of
            // the next 32 columns is in flight while the current ones are looked at.  (A single pass that keeps P in
            // registers until the reference is known to hold was measured no faster: 37.2 against 35.4 us.)
            float tmax = -INFINITY;
            {
                uint32_t sa[32], sb[32];
                tmem_ld_32cols(tm_s, sa);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < TC_KT / 32; ++c) {
                    uint32_t (&cur)[32] = (c & 1) ? sb : sa;
                    uint32_t (&nxt)[32] = (c & 1) ? sa : sb;
                    if (c + 1 < TC_KT / 32) tmem_ld_32cols(tm_s + (c + 1) * 32, nxt);
                    if (ti.valid >= (c + 1) * 32) {
#pragma unroll
                        for (int k = 0; k < 32; ++k) tmax = fmaxf(tmax, __uint_as_float(cur[k]));
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            if (c * 32 + k < ti.valid) tmax = fmaxf(tmax, __uint_as_float(cur[k]));
                    }
                    if (c + 1 < TC_KT / 32) tmem_ld_wait();
                }
            }
            tmax *= c2;                                 // log2 domain (the scale is > 0); finite: every tile has a key
            // move the reference only when the true max has run away from it (decided per warp, so that the
            // TMEM loads and stores below are executed by whole warps)
            const bool move = __any_sync(0xffffffffu, tmax > m_ref + TC_RESCALE_GAP);
            if (move) {
                const float m_new = fmaxf(m_ref, tmax);
                const float factor = fast_exp2(m_ref - m_new);   // exp2(-inf) = 0 on the first tile
                m_ref = m_new;
                l *= factor;
                if (t >= 1) {
                    // every MMA that adds to O must have landed before O is rescaled in place: tile t - 1 is the last
                    if (!mbar_wait(&bars->pv_done[j][(t - 1) & 1], ((t - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after_sync();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t ov[32];
                        tmem_ld_32cols(tm_o + c * 32, ov);
                        tmem_ld_wait();
#pragma unroll
                        for (int k = 0; k < 32; ++k) ov[k] = __float_as_uint(__uint_as_float(ov[k]) * factor);
                        tmem_st_32cols(tm_o + c * 32, ov);
                    }
                }
            }
            // second pass: P = exp2(s - m_ref) as packed bf16 over the columns S came from.  The 16 columns written
            // for keys [32 c, 32 c + 32) lie below column 16 c + 16, which this pass has already read.
            const float nm = -m_ref;
            float psum = 0.f;
            {
                uint32_t sa[32], sb[32];
                tmem_ld_32cols(tm_s, sa);
                tmem_ld_wait();
#pragma unroll
                for (int c = 0; c < TC_KT / 32; ++c) {
                    uint32_t (&cur)[32] = (c & 1) ? sb : sa;
                    uint32_t (&nxt)[32] = (c & 1) ? sa : sb;
                    if (c + 1 < TC_KT / 32) tmem_ld_32cols(tm_s + (c + 1) * 32, nxt);
                    uint32_t pk[16];
                    if (ti.valid >= (c + 1) * 32) {
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            const float e0 = fast_exp2(fmaf(__uint_as_float(cur[k]), c2, nm));
                            const float e1 = fast_exp2(fmaf(__uint_as_float(cur[k + 1]), c2, nm));
                            psum += e0 + e1;
                            pk[k >> 1] = pack_bf16(e0, e1);
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; k += 2) {
                            float e0 = fast_exp2(fmaf(__uint_as_float(cur[k]), c2, nm));
                            float e1 = fast_exp2(fmaf(__uint_as_float(cur[k + 1]), c2, nm));
                            if (c * 32 + k >= ti.valid) e0 = 0.f;
                            if (c * 32 + k + 1 >= ti.valid) e1 = 0.f;
                            psum += e0 + e1;
                            pk[k >> 1] = pack_bf16(e0, e1);
                        }
                    }
                    if (c + 1 < TC_KT / 32) tmem_ld_wait();      // (the next columns, [32 c + 32, +32), lie above the store below)
                    tmem_st_16cols(tm_s + c * 16, pk);
                }
            }
            tmem_st_wait();
            l += psum;
            if (ti.valid < TC_KT) {
                // V rows past the segment's end hold whatever lies behind it in memory: zero them so that
                // probability 0 times garbage cannot make a NaN (thread r clears 16-byte pieces of those rows;
                // both query tiles' warps do it, each before it releases its own second MMA)
                uint8_t* vt = kv_s + stage * S::KV_STAGE + KV_BYTES;
                const int n_bad = (TC_KT - ti.valid) * 8;       // 16-byte pieces per 64-column half
                for (int h2 = 0; h2 < NHALF; ++h2)
                    for (int q = r; q < n_bad; q += 128)
                        *reinterpret_cast<uint4*>(vt + h2 * HALF_K + ti.valid * 128 + q * 16) = make_uint4(0, 0, 0, 0);
                fence_proxy_async_smem();
            }
            tc_fence_before_sync();
            mbar_arrive(&bars->p_full[j][buf]);
        }
        if (ok && n_tiles > 0) ok = mbar_wait(&bars->pv_done[j][(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, abort_flag);
        tc_fence_after_sync();
        const float inv = l > 0.f ? 1.f / l : 0.f;
        // O rows leave through shared memory so that the global stores are coalesced (a thread holds one whole row,
        // and 32 lanes storing 16 bytes each to 32 different rows cost a request per lane).  The tile's Q rows are
        // no longer read (every S product has completed: the pipe runs the issuer's MMAs in order and the last P V
        // has landed), so each warp turns its 32 rows in the place its Q rows had, in the same swizzled layout.
        uint8_t* ot = q_s + j * S::Q_BYTES;
#pragma unroll
        for (int c2 = 0; c2 < D / 64; ++c2) {
            uint32_t oa[32], ob[32];
            tmem_ld_32cols(tm_o + c2 * 64, oa);          // (whole warp, also for rows that are not stored)
            tmem_ld_32cols(tm_o + c2 * 64 + 32, ob);
            tmem_ld_wait();
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const uint32_t (&ov)[32] = k < 4 ? oa : ob;
                const int k8 = (k & 3) * 8, cc = c2 * 8 + k;
                uint4 o;
                o.x = pack_bf16(__uint_as_float(ov[k8 + 0]) * inv, __uint_as_float(ov[k8 + 1]) * inv);
                o.y = pack_bf16(__uint_as_float(ov[k8 + 2]) * inv, __uint_as_float(ov[k8 + 3]) * inv);
                o.z = pack_bf16(__uint_as_float(ov[k8 + 4]) * inv, __uint_as_float(ov[k8 + 5]) * inv);
                o.w = pack_bf16(__uint_as_float(ov[k8 + 6]) * inv, __uint_as_float(ov[k8 + 7]) * inv);
                *reinterpret_cast<uint4*>(ot + (cc >> 3) * HALF_Q + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) = o;
            }
        }
        __syncwarp();
        {
            constexpr int CPR = D / 8;
            const int c = lane % CPR;
#pragma unroll
            for (int k = 0; k < CPR; ++k) {
                const int r2 = (warp & 3) * 32 + k * (32 / CPR) + lane / CPR;
                const int i2 = (blockIdx.x * QT + j) * pos_per_tile + r2 / p.g;
                const int h2 = kvh * p.g + r2 % p.g;
                if (ok && r2 < rows_in_tile && i2 < L_eff)
                    reinterpret_cast<uint4*>(p.out + ((q_token + i2) * p.Hq + h2) * D)[c] =
                        *reinterpret_cast<const uint4*>(ot + (c >> 3) * HALF_Q + r2 * 128 + (((c & 7) ^ (r2 & 7)) << 4));
            }
        }
        if (ok && live && p.lse != nullptr)
            p.lse[packed ? static_cast<size_t>(h) * p.total_tokens + seq_base + i
                         : (static_cast<size_t>(b) * p.Hq + h) * p.L + i] = l > 0.f ? (m_ref + log2f(l)) * LN2_F : -INFINITY;
    }

    // teardown
    tc_fence_before_sync();
    __syncthreads();
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
        if (threadIdx.x == 0) atomicOr(p.dev_status, DEV_WAIT_EXPIRED);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, S::TMEM_COLS);
    }
}

template <int D, int QT>
int launch_tc(const CUtensorMap* tm, const AttnParams& p, int q_tiles, cudaStream_t stream) {
    constexpr int SMEM = TcShape<D, QT>::SMEM;
    static std::atomic<uint64_t> smem_set{0};
    if (ensure_dynamic_smem(smem_set, attn_block_tc_kernel<D, QT>, SMEM) != DARE_OK) return DARE_ERR_CUDA;
    dim3 grid((q_tiles + QT - 1) / QT, p.B * p.Hkv, 1);
    attn_block_tc_kernel<D, QT><<<grid, TcShape<D, QT>::THREADS, SMEM, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], p); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

// The tensor-core tile is worth it when a tile's 128 rows are mostly real query rows.
bool use_tc_path(const AttnArgs& a) {
    const int g = a.Hq / a.Hkv;
    if (g > 128) return false;
    const int pos_per_tile = 128 / g;
    const int rows = (a.L < pos_per_tile ? a.L : pos_per_tile) * g;
    return rows >= 96;
}

// Combine KV-split partials: out = sum_s w_s o_s / sum_s w_s with w_s = exp(lse_s - max lse).
template <int D>
__global__ void attn_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse, int splits,
                                    size_t n_rows, int L, int Hq, __nv_bfloat16* __restrict__ out,
                                    float* __restrict__ lse) {
    const size_t row = static_cast<size_t>(blockIdx.x) * (blockDim.x / (D / 4)) + threadIdx.x / (D / 4);
    const int c4 = threadIdx.x % (D / 4);
    if (row >= n_rows) return;
    float mx = -INFINITY;
    for (int s = 0; s < splits; ++s) mx = fmaxf(mx, part_lse[s * n_rows + row]);
    float wsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s = 0; s < splits; ++s) {
        const float ls = part_lse[s * n_rows + row];
        if (ls == -INFINITY) continue;
        const float w = exp2f((ls - mx) * LOG2E_F);
        const float4 o = *reinterpret_cast<const float4*>(part_o + (s * n_rows + row) * D + c4 * 4);
        acc.x += w * o.x; acc.y += w * o.y; acc.z += w * o.z; acc.w += w * o.w;
        wsum += w;
    }
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(out + row * D + c4 * 4) = packed;
    if (lse != nullptr && c4 == 0) {
        // row = (b * L + i) * Hq + h  ->  lse[b, h, i]
        const size_t h = row % Hq, bi = row / Hq, i = bi % L, bb = bi / L;
        lse[(bb * Hq + h) * L + i] = wsum > 0.f ? mx + logf(wsum) : -INFINITY;
    }
}

template <int D, int NW, int KS, int KT, int STAGES, int CPS>
int launch_one(const CUtensorMap* tm, const AttnParams& p, int chunks, cudaStream_t stream) {
    constexpr int SMEM = att_smem_bytes<D, KT, STAGES>();
    static_assert((KS - 1) * NW * ((D / 8) * 4 + 4) * 32 * 4 <= STAGES * att_stage_bytes<D, KT>(), "merge buffer");
    static_assert(STAGES <= ATT_MAX_STAGES && KT <= KT_MAX && KT % (16 * KS) == 0, "variant");
    static std::atomic<uint64_t> smem_set{0};
    if (ensure_dynamic_smem(smem_set, attn_block_kernel<D, NW, KS, KT, STAGES, CPS>, SMEM) != DARE_OK) return DARE_ERR_CUDA;
    dim3 grid(chunks, p.B * p.Hkv, p.splits);
    attn_block_kernel<D, NW, KS, KT, STAGES, CPS><<<grid, (NW * KS + 1) * 32, SMEM, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], p); note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

// The warp-level kernel's variants by the number of packed query rows R per (rollout, KV head):
//   R <= 16   one row group, four key slices of a 64-key tile, 2 CTAs per SM
//   R <= 32   two row groups, two key slices of a 64-key tile, 2 CTAs per SM (32-key tiles with two warps and
//             4 CTAs per SM were measured slower: 58 against 45 us on 16 rollouts x 32 heads x 768 keys)
//   larger    four row groups per 64-row chunk, 64-key tiles, 2 CTAs per SM
struct WarpVariant { int nw, kt, per_sm; };
WarpVariant pick_variant(int R) {
    if (R <= 16) return {1, 64, 2};
    if (R <= 32) return {2, 64, 2};
    return {4, 64, 2};
}

}  // namespace

int attn_plan_splits(const dare_ctx* ctx, const AttnArgs& a) {
    if (use_tc_path(a)) return 1;
    const int g = a.Hq / a.Hkv;
    const int R = a.L * g;
    const WarpVariant var = pick_variant(R);
    const int nw = var.nw;
    const int chunks = (R + nw * 16 - 1) / (nw * 16);
    const long long units = static_cast<long long>(chunks) * a.B * a.Hkv;
    const long long slots = static_cast<long long>(ctx->sm_count) * var.per_sm;
    if (units >= slots) return 1;
    const int tiles = (a.prefix_cap + (a.k_blk ? a.L : 0) + a.suffix_cap + var.kt - 1) / var.kt;
    long long s = (slots + units - 1) / units;
    if (s > tiles / 2) s = tiles / 2;
    if (s > 32) s = 32;
    if (s < 1) s = 1;
    return static_cast<int>(s);
}

size_t attn_workspace_bytes(const AttnArgs& a, int splits) {
    if (splits <= 1) return 0;
    const size_t n_rows = static_cast<size_t>(a.B) * a.L * a.Hq;
    return static_cast<size_t>(splits) * n_rows * (a.d + 1) * sizeof(float);
}

int launch_attn(const dare_ctx* ctx, const AttnArgs& a, cudaStream_t stream) {
    AttnParams p;
    p.B = a.B; p.L = a.L; p.Hq = a.Hq; p.Hkv = a.Hkv; p.g = a.Hq / a.Hkv; p.R = a.L * p.g;
    p.prefix_cap = a.prefix_cap; p.suffix_cap = a.k_suf ? a.suffix_cap : 0;
    p.inplace = a.k_blk == nullptr; p.has_suffix = a.k_suf != nullptr && a.suffix_cap > 0;
    p.splits = attn_plan_splits(ctx, a);
    p.uniform_P = a.prefix_len_uniform;
    p.cu_seqlens = nullptr; p.total_tokens = 0;
    const float scale = a.scale != 0.f ? a.scale : 1.0f / sqrtf(static_cast<float>(a.d));
    p.scale_log2 = scale * LOG2E_F;
    p.q = static_cast<const __nv_bfloat16*>(a.q);
    p.prefix_len = a.prefix_len; p.suffix_len = a.suffix_len;
    p.out = static_cast<__nv_bfloat16*>(a.out); p.lse = a.lse;
    p.dev_status = ctx->dev_status;
    const size_t n_rows = static_cast<size_t>(a.B) * a.L * a.Hq;
    p.part_o = static_cast<float*>(ctx->workspace);
    p.part_lse = p.part_o + static_cast<size_t>(p.splits) * n_rows * a.d;

    CUtensorMap tm[6];
    const uint64_t units = static_cast<uint64_t>(a.B) * a.Hkv;
    const uint32_t KT = static_cast<uint32_t>(use_tc_path(a) ? TC_KT : pick_variant(p.R).kt);   // rows of a K/V tile
    int rc = make_tmap_bf16_2d(ctx, &tm[0], a.k_pre, units * a.prefix_cap, a.d, KT, 64);
    if (rc == DARE_OK) rc = make_tmap_bf16_2d(ctx, &tm[1], a.v_pre, units * a.prefix_cap, a.d, KT, 64);
    if (rc != DARE_OK) return rc;
    if (!p.inplace) {
        rc = make_tmap_bf16_2d(ctx, &tm[2], a.k_blk, units * a.L, a.d, KT, 64);
        if (rc == DARE_OK) rc = make_tmap_bf16_2d(ctx, &tm[3], a.v_blk, units * a.L, a.d, KT, 64);
        if (rc != DARE_OK) return rc;
    } else {
        tm[2] = tm[0]; tm[3] = tm[1];
    }
    if (p.has_suffix) {
        rc = make_tmap_bf16_2d(ctx, &tm[4], a.k_suf, units * a.suffix_cap, a.d, KT, 64);
        if (rc == DARE_OK) rc = make_tmap_bf16_2d(ctx, &tm[5], a.v_suf, units * a.suffix_cap, a.d, KT, 64);
        if (rc != DARE_OK) return rc;
    } else {
        tm[4] = tm[0]; tm[5] = tm[1];
    }

    if (use_tc_path(a)) {
        // two query tiles per CTA halve the K/V traffic, but only pay when the CTAs still fill the SMs
        const int pos_per_tile = 128 / p.g;
        const int q_tiles = (p.L + pos_per_tile - 1) / pos_per_tile;
        const long long pairs = static_cast<long long>((q_tiles + 1) / 2) * p.B * p.Hkv;
        if (q_tiles >= 2 && 4 * pairs >= 3LL * ctx->sm_count)
            return a.d == 128 ? launch_tc<128, 2>(tm, p, q_tiles, stream) : launch_tc<64, 2>(tm, p, q_tiles, stream);
        return a.d == 128 ? launch_tc<128, 1>(tm, p, q_tiles, stream) : launch_tc<64, 1>(tm, p, q_tiles, stream);
    }
    const int nw = pick_variant(p.R).nw;
    const int chunks = (p.R + nw * 16 - 1) / (nw * 16);
    if (a.d == 128) {
        rc = nw == 1 ? launch_one<128, 1, 4, 64, 3, 2>(tm, p, chunks, stream)
           : nw == 2 ? launch_one<128, 2, 2, 64, 3, 2>(tm, p, chunks, stream)
                     : launch_one<128, 4, 1, 64, 3, 2>(tm, p, chunks, stream);
    } else {
        rc = nw == 1 ? launch_one<64, 1, 4, 64, 3, 2>(tm, p, chunks, stream)
           : nw == 2 ? launch_one<64, 2, 2, 64, 3, 2>(tm, p, chunks, stream)
                     : launch_one<64, 4, 1, 64, 3, 2>(tm, p, chunks, stream);
    }
    if (rc != DARE_OK) return rc;
    if (p.splits > 1) {
        const int tpr = a.d / 4;                    // threads per row
        const int rows_per_block = 256 / tpr;
        const unsigned blocks = static_cast<unsigned>((n_rows + rows_per_block - 1) / rows_per_block);
        if (a.d == 128)
            attn_combine_kernel<128><<<blocks, 256, 0, stream>>>(p.part_o, p.part_lse, p.splits, n_rows, a.L, a.Hq, p.out, p.lse);
        else
            attn_combine_kernel<64><<<blocks, 256, 0, stream>>>(p.part_o, p.part_lse, p.splits, n_rows, a.L, a.Hq, p.out, p.lse);
        note_launch();
        if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
    }
    return DARE_OK;
}

// Packed variable-length bidirectional attention on the tcgen05 kernel: sequence s = "rollout" s, its tokens are the
// queries and, in place, the keys; K and V are 2-D [tokens, Hkv * d] views, a KV head is a column range.
int launch_attn_varlen(const dare_ctx* ctx, int total, int n_seqs, int max_seqlen, int Hq, int Hkv, int d, float scale,
                       const void* q, const void* k, const void* v, const int32_t* cu_seqlens, void* out, float* lse,
                       cudaStream_t stream) {
    AttnParams p = {};
    p.B = n_seqs; p.L = max_seqlen; p.Hq = Hq; p.Hkv = Hkv; p.g = Hq / Hkv; p.R = max_seqlen * p.g;
    p.prefix_cap = 0; p.suffix_cap = 0; p.inplace = 1; p.has_suffix = 0; p.splits = 1; p.uniform_P = 0;
    p.scale_log2 = (scale != 0.f ? scale : 1.0f / sqrtf(static_cast<float>(d))) * LOG2E_F;
    p.q = static_cast<const __nv_bfloat16*>(q);
    p.prefix_len = nullptr; p.suffix_len = nullptr;
    p.out = static_cast<__nv_bfloat16*>(out); p.lse = lse;
    p.part_o = nullptr; p.part_lse = nullptr;
    p.dev_status = ctx->dev_status;
    p.cu_seqlens = cu_seqlens; p.total_tokens = total;
    CUtensorMap tm[6];
    int rc = make_tmap_bf16_2d(ctx, &tm[0], k, static_cast<uint64_t>(total), static_cast<uint64_t>(Hkv) * d, TC_KT, 64);
    if (rc == DARE_OK) rc = make_tmap_bf16_2d(ctx, &tm[1], v, static_cast<uint64_t>(total), static_cast<uint64_t>(Hkv) * d, TC_KT, 64);
    if (rc != DARE_OK) return rc;
    tm[2] = tm[0]; tm[3] = tm[1]; tm[4] = tm[0]; tm[5] = tm[1];
    const int pos_per_tile = 128 / p.g;
    const int q_tiles = (max_seqlen + pos_per_tile - 1) / pos_per_tile;
    if (q_tiles >= 2) return d == 128 ? launch_tc<128, 2>(tm, p, q_tiles, stream) : launch_tc<64, 2>(tm, p, q_tiles, stream);
    return d == 128 ? launch_tc<128, 1>(tm, p, q_tiles, stream) : launch_tc<64, 1>(tm, p, q_tiles, stream);
}

}  // namespace dare
