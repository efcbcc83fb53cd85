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

constexpr int KT = 64;           // keys per tile
constexpr int ATT_STAGES = 3;
constexpr float LOG2E_F = 1.4426950408889634f;
constexpr float LN2_F = 0.6931471805599453f;

struct AttnParams {
    int B, L, Hq, Hkv, g, R;      // R = L * g packed query rows per (row, kv head)
    int prefix_cap, suffix_cap;
    int inplace, has_suffix, splits;
    int uniform_P;                // >= 0: every row's prefix length (used when prefix_len is NULL)
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
    uint64_t full[ATT_STAGES];
    uint64_t empty[ATT_STAGES];
    uint32_t abort_flag;
};

template <int D>
__host__ __device__ constexpr int att_stage_bytes() { return 2 * KT * D * 2; }
template <int D>
__host__ __device__ constexpr int att_smem_bytes() { return ATT_STAGES * att_stage_bytes<D>() + static_cast<int>(sizeof(AttBarriers)) + 1024; }

// Segment bookkeeping of one (row, kv head) unit: tiles of the prefix, then the block, then the suffix.
struct TileInfo {
    int seg;      // 0 prefix buffer, 1 block buffer, 2 suffix buffer
    int row0;     // first row of the tile in that buffer's 2-D [rows, D] view
    int valid;    // keys of the tile that exist (1..KT)
};

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
template <int D, int NW, int KS>
__global__ void __launch_bounds__((NW * KS + 1) * 32, (NW * KS + 1) * 32 <= 160 ? 2 : 1)
attn_block_kernel(const __grid_constant__ CUtensorMap tm_kpre, const __grid_constant__ CUtensorMap tm_vpre,
                  const __grid_constant__ CUtensorMap tm_kblk, const __grid_constant__ CUtensorMap tm_vblk,
                  const __grid_constant__ CUtensorMap tm_ksuf, const __grid_constant__ CUtensorMap tm_vsuf,
                  const AttnParams p) {
    constexpr int STAGE = att_stage_bytes<D>();
    constexpr int HALF = KT * 128;           // one 64-column half of a tile: 64 rows x 128 bytes
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

    if (threadIdx.x == 0) {
        for (int s = 0; s < ATT_STAGES; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], NCW);
        }
        bars->abort_flag = 0;
        fence_barrier_init();
    }
    __syncthreads();

    // lengths (clamped to capacity; a clamp is reported, never trapped on)
    int P = p.prefix_len ? p.prefix_len[b]
                         : (p.uniform_P >= 0 ? p.uniform_P : (p.inplace ? p.prefix_cap - p.L : p.prefix_cap));
    const int p_max = p.inplace ? p.prefix_cap - p.L : p.prefix_cap;
    int S = p.has_suffix ? (p.suffix_len ? p.suffix_len[b] : p.suffix_cap) : 0;
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
    float oacc[D / 8][4];
#pragma unroll
    for (int n = 0; n < D / 8; ++n) { oacc[n][0] = oacc[n][1] = oacc[n][2] = oacc[n][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    bool ok = true;

    if (warp == NCW) {
        // ---------------- producer
        if (lane == 0) {
            prefetch_tensormap(&tm_kpre);
            prefetch_tensormap(&tm_vpre);
            int stage = 0;
            uint32_t phase = 0;
            for (int t = t_begin; t < t_end; ++t) {
                const TileInfo ti = tile_info(t, n_pre, n_blk, len_pre, len_blk, S, base_pre, base_blk, base_suf);
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
        const size_t qoff0 = ((static_cast<size_t>(b) * p.L + i0) * p.Hq + h0) * D;
        const size_t qoff1 = ((static_cast<size_t>(b) * p.L + i1) * p.Hq + h1) * D;
        uint32_t qf[D / 16][4];
        {
            const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + qoff0);
            const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + qoff1);
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                qf[kk][0] = live0 ? q0[kk * 8 + tq] : 0u;
                qf[kk][1] = live1 ? q1[kk * 8 + tq] : 0u;
                qf[kk][2] = live0 ? q0[kk * 8 + 4 + tq] : 0u;
                qf[kk][3] = live1 ? q1[kk * 8 + 4 + tq] : 0u;
            }
        }
        int stage = 0;
        uint32_t phase = 0;
        const int mi = lane >> 3, rin = lane & 7;
        const int koff = ks * KPW;           // this warp's keys inside a tile: [koff, koff + KPW)
        for (int t = t_begin; t < t_end; ++t) {
            const TileInfo ti = tile_info(t, n_pre, n_blk, len_pre, len_blk, S, base_pre, base_blk, base_suf);
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
                // scale into the log2 domain, mask keys that do not exist, row max
                float tmax0 = -INFINITY, tmax1 = -INFINITY;
#pragma unroll
                for (int nb = 0; nb < KPW / 8; ++nb) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int key = koff + nb * 8 + tq * 2 + (e & 1);
                        float sv = sacc[nb][e] * p.scale_log2;
                        if (key >= ti.valid) sv = -INFINITY;
                        sacc[nb][e] = sv;
                    }
                    tmax0 = fmaxf(tmax0, fmaxf(sacc[nb][0], sacc[nb][1]));
                    tmax1 = fmaxf(tmax1, fmaxf(sacc[nb][2], sacc[nb][3]));
                }
                tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 1));
                tmax0 = fmaxf(tmax0, __shfl_xor_sync(0xffffffffu, tmax0, 2));
                tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 1));
                tmax1 = fmaxf(tmax1, __shfl_xor_sync(0xffffffffu, tmax1, 2));
                const float mn0 = fmaxf(m0, tmax0), mn1 = fmaxf(m1, tmax1);   // finite: the slice has >= 1 key
                const float a0 = fast_exp2(m0 - mn0), a1 = fast_exp2(m1 - mn1);
                m0 = mn0; m1 = mn1;
                float ps0 = 0.f, ps1 = 0.f;
                uint32_t pa[KPW / 16][4];
#pragma unroll
                for (int nb = 0; nb < KPW / 8; ++nb) {
                    const float e0 = fast_exp2(sacc[nb][0] - mn0), e1 = fast_exp2(sacc[nb][1] - mn0);
                    const float e2 = fast_exp2(sacc[nb][2] - mn1), e3 = fast_exp2(sacc[nb][3] - mn1);
                    ps0 += e0 + e1;
                    ps1 += e2 + e3;
                    pa[nb >> 1][(nb & 1) * 2 + 0] = pack_bf16(e0, e1);
                    pa[nb >> 1][(nb & 1) * 2 + 1] = pack_bf16(e2, e3);
                }
                l0 = l0 * a0 + ps0;
                l1 = l1 * a1 + ps1;
#pragma unroll
                for (int n = 0; n < D / 8; ++n) {
                    oacc[n][0] *= a0; oacc[n][1] *= a0;
                    oacc[n][2] *= a1; oacc[n][3] *= a1;
                }
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

template <int D, int NW, int KS>
int launch_one(const CUtensorMap* tm, const AttnParams& p, int chunks, cudaStream_t stream) {
    constexpr int SMEM = att_smem_bytes<D>();
    static_assert((KS - 1) * NW * ((D / 8) * 4 + 4) * 32 * 4 <= ATT_STAGES * att_stage_bytes<D>(), "merge buffer");
    if (cudaFuncSetAttribute(attn_block_kernel<D, NW, KS>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM) != cudaSuccess)
        return DARE_ERR_CUDA;
    dim3 grid(chunks, p.B * p.Hkv, p.splits);
    attn_block_kernel<D, NW, KS><<<grid, (NW * KS + 1) * 32, SMEM, stream>>>(tm[0], tm[1], tm[2], tm[3], tm[4], tm[5], p);
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int pick_warps(int R) { return R <= 16 ? 1 : (R <= 32 ? 2 : 4); }

}  // namespace

int attn_plan_splits(const dare_ctx* ctx, const AttnArgs& a) {
    const int g = a.Hq / a.Hkv;
    const int R = a.L * g;
    const int nw = pick_warps(R);
    const int chunks = (R + nw * 16 - 1) / (nw * 16);
    const long long units = static_cast<long long>(chunks) * a.B * a.Hkv;
    const int smem = a.d == 128 ? att_smem_bytes<128>() : att_smem_bytes<64>();
    int per_sm = (227 * 1024) / smem;
    if (per_sm > 8) per_sm = 8;
    const long long slots = static_cast<long long>(ctx->sm_count) * per_sm;
    if (units >= slots) return 1;
    const int tiles = (a.prefix_cap + (a.k_blk ? a.L : 0) + a.suffix_cap + KT - 1) / KT;
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

    const int nw = pick_warps(p.R);
    const int chunks = (p.R + nw * 16 - 1) / (nw * 16);
    if (a.d == 128) {
        rc = nw == 1 ? launch_one<128, 1, 4>(tm, p, chunks, stream)
           : nw == 2 ? launch_one<128, 2, 2>(tm, p, chunks, stream) : launch_one<128, 4, 1>(tm, p, chunks, stream);
    } else {
        rc = nw == 1 ? launch_one<64, 1, 4>(tm, p, chunks, stream)
           : nw == 2 ? launch_one<64, 2, 2>(tm, p, chunks, stream) : launch_one<64, 4, 1>(tm, p, chunks, stream);
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
        if (cudaGetLastError() != cudaSuccess) return DARE_ERR_CUDA;
    }
    return DARE_OK;
}

}  // namespace dare
