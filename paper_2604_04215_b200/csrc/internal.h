// Internal declarations shared by the translation units of libdare (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/dare.h"

typedef CUresult (*dare_encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                         const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                         CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                         CUtensorMapFloatOOBfill);

// Encoded tensor maps, kept per context.  A map is a pure function of (base address, rows, columns, box): it holds no
// state of the memory it describes, so an entry can never go stale -- a buffer that was freed and allocated again at
// the same address with the same shape gets the same, still correct, map.  The rollout passes the same buffers every
// step, so after the first step no call encodes anything.  Four-way set associative; a full set evicts in turn.
struct TmapCache {
    static constexpr int SETS = 256, WAYS = 4, SLOTS = SETS * WAYS;
    struct Slot {
        const void* base;
        uint64_t rows, cols;
        uint32_t box_rows, box_cols;
        bool valid;
        CUtensorMap map;
    };
    Slot slot[SLOTS];
    uint8_t next_way[SETS];
    uint64_t hits, misses;
};

struct dare_ctx {
    int device;
    int sm_count;
    void* workspace;
    size_t workspace_bytes;
    uint32_t* dev_status;   // device word, bits DARE_DEV_*
    dare_encode_tiled_fn encode_tiled;
    TmapCache* tmaps;       // host memory; NULL = encode on every call
    // side stream of the step (dare_denoise_block, highest priority): the LM head runs on it, forked from the caller's
    // stream (ev_fork) and joined back (ev_join); ev_mid marks the end of the head's row compaction, behind which the
    // attention is enqueued on the caller's stream.  NULL = none (the step then runs in sequence)
    cudaStream_t aux;
    cudaEvent_t ev_fork, ev_mid, ev_join;
};

#include <atomic>

namespace dare {

// Kernels this library has launched since it was loaded (counted on the host at every launch site; a launch that
// is replayed from a CUDA graph is counted per replay by whoever replays it).
extern std::atomic<uint64_t> g_kernel_launches;
inline void note_launch(uint64_t n = 1) { g_kernel_launches.fetch_add(n, std::memory_order_relaxed); }

// Raising a kernel's dynamic shared-memory limit is needed once per kernel and device, not per launch: `done` is a
// static of the launching function (one per kernel instantiation), bit d = set on device d.
template <typename Kernel>
inline int ensure_dynamic_smem(std::atomic<uint64_t>& done, Kernel kernel, int bytes) {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return DARE_ERR_CUDA;
    const uint64_t bit = (device >= 0 && device < 64) ? (uint64_t(1) << device) : 0;
    if (bit && (done.load(std::memory_order_acquire) & bit)) return DARE_OK;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess)
        return DARE_ERR_CUDA;
    if (bit) done.fetch_or(bit, std::memory_order_release);
    return DARE_OK;
}

// Makes `device` current for the lifetime of the object and puts the previous device back afterwards (the create
// and destroy calls allocate and free on the context's device whatever the caller's current device is).
class DeviceScope {
public:
    explicit DeviceScope(int device) : prev_(-1), ok_(false) {
        if (cudaGetDevice(&prev_) != cudaSuccess) { prev_ = -1; return; }
        ok_ = prev_ == device || cudaSetDevice(device) == cudaSuccess;
        if (prev_ == device) prev_ = -1;      // nothing to restore
    }
    ~DeviceScope() { if (prev_ >= 0) cudaSetDevice(prev_); }
    bool ok() const { return ok_; }
private:
    int prev_;
    bool ok_;
};

// The entry points launch on the CURRENT device with the context's workspace and status word: a context that
// belongs to another device must be refused before anything is enqueued.
inline int check_current_device(const dare_ctx* ctx) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) return DARE_ERR_CUDA;
    return dev == ctx->device ? DARE_OK : DARE_ERR_DEVICE;
}

// bf16 2-D row-major tensor [rows, cols] -> tensor map with a [box_rows, 64] box and 128-byte swizzle.
int make_tmap_bf16_2d(const dare_ctx* ctx, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                      uint32_t box_rows, uint32_t box_cols);

int launch_unmask_select(int32_t* tokens, int B, int64_t row_stride, int block_start, int L, const int32_t* pred,
                         const float* conf, int32_t mask_id, int mode, float threshold, int k, int32_t* n_committed,
                         int32_t* n_remaining, cudaStream_t stream);

// log p(target) per row = z_target - logsumexp z (and optionally logsumexp z); logits never stored.
int launch_lmhead_logprob(const dare_ctx* ctx, void* scratch, const void* hidden, int M, int D, const void* w, int V,
                          const int32_t* targets, int32_t mask_id, int exclude_mask_column, float* logprob, float* lse_out,
                          cudaStream_t stream);
// Sampling epilogue of the LM head (NULL = greedy): temperature, 64-bit seed and step counter of the generator.
// step_dev (optional, device): added to `step`; the head's last kernel then increments it, so that a step replayed
// from a CUDA graph draws fresh noise every time.
struct LmSampleArgs { float temperature; uint64_t seed; uint32_t step; uint32_t* step_dev = nullptr; };
size_t lmhead_workspace_bytes(int M, int D, int V, int sm_count, bool with_row_tokens, bool sampling);
// Token of LM-head row m (to skip committed rows) = row_tokens[(m / tok_L) * tok_row_stride + m % tok_L].
// Unmask selection folded into the head's last kernel (greedy head on a block of at most LMHEAD_SELECT_MAX_L
// positions whose tokens are given by row_tokens = tokens + block_start, tok_L = L): the caller then skips
// launch_unmask_select.  tokens_block is the same address as row_tokens, writable.
constexpr int LMHEAD_SELECT_MAX_L = 32;
struct LmSelectArgs { int32_t* tokens_block; int B; int mode; float threshold; int k; int32_t* n_committed; int32_t* n_remaining; };
int launch_lmhead(const dare_ctx* ctx, void* scratch, const void* hidden, int M, int D, const void* w, int V,
                  const int32_t* row_tokens, int tok_L, int64_t tok_row_stride, int32_t mask_id, int exclude_mask_column, int32_t* pred, float* conf,
                  cudaStream_t stream, const LmSampleArgs* sample, const LmSelectArgs* select = nullptr,
                  cudaEvent_t after_compaction = nullptr);    // non-NULL: recorded on `stream` behind the row compaction,
                                                              // i.e. just before the head's GEMM becomes ready to run

struct AttnArgs {
    int B, L, Hq, Hkv, d, prefix_cap, suffix_cap;
    float scale;
    const void* q;
    const void *k_pre, *v_pre;
    const int32_t* prefix_len;
    int prefix_len_uniform;   // used when prefix_len is NULL and this is >= 0 (internal callers)
    const void *k_blk, *v_blk;
    const void *k_suf, *v_suf;
    const int32_t* suffix_len;
    void* out;
    float* lse;
};
int attn_plan_splits(const dare_ctx* ctx, const AttnArgs& a);
size_t attn_workspace_bytes(const AttnArgs& a, int splits);
int launch_attn(const dare_ctx* ctx, const AttnArgs& a, cudaStream_t stream);
int launch_attn_varlen(const dare_ctx* ctx, int total, int n_seqs, int max_seqlen, int Hq, int Hkv, int d, float scale,
                       const void* q, const void* k, const void* v, const int32_t* cu_seqlens, void* out, float* lse,
                       cudaStream_t stream);

// ---- layer stack (gemm.cu, layers.cu)
enum { GEMM_EPI_STORE = 0, GEMM_EPI_RESIDUAL = 1, GEMM_EPI_SWIGLU = 2 };
// out[M, N] = epilogue(a[M, K] . w[N, K]^T), bf16 row-major, ldo = elements per output row.
//   STORE: out = acc.  RESIDUAL: out = res + acc (res may be out).  SWIGLU: out = silu(a w^T) * (a w2^T).
int launch_gemm(const dare_ctx* ctx, int epi, const void* a, int M, int K, const void* w, const void* w2, int N,
                void* out, const void* res, int ldo, cudaStream_t stream);
// out[8] = {row tiles per CTA, bn, output columns per tile, K splits, stages, row items, column tiles, resident clusters}
int gemm_plan_describe(const dare_ctx* ctx, int epi, int M, int N, int K, int* out);
int launch_embed(const void* emb, int D, int V, const int32_t* tokens, int64_t row_stride, int start, int length,
                 int n_rows, void* x, cudaStream_t stream);
int launch_rmsnorm(const void* x, int D, int n_rows, float eps, void* y, cudaStream_t stream);
int launch_rope_table(float* cs, int n_pos, int half, double base, cudaStream_t stream);
int launch_rope_kv_write(const void* qkv, int n_rows, int Hq, int Hkv, int d, int start, int length, const float* cs,
                         void* q_out, void* k_cache, void* v_cache, int cap, cudaStream_t stream);

}  // namespace dare
