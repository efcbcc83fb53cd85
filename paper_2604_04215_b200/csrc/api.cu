// C-ABI entry points: argument validation, context/workspace, tensor-map encoding, launches.
// Nothing here computes; every step of the path runs in the kernels of lmhead.cu, attn.cu and select.cu.
#include <math.h>
#include <new>
#include <stdlib.h>

#include "internal.h"

namespace dare {

std::atomic<uint64_t> g_kernel_launches{0};

int make_tmap_bf16_2d(const dare_ctx* ctx, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                      uint32_t box_rows, uint32_t box_cols) {
    TmapCache::Slot* slot = nullptr;
    if (ctx->tmaps) {
        // 64-bit finaliser over the whole key (allocations are aligned to hundreds of bytes, shapes are round numbers:
        // the raw low bits carry almost nothing)
        uint64_t h = reinterpret_cast<uintptr_t>(base) ^ (rows * 0x9E3779B97F4A7C15ull) ^ (cols * 0xC2B2AE3D27D4EB4Full) ^
                     (static_cast<uint64_t>(box_rows) << 40) ^ (static_cast<uint64_t>(box_cols) << 52);
        h ^= h >> 30; h *= 0xBF58476D1CE4E5B9ull;
        h ^= h >> 27; h *= 0x94D049BB133111EBull;
        h ^= h >> 31;
        const int set = static_cast<int>(h % TmapCache::SETS);
        TmapCache::Slot* ways = &ctx->tmaps->slot[set * TmapCache::WAYS];
        for (int i = 0; i < TmapCache::WAYS; ++i) {
            TmapCache::Slot& s = ways[i];
            if (s.valid && s.base == base && s.rows == rows && s.cols == cols && s.box_rows == box_rows &&
                s.box_cols == box_cols) {
                *out = s.map;
                ++ctx->tmaps->hits;
                return DARE_OK;
            }
        }
        ++ctx->tmaps->misses;
        slot = &ways[ctx->tmaps->next_way[set]];
        for (int i = 0; i < TmapCache::WAYS; ++i)       // an empty way first, else the set's next one in turn
            if (!ways[i].valid) { slot = &ways[i]; break; }
        if (slot->valid) ctx->tmaps->next_way[set] = static_cast<uint8_t>((ctx->tmaps->next_way[set] + 1) % TmapCache::WAYS);
    }
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};   // bytes, dimension 1
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode_tiled(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides,
                                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                   CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return DARE_ERR_CUDA;
    if (slot) {
        slot->base = base; slot->rows = rows; slot->cols = cols; slot->box_rows = box_rows; slot->box_cols = box_cols;
        slot->map = *out;
        slot->valid = true;
    }
    return DARE_OK;
}

}  // namespace dare

namespace {

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_attn(const dare_ctx* ctx, int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap, float scale,
               const void* q, const void* k_pre, const void* v_pre, const void* k_blk, const void* v_blk,
               const void* k_suf, const void* v_suf, const void* out, dare::AttnArgs* a) {
    if (!ctx || !q || !k_pre || !v_pre || !out) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if ((k_blk == nullptr) != (v_blk == nullptr)) return DARE_ERR_NULL;
    if ((k_suf == nullptr) != (v_suf == nullptr)) return DARE_ERR_NULL;
    if (B < 1 || L < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0) return DARE_ERR_SHAPE;
    if (d != 64 && d != 128) return DARE_ERR_SHAPE;
    if (static_cast<long long>(L) * (Hq / Hkv) > (1 << 20)) return DARE_ERR_SHAPE;
    if (prefix_cap < (k_blk ? 1 : L) || suffix_cap < 0) return DARE_ERR_SHAPE;
    if (k_suf && suffix_cap < 1) return DARE_ERR_SHAPE;
    if (static_cast<long long>(B) * Hkv * prefix_cap > 0x7fffffffLL) return DARE_ERR_SHAPE;
    if (!(scale >= 0.f) || isinf(scale)) return DARE_ERR_RANGE;
    if (!aligned16(q) || !aligned16(k_pre) || !aligned16(v_pre) || !aligned16(out) || !aligned16(k_blk) ||
        !aligned16(v_blk) || !aligned16(k_suf) || !aligned16(v_suf))
        return DARE_ERR_ALIGN;
    a->B = B; a->L = L; a->Hq = Hq; a->Hkv = Hkv; a->d = d; a->prefix_cap = prefix_cap; a->suffix_cap = suffix_cap;
    a->scale = scale; a->q = q; a->k_pre = k_pre; a->v_pre = v_pre; a->k_blk = k_blk; a->v_blk = v_blk;
    a->k_suf = k_suf; a->v_suf = v_suf; a->out = const_cast<void*>(out);
    a->prefix_len = nullptr; a->prefix_len_uniform = -1; a->suffix_len = nullptr; a->lse = nullptr;
    const int splits = dare::attn_plan_splits(ctx, *a);
    if (dare::attn_workspace_bytes(*a, splits) > ctx->workspace_bytes) return DARE_ERR_WORKSPACE;
    return DARE_OK;
}

int check_lmhead(const dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V, bool with_row_tokens,
                 const void* pred, const void* conf, bool sampling = false) {
    if (!ctx || !hidden || !w || !pred || !conf) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (M < 1 || D < 8 || D % 8 != 0 || V < 2) return DARE_ERR_SHAPE;
    if (!aligned16(hidden) || !aligned16(w)) return DARE_ERR_ALIGN;
    if (dare::lmhead_workspace_bytes(M, D, V, ctx->sm_count, with_row_tokens, sampling) > ctx->workspace_bytes)
        return DARE_ERR_WORKSPACE;
    return DARE_OK;
}

int check_select(const void* tokens, int B, int64_t row_stride, int block_start, int L, const void* pred,
                 const void* conf, int mode, float threshold, int k) {
    if (!tokens || !pred || !conf) return DARE_ERR_NULL;
    if (B < 1 || L < 1 || L > 4096) return DARE_ERR_SHAPE;
    if (block_start < 0 || row_stride < 1 || static_cast<int64_t>(block_start) + L > row_stride) return DARE_ERR_RANGE;
    if (mode != DARE_SELECT_THRESHOLD && mode != DARE_SELECT_TOPK) return DARE_ERR_RANGE;
    if (mode == DARE_SELECT_THRESHOLD && threshold != threshold) return DARE_ERR_RANGE;
    if (mode == DARE_SELECT_TOPK && k < 1) return DARE_ERR_RANGE;
    return DARE_OK;
}

}  // namespace

extern "C" {

int dare_create(dare_ctx** out, int device, size_t workspace_bytes) {
    if (!out) return DARE_ERR_NULL;
    *out = nullptr;
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) return DARE_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return DARE_ERR_CUDA;
    if (prop.major != 10) return DARE_ERR_UNSUPPORTED;
    dare::DeviceScope scope(device);      // the caller's current device is put back on return
    if (!scope.ok()) return DARE_ERR_CUDA;
    dare_ctx* ctx = new (std::nothrow) dare_ctx();
    if (!ctx) return DARE_ERR_CUDA;
    ctx->tmaps = new (std::nothrow) TmapCache();      // value-initialised: every slot invalid
    if (!ctx->tmaps) { delete ctx; return DARE_ERR_CUDA; }
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->workspace_bytes = workspace_bytes ? workspace_bytes : (size_t(256) << 20);
    ctx->workspace = nullptr;
    ctx->dev_status = nullptr;
    ctx->aux = nullptr; ctx->ev_fork = nullptr; ctx->ev_mid = nullptr; ctx->ev_join = nullptr;
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || fn == nullptr) {
        delete ctx->tmaps;
        delete ctx;
        return DARE_ERR_CUDA;
    }
    ctx->encode_tiled = reinterpret_cast<dare_encode_tiled_fn>(fn);
    int prio_low = 0, prio_high = 0;      // the side stream takes the highest priority (see dare_denoise_block)
    if (cudaDeviceGetStreamPriorityRange(&prio_low, &prio_high) != cudaSuccess) prio_high = 0;
    if (cudaMalloc(&ctx->workspace, ctx->workspace_bytes) != cudaSuccess ||
        cudaMalloc(reinterpret_cast<void**>(&ctx->dev_status), sizeof(uint32_t)) != cudaSuccess ||
        cudaMemset(ctx->dev_status, 0, sizeof(uint32_t)) != cudaSuccess ||
        cudaStreamCreateWithPriority(&ctx->aux, cudaStreamNonBlocking, prio_high) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_mid, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess) {
        if (ctx->workspace) cudaFree(ctx->workspace);
        if (ctx->dev_status) cudaFree(ctx->dev_status);
        if (ctx->aux) cudaStreamDestroy(ctx->aux);
        if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
        if (ctx->ev_mid) cudaEventDestroy(ctx->ev_mid);
        if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
        delete ctx->tmaps;
        delete ctx;
        return DARE_ERR_CUDA;
    }
    *out = ctx;
    return DARE_OK;
}

int dare_destroy(dare_ctx* ctx) {
    if (!ctx) return DARE_ERR_NULL;
    dare::DeviceScope scope(ctx->device);
    cudaFree(ctx->workspace);
    cudaFree(ctx->dev_status);
    if (ctx->aux) cudaStreamDestroy(ctx->aux);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_mid) cudaEventDestroy(ctx->ev_mid);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    delete ctx->tmaps;
    delete ctx;
    return DARE_OK;
}

int dare_tmap_cache_stats(const dare_ctx* ctx, uint64_t* hits, uint64_t* misses) {
    if (!ctx || !hits || !misses) return DARE_ERR_NULL;
    *hits = ctx->tmaps ? ctx->tmaps->hits : 0;
    *misses = ctx->tmaps ? ctx->tmaps->misses : 0;
    return DARE_OK;
}

const char* dare_status_string(int status) {
    switch (status) {
        case DARE_OK: return "ok";
        case DARE_ERR_NULL: return "a required pointer is NULL";
        case DARE_ERR_SHAPE: return "unsupported or inconsistent dimensions";
        case DARE_ERR_ALIGN: return "pointer or row size not 16-byte aligned";
        case DARE_ERR_RANGE: return "scalar argument out of range";
        case DARE_ERR_WORKSPACE: return "context workspace too small";
        case DARE_ERR_CUDA: return "CUDA call failed";
        case DARE_ERR_UNSUPPORTED: return "device is not sm_100";
        case DARE_ERR_DEVICE: return "the current CUDA device is not the one the context or buffers belong to";
        default: return "unknown status";
    }
}

int dare_device_status(dare_ctx* ctx, void* stream, uint32_t* host_out) {
    if (!ctx || !host_out) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(host_out, ctx->dev_status, sizeof(uint32_t), cudaMemcpyDeviceToHost, s) != cudaSuccess)
        return DARE_ERR_CUDA;
    if (cudaMemsetAsync(ctx->dev_status, 0, sizeof(uint32_t), s) != cudaSuccess) return DARE_ERR_CUDA;
    if (cudaStreamSynchronize(s) != cudaSuccess) return DARE_ERR_CUDA;
    return DARE_OK;
}

int dare_sm_count(const dare_ctx* ctx) { return ctx ? ctx->sm_count : DARE_ERR_NULL; }

uint64_t dare_kernel_launches(void) { return dare::g_kernel_launches.load(std::memory_order_relaxed); }

int dare_attn_block(dare_ctx* ctx, int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap, float scale,
                    const void* q, const void* k_pre, const void* v_pre, const int32_t* prefix_len, const void* k_blk,
                    const void* v_blk, const void* k_suf, const void* v_suf, const int32_t* suffix_len, void* out,
                    float* lse, void* stream) {
    dare::AttnArgs a;
    int rc = check_attn(ctx, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, scale, q, k_pre, v_pre, k_blk, v_blk, k_suf,
                        v_suf, out, &a);
    if (rc != DARE_OK) return rc;
    a.prefix_len = prefix_len; a.suffix_len = suffix_len; a.lse = lse;
    return dare::launch_attn(ctx, a, static_cast<cudaStream_t>(stream));
}

int dare_attn_varlen(dare_ctx* ctx, int total_tokens, int n_seqs, int max_seqlen, int Hq, int Hkv, int d, float scale,
                     const void* q, const void* k, const void* v, const int32_t* cu_seqlens, void* out, float* lse,
                     void* stream) {
    if (!ctx || !q || !k || !v || !cu_seqlens || !out) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (total_tokens < 1 || n_seqs < 1 || max_seqlen < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || Hq / Hkv > 128)
        return DARE_ERR_SHAPE;
    if (d != 64 && d != 128) return DARE_ERR_SHAPE;
    if (static_cast<long long>(n_seqs) * Hkv > 65535) return DARE_ERR_SHAPE;
    if (!(scale >= 0.f) || isinf(scale)) return DARE_ERR_RANGE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return DARE_ERR_ALIGN;
    return dare::launch_attn_varlen(ctx, total_tokens, n_seqs, max_seqlen, Hq, Hkv, d, scale, q, k, v, cu_seqlens, out, lse,
                                    static_cast<cudaStream_t>(stream));
}

int dare_lmhead_confidence(dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V,
                           const int32_t* row_tokens, int32_t mask_id, int exclude_mask_column, int32_t* pred,
                           float* conf, void* stream) {
    int rc = check_lmhead(ctx, hidden, M, D, w, V, row_tokens != nullptr, pred, conf);
    if (rc != DARE_OK) return rc;
    return dare::launch_lmhead(ctx, ctx->workspace, hidden, M, D, w, V, row_tokens, M, 0, mask_id, exclude_mask_column,
                               pred, conf, static_cast<cudaStream_t>(stream), nullptr);
}

int dare_lmhead_logprob(dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V, const int32_t* targets,
                        int32_t mask_id, int exclude_mask_column, float* logprob, float* lse, void* stream) {
    if (!targets) return DARE_ERR_NULL;
    int rc = check_lmhead(ctx, hidden, M, D, w, V, false, targets, logprob);
    if (rc != DARE_OK) return rc;
    return dare::launch_lmhead_logprob(ctx, ctx->workspace, hidden, M, D, w, V, targets, mask_id, exclude_mask_column,
                                       logprob, lse, static_cast<cudaStream_t>(stream));
}

int dare_lmhead_sample(dare_ctx* ctx, const void* hidden, int M, int D, const void* w, int V, const int32_t* row_tokens,
                       int32_t mask_id, int exclude_mask_column, float temperature, uint64_t seed, uint32_t step,
                       int32_t* pred, float* conf, void* stream) {
    int rc = check_lmhead(ctx, hidden, M, D, w, V, row_tokens != nullptr, pred, conf, true);
    if (rc != DARE_OK) return rc;
    if (!(temperature > 0.f) || isinf(temperature)) return DARE_ERR_RANGE;
    const dare::LmSampleArgs smp = {temperature, seed, step};
    return dare::launch_lmhead(ctx, ctx->workspace, hidden, M, D, w, V, row_tokens, M, 0, mask_id, exclude_mask_column,
                               pred, conf, static_cast<cudaStream_t>(stream), &smp);
}

int dare_unmask_select(dare_ctx* ctx, int32_t* tokens, int B, int64_t row_stride, int block_start, int L,
                       const int32_t* pred, const float* conf, int32_t mask_id, int mode, float threshold, int k,
                       int32_t* n_committed, int32_t* n_remaining, void* stream) {
    if (!ctx) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    int rc = check_select(tokens, B, row_stride, block_start, L, pred, conf, mode, threshold, k);
    if (rc != DARE_OK) return rc;
    return dare::launch_unmask_select(tokens, B, row_stride, block_start, L, pred, conf, mask_id, mode, threshold, k,
                                      n_committed, n_remaining, static_cast<cudaStream_t>(stream));
}

// The launches of one step, shared by the greedy and the sampled entry point (every argument has been validated).
static int enqueue_step(dare_ctx* ctx, const dare::AttnArgs& a, const void* hidden, int M, int D, const void* w, int V,
                        int32_t mask_id, int exclude_mask_column, const dare::LmSampleArgs* sample, int32_t* tokens,
                        int B, int L, int64_t row_stride, int block_start, int mode, float threshold, int k,
                        int32_t* pred, float* conf, int32_t* n_committed, int32_t* n_remaining, cudaStream_t s) {
    int rc = DARE_OK;
    // The LM head reads each row's current token straight from the token state: row m = (r, i) lives at
    // tokens[r * row_stride + block_start + i].
    //
    // Neither of the step's two halves reads what the other writes: the attention takes q and the caches and writes
    // attn_out (and lse); the head takes `hidden` and the token state and writes pred, conf and the tokens.  The
    // head's GEMM is a single wave of CTAs, one per SM, that finish up to a tenth of its duration apart (a CTA owns
    // 13 or 14 vocabulary tiles, and a tile is the unit of its work), and in that tail a third to a half of the SMs
    // have nothing to do.  So the head goes first, on the context's side stream (highest priority, ordered after
    // everything already on `stream`), and the attention is enqueued on `stream` behind the head's row compaction:
    // both the GEMM and the attention become ready at that point, the GEMM's CTAs take every SM, and the attention's
    // CTAs (which do not fit beside them) move into the SMs that the GEMM's early finishers leave.  `stream` joins
    // the side stream at the end, so everything the step wrote is ordered before what the caller enqueues next.
    // (Not when the attention splits K/V: its partials and the head's scratch share the workspace.)
    const bool overlap = ctx->aux && dare::attn_plan_splits(ctx, a) == 1;
    cudaStream_t head = s;
    if (overlap) {
        if (cudaEventRecord(ctx->ev_fork, s) != cudaSuccess || cudaStreamWaitEvent(ctx->aux, ctx->ev_fork, 0) != cudaSuccess)
            return DARE_ERR_CUDA;
        head = ctx->aux;
    } else {
        rc = dare::launch_attn(ctx, a, s);
        if (rc != DARE_OK) return rc;
    }
    if (sample == nullptr && L <= dare::LMHEAD_SELECT_MAX_L) {      // short blocks: the selection rides on the greedy head's merge kernel
        const dare::LmSelectArgs sel = {tokens + block_start, B, mode, threshold, k, n_committed, n_remaining};
        rc = dare::launch_lmhead(ctx, ctx->workspace, hidden, M, D, w, V, tokens + block_start, L, row_stride, mask_id,
                                 exclude_mask_column, pred, conf, head, nullptr, &sel, overlap ? ctx->ev_mid : nullptr);
    } else {
        rc = dare::launch_lmhead(ctx, ctx->workspace, hidden, M, D, w, V, tokens + block_start, L, row_stride, mask_id,
                                 exclude_mask_column, pred, conf, head, sample, nullptr, overlap ? ctx->ev_mid : nullptr);
        if (rc == DARE_OK)
            rc = dare::launch_unmask_select(tokens, B, row_stride, block_start, L, pred, conf, mask_id, mode, threshold, k,
                                            n_committed, n_remaining, head);
    }
    if (overlap) {
        // (also after an error above: `stream` must not be left without its join once the fork has been enqueued)
        int rc2 = DARE_OK;
        if (cudaStreamWaitEvent(s, ctx->ev_mid, 0) != cudaSuccess) rc2 = DARE_ERR_CUDA;
        if (rc == DARE_OK && rc2 == DARE_OK) rc2 = dare::launch_attn(ctx, a, s);
        if (cudaEventRecord(ctx->ev_join, ctx->aux) != cudaSuccess || cudaStreamWaitEvent(s, ctx->ev_join, 0) != cudaSuccess)
            rc2 = DARE_ERR_CUDA;
        if (rc == DARE_OK) rc = rc2;
    }
    return rc;
}

int dare_denoise_block(dare_ctx* ctx, int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap,
                       float scale, const void* q, const void* k_pre, const void* v_pre, const int32_t* prefix_len,
                       const void* k_blk, const void* v_blk, const void* k_suf, const void* v_suf,
                       const int32_t* suffix_len, void* attn_out, float* lse, const void* hidden, int D, const void* w,
                       int V, int32_t mask_id, int exclude_mask_column, int32_t* tokens, int64_t row_stride,
                       int block_start, int mode, float threshold, int k, int32_t* pred, float* conf,
                       int32_t* n_committed, int32_t* n_remaining, void* stream) {
    // validate everything first: on any error nothing is launched
    dare::AttnArgs a;
    int rc = check_attn(ctx, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, scale, q, k_pre, v_pre, k_blk, v_blk, k_suf,
                        v_suf, attn_out, &a);
    if (rc != DARE_OK) return rc;
    a.prefix_len = prefix_len; a.suffix_len = suffix_len; a.lse = lse;
    if (static_cast<long long>(B) * L > 0x7fffffffLL) return DARE_ERR_SHAPE;
    const int M = B * L;
    rc = check_lmhead(ctx, hidden, M, D, w, V, true, pred, conf);
    if (rc != DARE_OK) return rc;
    rc = check_select(tokens, B, row_stride, block_start, L, pred, conf, mode, threshold, k);
    if (rc != DARE_OK) return rc;
    return enqueue_step(ctx, a, hidden, M, D, w, V, mask_id, exclude_mask_column, nullptr, tokens, B, L, row_stride,
                        block_start, mode, threshold, k, pred, conf, n_committed, n_remaining,
                        static_cast<cudaStream_t>(stream));
}

// The step with the sampled head: as dare_denoise_block, the token of every masked row drawn by temperature +
// Gumbel-max sampling (dare_lmhead_sample), its confidence the temperature-1 probability of that token.
int dare_denoise_block_sampled(dare_ctx* ctx, int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap,
                               float scale, const void* q, const void* k_pre, const void* v_pre,
                               const int32_t* prefix_len, const void* k_blk, const void* v_blk, const void* k_suf,
                               const void* v_suf, const int32_t* suffix_len, void* attn_out, float* lse,
                               const void* hidden, int D, const void* w, int V, int32_t mask_id, int exclude_mask_column,
                               float temperature, uint64_t seed, uint32_t step, int32_t* tokens, int64_t row_stride,
                               int block_start, int mode, float threshold, int k, int32_t* pred, float* conf,
                               int32_t* n_committed, int32_t* n_remaining, void* stream) {
    dare::AttnArgs a;
    int rc = check_attn(ctx, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, scale, q, k_pre, v_pre, k_blk, v_blk, k_suf,
                        v_suf, attn_out, &a);
    if (rc != DARE_OK) return rc;
    a.prefix_len = prefix_len; a.suffix_len = suffix_len; a.lse = lse;
    if (static_cast<long long>(B) * L > 0x7fffffffLL) return DARE_ERR_SHAPE;
    const int M = B * L;
    rc = check_lmhead(ctx, hidden, M, D, w, V, true, pred, conf, true);
    if (rc != DARE_OK) return rc;
    if (!(temperature > 0.f) || isinf(temperature)) return DARE_ERR_RANGE;
    rc = check_select(tokens, B, row_stride, block_start, L, pred, conf, mode, threshold, k);
    if (rc != DARE_OK) return rc;
    const dare::LmSampleArgs smp = {temperature, seed, step};
    return enqueue_step(ctx, a, hidden, M, D, w, V, mask_id, exclude_mask_column, &smp, tokens, B, L, row_stride,
                        block_start, mode, threshold, k, pred, conf, n_committed, n_remaining,
                        static_cast<cudaStream_t>(stream));
}

}  // extern "C"
