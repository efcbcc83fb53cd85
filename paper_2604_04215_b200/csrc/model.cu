// The end-to-end denoising loop on a decoder-shaped stack (RMSNorm, fused QKV projection, RoPE, block
// attention against the in-place K/V cache, SwiGLU feed-forward, untied LM head): host-side sequencing only.
// Every arithmetic step is a kernel of gemm.cu, layers.cu, attn.cu, lmhead.cu or select.cu.
//
// A forward of the rows [start, start + length) of every rollout writes those rows' post-RoPE K/V into the
// cache at their positions and lets them attend to cache[0, start + length): with start = 0 this is the
// prefill (the prompt is one bidirectional segment); with start = a block's first position it is one
// denoising step's stack, or, once the block holds no mask, the refresh that leaves the block's final K/V in
// the cache before the prefix grows.
//
// A forward may also let its rows see cache[0, kv_len) with kv_len beyond the rows' own end: the positions
// behind the rows are then a cached suffix (whatever an earlier forward wrote there).  That is the dual cache
// of a fully bidirectional model: dare_generate_dual refreshes every position's K/V with one forward of the
// whole sequence before each block and runs the block's steps against prefix + block + suffix.
#include <math.h>
#include <cuda_bf16.h>
#include <new>

#include "internal.h"

struct dare_model {
    dare_ctx* ctx;
    dare_model_desc desc;
    const void* embedding;
    const void* lm_head;
    dare_layer_weights* layers;    // host copy of the caller's array (device pointers inside)
    float* rope_cs;                // [max_positions, d/2] (cos, sin)
    void *x, *h, *qkv, *q, *attn, *act;   // activations, max_rows each
    int32_t* host_counts;          // pinned: n_remaining of two steps in flight, [2][max_batch]
    int max_batch;
    cudaEvent_t ev[2];
    cudaStream_t work;             // the loop runs here: a block's step is captured once into a CUDA graph
    cudaEvent_t ev_in, ev_out;     // order the work stream after / before the caller's stream
    // sampled head (dare_model_set_sampling): temperature 0 = greedy; the device word counts the steps
    float sample_temperature;
    uint64_t sample_seed;
    uint32_t* step_counter;
};

namespace {

__global__ void set_word_kernel(uint32_t* p, uint32_t v) { *p = v; }

// Keys visible to the rows: cache[0, kv_len), start + length <= kv_len <= cap.
int forward_rows(dare_model* m, const int32_t* tokens, int B, int64_t row_stride, int start, int length, int kv_len,
                 void* k_cache, void* v_cache, int cap, void* hidden_out, cudaStream_t s) {
    using namespace dare;
    const dare_model_desc& c = m->desc;
    const int rows = B * length;
    const int nq = c.n_q_heads * c.head_dim, nkv = c.n_kv_heads * c.head_dim;
    int rc = launch_embed(m->embedding, c.hidden, c.vocab, tokens, row_stride, start, length, rows, m->x, s);
    if (rc != DARE_OK) return rc;
    const size_t layer_kv = static_cast<size_t>(B) * c.n_kv_heads * cap * c.head_dim;   // elements per layer
    for (int l = 0; l < c.n_layers; ++l) {
        const dare_layer_weights& w = m->layers[l];
        __nv_bfloat16* kc = static_cast<__nv_bfloat16*>(k_cache) + layer_kv * l;
        __nv_bfloat16* vc = static_cast<__nv_bfloat16*>(v_cache) + layer_kv * l;
        rc = launch_rmsnorm(m->x, c.hidden, rows, c.rms_eps, m->h, s);
        if (rc != DARE_OK) return rc;
        rc = launch_gemm(m->ctx, GEMM_EPI_STORE, m->h, rows, c.hidden, w.wqkv, nullptr, nq + 2 * nkv, m->qkv, nullptr,
                         nq + 2 * nkv, s);
        if (rc != DARE_OK) return rc;
        rc = launch_rope_kv_write(m->qkv, rows, c.n_q_heads, c.n_kv_heads, c.head_dim, start, length, m->rope_cs, m->q,
                                  kc, vc, cap, s);
        if (rc != DARE_OK) return rc;
        AttnArgs a;
        a.B = B; a.L = length; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.d = c.head_dim;
        a.prefix_cap = cap; a.suffix_cap = 0; a.scale = 0.f;
        a.q = m->q; a.k_pre = kc; a.v_pre = vc; a.prefix_len = nullptr;
        a.prefix_len_uniform = kv_len - length;   // in place: the kernel reads keys [0, this + length) of the cache
        a.k_blk = a.v_blk = a.k_suf = a.v_suf = nullptr; a.suffix_len = nullptr;
        a.out = m->attn; a.lse = nullptr;
        if (attn_workspace_bytes(a, attn_plan_splits(m->ctx, a)) > m->ctx->workspace_bytes) return DARE_ERR_WORKSPACE;
        rc = launch_attn(m->ctx, a, s);
        if (rc != DARE_OK) return rc;
        rc = launch_gemm(m->ctx, GEMM_EPI_RESIDUAL, m->attn, rows, nq, w.wo, nullptr, c.hidden, m->x, m->x, c.hidden, s);
        if (rc != DARE_OK) return rc;
        rc = launch_rmsnorm(m->x, c.hidden, rows, c.rms_eps, m->h, s);
        if (rc != DARE_OK) return rc;
        rc = launch_gemm(m->ctx, GEMM_EPI_SWIGLU, m->h, rows, c.hidden, w.wg, w.wu, c.ffn, m->act, nullptr, c.ffn, s);
        if (rc != DARE_OK) return rc;
        rc = launch_gemm(m->ctx, GEMM_EPI_RESIDUAL, m->act, rows, c.ffn, w.wd, nullptr, c.hidden, m->x, m->x, c.hidden, s);
        if (rc != DARE_OK) return rc;
    }
    return launch_rmsnorm(m->x, c.hidden, rows, c.rms_eps, hidden_out ? hidden_out : m->h, s);
}

int check_rows(const dare_model* m, const void* tokens, int B, int64_t row_stride, int start, int length, int kv_len,
               const void* k_cache, const void* v_cache, int cap) {
    if (!m || !tokens || !k_cache || !v_cache) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(m->ctx)) return rc;
    if (B < 1 || length < 1 || B > m->max_batch) return DARE_ERR_SHAPE;
    if (static_cast<long long>(B) * length > m->desc.max_rows) return DARE_ERR_SHAPE;
    if (start < 0 || static_cast<long long>(start) + length > cap || cap > m->desc.max_positions ||
        static_cast<long long>(start) + length > row_stride)
        return DARE_ERR_RANGE;
    if (kv_len < start + length || kv_len > cap) return DARE_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(k_cache) & 15u) || (reinterpret_cast<uintptr_t>(v_cache) & 15u)) return DARE_ERR_ALIGN;
    return DARE_OK;
}

int step_rows(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int start, int L, int kv_len, void* k_cache,
              void* v_cache, int cap, int mode, float threshold, int k, int32_t* pred, float* conf, int32_t* n_committed,
              int32_t* n_remaining, cudaStream_t s) {
    int rc = forward_rows(m, tokens, B, row_stride, start, L, kv_len, k_cache, v_cache, cap, nullptr, s);
    if (rc != DARE_OK) return rc;
    const int M = B * L;
    if (m->sample_temperature > 0.f) {          // sampled head, then the separate selection kernel
        dare::LmSampleArgs smp;
        smp.temperature = m->sample_temperature; smp.seed = m->sample_seed; smp.step = 0; smp.step_dev = m->step_counter;
        rc = dare::launch_lmhead(m->ctx, m->ctx->workspace, m->h, M, m->desc.hidden, m->lm_head, m->desc.vocab,
                                 tokens + start, L, row_stride, m->desc.mask_id, 1, pred, conf, s, &smp);
        if (rc != DARE_OK) return rc;
        return dare::launch_unmask_select(tokens, B, row_stride, start, L, pred, conf, m->desc.mask_id, mode, threshold,
                                          k, n_committed, n_remaining, s);
    }
    if (L <= dare::LMHEAD_SELECT_MAX_L) {      // short blocks: the selection rides on the head's merge kernel
        const dare::LmSelectArgs sel = {tokens + start, B, mode, threshold, k, n_committed, n_remaining};
        return dare::launch_lmhead(m->ctx, m->ctx->workspace, m->h, M, m->desc.hidden, m->lm_head, m->desc.vocab,
                                   tokens + start, L, row_stride, m->desc.mask_id, 1, pred, conf, s, nullptr, &sel);
    }
    rc = dare::launch_lmhead(m->ctx, m->ctx->workspace, m->h, M, m->desc.hidden, m->lm_head, m->desc.vocab,
                             tokens + start, L, row_stride, m->desc.mask_id, 1, pred, conf, s, nullptr);
    if (rc != DARE_OK) return rc;
    return dare::launch_unmask_select(tokens, B, row_stride, start, L, pred, conf, m->desc.mask_id, mode, threshold, k,
                                      n_committed, n_remaining, s);
}

int check_step(const dare_model* m, int B, int L, int mode, float threshold, int k, const void* pred, const void* conf) {
    if (!pred || !conf) return DARE_ERR_NULL;
    if (L > 4096) return DARE_ERR_SHAPE;
    if (mode != DARE_SELECT_THRESHOLD && mode != DARE_SELECT_TOPK) return DARE_ERR_RANGE;
    if (mode == DARE_SELECT_THRESHOLD && threshold != threshold) return DARE_ERR_RANGE;
    if (mode == DARE_SELECT_TOPK && k < 1) return DARE_ERR_RANGE;
    if (dare::lmhead_workspace_bytes(B * L, m->desc.hidden, m->desc.vocab, m->ctx->sm_count, true,
                                     m->sample_temperature > 0.f) > m->ctx->workspace_bytes)
        return DARE_ERR_WORKSPACE;
    return DARE_OK;
}

}  // namespace

extern "C" {

int dare_model_create(dare_ctx* ctx, const dare_model_desc* desc, const void* embedding,
                      const dare_layer_weights* layers, const void* lm_head, dare_model** out) {
    if (!ctx || !desc || !embedding || !layers || !lm_head || !out) return DARE_ERR_NULL;
    *out = nullptr;
    const dare_model_desc& c = *desc;
    if (c.n_layers < 1 || c.hidden < 8 || c.hidden % 8 || c.n_q_heads < 1 || c.n_kv_heads < 1 ||
        c.n_q_heads % c.n_kv_heads || (c.head_dim != 64 && c.head_dim != 128) || c.ffn < 8 || c.ffn % 8 || c.vocab < 2 ||
        c.max_positions < 1 || c.max_rows < 1 || c.max_batch < 1)
        return DARE_ERR_SHAPE;
    if (c.mask_id < 0 || c.mask_id >= c.vocab || !(c.rms_eps >= 0.f) || !(c.rope_base > 1.f)) return DARE_ERR_RANGE;
    for (int l = 0; l < c.n_layers; ++l)
        if (!layers[l].wqkv || !layers[l].wo || !layers[l].wg || !layers[l].wu || !layers[l].wd) return DARE_ERR_NULL;
    dare::DeviceScope scope(ctx->device);
    if (!scope.ok()) return DARE_ERR_CUDA;
    dare_model* m = new (std::nothrow) dare_model();
    if (!m) return DARE_ERR_CUDA;
    m->ctx = ctx; m->desc = c; m->embedding = embedding; m->lm_head = lm_head; m->max_batch = c.max_batch;
    m->layers = new (std::nothrow) dare_layer_weights[c.n_layers];
    m->rope_cs = nullptr; m->x = m->h = m->qkv = m->q = m->attn = m->act = nullptr; m->host_counts = nullptr;
    m->ev[0] = m->ev[1] = nullptr;
    m->work = nullptr; m->ev_in = m->ev_out = nullptr;
    m->sample_temperature = 0.f; m->sample_seed = 0; m->step_counter = nullptr;
    bool ok = m->layers != nullptr;
    if (ok) for (int l = 0; l < c.n_layers; ++l) m->layers[l] = layers[l];
    const size_t rows = static_cast<size_t>(c.max_rows);
    const size_t nq = static_cast<size_t>(c.n_q_heads) * c.head_dim, nkv = static_cast<size_t>(c.n_kv_heads) * c.head_dim;
    ok = ok && cudaMalloc(&m->rope_cs, sizeof(float) * 2 * c.max_positions * (c.head_dim / 2)) == cudaSuccess;
    ok = ok && cudaMalloc(&m->x, rows * c.hidden * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&m->h, rows * c.hidden * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&m->qkv, rows * (nq + 2 * nkv) * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&m->q, rows * nq * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&m->attn, rows * nq * 2) == cudaSuccess;
    ok = ok && cudaMalloc(&m->act, rows * c.ffn * 2) == cudaSuccess;
    ok = ok && cudaMalloc(reinterpret_cast<void**>(&m->step_counter), sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMemset(m->step_counter, 0, sizeof(uint32_t)) == cudaSuccess;
    ok = ok && cudaMallocHost(reinterpret_cast<void**>(&m->host_counts), sizeof(int32_t) * 2 * c.max_batch) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&m->ev[0], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&m->ev[1], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&m->ev_in, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&m->ev_out, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&m->work, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && dare::launch_rope_table(m->rope_cs, c.max_positions, c.head_dim / 2, static_cast<double>(c.rope_base),
                                       nullptr) == DARE_OK;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
    if (!ok) {
        dare_model_destroy(m);
        return DARE_ERR_CUDA;
    }
    *out = m;
    return DARE_OK;
}

int dare_model_destroy(dare_model* m) {
    if (!m) return DARE_ERR_NULL;
    dare::DeviceScope scope(m->ctx->device);
    cudaFree(m->rope_cs); cudaFree(m->x); cudaFree(m->h); cudaFree(m->qkv); cudaFree(m->q); cudaFree(m->attn);
    cudaFree(m->act);
    cudaFree(m->step_counter);
    if (m->host_counts) cudaFreeHost(m->host_counts);
    if (m->ev[0]) cudaEventDestroy(m->ev[0]);
    if (m->ev[1]) cudaEventDestroy(m->ev[1]);
    if (m->ev_in) cudaEventDestroy(m->ev_in);
    if (m->ev_out) cudaEventDestroy(m->ev_out);
    if (m->work) cudaStreamDestroy(m->work);
    delete[] m->layers;
    delete m;
    return DARE_OK;
}

int dare_model_set_sampling(dare_model* m, float temperature, uint64_t seed, uint32_t first_step, void* stream) {
    if (!m) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(m->ctx)) return rc;
    if (!(temperature >= 0.f) || isinf(temperature)) return DARE_ERR_RANGE;
    m->sample_temperature = temperature;
    m->sample_seed = seed;
    set_word_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(m->step_counter, first_step); dare::note_launch();
    return cudaGetLastError() == cudaSuccess ? DARE_OK : DARE_ERR_CUDA;
}

int dare_linear(dare_ctx* ctx, int epilogue, const void* a, int M, int K, const void* w, const void* w2, int N, void* out,
                const void* residual, void* stream) {
    if (!ctx || !a || !w || !out) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (epilogue == DARE_LINEAR_SWIGLU && !w2) return DARE_ERR_NULL;
    if (epilogue == DARE_LINEAR_RESIDUAL && !residual) return DARE_ERR_NULL;
    if (epilogue < DARE_LINEAR_STORE || epilogue > DARE_LINEAR_SWIGLU) return DARE_ERR_RANGE;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(a) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(w2) |
                           reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(residual);
    if (bits & 15u) return DARE_ERR_ALIGN;
    return dare::launch_gemm(ctx, epilogue, a, M, K, w, w2, N, out, residual, N, static_cast<cudaStream_t>(stream));
}

int dare_linear_plan(dare_ctx* ctx, int epilogue, int M, int K, int N, int* plan_out) {
    if (!ctx || !plan_out) return DARE_ERR_NULL;
    if (M < 1 || N < 8 || K < 8 || (N % 8) || (K % 8)) return DARE_ERR_SHAPE;
    if (epilogue < DARE_LINEAR_STORE || epilogue > DARE_LINEAR_SWIGLU) return DARE_ERR_RANGE;
    return dare::gemm_plan_describe(ctx, epilogue, M, N, K, plan_out);
}

int dare_rmsnorm(dare_ctx* ctx, const void* x, int n_rows, int D, float eps, void* y, void* stream) {
    if (!ctx || !x || !y) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(ctx)) return rc;
    if (n_rows < 1 || D < 8 || D % 8) return DARE_ERR_SHAPE;
    if (!(eps >= 0.f)) return DARE_ERR_RANGE;
    if ((reinterpret_cast<uintptr_t>(x) | reinterpret_cast<uintptr_t>(y)) & 15u) return DARE_ERR_ALIGN;
    return dare::launch_rmsnorm(x, D, n_rows, eps, y, static_cast<cudaStream_t>(stream));
}

int dare_rope_kv_write(dare_model* m, const void* qkv, int B, int length, int start, void* q_out, void* k_cache,
                       void* v_cache, int cache_cap, void* stream) {
    if (!m || !qkv || !q_out || !k_cache || !v_cache) return DARE_ERR_NULL;
    if (int rc = dare::check_current_device(m->ctx)) return rc;
    if (B < 1 || length < 1) return DARE_ERR_SHAPE;
    if (start < 0 || static_cast<long long>(start) + length > cache_cap || cache_cap > m->desc.max_positions)
        return DARE_ERR_RANGE;
    const uintptr_t bits = reinterpret_cast<uintptr_t>(qkv) | reinterpret_cast<uintptr_t>(q_out) |
                           reinterpret_cast<uintptr_t>(k_cache) | reinterpret_cast<uintptr_t>(v_cache);
    if (bits & 15u) return DARE_ERR_ALIGN;
    return dare::launch_rope_kv_write(qkv, B * length, m->desc.n_q_heads, m->desc.n_kv_heads, m->desc.head_dim, start,
                                      length, m->rope_cs, q_out, k_cache, v_cache, cache_cap,
                                      static_cast<cudaStream_t>(stream));
}

int dare_model_forward_window(dare_model* m, const int32_t* tokens, int B, int64_t row_stride, int start, int length,
                              int kv_len, void* k_cache, void* v_cache, int cache_cap, void* hidden_out, void* stream) {
    int rc = check_rows(m, tokens, B, row_stride, start, length, kv_len, k_cache, v_cache, cache_cap);
    if (rc != DARE_OK) return rc;
    return forward_rows(m, tokens, B, row_stride, start, length, kv_len, k_cache, v_cache, cache_cap, hidden_out,
                        static_cast<cudaStream_t>(stream));
}

int dare_model_forward(dare_model* m, const int32_t* tokens, int B, int64_t row_stride, int start, int length,
                       void* k_cache, void* v_cache, int cache_cap, void* hidden_out, void* stream) {
    return dare_model_forward_window(m, tokens, B, row_stride, start, length, start + length, k_cache, v_cache,
                                     cache_cap, hidden_out, stream);
}

int dare_model_step_window(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int block_start, int L, int kv_len,
                           void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k, int32_t* pred,
                           float* conf, int32_t* n_committed, int32_t* n_remaining, void* stream) {
    int rc = check_rows(m, tokens, B, row_stride, block_start, L, kv_len, k_cache, v_cache, cache_cap);
    if (rc == DARE_OK) rc = check_step(m, B, L, mode, threshold, k, pred, conf);
    if (rc != DARE_OK) return rc;
    return step_rows(m, tokens, B, row_stride, block_start, L, kv_len, k_cache, v_cache, cache_cap, mode, threshold, k,
                     pred, conf, n_committed, n_remaining, static_cast<cudaStream_t>(stream));
}

int dare_model_step(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int block_start, int L, void* k_cache,
                    void* v_cache, int cache_cap, int mode, float threshold, int k, int32_t* pred, float* conf,
                    int32_t* n_committed, int32_t* n_remaining, void* stream) {
    return dare_model_step_window(m, tokens, B, row_stride, block_start, L, block_start + L, k_cache, v_cache, cache_cap,
                                  mode, threshold, k, pred, conf, n_committed, n_remaining, stream);
}

}  // extern "C"

namespace {

// The previous block's graph: destroyed once its launches are known to have finished.
struct BlockGraph {
    cudaGraph_t graph = nullptr;
    cudaGraphExec_t exec = nullptr;
    void destroy() {
        if (exec) cudaGraphExecDestroy(exec);
        if (graph) cudaGraphDestroy(graph);
        exec = nullptr; graph = nullptr;
    }
};

// All denoising steps of one block on the model's work stream.  The step (about forty launches with fixed
// arguments) is captured once into a CUDA graph and replayed.
//
// A step whose block holds no mask any more does exactly what the refresh forward of the prefix-cache loop
// must do (the LM head finds no live row, the selection changes nothing, the stack rewrites the block's K/V
// from the committed tokens).  So step t + 1 is enqueued before step t's counts are read: when step t turns
// out to have finished the block, step t + 1 was the refresh, and the GPU never waits for the host.  (In the
// dual-cache loop that extra step is redundant and harmless: the next whole-sequence refresh rewrites the
// same K/V.)
int run_block(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int start, int L, int kv_len, void* k_cache,
              void* v_cache, int cap, int mode, float threshold, int k, int32_t* pred, float* conf, int32_t* n_remaining,
              BlockGraph* old, int* steps_taken) {
    cudaStream_t s = m->work;
    BlockGraph cur;
    if (cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return DARE_ERR_CUDA;
    const uint64_t launches_before = dare::g_kernel_launches.load();      // the capture itself launches nothing:
    int rc = step_rows(m, tokens, B, row_stride, start, L, kv_len, k_cache, v_cache, cap, mode, threshold, k, pred, conf,
                       nullptr, n_remaining, s);
    const uint64_t per_replay = dare::g_kernel_launches.load() - launches_before;
    dare::g_kernel_launches.fetch_sub(per_replay);                        // ... its kernels are counted per replay
    const cudaError_t end = cudaStreamEndCapture(s, &cur.graph);      // always ends the capture, also after an error
    if (rc == DARE_OK && (end != cudaSuccess || cur.graph == nullptr)) rc = DARE_ERR_CUDA;
    if (rc == DARE_OK && cudaGraphInstantiate(&cur.exec, cur.graph, 0) != cudaSuccess) rc = DARE_ERR_CUDA;
    int issued = 0, taken = -1;
    while (rc == DARE_OK && taken < 0) {
        if (issued > L + 1) { rc = DARE_ERR_CUDA; break; }   // cannot happen: every step commits a token per row
        const int slot = issued & 1;
        if (cudaGraphLaunch(cur.exec, s) != cudaSuccess ||
            cudaMemcpyAsync(m->host_counts + slot * m->max_batch, n_remaining, sizeof(int32_t) * B,
                            cudaMemcpyDeviceToHost, s) != cudaSuccess ||
            cudaEventRecord(m->ev[slot], s) != cudaSuccess) {
            rc = DARE_ERR_CUDA;
            break;
        }
        ++issued;
        dare::note_launch(per_replay);
        if (issued >= 2) {
            const int prev = (issued - 2) & 1;
            if (cudaEventSynchronize(m->ev[prev]) != cudaSuccess) { rc = DARE_ERR_CUDA; break; }
            old->destroy();      // a step of this block has finished, so every launch of the previous block has
            bool done = true;
            for (int r = 0; r < B; ++r) done = done && m->host_counts[prev * m->max_batch + r] == 0;
            if (done) taken = issued - 1;   // steps 0 .. issued-2 denoised; the last one issued found no mask
        }
    }
    if (old->exec) {      // (only if this block issued fewer than two steps or failed)
        cudaStreamSynchronize(s);
        old->destroy();
    }
    *old = cur;
    *steps_taken = taken;
    return rc;
}

// Order the model's work stream after the caller's stream (entry) / the caller's stream after it (exit).
int enter_work_stream(dare_model* m, cudaStream_t user) {
    if (cudaEventRecord(m->ev_in, user) != cudaSuccess || cudaStreamWaitEvent(m->work, m->ev_in, 0) != cudaSuccess)
        return DARE_ERR_CUDA;
    return DARE_OK;
}
int leave_work_stream(dare_model* m, cudaStream_t user, BlockGraph* old, int rc) {
    const bool synced = cudaStreamSynchronize(m->work) == cudaSuccess;
    old->destroy();
    if (rc != DARE_OK) return rc;
    if (!synced || cudaEventRecord(m->ev_out, m->work) != cudaSuccess ||
        cudaStreamWaitEvent(user, m->ev_out, 0) != cudaSuccess)
        return DARE_ERR_CUDA;
    return DARE_OK;
}

}  // namespace

extern "C" {

// The loops run on the model's own stream, ordered after the caller's stream at entry and before it at exit:
// the caller's stream (possibly the legacy default stream) may not allow a capture.

int dare_generate(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int prompt_len, int gen_len, int L,
                  void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k, int32_t* pred,
                  float* conf, int32_t* n_remaining, int32_t* steps_per_block, void* stream) {
    if (!n_remaining) return DARE_ERR_NULL;
    if (gen_len < 1 || L < 1 || gen_len % L != 0) return DARE_ERR_SHAPE;
    int rc = check_rows(m, tokens, B, row_stride, 0, prompt_len, prompt_len, k_cache, v_cache, cache_cap);
    if (rc == DARE_OK)
        rc = check_rows(m, tokens, B, row_stride, prompt_len + gen_len - L, L, prompt_len + gen_len, k_cache, v_cache,
                        cache_cap);
    if (rc == DARE_OK) rc = check_step(m, B, L, mode, threshold, k, pred, conf);
    if (rc != DARE_OK) return rc;
    cudaStream_t user = static_cast<cudaStream_t>(stream);
    rc = enter_work_stream(m, user);
    if (rc != DARE_OK) return rc;
    rc = forward_rows(m, tokens, B, row_stride, 0, prompt_len, prompt_len, k_cache, v_cache, cache_cap, nullptr, m->work);
    BlockGraph old;
    for (int b = 0; b < gen_len / L && rc == DARE_OK; ++b) {
        const int start = prompt_len + b * L;
        int taken = -1;
        if (m->sample_temperature > 0.f) {     // step n of block b draws with the counter (b << 16) + n
            set_word_kernel<<<1, 1, 0, m->work>>>(m->step_counter, static_cast<uint32_t>(b) << 16);
            dare::note_launch();
        }
        rc = run_block(m, tokens, B, row_stride, start, L, start + L, k_cache, v_cache, cache_cap, mode, threshold, k,
                       pred, conf, n_remaining, &old, &taken);
        if (rc == DARE_OK && steps_per_block) steps_per_block[b] = taken;
    }
    return leave_work_stream(m, user, &old, rc);
}

int dare_generate_dual(dare_model* m, int32_t* tokens, int B, int64_t row_stride, int prompt_len, int gen_len, int L,
                       void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k, int32_t* pred,
                       float* conf, int32_t* n_remaining, int32_t* steps_per_block, void* stream) {
    if (!n_remaining) return DARE_ERR_NULL;
    if (prompt_len < 0 || gen_len < 1 || L < 1 || gen_len % L != 0) return DARE_ERR_SHAPE;
    const int T = prompt_len + gen_len;
    int rc = check_rows(m, tokens, B, row_stride, 0, T, T, k_cache, v_cache, cache_cap);   // the refresh: all rows
    if (rc == DARE_OK) rc = check_step(m, B, L, mode, threshold, k, pred, conf);
    if (rc != DARE_OK) return rc;
    cudaStream_t user = static_cast<cudaStream_t>(stream);
    rc = enter_work_stream(m, user);
    if (rc != DARE_OK) return rc;
    BlockGraph old;
    for (int b = 0; b < gen_len / L && rc == DARE_OK; ++b) {
        const int start = prompt_len + b * L;
        rc = forward_rows(m, tokens, B, row_stride, 0, T, T, k_cache, v_cache, cache_cap, nullptr, m->work);
        if (rc != DARE_OK) break;
        int taken = -1;
        if (m->sample_temperature > 0.f) {
            set_word_kernel<<<1, 1, 0, m->work>>>(m->step_counter, static_cast<uint32_t>(b) << 16);
            dare::note_launch();
        }
        rc = run_block(m, tokens, B, row_stride, start, L, T, k_cache, v_cache, cache_cap, mode, threshold, k, pred, conf,
                       n_remaining, &old, &taken);
        if (rc == DARE_OK && steps_per_block) steps_per_block[b] = taken;
    }
    return leave_work_stream(m, user, &old, rc);
}

}  // extern "C"
