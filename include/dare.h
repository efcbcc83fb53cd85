/*
 * dare.h -- C ABI of the B200 (sm_100a) rollout denoising step for diffusion LLMs.
 *
 * One denoising step of the cached rollout the paper describes in Section 3.4
 * ("Rollout-side optimization for MDLMs": KV-cache reuse and repeated denoising on
 * partially fixed states) and Section 2.1 (block diffusion: bidirectional inside a
 * block, earlier blocks fixed):
 *
 *     dare_attn_block         block queries x (prefix cache + block + optional suffix cache), GQA
 *     dare_lmhead_confidence  LM head + vocabulary softmax -> (argmax token, max probability) per row,
 *                             logits never written to memory
 *     dare_unmask_select      confidence-threshold / per-block top-k commit on the int32 token state
 *     dare_denoise_block      the three above in one call (dare_denoise_block_sampled: with the sampled head)
 *     dare_model_* / dare_generate   the same step with a stack of transformer layers in between, and the
 *                             whole block-by-block loop (dare_linear, dare_rmsnorm, dare_rope_kv_write: its parts)
 *     dare_model_*_window / dare_generate_dual   the same with a cached suffix behind the block (dual cache)
 *     dare_lmhead_sample      the LM head with temperature + Gumbel-max sampling instead of the argmax
 *     dare_lmhead_logprob     log-probability of given tokens (cross-entropy), logits never written either
 *     dare_lmhead_logprob_backward   its gradient with respect to the hidden states and the weights
 *     dare_attn_varlen        bidirectional attention over packed variable-length sequences
 *     dare_forward_mask, dare_masked_nelbo   the forward (masking) process of Eq. 1 and the bound of Eq. 2
 *
 * Conventions
 *   - Every data pointer is a DEVICE pointer unless the comment says "host".  The caller owns every
 *     buffer; the library neither frees nor keeps them after the call's stream work has run.
 *   - All entry points enqueue work on `stream` (a cudaStream_t passed as void*, NULL = default
 *     stream) and return without synchronising, except where their comment says that they block
 *     (dare_device_status, dare_model_create, dare_generate, dare_generate_dual).  They allocate nothing; the only
 *     allocations are the workspace made once by dare_create and the buffers of dare_model_create.
 *   - bf16 tensors are dense, row-major, 16-byte aligned.
 *   - Return value: DARE_OK (0) or a negative dare_status.  On any error nothing has been launched.
 *   - Data-dependent anomalies (a per-row length beyond its capacity, a wait inside a kernel that
 *     ran out of its bounded time) never trap: they set bits in a device status word that
 *     dare_device_status reads.
 *   - One ctx serves one stream at a time (the workspace is shared by consecutive calls).
 *   - Work is launched on the CURRENT CUDA device, which must be the one the ctx was created on: every entry
 *     point that takes a ctx (or a model) returns DARE_ERR_DEVICE otherwise, before anything is enqueued.
 *     dare_create, dare_destroy, dare_model_create and dare_model_destroy work on the ctx's device and put the
 *     caller's current device back before they return.
 *   - A ctx keeps the TMA tensor maps it has encoded (keyed by base address, shape and tile box; a map depends on
 *     nothing else, so an entry never goes stale): a loop that passes the same buffers every step encodes each
 *     map once.  The kernels' shared-memory limits are likewise raised once per kernel and device.
 */
#ifndef DARE_H_
#define DARE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct dare_ctx dare_ctx;

typedef enum {
    DARE_OK = 0,
    DARE_ERR_NULL = -1,        /* a required pointer is NULL                                   */
    DARE_ERR_SHAPE = -2,       /* unsupported or inconsistent dimensions                       */
    DARE_ERR_ALIGN = -3,       /* pointer not 16-byte aligned / row size not a 16-byte multiple */
    DARE_ERR_RANGE = -4,       /* scalar out of range (k < 1, NaN threshold, mask id, window)   */
    DARE_ERR_WORKSPACE = -5,   /* ctx workspace too small for this call                         */
    DARE_ERR_CUDA = -6,        /* a CUDA runtime/driver call failed                             */
    DARE_ERR_UNSUPPORTED = -7, /* device is not sm_100                                          */
    DARE_ERR_DEVICE = -8       /* the current CUDA device is not the context's (or a buffer's) device */
} dare_status;

/* bits of the device status word */
#define DARE_DEV_LEN_CLAMPED 1u   /* a prefix/suffix length exceeded its capacity and was clamped */
#define DARE_DEV_WAIT_EXPIRED 2u  /* a bounded wait inside a kernel gave up; outputs are invalid  */

enum { DARE_SELECT_THRESHOLD = 0, DARE_SELECT_TOPK = 1 };

/* Create a context on `device` with a workspace of `workspace_bytes` (0 = library default, 256 MiB).
 * *out (host) receives the handle.  Allocates device memory; call outside any stream capture. */
int dare_create(dare_ctx** out, int device, size_t workspace_bytes);
int dare_destroy(dare_ctx* ctx);

/* Counters of the ctx's tensor-map cache since dare_create (HOST pointers): calls that found their map and
 * calls that had to encode one. */
int dare_tmap_cache_stats(const dare_ctx* ctx, uint64_t* hits, uint64_t* misses);

/* Static string for a status code (host pointer, never NULL). */
const char* dare_status_string(int status);

/* Synchronises `stream`, copies the device status word to *host_out (host) and clears it. */
int dare_device_status(dare_ctx* ctx, void* stream, uint32_t* host_out);

/* Number of SMs the ctx's device reports (launch shapes are sized from it). */
int dare_sm_count(const dare_ctx* ctx);

/* Kernels the library has launched in this process since it was loaded, counted on the host at each launch
 * (a step replayed from a CUDA graph counts its kernels once per replay).  Differences of two readings count
 * the launches in between. */
uint64_t dare_kernel_launches(void);

/*
 * Block-bidirectional attention against the caches (Section 2.1; Section 3.4).
 * For every row r, query head h (KV head h / (Hq/Hkv)) and block position i:
 *     o = softmax_j(scale * <q, k_j>) . v_j   over all visible keys j:
 *         prefix [0, prefix_len[r])  U  the block's own L keys  U  suffix [0, suffix_len[r]).
 * No mask inside the visible set (bidirectional).  bf16 in, fp32 accumulate, bf16 out.
 *
 *   q            bf16 [B, L, Hq, d]
 *   k_pre,v_pre  bf16 [B, Hkv, prefix_cap, d]
 *   prefix_len   int32 [B] or NULL (= prefix_cap, or prefix_cap - L when the block is in place)
 *   k_blk,v_blk  bf16 [B, Hkv, L, d]; both NULL => the block's K/V live in k_pre/v_pre at
 *                [prefix_len, prefix_len + L)
 *   k_suf,v_suf  bf16 [B, Hkv, suffix_cap, d] or both NULL (no dual cache)
 *   suffix_len   int32 [B] or NULL (= suffix_cap)
 *   out          bf16 [B, L, Hq, d]
 *   lse          fp32 [B, Hq, L] or NULL: natural-log sum of exp(scale * score)
 *   scale        softmax scale; 0 => 1/sqrt(d)
 * Supported: d in {64, 128}; Hq % Hkv == 0; L >= 1; L * (Hq/Hkv) <= 2^20.
 * Lengths beyond capacity are clamped and flagged in the device status word.
 */
int dare_attn_block(dare_ctx* ctx,
                    int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap, float scale,
                    const void* q,
                    const void* k_pre, const void* v_pre, const int32_t* prefix_len,
                    const void* k_blk, const void* v_blk,
                    const void* k_suf, const void* v_suf, const int32_t* suffix_len,
                    void* out, float* lse, void* stream);

/*
 * Bidirectional attention over packed variable-length sequences (Section 3.4: the training-side and log-prob
 * passes concatenate sequences without padding; each sequence attends to itself only).  Sequence s owns tokens
 * [cu_seqlens[s], cu_seqlens[s + 1]); every token of a sequence sees every token of that sequence.
 *
 *   q    bf16 [total_tokens, Hq, d]      k, v  bf16 [total_tokens, Hkv, d]      out  bf16 [total_tokens, Hq, d]
 *   cu_seqlens   int32 [n_seqs + 1], device, non-decreasing, cu_seqlens[0] = 0, cu_seqlens[n_seqs] = total_tokens
 *   max_seqlen   host value >= the longest sequence (sizes the launch; longer sequences would be cut off)
 *   lse          fp32 [Hq, total_tokens] or NULL
 * Runs on the tcgen05 attention kernel.  Supported: d in {64, 128}; Hq % Hkv == 0, Hq / Hkv <= 128;
 * n_seqs * Hkv <= 65535.  Empty sequences are allowed.
 */
int dare_attn_varlen(dare_ctx* ctx, int total_tokens, int n_seqs, int max_seqlen, int Hq, int Hkv, int d, float scale,
                     const void* q, const void* k, const void* v, const int32_t* cu_seqlens,
                     void* out, float* lse, void* stream);

/*
 * Fused LM head + vocabulary softmax (Section 3.4, the logits-free idea the paper cites for its fused
 * loss kernels, applied to decoding): for each row m,
 *     z = hidden[m] . w^T  (V logits, kept on chip);  z[mask_id] = -inf if exclude_mask_column;
 *     pred[m] = lowest index attaining max z;  conf[m] = exp(max z - logsumexp z).
 *
 *   hidden       bf16 [M, D]        w  bf16 [V, D]  (one row per vocabulary entry)
 *   row_tokens   int32 [M] or NULL: rows whose token != mask_id are already committed and get
 *                pred = that token, conf = -inf
 *   pred         int32 [M] out      conf  fp32 [M] out
 * Only rows that are still masked are evaluated (they are compacted on the device first).
 * Supported: D % 8 == 0, D >= 8; V >= 2; M >= 1.  Needs ctx workspace of 12 * M * min(#SMs, 2 * ceil(V/256))
 * bytes (partial (max, sum, argmax) triples per row), plus 2*M*D + 4*M + 2048 bytes when row_tokens is given.
 */
int dare_lmhead_confidence(dare_ctx* ctx,
                           const void* hidden, int M, int D, const void* w, int V,
                           const int32_t* row_tokens, int32_t mask_id, int exclude_mask_column,
                           int32_t* pred, float* conf, void* stream);

/*
 * Stochastic variant of dare_lmhead_confidence for rollouts that must differ from one another (Section 4.2:
 * several rollouts per prompt).  Per masked row, with z the logits as above:
 *     y_v = z_v / temperature + g_v,   g_v = -ln(-ln u_v),   pred = lowest index attaining max_v y_v
 *     conf = softmax(z)[pred] = exp(z_pred - logsumexp z)          (probability at temperature 1)
 * so pred is a sample of softmax(z / temperature) (Gumbel-max).  The uniforms come from the counter-based
 * generator Philox4x32 with 10 rounds (Salmon et al., SC 2011), key = (seed low word, seed high word), counter =
 * (v / 4, m, step, 0x44415245) where m is the row's index in `hidden`; element v uses output word v % 4, whose top
 * 23 bits k give u_v = (2 k + 1) / 2^24.  The same (seed, step) reproduces the same tokens; callers advance `step`
 * from one denoising step to the next.  Other arguments, skipped rows and limits as dare_lmhead_confidence;
 * temperature > 0; the workspace need is 20 * M * min(#SMs, ceil(V/256)) bytes (+ the row_tokens part).
 */
int dare_lmhead_sample(dare_ctx* ctx,
                       const void* hidden, int M, int D, const void* w, int V,
                       const int32_t* row_tokens, int32_t mask_id, int exclude_mask_column,
                       float temperature, uint64_t seed, uint32_t step,
                       int32_t* pred, float* conf, void* stream);

/*
 * Logits-free log-probability of given tokens (the idea the paper cites for its fused loss kernels, Section 3.4;
 * the rollout's old / reference log-probabilities and the likelihood estimators of Section 4.2 need exactly
 * this): for each row m
 *     logprob[m] = z[targets[m]] - logsumexp z,      z = hidden[m] . w^T,  z[mask_id] = -inf if exclude_mask_column
 * with the logits kept on chip as in dare_lmhead_confidence.  -logprob is the row's cross-entropy.
 *
 *   targets   int32 [M]: a target outside [0, V) (or the excluded column) gives logprob = -inf
 *   logprob   fp32 [M] out          lse  fp32 [M] out or NULL: logsumexp z
 * Every row is evaluated.  Limits as dare_lmhead_confidence; workspace 12 * M * min(#SMs, ceil(V/256)) bytes.
 */
int dare_lmhead_logprob(dare_ctx* ctx,
                        const void* hidden, int M, int D, const void* w, int V,
                        const int32_t* targets, int32_t mask_id, int exclude_mask_column,
                        float* logprob, float* lse, void* stream);

/*
 * Forward (corruption) process, Eq. 1: q(x_t | x_0) = Cat(alpha_t x_0 + (1 - alpha_t) m) with m the <MASK> state.
 * Every token of the window [start, start + length) of row b independently becomes mask_id with probability
 * p_mask[b] = 1 - alpha_t and keeps its value otherwise; tokens outside the window (the prompt) are copied.
 * The uniform of window position i of row b is output word i % 4 of Philox4x32-10 with key = seed and counter =
 * (i / 4, b, sample, 0x4D41534B), mapped to u = (2 k + 1) / 2^24 from its top 23 bits; masked iff u < p_mask[b].
 * `sample` numbers the Monte-Carlo draws (Section 4.2 uses 16 per sequence).
 *   x0  int32 [B, row_stride] in      xt  int32 [B, row_stride] out (may be x0: in place; otherwise only the
 *   window of xt is written)          p_mask  fp32 [B], device
 */
int dare_forward_mask(dare_ctx* ctx, const int32_t* x0, int32_t* xt, int B, int64_t row_stride, int start, int length,
                      const float* p_mask, int32_t mask_id, uint64_t seed, uint32_t sample, void* stream);

/*
 * Per-sequence term of the negative evidence lower bound, Eq. 2, for one draw (x_t, t):
 *     nelbo[b] = -(1 / t[b]) * sum over window positions l with x_t[b, l] = mask_id of logprob[b, l]
 * with logprob[b, l] = log p(x_0[b, l] | x_t) as dare_lmhead_logprob returns it for the window's rows.
 *   logprob  fp32 [B, length]     xt  int32 [B, row_stride]     t  fp32 [B] (device, > 0)
 *   nelbo    fp32 [B] out         n_masked  int32 [B] out or NULL
 */
int dare_masked_nelbo(dare_ctx* ctx, const float* logprob, const int32_t* xt, int B, int64_t row_stride, int start,
                      int length, int32_t mask_id, const float* t, float* nelbo, int32_t* n_masked, void* stream);

/*
 * Parallel unmask selection, in place on the token state (Section 3.4, "partially fixed states";
 * Section 4.2: block length 32, two tokens per step).  Per row, U = block positions whose token is
 * mask_id.  THRESHOLD: commit every i in U with conf > threshold, or the single most confident one
 * (lowest i on ties) if none passes.  TOPK: commit the min(k, #U) most confident (lower i first on
 * ties).  Committed: tokens[r, block_start + i] = pred[r, i].  Everything else is left as it is.
 * Comparisons are in fp32; NaN counts as -inf.
 *
 *   tokens       int32 [B, row_stride] in/out     pred int32 [B, L]     conf fp32 [B, L]
 *   n_committed, n_remaining   int32 [B] out, each may be NULL.  Here, in dare_denoise_block(_sampled) and in
 *                dare_model_step(_dual) these two may also point to page-locked host memory that the device can
 *                address (cudaHostAlloc / cudaHostRegister under unified addressing): the kernel stores the B
 *                integers with plain writes, so the host reads them after synchronising with the stream, without
 *                a copy back.  dare_generate(_dual) need device memory for n_remaining.
 * Supported: 1 <= L <= 4096; 0 <= block_start, block_start + L <= row_stride.
 */
int dare_unmask_select(dare_ctx* ctx,
                       int32_t* tokens, int B, int64_t row_stride, int block_start, int L,
                       const int32_t* pred, const float* conf,
                       int32_t mask_id, int mode, float threshold, int k,
                       int32_t* n_committed, int32_t* n_remaining, void* stream);

/*
 * One whole denoising step: dare_attn_block, dare_lmhead_confidence on the block's rows
 * (row_tokens taken from tokens[:, block_start : block_start + L], M = B * L), then
 * dare_unmask_select.  `hidden` is the LM-head input for the B*L block positions.  pred/conf are
 * caller-provided [B*L] buffers that also serve as the step's intermediate results.
 *
 * Ordering: everything the step reads is taken as `stream` has it when the call is made, and everything it
 * writes (attn_out, lse, pred, conf, tokens, the counts) is complete for whatever is enqueued on `stream`
 * afterwards.  Inside the step the attention and the head, neither of which reads what the other writes, are
 * not kept in sequence: the head runs on a stream of the context, forked from and joined back to `stream` by
 * events, and the attention's CTAs fill the SMs that the head's GEMM leaves early.  `hidden` and attn_out must
 * therefore not overlap (nor any other input of one half with an output of the other).  The fork and the join are
 * capturable in a CUDA graph like any event fork / join.
 */
int dare_denoise_block(dare_ctx* ctx,
                       int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap, float scale,
                       const void* q,
                       const void* k_pre, const void* v_pre, const int32_t* prefix_len,
                       const void* k_blk, const void* v_blk,
                       const void* k_suf, const void* v_suf, const int32_t* suffix_len,
                       void* attn_out, float* lse,
                       const void* hidden, int D, const void* w, int V,
                       int32_t mask_id, int exclude_mask_column,
                       int32_t* tokens, int64_t row_stride, int block_start,
                       int mode, float threshold, int k,
                       int32_t* pred, float* conf,
                       int32_t* n_committed, int32_t* n_remaining, void* stream);

/*
 * The same step with the sampled head (Section 4.2: several different rollouts per prompt): dare_attn_block,
 * dare_lmhead_sample on the block's rows (temperature, seed and step counter as there), then dare_unmask_select on
 * the sampled tokens and their temperature-1 probabilities.  Same buffers, rules and ordering as dare_denoise_block
 * (the head on the context's stream, the attention beside it); temperature must be finite and > 0 (DARE_ERR_RANGE
 * otherwise).
 */
int dare_denoise_block_sampled(dare_ctx* ctx, int B, int L, int Hq, int Hkv, int d, int prefix_cap, int suffix_cap,
                               float scale, const void* q, const void* k_pre, const void* v_pre,
                               const int32_t* prefix_len, const void* k_blk, const void* v_blk, const void* k_suf,
                               const void* v_suf, const int32_t* suffix_len, void* attn_out, float* lse,
                               const void* hidden, int D, const void* w, int V, int32_t mask_id,
                               int exclude_mask_column, float temperature, uint64_t seed, uint32_t step,
                               int32_t* tokens, int64_t row_stride, int block_start, int mode, float threshold, int k,
                               int32_t* pred, float* conf, int32_t* n_committed, int32_t* n_remaining, void* stream);

/*
 * ---------------------------------------------------------------------------------------------------------
 * End-to-end denoising loop on a decoder-shaped stack (the rollout of Section 3.4 with the layers in between;
 * Section 2.1: blocks are bidirectional inside and see the prompt and the earlier blocks).  The paper names no
 * architecture; the stack is pre-norm, without biases: per layer  h = RMSNorm(x);  q, k, v = h Wqkv^T;
 * RoPE(q, k) at the absolute position (channel c pairs with c + d/2, angle = position * base^(-2c/d));
 * block attention against the K/V cache;  x += attn Wo^T;  x += (silu(h2 Wg^T) * (h2 Wu^T)) Wd^T with
 * h2 = RMSNorm(x);  a final RMSNorm feeds the untied LM head.  RMSNorm has unit weight.
 * bf16 is stored after every RMSNorm, after the QKV projection, after RoPE, after attention, after each
 * residual addition (rounded once, after the add) and after the SwiGLU product; everything else is fp32.
 *
 * All weights are bf16, [out features, in features] row-major, 16-byte aligned, caller-owned DEVICE memory
 * that must stay valid while the model exists:
 *   embedding [V, D]; lm_head [V, D]; per layer wqkv [(Hq + 2 Hkv) d, D] (rows: q heads, k heads, v heads),
 *   wo [D, Hq d], wg [F, D], wu [F, D], wd [D, F].
 * K/V cache (caller-owned): k_cache and v_cache are bf16 [n_layers, B, Hkv, cache_cap, d]; position p of a
 * rollout lives at index p.
 */
typedef struct dare_model dare_model;

typedef struct {
    int n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab;
    int32_t mask_id;
    float rms_eps;          /* e.g. 1e-5 */
    float rope_base;        /* e.g. 10000 */
    int max_positions;      /* largest cache_cap any call will use (size of the RoPE table) */
    int max_rows;           /* largest B * length one forward processes (B * prompt length for the prefill) */
    int max_batch;          /* largest B */
} dare_model_desc;

typedef struct {
    const void *wqkv, *wo, *wg, *wu, *wd;   /* device pointers */
} dare_layer_weights;

/* Creates the model object: copies `layers` (HOST array of n_layers entries), allocates the activation
 * buffers for max_rows rows and builds the RoPE table.  Allocates and synchronises: call at set-up time.
 * The ctx must outlive the model and serves one stream at a time together with it. */
int dare_model_create(dare_ctx* ctx, const dare_model_desc* desc, const void* embedding,
                      const dare_layer_weights* layers, const void* lm_head, dare_model** out);
int dare_model_destroy(dare_model* model);

/*
 * Building blocks of the stack, exported so that each can be checked on its own.  All enqueue on `stream`.
 *
 * dare_linear:  out[M, N] = epilogue(a[M, K] . w[N, K]^T), bf16 row-major operands, fp32 accumulation.
 *   epilogue DARE_LINEAR_STORE:    out = acc
 *            DARE_LINEAR_RESIDUAL: out = residual + acc, rounded once (residual bf16 [M, N]; may be `out`)
 *            DARE_LINEAR_SWIGLU:   out = silu(a . w^T) * (a . w2^T)   (w, w2 both [N, K])
 *   Supported: N, K multiples of 8; pointers 16-byte aligned.
 * dare_rmsnorm: y[m, :] = x[m, :] / sqrt(mean(x[m, :]^2) + eps)   (x, y bf16 [n_rows, D], D % 8 == 0).
 * dare_rope_kv_write: row m = (b, i) of qkv [B * length, (Hq + 2 Hkv) d] at position start + i:
 *   q heads rotated -> q_out [B * length, Hq, d]; k heads rotated -> k_cache[b, :, start + i, :];
 *   v heads copied -> v_cache[b, :, start + i, :]  (caches bf16 [B, Hkv, cache_cap, d], one layer).
 */
enum { DARE_LINEAR_STORE = 0, DARE_LINEAR_RESIDUAL = 1, DARE_LINEAR_SWIGLU = 2 };
int dare_linear(dare_ctx* ctx, int epilogue, const void* a, int M, int K, const void* w, const void* w2, int N,
                void* out, const void* residual, void* stream);
/* The launch shape dare_linear picks for a problem (no launch): plan_out (HOST int[8]) = {row tiles per work
 * item, W rows per tile, output columns per tile, CTAs along K per output tile, pipeline stages, row items,
 * column tiles, clusters resident at once}.  M > 128: a work item is a PAIR of CTAs (a cluster of two) that
 * computes two row tiles with 256-row MMAs; entry 3 is the number of pairs along K (1 or 2; two pairs form a
 * cluster of four CTAs) and entry 7 the number of such clusters resident at once.
 * M <= 128: one CTA per (row tile, column tile, K slice); the K slices of a tile form a cluster and entry 7
 * is 0 without a K split. */
int dare_linear_plan(dare_ctx* ctx, int epilogue, int M, int K, int N, int* plan_out);
int dare_rmsnorm(dare_ctx* ctx, const void* x, int n_rows, int D, float eps, void* y, void* stream);
int dare_rope_kv_write(dare_model* model, const void* qkv, int B, int length, int start, void* q_out,
                       void* k_cache, void* v_cache, int cache_cap, void* stream);

/*
 * The rows [start, start + length) of every rollout through the whole stack: their post-RoPE K/V are
 * written into the cache at [start, start + length) and they attend to cache[0, start + length).
 * start = 0, length = prompt length is the prefill; start = a block's first position, length = L is the
 * refresh of a finished block.  tokens int32 [B, row_stride] (read only).  hidden_out: bf16
 * [B * length, D] final-RMSNorm hidden states, or NULL.  Enqueues on `stream`, no synchronisation.
 */
int dare_model_forward(dare_model* model, const int32_t* tokens, int B, int64_t row_stride, int start, int length,
                       void* k_cache, void* v_cache, int cache_cap, void* hidden_out, void* stream);

/*
 * One denoising step of block [block_start, block_start + L): dare_model_forward on the block's rows, the
 * LM head on the rows that are still masked, the unmask selection in place on `tokens`.
 * pred int32 [B * L], conf fp32 [B * L] (results of the step), n_committed / n_remaining int32 [B] or NULL.
 * Enqueues on `stream`, no synchronisation.
 */
int dare_model_step(dare_model* model, int32_t* tokens, int B, int64_t row_stride, int block_start, int L,
                    void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k,
                    int32_t* pred, float* conf, int32_t* n_committed, int32_t* n_remaining, void* stream);

/*
 * The whole loop: prefill of tokens[:, 0 : prompt_len], then for each block of L positions steps are repeated
 * until no rollout has a mask left in it (the batch moves block by block), then the block's K/V are refreshed
 * from the committed tokens and the prefix grows by L.  The host reads the per-step mask counts one step
 * behind the GPU, so the GPU never waits for it.  steps_per_block: HOST int32 [gen_len / L] or NULL.
 * n_remaining: device int32 [B] (scratch and last counts).  This call BLOCKS until the loop has finished.
 */
int dare_generate(dare_model* model, int32_t* tokens, int B, int64_t row_stride, int prompt_len, int gen_len, int L,
                  void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k,
                  int32_t* pred, float* conf, int32_t* n_remaining, int32_t* steps_per_block, void* stream);

/*
 * Backward of dare_lmhead_logprob (Section 3.4: the actor update differentiates the per-token log-probabilities;
 * the logits are recomputed, never stored).  For L = sum_m grad_logprob[m] * logprob[m]:
 *     dz[m, v]  = grad_logprob[m] * (1[v = targets[m]] - exp(z[m, v] - lse[m]))   (0 in the excluded column;
 *                 a row whose target is outside [0, V) or is the excluded column gets dz = 0)
 *     d_hidden  = dz . w           bf16 [M, D]
 *     d_w       = dz^T . hidden    bf16 [V, D]
 * hidden bf16 [M, D]; w bf16 [V, D]; w_t bf16 [D, V] = the transpose of w, kept by the caller (dare_transpose_bf16
 * makes it; it changes only when the weights do); targets int32 [M]; lse fp32 [M] = the logsumexp that
 * dare_lmhead_logprob returned for the same inputs; grad_logprob fp32 [M].
 * dz bf16 [M, V] and dzt bf16 [V, M]: caller-provided scratch for the gradient of the logits in both orientations
 * (2 * M * V * 2 bytes together: the caller bounds them by the rows it passes per call; d_w of several calls add up
 * on the caller's side).  Products accumulate in fp32 and are rounded to bf16 once.
 * Supported: M, D, V multiples of 8; the ctx workspace must hold M * D * 2 bytes (DARE_ERR_WORKSPACE otherwise).
 * Enqueues on `stream`, no synchronisation.
 *
 * dare_transpose_bf16: out [cols, rows] = transpose of in [rows, cols] (bf16, dense, out != in, rows <= 2 097 120).
 */
int dare_lmhead_logprob_backward(dare_ctx* ctx, const void* hidden, int M, int D, const void* w, const void* w_t,
                                 int V, const int32_t* targets, int32_t mask_id, int exclude_mask_column,
                                 const float* lse, const float* grad_logprob, void* dz, void* dzt, void* d_hidden,
                                 void* d_w, void* stream);
int dare_transpose_bf16(dare_ctx* ctx, const void* in, int rows, int cols, void* out, void* stream);

/*
 * Sampled head for the model calls (Section 4.2: several different rollouts per prompt).  After
 * dare_model_set_sampling(model, temperature > 0, seed, first_step, stream), dare_model_step, dare_model_step_window,
 * dare_generate and dare_generate_dual draw every masked row's token by temperature + Gumbel-max sampling
 * (dare_lmhead_sample; confidence = temperature-1 probability of the drawn token) instead of taking the argmax.
 * The generator's step counter lives on the device: the call sets it to first_step (enqueued on `stream`) and
 * every step adds one, so consecutive dare_model_step calls use first_step, first_step + 1, ...; the loops set it to
 * (block index << 16) at the start of each block, so step n of block b uses (b << 16) + n.  The generator's row
 * index is the row's index b * L + i among the block's rows.  temperature = 0 switches back to the argmax (the
 * default); negative, NaN or infinite values give DARE_ERR_RANGE.  The ctx workspace must cover the sampled head
 * (5 instead of 3 floats per partial), else the step calls return DARE_ERR_WORKSPACE.
 */
int dare_model_set_sampling(dare_model* model, float temperature, uint64_t seed, uint32_t first_step, void* stream);

/*
 * Dual cache (prefix and suffix) for a fully bidirectional masked model (Section 3.4, rollout with KV-cache
 * reuse): the rows [start, start + length) see cache[0 : kv_len) with kv_len >= start + length, i.e. also the
 * positions behind them, whose K/V are whatever an earlier forward left in the cache.
 *   dare_model_forward_window / dare_model_step_window: as dare_model_forward / dare_model_step with that extra
 *     argument (kv_len = start + length gives exactly those calls).  start + length <= kv_len <= cache_cap, else
 *     DARE_ERR_RANGE.  Enqueue on `stream`, no synchronisation.
 *   dare_generate_dual: for each block of L positions, first one forward of ALL rows [0, T), T = prompt_len +
 *     gen_len, seeing all of cache[0 : T) (this rewrites every position's K/V from the current tokens, the still
 *     masked later blocks included), then the block's steps against cache[0 : T) until no rollout has a mask
 *     left in it.  K/V outside the block are therefore as old as the last refresh while the block's tokens
 *     change: that staleness is the method's approximation.  The model needs max_rows >= B * T
 *     (DARE_ERR_SHAPE otherwise); prompt_len may be 0.  On return the cache holds, for each position, the K/V of
 *     the last forward that covered it.  Other arguments as dare_generate.  This call BLOCKS until the loop has
 *     finished.
 */
int dare_model_forward_window(dare_model* model, const int32_t* tokens, int B, int64_t row_stride, int start,
                              int length, int kv_len, void* k_cache, void* v_cache, int cache_cap, void* hidden_out,
                              void* stream);
int dare_model_step_window(dare_model* model, int32_t* tokens, int B, int64_t row_stride, int block_start, int L,
                           int kv_len, void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k,
                           int32_t* pred, float* conf, int32_t* n_committed, int32_t* n_remaining, void* stream);
int dare_generate_dual(dare_model* model, int32_t* tokens, int B, int64_t row_stride, int prompt_len, int gen_len,
                       int L, void* k_cache, void* v_cache, int cache_cap, int mode, float threshold, int k,
                       int32_t* pred, float* conf, int32_t* n_remaining, int32_t* steps_per_block, void* stream);

/*
 * Allocation-free variant of dare_lmhead_confidence.  (The paper has no counterpart for this entry
 * point; it exists for callers of this library that are not allowed to allocate device memory.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- inside another framework's allocator
 * or memory-budget hooks, in a plug-in that does not own the process's memory pool, or at a point of a
 * program where allocation would synchronise or fail.  Such callers cannot hold a dare_ctx, because
 * dare_create allocates the workspace.  Here the per-tile scratch of the LM head lives in a fixed array
 * of DARE_LMHEAD_STATIC_SCRATCH_BYTES inside the library's device image, which every GPU that loads the
 * library keeps resident until the process exits.  The call allocates nothing and frees nothing.
 *
 * Same arguments, results and arithmetic as dare_lmhead_confidence, without the ctx; it runs on the
 * CURRENT device.  Limits and rules:
 *   - The scratch the call needs (12 * M * min(#SMs, 2 * ceil(V/256)) bytes, plus 2*M*D + 4*M + 2048 bytes when
 *     row_tokens is given) must not exceed DARE_LMHEAD_STATIC_SCRATCH_BYTES, else DARE_ERR_WORKSPACE is
 *     returned and nothing is launched (use the ctx variant for larger problems).
 *   - The first call on each device looks up the device address of the scratch array and a driver entry
 *     point; make that first call before starting any stream capture.
 *   - All calls on a device share the one scratch array.  Nothing in it needs to start at zero: in a call
 *     that runs to completion every entry that is read has been written by that call.  Two calls whose GPU
 *     work overlaps (different streams, or several host threads) race on it: serialise them on one stream.
 *   - hidden, w, row_tokens, pred and conf must live on the current device (DARE_ERR_DEVICE otherwise).
 *   - Data-dependent status bits of this variant go to a word inside the library that
 *     dare_lmhead_static_status reads.  If DARE_DEV_WAIT_EXPIRED is set there, a bounded wait inside the
 *     kernel gave up: parts of the scratch were then NOT written by that call and its pred / conf may have
 *     been folded from an earlier call's leftovers -- discard them.
 */
#define DARE_LMHEAD_STATIC_SCRATCH_BYTES (8u << 20)
int dare_lmhead_confidence_static(const void* hidden, int M, int D, const void* w, int V,
                                  const int32_t* row_tokens, int32_t mask_id, int exclude_mask_column,
                                  int32_t* pred, float* conf, void* stream);
/* Synchronises `stream`, copies the status word of the allocation-free calls on the current device to
 * *host_out (host) and clears it.  Allocates nothing. */
int dare_lmhead_static_status(void* stream, uint32_t* host_out);

#ifdef __cplusplus
}
#endif
#endif /* DARE_H_ */
