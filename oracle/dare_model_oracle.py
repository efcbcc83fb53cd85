"""CPU oracle for the end-to-end denoising loop on a small decoder-shaped stack.  TEST INFRASTRUCTURE ONLY.

The paper (Section 3.4, rollout with KV-cache reuse; Section 2.1, "intra-block diffusion with inter-block
autoregression") gives no architecture; the workload names the parts: RMSNorm, RoPE, SwiGLU feed-forward,
untied LM head, no biases.  This module writes that stack out in float64, with an optional rounding to bf16
at exactly the places where the product path stores bf16 in memory, and states the loop twice:

  * ``forward_uncached``  the whole sequence at once under the block-causal visibility rule (the prompt is
    one bidirectional segment; generation block b sees the prompt, blocks < b and itself);
  * ``forward_block_cached`` + ``generate``  the cached loop: a step computes only the current block's rows,
    writes the block's post-RoPE K/V in place behind the prefix and attends to prefix + block; once a block
    has no mask left, one more forward (no LM head) rewrites its K/V from the committed tokens and the
    prefix grows by L.

  * ``generate_dual``  the loop of a fully bidirectional masked model with a prefix AND a suffix cache
    (Section 3.4, rollout with KV-cache reuse): before each block one forward of the whole sequence
    rewrites every position's K/V from the current tokens (the still-masked future blocks included); the
    block's steps then recompute only the block's rows against cached prefix + fresh block + cached suffix.
    The cached K/V outside the block go stale while the block's tokens change: that approximation is the
    algorithm, so the oracle follows its steps; what can be pinned exactly is pinned (a block forward right
    after a refresh reproduces the refresh; one block spanning the whole sequence is the uncached model).

That the two agree step by step is the pin of the cache recurrence (tests/test_oracle_model.py); the stack
itself is pinned against an independently written torch formulation (library attention with a boolean mask,
library rms_norm/silu, RoPE as a complex multiplication).  Nothing here is imported by the product path.

Rounding points (``rounded=True``): RMSNorm outputs; the fused QKV projection; q and k after RoPE;
attention output; the residual stream after each of the two additions (rounded once, after the add);
the SwiGLU product silu(g) * u (g and u themselves are not stored, hence not rounded).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional

import numpy as np

from . import dare_oracle as O


@dataclass
class ModelConfig:
    n_layers: int
    hidden: int          # D
    n_q_heads: int       # Hq
    n_kv_heads: int      # Hkv
    head_dim: int        # d
    ffn: int             # F
    vocab: int           # V
    mask_id: int
    rms_eps: float = 1e-5
    rope_base: float = 10000.0


@dataclass
class LayerWeights:
    wqkv: np.ndarray     # [(Hq + 2 Hkv) d, D]: rows = q heads, then k heads, then v heads
    wo: np.ndarray       # [D, Hq d]
    wg: np.ndarray       # [F, D]
    wu: np.ndarray       # [F, D]
    wd: np.ndarray       # [D, F]


@dataclass
class ModelWeights:
    embedding: np.ndarray          # [V, D]
    layers: List[LayerWeights]
    lm_head: np.ndarray            # [V, D]


def bf16_round(a):
    """Nearest bfloat16 (ties to even) of each element, returned as float64.

    The value is first rounded to float32 (what the product path accumulates in) and then to the 8-bit
    mantissa: add 0x7FFF plus the lowest kept bit, clear the low 16 bits.
    """
    a32 = np.asarray(a, dtype=np.float64).astype(np.float32)
    bits = a32.view(np.uint32).astype(np.uint64)
    rounded = ((bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000).astype(np.uint32)
    out = rounded.view(np.float32).astype(np.float64)
    return np.where(np.isfinite(a32), out, a32.astype(np.float64))


def _r(a, rounded):
    return bf16_round(a) if rounded else a


def rmsnorm(x, eps):
    """x / sqrt(mean(x^2) + eps) over the last axis (weight 1)."""
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps)


def rope(x, positions, base):
    """Rotary position embedding, half-split pairing: channel c pairs with c + d/2.

    x [T, H, d], positions int [T].  angle(p, c) = p * base^(-2c/d) for c in [0, d/2);
    out[c] = x[c] cos - x[c + d/2] sin;  out[c + d/2] = x[c + d/2] cos + x[c] sin.
    """
    T, H, d = x.shape
    half = d // 2
    inv_freq = base ** (-2.0 * np.arange(half, dtype=np.float64) / d)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]      # [T, half]
    cos, sin = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x2 * cos + x1 * sin], axis=-1)


def _split_qkv(qkv, cfg):
    T = qkv.shape[0]
    nq, nk = cfg.n_q_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim
    q = qkv[:, :nq].reshape(T, cfg.n_q_heads, cfg.head_dim)
    k = qkv[:, nq:nq + nk].reshape(T, cfg.n_kv_heads, cfg.head_dim)
    v = qkv[:, nq + nk:].reshape(T, cfg.n_kv_heads, cfg.head_dim)
    return q, k, v


def _ffn(x, lw, cfg, rounded):
    h2 = _r(rmsnorm(x, cfg.rms_eps), rounded)
    g = h2 @ lw.wg.T
    u = h2 @ lw.wu.T
    act = _r(g / (1.0 + np.exp(-g)) * u, rounded)          # silu(g) * u
    return _r(x + act @ lw.wd.T, rounded)


def segment_ids(prompt_len, gen_len, block_len):
    """0 for the prompt, 1 + b for the positions of generation block b."""
    seg = np.zeros(prompt_len + gen_len, dtype=np.int64)
    for j in range(gen_len):
        seg[prompt_len + j] = 1 + j // block_len
    return seg


def forward_uncached(cfg: ModelConfig, wts: ModelWeights, tokens_row, seg, rounded=True):
    """Whole sequence of ONE rollout, every layer, under the block-causal rule.

    tokens_row int [T]; seg int [T] (segment_ids): position i sees position j iff seg[j] <= seg[i].
    Returns (final-norm hidden states [T, D], list of per-layer (k [T,Hkv,d], v [T,Hkv,d]) after RoPE).
    """
    T = len(tokens_row)
    visible = seg[None, :] <= seg[:, None]                 # [T(query), T(key)]
    pos = np.arange(T)
    g = cfg.n_q_heads // cfg.n_kv_heads
    scale = 1.0 / np.sqrt(cfg.head_dim)
    x = wts.embedding[np.asarray(tokens_row)]
    kv = []
    for lw in wts.layers:
        h = _r(rmsnorm(x, cfg.rms_eps), rounded)
        qkv = _r(h @ lw.wqkv.T, rounded)
        q, k, v = _split_qkv(qkv, cfg)
        q = _r(rope(q, pos, cfg.rope_base), rounded)
        k = _r(rope(k, pos, cfg.rope_base), rounded)
        kv.append((k, v))
        o = np.zeros((T, cfg.n_q_heads, cfg.head_dim))
        for hq in range(cfg.n_q_heads):
            s = scale * (q[:, hq] @ k[:, hq // g].T)
            s = np.where(visible, s, -np.inf)
            e = np.exp(s - s.max(axis=1, keepdims=True))
            o[:, hq] = (e / e.sum(axis=1, keepdims=True)) @ v[:, hq // g]
        o = _r(o, rounded).reshape(T, -1)
        x = _r(x + o @ lw.wo.T, rounded)
        x = _ffn(x, lw, cfg, rounded)
    return _r(rmsnorm(x, cfg.rms_eps), rounded), kv


def new_cache(cfg: ModelConfig, batch, cap):
    """Per layer (k, v), each [B, Hkv, cap, d], zero-filled."""
    shp = (batch, cfg.n_kv_heads, cap, cfg.head_dim)
    return [(np.zeros(shp), np.zeros(shp)) for _ in range(cfg.n_layers)]


def forward_block_cached(cfg: ModelConfig, wts: ModelWeights, tokens, start, length, cache, rounded=True, kv_len=None):
    """The rows [start, start + length) of every rollout through the stack, against the cache.

    tokens int [B, row]; cache from new_cache, updated IN PLACE: each layer writes the rows' post-RoPE K/V at
    [start, start + length) and the rows attend to cache[0 : start + length) (everything before `start` is the
    prefix; the rows see each other).  With start = 0 and length = prompt length this is the prefill.
    With kv_len > start + length the rows also see cache[start + length : kv_len) as a suffix whose K/V are
    whatever an earlier forward left there (the dual cache of a fully bidirectional model).
    Returns the final-norm hidden states [B * length, D].
    """
    B = tokens.shape[0]
    end = start + length
    kv_len = end if kv_len is None else kv_len
    assert end <= kv_len <= cache[0][0].shape[2]
    pos = np.arange(start, start + length)
    x = wts.embedding[np.asarray(tokens)[:, start:start + length].reshape(-1)]     # [B*length, D]
    plen = np.full(B, start, dtype=np.int64)
    for li, lw in enumerate(wts.layers):
        kc, vc = cache[li]
        h = _r(rmsnorm(x, cfg.rms_eps), rounded)
        qkv = _r(h @ lw.wqkv.T, rounded)
        qs = np.zeros((B, length, cfg.n_q_heads, cfg.head_dim))
        for r in range(B):
            q, k, v = _split_qkv(qkv[r * length:(r + 1) * length], cfg)
            qs[r] = _r(rope(q, pos, cfg.rope_base), rounded)
            kc[r, :, start:start + length] = np.transpose(_r(rope(k, pos, cfg.rope_base), rounded), (1, 0, 2))
            vc[r, :, start:start + length] = np.transpose(v, (1, 0, 2))
        if kv_len == end:
            o, _ = O.attn_block(qs, kc, vc, plen)          # block stored in place behind the prefix
        else:                                              # ... and the cached suffix behind the block
            o, _ = O.attn_block(qs, kc[:, :, :end], vc[:, :, :end], plen, None, None,
                                kc[:, :, end:kv_len], vc[:, :, end:kv_len], None)
        o = _r(o, rounded).reshape(B * length, -1)
        x = _r(x + o @ lw.wo.T, rounded)
        x = _ffn(x, lw, cfg, rounded)
    return _r(rmsnorm(x, cfg.rms_eps), rounded)


def denoise_step_cached(cfg, wts, tokens, block_start, L, cache, mode, threshold, k, rounded=True):
    """One step of the loop: stack on the block's rows, LM head on the still-masked rows, selection."""
    hidden = forward_block_cached(cfg, wts, tokens, block_start, L, cache, rounded)
    B = tokens.shape[0]
    row_tokens = np.asarray(tokens)[:, block_start:block_start + L].reshape(B * L)
    lm = O.lmhead_confidence(hidden, wts.lm_head, row_tokens, cfg.mask_id, True)
    conf32 = lm["conf"].astype(np.float32)
    tok, nc, nr = O.unmask_select(tokens, block_start, L, lm["pred"], conf32, cfg.mask_id, mode, threshold, k)
    return {"hidden": hidden, "lm": lm, "tokens": tok, "n_committed": nc, "n_remaining": nr}


def generate(cfg, wts, tokens, prompt_len, gen_len, L, mode, threshold, k, rounded=True, on_step=None):
    """The cached loop: prefill, then per block repeat steps until no mask is left, then the refresh forward.

    The batch moves block-synchronously (a block ends when every rollout has committed all of it).
    Returns (tokens int32 [B, row], steps taken per block, cache).  on_step(block, step, tokens_before, result)
    is called after every step if given.
    """
    tok = np.array(tokens, dtype=np.int32, copy=True)
    B = tok.shape[0]
    cache = new_cache(cfg, B, prompt_len + gen_len)
    forward_block_cached(cfg, wts, tok, 0, prompt_len, cache, rounded)
    steps = []
    for b in range(gen_len // L):
        start = prompt_len + b * L
        n = 0
        while (tok[:, start:start + L] == cfg.mask_id).any():
            res = denoise_step_cached(cfg, wts, tok, start, L, cache, mode, threshold, k, rounded)
            if on_step is not None:
                on_step(b, n, tok, res)
            tok = res["tokens"]
            n += 1
        forward_block_cached(cfg, wts, tok, start, L, cache, rounded)   # K/V of the committed block
        steps.append(n)
    return tok, steps, cache


def denoise_step_dual(cfg, wts, tokens, block_start, L, kv_len, cache, mode, threshold, k, rounded=True):
    """One step with both caches: as denoise_step_cached, the block's rows seeing cache[0 : kv_len)."""
    hidden = forward_block_cached(cfg, wts, tokens, block_start, L, cache, rounded, kv_len=kv_len)
    B = tokens.shape[0]
    row_tokens = np.asarray(tokens)[:, block_start:block_start + L].reshape(B * L)
    lm = O.lmhead_confidence(hidden, wts.lm_head, row_tokens, cfg.mask_id, True)
    conf32 = lm["conf"].astype(np.float32)
    tok, nc, nr = O.unmask_select(tokens, block_start, L, lm["pred"], conf32, cfg.mask_id, mode, threshold, k)
    return {"hidden": hidden, "lm": lm, "tokens": tok, "n_committed": nc, "n_remaining": nr}


def generate_dual(cfg, wts, tokens, prompt_len, gen_len, L, mode, threshold, k, rounded=True, on_step=None,
                  on_refresh=None):
    """Dual-cache loop of a fully bidirectional model: per block, refresh every position's K/V with one forward
    of the whole sequence [0, T), T = prompt_len + gen_len, then denoise the block against cache[0 : T) until it
    holds no mask.  Blocks are taken left to right and the batch moves block-synchronously.

    Returns (tokens int32 [B, row], steps per block, cache).  on_refresh(block, tokens, hidden [B * T, D]) and
    on_step(block, step, tokens_before, result) are called if given.
    """
    tok = np.array(tokens, dtype=np.int32, copy=True)
    B = tok.shape[0]
    T = prompt_len + gen_len
    cache = new_cache(cfg, B, T)
    steps = []
    for b in range(gen_len // L):
        start = prompt_len + b * L
        hidden = forward_block_cached(cfg, wts, tok, 0, T, cache, rounded)          # the refresh
        if on_refresh is not None:
            on_refresh(b, tok, hidden)
        n = 0
        while (tok[:, start:start + L] == cfg.mask_id).any():
            res = denoise_step_dual(cfg, wts, tok, start, L, T, cache, mode, threshold, k, rounded)
            if on_step is not None:
                on_step(b, n, tok, res)
            tok = res["tokens"]
            n += 1
        steps.append(n)
    return tok, steps, cache


# ---------------------------------------------------------------------------------------------------------
# The cached loop with the sampled head (RL rollouts draw several different responses per prompt, Section 4.2).

STEP_BLOCK_SHIFT = 16      # generator step counter of step n of block b: (b << 16) + n


def denoise_step_cached_sampled(cfg, wts, tokens, block_start, L, cache, mode, threshold, k, temperature, seed, step,
                                rounded=True, kv_len=None):
    """One step of the loop with temperature + Gumbel-max sampling in place of the argmax (see
    dare_sampling_oracle.lmhead_sample): stack on the block's rows, sampled head on the still-masked rows (the
    generator is keyed by the row's index b * L + i in the block's row list and by `step`), selection on the
    sampled tokens' temperature-1 probabilities."""
    from . import dare_sampling_oracle as SO
    hidden = forward_block_cached(cfg, wts, tokens, block_start, L, cache, rounded, kv_len=kv_len)
    B = tokens.shape[0]
    row_tokens = np.asarray(tokens)[:, block_start:block_start + L].reshape(B * L)
    lm = SO.lmhead_sample(hidden, wts.lm_head, row_tokens, cfg.mask_id, True, temperature, seed, step)
    conf32 = lm["conf"].astype(np.float32)
    tok, nc, nr = O.unmask_select(tokens, block_start, L, lm["pred"], conf32, cfg.mask_id, mode, threshold, k)
    return {"hidden": hidden, "lm": lm, "tokens": tok, "n_committed": nc, "n_remaining": nr}


def generate_sampled(cfg, wts, tokens, prompt_len, gen_len, L, mode, threshold, k, temperature, seed, rounded=True,
                     on_step=None):
    """`generate` with the sampled head; step n of block b uses the generator step counter (b << 16) + n."""
    tok = np.array(tokens, dtype=np.int32, copy=True)
    B = tok.shape[0]
    cache = new_cache(cfg, B, prompt_len + gen_len)
    forward_block_cached(cfg, wts, tok, 0, prompt_len, cache, rounded)
    steps = []
    for b in range(gen_len // L):
        start = prompt_len + b * L
        n = 0
        while (tok[:, start:start + L] == cfg.mask_id).any():
            res = denoise_step_cached_sampled(cfg, wts, tok, start, L, cache, mode, threshold, k, temperature, seed,
                                              (b << STEP_BLOCK_SHIFT) + n, rounded)
            if on_step is not None:
                on_step(b, n, tok, res)
            tok = res["tokens"]
            n += 1
        forward_block_cached(cfg, wts, tok, start, L, cache, rounded)   # K/V of the committed block
        steps.append(n)
    return tok, steps, cache
