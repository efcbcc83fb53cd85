"""CPU oracle for the stochastic rollout epilogue (temperature + Gumbel-max sampling).  TEST INFRASTRUCTURE ONLY.

RL rollouts need several different samples per prompt (Section 4.2: rollout group size 8), so the denoising
step is also offered with a sampled instead of a greedy prediction: for each masked row

    y_v = z_v / T + g_v,   g_v = -ln(-ln u_v),   token = lowest index attaining max_v y_v,
    confidence = softmax(z)_token = exp(z_token - logsumexp z)        (temperature 1, raw logits)

where z are the LM-head logits (mask column excluded as in the greedy head) and u_v are uniforms in (0, 1).
By the Gumbel-max property the token is a sample of softmax(z / T).  The uniforms cannot be passed in (there
are M * V of them per step), so both sides implement one counter-based generator from its published
definition: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2,
3", SC 2011).  The counter is (v // 4, row, step, 0x44415245), the key the two halves of a 64-bit seed; element
v takes output word v % 4; its top 23 bits k give u = (2 k + 1) / 2^24, which is exact in float32.

Pins (tests/test_oracle_sampling.py): the generator against the known-answer vectors distributed with its
reference implementation; the uniforms' range and exactness in float32; the Gumbel moments; the sampling law
(token frequencies follow softmax(z / T)); T -> 0 recovers the greedy head; determinism in (seed, row, step);
perturbed_score against the sampled head's own winning score, rebuilt from the uniforms, and its row / step / seed
keys; denoise_step_sampled as the composition of the separately pinned attention, sampled head and selection, its
step invariants, and its T -> 0 limit (the greedy step); the forward process' marginals and window; the bound's
term on a hand-worked case.
"""
from __future__ import annotations

import numpy as np

from . import dare_oracle as O

PHILOX_M0 = np.uint64(0xD2511F53)
PHILOX_M1 = np.uint64(0xCD9E8D57)
PHILOX_W0 = np.uint32(0x9E3779B9)
PHILOX_W1 = np.uint32(0xBB67AE85)
COUNTER_TAG = 0x44415245
MASK32 = np.uint64(0xFFFFFFFF)


def philox4x32_10(counter, key):
    """Philox4x32-10.  counter: uint32 array [..., 4]; key: uint32 array [..., 2] (broadcastable).  Returns [..., 4].

    One round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2 (32 x 32 -> 64 bit products);
    c' = (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); between rounds the key is bumped by the Weyl constants.
    """
    c = np.array(np.broadcast_arrays(counter)[0], dtype=np.uint32, copy=True)
    k = np.array(key, dtype=np.uint32, copy=True)
    k = np.broadcast_to(k, c.shape[:-1] + (2,)).copy()
    c0, c1, c2, c3 = (c[..., i].copy() for i in range(4))
    k0, k1 = k[..., 0].copy(), k[..., 1].copy()
    for _ in range(10):
        p0 = PHILOX_M0 * c0.astype(np.uint64)
        p1 = PHILOX_M1 * c2.astype(np.uint64)
        hi0, lo0 = (p0 >> np.uint64(32)).astype(np.uint32), (p0 & MASK32).astype(np.uint32)
        hi1, lo1 = (p1 >> np.uint64(32)).astype(np.uint32), (p1 & MASK32).astype(np.uint32)
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = ((k0.astype(np.uint64) + np.uint64(PHILOX_W0)) & MASK32).astype(np.uint32)
        k1 = ((k1.astype(np.uint64) + np.uint64(PHILOX_W1)) & MASK32).astype(np.uint32)
    return np.stack([c0, c1, c2, c3], axis=-1)


def uniforms(seed, row, step, V):
    """u_v in (0, 1) for v in [0, V) of one (row, step): exact multiples of 2^-24, never 0 or 1."""
    n4 = (V + 3) // 4
    counter = np.zeros((n4, 4), dtype=np.uint32)
    counter[:, 0] = np.arange(n4, dtype=np.uint32)
    counter[:, 1] = np.uint32(row)
    counter[:, 2] = np.uint32(step)
    counter[:, 3] = np.uint32(COUNTER_TAG)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    words = philox4x32_10(counter, key).reshape(-1)[:V]
    k = (words >> np.uint32(9)).astype(np.float64)                 # top 23 bits
    return (2.0 * k + 1.0) / 16777216.0


def gumbel(u):
    """Standard Gumbel noise from a uniform: -ln(-ln u)."""
    return -np.log(-np.log(u))


def lmhead_sample(x, w, row_tokens=None, mask_id=-1, exclude_mask_column=True, temperature=1.0, seed=0, step=0):
    """Sampled LM head.  x [M, D], w [V, D] float64.  Rows whose row_tokens entry is not the mask id are skipped
    (pred = that token, conf = -inf), exactly as in the greedy head; the row index that keys the generator is the
    row's index in x.

    Returns dict: pred int32 [M]; conf float64 [M] = softmax(z)[pred]; logconf; gap_y float64 [M] = distance of
    the best perturbed score to the runner-up (to judge near-ties); y_best float64 [M].
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    M, V = x.shape[0], w.shape[0]
    pred = np.zeros(M, dtype=np.int32)
    conf = np.full(M, -np.inf)
    logconf = np.full(M, -np.inf)
    gap = np.full(M, np.inf)
    ybest = np.full(M, -np.inf)
    for m in range(M):
        if row_tokens is not None and row_tokens[m] != mask_id:
            pred[m] = row_tokens[m]
            continue
        z = w @ x[m]
        if exclude_mask_column and 0 <= mask_id < V:
            z[mask_id] = -np.inf
        y = z / temperature + gumbel(uniforms(seed, m, step, V))
        t = int(np.argmax(y))                                      # first (lowest) index of the maximum
        zmax = z.max()
        lse = zmax + np.log(np.exp(z - zmax).sum())
        pred[m] = t
        logconf[m] = z[t] - lse
        conf[m] = np.exp(logconf[m])
        y2 = y.copy()
        y2[t] = -np.inf
        gap[m] = y[t] - y2.max()
        ybest[m] = y[t]
    return {"pred": pred, "conf": conf, "logconf": logconf, "gap_y": gap, "y_best": ybest}


def perturbed_score(x_row, w, token, row, mask_id=-1, exclude_mask_column=True, temperature=1.0, seed=0, step=0):
    """y_token of one row (used to judge whether a differing token was a near-tie)."""
    z = np.asarray(w, dtype=np.float64) @ np.asarray(x_row, dtype=np.float64)
    if exclude_mask_column and 0 <= mask_id < z.shape[0]:
        z[mask_id] = -np.inf
    return float(z[token] / temperature + gumbel(uniforms(seed, row, step, z.shape[0]))[token])


def denoise_step_sampled(q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len, x, w, tokens, block_start,
                         L, mask_id, mode, threshold, k, temperature, seed, step, exclude_mask_column=True):
    """One denoising step with the sampled head in place of the greedy one (attention and selection unchanged)."""
    o, lse = O.attn_block(q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len)
    B = tokens.shape[0]
    row_tokens = np.asarray(tokens)[:, block_start:block_start + L].reshape(B * L)
    lm = lmhead_sample(x, w, row_tokens, mask_id, exclude_mask_column, temperature, seed, step)
    tok, nc, nr = O.unmask_select(tokens, block_start, L, lm["pred"], lm["conf"].astype(np.float32), mask_id, mode,
                                  threshold, k)
    return {"attn_out": o, "lse": lse, "lm": lm, "tokens": tok, "n_committed": nc, "n_remaining": nr}


# ---------------------------------------------------------------------------------------------------------
# Forward (corruption) process and the Monte-Carlo likelihood bound that uses it.

MASK_TAG = 0x4D41534B


def forward_mask(x0, start, length, p_mask, mask_id, seed, sample):
    """Eq. 1 (forward process with the absorbing <MASK> state): each token of the window [start, start + length)
    of row b independently stays x_0 with probability alpha_t = 1 - p_mask[b] and becomes <MASK> otherwise;
    tokens outside the window (the prompt) are kept.

    The uniform of position i of row b is word i % 4 of Philox4x32-10(counter = (i // 4, b, sample, MASK_TAG),
    key = seed), mapped to u = (2 k + 1) / 2^24 as in `uniforms`; the token is masked iff u < p_mask[b]
    (compared in float32: u is exact there).  Returns a new int32 array.
    """
    x = np.array(x0, dtype=np.int32, copy=True)
    B = x.shape[0]
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint32)
    n4 = (length + 3) // 4
    for b in range(B):
        counter = np.zeros((n4, 4), dtype=np.uint32)
        counter[:, 0] = np.arange(n4, dtype=np.uint32)
        counter[:, 1] = np.uint32(b)
        counter[:, 2] = np.uint32(sample)
        counter[:, 3] = np.uint32(MASK_TAG)
        words = philox4x32_10(counter, key).reshape(-1)[:length]
        u = ((2.0 * (words >> np.uint32(9)).astype(np.float64) + 1.0) / 16777216.0).astype(np.float32)
        hit = u < np.float32(p_mask[b])
        x[b, start:start + length][hit] = mask_id
    return x


def masked_nelbo(logprob, xt, start, length, mask_id, t):
    """Eq. 2, the per-sequence term of the negative evidence lower bound for one (x_t, t) draw:
        nelbo[b] = -(1 / t[b]) * sum over window positions l with x_t[b, l] = <MASK> of log p(x_0[b, l] | x_t).
    logprob float [B, length] holds log p(x_0^l | x_t) for every window position (entries at unmasked positions are
    ignored).  Returns (nelbo float64 [B], n_masked int32 [B])."""
    lp = np.asarray(logprob, dtype=np.float64).reshape(len(t), length)
    m = np.asarray(xt)[:, start:start + length] == mask_id
    s = np.where(m, lp, 0.0).sum(axis=1)
    return -s / np.asarray(t, dtype=np.float64), m.sum(axis=1).astype(np.int32)
