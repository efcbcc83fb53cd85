"""CPU oracle for the dLLM rollout denoising step.  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 statement of what one denoising step of the cached rollout
computes (paper Section 3.4, "Rollout-side optimization for MDLMs": repeated
denoising on partially fixed states with KV-cache reuse; Section 2.1, block
structure: bidirectional inside a block, earlier blocks fixed).  Only tests,
the smoke check and the benchmark's CPU-baseline leg may import this module;
the product path never does, and this module imports nothing of the product.

The paper prints no formula for the step, so each function writes out the
textbook definition the step reaches exactly (softmax attention over the
visible keys; softmax over the vocabulary; a selection rule), with the
readings listed in the design notes.  numpy matmul is used as a library step;
there is no tiling, streaming or fusion here.

Pins (tests/test_oracle_*.py): attention against a library full-sequence
attention with an explicit boolean mask, closed forms and invariances;
LM head against library log-softmax, closed forms (uniform logits, planted
column); selection against a brute-force sort, counting invariants and
hand-written cases under tests/golden/.  Numeric values on the five
workloads themselves are not printed by the paper: "parity unpinned" by the
paper for those values; they are pinned only through the checks above.
"""
from __future__ import annotations

import numpy as np

SELECT_THRESHOLD = 0
SELECT_TOPK = 1


def _visible_keys(k_pre, v_pre, P, k_blk, v_blk, L, k_suf, v_suf, S):
    """Concatenate the keys/values a block query may see: prefix [0,P), the block itself, suffix [0,S).

    Section 2.1 (block diffusion): a block conditions on the preceding blocks and on itself; the dual
    (suffix) cache adds the still-masked positions after the block as further visible keys.
    """
    if k_blk is None:  # block stored in place, right after the prefix
        ks = [k_pre[:P + L]]
        vs = [v_pre[:P + L]]
    else:
        ks = [k_pre[:P], k_blk]
        vs = [v_pre[:P], v_blk]
    if k_suf is not None and S > 0:
        ks.append(k_suf[:S])
        vs.append(v_suf[:S])
    return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)


def attn_block(q, k_pre, v_pre, prefix_len, k_blk=None, v_blk=None,
               k_suf=None, v_suf=None, suffix_len=None, scale=None):
    """Block-bidirectional attention of the current block's queries against the caches.

    q [B,L,Hq,d]; k_pre/v_pre [B,Hkv,Pcap,d]; k_blk/v_blk [B,Hkv,L,d] or None (in place);
    k_suf/v_suf [B,Hkv,Scap,d] or None; prefix_len/suffix_len int [B] (None = full capacity).
    All float64 (exact images of the bf16 inputs).  Query head h reads KV head h // (Hq/Hkv).

    For each (row, head, position): s_j = scale * <q, k_j>; p = softmax_j(s); o = sum_j p_j v_j;
    lse = log sum_j exp(s_j).  Returns (o [B,L,Hq,d], lse [B,Hq,L]) in float64.
    """
    q = np.asarray(q, dtype=np.float64)
    B, L, Hq, d = q.shape
    Hkv = k_pre.shape[1]
    assert Hq % Hkv == 0
    g = Hq // Hkv
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((B, L, Hq, d), dtype=np.float64)
    lse = np.zeros((B, Hq, L), dtype=np.float64)
    for r in range(B):
        if prefix_len is not None:
            P = int(prefix_len[r])
        else:
            P = k_pre.shape[2] - (L if k_blk is None else 0)
        S = 0
        if k_suf is not None:
            S = int(suffix_len[r]) if suffix_len is not None else k_suf.shape[2]
        for h in range(Hq):
            kv = h // g
            K, Vv = _visible_keys(np.asarray(k_pre[r, kv], dtype=np.float64), np.asarray(v_pre[r, kv], dtype=np.float64), P,
                                  None if k_blk is None else np.asarray(k_blk[r, kv], dtype=np.float64),
                                  None if v_blk is None else np.asarray(v_blk[r, kv], dtype=np.float64), L,
                                  None if k_suf is None else np.asarray(k_suf[r, kv], dtype=np.float64),
                                  None if v_suf is None else np.asarray(v_suf[r, kv], dtype=np.float64), S)
            s = scale * (q[r, :, h, :] @ K.T)                 # [L, T]
            m = s.max(axis=1, keepdims=True)
            e = np.exp(s - m)
            den = e.sum(axis=1, keepdims=True)
            p = e / den
            out[r, :, h, :] = p @ Vv
            lse[r, h, :] = (m + np.log(den))[:, 0]
    return out, lse


def attn_varlen(q, k, v, cu_seqlens, scale=None):
    """Bidirectional attention over packed variable-length sequences (Section 3.4, training-side and log-prob
    passes: sequences are concatenated without padding and each attends to itself only).

    q [T, Hq, d]; k, v [T, Hkv, d] float64 with T = total tokens; cu_seqlens int [n + 1], sequence s owns tokens
    [cu_seqlens[s], cu_seqlens[s + 1]).  Query head h reads KV head h // (Hq / Hkv); every token of a sequence
    sees every token of the same sequence.  Returns (o [T, Hq, d], lse [Hq, T]).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, Hq, d = q.shape
    g = Hq // k.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros_like(q)
    lse = np.full((Hq, T), -np.inf)
    for s in range(len(cu_seqlens) - 1):
        a, b = int(cu_seqlens[s]), int(cu_seqlens[s + 1])
        if b <= a:
            continue
        for h in range(Hq):
            sc = scale * (q[a:b, h] @ k[a:b, h // g].T)
            m = sc.max(axis=1, keepdims=True)
            e = np.exp(sc - m)
            den = e.sum(axis=1, keepdims=True)
            out[a:b, h] = (e / den) @ v[a:b, h // g]
            lse[h, a:b] = (m + np.log(den))[:, 0]
    return out, lse


def lmhead_confidence(x, w, row_tokens=None, mask_id=-1, exclude_mask_column=True):
    """LM head + vocabulary softmax -> greedy token and its probability, per masked row.

    x [M,D], w [V,D] float64.  z = x w^T (all V logits); if ``exclude_mask_column`` the mask id's logit
    is -inf (a commit must remove a mask, Eq. 1's absorbing state is never a prediction);
    token = lowest index attaining max z; confidence = exp(max z - logsumexp z) = max_v softmax(z)_v.
    Rows whose ``row_tokens`` entry is not the mask id are skipped: pred = that token, conf = -inf.

    Returns dict with pred int32 [M], conf float64 [M], logconf float64 [M] (= max - lse),
    second float64 [M] (runner-up probability) and gap_logit float64 [M] (top-2 logit gap).
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    M = x.shape[0]
    V = w.shape[0]
    z = x @ w.T                                               # [M, V]
    if exclude_mask_column and 0 <= mask_id < V:
        z[:, mask_id] = -np.inf
    pred = np.argmax(z, axis=1).astype(np.int32)              # first (lowest) index of the maximum
    zmax = z[np.arange(M), pred]
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    logconf = zmax - lse
    conf = np.exp(logconf)
    z2 = z.copy()
    z2[np.arange(M), pred] = -np.inf
    second_logit = z2.max(axis=1)
    second = np.exp(second_logit - lse)
    gap_logit = zmax - second_logit
    if row_tokens is not None:
        rt = np.asarray(row_tokens)
        skip = rt != mask_id
        pred = np.where(skip, rt, pred).astype(np.int32)
        conf = np.where(skip, -np.inf, conf)
        logconf = np.where(skip, -np.inf, logconf)
        second = np.where(skip, 0.0, second)
        gap_logit = np.where(skip, np.inf, gap_logit)
    return {"pred": pred, "conf": conf, "logconf": logconf, "second": second, "gap_logit": gap_logit}


def lmhead_logprob(x, w, targets, mask_id=-1, exclude_mask_column=False):
    """Log-probability of given tokens under the LM head's softmax, per row (Section 3.4: logits-free loss).

    x [M, D], w [V, D] float64; targets int [M].  z = x w^T; the mask id's logit is -inf if
    ``exclude_mask_column``; logprob[m] = z[m, targets[m]] - logsumexp z[m].  A target outside [0, V) (or the
    excluded column) gives -inf.  Returns (logprob float64 [M], lse float64 [M]).
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    M, V = x.shape[0], w.shape[0]
    z = x @ w.T
    if exclude_mask_column and 0 <= mask_id < V:
        z[:, mask_id] = -np.inf
    zmax = z.max(axis=1)
    lse = zmax + np.log(np.exp(z - zmax[:, None]).sum(axis=1))
    t = np.asarray(targets)
    ok = (t >= 0) & (t < V)
    zt = np.where(ok, z[np.arange(M), np.where(ok, t, 0)], -np.inf)
    return zt - lse, lse


def lmhead_logprob_backward(x, w, targets, grad_logprob, mask_id=-1, exclude_mask_column=False):
    """Gradient of sum_m grad_logprob[m] * logprob[m] (lmhead_logprob) with respect to x and w: the backward of
    the logits-free loss of Section 3.4 (the actor update differentiates the per-token log-probabilities).

    With p = softmax(z) over the non-excluded columns:  d logprob[m] / d z[m, v] = 1[v = targets[m]] - p[m, v]
    (0 in the excluded column), so
        dz = grad_logprob[:, None] * (onehot(targets) - p),   dx = dz @ w,   dw = dz^T @ x.
    Rows whose target is outside [0, V) or is the excluded column have logprob = -inf and take no part
    (their dz is 0).  Returns (dx float64 [M, D], dw float64 [V, D], dz float64 [M, V]).
    """
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    g = np.asarray(grad_logprob, dtype=np.float64)
    M, V = x.shape[0], w.shape[0]
    z = x @ w.T
    excluded = exclude_mask_column and 0 <= mask_id < V
    if excluded:
        z[:, mask_id] = -np.inf
    e = np.exp(z - z.max(axis=1, keepdims=True))
    p = e / e.sum(axis=1, keepdims=True)
    t = np.asarray(targets)
    ok = (t >= 0) & (t < V)
    if excluded:
        ok &= t != mask_id
    onehot = np.zeros((M, V))
    onehot[np.nonzero(ok)[0], t[ok]] = 1.0
    dz = g[:, None] * (onehot - p)
    dz[~ok] = 0.0
    return dz @ w, dz.T @ x, dz


def token_probability(x_row, w, token, mask_id=-1, exclude_mask_column=True):
    """Softmax probability of one given token for one row (used to judge near-ties)."""
    z = np.asarray(w, dtype=np.float64) @ np.asarray(x_row, dtype=np.float64)
    if exclude_mask_column and 0 <= mask_id < z.shape[0]:
        z[mask_id] = -np.inf
    m = z.max()
    return float(np.exp(z[token] - m) / np.exp(z - m).sum())


def unmask_select(tokens, block_start, L, pred, conf, mask_id, mode, threshold=0.0, k=1):
    """Parallel unmask selection on the int32 token state (returns a new array; input untouched).

    tokens int32 [B, row]; pred int32 [B, L]; conf float32 [B, L] (compared in float32 exactly as
    given; NaN counts as -inf).  U = masked positions of the block in a row.
      THRESHOLD: C = {i in U : conf_i > threshold}; if C is empty and U is not, C = {the i in U with
                 the largest conf, lowest i on ties}  (at least one commit per step).
      TOPK:      C = the min(k, #U) members of U with the largest conf, lower i first on ties.
    tokens[block_start + i] = pred_i for i in C; every other position keeps its value, so the
    low-confidence positions stay <MASK> and committed tokens are never revisited (Section 3.4,
    "partially fixed states").  Returns (tokens_new, n_committed int32 [B], n_remaining int32 [B]).
    """
    tok = np.array(tokens, dtype=np.int32, copy=True)
    pred = np.asarray(pred, dtype=np.int32).reshape(tok.shape[0], L)
    conf = np.asarray(conf, dtype=np.float32).reshape(tok.shape[0], L)
    B = tok.shape[0]
    n_committed = np.zeros(B, dtype=np.int32)
    n_remaining = np.zeros(B, dtype=np.int32)
    thr = np.float32(threshold)
    for r in range(B):
        U = [i for i in range(L) if tok[r, block_start + i] == mask_id]
        c = {i: (np.float32(-np.inf) if np.isnan(conf[r, i]) else conf[r, i]) for i in U}
        order = sorted(U, key=lambda i: (-float(c[i]), i))   # by confidence descending, index ascending
        if mode == SELECT_THRESHOLD:
            C = [i for i in U if c[i] > thr]
            if not C and U:
                C = [order[0]]
        elif mode == SELECT_TOPK:
            C = order[:min(int(k), len(U))]
        else:
            raise ValueError("mode")
        for i in C:
            tok[r, block_start + i] = pred[r, i]
        n_committed[r] = len(C)
        n_remaining[r] = len(U) - len(C)
    return tok, n_committed, n_remaining


def denoise_step(q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len,
                 x, w, tokens, block_start, L, mask_id, mode, threshold, k,
                 exclude_mask_column=True, scale=None):
    """One denoising step: attention, LM head on the still-masked rows, selection.

    In the single-layer workloads the LM-head input x is given independently of the attention output
    (both are checked); the selection consumes the LM head's confidences rounded to float32.
    """
    o, lse = attn_block(q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len, scale)
    B = tokens.shape[0]
    row_tokens = np.asarray(tokens)[:, block_start:block_start + L].reshape(B * L)
    lm = lmhead_confidence(x, w, row_tokens, mask_id, exclude_mask_column)
    conf32 = lm["conf"].astype(np.float32)
    tok, nc, nr = unmask_select(tokens, block_start, L, lm["pred"], conf32, mask_id, mode, threshold, k)
    return {"attn_out": o, "lse": lse, "lm": lm, "tokens": tok, "n_committed": nc, "n_remaining": nr}
