"""Pins for the oracle of the end-to-end loop (oracle/dare_model_oracle.py), CPU only.

The paper prints no values for this loop, so the oracle is tied down by what the mathematics fixes:
  * the cache recurrence: the cached loop equals, step by step, a from-scratch forward of the whole sequence
    under the block-causal visibility rule;
  * the stack itself: an independently written torch formulation (library attention with a boolean mask,
    library rms_norm / silu, RoPE as a complex multiplication on re-paired channels);
  * RoPE: position 0 is the identity, norms are kept, scores depend only on position differences;
  * RMSNorm: unit root-mean-square; bf16 rounding: torch's own conversion, including ties;
  * the dual cache: the refresh is the fully bidirectional forward; a window forward right after a refresh
    reproduces the refresh's rows and leaves the cache unchanged; it writes only its own rows, reads the suffix
    and nothing beyond kv_len; one block over the whole sequence makes the loop the uncached model;
  * loop counts: every rollout commits exactly G tokens; steps per block = ceil(L / k) under top-k and
    at most L under the threshold rule; prompt tokens never change; same seed, same tokens.
"""
import numpy as np
import pytest
import torch

from oracle import dare_model_oracle as MO
from oracle import dare_oracle as O
from paper_2604_04215_b200 import inputs as I


def _cfg(mw):
    return MO.ModelConfig(mw.n_layers, mw.hidden, mw.n_q_heads, mw.n_kv_heads, mw.head_dim, mw.ffn, mw.vocab,
                          mw.mask_id, mw.rms_eps, mw.rope_base)


def _weights(mw):
    w = I.make_model_weights(mw)
    f = lambda t: t.to(torch.float64).numpy()
    layers = [MO.LayerWeights(f(l["wqkv"]), f(l["wo"]), f(l["wg"]), f(l["wu"]), f(l["wd"])) for l in w["layers"]]
    return MO.ModelWeights(f(w["embedding"]), layers, f(w["lm_head"]))


def _small(**kw):
    base = I.MODEL_WORKLOADS["loop_small"]
    d = dict(base.__dict__)
    d.update(dict(n_layers=2, hidden=64, n_q_heads=4, n_kv_heads=2, head_dim=16, ffn=96, vocab=128, mask_id=100,
                  batch=2, prompt_len=5, gen_len=12, block_len=4))
    d.update(kw)
    return I.ModelWorkload(**d)


def test_bf16_round_is_torch_conversion_including_ties():
    rng = np.random.default_rng(0)
    a = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096),
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(1.0 + 2.0 ** -8), 0.0, 1e-40, 3.0e38])])
    want = torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(MO.bf16_round(a), want)
    # the two tie cases round to the even mantissa: 1 + 2^-8 -> 1, 1 + 3*2^-8 -> 1 + 2^-6
    assert MO.bf16_round(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert MO.bf16_round(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_rope_properties():
    rng = np.random.default_rng(1)
    T, H, d = 7, 3, 16
    q, k = rng.standard_normal((T, H, d)), rng.standard_normal((T, H, d))
    # position 0 is the identity; rotations keep the norm of every (c, c + d/2) pair
    np.testing.assert_allclose(MO.rope(q, np.zeros(T, dtype=int), 10000.0), q, atol=0)
    pos = np.array([0, 1, 2, 5, 9, 100, 511])
    rq = MO.rope(q, pos, 10000.0)
    np.testing.assert_allclose(rq[..., :8] ** 2 + rq[..., 8:] ** 2, q[..., :8] ** 2 + q[..., 8:] ** 2, rtol=1e-12)
    # scores depend only on the position difference
    s1 = np.einsum("thd,shd->hts", MO.rope(q, pos, 10000.0), MO.rope(k, pos, 10000.0))
    s2 = np.einsum("thd,shd->hts", MO.rope(q, pos + 37, 10000.0), MO.rope(k, pos + 37, 10000.0))
    np.testing.assert_allclose(s1, s2, atol=1e-10)
    # a hand-worked pair: d = 2, position 1, base irrelevant (c = 0): rotation by 1 radian
    out = MO.rope(np.array([[[1.0, 0.0]]]), np.array([1]), 10000.0)
    np.testing.assert_allclose(out[0, 0], [np.cos(1.0), np.sin(1.0)], atol=1e-15)
    # channel c turns at base^(-2c/d): d = 4, c = 1 -> 1/100 radian per position
    out = MO.rope(np.array([[[0.0, 1.0, 0.0, 0.0]]]), np.array([3]), 10000.0)
    np.testing.assert_allclose(out[0, 0], [0.0, np.cos(0.03), 0.0, np.sin(0.03)], atol=1e-15)


def test_rmsnorm_has_unit_rms():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((5, 64)) * 7.0
    y = MO.rmsnorm(x, 0.0)
    np.testing.assert_allclose(np.sqrt((y * y).mean(axis=-1)), 1.0, rtol=1e-12)
    np.testing.assert_allclose(MO.rmsnorm(x, 1e-5), x / np.sqrt((x * x).mean(-1, keepdims=True) + 1e-5), rtol=1e-15)


def _torch_stack(cfg, wts, tokens_row, seg):
    """The same architecture written differently, in torch float64: library attention with a boolean mask,
    library rms_norm and silu, RoPE as multiplication by e^{i angle} of the complex number (x_c, x_{c+d/2})."""
    F = torch.nn.functional
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    T = len(tokens_row)
    d, Hq, Hkv = cfg.head_dim, cfg.n_q_heads, cfg.n_kv_heads
    x = t(wts.embedding)[torch.as_tensor(np.asarray(tokens_row), dtype=torch.long)]
    mask = torch.from_numpy(seg[None, :] <= seg[:, None])
    inv = torch.tensor(cfg.rope_base, dtype=torch.float64) ** (-torch.arange(0, d, 2, dtype=torch.float64) / d)
    rot = torch.polar(torch.ones(T, d // 2, dtype=torch.float64), torch.arange(T, dtype=torch.float64)[:, None] * inv)

    def rope(v):   # v [T, H, d]
        z = torch.complex(v[..., :d // 2], v[..., d // 2:]) * rot[:, None, :]
        return torch.cat([z.real, z.imag], dim=-1)

    for lw in wts.layers:
        h = F.rms_norm(x, (cfg.hidden,), eps=cfg.rms_eps)
        qkv = F.linear(h, t(lw.wqkv))
        q = rope(qkv[:, :Hq * d].view(T, Hq, d)).transpose(0, 1)
        k = rope(qkv[:, Hq * d:(Hq + Hkv) * d].view(T, Hkv, d)).transpose(0, 1)
        v = qkv[:, (Hq + Hkv) * d:].view(T, Hkv, d).transpose(0, 1)
        k = k.repeat_interleave(Hq // Hkv, dim=0)
        v = v.repeat_interleave(Hq // Hkv, dim=0)
        o = F.scaled_dot_product_attention(q[None], k[None], v[None], attn_mask=mask[None, None])[0]
        x = x + F.linear(o.transpose(0, 1).reshape(T, Hq * d), t(lw.wo))
        h2 = F.rms_norm(x, (cfg.hidden,), eps=cfg.rms_eps)
        x = x + F.linear(F.silu(F.linear(h2, t(lw.wg))) * F.linear(h2, t(lw.wu)), t(lw.wd))
    return F.rms_norm(x, (cfg.hidden,), eps=cfg.rms_eps).numpy()


@pytest.mark.parametrize("gqa", [False, True])
def test_uncached_forward_matches_independent_torch_formulation(gqa):
    mw = _small(n_kv_heads=2 if gqa else 4)
    cfg, wts = _cfg(mw), _weights(mw)
    tok = I.fresh_model_tokens(mw).numpy()
    tok[:, mw.prompt_len:mw.prompt_len + 6] = 3             # some committed generation tokens
    seg = MO.segment_ids(mw.prompt_len, mw.gen_len, mw.block_len)
    got, _ = MO.forward_uncached(cfg, wts, tok[0], seg, rounded=False)
    want = _torch_stack(cfg, wts, tok[0], seg)
    np.testing.assert_allclose(got, want, atol=1e-10)
    # the weights are tiny (sigma 0.02): make sure the check is not vacuous
    assert np.abs(want).max() > 0.5 and np.abs(got - np.roll(want, 1, axis=0)).max() > 1e-3


def test_block_causal_rule():
    seg = MO.segment_ids(3, 4, 2)
    np.testing.assert_array_equal(seg, [0, 0, 0, 1, 1, 2, 2])
    mw = _small()
    cfg, wts = _cfg(mw), _weights(mw)
    tok = I.fresh_model_tokens(mw).numpy()[0]
    seg = MO.segment_ids(mw.prompt_len, mw.gen_len, mw.block_len)
    base, _ = MO.forward_uncached(cfg, wts, tok, seg, rounded=False)
    # changing a token of the LAST block leaves every earlier position's output untouched, and changes its own block
    tok2 = tok.copy()
    tok2[-1] = 7
    out2, _ = MO.forward_uncached(cfg, wts, tok2, seg, rounded=False)
    first_of_last = mw.prompt_len + mw.gen_len - mw.block_len
    np.testing.assert_array_equal(out2[:first_of_last], base[:first_of_last])
    assert np.abs(out2[first_of_last:] - base[first_of_last:]).min(axis=1).max() > 0
    # the prompt is bidirectional: changing its last token changes its first position
    tok3 = tok.copy()
    tok3[mw.prompt_len - 1] = (tok3[mw.prompt_len - 1] + 1) % 90
    out3, _ = MO.forward_uncached(cfg, wts, tok3, seg, rounded=False)
    assert np.abs(out3[0] - base[0]).max() > 0


@pytest.mark.parametrize("rounded", [False, True])
@pytest.mark.parametrize("mode,k", [(O.SELECT_THRESHOLD, 1), (O.SELECT_TOPK, 3)])
def test_cached_loop_equals_uncached_forward_step_by_step(rounded, mode, k):
    mw = _small(batch=2)
    cfg, wts = _cfg(mw), _weights(mw)
    tok0 = I.fresh_model_tokens(mw).numpy()
    seg = MO.segment_ids(mw.prompt_len, mw.gen_len, mw.block_len)
    L = mw.block_len
    seen = []

    def on_step(b, n, tok_before, res):
        start = mw.prompt_len + b * L
        for r in range(mw.batch):
            full, _ = MO.forward_uncached(cfg, wts, tok_before[r], seg, rounded)
            got = res["hidden"][r * L:(r + 1) * L]
            if rounded:
                # identical rounding points; a last-bit difference of the two summation orders can move one
                # bf16 rounding, so allow one bf16 step on O(1) values
                np.testing.assert_allclose(got, full[start:start + L], atol=2e-2)
                assert np.abs(got - full[start:start + L]).mean() < 1e-4
            else:
                np.testing.assert_allclose(got, full[start:start + L], atol=1e-9)
            lm = O.lmhead_confidence(full[start:start + L], wts.lm_head, tok_before[r, start:start + L], cfg.mask_id)
            if not rounded:
                np.testing.assert_array_equal(lm["pred"], res["lm"]["pred"][r * L:(r + 1) * L])
        seen.append((b, n))

    tok, steps, cache = MO.generate(cfg, wts, tok0, mw.prompt_len, mw.gen_len, L, mode, 0.9, k, rounded, on_step)
    assert len(seen) == sum(steps)
    # counts: every rollout commits all G tokens, nothing of the prompt changes
    assert (tok[:, mw.prompt_len:] != cfg.mask_id).all()
    np.testing.assert_array_equal(tok[:, :mw.prompt_len], tok0[:, :mw.prompt_len])
    if mode == O.SELECT_TOPK:
        assert steps == [-(-L // k)] * (mw.gen_len // L)
    else:
        assert all(1 <= s <= L for s in steps)
    # after the loop the cache holds the K/V of the final sequence (the refresh forward did its job)
    for r in range(mw.batch):
        _, kv = MO.forward_uncached(cfg, wts, tok[r], seg, rounded)
        for li, (k_full, v_full) in enumerate(kv):
            tol = 2e-2 if rounded else 1e-9
            np.testing.assert_allclose(cache[li][0][r], np.transpose(k_full, (1, 0, 2)), atol=tol)
            np.testing.assert_allclose(cache[li][1][r], np.transpose(v_full, (1, 0, 2)), atol=tol)


def test_generate_is_deterministic():
    mw = _small(batch=1, gen_len=8)
    cfg, wts = _cfg(mw), _weights(mw)
    tok0 = I.fresh_model_tokens(mw).numpy()
    a = MO.generate(cfg, wts, tok0, mw.prompt_len, mw.gen_len, mw.block_len, O.SELECT_THRESHOLD, 0.9, 1)
    b = MO.generate(cfg, wts, tok0, mw.prompt_len, mw.gen_len, mw.block_len, O.SELECT_THRESHOLD, 0.9, 1)
    np.testing.assert_array_equal(a[0], b[0])
    assert a[1] == b[1]


# ---------------------------------------------------------------------------------------------------------
# Dual cache (prefix + suffix) of a fully bidirectional model

def test_refresh_is_the_fully_bidirectional_forward():
    """The refresh forward (all rows, all keys) equals the uncached forward with every position in one segment."""
    mw = _small(batch=2)
    cfg, wts = _cfg(mw), _weights(mw)
    tok = I.fresh_model_tokens(mw).numpy()
    T = mw.prompt_len + mw.gen_len
    cache = MO.new_cache(cfg, mw.batch, T)
    hid = MO.forward_block_cached(cfg, wts, tok, 0, T, cache, rounded=False)
    for r in range(mw.batch):
        full, kv = MO.forward_uncached(cfg, wts, tok[r, :T], np.zeros(T, dtype=np.int64), rounded=False)
        np.testing.assert_allclose(hid[r * T:(r + 1) * T], full, atol=1e-9)
        for li, (k_full, v_full) in enumerate(kv):
            np.testing.assert_allclose(cache[li][0][r], np.transpose(k_full, (1, 0, 2)), atol=1e-9)
            np.testing.assert_allclose(cache[li][1][r], np.transpose(v_full, (1, 0, 2)), atol=1e-9)


@pytest.mark.parametrize("start,length", [(5, 4), (0, 5), (13, 4), (7, 3)])
def test_window_forward_right_after_a_refresh_reproduces_it(start, length):
    """With unchanged tokens the cached K/V are exact, so a window forward over prefix + block + suffix gives the
    refresh's own rows and leaves the cache as it was: pins the visibility (all of [0, kv_len)), the in-place
    positions and RoPE offsets of the window, for a window at the start, in the middle and at the end."""
    mw = _small(batch=2)
    cfg, wts = _cfg(mw), _weights(mw)
    tok = I.fresh_model_tokens(mw).numpy()
    T = mw.prompt_len + mw.gen_len
    cache = MO.new_cache(cfg, mw.batch, T)
    hid = MO.forward_block_cached(cfg, wts, tok, 0, T, cache, rounded=False).reshape(mw.batch, T, -1)
    before = [(k.copy(), v.copy()) for k, v in cache]
    win = MO.forward_block_cached(cfg, wts, tok, start, length, cache, rounded=False, kv_len=T)
    np.testing.assert_allclose(win.reshape(mw.batch, length, -1), hid[:, start:start + length], atol=1e-9)
    for (k0, v0), (k1, v1) in zip(before, cache):
        np.testing.assert_allclose(k1, k0, atol=1e-9)
        np.testing.assert_allclose(v1, v0, atol=1e-9)
    # a window that cannot see the suffix differs (unless it is the last one)
    if start + length < T:
        cut = MO.forward_block_cached(cfg, wts, tok, start, length, [(k.copy(), v.copy()) for k, v in before],
                                      rounded=False)
        assert np.abs(cut - win).max() > 1e-6


def test_window_forward_writes_only_its_own_rows_and_reads_the_suffix():
    mw = _small(batch=1)
    cfg, wts = _cfg(mw), _weights(mw)
    tok = I.fresh_model_tokens(mw).numpy()
    T = mw.prompt_len + mw.gen_len
    start, L = mw.prompt_len, mw.block_len
    cache = MO.new_cache(cfg, 1, T)
    MO.forward_block_cached(cfg, wts, tok, 0, T, cache, rounded=False)
    before = [(k.copy(), v.copy()) for k, v in cache]
    tok2 = tok.copy()
    tok2[0, start + 1] = 9                                              # a committed token inside the block
    out = MO.forward_block_cached(cfg, wts, tok2, start, L, cache, rounded=False, kv_len=T)
    for (k0, v0), (k1, v1) in zip(before, cache):
        np.testing.assert_array_equal(k1[:, :, :start], k0[:, :, :start])
        np.testing.assert_array_equal(k1[:, :, start + L:], k0[:, :, start + L:])
        np.testing.assert_array_equal(v1[:, :, start + L:], v0[:, :, start + L:])
    assert np.abs(cache[0][0][:, :, start + 1] - before[0][0][:, :, start + 1]).max() > 0
    # the suffix is read: perturbing a cached suffix value changes the block's output
    cache2 = [(k.copy(), v.copy()) for k, v in cache]
    cache2[0][1][0, :, T - 1] += 1.0
    out2 = MO.forward_block_cached(cfg, wts, tok2, start, L, cache2, rounded=False, kv_len=T)
    assert np.abs(out2 - out).max() > 1e-6
    # keys at and beyond kv_len are not read
    cache3 = [(k.copy(), v.copy()) for k, v in cache]
    cache3[0][1][0, :, T - 1] += 1.0
    out3 = MO.forward_block_cached(cfg, wts, tok2, start, L, cache3, rounded=False, kv_len=T - 1)
    out4 = MO.forward_block_cached(cfg, wts, tok2, start, L, [(k.copy(), v.copy()) for k, v in cache], rounded=False,
                                   kv_len=T - 1)
    np.testing.assert_array_equal(out3, out4)


@pytest.mark.parametrize("mode,k", [(O.SELECT_THRESHOLD, 1), (O.SELECT_TOPK, 3)])
def test_dual_loop_with_one_block_over_everything_is_the_uncached_model(mode, k):
    """No prompt and a single block spanning the whole sequence: nothing is ever stale, so every step of the
    dual-cache loop equals a from-scratch fully bidirectional forward of the current tokens."""
    mw = _small(batch=2, prompt_len=0, gen_len=8, block_len=8)
    cfg, wts = _cfg(mw), _weights(mw)
    tok0 = I.fresh_model_tokens(mw).numpy()
    seen = []

    def on_step(b, n, tok_before, res):
        for r in range(mw.batch):
            full, _ = MO.forward_uncached(cfg, wts, tok_before[r, :8], np.zeros(8, dtype=np.int64), rounded=False)
            np.testing.assert_allclose(res["hidden"][r * 8:(r + 1) * 8], full, atol=1e-9)
        seen.append(n)

    tok, steps, _ = MO.generate_dual(cfg, wts, tok0, 0, 8, 8, mode, 0.9, k, rounded=False, on_step=on_step)
    assert len(seen) == steps[0] and (tok[:, :8] != cfg.mask_id).all()
    if mode == O.SELECT_TOPK:
        assert steps == [3]


def test_dual_loop_counts_and_first_step_of_each_block():
    """Several blocks: the first step of a block (tokens unchanged since the refresh) equals the refresh's rows for
    that block; later steps see stale K/V outside the block and differ from a from-scratch forward; counts hold."""
    mw = _small(batch=2)
    cfg, wts = _cfg(mw), _weights(mw)
    tok0 = I.fresh_model_tokens(mw).numpy()
    T, L, P = mw.prompt_len + mw.gen_len, mw.block_len, mw.prompt_len
    refreshed = {}
    stale_seen = []

    def on_refresh(b, tok, hidden):
        refreshed[b] = hidden.reshape(mw.batch, T, -1).copy()

    def on_step(b, n, tok_before, res):
        start = P + b * L
        got = res["hidden"].reshape(mw.batch, L, -1)
        if n == 0:
            np.testing.assert_allclose(got, refreshed[b][:, start:start + L], atol=1e-9)
        else:
            full = np.stack([MO.forward_uncached(cfg, wts, tok_before[r, :T], np.zeros(T, dtype=np.int64), False)[0]
                             for r in range(mw.batch)])
            stale_seen.append(np.abs(got - full[:, start:start + L]).max())

    tok, steps, _ = MO.generate_dual(cfg, wts, tok0, P, mw.gen_len, L, O.SELECT_TOPK, 0.9, 2, rounded=False,
                                     on_step=on_step, on_refresh=on_refresh)
    assert steps == [2] * (mw.gen_len // L) and sorted(refreshed) == list(range(mw.gen_len // L))
    assert (tok[:, P:] != cfg.mask_id).all()
    np.testing.assert_array_equal(tok[:, :P], tok0[:, :P])
    assert min(stale_seen) > 1e-6                   # staleness is real: the cached loop is an approximation
    a = MO.generate_dual(cfg, wts, tok0, P, mw.gen_len, L, O.SELECT_TOPK, 0.9, 2)
    b = MO.generate_dual(cfg, wts, tok0, P, mw.gen_len, L, O.SELECT_TOPK, 0.9, 2)
    np.testing.assert_array_equal(a[0], b[0])


# ---------------------------------------------------------------------------------------------------------
# The loop with the sampled head

def test_sampled_loop_limits_counts_and_determinism():
    """T -> 0 gives the greedy loop's tokens; the same seed the same tokens, another seed others; every rollout
    commits all G tokens under top-k in ceil(L / k) steps per block; steps of different blocks and different steps
    of a block use different generator counters (identical hidden rows would otherwise repeat their draws)."""
    mw = _small(batch=2)
    cfg, wts = _cfg(mw), _weights(mw)
    tok0 = I.fresh_model_tokens(mw).numpy()
    P, G, L = mw.prompt_len, mw.gen_len, mw.block_len
    greedy, gsteps, _ = MO.generate(cfg, wts, tok0, P, G, L, O.SELECT_TOPK, 0.9, 2, rounded=False)
    cold, csteps, _ = MO.generate_sampled(cfg, wts, tok0, P, G, L, O.SELECT_TOPK, 0.9, 2, 1e-7, 5, rounded=False)
    np.testing.assert_array_equal(cold, greedy)
    assert csteps == gsteps == [2] * (G // L)
    seen = []
    a, _, _ = MO.generate_sampled(cfg, wts, tok0, P, G, L, O.SELECT_TOPK, 0.9, 2, 1.0, 5, rounded=False,
                                  on_step=lambda b, n, t, r: seen.append((b, n)))
    b_, _, _ = MO.generate_sampled(cfg, wts, tok0, P, G, L, O.SELECT_TOPK, 0.9, 2, 1.0, 5, rounded=False)
    c, _, _ = MO.generate_sampled(cfg, wts, tok0, P, G, L, O.SELECT_TOPK, 0.9, 2, 1.0, 6, rounded=False)
    np.testing.assert_array_equal(a, b_)
    assert (a != c).any() and (a != greedy).any()
    assert (a[:, P:] != cfg.mask_id).all() and (a[:, :P] == tok0[:, :P]).all()
    assert seen == [(b, n) for b in range(G // L) for n in range(2)]
    # the step counter reaches the generator: the same state sampled under two counters differs
    cache = MO.new_cache(cfg, mw.batch, P + G)
    MO.forward_block_cached(cfg, wts, tok0, 0, P, cache, False)
    r1 = MO.denoise_step_cached_sampled(cfg, wts, tok0, P, L, [(k.copy(), v.copy()) for k, v in cache], O.SELECT_TOPK,
                                        0.9, 2, 1.0, 5, (0 << 16) + 0, False)
    r2 = MO.denoise_step_cached_sampled(cfg, wts, tok0, P, L, [(k.copy(), v.copy()) for k, v in cache], O.SELECT_TOPK,
                                        0.9, 2, 1.0, 5, (1 << 16) + 0, False)
    assert (r1["lm"]["pred"] != r2["lm"]["pred"]).any()
    np.testing.assert_allclose(r1["hidden"], r2["hidden"], atol=0)
