"""Pins for the oracle's block attention (CPU only).

The oracle is checked against things other than itself: torch's library attention over the whole
sequence with an explicit boolean visibility mask, closed forms, and invariances.
"""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O


def _rand(rng, *shape):
    return rng.standard_normal(shape)


def _library_fullseq(q, k_pre, v_pre, plen, k_blk, v_blk, k_suf, v_suf, slen):
    """Full-sequence attention by torch's SDPA (fp64) with a boolean mask; block rows extracted.

    The sequence is [prefix capacity | block | suffix capacity]; a key is visible to a block query iff
    it is a valid prefix entry, a block entry or a valid suffix entry.  KV heads are replicated so that
    consecutive query heads share one (the GQA mapping being pinned).
    """
    B, L, Hq, d = q.shape
    Hkv, Pcap = k_pre.shape[1], k_pre.shape[2]
    Scap = 0 if k_suf is None else k_suf.shape[2]
    g = Hq // Hkv
    T = Pcap + L + Scap
    outs = np.zeros_like(q)
    for r in range(B):
        K = np.concatenate([k_pre[r], k_blk[r]] + ([k_suf[r]] if Scap else []), axis=1)   # [Hkv,T,d]
        V = np.concatenate([v_pre[r], v_blk[r]] + ([v_suf[r]] if Scap else []), axis=1)
        K = np.repeat(K, g, axis=0)
        V = np.repeat(V, g, axis=0)
        vis = np.zeros(T, dtype=bool)
        vis[:plen[r]] = True
        vis[Pcap:Pcap + L] = True
        if Scap:
            vis[Pcap + L:Pcap + L + slen[r]] = True
        # queries for every position of the sequence; only the block's rows carry the real q
        Qfull = np.zeros((Hq, T, d))
        Qfull[:, Pcap:Pcap + L, :] = np.transpose(q[r], (1, 0, 2))
        mask = np.broadcast_to(vis[None, :], (T, T)).copy()
        o = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(Qfull)[None], torch.from_numpy(K)[None], torch.from_numpy(V)[None],
            attn_mask=torch.from_numpy(mask)[None, None])
        outs[r] = np.transpose(o[0, :, Pcap:Pcap + L, :].numpy(), (1, 0, 2))
    return outs


@pytest.mark.parametrize("B,L,Hq,Hkv,d,Pcap,Scap", [
    (2, 4, 4, 4, 8, 7, 0), (3, 5, 6, 2, 16, 9, 6), (1, 32, 7, 1, 8, 20, 3), (2, 3, 4, 1, 4, 1, 1)])
def test_against_library_fullseq_attention(B, L, Hq, Hkv, d, Pcap, Scap):
    rng = np.random.default_rng(B * 100 + L)
    q = _rand(rng, B, L, Hq, d)
    k_pre, v_pre = _rand(rng, B, Hkv, Pcap, d), _rand(rng, B, Hkv, Pcap, d)
    k_blk, v_blk = _rand(rng, B, Hkv, L, d), _rand(rng, B, Hkv, L, d)
    k_suf = v_suf = slen = None
    if Scap:
        k_suf, v_suf = _rand(rng, B, Hkv, Scap, d), _rand(rng, B, Hkv, Scap, d)
        slen = rng.integers(0, Scap + 1, B)
    plen = rng.integers(0, Pcap + 1, B)
    o, lse = O.attn_block(q, k_pre, v_pre, plen, k_blk, v_blk, k_suf, v_suf, slen)
    ref = _library_fullseq(q, k_pre, v_pre, plen, k_blk, v_blk, k_suf, v_suf, slen)
    np.testing.assert_allclose(o, ref, rtol=0, atol=1e-12)


def test_inplace_block_equals_separate_block():
    rng = np.random.default_rng(5)
    B, L, Hq, Hkv, d, Pcap = 2, 4, 4, 2, 8, 12
    q = _rand(rng, B, L, Hq, d)
    k_pre, v_pre = _rand(rng, B, Hkv, Pcap, d), _rand(rng, B, Hkv, Pcap, d)
    plen = np.array([3, 8])
    k_blk = np.stack([k_pre[r, :, plen[r]:plen[r] + L] for r in range(B)])
    v_blk = np.stack([v_pre[r, :, plen[r]:plen[r] + L] for r in range(B)])
    o1, l1 = O.attn_block(q, k_pre, v_pre, plen, None, None)
    o2, l2 = O.attn_block(q, k_pre, v_pre, plen, k_blk, v_blk)
    np.testing.assert_allclose(o1, o2, atol=1e-14)
    np.testing.assert_allclose(l1, l2, atol=1e-14)


def test_zero_query_gives_mean_of_visible_values_and_log_count():
    rng = np.random.default_rng(1)
    B, L, Hq, Hkv, d, Pcap, Scap = 2, 3, 4, 2, 8, 10, 5
    q = np.zeros((B, L, Hq, d))
    k_pre, v_pre = _rand(rng, B, Hkv, Pcap, d), _rand(rng, B, Hkv, Pcap, d)
    k_blk, v_blk = _rand(rng, B, Hkv, L, d), _rand(rng, B, Hkv, L, d)
    k_suf, v_suf = _rand(rng, B, Hkv, Scap, d), _rand(rng, B, Hkv, Scap, d)
    plen, slen = np.array([4, 10]), np.array([0, 5])
    o, lse = O.attn_block(q, k_pre, v_pre, plen, k_blk, v_blk, k_suf, v_suf, slen)
    for r in range(B):
        for h in range(Hq):
            kv = h // 2
            vis = np.concatenate([v_pre[r, kv, :plen[r]], v_blk[r, kv], v_suf[r, kv, :slen[r]]])
            for i in range(L):
                np.testing.assert_allclose(o[r, i, h], vis.mean(axis=0), atol=1e-13)
                assert abs(lse[r, h, i] - np.log(len(vis))) < 1e-13


def test_dominant_key_selects_its_value():
    rng = np.random.default_rng(2)
    B, L, Hq, d, Pcap = 1, 2, 1, 4, 6
    q = np.zeros((B, L, Hq, d)); q[..., 0] = 1.0
    k_pre = 0.01 * _rand(rng, B, 1, Pcap, d); v_pre = _rand(rng, B, 1, Pcap, d)
    k_blk = 0.01 * _rand(rng, B, 1, L, d); v_blk = _rand(rng, B, 1, L, d)
    k_pre[0, 0, 3, 0] = 200.0   # score = 200/sqrt(4) = 100 above everything else
    o, _ = O.attn_block(q, k_pre, v_pre, np.array([Pcap]), k_blk, v_blk)
    np.testing.assert_allclose(o[0, :, 0], np.broadcast_to(v_pre[0, 0, 3], (L, d)), atol=1e-12)


def test_single_key_returns_block_value():
    rng = np.random.default_rng(3)
    q = _rand(rng, 1, 1, 2, 4)
    k_pre, v_pre = np.zeros((1, 2, 0, 4)), np.zeros((1, 2, 0, 4))
    k_blk, v_blk = _rand(rng, 1, 2, 1, 4), _rand(rng, 1, 2, 1, 4)
    o, lse = O.attn_block(q, k_pre, v_pre, np.array([0]), k_blk, v_blk)
    np.testing.assert_allclose(o[0, 0], v_blk[0, :, 0], atol=1e-15)
    s = (q[0, 0] * k_blk[0, :, 0]).sum(-1) / 2.0     # 1/sqrt(4)
    np.testing.assert_allclose(lse[0, :, 0], s, atol=1e-14)


def test_segment_and_permutation_invariance():
    """Moving keys between prefix / block / suffix, or permuting inside the prefix, changes nothing."""
    rng = np.random.default_rng(4)
    B, L, H, d = 1, 3, 2, 8
    q = _rand(rng, B, L, H, d)
    K, V = _rand(rng, H, 11, d), _rand(rng, H, 11, d)
    # split A: prefix 5, block 3, suffix 3 ; split B: prefix 8 (5 old + old suffix, permuted), block same, no suffix
    oA, lA = O.attn_block(q, K[None, :, :5], V[None, :, :5], np.array([5]), K[None, :, 5:8], V[None, :, 5:8],
                          K[None, :, 8:], V[None, :, 8:], np.array([3]))
    perm = rng.permutation(8)
    pre_idx = np.concatenate([np.arange(5), np.arange(8, 11)])[perm]
    oB, lB = O.attn_block(q, K[None][:, :, pre_idx], V[None][:, :, pre_idx], np.array([8]), K[None, :, 5:8], V[None, :, 5:8])
    np.testing.assert_allclose(oA, oB, atol=1e-13)
    np.testing.assert_allclose(lA, lB, atol=1e-13)


def test_probabilities_bound_output_by_value_range():
    rng = np.random.default_rng(6)
    q = 3 * _rand(rng, 2, 4, 2, 8)
    kp, vp = _rand(rng, 2, 2, 9, 8), _rand(rng, 2, 2, 9, 8)
    kb, vb = _rand(rng, 2, 2, 4, 8), _rand(rng, 2, 2, 4, 8)
    plen = np.array([9, 2])
    o, _ = O.attn_block(q, kp, vp, plen, kb, vb)
    for r in range(2):
        for h in range(2):
            vis = np.concatenate([vp[r, h, :plen[r]], vb[r, h]])
            assert (o[r, :, h] <= vis.max(0) + 1e-12).all() and (o[r, :, h] >= vis.min(0) - 1e-12).all()


def test_split_merge_of_partial_softmax_matches_unsplit():
    """Combining (lse, o) of two key partitions reproduces the unsplit result (what a KV-split relies on)."""
    rng = np.random.default_rng(7)
    B, L, H, d, P = 1, 2, 1, 4, 10
    q = _rand(rng, B, L, H, d)
    kp, vp = _rand(rng, B, H, P, d), _rand(rng, B, H, P, d)
    kb, vb = _rand(rng, B, H, L, d), _rand(rng, B, H, L, d)
    o, lse = O.attn_block(q, kp, vp, np.array([P]), kb, vb)
    # partition: prefix only handled as "block-less" by giving a zero-length trick: use prefix part as its own block
    o1, l1 = O.attn_block(q, kp[:, :, :0], vp[:, :, :0], np.array([0]), kp, vp)      # keys = old prefix
    o2, l2 = O.attn_block(q, kp[:, :, :0], vp[:, :, :0], np.array([0]), kb, vb)      # keys = old block
    l1t, l2t = np.transpose(l1, (0, 2, 1))[..., None], np.transpose(l2, (0, 2, 1))[..., None]
    m = np.maximum(l1t, l2t)
    w1, w2 = np.exp(l1t - m), np.exp(l2t - m)
    merged = (o1 * w1 + o2 * w2) / (w1 + w2)
    np.testing.assert_allclose(merged, o, atol=1e-13)
    np.testing.assert_allclose((m + np.log(w1 + w2))[..., 0], np.transpose(lse, (0, 2, 1)), atol=1e-13)


def test_varlen_is_block_diagonal_library_attention_and_per_sequence_block_attention():
    """attn_varlen against torch attention over the packed tokens with a block-diagonal mask, and against
    attn_block run sequence by sequence (no prefix, the sequence as the in-place block)."""
    rng = np.random.default_rng(21)
    lens = [5, 1, 17, 0, 9]
    cu = np.concatenate([[0], np.cumsum(lens)])
    T, Hq, Hkv, d = int(cu[-1]), 6, 2, 8
    q, k, v = rng.standard_normal((T, Hq, d)), rng.standard_normal((T, Hkv, d)), rng.standard_normal((T, Hkv, d))
    o, lse = O.attn_varlen(q, k, v, cu)
    seg = np.repeat(np.arange(len(lens)), lens)
    mask = torch.from_numpy(seg[:, None] == seg[None, :])
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(Hq // Hkv, dim=0)[None]
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, attn_mask=mask[None, None])[0].permute(1, 0, 2)
    np.testing.assert_allclose(o, want.numpy(), atol=1e-12)
    for s, n in enumerate(lens):
        if n == 0:
            continue
        a, b = cu[s], cu[s + 1]
        kc = np.transpose(k[a:b], (1, 0, 2))[None]
        vc = np.transpose(v[a:b], (1, 0, 2))[None]
        ob, lb = O.attn_block(q[a:b][None], kc, vc, np.array([0]))
        np.testing.assert_allclose(o[a:b], ob[0], atol=1e-12)
        np.testing.assert_allclose(lse[:, a:b], lb[0], atol=1e-12)
    # a token of one sequence does not influence another sequence
    k2 = k.copy()
    k2[cu[2]] += 3.0
    o2, _ = O.attn_varlen(q, k2, v, cu)
    np.testing.assert_array_equal(o2[:cu[2]], o[:cu[2]])
    np.testing.assert_array_equal(o2[cu[3]:], o[cu[3]:])
    assert np.abs(o2[cu[2]:cu[3]] - o[cu[2]:cu[3]]).max() > 1e-3
