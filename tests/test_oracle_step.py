"""Pins for the oracle's whole denoising step and for the seeded input generators (CPU only)."""
import numpy as np
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import inputs as I


def _f64(t):
    return None if t is None else t.to(torch.float64).numpy()


def _tiny(**kw):
    return I.scaled(I.WORKLOADS["tiny"], vocab=512, mask_id=511, hidden=64, prompt_len=16, **kw)


def _run_step(si, tokens, mode, thr, k):
    wl = si.wl
    return O.denoise_step(_f64(si.q), _f64(si.k_pre), _f64(si.v_pre), si.prefix_len.numpy(), _f64(si.k_blk),
                          _f64(si.v_blk), _f64(si.k_suf), _f64(si.v_suf),
                          None if si.suffix_len is None else si.suffix_len.numpy(), _f64(si.x), _f64(si.w),
                          tokens, si.block_start, wl.block_len, wl.mask_id, mode, thr, k)


def test_frozen_inputs_commit_in_descending_confidence_order():
    """With the same hidden states at every iteration, top-k steps commit the first step's ranking, k at a time."""
    wl = _tiny(batch=2)
    si = I.make_step(wl, step=0)
    tokens = si.tokens.numpy()
    first = _run_step(si, tokens, O.SELECT_TOPK, 0.0, 3)
    conf0 = first["lm"]["conf"].reshape(wl.batch, wl.block_len)
    rank = np.argsort(-conf0, axis=1, kind="stable")
    cur, t = tokens, 0
    while (cur[:, si.block_start:] == wl.mask_id).any():
        res = _run_step(si, cur, O.SELECT_TOPK, 0.0, 3)
        t += 1
        for r in range(wl.batch):
            done = set(np.nonzero(res["tokens"][r, si.block_start:] != wl.mask_id)[0].tolist())
            assert done == set(rank[r, :min(3 * t, wl.block_len)].tolist())
        # committed tokens never change
        keep = cur != wl.mask_id
        assert (res["tokens"][keep] == cur[keep]).all()
        cur = res["tokens"]
    assert t == -(-wl.block_len // 3)


def test_step_outputs_are_consistent():
    wl = _tiny(batch=2, suffix_cap=8)
    si = I.make_step(wl, step=1, planted=True)
    res = _run_step(si, si.tokens.numpy(), O.SELECT_THRESHOLD, 0.9, 1)
    conf = res["lm"]["conf"]
    assert ((conf > 0) & (conf <= 1)).all()
    np.testing.assert_allclose(np.exp(res["lm"]["logconf"]), conf, rtol=1e-14)
    # planted inputs: most rows predict their planted column, confidences spread out
    hit = (res["lm"]["pred"] == si.extras["planted_cols"].numpy()).mean()
    assert hit > 0.9 and conf.min() < 0.5 < conf.max()
    above = (conf.astype(np.float32).reshape(2, -1) > np.float32(0.9)).sum(1)
    np.testing.assert_array_equal(res["n_committed"], np.maximum(above, 1))
    assert (res["tokens"] != wl.mask_id).sum() - (si.tokens.numpy() != wl.mask_id).sum() == res["n_committed"].sum()


def test_generators_are_deterministic_and_shaped():
    wl = I.scaled(I.WORKLOADS["dualcache"], batch=3, prompt_len=64, suffix_cap=32, vocab=1024, mask_id=1000,
                  hidden=128, n_q_heads=4, n_kv_heads=4, ragged=True)
    a, b = I.make_step(wl, step=2), I.make_step(wl, step=2)
    for name in ("q", "k_pre", "v_pre", "k_blk", "k_suf", "x", "w", "tokens", "prefix_len", "suffix_len"):
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    c = I.make_step(wl, step=3)
    assert not torch.equal(a.x, c.x) and torch.equal(a.w, c.w)
    assert a.q.shape == (3, 4, 4, 128) and a.k_pre.shape == (3, 4, 68, 128) and a.k_suf.shape == (3, 4, 32, 128)
    assert (a.prefix_len % 4 == 0).all() and (a.prefix_len >= 4).all() and (a.prefix_len <= 64).all()
    assert (a.suffix_len <= 32).all() and a.w.dtype == torch.bfloat16
    assert (a.tokens[:, :64] != wl.mask_id).all() and (a.tokens[:, 64:] == wl.mask_id).all()
    assert abs(float(a.w.float().std()) - 0.02) < 2e-3 and abs(float(a.x.float().std()) - 1.0) < 0.05
