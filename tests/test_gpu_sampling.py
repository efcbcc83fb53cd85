"""GPU parity of the stochastic rollout epilogue (dare_lmhead_sample) against its fp64 oracle.

The sampled token is an argmax of perturbed scores y = z / T + g, so the rule for the greedy head carries over:
tokens must agree wherever the oracle's best score leads the runner-up by more than 1e-3; where they differ, the
GPU's token must be a near-tie (its oracle score within 1e-3 of the best).  Confidences within 1e-3 absolute and
2e-2 in log.  The uniforms come from the same published counter-based generator on both sides.
"""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from oracle import dare_sampling_oracle as SO
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import CONF_ABS, LOGCONF_ABS, f64

pytestmark = pytest.mark.gpu

GAP_Y = 1e-3


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    c.close()


def _check(pred_t, conf_t, ref, x64, w64, rows, mask_id, excl, T, seed, step):
    pred, conf = pred_t.cpu().numpy(), conf_t.cpu().numpy().astype(np.float64)
    live = np.isfinite(ref["conf"])
    assert (pred[~live] == ref["pred"][~live]).all() and np.isneginf(conf[~live]).all()
    must = live & (ref["gap_y"] > GAP_Y)
    assert (pred[must] == ref["pred"][must]).all(), "sampled token differs where the best score leads by more than 1e-3"
    for m in np.nonzero(live & (pred != ref["pred"]))[0]:
        y = SO.perturbed_score(x64[m], w64, int(pred[m]), int(rows[m]), mask_id, excl, T, seed, step)
        assert y >= ref["y_best"][m] - GAP_Y
    same = live & (pred == ref["pred"])
    assert np.abs(conf[same] - ref["conf"][same]).max(initial=0) <= CONF_ABS
    assert np.abs(np.log(conf[same]) - ref["logconf"][same]).max(initial=0) <= LOGCONF_ABS
    assert same.sum() >= 0.9 * live.sum() - 1
    return int((live & (pred != ref["pred"])).sum())


def _case(ctx, M, D, V, mu, T, seed, step, with_rows=False, excl=True, planted=False):
    wl = I.scaled(I.WORKLOADS["tiny"], hidden=D, vocab=V, mask_id=mu, seed=seed & 0xFFFF)
    x = I.normal_bf16(seed & 0xFFFF, I.TID_X, (M, D))
    w = I.normal_bf16(seed & 0xFFFF, I.TID_W, (V, D), 0.02 if not planted else 0.05)
    if planted:
        x, _ = I.plant_confidences(wl, x, w, 0)
    rt = None
    if with_rows:
        rt = I.uniform_int(seed & 0xFFFF, I.TID_TOK, (M,), 0, V - 1)
        rt[::3] = mu
    ref = SO.lmhead_sample(f64(x), f64(w), None if rt is None else rt.numpy(), mu, excl, T, seed, step)
    pred, conf = dare.dare_lmhead_sample(ctx, x.cuda(), w.cuda(), None if rt is None else rt.cuda(), mu, excl, T, seed, step)
    torch.cuda.synchronize()
    _check(pred, conf, ref, f64(x), f64(w), np.arange(M), mu, excl, T, seed, step)
    assert ctx.device_status() == 0
    return pred, conf, ref


@pytest.mark.parametrize("M,D,V,mu,T,seed,step,with_rows", [
    (32, 256, 4096, 4095, 1.0, 0, 0, False),                      # the tiny workload's head
    (300, 1024, 2560 + 40, 2599, 0.7, 0x1234567890ABCDEF, 7, True),   # several row and vocabulary tiles, tails, 64-bit seed
    (130, 64, 520, 5, 1.5, 3, 4000000000, True),                  # high temperature, large step counter
    (9, 8, 2, 1, 1.0, 1, 1, False),                               # two-entry vocabulary with the mask excluded: one choice
])
def test_sample_matches_oracle(ctx, M, D, V, mu, T, seed, step, with_rows):
    _case(ctx, M, D, V, mu, T, seed, step, with_rows)


def test_sample_with_spread_confidences_and_raw_softmax(ctx):
    pred, conf, ref = _case(ctx, 96, 256, 1024, 1023, 1.0, 11, 2, planted=True)
    c = conf.cpu().numpy()
    assert (c > 0.3).sum() >= 5 and (c < 0.1).sum() >= 5            # not all in one corner
    _case(ctx, 96, 256, 1024, 7, 1.0, 12, 3, excl=False)              # mask column kept in the softmax


def test_sample_is_reproducible_and_keyed_by_seed_step_and_row(ctx):
    M, D, V, mu = 200, 128, 3000, 2999
    x = I.normal_bf16(5, I.TID_X, (M, D)).cuda()
    w = I.normal_bf16(5, I.TID_W, (V, D), 0.02).cuda()
    a = dare.dare_lmhead_sample(ctx, x, w, None, mu, True, 1.0, 42, 0)[0].clone()
    b = dare.dare_lmhead_sample(ctx, x, w, None, mu, True, 1.0, 42, 0)[0].clone()
    c = dare.dare_lmhead_sample(ctx, x, w, None, mu, True, 1.0, 42, 1)[0].clone()
    d = dare.dare_lmhead_sample(ctx, x, w, None, mu, True, 1.0, 43, 0)[0].clone()
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    assert (a != c).float().mean() > 0.9 and (a != d).float().mean() > 0.9
    # identical hidden rows still draw different tokens (the row index keys the generator)
    x1 = x[:1].repeat(M, 1).contiguous()
    e = dare.dare_lmhead_sample(ctx, x1, w, None, mu, True, 1.0, 42, 0)[0]
    assert len(torch.unique(e)) > M // 2
    # rows skipped by row_tokens do not shift the other rows' streams
    rt = torch.full((M,), mu, dtype=torch.int32)
    rt[::2] = 3
    f = dare.dare_lmhead_sample(ctx, x, w, rt.cuda(), mu, True, 1.0, 42, 0)[0]
    torch.cuda.synchronize()
    assert torch.equal(f[1::2], a[1::2]) and (f[::2] == 3).all()


def test_low_temperature_gives_the_greedy_tokens(ctx):
    M, D, V, mu = 128, 256, 4096, 4095
    x = I.normal_bf16(6, I.TID_X, (M, D))
    w = I.normal_bf16(6, I.TID_W, (V, D), 0.02)
    g = O.lmhead_confidence(f64(x), f64(w), None, mu, True)
    pred, conf = dare.dare_lmhead_sample(ctx, x.cuda(), w.cuda(), None, mu, True, 1e-4, 9, 0)
    torch.cuda.synchronize()
    clear = g["gap_logit"] > 0.02                                     # noise / T-scaled gap: 1e-4 * 20 << 0.02
    assert clear.sum() > M // 2
    assert (pred.cpu().numpy()[clear] == g["pred"][clear]).all()
    assert np.abs(conf.cpu().numpy()[clear] - g["conf"][clear]).max() <= CONF_ABS


def test_token_frequencies_follow_softmax(ctx):
    """Gumbel-max on the GPU: 4096 copies of one row, small vocabulary, frequencies against softmax(z / T)."""
    M, D, V, mu, T = 4096, 64, 40, 39, 0.8
    x1 = I.normal_bf16(7, I.TID_X, (1, D))
    w = I.normal_bf16(7, I.TID_W, (V, D), 0.25)
    x = x1.repeat(M, 1).contiguous()
    pred, _ = dare.dare_lmhead_sample(ctx, x.cuda(), w.cuda(), None, mu, True, T, 2024, 5)
    torch.cuda.synchronize()
    z = f64(w) @ f64(x1)[0]
    z[mu] = -np.inf
    p = np.exp(z / T - (z / T)[np.isfinite(z)].max())
    p /= p.sum()
    freq = np.bincount(pred.cpu().numpy(), minlength=V) / M
    assert freq[mu] == 0
    assert np.abs(freq - p).max() < 4.0 * np.sqrt(0.25 / M)
    assert p.max() < 0.6                                             # the distribution is not degenerate


def test_bad_arguments(ctx):
    x = torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_lmhead_sample(ctx, x, w, None, 3, True, 0.0, 1, 1, check=False) == -4      # temperature must be > 0
    assert dare.dare_lmhead_sample(ctx, x, w, None, 3, True, float("nan"), 1, 1, check=False) == -4
    assert dare.dare_lmhead_sample(ctx, x, w, None, 3, True, float("inf"), 1, 1, check=False) == -4


def test_llada8b_full_size_sampled_rows(ctx):
    """Full-size head (512 x 4096 x 126464): 16 sampled rows against the oracle, everything else by properties."""
    wl = I.WORKLOADS["llada8b"]
    rng = np.random.default_rng(3)
    w = I.make_weights(wl)
    x = I.normal_bf16(0, I.TID_X, (wl.M, wl.hidden))
    rt = torch.full((wl.M,), wl.mask_id, dtype=torch.int32)
    rt[rng.random(wl.M) < 0.3] = 11
    T, seed, step = 1.0, 77, 19
    pred, conf = dare.dare_lmhead_sample(ctx, x.cuda(), w.cuda(), rt.cuda(), wl.mask_id, True, T, seed, step)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    masked = np.nonzero(rt.numpy() == wl.mask_id)[0]
    rows = np.sort(rng.choice(masked, size=16, replace=False))
    w64, x64 = f64(w), f64(x[rows])
    # the oracle keys its generator by the row index in the array it is given: evaluate row by row at the true index
    for n, m in enumerate(rows):
        z = w64 @ x64[n]
        z[wl.mask_id] = -np.inf
        y = z / T + SO.gumbel(SO.uniforms(seed, int(m), step, wl.vocab))
        t = int(np.argmax(y))
        second = np.partition(y, -2)[-2]
        got = int(pred[m])
        if y[t] - second > GAP_Y:
            assert got == t
        else:
            assert y[got] >= y[t] - GAP_Y
        lse = z[np.isfinite(z)].max() + np.log(np.exp(z - z[np.isfinite(z)].max()).sum())
        if got == t:
            assert abs(float(conf[m]) - np.exp(z[t] - lse)) <= CONF_ABS
            assert abs(np.log(float(conf[m])) - (z[t] - lse)) <= LOGCONF_ABS
    p_all, c_all = pred.cpu().numpy(), conf.cpu().numpy()
    done = rt.numpy() != wl.mask_id
    assert (p_all[done] == 11).all() and np.isneginf(c_all[done]).all()
    assert ((c_all[~done] > 0) & (c_all[~done] <= 1.0)).all()
    assert (p_all[~done] != wl.mask_id).all() and (p_all[~done] >= 0).all() and (p_all[~done] < wl.vocab).all()
    assert len(np.unique(p_all[~done])) > 0.9 * (~done).sum()          # high-entropy logits: almost all tokens differ


def test_sampled_step_on_the_tiny_workload(ctx):
    """dare_denoise_block_sampled over 6 iterations of config 1 (planted confidences, so that the threshold rule
    commits varying numbers of tokens): attention and sampled head against the oracle from the GPU's pre-step state,
    selection bit-exact from the GPU's own tokens and confidences."""
    from _util import check_attn
    wl = I.WORKLOADS["tiny"]
    w = I.make_weights(wl)
    caches = I.make_caches(wl)
    wd, kp, vp = w.cuda(), caches[0].cuda(), caches[1].cuda()
    tok_d = I.fresh_tokens(wl).cuda()
    T, seed = 0.9, 0xC0FFEE1234
    w64 = f64(w)
    for it in range(6):
        si = I.make_step(wl, step=it, planted=True, w=w, caches=caches)
        pre = tok_d.cpu().numpy()
        attn_out = torch.empty_like(si.q, device="cuda")
        pred = torch.empty(wl.M, dtype=torch.int32, device="cuda")
        conf = torch.empty(wl.M, dtype=torch.float32, device="cuda")
        nc = torch.zeros(wl.batch, dtype=torch.int32, device="cuda")
        nr = torch.zeros(wl.batch, dtype=torch.int32, device="cuda")
        dare.dare_denoise_block_sampled(ctx, si.q.cuda(), kp, vp, si.prefix_len.cuda(), si.k_blk.cuda(), si.v_blk.cuda(),
                                        None, None, None, attn_out, None, si.x.cuda(), wd, wl.mask_id, True, T, seed, it,
                                        tok_d, si.block_start, wl.mode, wl.threshold, wl.k, pred, conf, nc, nr)
        torch.cuda.synchronize()
        assert ctx.device_status() == 0
        ref = SO.denoise_step_sampled(f64(si.q), f64(si.k_pre), f64(si.v_pre), si.prefix_len.numpy(), f64(si.k_blk),
                                      f64(si.v_blk), None, None, None, f64(si.x), w64, pre, si.block_start, wl.block_len,
                                      wl.mask_id, wl.mode, wl.threshold, wl.k, T, seed, it)
        check_attn(attn_out, ref["attn_out"])
        rows = pre[:, si.block_start:si.block_start + wl.block_len].reshape(-1)
        _check(pred, conf, ref["lm"], f64(si.x), w64, rows, wl.mask_id, True, T, seed, it)
        want, wnc, wnr = O.unmask_select(pre, si.block_start, wl.block_len, pred.cpu().numpy(), conf.cpu().numpy(),
                                         wl.mask_id, wl.mode, wl.threshold, wl.k)
        np.testing.assert_array_equal(tok_d.cpu().numpy(), want)
        np.testing.assert_array_equal(nc.cpu().numpy(), wnc)
        np.testing.assert_array_equal(nr.cpu().numpy(), wnr)
        assert wnc.min() >= 1 or (rows != wl.mask_id).all()
    assert dare.dare_denoise_block_sampled(ctx, si.q.cuda(), kp, vp, si.prefix_len.cuda(), si.k_blk.cuda(),
                                           si.v_blk.cuda(), None, None, None, attn_out, None, si.x.cuda(), wd, wl.mask_id,
                                           True, 0.0, seed, 0, tok_d, si.block_start, wl.mode, wl.threshold, wl.k, pred,
                                           conf, nc, nr, check=False) == -4
