"""GPU parity of the logits-free log-probability head (dare_lmhead_logprob) against the fp64 oracle.

Bars: log-probability within 2e-2 absolute (the bar used for the log-confidence of the greedy head; the error is
the bf16 products' fp32 accumulation over D plus the fast exponentials of the partition sum), log-sum-exp likewise.
"""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import LOGCONF_ABS, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    c.close()


def _case(ctx, M, D, V, mu, excl, seed, planted=False):
    wl = I.scaled(I.WORKLOADS["tiny"], hidden=D, vocab=V, mask_id=mu, seed=seed)
    x = I.normal_bf16(seed, I.TID_X, (M, D))
    w = I.normal_bf16(seed, I.TID_W, (V, D), 0.05 if planted else 0.02)
    t = I.uniform_int(seed, I.TID_TOK, (M,), 0, V - 1)
    if planted:
        x, cols = I.plant_confidences(wl, x, w, 0)
        t[::2] = cols[::2].to(torch.int32)                     # half of the targets are the planted (likely) tokens
    lp_ref, lse_ref = O.lmhead_logprob(f64(x), f64(w), t.numpy(), mu, excl)
    lse = torch.empty(M, dtype=torch.float32, device="cuda")
    lp = dare.dare_lmhead_logprob(ctx, x.cuda(), w.cuda(), t.cuda(), mu, excl, lse=lse)
    torch.cuda.synchronize()
    got, got_lse = lp.cpu().double().numpy(), lse.cpu().double().numpy()
    fin = np.isfinite(lp_ref)
    assert np.isneginf(got[~fin]).all()
    assert np.abs(got[fin] - lp_ref[fin]).max() <= LOGCONF_ABS
    assert np.abs(got_lse - lse_ref).max() <= LOGCONF_ABS
    assert ctx.device_status() == 0
    return got, lp_ref


@pytest.mark.parametrize("M,D,V,mu,excl", [
    (32, 256, 4096, 4095, False),
    (300, 1024, 2560 + 40, 2599, True),       # several row and vocabulary tiles with tails; excluded column
    (130, 64, 520, 5, False),
    (1, 8, 2, 1, False),
])
def test_logprob_matches_oracle(ctx, M, D, V, mu, excl):
    _case(ctx, M, D, V, mu, excl, seed=M + V)


def test_logprob_of_likely_and_unlikely_targets(ctx):
    got, ref = _case(ctx, 128, 256, 1024, 1023, False, seed=4, planted=True)
    assert (ref > np.log(0.3)).sum() >= 5 and (ref < np.log(1e-3)).sum() >= 5    # both regimes are present


def test_logprob_bad_targets_and_consistency_with_the_greedy_head(ctx):
    M, D, V, mu = 64, 128, 1000, 999
    x = I.normal_bf16(8, I.TID_X, (M, D)).cuda()
    w = I.normal_bf16(8, I.TID_W, (V, D), 0.05).cuda()
    pred, conf = dare.dare_lmhead_confidence(ctx, x, w, None, mu, True)
    lp = dare.dare_lmhead_logprob(ctx, x, w, pred, mu, True)          # log-probability of the greedy token = log confidence
    torch.cuda.synchronize()
    assert torch.allclose(lp, conf.log(), atol=1e-4)
    t = pred.clone()
    t[0], t[1], t[2] = -1, V, mu                                      # out of range twice, then the excluded column
    lp2 = dare.dare_lmhead_logprob(ctx, x, w, t, mu, True)
    torch.cuda.synchronize()
    assert torch.isneginf(lp2[:3]).all() and torch.equal(lp2[3:], lp[3:])
    assert dare.dare_lmhead_logprob(ctx, x, w, None, mu, True, check=False) == -1


def test_logprob_full_size_sampled_rows(ctx):
    wl = I.WORKLOADS["llada8b"]
    rng = np.random.default_rng(5)
    w = I.make_weights(wl)
    x = I.normal_bf16(0, I.TID_X, (wl.M, wl.hidden))
    t = I.uniform_int(1, I.TID_TOK, (wl.M,), 0, wl.vocab - 1)
    lp = dare.dare_lmhead_logprob(ctx, x.cuda(), w.cuda(), t.cuda(), wl.mask_id, False)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    rows = np.sort(rng.choice(wl.M, size=24, replace=False))
    ref, _ = O.lmhead_logprob(f64(x[rows]), f64(w), t.numpy()[rows], wl.mask_id, False)
    assert np.abs(lp.cpu().double().numpy()[rows] - ref).max() <= LOGCONF_ABS
    assert torch.isfinite(lp).all() and (lp < 0).all()
