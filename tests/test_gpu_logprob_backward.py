"""GPU parity of the backward of the log-probability head (dare_lmhead_logprob_backward) against the fp64 oracle.

Three things are checked, each with the bar its arithmetic gives:
  * dz = g (onehot - softmax), stored as bf16: the softmax inherits the forward head's error (2e-2 in log, the
    bar of the log-probability itself), so |dz - ref| <= 3e-2 |g| p + one bf16 step of the value; the transposed
    copy equals the first one bit for bit;
  * the two products on their own (d_hidden = dz . w, d_w = dz^T . hidden) against fp64 products of the GPU's own
    bf16 dz: one bf16 step of the result plus the fp32 accumulation floor;
  * end to end against the oracle's dx and dw: relative L2 error <= 2e-2 (dz is rounded to bf16 before the
    products, and carries the softmax error above).
"""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import f64

pytestmark = pytest.mark.gpu

BF16_STEP = 2.0 ** -7
REL_L2 = 2e-2


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    c.close()


def _inputs(M, D, V, mu, seed, excl):
    x = I.normal_bf16(seed, I.TID_X, (M, D))
    w = I.normal_bf16(seed, I.TID_W, (V, D), 0.05)
    t = I.uniform_int(seed, I.TID_TOK, (M,), 0, V - 1)
    if M >= 8:
        t[1] = -1                                   # outside the vocabulary: no gradient
        t[3] = mu                                   # the excluded column as a target (only matters with excl)
    g = I.normal_bf16(seed, I.TID_Q, (M,)).float()
    g[5 % M] = 0.0
    return x, w, t, g


def _run(ctx, x, w, t, g, mu, excl):
    xd, wd = x.cuda(), w.cuda()
    w_t = dare.dare_transpose_bf16(ctx, wd)
    lse = torch.empty(x.shape[0], dtype=torch.float32, device="cuda")
    dare.dare_lmhead_logprob(ctx, xd, wd, t.cuda(), mu, excl, lse=lse)
    out = dare.dare_lmhead_logprob_backward(ctx, xd, wd, w_t, t.cuda(), lse, g.cuda(), mu, excl)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    return out, w_t


def _rel_l2(got, ref):
    return np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)


def _close_product(got_t, ref, k_terms_abs):
    """bf16 result of an fp32-accumulated product: one bf16 step of the value plus the accumulation floor."""
    got = got_t.float().cpu().double().numpy()
    assert np.isfinite(got).all()
    bound = BF16_STEP * np.abs(ref) + 1e-5 * k_terms_abs + 1e-9
    assert (np.abs(got - ref) <= bound).all(), f"max excess {(np.abs(got - ref) - bound).max()}"


@pytest.mark.parametrize("M,D,V,mu,excl", [
    (32, 256, 4096, 4095, False),
    (304, 1024, 2600, 2599, True),          # several row and vocabulary tiles with tails; excluded column
    (136, 64, 520, 5, True),
    (8, 8, 8, 1, False),
])
def test_backward_matches_oracle(ctx, M, D, V, mu, excl):
    x, w, t, g = _inputs(M, D, V, mu, M + V, excl)
    (d_hidden, d_w, dz, dzt), w_t = _run(ctx, x, w, t, g, mu, excl)
    assert torch.equal(w_t.cpu(), w.t().contiguous())
    dx_ref, dw_ref, dz_ref = O.lmhead_logprob_backward(f64(x), f64(w), t.numpy(), g.double().numpy(), mu, excl)

    # ---- dz and its transpose
    assert torch.equal(dzt, dz.t().contiguous())
    got_dz = dz.float().cpu().double().numpy()
    ga = np.abs(g.double().numpy())[:, None]
    onehot = np.zeros_like(dz_ref)
    ok = (t.numpy() >= 0) & (t.numpy() < V) & ~((t.numpy() == mu) & excl)
    onehot[np.nonzero(ok)[0], t.numpy()[ok]] = 1.0
    with np.errstate(divide="ignore", invalid="ignore"):
        p = np.where(ga > 0, onehot - dz_ref / np.where(ga > 0, g.double().numpy()[:, None], 1.0), 0.0)
    bound = 3e-2 * ga * np.abs(p) + 2.0 ** -8 * np.abs(dz_ref) + 1e-9
    assert (np.abs(got_dz - dz_ref) <= bound).all()
    assert (got_dz[~ok] == 0).all()                                   # rows without a valid target
    if excl:
        assert (got_dz[:, mu] == 0).all()

    # ---- the two products on their own, from the GPU's dz
    _close_product(d_hidden, got_dz @ f64(w), np.abs(got_dz) @ np.abs(f64(w)))
    _close_product(d_w, got_dz.T @ f64(x), np.abs(got_dz).T @ np.abs(f64(x)))

    # ---- end to end
    assert _rel_l2(d_hidden.float().cpu().double().numpy(), dx_ref) <= REL_L2
    assert _rel_l2(d_w.float().cpu().double().numpy(), dw_ref) <= REL_L2


def test_backward_rejects_bad_arguments(ctx):
    x = torch.zeros(16, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(24, 64, dtype=torch.bfloat16, device="cuda")
    w_t = torch.zeros(64, 24, dtype=torch.bfloat16, device="cuda")
    t = torch.zeros(16, dtype=torch.int32, device="cuda")
    f = torch.zeros(16, dtype=torch.float32, device="cuda")
    assert dare.dare_lmhead_logprob_backward(ctx, x[:12], w, w_t, t[:12], f[:12], f[:12], check=False) == -2   # M % 8
    w20 = torch.zeros(20, 64, dtype=torch.bfloat16, device="cuda")
    w20_t = torch.zeros(64, 20, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_lmhead_logprob_backward(ctx, x, w20, w20_t, t, f, f, check=False) == -2                 # V % 8
    assert dare.dare_transpose_bf16(ctx, x, out=x, check=False) == -4                                        # in place


def test_backward_full_size_sampled(ctx):
    """LLaDA-8B-shaped head (512 x 4096 x 126464): dz of 12 sampled rows and d_hidden of those rows against the
    oracle (rows are independent); d_w on sampled vocabulary rows against the fp64 product of the GPU's own dz."""
    wl = I.WORKLOADS["llada8b"]
    rng = np.random.default_rng(5)
    w = I.make_weights(wl)
    x = I.normal_bf16(0, I.TID_X, (wl.M, wl.hidden))
    t = I.uniform_int(0, I.TID_TOK, (wl.M,), 0, wl.vocab - 1)
    g = I.normal_bf16(0, I.TID_Q, (wl.M,)).float()
    (d_hidden, d_w, dz, dzt), _ = _run(ctx, x, w, t, g, wl.mask_id, True)
    rows = np.sort(rng.choice(wl.M, size=12, replace=False))
    w64 = f64(w)
    dx_ref, _, dz_ref = O.lmhead_logprob_backward(f64(x[rows]), w64, t.numpy()[rows], g.double().numpy()[rows],
                                                  wl.mask_id, True)
    got_dz = dz[rows].float().cpu().double().numpy()
    # away from a row's target column dz = -g p, so the softmax bar (3e-2 relative) applies to dz itself; at the
    # target column dz = g (1 - p) with p ~ 1e-5 here: one bf16 step
    assert (np.abs(got_dz - dz_ref) <= 3e-2 * np.abs(dz_ref) + 1e-9).all()
    assert _rel_l2(got_dz, dz_ref) <= 1e-2
    assert _rel_l2(d_hidden[rows].float().cpu().double().numpy(), dx_ref) <= REL_L2
    assert torch.equal(dzt[:, rows[0]], dz[rows[0]])
    cols = np.sort(rng.choice(wl.vocab, size=24, replace=False))
    cols[0] = int(t[rows[0]])                                       # one column that is some row's target
    dz_cols = dz[:, cols].float().cpu().double().numpy()            # [M, 24]
    ref_dw = dz_cols.T @ f64(x)
    _close_product(d_w[cols], ref_dw, np.abs(dz_cols).T @ np.abs(f64(x)))
    assert (d_w[wl.mask_id] == 0).all()
