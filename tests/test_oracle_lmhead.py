"""Pins for the oracle's LM head + vocabulary softmax (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O


def test_against_library_log_softmax():
    rng = np.random.default_rng(0)
    M, D, V, mu = 9, 16, 50, 17
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D))
    r = O.lmhead_confidence(x, w, None, mu, True)
    z = torch.from_numpy(x) @ torch.from_numpy(w).T
    z[:, mu] = -float("inf")
    lp = torch.log_softmax(z, dim=1)
    best, idx = lp.max(dim=1)
    np.testing.assert_array_equal(r["pred"], idx.numpy().astype(np.int32))
    np.testing.assert_allclose(r["logconf"], best.numpy(), atol=1e-12)
    np.testing.assert_allclose(r["conf"], best.exp().numpy(), atol=1e-13)
    top2 = torch.topk(lp, 2, dim=1).values
    np.testing.assert_allclose(r["second"], top2[:, 1].exp().numpy(), atol=1e-13)
    np.testing.assert_allclose(r["gap_logit"], (top2[:, 0] - top2[:, 1]).numpy(), atol=1e-12)
    assert (r["pred"] != mu).all()


def test_without_exclusion_matches_raw_softmax():
    rng = np.random.default_rng(1)
    x, w = rng.standard_normal((4, 8)), rng.standard_normal((12, 8))
    w[5] = 10 * x[2] / np.linalg.norm(x[2])          # make column 5 the clear winner for row 2
    r = O.lmhead_confidence(x, w, None, 5, False)
    p = torch.softmax(torch.from_numpy(x @ w.T), dim=1).numpy()
    np.testing.assert_allclose(r["conf"], p.max(1), atol=1e-13)
    assert r["pred"][2] == 5
    r2 = O.lmhead_confidence(x, w, None, 5, True)
    assert r2["pred"][2] != 5


@pytest.mark.parametrize("mu", [0, 3, 9])
def test_uniform_logits_closed_form_and_lowest_index_tie_break(mu):
    """Identical weight rows: every admissible column ties; conf = 1/(V-1); token = lowest admissible id."""
    rng = np.random.default_rng(2)
    M, D, V = 5, 8, 10
    x = rng.standard_normal((M, D))
    w = np.tile(rng.standard_normal((1, D)), (V, 1))
    r = O.lmhead_confidence(x, w, None, mu, True)
    np.testing.assert_allclose(r["conf"], 1.0 / (V - 1), rtol=1e-13)
    assert (r["pred"] == (1 if mu == 0 else 0)).all()
    r0 = O.lmhead_confidence(np.zeros((M, D)), rng.standard_normal((V, D)), None, mu, True)
    np.testing.assert_allclose(r0["conf"], 1.0 / (V - 1), rtol=1e-13)
    assert (r0["pred"] == (1 if mu == 0 else 0)).all()


def test_planted_column_closed_form():
    """Orthonormal weight rows: x = a e_c gives z_c = a and zero elsewhere, so conf = e^a / (e^a + V' - 1)."""
    V, D, mu = 6, 8, 5
    w = np.eye(V, D)
    a = np.array([0.5, 2.0, 7.0])
    cols = np.array([1, 4, 0])
    x = np.zeros((3, D)); x[np.arange(3), cols] = a
    r = O.lmhead_confidence(x, w, None, mu, True)
    np.testing.assert_array_equal(r["pred"], cols)
    np.testing.assert_allclose(r["conf"], np.exp(a) / (np.exp(a) + (V - 1) - 1), rtol=1e-13)
    np.testing.assert_allclose(r["second"], 1.0 / (np.exp(a) + (V - 1) - 1), rtol=1e-13)
    np.testing.assert_allclose(r["gap_logit"], a, rtol=1e-13)


def test_transposed_weight_would_be_caught():
    """A non-square, asymmetric case where x w^T differs from any transposed reading."""
    x = np.array([[1.0, 0.0, 0.0]])
    w = np.array([[0.0, 5.0, 0.0], [3.0, 0.0, 0.0], [0.0, 0.0, 9.0], [1.0, 1.0, 1.0]])
    r = O.lmhead_confidence(x, w, None, -1, False)
    assert r["pred"][0] == 1
    z = np.array([0.0, 3.0, 0.0, 1.0])
    np.testing.assert_allclose(r["conf"][0], np.exp(3.0) / np.exp(z).sum(), rtol=1e-14)


def test_committed_rows_are_skipped():
    rng = np.random.default_rng(3)
    x, w = rng.standard_normal((6, 4)), rng.standard_normal((9, 4))
    rt = np.array([8, 2, 8, 8, 0, 8], dtype=np.int32)
    r = O.lmhead_confidence(x, w, rt, 8, True)
    full = O.lmhead_confidence(x, w, None, 8, True)
    for m in range(6):
        if rt[m] == 8:
            assert r["pred"][m] == full["pred"][m] and r["conf"][m] == full["conf"][m]
        else:
            assert r["pred"][m] == rt[m] and r["conf"][m] == -np.inf


def test_confidence_bounds_and_token_probability():
    rng = np.random.default_rng(4)
    M, D, V, mu = 20, 32, 40, 39
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D))
    r = O.lmhead_confidence(x, w, None, mu, True)
    assert (r["conf"] >= 1.0 / (V - 1) - 1e-15).all() and (r["conf"] <= 1.0).all()
    assert (r["second"] <= r["conf"]).all()
    for m in range(M):
        assert abs(O.token_probability(x[m], w, int(r["pred"][m]), mu, True) - r["conf"][m]) < 1e-14
        tot = sum(O.token_probability(x[m], w, v, mu, True) for v in range(V))
        assert abs(tot - 1.0) < 1e-12


def test_logprob_is_library_log_softmax_gather_and_cross_entropy():
    """lmhead_logprob against torch: log_softmax + gather, and -cross_entropy; closed forms; exclusion; bad targets."""
    rng = np.random.default_rng(11)
    M, D, V = 13, 24, 97
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D))
    t = rng.integers(0, V, M)
    lp, lse = O.lmhead_logprob(x, w, t)
    z = torch.from_numpy(x) @ torch.from_numpy(w).T
    want = torch.log_softmax(z, dim=1).gather(1, torch.from_numpy(t)[:, None])[:, 0].numpy()
    np.testing.assert_allclose(lp, want, atol=1e-12)
    np.testing.assert_allclose(-lp, torch.nn.functional.cross_entropy(z, torch.from_numpy(t), reduction="none").numpy(), atol=1e-12)
    np.testing.assert_allclose(lse, torch.logsumexp(z, dim=1).numpy(), atol=1e-12)
    # identical weight rows: every token has probability 1 / V (1 / (V - 1) with one column excluded)
    w1 = np.tile(rng.standard_normal((1, D)), (V, 1))
    np.testing.assert_allclose(O.lmhead_logprob(x, w1, t)[0], -np.log(V), atol=1e-12)
    t2 = np.where(t == 5, 6, t)
    np.testing.assert_allclose(O.lmhead_logprob(x, w1, t2, 5, True)[0], -np.log(V - 1), atol=1e-12)
    # the excluded column and out-of-range targets have probability zero
    bad = np.array([5, -1, V, 3])
    lpb, _ = O.lmhead_logprob(x[:4], w, bad, 5, True)
    assert np.isneginf(lpb[:3]).all() and np.isfinite(lpb[3])
    # exp(logprob) summed over all targets is 1; consistent with the greedy head's confidence
    allp = np.stack([np.exp(O.lmhead_logprob(x[:2], w, np.full(2, v))[0]) for v in range(V)], axis=1)
    np.testing.assert_allclose(allp.sum(axis=1), 1.0, atol=1e-12)
    g = O.lmhead_confidence(x, w, None, -1, False)
    np.testing.assert_allclose(np.exp(O.lmhead_logprob(x, w, g["pred"])[0]), g["conf"], rtol=1e-12)


def test_logprob_backward_is_autograd_and_finite_differences():
    """lmhead_logprob_backward against torch autograd of log_softmax + gather (a library routine written
    independently of the oracle), against central differences of the oracle's own forward, and by invariants."""
    import torch
    rng = np.random.default_rng(11)
    M, D, V, mu = 7, 12, 23, 5
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D)) * 0.5
    t = rng.integers(0, V, M)
    t[t == mu] = 6
    g = rng.standard_normal(M)
    for excl in (False, True):
        dx, dw, dz = O.lmhead_logprob_backward(x, w, t, g, mu, excl)
        xt = torch.tensor(x, requires_grad=True)
        wt = torch.tensor(w, requires_grad=True)
        z = xt @ wt.T
        if excl:
            z = z.masked_fill(torch.arange(V)[None, :] == mu, float("-inf"))
        lp = torch.log_softmax(z, dim=1).gather(1, torch.tensor(t)[:, None])[:, 0]
        (lp * torch.tensor(g)).sum().backward()
        np.testing.assert_allclose(dx, xt.grad.numpy(), atol=1e-12)
        np.testing.assert_allclose(dw, wt.grad.numpy(), atol=1e-12)
        # invariants: each row of dz sums to 0 (softmax is shift invariant); the excluded column gets nothing
        np.testing.assert_allclose(dz.sum(axis=1), 0.0, atol=1e-12)
        if excl:
            assert (dz[:, mu] == 0).all() and (dw[mu] == 0).all()
    # central differences of the forward oracle on a few coordinates
    f = lambda xx, ww: float((g * O.lmhead_logprob(xx, ww, t, mu, True)[0]).sum())
    dx, dw, _ = O.lmhead_logprob_backward(x, w, t, g, mu, True)
    h = 1e-6
    for (i, j) in [(0, 0), (3, 7), (6, 11)]:
        xp, xm = x.copy(), x.copy()
        xp[i, j] += h
        xm[i, j] -= h
        assert abs((f(xp, w) - f(xm, w)) / (2 * h) - dx[i, j]) < 1e-6
    for (v, j) in [(0, 0), (int(t[2]), 3), (22, 11)]:
        wp, wm = w.copy(), w.copy()
        wp[v, j] += h
        wm[v, j] -= h
        assert abs((f(x, wp) - f(x, wm)) / (2 * h) - dw[v, j]) < 1e-6
    # a row with zero upstream gradient, an out-of-range target or the excluded column as target contributes nothing
    g2 = g.copy()
    g2[1] = 0.0
    t2 = t.copy()
    t2[2], t2[4] = -1, mu
    dx2, dw2, dz2 = O.lmhead_logprob_backward(x, w, t2, g2, mu, True)
    assert (dz2[[1, 2, 4]] == 0).all() and (dx2[[1, 2, 4]] == 0).all()
    keep = np.array([0, 3, 5, 6])
    dxk, dwk, _ = O.lmhead_logprob_backward(x[keep], w, t2[keep], g2[keep], mu, True)
    np.testing.assert_allclose(dw2, dwk, atol=1e-12)
    np.testing.assert_allclose(dx2[keep], dxk, atol=1e-12)
