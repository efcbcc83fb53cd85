"""Pins for the oracle's unmask selection (CPU only)."""
import os

import numpy as np
import pytest

from oracle import dare_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "select_cases.txt")


def _cases():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            head, tok, pred, conf, exp, cnt = [s.split() for s in line.split("|")]
            out.append((head[0], float(head[1]), int(head[2]), int(head[3]), int(head[4]),
                        [int(t) for t in tok], [int(t) for t in pred], [float(c) for c in conf],
                        [int(t) for t in exp], int(cnt[0]), int(cnt[1])))
    return out


@pytest.mark.parametrize("case", _cases())
def test_hand_worked_cases(case):
    mode, par, mu, bs, L, tok, pred, conf, exp, nc, nr = case
    m = O.SELECT_THRESHOLD if mode == "threshold" else O.SELECT_TOPK
    t, c, r = O.unmask_select(np.array([tok], np.int32), bs, L, np.array([pred]), np.array([conf], np.float32),
                              mu, m, threshold=par, k=int(par) if mode == "topk" else 1)
    assert t[0].tolist() == exp and int(c[0]) == nc and int(r[0]) == nr


def _second_opinion(tok, bs, L, pred, conf, mu, mode, thr, k):
    """Written differently on purpose: a scan for the threshold rule, repeated max-extraction for top-k."""
    tok = tok.copy()
    for r in range(tok.shape[0]):
        masked = np.array([tok[r, bs + i] == mu for i in range(L)])
        c = np.where(np.isnan(conf[r]), -np.inf, conf[r]).astype(np.float32)
        chosen = np.zeros(L, bool)
        if mode == O.SELECT_THRESHOLD:
            chosen = masked & (c > np.float32(thr))
            if masked.any() and not chosen.any():
                best = -1
                for i in range(L):
                    if masked[i] and (best < 0 or c[i] > c[best]):
                        best = i
                chosen[best] = True
        else:
            avail = masked.copy()
            for _ in range(min(k, int(masked.sum()))):
                best = -1
                for i in range(L):
                    if avail[i] and (best < 0 or c[i] > c[best]):
                        best = i
                chosen[best] = True
                avail[best] = False
        for i in range(L):
            if chosen[i]:
                tok[r, bs + i] = pred[r, i]
    return tok


@pytest.mark.parametrize("seed", range(30))
def test_random_against_second_implementation_and_invariants(seed):
    rng = np.random.default_rng(seed)
    B, L = int(rng.integers(1, 5)), int(rng.integers(1, 40))
    bs = int(rng.integers(0, 5)); tail = int(rng.integers(0, 4))
    mu = 1000
    tok = rng.integers(0, 999, (B, bs + L + tail)).astype(np.int32)
    blockmask = rng.random((B, L)) < rng.random()
    tok[:, bs:bs + L][blockmask] = mu
    tok[:, :bs][rng.random((B, bs)) < 0.3] = mu      # masks outside the block must be left alone
    pred = rng.integers(0, 999, (B, L)).astype(np.int32)
    conf = rng.random((B, L)).astype(np.float32)
    conf[rng.random((B, L)) < 0.3] = np.float32(0.5)  # ties
    if seed % 5 == 0:
        conf[rng.random((B, L)) < 0.1] = np.nan
    mode = O.SELECT_THRESHOLD if seed % 2 == 0 else O.SELECT_TOPK
    thr, k = float(rng.choice([0.3, 0.5, 0.9, 2.0, -1.0])), int(rng.integers(1, 6))
    new, nc, nr = O.unmask_select(tok, bs, L, pred, conf, mu, mode, thr, k)
    np.testing.assert_array_equal(new, _second_opinion(tok, bs, L, pred, conf, mu, mode, thr, k))
    changed = new != tok
    assert not changed[:, :bs].any() and not changed[:, bs + L:].any()
    assert (tok[changed] == mu).all()                           # only masks change
    was_masked = (tok[:, bs:bs + L] == mu)
    U = was_masked.sum(1)
    np.testing.assert_array_equal(nc + nr, U)
    for r in range(B):
        c = np.where(np.isnan(conf[r]), -np.inf, conf[r])
        if mode == O.SELECT_TOPK:
            assert nc[r] == min(k, U[r])
        else:
            above = int((was_masked[r] & (c > np.float32(thr))).sum())
            assert nc[r] == (max(1, above) if U[r] else 0)
        # every committed position carries its prediction
        for i in range(L):
            if was_masked[r, i] and new[r, bs + i] != mu:
                assert new[r, bs + i] == pred[r, i]


def test_limits_of_threshold_and_k():
    mu, L = 50, 8
    tok = np.full((1, L), mu, np.int32)
    pred = np.arange(L, dtype=np.int32)[None]
    conf = np.linspace(0.1, 0.8, L, dtype=np.float32)[None]
    t, nc, nr = O.unmask_select(tok, 0, L, pred, conf, mu, O.SELECT_THRESHOLD, threshold=-np.inf)
    assert nc[0] == L and nr[0] == 0 and (t[0] == pred[0]).all()
    t, nc, nr = O.unmask_select(tok, 0, L, pred, conf, mu, O.SELECT_TOPK, k=L + 3)
    assert nc[0] == L and (t[0] == pred[0]).all()
    # tau >= 1: exactly one commit per step, so exactly L steps, in descending-confidence order
    order = []
    cur = tok
    for _ in range(L):
        new, nc, nr = O.unmask_select(cur, 0, L, pred, conf, mu, O.SELECT_THRESHOLD, threshold=1.0)
        assert nc[0] == 1
        order.append(int(np.nonzero(new[0] != cur[0])[0][0]))
        cur = new
    assert order == list(range(L - 1, -1, -1)) and (cur != mu).all()


def test_comparison_is_done_in_float32():
    """0.9 as float32 is 0.89999998; a float32 confidence equal to it must not pass a strict '>'."""
    mu = 9
    tok = np.array([[mu, mu]], np.int32)
    conf = np.array([[np.float32(0.9), np.nextafter(np.float32(0.9), np.float32(1))]], np.float32)
    t, nc, _ = O.unmask_select(tok, 0, 2, np.array([[1, 2]]), conf, mu, O.SELECT_THRESHOLD, threshold=0.9)
    assert t[0].tolist() == [mu, 2] and nc[0] == 1
