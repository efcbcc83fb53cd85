"""Pins for the oracle of the stochastic rollout epilogue (oracle/dare_sampling_oracle.py), CPU only.

  * the counter-based generator against the known-answer vectors published with its reference implementation
    (tests/golden/philox4x32_10_kat.txt);
  * the uniforms: inside (0, 1), exact in float32, flat histogram, different for different (seed, row, step);
  * the Gumbel transform: closed-form values, mean = Euler's constant, variance = pi^2 / 6;
  * the sampling law (Gumbel-max): token frequencies follow softmax(z / T), checked on a small vocabulary;
  * limits: T -> 0 gives the greedy head's token; the confidence is the temperature-1 probability of the token;
    committed rows are skipped; the mask column is never sampled;
  * perturbed_score (which judges near-ties in the GPU tests): equals the sampled head's winning score at its token,
    stays below it elsewhere, is rebuilt from the uniforms, and depends on the row, step and seed keys;
  * denoise_step_sampled: equals attention + sampled head + selection on the same inputs, keeps committed tokens and
    everything outside the block, and turns into the greedy step as T -> 0.
"""
import os

import numpy as np

from oracle import dare_oracle as O
from oracle import dare_sampling_oracle as SO

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")


def test_philox_known_answers():
    n = 0
    for line in open(GOLDEN):
        line = line.split("#")[0].strip()
        if not line:
            continue
        w = [int(t, 16) for t in line.split()]
        ctr, key, want = w[0:4], w[4:6], w[6:10]
        got = SO.philox4x32_10(np.array(ctr, dtype=np.uint32), np.array(key, dtype=np.uint32))
        assert [int(v) for v in got] == want
        n += 1
    assert n == 3


def test_philox_is_a_bijection_of_the_counter_and_vectorises():
    ctr = np.zeros((1000, 4), dtype=np.uint32)
    ctr[:, 0] = np.arange(1000)
    out = SO.philox4x32_10(ctr, np.array([7, 9], dtype=np.uint32))
    assert len({tuple(r) for r in out.tolist()}) == 1000
    one = SO.philox4x32_10(np.array([17, 0, 0, 0], dtype=np.uint32), np.array([7, 9], dtype=np.uint32))
    np.testing.assert_array_equal(out[17], one)


def test_uniforms_are_exact_float32_in_the_open_interval():
    u = SO.uniforms(seed=0x1234_5678_9ABC_DEF0, row=3, step=5, V=100003)
    assert u.shape == (100003,)
    assert u.min() > 0.0 and u.max() < 1.0
    np.testing.assert_array_equal(u.astype(np.float32).astype(np.float64), u)
    np.testing.assert_array_equal((u * 2 ** 24) % 2, 1.0)                 # odd multiples of 2^-24
    hist, _ = np.histogram(u, bins=20, range=(0, 1))
    assert np.abs(hist / len(u) - 0.05).max() < 0.004
    assert abs(u.mean() - 0.5) < 0.004
    # a different row, step or seed gives a different stream; the same triple the same one
    base = SO.uniforms(1, 2, 3, 64)
    np.testing.assert_array_equal(base, SO.uniforms(1, 2, 3, 64))
    for other in (SO.uniforms(2, 2, 3, 64), SO.uniforms(1, 3, 3, 64), SO.uniforms(1, 2, 4, 64),
                  SO.uniforms(1 + (1 << 32), 2, 3, 64)):
        assert (other != base).mean() > 0.9
    # element v is word v % 4 of block v // 4: a longer request extends a shorter one
    np.testing.assert_array_equal(SO.uniforms(1, 2, 3, 70)[:64], base)


def test_gumbel_closed_forms_and_moments():
    np.testing.assert_allclose(SO.gumbel(np.array([np.exp(-1.0)])), [0.0], atol=1e-15)
    np.testing.assert_allclose(SO.gumbel(np.array([np.exp(-np.e)])), [-1.0], atol=1e-15)
    g = SO.gumbel(SO.uniforms(11, 0, 0, 400000))
    assert abs(g.mean() - 0.5772156649) < 0.01
    assert abs(g.var() - np.pi ** 2 / 6) < 0.03


def test_sampling_law_follows_softmax_of_scaled_logits():
    rng = np.random.default_rng(0)
    V, D, T = 12, 8, 0.7
    w = rng.standard_normal((V, D))
    x = np.tile(rng.standard_normal((1, D)), (4000, 1))                   # the same row 4000 times: rows differ in noise only
    mask_id = 5
    res = SO.lmhead_sample(x, w, None, mask_id, True, T, seed=99, step=1)
    z = w @ x[0]
    z[mask_id] = -np.inf
    p = np.exp(z / T - (z / T)[np.isfinite(z)].max())
    p /= p.sum()
    freq = np.bincount(res["pred"], minlength=V) / len(x)
    assert freq[mask_id] == 0
    assert np.abs(freq - p).max() < 4.0 * np.sqrt(0.25 / len(x))          # 4 sigma of a binomial proportion
    # confidence = temperature-1 probability of the sampled token
    p1 = np.exp(z - z[np.isfinite(z)].max())
    p1 /= p1.sum()
    np.testing.assert_allclose(res["conf"], p1[res["pred"]], rtol=1e-12)


def test_low_temperature_recovers_the_greedy_head_and_rows_are_skipped():
    rng = np.random.default_rng(1)
    M, V, D = 9, 200, 16
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D))
    row_tokens = np.full(M, 150)
    row_tokens[[2, 6]] = 17                                                 # committed rows
    greedy = O.lmhead_confidence(x, w, row_tokens, 150, True)
    res = SO.lmhead_sample(x, w, row_tokens, 150, True, temperature=1e-6, seed=5, step=0)
    np.testing.assert_array_equal(res["pred"], greedy["pred"])
    np.testing.assert_allclose(res["conf"][np.isfinite(res["conf"])], greedy["conf"][np.isfinite(greedy["conf"])], rtol=1e-12)
    assert np.isneginf(res["conf"][[2, 6]]).all() and (res["pred"][[2, 6]] == 17).all()
    # at T = 1 the samples differ from the greedy tokens somewhere, and change with the step
    a = SO.lmhead_sample(x, w, None, 150, True, 1.0, seed=5, step=0)["pred"]
    b = SO.lmhead_sample(x, w, None, 150, True, 1.0, seed=5, step=1)["pred"]
    assert (a != greedy["pred"]).any() and (a != b).any()
    assert (a != 150).all() and (b != 150).all()


def test_forward_process_marginals_window_and_limits():
    """Eq. 1: P(x_t = x_0) = alpha_t per token, independently; only the window is touched; limits p = 0 and p = 1."""
    rng = np.random.default_rng(2)
    B, T, start, length, mask_id = 6, 5000, 100, 4800, 99
    x0 = rng.integers(0, 90, (B, T)).astype(np.int32)
    p = np.array([0.0, 0.1, 0.5, 0.9, 1.0, 0.3], dtype=np.float32)
    xt = SO.forward_mask(x0, start, length, p, mask_id, seed=5, sample=0)
    np.testing.assert_array_equal(xt[:, :start], x0[:, :start])
    np.testing.assert_array_equal(xt[:, start + length:], x0[:, start + length:])
    win, win0 = xt[:, start:start + length], x0[:, start:start + length]
    assert ((win == mask_id) | (win == win0)).all()                   # a token is either kept or absorbed
    frac = (win == mask_id).mean(axis=1)
    assert frac[0] == 0.0 and frac[4] == 1.0
    assert np.abs(frac - p).max() < 4 * np.sqrt(0.25 / length)
    # neighbouring positions are masked independently: P(both) = p^2
    both = ((win[2, :-1] == mask_id) & (win[2, 1:] == mask_id)).mean()
    assert abs(both - 0.25) < 0.03
    # another Monte-Carlo sample or seed gives another pattern; the same arguments the same one
    np.testing.assert_array_equal(xt, SO.forward_mask(x0, start, length, p, mask_id, 5, 0))
    assert (SO.forward_mask(x0, start, length, p, mask_id, 5, 1) != xt).any()
    assert (SO.forward_mask(x0, start, length, p, mask_id, 6, 0) != xt).any()
    # a larger p masks a superset (same uniforms, higher threshold)
    hi = SO.forward_mask(x0, start, length, np.minimum(p + 0.2, 1.0).astype(np.float32), mask_id, 5, 0)
    assert ((xt == mask_id) <= (hi == mask_id)).all()


def test_masked_nelbo_hand_worked():
    """Eq. 2 on a hand-worked case: only masked window positions count, scaled by 1 / t."""
    mask_id = 9
    xt = np.array([[1, 9, 3, 9, 9, 2], [4, 4, 9, 4, 4, 4]], dtype=np.int32)
    lp = np.log(np.array([[0.5, 0.25, 0.125, 0.5], [0.1, 0.2, 0.3, 0.4]]))         # window = positions 1..4
    nelbo, n = SO.masked_nelbo(lp, xt, 1, 4, mask_id, np.array([0.5, 0.25]))
    # row 0: window tokens 9 3 9 9 -> masked at window offsets 0, 2, 3: -(ln .5 + ln .125 + ln .5) / 0.5
    # row 1: window tokens 4 9 4 4 -> masked at offset 1: -ln .2 / 0.25
    np.testing.assert_allclose(nelbo, [2 * (np.log(2) + np.log(8) + np.log(2)), 4 * np.log(5)], rtol=1e-14)
    np.testing.assert_array_equal(n, [3, 1])
    # with every window token masked at t = 1 it is the summed cross-entropy
    xt2 = np.full((2, 6), mask_id, dtype=np.int32)
    nelbo2, _ = SO.masked_nelbo(lp, xt2, 1, 4, mask_id, np.array([1.0, 1.0]))
    np.testing.assert_allclose(nelbo2, -lp.sum(axis=1), rtol=1e-14)


def test_perturbed_score_is_the_winning_score_of_the_sampled_head_and_is_keyed_by_row_and_step():
    """perturbed_score judges near-ties in the GPU tests, so a wrong row, step or seed key, a dropped temperature or
    a forgotten mask column there must show: at the sampled token it has to reproduce the head's own best score,
    at every other token it has to stay below it, and it is rebuilt here from the uniforms without the function."""
    rng = np.random.default_rng(3)
    M, V, D, mask_id, T, seed, step = 7, 90, 12, 40, 0.6, 0xABCDEF0123, 9
    x, w = rng.standard_normal((M, D)), rng.standard_normal((V, D))
    res = SO.lmhead_sample(x, w, None, mask_id, True, T, seed, step)
    for m in range(M):
        ys = np.array([SO.perturbed_score(x[m], w, v, m, mask_id, True, T, seed, step) for v in range(V)])
        assert int(np.argmax(ys)) == res["pred"][m]
        assert ys[res["pred"][m]] == res["y_best"][m]
        assert ys[mask_id] == -np.inf                                       # the excluded column can never win
        second = np.sort(ys)[-2]
        np.testing.assert_allclose(res["gap_y"][m], ys.max() - second, rtol=1e-12)
        # rebuilt from the definition: z / T - ln(-ln u), u of (seed, row m, step)
        u = SO.uniforms(seed, m, step, V)
        z = w @ x[m]
        want = z / T - np.log(-np.log(u))
        keep = np.arange(V) != mask_id
        np.testing.assert_allclose(ys[keep], want[keep], rtol=1e-13)
        # another row, step or seed key gives other scores; without the exclusion flag the mask column is finite
        assert SO.perturbed_score(x[m], w, 3, m + 1, mask_id, True, T, seed, step) != ys[3]
        assert SO.perturbed_score(x[m], w, 3, m, mask_id, True, T, seed, step + 1) != ys[3]
        assert SO.perturbed_score(x[m], w, 3, m, mask_id, True, T, seed + 1, step) != ys[3]
        assert np.isfinite(SO.perturbed_score(x[m], w, mask_id, m, mask_id, False, T, seed, step))


def _tiny_step_inputs(rng, B=2, L=4, Hq=2, Hkv=1, d=8, P=5, V=30, mask_id=29):
    D = Hq * d
    q = rng.standard_normal((B, L, Hq, d))
    k_pre, v_pre = rng.standard_normal((B, Hkv, P + L, d)), rng.standard_normal((B, Hkv, P + L, d))
    plen = np.array([P, P - 2][:B])
    x, w = rng.standard_normal((B * L, D)), rng.standard_normal((V, D))
    tokens = rng.integers(0, mask_id, (B, P + L + 3)).astype(np.int32)
    tokens[:, P:P + L] = mask_id
    tokens[0, P + 1] = 4                                                    # one position already committed
    return q, k_pre, v_pre, plen, x, w, tokens, P, L, mask_id


def test_sampled_step_is_attention_plus_sampled_head_plus_selection_and_reduces_to_the_greedy_step():
    rng = np.random.default_rng(4)
    q, k_pre, v_pre, plen, x, w, tokens, P, L, mask_id = _tiny_step_inputs(rng)
    T, seed, step = 0.8, 77, 3
    for mode, thr, k in ((O.SELECT_THRESHOLD, 0.2, 0), (O.SELECT_TOPK, 0.0, 2)):
        res = SO.denoise_step_sampled(q, k_pre, v_pre, plen, None, None, None, None, None, x, w, tokens, P, L, mask_id,
                                      mode, thr, k, T, seed, step)
        # composition of the three separately pinned parts, on the same inputs
        o, lse = O.attn_block(q, k_pre, v_pre, plen)
        np.testing.assert_array_equal(res["attn_out"], o)
        np.testing.assert_array_equal(res["lse"], lse)
        lm = SO.lmhead_sample(x, w, tokens[:, P:P + L].reshape(-1), mask_id, True, T, seed, step)
        np.testing.assert_array_equal(res["lm"]["pred"], lm["pred"])
        np.testing.assert_array_equal(res["lm"]["conf"], lm["conf"])
        tok, nc, nr = O.unmask_select(tokens, P, L, lm["pred"], lm["conf"].astype(np.float32), mask_id, mode, thr, k)
        np.testing.assert_array_equal(res["tokens"], tok)
        np.testing.assert_array_equal(res["n_committed"], nc)
        np.testing.assert_array_equal(res["n_remaining"], nr)
        # invariants of a step: committed positions and everything outside the block keep their tokens; a commit
        # removes a mask; the committed row of the block echoes its token with confidence -inf
        assert res["tokens"][0, P + 1] == 4 and res["lm"]["pred"][1] == 4 and np.isneginf(res["lm"]["conf"][1])
        outside = np.ones_like(tokens, dtype=bool)
        outside[:, P:P + L] = False
        np.testing.assert_array_equal(res["tokens"][outside], tokens[outside])
        assert (nc >= 1).all() and (nc + nr == (tokens[:, P:P + L] == mask_id).sum(axis=1)).all()
        # T -> 0: the sampled step is the greedy step
        cold = SO.denoise_step_sampled(q, k_pre, v_pre, plen, None, None, None, None, None, x, w, tokens, P, L, mask_id,
                                       mode, thr, k, 1e-7, seed, step)
        greedy = O.denoise_step(q, k_pre, v_pre, plen, None, None, None, None, None, x, w, tokens, P, L, mask_id, mode,
                                thr, k)
        np.testing.assert_array_equal(cold["tokens"], greedy["tokens"])
        np.testing.assert_array_equal(cold["n_committed"], greedy["n_committed"])
        np.testing.assert_allclose(cold["lm"]["conf"], greedy["lm"]["conf"], rtol=1e-12)
    # the step index keys the noise: another step draws other tokens somewhere
    a = SO.denoise_step_sampled(q, k_pre, v_pre, plen, None, None, None, None, None, x, w, tokens, P, L, mask_id,
                                O.SELECT_TOPK, 0.0, 4, 1.5, seed, 0)["lm"]["pred"]
    b = SO.denoise_step_sampled(q, k_pre, v_pre, plen, None, None, None, None, None, x, w, tokens, P, L, mask_id,
                                O.SELECT_TOPK, 0.0, 4, 1.5, seed, 1)["lm"]["pred"]
    assert (a != b).any()
