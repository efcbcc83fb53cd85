"""GPU parity: every kernel, through the C ABI, against the fp64 CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import check_attn, check_lmhead, dev, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    torch.cuda.synchronize()
    assert c.device_status() == 0
    c.close()


# ----------------------------------------------------------------------------- selection (bit-exact)
@pytest.mark.parametrize("seed", range(12))
def test_select_bit_exact(ctx, seed):
    rng = np.random.default_rng(seed)
    B = int(rng.integers(1, 70))
    L = int(rng.choice([1, 4, 32, 33, 200, 1024]))
    bs, tail = int(rng.integers(0, 40)), int(rng.integers(0, 9))
    mu = 126336
    tok = rng.integers(0, 126000, (B, bs + L + tail)).astype(np.int32)
    tok[:, bs:bs + L][rng.random((B, L)) < rng.random()] = mu
    tok[:, :bs][rng.random((B, bs)) < 0.2] = mu
    pred = rng.integers(0, 126000, (B, L)).astype(np.int32)
    conf = rng.random((B, L)).astype(np.float32)
    conf[rng.random((B, L)) < 0.25] = np.float32(0.5)
    if seed % 3 == 0:
        conf[rng.random((B, L)) < 0.05] = np.nan
    if seed % 4 == 1:
        conf[rng.random((B, L)) < 0.3] = -np.inf          # committed rows' confidences from the LM head
    mode = O.SELECT_THRESHOLD if seed % 2 == 0 else O.SELECT_TOPK
    thr, k = float(rng.choice([0.3, 0.9, 0.95, 1.5])), int(rng.integers(1, 5))
    want, nc, nr = O.unmask_select(tok, bs, L, pred, conf, mu, mode, thr, k)
    t = torch.from_numpy(tok).cuda()
    ncd = torch.zeros(B, dtype=torch.int32, device="cuda")
    nrd = torch.zeros(B, dtype=torch.int32, device="cuda")
    dare.dare_unmask_select(ctx, t, bs, L, torch.from_numpy(pred).cuda(), torch.from_numpy(conf).cuda(), mu, mode,
                            thr, k, ncd, nrd)
    np.testing.assert_array_equal(t.cpu().numpy(), want)
    np.testing.assert_array_equal(ncd.cpu().numpy(), nc)
    np.testing.assert_array_equal(nrd.cpu().numpy(), nr)


def test_select_empty_block_and_all_committed(ctx):
    mu = 7
    tok = np.array([[1, 2, 3, 4], [mu, mu, mu, mu]], np.int32)
    pred = np.array([[9, 9, 9, 9], [10, 11, 12, 13]], np.int32)
    conf = np.array([[.9, .9, .9, .9], [.1, .2, .3, .4]], np.float32)
    t = torch.from_numpy(tok).cuda()
    nc = torch.zeros(2, dtype=torch.int32, device="cuda")
    nr = torch.zeros(2, dtype=torch.int32, device="cuda")
    dare.dare_unmask_select(ctx, t, 0, 4, torch.from_numpy(pred).cuda(), torch.from_numpy(conf).cuda(), mu,
                            dare.SELECT_TOPK, 0.0, 8, nc, nr)
    assert t.cpu().tolist() == [[1, 2, 3, 4], [10, 11, 12, 13]]
    assert nc.cpu().tolist() == [0, 4] and nr.cpu().tolist() == [0, 0]


# ----------------------------------------------------------------------------- LM head
def _lm_case(ctx, M, D, V, mu, seed, sigma_w=0.02, planted=False, excl=True, with_rows=False):
    wl = I.scaled(I.WORKLOADS["tiny"], batch=M, block_len=1, hidden=D, vocab=V, mask_id=mu, seed=seed)
    x = I.normal_bf16(seed, I.TID_X, (M, D))
    w = I.normal_bf16(seed, I.TID_W, (V, D), sigma_w)
    if planted:
        x, _ = I.plant_confidences(wl, x, w, 0)
    rt = None
    if with_rows:
        rt = I.uniform_int(seed, I.TID_TOK, (M,), 0, V - 1)
        rt[::3] = mu
    ref = O.lmhead_confidence(f64(x), f64(w), None if rt is None else rt.numpy(), mu, excl)
    pred, conf = dare.dare_lmhead_confidence(ctx, x.cuda(), w.cuda(), dev(rt), mu, excl)
    torch.cuda.synchronize()
    return check_lmhead(pred, conf, ref, f64(x), f64(w), mu, excl, O), ref, pred, conf


@pytest.mark.parametrize("M,D,V,mu", [
    (32, 256, 4096, 4095),        # the tiny workload's LM head
    (128, 64, 256, 255),          # one tile exactly, one K slice
    (200, 328, 1000, 17),         # ragged rows, K tail (328 = 5*64 + 8), ragged vocabulary
    (300, 1024, 2560 + 40, 2599), # several row tiles and vocabulary tiles, tail in both
    (1, 8, 2, 0),                 # the smallest legal problem
])
def test_lmhead_matches_oracle(ctx, M, D, V, mu):
    _lm_case(ctx, M, D, V, mu, seed=M + V)


def test_lmhead_planted_confidences_spread_and_match(ctx):
    n_diff, ref, pred, conf = _lm_case(ctx, 256, 512, 8192, 8000, seed=3, planted=True)
    c = ref["conf"]
    assert c.min() < 0.3 and c.max() > 0.9            # the 1e-3 bars bite on these
    assert n_diff == 0


def test_lmhead_without_exclusion_and_with_committed_rows(ctx):
    _lm_case(ctx, 96, 256, 1024, 5, seed=5, excl=False)
    _lm_case(ctx, 130, 256, 1024, 1023, seed=6, with_rows=True)


@pytest.mark.parametrize("M,D,V,mu,with_rows", [
    (256, 320, 2600, 7, False),        # 256 rows known on the host: the swapped-operand path (vocabulary on the lanes)
    (500, 128, 1000, 999, False),      # four row tiles, ragged last one (two chunks would be 256 long): row-major CTA pairs
    (600, 256, 2048, 5, True),         # 200 masked rows, known only on the device: swapped path, N = 208
    (1500, 64, 1200, 3, True),         # 500 masked rows = four tiles, known only on the device: pairs
    (1400, 64, 1200, 3, True),         # 467 masked rows: swapped path, two chunks of N = 240
    (900, 64, 1200, 3, True),          # 300 masked rows = three tiles: one pair of tiles and a single tile
    (560, 128, 1000, 999, False),      # five row tiles known on the host: pairs for four, single CTAs for the fifth
    (640, 128, 1000, 999, False),      # 640 rows known on the host: swapped path, three chunks of N = 224
    (1900, 64, 1200, 3, True),         # ~634 masked rows, known only on the device: three chunks
    (2560, 64, 1200, 3, True),         # ~855 masked rows: four chunks of N = 224
    (1100, 64, 1200, 3, False),        # nine row tiles (beyond the swapped path's range): four tile pairs and a single tile
    (300, 1024, 2600, 2599, False),    # three tiles on a small grid (16 clusters: 10 run the pair, 12 CTAs the third tile)
    (72, 200, 700, 0, False),          # swapped path, each CTA of a pair loads 40 rows as boxes of 32 + 8
    (330, 64, 520, 519, True),         # 110 masked rows: N = 112, one box of 64 rows per CTA covers its 56
])
def test_lmhead_single_and_pair_modes(ctx, M, D, V, mu, with_rows):
    """The greedy head's one kernel has three GEMM paths, picked by the number of live rows (on the device when rows
    are skipped): the swapped-operand path on CTA pairs up to 256 rows and, in chunks, for counts up to 1024 that cut
    into chunks of 208 to 240 rows; otherwise row-major tiles of 128 rows, on CTA pairs when the tiles come in twos,
    and for an odd count on pairs for all but the last tile while the CTAs of the remaining clusters work on that one
    singly."""
    _lm_case(ctx, M, D, V, mu, seed=M + D, with_rows=with_rows)


def test_lmhead_tie_break_lowest_index_and_mask_column(ctx):
    """Identical weight rows: all admissible columns tie exactly; lowest admissible id wins, conf = 1/(V-1)."""
    M, D, V = 64, 128, 700
    x = I.normal_bf16(1, I.TID_X, (M, D))
    w = I.normal_bf16(1, I.TID_W, (1, D), 0.05).repeat(V, 1).contiguous()
    for mu, want in ((0, 1), (300, 0)):
        pred, conf = dare.dare_lmhead_confidence(ctx, x.cuda(), w.cuda(), None, mu, True)
        assert (pred.cpu() == want).all()
        np.testing.assert_allclose(conf.cpu().numpy(), 1.0 / (V - 1), rtol=1e-4)


def test_lmhead_is_deterministic(ctx):
    x = I.normal_bf16(2, I.TID_X, (256, 512)).cuda()
    w = I.normal_bf16(2, I.TID_W, (5000, 512), 0.02).cuda()
    p1, c1 = dare.dare_lmhead_confidence(ctx, x, w, None, 4999, True)
    p2, c2 = dare.dare_lmhead_confidence(ctx, x, w, None, 4999, True)
    assert torch.equal(p1, p2) and torch.equal(c1, c2)


# ----------------------------------------------------------------------------- attention
def _attn_case(ctx, B, L, Hq, Hkv, d, P, S=0, ragged=False, inplace=False, seed=0, want_lse=True):
    wl = I.scaled(I.WORKLOADS["tiny"], batch=B, block_len=L, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d,
                  prompt_len=P, gen_len=L, suffix_cap=S, ragged=ragged, seed=seed, hidden=64, vocab=64, mask_id=63)
    k_pre, v_pre, k_suf, v_suf = I.make_caches(wl)
    plen, slen = I.make_lengths(wl, 0)
    q, k_blk, v_blk, _ = I.make_step_activations(wl, 0, inplace)
    o_ref, lse_ref = O.attn_block(f64(q), f64(k_pre), f64(v_pre), plen.numpy(), f64(k_blk), f64(v_blk), f64(k_suf),
                                  f64(v_suf), None if slen is None else slen.numpy())
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device="cuda") if want_lse else None
    out = dare.dare_attn_block(ctx, q.cuda(), k_pre.cuda(), v_pre.cuda(), plen.cuda(), dev(k_blk), dev(v_blk),
                               dev(k_suf), dev(v_suf), dev(slen), None, lse)
    torch.cuda.synchronize()
    check_attn(out, o_ref)
    if want_lse:
        assert np.abs(lse.cpu().double().numpy() - lse_ref).max() < 2e-2
    return out


@pytest.mark.parametrize("B,L,Hq,Hkv,d,P,S,ragged,inplace", [
    (1, 32, 4, 4, 64, 64, 0, False, False),      # the tiny workload
    (2, 32, 4, 4, 128, 200, 0, False, False),    # ragged tail tile in the prefix (200 = 3*64 + 8)
    (3, 32, 14, 2, 128, 300, 0, False, False),   # GQA group of 7: 224 packed rows, four query chunks
    (2, 4, 8, 8, 128, 1024, 256, True, False),   # dual cache, block of 4, ragged per-row lengths
    (2, 32, 8, 8, 128, 512, 0, False, True),     # block stored in place behind the prefix
    (1, 5, 6, 3, 64, 0 + 16, 7, True, False),    # odd sizes everywhere
    (4, 32, 2, 1, 64, 2048, 0, False, False),    # long prefix, few units: KV splits + combine
    (1, 1, 1, 1, 64, 16, 0, False, True),        # a single query
    # shapes that fill a 128-row tensor-core tile (tcgen05 path)
    (2, 128, 4, 4, 64, 100, 0, False, False),    # one full tile per head, head_dim 64, ragged prefix tile
    (2, 40, 8, 2, 128, 300, 70, True, False),    # GQA group of 4: 32 positions per tile, two tiles, dual cache, ragged
    (2, 100, 6, 2, 128, 0 + 8, 0, False, True),  # group of 3: 42 positions x 3 heads = 126 rows per tile, in place
    (1, 300, 2, 2, 64, 64, 0, False, True),      # prefill-like: three tiles of 128 rows, block in place
    (60, 256, 2, 2, 128, 200, 0, False, False),  # enough units for two query tiles per CTA (and a third, single one)
    (30, 130, 4, 4, 64, 70, 20, True, False),    # two query tiles per CTA, head_dim 64, second tile nearly empty
])
def test_attention_matches_oracle(ctx, B, L, Hq, Hkv, d, P, S, ragged, inplace):
    _attn_case(ctx, B, L, Hq, Hkv, d, P, S, ragged, inplace, seed=B + L + P)


@pytest.mark.parametrize("L", [8, 128])
def test_attention_zero_prefix_and_garbage_behind_lengths(ctx, L):
    """prefix_len = 0 for some rows, and NaNs planted behind every valid length must not leak in (both kernels)."""
    B, H, d, P, S = 3, 2, 64, 96, 40
    wl = I.scaled(I.WORKLOADS["tiny"], batch=B, block_len=L, n_q_heads=H, n_kv_heads=H, head_dim=d, prompt_len=P,
                  gen_len=L, suffix_cap=S, seed=9)
    k_pre, v_pre, k_suf, v_suf = I.make_caches(wl)
    k_pre, v_pre = k_pre[:, :, :P].contiguous(), v_pre[:, :, :P].contiguous()
    q, k_blk, v_blk, _ = I.make_step_activations(wl, 0)
    plen = torch.tensor([0, 37, 96], dtype=torch.int32)
    slen = torch.tensor([40, 0, 13], dtype=torch.int32)
    o_ref, _ = O.attn_block(f64(q), f64(k_pre), f64(v_pre), plen.numpy(), f64(k_blk), f64(v_blk), f64(k_suf),
                            f64(v_suf), slen.numpy())
    for r in range(B):
        k_pre[r, :, plen[r]:] = float("nan"); v_pre[r, :, plen[r]:] = float("nan")
        k_suf[r, :, slen[r]:] = float("inf"); v_suf[r, :, slen[r]:] = float("nan")
    out = dare.dare_attn_block(ctx, q.cuda(), k_pre.cuda(), v_pre.cuda(), plen.cuda(), k_blk.cuda(), v_blk.cuda(),
                               k_suf.cuda(), v_suf.cuda(), slen.cuda())
    check_attn(out, o_ref)


def test_attention_length_beyond_capacity_is_clamped_and_flagged(ctx):
    B, L, H, d, P = 1, 4, 1, 64, 32
    wl = I.scaled(I.WORKLOADS["tiny"], batch=B, block_len=L, n_q_heads=H, n_kv_heads=H, head_dim=d, prompt_len=P,
                  gen_len=L, seed=4)
    k_pre, v_pre, _, _ = I.make_caches(wl)
    k_pre, v_pre = k_pre[:, :, :P].contiguous(), v_pre[:, :, :P].contiguous()
    q, k_blk, v_blk, _ = I.make_step_activations(wl, 0)
    assert ctx.device_status() == 0
    out = dare.dare_attn_block(ctx, q.cuda(), k_pre.cuda(), v_pre.cuda(), torch.tensor([999], dtype=torch.int32).cuda(),
                               k_blk.cuda(), v_blk.cuda())
    assert ctx.device_status() == dare.DEV_LEN_CLAMPED
    o_ref, _ = O.attn_block(f64(q), f64(k_pre), f64(v_pre), np.array([P]), f64(k_blk), f64(v_blk))
    check_attn(out, o_ref)
    assert ctx.device_status() == 0


# ----------------------------------------------------------------------------- whole step, tiny workload
def test_tiny_workload_eight_iterations(ctx):
    """Config 1: batch 1, prompt 64, one block of 32 masks, vocab 4096, tau 0.9, 8 iterations; the oracle is
    evaluated from the GPU's pre-step state at every iteration (teacher forcing)."""
    wl = I.WORKLOADS["tiny"]
    w = I.make_weights(wl)
    caches = I.make_caches(wl)
    tok_d = I.fresh_tokens(wl).cuda()
    wd, kp, vp = w.cuda(), caches[0].cuda(), caches[1].cuda()
    for planted in (False, True):
        tok_d = I.fresh_tokens(wl).cuda()
        total = 0
        for it in range(8):
            si = I.make_step(wl, step=it, planted=planted, w=w, caches=caches)
            pre = tok_d.cpu().numpy()
            attn_out = torch.empty_like(si.q, device="cuda")
            pred = torch.empty(wl.M, dtype=torch.int32, device="cuda")
            conf = torch.empty(wl.M, dtype=torch.float32, device="cuda")
            # the planted pass takes the counts in page-locked host memory, which the step's last kernel writes itself
            nc = torch.full((wl.batch,), -1, dtype=torch.int32, device="cuda")
            nr = torch.full((wl.batch,), -1, dtype=torch.int32, device="cuda")
            if planted:
                nc, nr = nc.cpu().pin_memory(), nr.cpu().pin_memory()
            dare.dare_denoise_block(ctx, si.q.cuda(), kp, vp, si.prefix_len.cuda(), si.k_blk.cuda(), si.v_blk.cuda(),
                                    None, None, None, attn_out, None, si.x.cuda(), wd, wl.mask_id, True, tok_d,
                                    si.block_start, wl.mode, wl.threshold, wl.k, pred, conf, nc, nr)
            torch.cuda.synchronize()
            ref = O.denoise_step(f64(si.q), f64(si.k_pre), f64(si.v_pre), si.prefix_len.numpy(), f64(si.k_blk),
                                 f64(si.v_blk), None, None, None, f64(si.x), f64(si.w), pre, si.block_start,
                                 wl.block_len, wl.mask_id, wl.mode, wl.threshold, wl.k)
            check_attn(attn_out, ref["attn_out"])
            check_lmhead(pred, conf, ref["lm"], f64(si.x), f64(si.w), wl.mask_id, True, O)
            # selection: bit-exact given the GPU's own predictions and confidences
            want, wnc, wnr = O.unmask_select(pre, si.block_start, wl.block_len, pred.cpu().numpy(),
                                             conf.cpu().numpy(), wl.mask_id, wl.mode, wl.threshold, wl.k)
            np.testing.assert_array_equal(tok_d.cpu().numpy(), want)
            np.testing.assert_array_equal(nc.cpu().numpy(), wnc)
            np.testing.assert_array_equal(nr.cpu().numpy(), wnr)
            total += int(wnc.sum())
            assert wnc.min() >= 1 or (pre[:, si.block_start:] != wl.mask_id).all()
        if not planted:
            assert total == 8          # as stated, random logits never pass tau = 0.9: one commit per iteration
        else:
            assert total > 8           # planted confidences exercise the threshold branch


def test_step_replays_from_a_cuda_graph(ctx):
    """The step forks its LM head onto a stream of the context and joins it back by events: captured into a CUDA graph
    on the caller's stream, a replay must give what the eager call gives (tokens, counts, attention output)."""
    wl = I.WORKLOADS["tiny"]
    w = I.make_weights(wl)
    caches = I.make_caches(wl)
    wd, kp, vp = w.cuda(), caches[0].cuda(), caches[1].cuda()
    si = I.make_step(wl, step=0, planted=True, w=w, caches=caches)
    q, plen, kb, vb, x = si.q.cuda(), si.prefix_len.cuda(), si.k_blk.cuda(), si.v_blk.cuda(), si.x.cuda()
    tok0 = I.fresh_tokens(wl).cuda()
    bufs = {}
    for name in ("eager", "graph"):
        bufs[name] = dict(tok=tok0.clone(), out=torch.zeros_like(q), pred=torch.zeros(wl.M, dtype=torch.int32, device="cuda"),
                          conf=torch.zeros(wl.M, dtype=torch.float32, device="cuda"),
                          nc=torch.zeros(wl.batch, dtype=torch.int32, device="cuda"),
                          nr=torch.zeros(wl.batch, dtype=torch.int32, device="cuda"))

    def step(b, stream=None):
        dare.dare_denoise_block(ctx, q, kp, vp, plen, kb, vb, None, None, None, b["out"], None, x, wd, wl.mask_id, True,
                                b["tok"], si.block_start, wl.mode, wl.threshold, wl.k, b["pred"], b["conf"], b["nc"], b["nr"],
                                stream=stream)

    step(bufs["eager"])                          # (also raises the kernels' shared-memory limits before the capture)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step(bufs["graph"], stream=torch.cuda.current_stream())
    bufs["graph"]["tok"].copy_(tok0)             # whatever ran or did not run during the capture: start over
    g.replay()
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    for key in ("tok", "out", "pred", "conf", "nc", "nr"):
        assert torch.equal(bufs["eager"][key], bufs["graph"][key]), key
    assert int(bufs["graph"]["nc"].sum()) >= 1


# ----------------------------------------------------------------------------- ABI error behaviour
def test_bad_arguments_are_rejected_before_any_launch(ctx):
    q = torch.zeros(1, 4, 2, 64, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(1, 2, 16, 64, dtype=torch.bfloat16, device="cuda")
    kb = torch.zeros(1, 2, 4, 64, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_attn_block(ctx, q, k, k, None, kb, None, check=False) == -1          # v_blk missing
    q3 = torch.zeros(1, 4, 3, 64, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_attn_block(ctx, q3, k, k, None, kb, kb, check=False) == -2           # 3 % 2 != 0
    q96 = torch.zeros(1, 4, 2, 96, dtype=torch.bfloat16, device="cuda")
    k96 = torch.zeros(1, 2, 16, 96, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_attn_block(ctx, q96, k96, k96, None, None, None, check=False) == -2  # head_dim 96
    x = torch.zeros(4, 12, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(8, 12, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_lmhead_confidence(ctx, x, w, check=False) == -2                      # D % 8 != 0
    buf = torch.zeros(4 * 16 + 1, dtype=torch.bfloat16, device="cuda")[1:].view(4, 16)
    w16 = torch.zeros(8, 16, dtype=torch.bfloat16, device="cuda")
    rc = load_rc = dare.load().dare_lmhead_confidence(ctx.handle, buf.data_ptr(), 4, 16, w16.data_ptr(), 8, None, 0, 1,
                                                      torch.zeros(4, dtype=torch.int32, device="cuda").data_ptr(),
                                                      torch.zeros(4, device="cuda").data_ptr(), None)
    assert rc == -3                                                                        # misaligned pointer
    tok = torch.zeros(2, 8, dtype=torch.int32, device="cuda")
    p = torch.zeros(2, 4, dtype=torch.int32, device="cuda")
    c = torch.zeros(2, 4, device="cuda")
    assert dare.dare_unmask_select(ctx, tok, 6, 4, p, c, 0, dare.SELECT_TOPK, 0.0, 1, check=False) == -4   # window
    assert dare.dare_unmask_select(ctx, tok, 0, 4, p, c, 0, dare.SELECT_TOPK, 0.0, 0, check=False) == -4   # k < 1
    assert dare.dare_unmask_select(ctx, tok, 0, 4, p, c, 0, 0, float("nan"), 1, check=False) == -4          # NaN tau
    assert dare.dare_unmask_select(ctx, tok, 0, 4, p, c, 0, 5, 0.5, 1, check=False) == -4                   # mode
    small = dare.Context(0, workspace_bytes=4096)
    xb = torch.zeros(256, 64, dtype=torch.bfloat16, device="cuda")
    wb = torch.zeros(4096, 64, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_lmhead_confidence(small, xb, wb, check=False) == -5                   # workspace too small
    small.close()
    torch.cuda.synchronize()


def test_tensor_map_cache_hits_on_the_same_buffers_and_misses_on_new_ones():
    """The context keeps encoded tensor maps keyed by (address, shape, box).  The same step on the same buffers must
    hit; other buffers of the same shapes must miss and still give the right result (each against the oracle); a
    buffer freed and allocated again with another shape, possibly at the same address, must give the new shape's
    result."""
    wl = I.scaled(I.WORKLOADS["tiny"], batch=3)
    ctx = dare.Context(0)

    def run(si, bufs=None):
        d = bufs or {k: getattr(si, k).cuda() for k in ("q", "k_pre", "v_pre", "k_blk", "v_blk", "x", "w")}
        tok = si.tokens.cuda()
        out = torch.empty_like(d["q"])
        pred = torch.empty(wl.M, dtype=torch.int32, device="cuda")
        conf = torch.empty(wl.M, dtype=torch.float32, device="cuda")
        dare.dare_denoise_block(ctx, d["q"], d["k_pre"], d["v_pre"], si.prefix_len.cuda(), d["k_blk"], d["v_blk"], None,
                                None, None, out, None, d["x"], d["w"], wl.mask_id, True, tok, si.block_start, wl.mode,
                                wl.threshold, wl.k, pred, conf, None, None)
        torch.cuda.synchronize()
        ref = O.denoise_step(f64(si.q), f64(si.k_pre), f64(si.v_pre), si.prefix_len.numpy(), f64(si.k_blk), f64(si.v_blk),
                             None, None, None, f64(si.x), f64(si.w), si.tokens.numpy(), si.block_start, wl.block_len,
                             wl.mask_id, wl.mode, wl.threshold, wl.k)
        check_attn(out, ref["attn_out"])
        check_lmhead(pred, conf, ref["lm"], f64(si.x), f64(si.w), wl.mask_id, True, O)
        return d

    a = I.make_step(wl, step=0, planted=True)
    b = I.make_step(wl, step=1, planted=True)
    bufs_a = run(a)
    h0, m0 = ctx.tmap_cache_stats()
    assert m0 > 0
    run(a, bufs_a)                                   # same buffers: every map is found
    h1, m1 = ctx.tmap_cache_stats()
    assert m1 == m0 and h1 - h0 == h0 + m0         # as many look-ups as the first run made, all found
    bufs_b = run(b)                                  # same shapes at other addresses: encoded anew, results of b
    h2, m2 = ctx.tmap_cache_stats()
    assert m2 > m1
    run(a, bufs_a)                                   # and a's maps are still right
    # free a's LM-head input and let the allocator hand the memory out again for another shape
    M, D = bufs_a["x"].shape
    del bufs_a, bufs_b
    x2 = I.normal_bf16(5, I.TID_X, (2 * M, D // 2))
    w2 = I.normal_bf16(5, I.TID_W, (300, D // 2), 0.05)
    pred, conf = dare.dare_lmhead_confidence(ctx, x2.cuda(), w2.cuda(), None, 7, True)
    torch.cuda.synchronize()
    ref = O.lmhead_confidence(f64(x2), f64(w2), None, 7, True)
    check_lmhead(pred, conf, ref, f64(x2), f64(w2), 7, True, O)
    assert ctx.device_status() == 0
    ctx.close()


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.device_count() < 2, reason="needs two GPUs")
def test_context_of_another_device_is_refused():
    """Nothing is launched: the call returns DARE_ERR_DEVICE before it touches the other GPU's workspace."""
    ctx = dare.Context(1)
    assert torch.cuda.current_device() == 0          # dare_create put the current device back
    tok = torch.zeros(2, 8, dtype=torch.int32, device="cuda:0")
    pred = torch.zeros(2, 4, dtype=torch.int32, device="cuda:0")
    conf = torch.zeros(2, 4, dtype=torch.float32, device="cuda:0")
    assert dare.dare_unmask_select(ctx, tok, 0, 4, pred, conf, 5, dare.SELECT_TOPK, 0.0, 1, check=False) == -8
    ctx.close()
