"""GPU parity of the forward (masking) process, Eq. 1, and of the per-sequence NELBO term, Eq. 2, against the oracle.
The masking decision compares an exactly representable uniform with p in float32 on both sides: bit-exact.  The
NELBO term is a float32 sum of up to a few thousand log-probabilities against a float64 one: relative 1e-5."""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from oracle import dare_sampling_oracle as SO
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    c.close()


@pytest.mark.parametrize("B,T,start,length,seed,sample", [
    (6, 700, 100, 513, 5, 0), (3, 64, 0, 64, 0x0123456789ABCDEF, 15), (1, 9, 4, 1, 1, 4000000000), (16, 768, 512, 256, 9, 3)])
def test_forward_mask_bit_exact(ctx, B, T, start, length, seed, sample):
    mask_id = 126336
    x0 = I.uniform_int(seed & 0xFFFF, I.TID_TOK, (B, T), 0, 126000)
    p = torch.linspace(0.0, 1.0, B, dtype=torch.float32) if B > 1 else torch.tensor([0.37])
    want = SO.forward_mask(x0.numpy(), start, length, p.numpy(), mask_id, seed, sample)
    got = dare.dare_forward_mask(ctx, x0.cuda(), start, length, p.cuda(), mask_id, seed, sample)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(got.cpu().numpy(), want)
    # in place gives the same result
    x = x0.cuda()
    dare.dare_forward_mask(ctx, x, start, length, p.cuda(), mask_id, seed, sample, xt=x)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(x.cpu().numpy(), want)


def test_masked_nelbo_and_the_whole_estimator(ctx):
    """Eq. 1 -> log-probability head -> Eq. 2 on the GPU against the same chain in the oracle, for 4 draws."""
    B, T, start, length, D, V, mask_id = 4, 96, 32, 64, 128, 1000, 999
    x0 = I.uniform_int(3, I.TID_TOK, (B, T), 0, V - 2)
    w = I.normal_bf16(3, I.TID_W, (V, D), 0.05)
    t = torch.tensor([0.2, 0.5, 0.8, 1.0], dtype=torch.float32)
    est_gpu, est_ref = np.zeros(B), np.zeros(B)
    for sample in range(4):
        xt = dare.dare_forward_mask(ctx, x0.cuda(), start, length, t.cuda(), mask_id, 77, sample)
        xt_ref = SO.forward_mask(x0.numpy(), start, length, t.numpy(), mask_id, 77, sample)
        # stand-in for the network: hidden states drawn per draw (what matters here is the chain after them)
        h = I.normal_bf16(3, I.TID_X, (B * length, D), 1.0, step=sample)
        targets = x0[:, start:start + length].contiguous().view(-1)
        lp = dare.dare_lmhead_logprob(ctx, h.cuda(), w.cuda(), targets.cuda(), mask_id, False)
        n = torch.zeros(B, dtype=torch.int32, device="cuda")
        nelbo = dare.dare_masked_nelbo(ctx, lp, xt, start, length, mask_id, t.cuda(), n_masked=n)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(xt.cpu().numpy(), xt_ref)
        # Eq. 2 alone, from the GPU's own log-probabilities: float32 sum against float64
        want, n_ref = SO.masked_nelbo(lp.cpu().numpy(), xt_ref, start, length, mask_id, t.numpy())
        np.testing.assert_allclose(nelbo.cpu().numpy(), want, rtol=1e-5)
        np.testing.assert_array_equal(n.cpu().numpy(), n_ref)
        # the whole chain against the oracle's own log-probabilities
        lp_ref, _ = O.lmhead_logprob(f64(h), f64(w), targets.numpy(), mask_id, False)
        ref, _ = SO.masked_nelbo(lp_ref, xt_ref, start, length, mask_id, t.numpy())
        assert np.abs(nelbo.cpu().numpy() - ref).max() <= 2e-2 * n_ref.max() / t.min().item()
        est_gpu += nelbo.cpu().numpy() / 4
        est_ref += ref / 4
    np.testing.assert_allclose(est_gpu, est_ref, rtol=2e-3)
    assert ctx.device_status() == 0


def test_diffusion_bad_arguments(ctx):
    x = torch.zeros(2, 16, dtype=torch.int32, device="cuda")
    p = torch.zeros(2, dtype=torch.float32, device="cuda")
    assert dare.dare_forward_mask(ctx, x, 8, 9, p, 5, 1, 0, check=False) == -4          # window beyond the row
    assert dare.dare_forward_mask(ctx, x, 0, 0, p, 5, 1, 0, check=False) == -2
    lp = torch.zeros(2, 8, dtype=torch.float32, device="cuda")
    assert dare.dare_masked_nelbo(ctx, lp, x, 12, 8, 5, p, check=False) == -4
