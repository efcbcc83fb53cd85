"""GPU parity of the packed variable-length bidirectional attention (dare_attn_varlen) against the fp64 oracle.
Same bars as the block attention: max-abs 2e-2, relative-L2 5e-3, log-sum-exp 2e-2."""
import numpy as np
import pytest
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import check_attn, f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    c = dare.Context(0)
    yield c
    c.close()


def _case(ctx, lens, Hq, Hkv, d, seed, max_seqlen=None):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    q = I.normal_bf16(seed, I.TID_Q, (T, Hq, d))
    k = I.normal_bf16(seed, I.TID_KPRE, (T, Hkv, d))
    v = I.normal_bf16(seed, I.TID_VPRE, (T, Hkv, d))
    o_ref, lse_ref = O.attn_varlen(f64(q), f64(k), f64(v), cu)
    lse = torch.full((Hq, T), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.zeros_like(q, device="cuda")
    dare.dare_attn_varlen(ctx, q.cuda(), k.cuda(), v.cuda(), torch.from_numpy(cu).cuda(), max_seqlen or max(lens), out, lse)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    check_attn(out, o_ref)
    assert np.abs(lse.cpu().double().numpy() - lse_ref).max() < 2e-2
    return out


@pytest.mark.parametrize("lens,Hq,Hkv,d", [
    ([64, 128, 37], 4, 4, 64),                 # one query tile per sequence, ragged last key tile
    ([5, 1, 17, 0, 9, 300], 6, 2, 128),        # tiny, single-token and empty sequences beside a long one; GQA group of 3
    ([257, 130, 511], 2, 2, 128),              # several query tiles per sequence (two per CTA), odd lengths
    ([200] * 40, 8, 8, 64),                    # many sequences x heads
    ([96, 33], 14, 2, 128),                    # group of 7: 18 positions per tile
])
def test_varlen_matches_oracle(ctx, lens, Hq, Hkv, d):
    _case(ctx, lens, Hq, Hkv, d, seed=len(lens) + Hq)


def test_varlen_max_seqlen_may_overestimate_and_sequences_do_not_mix(ctx):
    lens = [70, 50, 90]
    a = _case(ctx, lens, 4, 4, 64, seed=3, max_seqlen=400)         # a loose bound only costs idle CTAs
    b = _case(ctx, lens, 4, 4, 64, seed=3)
    assert torch.equal(a, b)
    # one packed call equals the sequences run one at a time
    cu = np.concatenate([[0], np.cumsum(lens)])
    q = I.normal_bf16(3, I.TID_Q, (int(cu[-1]), 4, 64)).cuda()
    k = I.normal_bf16(3, I.TID_KPRE, (int(cu[-1]), 4, 64)).cuda()
    v = I.normal_bf16(3, I.TID_VPRE, (int(cu[-1]), 4, 64)).cuda()
    for s, n in enumerate(lens):
        sl = slice(int(cu[s]), int(cu[s + 1]))
        one = dare.dare_attn_varlen(ctx, q[sl].contiguous(), k[sl].contiguous(), v[sl].contiguous(),
                                    torch.tensor([0, n], dtype=torch.int32, device="cuda"), n)
        torch.cuda.synchronize()
        assert torch.equal(one, a[sl])


def test_varlen_bad_arguments(ctx):
    q = torch.zeros(16, 4, 64, dtype=torch.bfloat16, device="cuda")
    k = torch.zeros(16, 3, 64, dtype=torch.bfloat16, device="cuda")
    cu = torch.tensor([0, 16], dtype=torch.int32, device="cuda")
    assert dare.dare_attn_varlen(ctx, q, k, k, cu, 16, check=False) == -2           # 4 query heads over 3 KV heads
    q96 = torch.zeros(16, 4, 96, dtype=torch.bfloat16, device="cuda")
    assert dare.dare_attn_varlen(ctx, q96, q96, q96, cu, 16, check=False) == -2     # head_dim 96
    assert dare.dare_attn_varlen(ctx, q, q, q, cu, 0, check=False) == -2            # max_seqlen < 1
