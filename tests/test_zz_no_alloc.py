"""The allocation-free LM-head entry point against the context-based one.

This file is named so that pytest collects it last: a run that stops at the first failure has then already
run every other test.  It must pass alone in a fresh process and after the rest of the suite.

dare_lmhead_confidence_static serves callers that cannot call cudaMalloc (and therefore cannot create a
context): its scratch is a fixed array inside the library.  Same kernels, so the results must agree with
dare_lmhead_confidence on the same inputs within the LM-head bars of the other tests -- here they are
required to be identical.  Two different problems are run back to back because the scratch array keeps the
previous call's contents.  The results are also held against the fp64 oracle directly, with the same bars as the
context-based entry point.
"""
import pytest
import torch

from oracle import dare_oracle as O
from paper_2604_04215_b200 import binding as dare
from paper_2604_04215_b200 import inputs as I

from _util import check_lmhead, f64

pytestmark = pytest.mark.gpu


def _problem(seed, M, D, V, mu, with_rows):
    x = I.normal_bf16(seed, I.TID_X, (M, D)).cuda()
    w = I.normal_bf16(seed, I.TID_W, (V, D), 0.02).cuda()
    rt = None
    if with_rows:
        rt = I.uniform_int(seed, I.TID_TOK, (M,), 0, V - 1)
        rt[::2] = mu
        rt = rt.cuda()
    return x, w, rt, mu


def test_static_entry_matches_context_entry_on_two_calls_in_a_row():
    ctx = dare.Context(0)
    problems = [_problem(11, 300, 512, 5000, 4999, True),     # larger first ...
                _problem(12, 70, 264, 1000, 3, False)]        # ... then smaller: stale scratch must not matter
    want = [dare.dare_lmhead_confidence(ctx, x, w, rt, mu, True) for x, w, rt, mu in problems]
    # outputs for two rounds over the two problems, made before the calls: nothing is allocated in between
    outs = [[(torch.empty(x.shape[0], dtype=torch.int32, device="cuda"),
              torch.empty(x.shape[0], dtype=torch.float32, device="cuda")) for x, _, _, _ in problems]
            for _ in range(2)]
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for round_ in range(2):
        for (x, w, rt, mu), (p, c) in zip(problems, outs[round_]):
            dare.dare_lmhead_confidence_static(x, w, rt, mu, True, p, c)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before          # the device's free memory did not move
    for round_ in range(2):
        for (p, c), (wp, wc) in zip(outs[round_], want):
            assert torch.equal(p, wp)
            live = torch.isfinite(wc)
            assert torch.equal(torch.isfinite(c), live)
            assert (c[live] - wc[live]).abs().max().item() <= 1e-3      # the suite's confidence bar
            assert torch.equal(c[live], wc[live])                        # and in fact bit-identical
    # against the oracle itself, not only against the other entry point
    for (x, w, rt, mu), (p, c) in zip(problems, outs[1]):
        x64, w64 = f64(x.cpu()), f64(w.cpu())
        ref = O.lmhead_confidence(x64, w64, None if rt is None else rt.cpu().numpy(), mu, True)
        check_lmhead(p, c, ref, x64, w64, mu, True, O)
    assert dare.dare_lmhead_static_status() == 0                 # no clamp, no expired wait in any of the calls
    ctx.close()


def test_static_entry_rejects_problems_beyond_its_scratch():
    M, V = 8192, 126464                      # 12 * 8192 * 148 bytes > 8 MiB
    x = torch.zeros(M, 64, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(V, 64, dtype=torch.bfloat16, device="cuda")
    rc = dare.dare_lmhead_confidence_static(x, w, None, 0, True, check=False)
    assert rc == -5
    assert b"workspace" in dare.load().dare_status_string(rc)
    torch.cuda.synchronize()
