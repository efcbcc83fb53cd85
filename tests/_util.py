"""Helpers shared by the tests: conversions between the generator's CPU tensors, the oracle's float64
arrays and device memory, and the parity criteria."""
import numpy as np
import torch


def f64(t):
    return None if t is None else t.to(torch.float64).numpy()


def dev(t):
    return None if t is None else t.cuda()


def i32np(t):
    return None if t is None else t.numpy().astype(np.int32)


# Parity bars (bf16 inputs, fp32 accumulation, against the fp64 oracle)
ATTN_MAX_ABS = 2e-2
ATTN_REL_L2 = 5e-3
CONF_ABS = 1e-3
LOGCONF_ABS = 2e-2     # supplement: synthetic confidences are ~1e-3, so the absolute bar alone is loose
GAP_PROB = 1e-3


def check_attn(out_gpu, o_ref):
    got = out_gpu.float().cpu().double().numpy()
    err = np.abs(got - o_ref).max()
    rel = np.linalg.norm(got - o_ref) / max(np.linalg.norm(o_ref), 1e-30)
    assert np.isfinite(got).all()
    assert err <= ATTN_MAX_ABS, f"attention max-abs {err}"
    assert rel <= ATTN_REL_L2, f"attention rel-L2 {rel}"
    return err, rel


def check_lmhead(pred_gpu, conf_gpu, ref, x64=None, w64=None, mask_id=-1, excl=True, oracle=None):
    """ref = oracle.lmhead_confidence(...) dict.  Tokens must match wherever the oracle's top-2 probability gap
    exceeds 1e-3; elsewhere the GPU's token must lie in the near-tie set (its oracle probability within 1e-3 of
    the maximum).  Confidence within 1e-3 absolute and 2e-2 in log."""
    pred = pred_gpu.cpu().numpy()
    conf = conf_gpu.cpu().numpy().astype(np.float64)
    live = np.isfinite(ref["conf"])
    # skipped rows: token echoed, -inf confidence
    assert (pred[~live] == ref["pred"][~live]).all()
    assert np.isneginf(conf[~live]).all()
    gap = ref["conf"] - ref["second"]
    must = live & (gap > GAP_PROB)
    assert (pred[must] == ref["pred"][must]).all(), "argmax differs where the top-2 gap exceeds 1e-3"
    diff = live & (pred != ref["pred"])
    assert diff.sum() <= (live & (gap <= GAP_PROB)).sum()
    if diff.any():
        # a differing token is only acceptable as a near-tie, which takes the oracle to judge: the GPU's token must be
        # within 1e-3 of the maximum probability, and the GPU's confidence must be that token's probability
        assert oracle is not None, "tokens differ and no oracle inputs were given to judge the near-tie"
        for m in np.nonzero(diff)[0]:
            pr = oracle.token_probability(x64[m], w64, int(pred[m]), mask_id, excl)
            assert pr >= ref["conf"][m] - GAP_PROB
            assert abs(conf[m] - pr) <= CONF_ABS
            assert abs(np.log(conf[m]) - np.log(pr)) <= LOGCONF_ABS
    same = live & (pred == ref["pred"])
    assert np.abs(conf[same] - ref["conf"][same]).max(initial=0) <= CONF_ABS
    assert np.abs(np.log(conf[same]) - ref["logconf"][same]).max(initial=0) <= LOGCONF_ABS
    return int(diff.sum())
