"""Seeded synthetic inputs for the rollout denoising step.

This module only draws numbers and lays them out; it contains none of the
method's arithmetic (no attention, no softmax, no selection).  Both the CUDA
tests/bench and the CPU oracle's tests take their inputs from here so that the
two sides see the same bits.

Every tensor is a function of ``(seed, tensor_id, step)`` through a seeded
``torch.Generator`` on the CPU: N(0, sigma) drawn in fp32, rounded to bf16
(round-to-nearest-even).  Token ids are int32.

The workloads stand in for the paper's rollouts (Section 4.2, "Implementation
Details": block length 32, response 256/512 with 128/256 diffusion steps, i.e.
two tokens per step) on LLaDA-, Dream- and SDAR-shaped models; the trained
checkpoints and prompt datasets are not available, so shapes are kept and
values are random.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import torch

# tensor ids (kept stable: they key the random streams)
TID_Q, TID_KPRE, TID_VPRE, TID_KBLK, TID_VBLK, TID_KSUF, TID_VSUF = 1, 2, 3, 4, 5, 6, 7
TID_X, TID_W, TID_PLEN, TID_SLEN, TID_PLANT, TID_TOK = 8, 9, 10, 11, 12, 13
TID_EMB, TID_LAYER0 = 14, 32     # layer l uses ids TID_LAYER0 + 8*l + {0: wqkv, 1: wo, 2: wg, 3: wu, 4: wd}

SELECT_THRESHOLD = 0
SELECT_TOPK = 1


def _gen(seed: int, tensor_id: int, step: int = 0) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed(((int(seed) & 0xFFFF) << 40) ^ ((int(tensor_id) & 0xFFFF) << 20) ^ (int(step) & 0xFFFFF))
    return g


def normal_bf16(seed: int, tensor_id: int, shape, sigma: float = 1.0, step: int = 0) -> torch.Tensor:
    """N(0, sigma) in bf16 on the CPU; generated along dim 0 in slabs to bound the fp32 temporary."""
    shape = tuple(int(s) for s in shape)
    g = _gen(seed, tensor_id, step)
    out = torch.empty(shape, dtype=torch.bfloat16)
    if out.numel() == 0:
        return out
    rows = shape[0]
    per_row = out.numel() // rows
    slab = max(1, (1 << 26) // max(per_row, 1))
    for r0 in range(0, rows, slab):
        r1 = min(rows, r0 + slab)
        t = torch.randn((r1 - r0,) + shape[1:], generator=g, dtype=torch.float32)
        out[r0:r1] = (t * sigma).to(torch.bfloat16)
    return out


def uniform_int(seed: int, tensor_id: int, shape, lo: int, hi: int, step: int = 0) -> torch.Tensor:
    """Integers uniform in [lo, hi] (inclusive), int32."""
    g = _gen(seed, tensor_id, step)
    return torch.randint(lo, hi + 1, tuple(shape), generator=g, dtype=torch.int64).to(torch.int32)


@dataclass
class Workload:
    """Shape of one denoising-step workload (names follow the paper's notation where it has one)."""
    name: str
    batch: int            # B rollouts
    block_len: int        # L, block length (Section 4.2: 32)
    n_q_heads: int        # Hq
    n_kv_heads: int       # Hkv
    head_dim: int         # d
    hidden: int           # D
    vocab: int            # V
    mask_id: int          # the absorbing <MASK> token id (Eq. 1)
    prompt_len: int       # P0
    gen_len: int          # G (generation length, a multiple of block_len)
    mode: int             # SELECT_THRESHOLD / SELECT_TOPK
    threshold: float = 0.9
    k: int = 1
    suffix_cap: int = 0   # dual (suffix) cache capacity; 0 = prefix cache only
    ragged: bool = False  # per-row prefix/suffix lengths (config 4's parity case)
    seed: int = 0

    @property
    def prefix_cap(self) -> int:
        return self.prompt_len + self.gen_len

    @property
    def n_blocks(self) -> int:
        return self.gen_len // self.block_len

    @property
    def M(self) -> int:
        return self.batch * self.block_len


# The five configurations.  WORKLOADS["llada8b"] is the one the headline metric is quoted on.
WORKLOADS = {
    "tiny": Workload("tiny", 1, 32, 4, 4, 64, 256, 4096, 4095, 64, 32, SELECT_THRESHOLD, threshold=0.9, seed=0),
    "llada8b": Workload("llada8b", 16, 32, 32, 32, 128, 4096, 126464, 126336, 512, 256, SELECT_TOPK, k=2, seed=0),
    "dream7b": Workload("dream7b", 32, 32, 28, 4, 128, 3584, 152064, 151666, 1024, 512, SELECT_THRESHOLD,
                        threshold=0.9, seed=0),
    "dualcache": Workload("dualcache", 64, 4, 32, 32, 128, 4096, 126464, 126336, 4096, 4, SELECT_THRESHOLD,
                          threshold=0.95, suffix_cap=1024, seed=0),
}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for small parity cases)."""
    d = dict(w.__dict__)
    d.update(kw)
    return Workload(**d)


@dataclass
class StepInputs:
    """All operands of one denoising step, on the CPU.  bf16 tensors unless noted."""
    wl: Workload
    q: torch.Tensor                    # [B, L, Hq, d]
    k_pre: torch.Tensor                # [B, Hkv, prefix_cap, d]
    v_pre: torch.Tensor
    prefix_len: torch.Tensor           # int32 [B]
    k_blk: Optional[torch.Tensor]      # [B, Hkv, L, d] or None (block stored in k_pre at [prefix_len, +L))
    v_blk: Optional[torch.Tensor]
    k_suf: Optional[torch.Tensor]      # [B, Hkv, suffix_cap, d] or None
    v_suf: Optional[torch.Tensor]
    suffix_len: Optional[torch.Tensor]  # int32 [B] or None
    x: torch.Tensor                    # [M, D] hidden states entering the LM head
    w: torch.Tensor                    # [V, D] LM-head weight (mathematical shape D x V, stored K-major)
    tokens: torch.Tensor               # int32 [B, row_stride]
    row_stride: int
    block_start: int
    extras: dict = field(default_factory=dict)


def make_lengths(wl: Workload, block_index: int = 0):
    """Per-row prefix and suffix lengths.  Non-ragged: prompt + completed blocks, full suffix."""
    B = wl.batch
    if wl.ragged:
        # multiples of 4 drawn per row (the dual-cache parity case)
        lo = max(1, wl.prompt_len // 16)
        plen = 4 * uniform_int(wl.seed, TID_PLEN, (B,), lo, max(lo, wl.prompt_len // 4))
        plen = plen + block_index * wl.block_len
        slen = None
        if wl.suffix_cap:
            slo = max(1, wl.suffix_cap // 16)
            slen = 4 * uniform_int(wl.seed, TID_SLEN, (B,), slo, max(slo, wl.suffix_cap // 4))
    else:
        plen = torch.full((B,), wl.prompt_len + block_index * wl.block_len, dtype=torch.int32)
        slen = torch.full((B,), wl.suffix_cap, dtype=torch.int32) if wl.suffix_cap else None
    return plen.to(torch.int32), (slen.to(torch.int32) if slen is not None else None)


def make_weights(wl: Workload) -> torch.Tensor:
    """LM-head weight, N(0, 0.02), stored [V, D]."""
    return normal_bf16(wl.seed, TID_W, (wl.vocab, wl.hidden), 0.02)


def make_caches(wl: Workload, inplace_block: bool = False):
    """Prefix (and optional suffix) K/V caches filled with N(0,1) over their whole capacity."""
    shp = (wl.batch, wl.n_kv_heads, wl.prefix_cap, wl.head_dim)
    k_pre = normal_bf16(wl.seed, TID_KPRE, shp)
    v_pre = normal_bf16(wl.seed, TID_VPRE, shp)
    k_suf = v_suf = None
    if wl.suffix_cap:
        sshp = (wl.batch, wl.n_kv_heads, wl.suffix_cap, wl.head_dim)
        k_suf = normal_bf16(wl.seed, TID_KSUF, sshp)
        v_suf = normal_bf16(wl.seed, TID_VSUF, sshp)
    return k_pre, v_pre, k_suf, v_suf


def fresh_tokens(wl: Workload) -> torch.Tensor:
    """Token state [B, prompt+gen]: uniform prompt ids (never the mask id), generation region all <MASK>."""
    B = wl.batch
    row = wl.prompt_len + wl.gen_len
    tok = uniform_int(wl.seed, TID_TOK, (B, row), 0, wl.vocab - 2)
    tok = torch.where(tok >= wl.mask_id, tok + 1, tok).to(torch.int32)  # skip the mask id
    tok[:, wl.prompt_len:] = wl.mask_id
    return tok.contiguous()


def make_step_activations(wl: Workload, step: int, inplace_block: bool = False):
    """Per-step activations: block queries, block K/V (unless in place) and LM-head inputs."""
    B, L = wl.batch, wl.block_len
    q = normal_bf16(wl.seed, TID_Q, (B, L, wl.n_q_heads, wl.head_dim), 1.0, step)
    k_blk = v_blk = None
    if not inplace_block:
        k_blk = normal_bf16(wl.seed, TID_KBLK, (B, wl.n_kv_heads, L, wl.head_dim), 1.0, step)
        v_blk = normal_bf16(wl.seed, TID_VBLK, (B, wl.n_kv_heads, L, wl.head_dim), 1.0, step)
    x = normal_bf16(wl.seed, TID_X, (B * L, wl.hidden), 1.0, step)
    return q, k_blk, v_blk, x


def plant_confidences(wl: Workload, x: torch.Tensor, w: torch.Tensor, step: int = 0,
                      p_lo: float = 0.05, p_hi: float = 0.999):
    """Planted companion inputs: push each LM-head row towards one random column.

    For row m a column c (never the mask id) and a target probability p* in
    [p_lo, p_hi] are drawn; ``a * W[c] / |W[c]|^2`` is added to x[m] with
    ``a = logit(p*) + ln V + sigma^2/2`` where sigma^2 = 0.02^2 * D is the variance
    of the background logits, so the realised confidence lands near p* and the
    confidences spread over (0, 1).  Returns (x_planted bf16, columns int64).
    This only shapes the *inputs*; what the step does with them is not computed here.
    """
    M, D = x.shape
    V = w.shape[0]
    g = _gen(wl.seed, TID_PLANT, step)
    cols = torch.randint(0, V - 1, (M,), generator=g, dtype=torch.int64)
    cols = torch.where(cols >= wl.mask_id, cols + 1, cols)
    pstar = p_lo + (p_hi - p_lo) * torch.rand((M,), generator=g, dtype=torch.float64)
    sigma2 = (0.02 ** 2) * D
    import math
    a = torch.log(pstar / (1 - pstar)) + math.log(V) + sigma2 / 2
    wc = w[cols].to(torch.float64)
    delta = a[:, None] * wc / (wc * wc).sum(dim=1, keepdim=True)
    xp = (x.to(torch.float64) + delta).to(torch.float32).to(torch.bfloat16)
    return xp, cols


def make_step(wl: Workload, step: int = 0, block_index: int = 0, inplace_block: bool = False,
              planted: bool = False, w: Optional[torch.Tensor] = None, caches=None,
              tokens: Optional[torch.Tensor] = None) -> StepInputs:
    """Assemble every operand of one step (weights/caches are reused when passed in)."""
    if w is None:
        w = make_weights(wl)
    if caches is None:
        caches = make_caches(wl)
    k_pre, v_pre, k_suf, v_suf = caches
    plen, slen = make_lengths(wl, block_index)
    q, k_blk, v_blk, x = make_step_activations(wl, step, inplace_block)
    extras = {}
    if planted:
        x, cols = plant_confidences(wl, x, w, step)
        extras["planted_cols"] = cols
    if tokens is None:
        tokens = fresh_tokens(wl)
    return StepInputs(wl, q, k_pre, v_pre, plen, k_blk, v_blk, k_suf, v_suf, slen, x, w, tokens,
                      tokens.shape[1], wl.prompt_len + block_index * wl.block_len, extras)


# ---------------------------------------------------------------------------------------------------
# The end-to-end loop workload: a random-init decoder-shaped stack (RMSNorm, RoPE, SwiGLU, untied LM head).

@dataclass
class ModelWorkload:
    """Shape of the end-to-end denoising loop on a small stack of layers."""
    name: str
    n_layers: int
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    mask_id: int
    batch: int
    prompt_len: int
    gen_len: int
    block_len: int
    mode: int
    threshold: float = 0.9
    k: int = 1
    rms_eps: float = 1e-5
    rope_base: float = 10000.0
    seed: int = 0

    @property
    def row_len(self) -> int:
        return self.prompt_len + self.gen_len


MODEL_WORKLOADS = {
    # the 4-layer LLaDA-shaped loop
    "llada_loop": ModelWorkload("llada_loop", 4, 4096, 32, 32, 128, 12288, 126464, 126336, 16, 512, 256, 32,
                                SELECT_THRESHOLD, threshold=0.9),
    # small cases for element-by-element parity
    "loop_small": ModelWorkload("loop_small", 2, 256, 4, 4, 64, 768, 4096, 4095, 2, 48, 64, 32,
                                SELECT_THRESHOLD, threshold=0.9),
    # block diffusion with short blocks (SDAR / LLaDA2-style: block of 4, causal across blocks)
    "loop_small_bd4": ModelWorkload("loop_small_bd4", 2, 256, 4, 2, 64, 512, 1024, 1000, 3, 24, 16, 4,
                                    SELECT_THRESHOLD, threshold=0.95),
    "loop_small_gqa": ModelWorkload("loop_small_gqa", 3, 512, 4, 2, 128, 1280, 2048, 2000, 3, 40, 32, 16,
                                    SELECT_TOPK, k=3),
}


def make_model_weights(mw: ModelWorkload):
    """All weights of the stack, N(0, 0.02) bf16, stored [out features, in features] (K-major).

    Returns dict: embedding [V, D], lm_head [V, D], layers = list of dicts with wqkv [(Hq+2Hkv)d, D] (rows:
    q heads, k heads, v heads), wo [D, Hq d], wg [F, D], wu [F, D], wd [D, F].
    """
    D, F = mw.hidden, mw.ffn
    nq, nk = mw.n_q_heads * mw.head_dim, mw.n_kv_heads * mw.head_dim
    layers = []
    for l in range(mw.n_layers):
        t = TID_LAYER0 + 8 * l
        layers.append({"wqkv": normal_bf16(mw.seed, t + 0, (nq + 2 * nk, D), 0.02),
                       "wo": normal_bf16(mw.seed, t + 1, (D, nq), 0.02),
                       "wg": normal_bf16(mw.seed, t + 2, (F, D), 0.02),
                       "wu": normal_bf16(mw.seed, t + 3, (F, D), 0.02),
                       "wd": normal_bf16(mw.seed, t + 4, (D, F), 0.02)})
    return {"embedding": normal_bf16(mw.seed, TID_EMB, (mw.vocab, D), 0.02),
            "lm_head": normal_bf16(mw.seed, TID_W, (mw.vocab, D), 0.02), "layers": layers}


def fresh_model_tokens(mw: ModelWorkload) -> torch.Tensor:
    """Token state [B, prompt + gen]: uniform prompt ids (never the mask id), generation region all <MASK>."""
    tok = uniform_int(mw.seed, TID_TOK, (mw.batch, mw.row_len), 0, mw.vocab - 2)
    tok = torch.where(tok >= mw.mask_id, tok + 1, tok).to(torch.int32)
    tok[:, mw.prompt_len:] = mw.mask_id
    return tok.contiguous()
