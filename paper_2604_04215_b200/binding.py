"""ctypes binding of libdare.so: argument marshalling only.

The functions carry the names of the C entry points (include/dare.h).  Tensors are torch CUDA tensors
used purely as device memory; every step runs inside the library's kernels.  There is no fallback: if
the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdare.so")

SELECT_THRESHOLD = 0
SELECT_TOPK = 1
DEV_LEN_CLAMPED = 1
DEV_WAIT_EXPIRED = 2

EXPORTS = ["dare_create", "dare_destroy", "dare_status_string", "dare_device_status", "dare_sm_count",
           "dare_tmap_cache_stats", "dare_lmhead_static_status", "dare_kernel_launches",
           "dare_attn_block", "dare_attn_varlen", "dare_lmhead_confidence", "dare_unmask_select", "dare_denoise_block", "dare_denoise_block_sampled",
           "dare_lmhead_confidence_static", "dare_lmhead_sample", "dare_lmhead_logprob", "dare_lmhead_logprob_backward", "dare_transpose_bf16", "dare_forward_mask", "dare_masked_nelbo", "dare_model_create", "dare_model_destroy", "dare_model_forward",
           "dare_model_step", "dare_generate", "dare_model_set_sampling", "dare_model_forward_window", "dare_model_step_window", "dare_generate_dual",
           "dare_linear", "dare_linear_plan", "dare_rmsnorm", "dare_rope_kv_write"]

_lib = None


class DareError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load().dare_status_string(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


def load():
    """Load the shared library (built in-tree by paper_2604_04215_b200.build); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2604_04215_b200.build` "
                           "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_float
    lib.dare_create.argtypes = [C.POINTER(vp), i32, C.c_size_t]
    lib.dare_create.restype = i32
    lib.dare_destroy.argtypes = [vp]
    lib.dare_destroy.restype = i32
    lib.dare_status_string.argtypes = [i32]
    lib.dare_status_string.restype = C.c_char_p
    lib.dare_device_status.argtypes = [vp, vp, C.POINTER(C.c_uint32)]
    lib.dare_device_status.restype = i32
    lib.dare_sm_count.argtypes = [vp]
    lib.dare_sm_count.restype = i32
    lib.dare_tmap_cache_stats.argtypes = [vp, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    lib.dare_tmap_cache_stats.restype = i32
    lib.dare_kernel_launches.argtypes = []
    lib.dare_kernel_launches.restype = C.c_uint64
    lib.dare_lmhead_static_status.argtypes = [vp, C.POINTER(C.c_uint32)]
    lib.dare_lmhead_static_status.restype = i32
    attn_args = [i32] * 7 + [f32] + [vp] * 12
    lib.dare_attn_block.argtypes = [vp] + attn_args
    lib.dare_attn_block.restype = i32
    lib.dare_attn_varlen.argtypes = [vp] + [i32] * 6 + [f32] + [vp] * 7
    lib.dare_attn_varlen.restype = i32
    lib.dare_lmhead_confidence.argtypes = [vp, vp, i32, i32, vp, i32, vp, i32, i32, vp, vp, vp]
    lib.dare_lmhead_confidence.restype = i32
    lib.dare_lmhead_confidence_static.argtypes = [vp, i32, i32, vp, i32, vp, i32, i32, vp, vp, vp]
    lib.dare_lmhead_confidence_static.restype = i32
    lib.dare_lmhead_sample.argtypes = [vp, vp, i32, i32, vp, i32, vp, i32, i32, f32, C.c_uint64, C.c_uint32, vp, vp, vp]
    lib.dare_lmhead_sample.restype = i32
    lib.dare_lmhead_logprob.argtypes = [vp, vp, i32, i32, vp, i32, vp, i32, i32, vp, vp, vp]
    lib.dare_lmhead_logprob.restype = i32
    lib.dare_lmhead_logprob_backward.argtypes = [vp, vp, i32, i32, vp, vp, i32, vp, i32, i32, vp, vp, vp, vp, vp, vp, vp]
    lib.dare_lmhead_logprob_backward.restype = i32
    lib.dare_transpose_bf16.argtypes = [vp, vp, i32, i32, vp, vp]
    lib.dare_transpose_bf16.restype = i32
    lib.dare_forward_mask.argtypes = [vp, vp, vp, i32, i64, i32, i32, vp, i32, C.c_uint64, C.c_uint32, vp]
    lib.dare_forward_mask.restype = i32
    lib.dare_masked_nelbo.argtypes = [vp, vp, vp, i32, i64, i32, i32, i32, vp, vp, vp, vp]
    lib.dare_masked_nelbo.restype = i32
    lib.dare_unmask_select.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, i32, i32, f32, i32, vp, vp, vp]
    lib.dare_unmask_select.restype = i32
    lib.dare_denoise_block.argtypes = ([vp] + [i32] * 7 + [f32] + [vp] * 11 +   # attention operands .. lse
                                       [vp, i32, vp, i32, i32, i32,              # hidden, D, w, V, mask, excl
                                        vp, i64, i32, i32, f32, i32,             # tokens, stride, start, mode, thr, k
                                        vp, vp, vp, vp, vp])                     # pred, conf, n_comm, n_rem, stream
    lib.dare_denoise_block.restype = i32
    lib.dare_denoise_block_sampled.argtypes = ([vp] + [i32] * 7 + [f32] + [vp] * 11 +
                                               [vp, i32, vp, i32, i32, i32, f32, C.c_uint64, C.c_uint32,
                                                vp, i64, i32, i32, f32, i32, vp, vp, vp, vp, vp])
    lib.dare_denoise_block_sampled.restype = i32
    lib.dare_model_create.argtypes = [vp, C.POINTER(ModelDesc), vp, C.POINTER(LayerWeights), vp, C.POINTER(vp)]
    lib.dare_model_create.restype = i32
    lib.dare_model_destroy.argtypes = [vp]
    lib.dare_model_destroy.restype = i32
    lib.dare_model_forward.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, i32, vp, vp]
    lib.dare_model_forward.restype = i32
    lib.dare_model_step.argtypes = [vp, vp, i32, i64, i32, i32, vp, vp, i32, i32, f32, i32, vp, vp, vp, vp, vp]
    lib.dare_model_step.restype = i32
    lib.dare_generate.argtypes = [vp, vp, i32, i64, i32, i32, i32, vp, vp, i32, i32, f32, i32, vp, vp, vp,
                                  C.POINTER(C.c_int32), vp]
    lib.dare_generate.restype = i32
    lib.dare_model_set_sampling.argtypes = [vp, f32, C.c_uint64, C.c_uint32, vp]
    lib.dare_model_set_sampling.restype = i32
    lib.dare_model_forward_window.argtypes = [vp, vp, i32, i64, i32, i32, i32, vp, vp, i32, vp, vp]
    lib.dare_model_forward_window.restype = i32
    lib.dare_model_step_window.argtypes = [vp, vp, i32, i64, i32, i32, i32, vp, vp, i32, i32, f32, i32, vp, vp, vp, vp, vp]
    lib.dare_model_step_window.restype = i32
    lib.dare_generate_dual.argtypes = lib.dare_generate.argtypes
    lib.dare_generate_dual.restype = i32
    lib.dare_linear.argtypes = [vp, i32, vp, i32, i32, vp, vp, i32, vp, vp, vp]
    lib.dare_linear.restype = i32
    lib.dare_linear_plan.argtypes = [vp, i32, i32, i32, i32, C.POINTER(C.c_int)]
    lib.dare_linear_plan.restype = i32
    lib.dare_rmsnorm.argtypes = [vp, vp, i32, i32, f32, vp, vp]
    lib.dare_rmsnorm.restype = i32
    lib.dare_rope_kv_write.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, i32, vp]
    lib.dare_rope_kv_write.restype = i32
    _lib = lib
    return lib


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int), ("hidden", C.c_int), ("n_q_heads", C.c_int), ("n_kv_heads", C.c_int),
                ("head_dim", C.c_int), ("ffn", C.c_int), ("vocab", C.c_int), ("mask_id", C.c_int32),
                ("rms_eps", C.c_float), ("rope_base", C.c_float), ("max_positions", C.c_int),
                ("max_rows", C.c_int), ("max_batch", C.c_int)]


class LayerWeights(C.Structure):
    _fields_ = [("wqkv", C.c_void_p), ("wo", C.c_void_p), ("wg", C.c_void_p), ("wu", C.c_void_p),
                ("wd", C.c_void_p)]


def _ptr(t: Optional[torch.Tensor], dtype=None):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    # the library launches on the current device (and refuses a context of another one): the buffers must live there
    if t.device.index != torch.cuda.current_device():
        raise ValueError(f"tensor on cuda:{t.device.index}, but the current device is cuda:{torch.cuda.current_device()}")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"expected dtype {dtype}, got {t.dtype}")
    return C.c_void_p(t.data_ptr())


def _count_ptr(t: Optional[torch.Tensor]):
    """The per-rollout count outputs (n_committed, n_remaining): a device tensor, or a page-locked host tensor (the
    kernel then stores its B integers straight into host memory and the caller needs no copy back)."""
    if t is not None and not t.is_cuda:
        if not t.is_pinned() or not t.is_contiguous():
            raise ValueError("a host tensor for the counts must be page-locked (pin_memory()) and contiguous")
        if t.dtype != torch.int32:
            raise ValueError(f"expected dtype {torch.int32}, got {t.dtype}")
        return C.c_void_p(t.data_ptr())
    return _ptr(t, torch.int32)


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


class Context:
    """Owns a dare_ctx (workspace + device status word) on one device."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        lib = load()
        h = C.c_void_p()
        rc = lib.dare_create(C.byref(h), int(device), int(workspace_bytes))
        if rc != 0:
            raise DareError(rc, "dare_create")
        self.handle = h
        self.device = device

    def close(self):
        if getattr(self, "handle", None):
            load().dare_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def sm_count(self) -> int:
        return load().dare_sm_count(self.handle)

    def tmap_cache_stats(self):
        """(hits, misses) of the context's tensor-map cache since it was created."""
        hits, misses = C.c_uint64(0), C.c_uint64(0)
        rc = load().dare_tmap_cache_stats(self.handle, C.byref(hits), C.byref(misses))
        if rc != 0:
            raise DareError(rc, "dare_tmap_cache_stats")
        return int(hits.value), int(misses.value)

    def device_status(self, stream=None) -> int:
        out = C.c_uint32(0)
        rc = load().dare_device_status(self.handle, _stream(stream), C.byref(out))
        if rc != 0:
            raise DareError(rc, "dare_device_status")
        return int(out.value)


def dare_attn_block(ctx: Context, q, k_pre, v_pre, prefix_len=None, k_blk=None, v_blk=None, k_suf=None, v_suf=None,
                    suffix_len=None, out=None, lse=None, scale: float = 0.0, stream=None, check: bool = True):
    B, L, Hq, d = q.shape
    Hkv, prefix_cap = k_pre.shape[1], k_pre.shape[2]
    suffix_cap = k_suf.shape[2] if k_suf is not None else 0
    if out is None:
        out = torch.empty_like(q)
    bf = torch.bfloat16
    rc = load().dare_attn_block(ctx.handle, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, float(scale),
                                _ptr(q, bf), _ptr(k_pre, bf), _ptr(v_pre, bf), _ptr(prefix_len, torch.int32),
                                _ptr(k_blk, bf), _ptr(v_blk, bf), _ptr(k_suf, bf), _ptr(v_suf, bf),
                                _ptr(suffix_len, torch.int32), _ptr(out, bf), _ptr(lse, torch.float32),
                                _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_attn_block")
    return out if check else rc


def dare_attn_varlen(ctx: Context, q, k, v, cu_seqlens, max_seqlen: int, out=None, lse=None, scale: float = 0.0,
                     stream=None, check: bool = True):
    total, Hq, d = q.shape
    Hkv = k.shape[1]
    if out is None:
        out = torch.empty_like(q)
    bf = torch.bfloat16
    rc = load().dare_attn_varlen(ctx.handle, total, cu_seqlens.numel() - 1, int(max_seqlen), Hq, Hkv, d, float(scale),
                                 _ptr(q, bf), _ptr(k, bf), _ptr(v, bf), _ptr(cu_seqlens, torch.int32), _ptr(out, bf),
                                 _ptr(lse, torch.float32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_attn_varlen")
    return out if check else rc


def dare_lmhead_confidence(ctx: Context, hidden, w, row_tokens=None, mask_id: int = -1,
                           exclude_mask_column: bool = True, pred=None, conf=None, stream=None, check: bool = True):
    M, D = hidden.shape
    V = w.shape[0]
    if pred is None:
        pred = torch.empty(M, dtype=torch.int32, device=hidden.device)
    if conf is None:
        conf = torch.empty(M, dtype=torch.float32, device=hidden.device)
    rc = load().dare_lmhead_confidence(ctx.handle, _ptr(hidden, torch.bfloat16), M, D, _ptr(w, torch.bfloat16), V,
                                       _ptr(row_tokens, torch.int32), int(mask_id), int(bool(exclude_mask_column)),
                                       _ptr(pred, torch.int32), _ptr(conf, torch.float32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_lmhead_confidence")
    return (pred, conf) if check else rc


def dare_lmhead_sample(ctx: Context, hidden, w, row_tokens=None, mask_id: int = -1, exclude_mask_column: bool = True,
                       temperature: float = 1.0, seed: int = 0, step: int = 0, pred=None, conf=None, stream=None,
                       check: bool = True):
    M, D = hidden.shape
    V = w.shape[0]
    if pred is None:
        pred = torch.empty(M, dtype=torch.int32, device=hidden.device)
    if conf is None:
        conf = torch.empty(M, dtype=torch.float32, device=hidden.device)
    rc = load().dare_lmhead_sample(ctx.handle, _ptr(hidden, torch.bfloat16), M, D, _ptr(w, torch.bfloat16), V,
                                   _ptr(row_tokens, torch.int32), int(mask_id), int(bool(exclude_mask_column)),
                                   float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF,
                                   _ptr(pred, torch.int32), _ptr(conf, torch.float32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_lmhead_sample")
    return (pred, conf) if check else rc


def dare_lmhead_logprob(ctx: Context, hidden, w, targets, mask_id: int = -1, exclude_mask_column: bool = False,
                        logprob=None, lse=None, stream=None, check: bool = True):
    M, D = hidden.shape
    V = w.shape[0]
    if logprob is None:
        logprob = torch.empty(M, dtype=torch.float32, device=hidden.device)
    rc = load().dare_lmhead_logprob(ctx.handle, _ptr(hidden, torch.bfloat16), M, D, _ptr(w, torch.bfloat16), V,
                                    _ptr(targets, torch.int32), int(mask_id), int(bool(exclude_mask_column)),
                                    _ptr(logprob, torch.float32), _ptr(lse, torch.float32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_lmhead_logprob")
    return logprob if check else rc


def dare_transpose_bf16(ctx: Context, a, out=None, stream=None, check: bool = True):
    rows, cols = a.shape
    if out is None:
        out = torch.empty(cols, rows, dtype=torch.bfloat16, device=a.device)
    rc = load().dare_transpose_bf16(ctx.handle, _ptr(a, torch.bfloat16), rows, cols, _ptr(out, torch.bfloat16),
                                    _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_transpose_bf16")
    return out if check else rc


def dare_lmhead_logprob_backward(ctx: Context, hidden, w, w_t, targets, lse, grad_logprob, mask_id: int = -1,
                                 exclude_mask_column: bool = False, dz=None, dzt=None, d_hidden=None, d_w=None,
                                 stream=None, check: bool = True):
    """Gradient of sum(grad_logprob * logprob) with respect to hidden and w.  Returns (d_hidden, d_w, dz, dzt)."""
    M, D = hidden.shape
    V = w.shape[0]
    bf, dev = torch.bfloat16, hidden.device
    dz = torch.empty(M, V, dtype=bf, device=dev) if dz is None else dz
    dzt = torch.empty(V, M, dtype=bf, device=dev) if dzt is None else dzt
    d_hidden = torch.empty(M, D, dtype=bf, device=dev) if d_hidden is None else d_hidden
    d_w = torch.empty(V, D, dtype=bf, device=dev) if d_w is None else d_w
    rc = load().dare_lmhead_logprob_backward(ctx.handle, _ptr(hidden, bf), M, D, _ptr(w, bf), _ptr(w_t, bf), V,
                                             _ptr(targets, torch.int32), int(mask_id), int(bool(exclude_mask_column)),
                                             _ptr(lse, torch.float32), _ptr(grad_logprob, torch.float32), _ptr(dz, bf),
                                             _ptr(dzt, bf), _ptr(d_hidden, bf), _ptr(d_w, bf), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_lmhead_logprob_backward")
    return (d_hidden, d_w, dz, dzt) if check else rc


def dare_forward_mask(ctx: Context, x0, start: int, length: int, p_mask, mask_id: int, seed: int, sample: int, xt=None,
                      stream=None, check: bool = True):
    """Eq. 1.  Returns xt (a fresh copy of x0 with the window corrupted unless xt is given; xt may be x0)."""
    B, row_stride = x0.shape
    if xt is None:
        xt = x0.clone()
    rc = load().dare_forward_mask(ctx.handle, _ptr(x0, torch.int32), _ptr(xt, torch.int32), B, row_stride, int(start),
                                  int(length), _ptr(p_mask, torch.float32), int(mask_id), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                  int(sample) & 0xFFFFFFFF, _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_forward_mask")
    return xt if check else rc


def dare_masked_nelbo(ctx: Context, logprob, xt, start: int, length: int, mask_id: int, t, nelbo=None, n_masked=None,
                      stream=None, check: bool = True):
    """Eq. 2, one draw: nelbo [B]."""
    B, row_stride = xt.shape
    if nelbo is None:
        nelbo = torch.empty(B, dtype=torch.float32, device=xt.device)
    rc = load().dare_masked_nelbo(ctx.handle, _ptr(logprob, torch.float32), _ptr(xt, torch.int32), B, row_stride,
                                  int(start), int(length), int(mask_id), _ptr(t, torch.float32),
                                  _ptr(nelbo, torch.float32), _ptr(n_masked, torch.int32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_masked_nelbo")
    return nelbo if check else rc


LMHEAD_STATIC_SCRATCH_BYTES = 8 << 20


def dare_lmhead_confidence_static(hidden, w, row_tokens=None, mask_id: int = -1, exclude_mask_column: bool = True,
                                  pred=None, conf=None, stream=None, check: bool = True):
    """The LM head for callers that may not allocate device memory: no context, fixed scratch inside the library.

    pred and conf should be passed in by such callers (they are only created here as a convenience for tests).
    Runs on the current device; calls that overlap on the GPU race on the shared scratch.
    """
    M, D = hidden.shape
    V = w.shape[0]
    if pred is None:
        pred = torch.empty(M, dtype=torch.int32, device=hidden.device)
    if conf is None:
        conf = torch.empty(M, dtype=torch.float32, device=hidden.device)
    rc = load().dare_lmhead_confidence_static(_ptr(hidden, torch.bfloat16), M, D, _ptr(w, torch.bfloat16), V,
                                              _ptr(row_tokens, torch.int32), int(mask_id),
                                              int(bool(exclude_mask_column)), _ptr(pred, torch.int32),
                                              _ptr(conf, torch.float32), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_lmhead_confidence_static")
    return (pred, conf) if check else rc


def dare_kernel_launches() -> int:
    """Kernels launched by the library in this process so far (host-side count)."""
    return int(load().dare_kernel_launches())


def dare_lmhead_static_status(stream=None) -> int:
    """Reads and clears the status word of the allocation-free LM-head calls on the current device (blocks)."""
    out = C.c_uint32(0)
    rc = load().dare_lmhead_static_status(_stream(stream), C.byref(out))
    if rc != 0:
        raise DareError(rc, "dare_lmhead_static_status")
    return int(out.value)


def dare_unmask_select(ctx: Context, tokens, block_start: int, L: int, pred, conf, mask_id: int, mode: int,
                       threshold: float = 0.0, k: int = 1, n_committed=None, n_remaining=None, stream=None,
                       check: bool = True):
    B, row_stride = tokens.shape
    rc = load().dare_unmask_select(ctx.handle, _ptr(tokens, torch.int32), B, row_stride, int(block_start), int(L),
                                   _ptr(pred, torch.int32), _ptr(conf, torch.float32), int(mask_id), int(mode),
                                   float(threshold), int(k), _count_ptr(n_committed),
                                   _count_ptr(n_remaining), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_unmask_select")
    return rc


def dare_denoise_block(ctx: Context, q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len,
                       attn_out, lse, hidden, w, mask_id: int, exclude_mask_column: bool, tokens, block_start: int,
                       mode: int, threshold: float, k: int, pred, conf, n_committed=None, n_remaining=None,
                       scale: float = 0.0, stream=None, check: bool = True):
    B, L, Hq, d = q.shape
    Hkv, prefix_cap = k_pre.shape[1], k_pre.shape[2]
    suffix_cap = k_suf.shape[2] if k_suf is not None else 0
    D = hidden.shape[1]
    V = w.shape[0]
    bf = torch.bfloat16
    rc = load().dare_denoise_block(
        ctx.handle, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, float(scale),
        _ptr(q, bf), _ptr(k_pre, bf), _ptr(v_pre, bf), _ptr(prefix_len, torch.int32), _ptr(k_blk, bf), _ptr(v_blk, bf),
        _ptr(k_suf, bf), _ptr(v_suf, bf), _ptr(suffix_len, torch.int32), _ptr(attn_out, bf), _ptr(lse, torch.float32),
        _ptr(hidden, bf), D, _ptr(w, bf), V, int(mask_id), int(bool(exclude_mask_column)),
        _ptr(tokens, torch.int32), tokens.shape[1], int(block_start), int(mode), float(threshold), int(k),
        _ptr(pred, torch.int32), _ptr(conf, torch.float32), _count_ptr(n_committed),
        _count_ptr(n_remaining), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_denoise_block")
    return rc


def dare_denoise_block_sampled(ctx: Context, q, k_pre, v_pre, prefix_len, k_blk, v_blk, k_suf, v_suf, suffix_len,
                               attn_out, lse, hidden, w, mask_id: int, exclude_mask_column: bool, temperature: float,
                               seed: int, step: int, tokens, block_start: int, mode: int, threshold: float, k: int,
                               pred, conf, n_committed=None, n_remaining=None, scale: float = 0.0, stream=None,
                               check: bool = True):
    B, L, Hq, d = q.shape
    Hkv, prefix_cap = k_pre.shape[1], k_pre.shape[2]
    suffix_cap = k_suf.shape[2] if k_suf is not None else 0
    D = hidden.shape[1]
    V = w.shape[0]
    bf = torch.bfloat16
    rc = load().dare_denoise_block_sampled(
        ctx.handle, B, L, Hq, Hkv, d, prefix_cap, suffix_cap, float(scale),
        _ptr(q, bf), _ptr(k_pre, bf), _ptr(v_pre, bf), _ptr(prefix_len, torch.int32), _ptr(k_blk, bf), _ptr(v_blk, bf),
        _ptr(k_suf, bf), _ptr(v_suf, bf), _ptr(suffix_len, torch.int32), _ptr(attn_out, bf), _ptr(lse, torch.float32),
        _ptr(hidden, bf), D, _ptr(w, bf), V, int(mask_id), int(bool(exclude_mask_column)), float(temperature),
        int(seed) & 0xFFFFFFFFFFFFFFFF, int(step) & 0xFFFFFFFF,
        _ptr(tokens, torch.int32), tokens.shape[1], int(block_start), int(mode), float(threshold), int(k),
        _ptr(pred, torch.int32), _ptr(conf, torch.float32), _count_ptr(n_committed),
        _count_ptr(n_remaining), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_denoise_block_sampled")
    return rc


LINEAR_STORE, LINEAR_RESIDUAL, LINEAR_SWIGLU = 0, 1, 2


def dare_linear(ctx: Context, epilogue: int, a, w, w2=None, residual=None, out=None, stream=None, check: bool = True):
    M, K = a.shape
    N = w.shape[0]
    bf = torch.bfloat16
    if out is None:
        out = torch.empty(M, N, dtype=bf, device=a.device)
    rc = load().dare_linear(ctx.handle, int(epilogue), _ptr(a, bf), M, K, _ptr(w, bf), _ptr(w2, bf), N, _ptr(out, bf),
                            _ptr(residual, bf), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_linear")
    return out if check else rc


def dare_linear_plan(ctx: Context, epilogue: int, M: int, K: int, N: int):
    """The launch shape dare_linear would use: dict of the eight plan numbers."""
    out = (C.c_int * 8)()
    rc = load().dare_linear_plan(ctx.handle, int(epilogue), int(M), int(K), int(N), out)
    if rc != 0:
        raise DareError(rc, "dare_linear_plan")
    keys = ("row_tiles", "w_rows", "out_cols", "k_splits", "stages", "row_items", "col_tiles", "resident_clusters")
    return dict(zip(keys, list(out)))


def dare_rmsnorm(ctx: Context, x, eps: float, y=None, stream=None, check: bool = True):
    n_rows, D = x.shape
    if y is None:
        y = torch.empty_like(x)
    rc = load().dare_rmsnorm(ctx.handle, _ptr(x, torch.bfloat16), n_rows, D, float(eps), _ptr(y, torch.bfloat16),
                             _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_rmsnorm")
    return y if check else rc


class Model:
    """Owns a dare_model: the caller's weight tensors (kept alive here), activation buffers, the RoPE table."""

    def __init__(self, ctx: Context, *, n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab, mask_id,
                 embedding, layers, lm_head, max_positions, max_rows, max_batch, rms_eps=1e-5, rope_base=10000.0):
        lib = load()
        bf = torch.bfloat16
        self.ctx = ctx
        self._keep = (embedding, layers, lm_head)
        self.desc = ModelDesc(n_layers, hidden, n_q_heads, n_kv_heads, head_dim, ffn, vocab, mask_id, rms_eps,
                              rope_base, max_positions, max_rows, max_batch)
        arr = (LayerWeights * n_layers)()
        for i, l in enumerate(layers):
            arr[i] = LayerWeights(*[_ptr(l[k], bf).value for k in ("wqkv", "wo", "wg", "wu", "wd")])
        h = C.c_void_p()
        rc = lib.dare_model_create(ctx.handle, C.byref(self.desc), _ptr(embedding, bf), arr, _ptr(lm_head, bf),
                                   C.byref(h))
        if rc != 0:
            raise DareError(rc, "dare_model_create")
        self.handle = h

    def close(self):
        if getattr(self, "handle", None):
            load().dare_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def new_cache(self, batch: int, cap: int, device="cuda"):
        shp = (self.desc.n_layers, batch, self.desc.n_kv_heads, cap, self.desc.head_dim)
        return (torch.zeros(shp, dtype=torch.bfloat16, device=device),
                torch.zeros(shp, dtype=torch.bfloat16, device=device))


def dare_rope_kv_write(model: Model, qkv, B: int, length: int, start: int, q_out, k_cache, v_cache, stream=None):
    bf = torch.bfloat16
    rc = load().dare_rope_kv_write(model.handle, _ptr(qkv, bf), B, length, start, _ptr(q_out, bf), _ptr(k_cache, bf),
                                   _ptr(v_cache, bf), k_cache.shape[-2], _stream(stream))
    if rc != 0:
        raise DareError(rc, "dare_rope_kv_write")


def dare_model_forward(model: Model, tokens, start: int, length: int, k_cache, v_cache, hidden_out=None, stream=None,
                       check: bool = True):
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    rc = load().dare_model_forward(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(start), int(length),
                                   _ptr(k_cache, bf), _ptr(v_cache, bf), k_cache.shape[3], _ptr(hidden_out, bf),
                                   _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_model_forward")
    return rc


def dare_model_step(model: Model, tokens, block_start: int, L: int, k_cache, v_cache, mode: int, threshold: float,
                    k: int, pred, conf, n_committed=None, n_remaining=None, stream=None, check: bool = True):
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    rc = load().dare_model_step(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(block_start), int(L),
                                _ptr(k_cache, bf), _ptr(v_cache, bf), k_cache.shape[3], int(mode), float(threshold),
                                int(k), _ptr(pred, torch.int32), _ptr(conf, torch.float32),
                                _count_ptr(n_committed), _count_ptr(n_remaining), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_model_step")
    return rc


def dare_generate(model: Model, tokens, prompt_len: int, gen_len: int, L: int, k_cache, v_cache, mode: int,
                  threshold: float, k: int, pred, conf, n_remaining, stream=None, check: bool = True):
    """Runs the whole loop (blocks until done); returns the list of denoising steps taken per block."""
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    steps = (C.c_int32 * (gen_len // L))()
    rc = load().dare_generate(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(prompt_len), int(gen_len),
                              int(L), _ptr(k_cache, bf), _ptr(v_cache, bf), k_cache.shape[3], int(mode),
                              float(threshold), int(k), _ptr(pred, torch.int32), _ptr(conf, torch.float32),
                              _ptr(n_remaining, torch.int32), steps, _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_generate")
    return list(steps) if check else rc


def dare_model_forward_window(model: Model, tokens, start: int, length: int, kv_len: int, k_cache, v_cache,
                              hidden_out=None, stream=None, check: bool = True):
    """dare_model_forward with the rows seeing cache[0 : kv_len) (a cached suffix behind them)."""
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    rc = load().dare_model_forward_window(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(start),
                                          int(length), int(kv_len), _ptr(k_cache, bf), _ptr(v_cache, bf),
                                          k_cache.shape[3], _ptr(hidden_out, bf), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_model_forward_window")
    return rc


def dare_model_step_window(model: Model, tokens, block_start: int, L: int, kv_len: int, k_cache, v_cache, mode: int,
                           threshold: float, k: int, pred, conf, n_committed=None, n_remaining=None, stream=None,
                           check: bool = True):
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    rc = load().dare_model_step_window(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(block_start), int(L),
                                       int(kv_len), _ptr(k_cache, bf), _ptr(v_cache, bf), k_cache.shape[3], int(mode),
                                       float(threshold), int(k), _ptr(pred, torch.int32), _ptr(conf, torch.float32),
                                       _count_ptr(n_committed), _count_ptr(n_remaining), _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_model_step_window")
    return rc


def dare_generate_dual(model: Model, tokens, prompt_len: int, gen_len: int, L: int, k_cache, v_cache, mode: int,
                       threshold: float, k: int, pred, conf, n_remaining, stream=None, check: bool = True):
    """The dual-cache loop (blocks until done); returns the list of denoising steps taken per block."""
    B, row_stride = tokens.shape
    bf = torch.bfloat16
    steps = (C.c_int32 * (gen_len // L))()
    rc = load().dare_generate_dual(model.handle, _ptr(tokens, torch.int32), B, row_stride, int(prompt_len),
                                   int(gen_len), int(L), _ptr(k_cache, bf), _ptr(v_cache, bf), k_cache.shape[3],
                                   int(mode), float(threshold), int(k), _ptr(pred, torch.int32),
                                   _ptr(conf, torch.float32), _ptr(n_remaining, torch.int32), steps, _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_generate_dual")
    return list(steps) if check else rc


def dare_model_set_sampling(model: Model, temperature: float, seed: int = 0, first_step: int = 0, stream=None,
                            check: bool = True):
    """temperature > 0: the model's step and loop calls sample; 0: back to the argmax."""
    rc = load().dare_model_set_sampling(model.handle, float(temperature), int(seed) & 0xFFFFFFFFFFFFFFFF,
                                        int(first_step) & 0xFFFFFFFF, _stream(stream))
    if rc != 0 and check:
        raise DareError(rc, "dare_model_set_sampling")
    return rc
