"""Thin ctypes binding over the C-ABI library declared in ``include/earn.h``.

Argument marshalling only: every function here packs pointers and sizes and
calls the entry point of the same name; all arithmetic runs in the CUDA
kernels.  Tensors are torch CUDA tensors used purely as device memory; the
stream is torch's current stream.  A missing library raises — there is no
fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libearn.so")

EARN_OK, EARN_ERR_INVALID_ARG, EARN_ERR_UNSUPPORTED, EARN_ERR_WORKSPACE, EARN_ERR_CUDA, EARN_ERR_TIMEOUT = range(6)
EARN_F32, EARN_BF16 = 0, 1
PAGE_TOKENS = 16


class EarnModel(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("split_k", C.c_int32), ("n_q_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("dtype", C.c_int32),
                ("softmax_scale", C.c_float)]


class EarnBatch(C.Structure):
    _fields_ = [("batch", C.c_int32), ("total_tokens", C.c_int32), ("max_seqlen", C.c_int32),
                ("cu_seqlens", C.c_void_p), ("cu_seqlens_host", C.c_void_p),
                ("n_head_reg", C.c_int32), ("n_tail_reg", C.c_int32)]


class EarnCache(C.Structure):
    _fields_ = [("k_shared", C.c_void_p), ("v_shared", C.c_void_p), ("block_table", C.c_void_p),
                ("pages_per_seq", C.c_int32), ("n_pages", C.c_int32),
                ("k_priv", C.c_void_p), ("v_priv", C.c_void_p), ("lineage", C.c_void_p),
                ("beams", C.c_int32), ("max_new", C.c_int32), ("reg_idx", C.c_void_p),
                ("priv_block_table", C.c_void_p), ("priv_pages_per_beam", C.c_int32), ("n_priv_pages", C.c_int32)]


class EarnProj(C.Structure):
    _fields_ = [("d_model", C.c_int32), ("max_pos", C.c_int32), ("rms_eps", C.c_float), ("x_is_compact", C.c_int32),
                ("rope_cos", C.c_void_p), ("rope_sin", C.c_void_p)]


SYMBOLS = {
    "earn_workspace_bytes": (C.c_size_t, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32]),
    "earn_workspace_init": (C.c_int, [C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_device_status": (C.c_int, [C.c_void_p, C.c_void_p]),
    "earn_selftest_wait_timeout": (C.c_int, [C.c_void_p, C.c_size_t, C.c_int64, C.c_void_p]),
    "earn_prefill_attn": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_void_p, C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_compact_kv": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_void_p, C.c_void_p,
                                  C.c_void_p, C.c_void_p, C.POINTER(EarnCache), C.c_void_p]),
    "earn_register_qkv": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.POINTER(EarnProj), C.c_void_p,
                                    C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(EarnCache), C.c_void_p, C.c_void_p,
                                    C.c_size_t, C.c_void_p]),
    "earn_register_attn": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_void_p,
                                     C.POINTER(EarnCache), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_compact_register_attn": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_void_p, C.c_void_p,
                                             C.c_void_p, C.POINTER(EarnCache), C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_decode_attn": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_int32, C.c_void_p,
                                   C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(EarnCache), C.c_void_p,
                                   C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_decode_attn_static": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_int32, C.c_void_p,
                                          C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(EarnCache), C.c_void_p,
                                          C.c_void_p]),
    "earn_beam_reparent": (C.c_int, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_void_p]),
    "earn_train_workspace_bytes": (C.c_size_t, [C.POINTER(EarnModel), C.POINTER(EarnBatch)]),
    "earn_train_attn_fwd": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_train_attn_bwd": (C.c_int, [C.POINTER(EarnModel), C.POINTER(EarnBatch), C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_beam_topk_workspace_bytes": (C.c_size_t, [C.c_int32, C.c_int32, C.c_int32]),
    "earn_beam_topk": (C.c_int, [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                 C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]),
    "earn_launch_count": (C.c_uint64, []),
    "earn_status_string": (C.c_char_p, [C.c_int]),
    "earn_version": (C.c_int32, []),
}

_lib = None


def lib() -> C.CDLL:
    """Load libearn.so (once).  Raises if it has not been built — nothing stands in for it."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2507_00715_b200.build` "
                               "(or __graft_entry__.build()) first; there is no fallback implementation")
        handle = C.CDLL(LIB_PATH)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


class EarnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().earn_status_string(status).decode()
        super().__init__(f"{where}: {msg} (status {status})")


def _check(status: int, where: str) -> None:
    if status != EARN_OK:
        raise EarnError(status, where)


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    return int(t)


def _stream() -> Optional[int]:
    return torch.cuda.current_stream().cuda_stream or None


def make_model(n_layers, split_k, n_q_heads, n_kv_heads, head_dim, dtype, softmax_scale=0.0) -> EarnModel:
    code = {torch.float32: EARN_F32, torch.bfloat16: EARN_BF16, "f32": EARN_F32, "bf16": EARN_BF16}.get(dtype, dtype)
    return EarnModel(n_layers, split_k, n_q_heads, n_kv_heads, head_dim, int(code), float(softmax_scale))


class Batch:
    """Owns the host and device copies of cu_seqlens behind an earn_batch_t."""

    def __init__(self, cu_seqlens_host: np.ndarray, r_head: int, r_tail: int, device="cuda",
                 cu_seqlens_dev: Optional[torch.Tensor] = None):
        self.cu_host = np.ascontiguousarray(cu_seqlens_host, dtype=np.int32)
        self.cu_dev = cu_seqlens_dev if cu_seqlens_dev is not None else torch.from_numpy(self.cu_host).to(device)
        n = len(self.cu_host) - 1
        lens = np.diff(self.cu_host) if n > 0 else np.zeros(0, dtype=np.int32)
        self.c = EarnBatch(n, int(self.cu_host[-1]) if n >= 0 and len(self.cu_host) else 0,
                           int(lens.max()) if n > 0 else 0, self.cu_dev.data_ptr(),
                           self.cu_host.ctypes.data, r_head, r_tail)

    @property
    def batch(self) -> int:
        return self.c.batch

    @property
    def n_regs(self) -> int:
        return self.c.n_head_reg + self.c.n_tail_reg


def make_cache(k_shared=None, v_shared=None, block_table=None, pages_per_seq=0, n_pages=0, k_priv=None, v_priv=None,
               lineage=None, beams=1, max_new=1, reg_idx=None, priv_block_table=None, priv_pages_per_beam=0,
               n_priv_pages=0) -> EarnCache:
    return EarnCache(_ptr(k_shared), _ptr(v_shared), _ptr(block_table), pages_per_seq, n_pages, _ptr(k_priv),
                     _ptr(v_priv), _ptr(lineage), beams, max_new, _ptr(reg_idx), _ptr(priv_block_table),
                     priv_pages_per_beam, n_priv_pages)


def earn_version() -> int:
    return lib().earn_version()


def earn_launch_count() -> int:
    return int(lib().earn_launch_count())


def earn_workspace_bytes(model: EarnModel, batch: Batch, beams: int) -> int:
    return lib().earn_workspace_bytes(C.byref(model), C.byref(batch.c), beams)


def earn_workspace_init(workspace: torch.Tensor) -> None:
    _check(lib().earn_workspace_init(_ptr(workspace), workspace.numel() * workspace.element_size(), _stream()),
           "earn_workspace_init")


def earn_device_status(workspace: torch.Tensor) -> int:
    return lib().earn_device_status(_ptr(workspace), _stream())


def earn_selftest_wait_timeout(workspace: torch.Tensor, limit_cycles: int) -> None:
    _check(lib().earn_selftest_wait_timeout(_ptr(workspace), workspace.numel() * workspace.element_size(),
                                            int(limit_cycles), _stream()), "earn_selftest_wait_timeout")


def _ws(workspace):
    if workspace is None:
        return None, 0
    return _ptr(workspace), workspace.numel() * workspace.element_size()


def earn_prefill_attn(model, batch: Batch, layer, q, k, v, o, lse=None, workspace=None) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_prefill_attn(C.byref(model), C.byref(batch.c), layer, _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                   _ptr(lse), p, n, _stream()), "earn_prefill_attn")


def earn_compact_kv(model, batch: Batch, layer, k, v, cache: EarnCache, q=None, q_reg=None) -> None:
    _check(lib().earn_compact_kv(C.byref(model), C.byref(batch.c), layer, _ptr(k), _ptr(v), _ptr(q), _ptr(q_reg),
                                 C.byref(cache), _stream()), "earn_compact_kv")


def make_proj(d_model: int, rope_cos: torch.Tensor, rope_sin: torch.Tensor, rms_eps: float = 1e-6,
              x_is_compact: bool = False) -> EarnProj:
    """rope_cos / rope_sin: device fp32 [max_pos, D/2], kept alive by the caller."""
    return EarnProj(d_model, rope_cos.shape[0], rms_eps, int(x_is_compact), _ptr(rope_cos), _ptr(rope_sin))


def earn_register_qkv(model, batch: Batch, layer, proj: EarnProj, x, w_norm, w_qkv, x_norm_scratch, cache: EarnCache,
                      q_reg, workspace=None) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_register_qkv(C.byref(model), C.byref(batch.c), layer, C.byref(proj), _ptr(x), _ptr(w_norm),
                                   _ptr(w_qkv), _ptr(x_norm_scratch), C.byref(cache), _ptr(q_reg), p, n, _stream()),
           "earn_register_qkv")


def earn_register_attn(model, batch: Batch, layer, q_reg, cache: EarnCache, o_reg, workspace=None) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_register_attn(C.byref(model), C.byref(batch.c), layer, _ptr(q_reg), C.byref(cache), _ptr(o_reg),
                                    p, n, _stream()), "earn_register_attn")


def earn_compact_register_attn(model, batch: Batch, layer, q, k, v, cache: EarnCache, o_reg, workspace=None) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_compact_register_attn(C.byref(model), C.byref(batch.c), layer, _ptr(q), _ptr(k), _ptr(v),
                                            C.byref(cache), _ptr(o_reg), p, n, _stream()), "earn_compact_register_attn")


def earn_decode_attn(model, batch: Batch, layer, step, q, k_new, v_new, cache: EarnCache, o, k_full=None, v_full=None,
                     workspace=None) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_decode_attn(C.byref(model), C.byref(batch.c), layer, step, _ptr(q), _ptr(k_new), _ptr(v_new),
                                  _ptr(k_full), _ptr(v_full), C.byref(cache), _ptr(o), p, n, _stream()),
           "earn_decode_attn")


STATIC_SCRATCH_BYTES = 8 << 20


def earn_decode_attn_static(model, batch: Batch, layer, step, q, k_new, v_new, cache: EarnCache, o, k_full=None,
                            v_full=None) -> None:
    """earn_decode_attn without a workspace argument: the library's built-in scratch array is used, so the
    caller needs no device allocation of its own (batches that need more than STATIC_SCRATCH_BYTES raise)."""
    _check(lib().earn_decode_attn_static(C.byref(model), C.byref(batch.c), layer, step, _ptr(q), _ptr(k_new),
                                         _ptr(v_new), _ptr(k_full), _ptr(v_full), C.byref(cache), _ptr(o), _stream()),
           "earn_decode_attn_static")


def earn_beam_reparent(batch: int, beams: int, max_new: int, step: int, parent, lineage_in, lineage_out) -> None:
    _check(lib().earn_beam_reparent(batch, beams, max_new, step, _ptr(parent), _ptr(lineage_in), _ptr(lineage_out),
                                    _stream()), "earn_beam_reparent")


def earn_beam_topk_workspace_bytes(batch: int, beams: int, vocab: int) -> int:
    return lib().earn_beam_topk_workspace_bytes(batch, beams, vocab)


def earn_beam_topk(batch: int, beams: int, n_live: int, vocab: int, logprobs, beam_scores, parent, token, new_scores,
                   workspace) -> None:
    """logprobs fp32 [B*W, vocab], beam_scores fp32 [B*W] or None -> parent, token int32 [B*W], new_scores fp32 [B*W]."""
    p, n = _ws(workspace)
    _check(lib().earn_beam_topk(batch, beams, n_live, vocab, _ptr(logprobs), _ptr(beam_scores), _ptr(parent), _ptr(token),
                                _ptr(new_scores), p, n, _stream()), "earn_beam_topk")


def earn_train_workspace_bytes(model: EarnModel, batch: Batch) -> int:
    return lib().earn_train_workspace_bytes(C.byref(model), C.byref(batch.c))


def earn_train_attn_fwd(model, batch: Batch, layer, n_target, q, k, v, o, lse, workspace) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_train_attn_fwd(C.byref(model), C.byref(batch.c), layer, n_target, _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                     _ptr(lse), p, n, _stream()), "earn_train_attn_fwd")


def earn_train_attn_bwd(model, batch: Batch, layer, n_target, q, k, v, o, lse, d_o, dq, dk, dv, workspace) -> None:
    p, n = _ws(workspace)
    _check(lib().earn_train_attn_bwd(C.byref(model), C.byref(batch.c), layer, n_target, _ptr(q), _ptr(k), _ptr(v), _ptr(o),
                                     _ptr(lse), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), p, n, _stream()),
           "earn_train_attn_bwd")
