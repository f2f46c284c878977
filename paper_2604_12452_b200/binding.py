"""Thin ctypes binding of the LCA C ABI (include/lca.h).

The functions named ``lca_*`` take the same arguments as the C entry points; tensors may be
passed as torch tensors (their device pointer is taken), raw integer addresses, or None.  They
return the integer status.  The helpers below them (``condense``, ``prefill_attention``,
``decode_attention``) only allocate outputs / workspace with torch and check the status; every
step of the method runs inside the CUDA library.  There is no CPU fallback: importing this
module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import math
import os
from typing import Optional

import torch

from . import build as _build

LCA_OK = 0
LCA_VARIANT_MLA, LCA_VARIANT_GQA = 0, 1
LCA_WS_CONDENSE, LCA_WS_PREFILL, LCA_WS_DECODE, LCA_WS_UPDATE = 0, 1, 2, 3
LCA_WS_CONDENSE_VARLEN, LCA_WS_PREFILL_VARLEN = 4, 5
LCA_STATIC_SCRATCH_BYTES = 1 << 20
LCA_ERR_STATIC_SCRATCH_EXCEEDED = -7
LCA_ERR_DEVICE_TIMEOUT = -6
ATTN_AUTO, ATTN_SCALAR, ATTN_TENSOR = 0, 1, 2
REDUCE_DEFAULT, REDUCE_MAXPOOL, REDUCE_MEANPOOL, REDUCE_WEIGHTED, REDUCE_MAXSEL = 0, 1, 2, 3, 4


class LcaParams(C.Structure):
    """Mirror of ``lca_params`` (Alg. 1 REQUIRE line + head layout)."""
    _fields_ = [("variant", C.c_int32), ("batch", C.c_int32), ("seq_len", C.c_int32),
                ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("d_sem", C.c_int32),
                ("d_pos", C.c_int32), ("group_size", C.c_int32), ("window", C.c_int32),
                ("n_summary_q", C.c_int32), ("softmax_scale", C.c_float),
                ("rep_logit_bias", C.c_float), ("sem_reducer", C.c_int32), ("pos_reducer", C.c_int32)]


class LcaError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {lca_status_string(status)} ({status})")


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with paper_2604_12452_b200.build.build() "
                          "(python __graft_entry__.py); there is no fallback path")
    lib = C.CDLL(path)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    P = C.POINTER(LcaParams)
    lib.lca_version.restype = C.c_int
    lib.lca_status_string.restype = C.c_char_p
    lib.lca_status_string.argtypes = [C.c_int]
    lib.lca_launch_count.restype = i64
    lib.lca_set_attention_impl.restype = C.c_int
    lib.lca_set_attention_impl.argtypes = [C.c_int]
    lib.lca_partition.restype = C.c_int
    lib.lca_partition.argtypes = [P, C.POINTER(i32), C.POINTER(i32)]
    lib.lca_workspace_bytes.restype = sz
    lib.lca_workspace_bytes.argtypes = [P, i32]
    lib.lca_condense.restype = C.c_int
    lib.lca_condense.argtypes = [P, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lca_condense_static_scratch.restype = C.c_int
    lib.lca_condense_static_scratch.argtypes = [P, vp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.lca_prefill_attention.restype = C.c_int
    lib.lca_prefill_attention.argtypes = [P, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lca_decode_attention.restype = C.c_int
    lib.lca_decode_attention.argtypes = [P, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, sz, vp]
    lib.lca_decode_update.restype = C.c_int
    lib.lca_decode_update.argtypes = [P, vp, vp, i64, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.lca_ring_from_packed.restype = C.c_int
    lib.lca_ring_from_packed.argtypes = [P, vp, vp, vp, vp, i32, vp, vp, i32, vp, vp]
    lib.lca_decode_attention_ring.restype = C.c_int
    lib.lca_decode_attention_ring.argtypes = [P, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, sz, vp]
    lib.lca_decode_update_ring.restype = C.c_int
    lib.lca_decode_update_ring.argtypes = [P, vp, vp, i64, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.lca_decode_step_update_ring.restype = C.c_int
    lib.lca_decode_step_update_ring.argtypes = [P, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    pi32, pi64 = C.POINTER(i32), C.POINTER(i64)
    lib.lca_varlen_layout.restype = C.c_int
    lib.lca_varlen_layout.argtypes = [P, pi32, pi64, pi64, pi64]
    lib.lca_condense_varlen.restype = C.c_int
    lib.lca_condense_varlen.argtypes = [P, pi32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lca_prefill_attention_varlen.restype = C.c_int
    lib.lca_prefill_attention_varlen.argtypes = [P, pi32, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.lca_latent_to_value.restype = C.c_int
    lib.lca_latent_to_value.argtypes = [vp, vp, vp, i64, i32, i32, i32, vp]
    lib.lca_selftest_bounded_wait.restype = C.c_int
    lib.lca_selftest_bounded_wait.argtypes = [i64, vp]
    lib.lca_last_device_status.restype = C.c_int
    lib.lca_last_device_status.argtypes = [vp]
    return lib


_lib = _load()


def _ptr(x):
    if x is None:
        return None
    if isinstance(x, torch.Tensor):
        if not x.is_contiguous():
            raise ValueError("the LCA entry points take dense row-major tensors: call .contiguous() first")
        return C.c_void_p(x.data_ptr())
    return C.c_void_p(int(x))


def _nbytes(x) -> int:
    return 0 if x is None else x.numel() * x.element_size()


def _stream(stream):
    if stream is None:
        if not torch.cuda.is_available():      # host-side validation calls on a GPU-less machine
            return C.c_void_p(0)
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, torch.cuda.Stream):
        return C.c_void_p(stream.cuda_stream)
    return C.c_void_p(int(stream))


# ------------------------------------------------------------------ raw entry points (same names)
def lca_version() -> int:
    return int(_lib.lca_version())


def lca_status_string(status: int) -> str:
    return _lib.lca_status_string(int(status)).decode()


def lca_launch_count() -> int:
    return int(_lib.lca_launch_count())


def lca_set_attention_impl(impl: int) -> int:
    return int(_lib.lca_set_attention_impl(int(impl)))


def lca_partition(params: LcaParams):
    m, k = C.c_int32(), C.c_int32()
    st = _lib.lca_partition(C.byref(params), C.byref(m), C.byref(k))
    if st != LCA_OK:
        raise LcaError(st, "lca_partition")
    return int(m.value), int(k.value)


def lca_workspace_bytes(params: LcaParams, which: int) -> int:
    return int(_lib.lca_workspace_bytes(C.byref(params), int(which)))


def lca_condense(params, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, kv_sem, kv_pos,
                 cache_sem, cache_pos, anchor_idx, scores_opt, ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_condense(C.byref(params), _ptr(q_tail_sem), _ptr(q_tail_pos),
                                 int(q_tail_batch_stride), _ptr(qbar_opt), _ptr(kv_sem), _ptr(kv_pos),
                                 _ptr(cache_sem), _ptr(cache_pos), _ptr(anchor_idx), _ptr(scores_opt),
                                 _ptr(ws), wsb, _stream(stream)))


def lca_condense_static_scratch(params, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, kv_sem,
                                kv_pos, cache_sem, cache_pos, anchor_idx, scores_opt, stream=None) -> int:
    """lca_condense without a workspace argument: the scratch is a fixed array inside the library
    (for callers that must not allocate device memory).  Same outputs, bit for bit."""
    return int(_lib.lca_condense_static_scratch(C.byref(params), _ptr(q_tail_sem), _ptr(q_tail_pos),
                                                int(q_tail_batch_stride), _ptr(qbar_opt), _ptr(kv_sem),
                                                _ptr(kv_pos), _ptr(cache_sem), _ptr(cache_pos),
                                                _ptr(anchor_idx), _ptr(scores_opt), _stream(stream)))


def lca_prefill_attention(params, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos, out, lse_opt,
                          ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_prefill_attention(C.byref(params), _ptr(q_sem), _ptr(q_pos), _ptr(kv_sem),
                                          _ptr(kv_pos), _ptr(cache_sem), _ptr(cache_pos), _ptr(out),
                                          _ptr(lse_opt), _ptr(ws), wsb, _stream(stream)))


def lca_decode_attention(params, q_sem, q_pos, cache_sem, cache_pos, cache_rows, cache_row_capacity,
                         n_rep, out, lse_opt, ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_decode_attention(C.byref(params), _ptr(q_sem), _ptr(q_pos), _ptr(cache_sem),
                                         _ptr(cache_pos), _ptr(cache_rows), int(cache_row_capacity),
                                         int(n_rep), _ptr(out), _ptr(lse_opt), _ptr(ws), wsb,
                                         _stream(stream)))


def lca_decode_update(params, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, cache_sem, cache_pos,
                      cache_row_capacity, n_rep, cache_rows, anchor_out, ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_decode_update(C.byref(params), _ptr(q_tail_sem), _ptr(q_tail_pos), int(q_tail_batch_stride),
                                      _ptr(qbar_opt), _ptr(cache_sem), _ptr(cache_pos), int(cache_row_capacity),
                                      _ptr(n_rep), _ptr(cache_rows), _ptr(anchor_out), _ptr(ws), wsb, _stream(stream)))


def lca_ring_from_packed(params, packed_sem, packed_pos, packed_rows, n_rep, packed_row_capacity, ring_sem, ring_pos,
                         ring_row_capacity, n_tok_out, stream=None) -> int:
    return int(_lib.lca_ring_from_packed(C.byref(params), _ptr(packed_sem), _ptr(packed_pos), _ptr(packed_rows), _ptr(n_rep),
                                         int(packed_row_capacity), _ptr(ring_sem), _ptr(ring_pos), int(ring_row_capacity),
                                         _ptr(n_tok_out), _stream(stream)))


def lca_decode_attention_ring(params, q_sem, q_pos, ring_sem, ring_pos, n_rep, n_tok, ring_row_capacity, out, lse_opt,
                              ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_decode_attention_ring(C.byref(params), _ptr(q_sem), _ptr(q_pos), _ptr(ring_sem), _ptr(ring_pos),
                                              _ptr(n_rep), _ptr(n_tok), int(ring_row_capacity), _ptr(out), _ptr(lse_opt),
                                              _ptr(ws), wsb, _stream(stream)))


def lca_decode_update_ring(params, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, ring_sem, ring_pos,
                           ring_row_capacity, n_rep, n_tok, anchor_out, ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_decode_update_ring(C.byref(params), _ptr(q_tail_sem), _ptr(q_tail_pos), int(q_tail_batch_stride),
                                           _ptr(qbar_opt), _ptr(ring_sem), _ptr(ring_pos), int(ring_row_capacity),
                                           _ptr(n_rep), _ptr(n_tok), _ptr(anchor_out), _ptr(ws), wsb, _stream(stream)))


def lca_decode_step_update_ring(params, q_sem, q_pos, qsum, qcount, ring_sem, ring_pos, ring_row_capacity, n_rep, n_tok,
                                anchor_out, ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_decode_step_update_ring(C.byref(params), _ptr(q_sem), _ptr(q_pos), _ptr(qsum), _ptr(qcount),
                                                _ptr(ring_sem), _ptr(ring_pos), int(ring_row_capacity), _ptr(n_rep),
                                                _ptr(n_tok), _ptr(anchor_out), _ptr(ws), wsb, _stream(stream)))


def _lens(seq_lens):
    return (C.c_int32 * len(seq_lens))(*[int(x) for x in seq_lens])


def lca_varlen_layout(params, seq_lens):
    """(token_offsets, cache_row_offsets, group_offsets): lists of batch + 1 prefix sums."""
    n = params.batch + 1
    tok, cache, grp = (C.c_int64 * n)(), (C.c_int64 * n)(), (C.c_int64 * n)()
    st = _lib.lca_varlen_layout(C.byref(params), _lens(seq_lens), tok, cache, grp)
    if st != LCA_OK:
        raise LcaError(st, "lca_varlen_layout")
    return list(tok), list(cache), list(grp)


def lca_condense_varlen(params, seq_lens, q_sem, q_pos, qbar_opt, kv_sem, kv_pos, cache_sem, cache_pos, anchor_idx,
                        ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_condense_varlen(C.byref(params), _lens(seq_lens), _ptr(q_sem), _ptr(q_pos), _ptr(qbar_opt),
                                        _ptr(kv_sem), _ptr(kv_pos), _ptr(cache_sem), _ptr(cache_pos), _ptr(anchor_idx),
                                        _ptr(ws), wsb, _stream(stream)))


def lca_prefill_attention_varlen(params, seq_lens, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos, out, lse_opt,
                                 ws, ws_bytes=None, stream=None) -> int:
    wsb = _nbytes(ws) if ws_bytes is None else int(ws_bytes)
    return int(_lib.lca_prefill_attention_varlen(C.byref(params), _lens(seq_lens), _ptr(q_sem), _ptr(q_pos), _ptr(kv_sem),
                                                 _ptr(kv_pos), _ptr(cache_sem), _ptr(cache_pos), _ptr(out), _ptr(lse_opt),
                                                 _ptr(ws), wsb, _stream(stream)))


def lca_latent_to_value(attn_latent, w_uv, out_v, n_tokens, n_heads, d_latent, d_v, stream=None) -> int:
    return int(_lib.lca_latent_to_value(_ptr(attn_latent), _ptr(w_uv), _ptr(out_v), int(n_tokens), int(n_heads),
                                        int(d_latent), int(d_v), _stream(stream)))


def lca_selftest_bounded_wait(limit_cycles: int, stream=None) -> int:
    return int(_lib.lca_selftest_bounded_wait(int(limit_cycles), _stream(stream)))


def lca_last_device_status(stream=None) -> int:
    return int(_lib.lca_last_device_status(_stream(stream)))


# ----------------------------------------------------------------------- allocation helpers
def make_params(variant: str, batch: int, seq_len: int, n_q_heads: int, n_kv_heads: int, d_sem: int,
                d_pos: int, group_size: int, window: int, softmax_scale: float,
                n_summary_q: int = 0, rep_logit_bias: float = 0.0) -> LcaParams:
    v = LCA_VARIANT_MLA if variant == "mla" else LCA_VARIANT_GQA
    return LcaParams(v, batch, seq_len, n_q_heads, n_kv_heads, d_sem, d_pos, group_size, window,
                     n_summary_q, softmax_scale, rep_logit_bias, 0, 0)


def params_from_config(cfg, batch: Optional[int] = None, **kw) -> LcaParams:
    d_pos = cfg.d_pos if cfg.variant == "mla" else cfg.d_sem
    p = make_params(cfg.variant, cfg.batch if batch is None else batch, cfg.seq_len, cfg.n_q_heads,
                    cfg.n_kv_heads, cfg.d_sem, d_pos, cfg.group_size, cfg.window, cfg.softmax_scale)
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def _check(st: int, where: str):
    if st != LCA_OK:
        raise LcaError(st, where)


def workspace(params: LcaParams, which: int, device) -> Optional[torch.Tensor]:
    n = lca_workspace_bytes(params, which)
    return torch.empty(max(n, 16), dtype=torch.uint8, device=device)


def condense(params: LcaParams, q_tail_sem, q_tail_pos, kv_sem, kv_pos, qbar: Optional[torch.Tensor] = None,
             q_tail_batch_stride: Optional[int] = None, want_scores: bool = False, out=None, ws=None,
             stream=None):
    """Allocate the condensed cache and run lca_condense.  Returns dict(cache_sem, cache_pos,
    anchor_idx, scores, m, k)."""
    dev = kv_sem.device
    m, k = lca_partition(params)
    B, Hkv = params.batch, params.n_kv_heads
    if out is None:
        out = dict(cache_sem=torch.empty((B, m + k, Hkv, params.d_sem), dtype=torch.bfloat16, device=dev),
                   cache_pos=torch.empty((B, m + k, Hkv, params.d_pos), dtype=torch.bfloat16, device=dev),
                   anchor_idx=torch.empty((B, max(m, 1), Hkv), dtype=torch.int32, device=dev))
    scores = torch.empty((B, Hkv, max(m, 1) * params.group_size), dtype=torch.float64, device=dev) if want_scores else None
    if ws is None:
        ws = workspace(params, LCA_WS_CONDENSE, dev)
    n = params.n_summary_q if params.n_summary_q > 0 else params.group_size
    n = min(n, params.seq_len)
    stride = n if q_tail_batch_stride is None else q_tail_batch_stride
    st = lca_condense(params, q_tail_sem, q_tail_pos, stride, qbar, kv_sem, kv_pos, out["cache_sem"],
                      out["cache_pos"], out["anchor_idx"], scores, ws, stream=stream)
    _check(st, "lca_condense")
    res = dict(out)
    res.update(scores=scores, m=m, k=k, ws=ws)
    return res


def prefill_attention(params: LcaParams, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos, out=None,
                      want_lse: bool = False, ws=None, stream=None):
    dev = kv_sem.device
    B, L, H = params.batch, params.seq_len, params.n_q_heads
    if out is None:
        out = torch.empty((B, L, H, params.d_sem), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, L, H), dtype=torch.float32, device=dev) if want_lse else None
    if ws is None:
        ws = workspace(params, LCA_WS_PREFILL, dev)
    st = lca_prefill_attention(params, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos, out, lse, ws,
                               stream=stream)
    _check(st, "lca_prefill_attention")
    return out, lse


def decode_attention(params: LcaParams, q_sem, q_pos, cache_sem, cache_pos, cache_rows, n_rep: int,
                     out=None, want_lse: bool = False, ws=None, stream=None):
    dev = cache_sem.device
    B, H = params.batch, params.n_q_heads
    cap = cache_sem.shape[1]
    if out is None:
        out = torch.empty((B, H, params.d_sem), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, H), dtype=torch.float32, device=dev) if want_lse else None
    if ws is None:
        ws = workspace(params, LCA_WS_DECODE, dev)
    st = lca_decode_attention(params, q_sem, q_pos, cache_sem, cache_pos, cache_rows, cap, n_rep, out, lse,
                              ws, stream=stream)
    _check(st, "lca_decode_attention")
    return out, lse


def condense_varlen(params: LcaParams, seq_lens, q_sem, q_pos, kv_sem, kv_pos, qbar: Optional[torch.Tensor] = None,
                    stream=None):
    """Packed batch of sequences of different lengths: allocate the packed cache and run lca_condense_varlen.
    Returns dict(cache_sem, cache_pos, anchor_idx, token_offsets, cache_row_offsets, group_offsets)."""
    dev = kv_sem.device
    p = LcaParams.from_buffer_copy(params)
    p.batch, p.seq_len = len(seq_lens), max(seq_lens)
    tok, cache, grp = lca_varlen_layout(p, seq_lens)
    Hkv = p.n_kv_heads
    out = dict(cache_sem=torch.empty((cache[-1], Hkv, p.d_sem), dtype=torch.bfloat16, device=dev),
               cache_pos=torch.empty((cache[-1], Hkv, p.d_pos), dtype=torch.bfloat16, device=dev),
               anchor_idx=torch.empty((max(grp[-1], 1), Hkv), dtype=torch.int32, device=dev))
    ws = workspace(p, LCA_WS_CONDENSE_VARLEN, dev)
    st = lca_condense_varlen(p, seq_lens, q_sem, q_pos, qbar, kv_sem, kv_pos, out["cache_sem"], out["cache_pos"],
                             out["anchor_idx"], ws, stream=stream)
    _check(st, "lca_condense_varlen")
    out.update(token_offsets=tok, cache_row_offsets=cache, group_offsets=grp, ws=ws)
    return out


def prefill_attention_varlen(params: LcaParams, seq_lens, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos,
                             want_lse: bool = False, stream=None):
    dev = kv_sem.device
    p = LcaParams.from_buffer_copy(params)
    p.batch, p.seq_len = len(seq_lens), max(seq_lens)
    T, H = sum(seq_lens), p.n_q_heads
    out = torch.empty((T, H, p.d_sem), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((T, H), dtype=torch.float32, device=dev) if want_lse else None
    ws = workspace(p, LCA_WS_PREFILL_VARLEN, dev)
    st = lca_prefill_attention_varlen(p, seq_lens, q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos, out, lse, ws,
                                      stream=stream)
    _check(st, "lca_prefill_attention_varlen")
    return out, lse


def latent_to_value(attn_latent: torch.Tensor, w_uv: torch.Tensor, out=None, stream=None):
    """out_v[..., h, :] = attn_latent[..., h, :] @ w_uv[h]  (attn_latent [..., H, d_latent], w_uv [H, d_latent, d_v])."""
    H, d_latent, d_v = w_uv.shape
    n_tokens = attn_latent.numel() // (H * d_latent)
    if out is None:
        out = torch.empty(attn_latent.shape[:-1] + (d_v,), dtype=torch.bfloat16, device=attn_latent.device)
    _check(lca_latent_to_value(attn_latent, w_uv, out, n_tokens, H, d_latent, d_v, stream=stream), "lca_latent_to_value")
    return out


def decode_update(params: LcaParams, q_tail_sem, q_tail_pos, cache_sem, cache_pos, n_rep, cache_rows,
                  qbar: Optional[torch.Tensor] = None, ws=None, stream=None):
    """Run lca_decode_update in place on the cache buffers and counters; returns anchor offsets [B, Hkv]."""
    dev = cache_sem.device
    anchor = torch.empty((params.batch, params.n_kv_heads), dtype=torch.int32, device=dev)
    if ws is None:
        ws = workspace(params, LCA_WS_UPDATE, dev)
    n = params.n_summary_q if params.n_summary_q > 0 else params.group_size
    st = lca_decode_update(params, q_tail_sem, q_tail_pos, n, qbar, cache_sem, cache_pos, cache_sem.shape[1], n_rep,
                           cache_rows, anchor, ws, stream=stream)
    _check(st, "lca_decode_update")
    return anchor


def ring_from_packed(params: LcaParams, packed_sem, packed_pos, packed_rows, n_rep, ring_row_capacity: int, stream=None):
    """Allocate zeroed ring buffers and fill them from a packed cache.  Returns (ring_sem, ring_pos, n_tok [B] int32)."""
    dev = packed_sem.device
    B = params.batch
    ring_sem = torch.zeros((B, ring_row_capacity) + tuple(packed_sem.shape[2:]), dtype=torch.bfloat16, device=dev)
    ring_pos = torch.zeros((B, ring_row_capacity) + tuple(packed_pos.shape[2:]), dtype=torch.bfloat16, device=dev)
    n_tok = torch.empty((B,), dtype=torch.int32, device=dev)
    st = lca_ring_from_packed(params, packed_sem, packed_pos, packed_rows, n_rep, packed_sem.shape[1], ring_sem, ring_pos,
                              ring_row_capacity, n_tok, stream=stream)
    _check(st, "lca_ring_from_packed")
    return ring_sem, ring_pos, n_tok


def decode_attention_ring(params: LcaParams, q_sem, q_pos, ring_sem, ring_pos, n_rep, n_tok, out=None,
                          want_lse: bool = False, ws=None, stream=None):
    dev = ring_sem.device
    B, H = params.batch, params.n_q_heads
    if out is None:
        out = torch.empty((B, H, params.d_sem), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((B, H), dtype=torch.float32, device=dev) if want_lse else None
    if ws is None:
        ws = workspace(params, LCA_WS_DECODE, dev)
    st = lca_decode_attention_ring(params, q_sem, q_pos, ring_sem, ring_pos, n_rep, n_tok, ring_sem.shape[1], out, lse,
                                   ws, stream=stream)
    _check(st, "lca_decode_attention_ring")
    return out, lse


def decode_update_ring(params: LcaParams, q_tail_sem, q_tail_pos, ring_sem, ring_pos, n_rep, n_tok,
                       qbar: Optional[torch.Tensor] = None, ws=None, stream=None):
    """Run lca_decode_update_ring in place on the ring buffers and n_rep; returns anchor offsets [B, Hkv]."""
    dev = ring_sem.device
    anchor = torch.empty((params.batch, params.n_kv_heads), dtype=torch.int32, device=dev)
    if ws is None:
        ws = workspace(params, LCA_WS_UPDATE, dev)
    n = params.n_summary_q if params.n_summary_q > 0 else params.group_size
    st = lca_decode_update_ring(params, q_tail_sem, q_tail_pos, n, qbar, ring_sem, ring_pos, ring_sem.shape[1], n_rep,
                                n_tok, anchor, ws, stream=stream)
    _check(st, "lca_decode_update_ring")
    return anchor


def decode_step_update_ring(params: LcaParams, q_sem, q_pos, qsum, qcount, ring_sem, ring_pos, n_rep, n_tok, ws=None,
                            anchor=None, stream=None):
    """Run lca_decode_step_update_ring in place (qsum [B, Hkv, dk] float64, qcount [B] int32); returns anchor offsets."""
    dev = ring_sem.device
    if anchor is None:
        anchor = torch.empty((params.batch, params.n_kv_heads), dtype=torch.int32, device=dev)
    if ws is None:
        ws = workspace(params, LCA_WS_UPDATE, dev)
    st = lca_decode_step_update_ring(params, q_sem, q_pos, qsum, qcount, ring_sem, ring_pos, ring_sem.shape[1], n_rep, n_tok,
                                     anchor, ws, stream=stream)
    _check(st, "lca_decode_step_update_ring")
    return anchor
