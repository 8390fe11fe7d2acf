"""Python face of the C-ABI library `libgvote.so` (declared in include/gvote.h).

Argument marshalling only: every function takes torch tensors (for device memory and the
current stream), checks dtype/device, and passes raw pointers, strides and sizes to the
entry point of the same name.  No step of the pass is computed here, and there is no
fallback: a missing library raises at the first call.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libgvote.so")
_lib = None

GVOTE_OK = 0
SEL_TOPK_C0, SEL_TOPP = 0, 1
DTYPE_F32, DTYPE_BF16 = 0, 1

EXPORTS = (
    "gvote_workspace_bytes", "gvote_workspace_queries", "gvote_fit", "gvote_fit_update", "gvote_fit_finish", "gvote_fit_static", "gvote_sample", "gvote_project", "gvote_vote", "gvote_select",
    "gvote_compact", "gvote_pack", "gvote_overlap", "gvote_compress", "gvote_compress_moments", "gvote_recompress", "gvote_compress_host", "gvote_host_arena_release",
    "gvote_poll_status", "gvote_clear_status", "gvote_exact_heads", "gvote_profile_enable", "gvote_profile_report", "gvote_launch_count", "gvote_status_string", "gvote_last_cuda_error",
)


class GVoteParams(ctypes.Structure):
    """Mirror of `gvote_params` (same field order and C types)."""
    _fields_ = [
        ("d_h", ctypes.c_int32), ("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32),
        ("d_k", ctypes.c_int32), ("rope_theta", ctypes.c_double), ("S", ctypes.c_int32),
        ("p_nuc", ctypes.c_float), ("n_f", ctypes.c_int32), ("n_s", ctypes.c_int32),
        ("sel_mode", ctypes.c_int32), ("include_c0", ctypes.c_int32), ("seed", ctypes.c_uint64),
        ("layer_id", ctypes.c_uint32), ("h_dtype", ctypes.c_int32),
    ]


class GVoteError(RuntimeError):
    def __init__(self, status: int, where: str):
        lib = load()
        msg = lib.gvote_status_string(status).decode()
        cuda = lib.gvote_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({status})" + (f": {cuda}" if status == -5 and cuda else ""))
        self.status = status


def load():
    """Load libgvote.so (built by `python -m paper_2509_03136_b200.build`).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2509_03136_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(_LIB_PATH)
    P, vp, i32, i64, sz = ctypes.POINTER(GVoteParams), ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    lib.gvote_workspace_bytes.restype = sz
    lib.gvote_workspace_bytes.argtypes = [P, i32, i64, i64]
    lib.gvote_workspace_queries.restype = sz
    lib.gvote_workspace_queries.argtypes = [P, i32, i64, i64]
    lib.gvote_fit.restype = i32
    lib.gvote_fit.argtypes = [P, vp, i64, vp, i32, i64, i64, vp, vp, vp, sz, vp]
    lib.gvote_fit_update.restype = i32
    lib.gvote_fit_update.argtypes = [P, vp, i64, vp, i32, i64, i64, vp, vp, sz, vp]
    lib.gvote_fit_finish.restype = i32
    lib.gvote_fit_finish.argtypes = [P, vp, i32, vp, vp, vp]
    lib.gvote_compress_moments.restype = i32
    lib.gvote_compress_moments.argtypes = [P, vp, vp, vp, vp, i64, vp, vp, vp, i64, i64, vp, i32, i64, i64, vp, vp, vp,
                                           vp, sz, vp]
    lib.gvote_recompress.restype = i32
    lib.gvote_recompress.argtypes = [P, vp, vp, vp, vp, i64, vp, vp, vp, i64, i64, vp, vp, vp, vp, i32, i64, i64, vp, vp,
                                     vp, vp, sz, vp]
    lib.gvote_fit_static.restype = i32
    lib.gvote_fit_static.argtypes = [P, vp, i64, vp, i32, i64, vp, vp, vp]
    lib.gvote_sample.restype = i32
    lib.gvote_sample.argtypes = [P, vp, vp, i32, vp, vp, vp]
    lib.gvote_project.restype = i32
    lib.gvote_project.argtypes = [P, vp, vp, vp, i64, vp, vp, i32, vp, vp, sz, vp]
    lib.gvote_vote.restype = i32
    lib.gvote_vote.argtypes = [P, vp, vp, i64, i64, vp, i32, i64, i64, vp, vp, vp, vp, vp, sz, vp]
    lib.gvote_select.restype = i32
    lib.gvote_select.argtypes = [P, vp, vp, vp, i64, vp, vp, i64, i64, vp, i32, i64, i64, vp, vp, vp, vp, vp, sz, vp]
    lib.gvote_compact.restype = i32
    lib.gvote_compact.argtypes = [P, vp, vp, i64, i64, vp, vp, i32, i64, i64, vp, vp, sz, vp]
    lib.gvote_overlap.restype = i32
    lib.gvote_overlap.argtypes = [P, vp, vp, i64, i64, vp, vp, i32, i64, i64, vp, vp, sz, vp]
    lib.gvote_pack.restype = i32
    lib.gvote_pack.argtypes = [P, vp, vp, i64, i64, vp, vp, i32, i64, i64, vp, vp, i64, vp, vp, vp, sz, vp]
    lib.gvote_compress.restype = i32
    lib.gvote_compress.argtypes = [P, vp, i64, vp, vp, i64, vp, vp, vp, i64, i64, vp, i32, i64, i64, vp, vp, vp,
                                   vp, sz, vp]
    lib.gvote_compress_host.restype = i32
    lib.gvote_compress_host.argtypes = [P, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
    lib.gvote_host_arena_release.restype = None
    lib.gvote_host_arena_release.argtypes = []
    lib.gvote_poll_status.restype = i32
    lib.gvote_poll_status.argtypes = [vp, vp]
    lib.gvote_clear_status.restype = i32
    lib.gvote_clear_status.argtypes = [vp, vp]
    lib.gvote_exact_heads.restype = i64
    lib.gvote_exact_heads.argtypes = [vp, vp]
    lib.gvote_profile_enable.restype = None
    lib.gvote_profile_enable.argtypes = [i32]
    lib.gvote_profile_report.restype = sz
    lib.gvote_profile_report.argtypes = [ctypes.c_char_p, sz]
    lib.gvote_launch_count.restype = i64
    lib.gvote_launch_count.argtypes = []
    lib.gvote_status_string.restype = ctypes.c_char_p
    lib.gvote_status_string.argtypes = [i32]
    lib.gvote_last_cuda_error.restype = ctypes.c_char_p
    lib.gvote_last_cuda_error.argtypes = []
    _lib = lib
    return lib


# ----------------------------------------------------------------------------- helpers
def make_params(*, d_h: int, n_q_heads: int, n_kv_heads: int, d_k: int, rope_theta: float, S: int,
                p_nuc: float, n_f: int, n_s: int, seed: int, layer_id: int = 0, sel_mode: int = SEL_TOPK_C0,
                include_c0: bool = False, h_dtype: int = DTYPE_F32) -> GVoteParams:
    return GVoteParams(d_h, n_q_heads, n_kv_heads, d_k, float(rope_theta), S, float(p_nuc), n_f, n_s, sel_mode,
                       int(bool(include_c0)), int(seed) & 0xFFFFFFFFFFFFFFFF, int(layer_id) & 0xFFFFFFFF, h_dtype)


def params_from_config(cfg, layer_id: int = 0, **kw) -> GVoteParams:
    """Parameters for a `synth.GVoteConfig`."""
    return make_params(d_h=cfg.d_h, n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, d_k=cfg.d_k,
                       rope_theta=cfg.rope_theta, S=cfg.S, p_nuc=cfg.p_nuc, n_f=cfg.n_f, n_s=cfg.n_s,
                       seed=cfg.seed, layer_id=layer_id, **kw)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(status: int, where: str) -> None:
    if status != GVOTE_OK:
        raise GVoteError(status, where)


def _dev(t: torch.Tensor, dtype, name: str, dense: bool = True) -> torch.Tensor:
    if not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    if dense and not t.is_contiguous():
        raise TypeError(f"{name} must be contiguous")
    if not dense and t.stride(-1) != 1:
        raise TypeError(f"{name} must be contiguous along its last dimension")
    return t


def mask_row_words(total_tokens: int, batch: int) -> int:
    return (total_tokens >> 5) + batch


def mask_word_offset(cu_r: int, r: int) -> int:
    return (cu_r >> 5) + r


def batch_geometry(cu_seqlens_host: Sequence[int]) -> Tuple[int, int, int]:
    """(batch, total_tokens, max_N) from host-side cumulative lengths."""
    cu = [int(x) for x in cu_seqlens_host]
    return len(cu) - 1, cu[-1], max((b - a for a, b in zip(cu[:-1], cu[1:])), default=0)


def gvote_workspace_bytes(p: GVoteParams, batch: int, total_tokens: int, max_N: int) -> int:
    return int(load().gvote_workspace_bytes(ctypes.byref(p), batch, total_tokens, max_N))


def workspace_queries(p: GVoteParams, ws: torch.Tensor, batch: int, total_tokens: int, max_N: int) -> torch.Tensor:
    """The rotated queries a whole-pass call left in `ws`: a bf16 view [batch, n_kv_heads, G*(S+1), d_k]."""
    off = int(load().gvote_workspace_queries(ctypes.byref(p), batch, total_tokens, max_N))
    if off == 0:
        raise GVoteError(-1, "gvote_workspace_queries")
    G = p.n_q_heads // p.n_kv_heads
    n = batch * p.n_kv_heads * G * (p.S + 1) * p.d_k
    return ws[off:off + 2 * n].view(torch.bfloat16).view(batch, p.n_kv_heads, G * (p.S + 1), p.d_k)


def alloc_workspace(p: GVoteParams, batch: int, total_tokens: int, max_N: int, device="cuda",
                    softmax_dump: bool = False) -> torch.Tensor:
    """A zero-filled workspace for these parameters.  softmax_dump=True sizes it for calls that ask
    gvote_vote / gvote_select for the softmax rows (dbg_probs): those keep the fp32 logits of every row,
    like the per-sample top-p mode, so the size is that mode's."""
    if softmax_dump and p.sel_mode != SEL_TOPP:
        q = GVoteParams.from_buffer_copy(p)
        q.sel_mode = SEL_TOPP
        p = q
    n = gvote_workspace_bytes(p, batch, total_tokens, max_N)
    if n == 0:
        raise GVoteError(-1, "gvote_workspace_bytes")
    return torch.zeros(n, dtype=torch.uint8, device=device)


# ----------------------------------------------------------------------------- entry points
def gvote_fit(p, h, cu_seqlens, geom, mu, var, ws) -> None:
    batch, total, max_N = geom
    _dev(h, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h", dense=False)
    _dev(cu_seqlens, torch.int32, "cu_seqlens"); _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var")
    _check(load().gvote_fit(ctypes.byref(p), _ptr(h), h.stride(0), _ptr(cu_seqlens), batch, total, max_N,
                            _ptr(mu), _ptr(var), _ptr(ws), ws.numel(), _stream()), "gvote_fit")


def gvote_fit_update(p, h_block, cu_block, geom, state, ws) -> None:
    """Fold one block of hidden-state rows (requests packed by cu_block) into the running moments
    `state` [batch, 3, d_h] float64 (zero-filled before the first block)."""
    batch, total, max_rows = geom
    _dev(h_block, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h_block", dense=False)
    _dev(cu_block, torch.int32, "cu_block"); _dev(state, torch.float64, "state")
    _check(load().gvote_fit_update(ctypes.byref(p), _ptr(h_block), h_block.stride(0), _ptr(cu_block), batch, total,
                                   max_rows, _ptr(state), _ptr(ws), ws.numel(), _stream()), "gvote_fit_update")


def gvote_fit_finish(p, state, batch, mu, var) -> None:
    _dev(state, torch.float64, "state"); _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var")
    _check(load().gvote_fit_finish(ctypes.byref(p), _ptr(state), batch, _ptr(mu), _ptr(var), _stream()),
           "gvote_fit_finish")


def gvote_compress_moments(p, mu, var, h_last, W_q, b_q, K, V, cu_seqlens, geom, mask, budget, b_step, ws) -> None:
    batch, total, max_N = geom
    _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var")
    _dev(h_last, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h_last")
    _dev(W_q, torch.bfloat16, "W_q", dense=False); _dev(K, torch.bfloat16, "K", dense=False); _dev(V, torch.bfloat16, "V", dense=False)
    _dev(mask, torch.int32, "mask"); _dev(budget, torch.int32, "budget"); _dev(b_step, torch.int32, "b_step")
    if K.stride() != V.stride():
        raise ValueError("K and V must share strides")
    _check(load().gvote_compress_moments(ctypes.byref(p), _ptr(mu), _ptr(var), _ptr(h_last), _ptr(W_q), W_q.stride(0),
                                         _ptr(b_q), _ptr(K), _ptr(V), K.stride(1), K.stride(0), _ptr(cu_seqlens),
                                         batch, total, max_N, _ptr(mask), _ptr(budget), _ptr(b_step), _ptr(ws),
                                         ws.numel(), _stream()), "gvote_compress_moments")


def gvote_recompress(p, mu, var, h_last, W_q, b_q, K, V, cu_seqlens, kv_len, seq_len, token_pos, geom, mask, budget,
                     b_step, ws) -> None:
    """The pass on a cache pruned before: kv_len [batch, n_kv_heads] rows per head, seq_len [batch] tokens
    seen, token_pos [n_kv_heads, total] slot -> position map (or None), compacted with the rows."""
    batch, total, max_N = geom
    _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var")
    _dev(h_last, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h_last")
    _dev(W_q, torch.bfloat16, "W_q", dense=False); _dev(K, torch.bfloat16, "K", dense=False); _dev(V, torch.bfloat16, "V", dense=False)
    _dev(mask, torch.int32, "mask"); _dev(budget, torch.int32, "budget"); _dev(b_step, torch.int32, "b_step")
    for t, name in ((kv_len, "kv_len"), (seq_len, "seq_len"), (token_pos, "token_pos")):
        if t is not None:                      # a missing kv_len or seq_len is the library's to refuse
            _dev(t, torch.int32, name)
    if K.stride() != V.stride():
        raise ValueError("K and V must share strides")
    _check(load().gvote_recompress(ctypes.byref(p), _ptr(mu), _ptr(var), _ptr(h_last), _ptr(W_q), W_q.stride(0),
                                   _ptr(b_q), _ptr(K), _ptr(V), K.stride(1), K.stride(0), _ptr(cu_seqlens),
                                   _ptr(kv_len), _ptr(seq_len), _ptr(token_pos), batch, total, max_N, _ptr(mask),
                                   _ptr(budget), _ptr(b_step), _ptr(ws), ws.numel(), _stream()), "gvote_recompress")


FIT_STATIC_MAX_ENTRIES = 131072


def gvote_fit_static(p, h, cu_seqlens, batch: int, max_N: int, mu, var) -> None:
    """`gvote_fit` for callers that cannot ask for device memory where they stand (an allocator
    callback, a serving loop with a frozen pool): no workspace argument, the partial sums go to
    a fixed array inside the library.  Needs batch * d_h <= FIT_STATIC_MAX_ENTRIES; calls that
    could overlap on the GPU must be serialised by the caller, they share that array."""
    _dev(h, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h", dense=False)
    _dev(cu_seqlens, torch.int32, "cu_seqlens"); _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var")
    _check(load().gvote_fit_static(ctypes.byref(p), _ptr(h), h.stride(0), _ptr(cu_seqlens), batch, max_N,
                                   _ptr(mu), _ptr(var), _stream()), "gvote_fit_static")


def gvote_sample(p, mu, var, batch, H_tilde, raw=None) -> None:
    _dev(mu, torch.float32, "mu"); _dev(var, torch.float32, "var"); _dev(H_tilde, torch.float32, "H_tilde")
    if raw is not None:
        _dev(raw, torch.int32, "raw")
    _check(load().gvote_sample(ctypes.byref(p), _ptr(mu), _ptr(var), batch, _ptr(H_tilde), _ptr(raw), _stream()),
           "gvote_sample")


def gvote_project(p, H_tilde, h_last, W_q, b_q, cu_seqlens, batch, Q, ws) -> None:
    _dev(H_tilde, torch.float32, "H_tilde"); _dev(W_q, torch.bfloat16, "W_q", dense=False); _dev(Q, torch.bfloat16, "Q")
    _dev(h_last, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h_last")
    _check(load().gvote_project(ctypes.byref(p), _ptr(H_tilde), _ptr(h_last), _ptr(W_q), W_q.stride(0), _ptr(b_q),
                                _ptr(cu_seqlens), batch, _ptr(Q), _ptr(ws), ws.numel(), _stream()), "gvote_project")


def gvote_vote(p, Q, K, cu_seqlens, geom, mask, budget, b_step, ws, dbg_probs=None) -> None:
    batch, total, max_N = geom
    _dev(Q, torch.bfloat16, "Q"); _dev(K, torch.bfloat16, "K", dense=False); _dev(mask, torch.int32, "mask")
    _dev(budget, torch.int32, "budget"); _dev(b_step, torch.int32, "b_step")
    _check(load().gvote_vote(ctypes.byref(p), _ptr(Q), _ptr(K), K.stride(1), K.stride(0), _ptr(cu_seqlens), batch,
                             total, max_N, _ptr(mask), _ptr(budget), _ptr(b_step), _ptr(dbg_probs), _ptr(ws),
                             ws.numel(), _stream()), "gvote_vote")


def gvote_select(p, H_tilde, h_last, W_q, b_q, K, cu_seqlens, geom, mask, budget, b_step, ws, dbg_probs=None) -> None:
    batch, total, max_N = geom
    _dev(H_tilde, torch.float32, "H_tilde"); _dev(W_q, torch.bfloat16, "W_q", dense=False); _dev(K, torch.bfloat16, "K", dense=False)
    _check(load().gvote_select(ctypes.byref(p), _ptr(H_tilde), _ptr(h_last), _ptr(W_q), W_q.stride(0), _ptr(b_q),
                               _ptr(K), K.stride(1), K.stride(0), _ptr(cu_seqlens), batch, total, max_N, _ptr(mask),
                               _ptr(budget), _ptr(b_step), _ptr(dbg_probs), _ptr(ws), ws.numel(), _stream()),
           "gvote_select")


def gvote_compact(p, K, V, mask, cu_seqlens, geom, budget, ws) -> None:
    batch, total, max_N = geom
    _dev(K, torch.bfloat16, "K", dense=False); _dev(V, torch.bfloat16, "V", dense=False); _dev(mask, torch.int32, "mask")
    if K.stride() != V.stride():
        raise ValueError("K and V must share strides")
    _check(load().gvote_compact(ctypes.byref(p), _ptr(K), _ptr(V), K.stride(1), K.stride(0), _ptr(mask),
                                _ptr(cu_seqlens), batch, total, max_N, _ptr(budget), _ptr(ws), ws.numel(), _stream()),
           "gvote_compact")


def gvote_overlap(p, Q, K, mask, cu_seqlens, geom, overlap, ws) -> None:
    """Share of each query head's current-query attention that falls on the kept keys (Section 3.3)."""
    batch, total, max_N = geom
    _dev(Q, torch.bfloat16, "Q"); _dev(K, torch.bfloat16, "K", dense=False); _dev(mask, torch.int32, "mask")
    _dev(overlap, torch.float32, "overlap")
    _check(load().gvote_overlap(ctypes.byref(p), _ptr(Q), _ptr(K), K.stride(1), K.stride(0), _ptr(mask),
                                _ptr(cu_seqlens), batch, total, max_N, _ptr(overlap), _ptr(ws), ws.numel(), _stream()),
           "gvote_overlap")


def gvote_pack(p, K, V, mask, cu_seqlens, geom, K_packed, V_packed, cu_seqlens_k, budget, ws) -> None:
    batch, total, max_N = geom
    _dev(K, torch.bfloat16, "K", dense=False); _dev(V, torch.bfloat16, "V", dense=False); _dev(mask, torch.int32, "mask")
    _dev(K_packed, torch.bfloat16, "K_packed"); _dev(V_packed, torch.bfloat16, "V_packed")
    _dev(cu_seqlens_k, torch.int32, "cu_seqlens_k"); _dev(budget, torch.int32, "budget")
    if K.stride() != V.stride():
        raise ValueError("K and V must share strides")
    if K_packed.shape != V_packed.shape or K_packed.dim() != 2 or K_packed.shape[1] != p.d_k:
        raise ValueError("K_packed and V_packed must be [rows, d_k]")
    _check(load().gvote_pack(ctypes.byref(p), _ptr(K), _ptr(V), K.stride(1), K.stride(0), _ptr(mask), _ptr(cu_seqlens),
                             batch, total, max_N, _ptr(K_packed), _ptr(V_packed), K_packed.shape[0],
                             _ptr(cu_seqlens_k), _ptr(budget), _ptr(ws), ws.numel(), _stream()), "gvote_pack")


def gvote_compress(p, h, W_q, b_q, K, V, cu_seqlens, geom, mask, budget, b_step, ws, h_last=None) -> None:
    batch, total, max_N = geom
    _dev(h, torch.float32 if p.h_dtype == DTYPE_F32 else torch.bfloat16, "h", dense=False)
    _dev(W_q, torch.bfloat16, "W_q", dense=False); _dev(K, torch.bfloat16, "K", dense=False); _dev(V, torch.bfloat16, "V", dense=False)
    _dev(mask, torch.int32, "mask"); _dev(budget, torch.int32, "budget"); _dev(b_step, torch.int32, "b_step")
    if K.stride() != V.stride():
        raise ValueError("K and V must share strides")
    _check(load().gvote_compress(ctypes.byref(p), _ptr(h), h.stride(0), _ptr(h_last), _ptr(W_q), W_q.stride(0),
                                 _ptr(b_q), _ptr(K), _ptr(V), K.stride(1), K.stride(0), _ptr(cu_seqlens), batch,
                                 total, max_N, _ptr(mask), _ptr(budget), _ptr(b_step), _ptr(ws), ws.numel(),
                                 _stream()), "gvote_compress")


def gvote_compress_host(p, h, W_q, b_q, K, V, cu_seqlens, mask, budget, b_step) -> None:
    """Host-memory variant: every tensor is a CPU tensor (pinned for full copy speed); K and V are
    compacted in place in host memory; returns after the device work has completed."""
    for name, t in (("h", h), ("W_q", W_q), ("K", K), ("V", V), ("cu_seqlens", cu_seqlens), ("mask", mask),
                    ("budget", budget), ("b_step", b_step)):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError(f"{name} must be a contiguous CPU tensor")
    batch = cu_seqlens.numel() - 1
    _check(load().gvote_compress_host(ctypes.byref(p), _ptr(h), _ptr(W_q), _ptr(b_q), _ptr(K), _ptr(V),
                                      _ptr(cu_seqlens), batch, _ptr(mask), _ptr(budget), _ptr(b_step)),
           "gvote_compress_host")


def gvote_host_arena_release() -> None:
    load().gvote_host_arena_release()


def gvote_poll_status(ws) -> int:
    return int(load().gvote_poll_status(_ptr(ws), _stream()))


def gvote_clear_status(ws) -> None:
    _check(load().gvote_clear_status(_ptr(ws), _stream()), "gvote_clear_status")


def gvote_exact_heads(ws) -> int:
    """(request, KV head) pairs the default mode had to select again by the exact route since the
    status block was last cleared."""
    return int(load().gvote_exact_heads(_ptr(ws), _stream()))


def gvote_profile_enable(on: bool) -> None:
    load().gvote_profile_enable(1 if on else 0)


def gvote_profile_report() -> dict:
    """{kernel name: (launches, total milliseconds)} since profiling was enabled."""
    lib = load()
    cap = 1 << 16
    buf = ctypes.create_string_buffer(cap)
    lib.gvote_profile_report(buf, cap)
    out = {}
    for line in buf.value.decode().splitlines():
        name, n, ms = line.split()
        out[name] = (int(n), float(ms))
    return out


def gvote_launch_count() -> int:
    return int(load().gvote_launch_count())


def gvote_status_string(status: int) -> str:
    return load().gvote_status_string(status).decode()


# ----------------------------------------------------------------------------- tensor plumbing
def bf16_from_bits(bits: np.ndarray, device="cuda", pin: bool = False) -> torch.Tensor:
    """uint16 bit patterns -> torch.bfloat16 tensor (no value change)."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    if device == "cpu":
        return t.pin_memory() if pin else t
    return t.to(device)


def bits_from_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def unpack_mask(mask_row: np.ndarray, word_offset: int, N: int) -> np.ndarray:
    """Bits of one request in one head's mask row -> bool [N]."""
    words = np.ascontiguousarray(mask_row[word_offset:word_offset + (N + 31) // 32]).view(np.uint32)
    bits = np.unpackbits(words.view(np.uint8), bitorder="little")
    return bits[:N].astype(bool)
