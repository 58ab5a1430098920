"""Thin ctypes binding of the C ABI declared in include/specext.h.

The functions here carry the same names as the C entry points and only marshal arguments
(device pointers, strides, the current CUDA stream); every step of the path runs in the library's
kernels.  There is no CPU fallback: if the shared library is missing or a tensor is not on a CUDA
device the call raises.
"""
from __future__ import annotations

import ctypes
import math
import os
from typing import Optional, Tuple

import torch

from . import build as _build

SPECEXT_OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE", 4: "BAD_TREE", 5: "TIMEOUT",
                6: "CUDA"}


class SpecextError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where} failed: SPECEXT_ERR_{STATUS_NAMES.get(code, code)} "
                         f"({lib().specext_status_string(code).decode()})")


class AttnDesc(ctypes.Structure):
    """Mirror of specext_attn_desc."""
    _fields_ = [("n_q_heads", ctypes.c_int32), ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
                ("prefix_len", ctypes.c_int32), ("n_tree", ctypes.c_int32), ("chunk_size", ctypes.c_int32),
                ("softmax_scale", ctypes.c_float), ("want_chunk_score", ctypes.c_int32),
                ("q_stride_t", ctypes.c_int64), ("q_stride_h", ctypes.c_int64),
                ("kv_stride_l", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
                ("tkv_stride_t", ctypes.c_int64), ("tkv_stride_h", ctypes.c_int64),
                ("o_stride_t", ctypes.c_int64), ("o_stride_h", ctypes.c_int64)]


_LIB: Optional[ctypes.CDLL] = None


def bind(path: str) -> ctypes.CDLL:
    """Loads a build of the library and declares the signatures of include/specext.h on it."""
    L = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    L.specext_verify_attn_workspace.restype = sz
    L.specext_verify_attn_workspace.argtypes = [ctypes.POINTER(AttnDesc)]
    L.specext_verify_attn.restype = ctypes.c_int
    L.specext_verify_attn.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 9 + [vp, sz, vp, vp]
    L.specext_verify_attn_static_scratch.restype = ctypes.c_int
    L.specext_verify_attn_static_scratch.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 9 + [vp, vp]
    L.specext_select_chunks.restype = ctypes.c_int
    L.specext_select_chunks.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
    L.specext_gather_kv.restype = ctypes.c_int
    L.specext_gather_kv.argtypes = [vp, vp, i32, i32, i32, i32, i32, i64, i64, i64, vp, vp, i32, vp, vp, vp,
                                    vp, vp]
    L.specext_draft_attn.restype = ctypes.c_int
    L.specext_draft_attn.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 9 + [vp, sz, vp, vp]
    L.specext_prefill_attn.restype = ctypes.c_int
    L.specext_prefill_attn.argtypes = [ctypes.POINTER(AttnDesc)] + [vp] * 7
    L.specext_select_gather.restype = ctypes.c_int
    L.specext_select_gather.argtypes = [vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp, i32, i32, i32, i64, i64,
                                        i64, vp, vp, vp, vp, vp, vp, vp]
    L.specext_read_status.restype = ctypes.c_int
    L.specext_read_status.argtypes = [vp, vp]
    L.specext_status_string.restype = ctypes.c_char_p
    L.specext_status_string.argtypes = [ctypes.c_int]
    L.specext_launch_count.restype = i64
    L.specext_launch_count.argtypes = []
    return L


def lib() -> ctypes.CDLL:
    """Loads libspecext.so (built in-tree by build.py); raises if it is not there."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = _build.LIB_PATH
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -m paper_2505_20776_b200.build` "
                           "(there is no fallback path)")
    _LIB = bind(path)
    return _LIB


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("specext operates on CUDA tensors only (there is no CPU path)")
    return t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _check(code: int, where: str) -> None:
    if code != SPECEXT_OK:
        raise SpecextError(code, where)


def _bf16_3d(t: torch.Tensor, name: str) -> None:
    if t.dtype != torch.bfloat16 or t.dim() != 3 or t.stride(2) != 1:
        raise ValueError(f"{name} must be a bf16 [.][heads][head_dim] tensor with contiguous head_dim")


def make_attn_desc(Q: torch.Tensor, K_prefix: torch.Tensor, K_tree: torch.Tensor, O: torch.Tensor,
                   prefix_len: int, chunk_size: int, softmax_scale: float = 0.0,
                   want_chunk_score: bool = False) -> AttnDesc:
    """Fills a specext_attn_desc from tensor shapes and strides (V tensors share K's strides)."""
    for t, n in ((Q, "Q"), (K_prefix, "K_prefix"), (K_tree, "K_tree"), (O, "O")):
        _bf16_3d(t, n)
    T, Hq, D = Q.shape
    d = AttnDesc()
    d.n_q_heads, d.n_kv_heads, d.head_dim = Hq, K_tree.shape[1], D
    d.prefix_len, d.n_tree, d.chunk_size = int(prefix_len), T, int(chunk_size)
    d.softmax_scale = float(softmax_scale)
    d.want_chunk_score = 1 if want_chunk_score else 0
    d.q_stride_t, d.q_stride_h = Q.stride(0), Q.stride(1)
    d.kv_stride_l, d.kv_stride_h = K_prefix.stride(0), K_prefix.stride(1)
    d.tkv_stride_t, d.tkv_stride_h = K_tree.stride(0), K_tree.stride(1)
    d.o_stride_t, d.o_stride_h = O.stride(0), O.stride(1)
    return d


def specext_verify_attn_workspace(desc: AttnDesc) -> int:
    return int(lib().specext_verify_attn_workspace(ctypes.byref(desc)))


def specext_verify_attn(desc: AttnDesc, Q: torch.Tensor, K_prefix: torch.Tensor, V_prefix: torch.Tensor,
                        K_tree: torch.Tensor, V_tree: torch.Tensor, parent: torch.Tensor, O: torch.Tensor,
                        lse: torch.Tensor, chunk_score: Optional[torch.Tensor], workspace: torch.Tensor,
                        device_status: torch.Tensor) -> None:
    """Enqueues one verification attention call on the current stream (see include/specext.h)."""
    if V_prefix.stride() != K_prefix.stride() or V_tree.stride() != K_tree.stride():
        raise ValueError("V tensors must have the strides of the matching K tensors")
    if parent.dtype != torch.int32 or lse.dtype != torch.float32 or device_status.dtype != torch.int32:
        raise ValueError("parent/device_status must be int32 and lse fp32")
    if chunk_score is not None and chunk_score.dtype != torch.float32:
        raise ValueError("chunk_score must be fp32")
    rc = lib().specext_verify_attn(ctypes.byref(desc), _ptr(Q), _ptr(K_prefix), _ptr(V_prefix), _ptr(K_tree),
                                   _ptr(V_tree), _ptr(parent), _ptr(O), _ptr(lse), _ptr(chunk_score),
                                   _ptr(workspace), workspace.numel() * workspace.element_size(),
                                   _ptr(device_status), _stream())
    _check(rc, "specext_verify_attn")


def specext_draft_attn(desc: AttnDesc, Q: torch.Tensor, K_cache: torch.Tensor, V_cache: torch.Tensor,
                       n_tokens: torch.Tensor, K_tree: torch.Tensor, V_tree: torch.Tensor, parent: torch.Tensor,
                       O: torch.Tensor, lse: torch.Tensor, workspace: torch.Tensor,
                       device_status: torch.Tensor) -> None:
    """Enqueues the draft model's attention over a compact cache whose length is an int32 on the device."""
    if V_cache.stride() != K_cache.stride() or V_tree.stride() != K_tree.stride():
        raise ValueError("V tensors must have the strides of the matching K tensors")
    if (parent.dtype != torch.int32 or lse.dtype != torch.float32 or device_status.dtype != torch.int32 or
            n_tokens.dtype != torch.int32):
        raise ValueError("parent/device_status/n_tokens must be int32 and lse fp32")
    rc = lib().specext_draft_attn(ctypes.byref(desc), _ptr(Q), _ptr(K_cache), _ptr(V_cache), _ptr(n_tokens),
                                  _ptr(K_tree), _ptr(V_tree), _ptr(parent), _ptr(O), _ptr(lse), _ptr(workspace),
                                  workspace.numel() * workspace.element_size(), _ptr(device_status), _stream())
    _check(rc, "specext_draft_attn")


def specext_prefill_attn(Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, O: torch.Tensor, lse: torch.Tensor,
                         device_status: torch.Tensor, softmax_scale: float = 0.0) -> None:
    """Enqueues the prefill (causal self-attention) of a prompt: Q, O [L][Hq][128], K, V [L][Hkv][128], lse [Hq][L]."""
    for t, n in ((Q, "Q"), (K, "K"), (V, "V"), (O, "O")):
        _bf16_3d(t, n)
    if K.stride() != V.stride() or lse.dtype != torch.float32 or device_status.dtype != torch.int32:
        raise ValueError("K and V must share strides; lse must be fp32 and device_status int32")
    L, Hq, D = Q.shape
    if K.shape[0] < L or O.shape != Q.shape or lse.numel() < Hq * L or not lse.is_contiguous():
        raise ValueError("shapes: K, V [>=L][Hkv][D], O like Q, lse contiguous [Hq][L]")
    d = AttnDesc()
    d.n_q_heads, d.n_kv_heads, d.head_dim = Hq, K.shape[1], D
    d.prefix_len, d.n_tree, d.chunk_size = L, 1, 32
    d.softmax_scale, d.want_chunk_score = float(softmax_scale), 0
    d.q_stride_t, d.q_stride_h = Q.stride(0), Q.stride(1)
    d.kv_stride_l, d.kv_stride_h = K.stride(0), K.stride(1)
    d.tkv_stride_t, d.tkv_stride_h = K.stride(0), K.stride(1)
    d.o_stride_t, d.o_stride_h = O.stride(0), O.stride(1)
    rc = lib().specext_prefill_attn(ctypes.byref(d), _ptr(Q), _ptr(K), _ptr(V), _ptr(O), _ptr(lse),
                                    _ptr(device_status), _stream())
    _check(rc, "specext_prefill_attn")


STATIC_SCRATCH_BYTES = 32 << 20


def specext_verify_attn_static_scratch(desc: AttnDesc, Q: torch.Tensor, K_prefix: torch.Tensor,
                                       V_prefix: torch.Tensor, K_tree: torch.Tensor, V_tree: torch.Tensor,
                                       parent: torch.Tensor, O: torch.Tensor, lse: torch.Tensor,
                                       chunk_score: Optional[torch.Tensor], device_status: torch.Tensor) -> None:
    """specext_verify_attn without a workspace argument: for callers that may not allocate device memory.

    The scratch is a fixed 32 MiB array inside the library; shapes that need more raise
    SPECEXT_ERR_WORKSPACE.  Calls on one device share that array and must not overlap on the GPU.
    The first call on a device should be made outside of stream capture.
    """
    if V_prefix.stride() != K_prefix.stride() or V_tree.stride() != K_tree.stride():
        raise ValueError("V tensors must have the strides of the matching K tensors")
    rc = lib().specext_verify_attn_static_scratch(ctypes.byref(desc), _ptr(Q), _ptr(K_prefix), _ptr(V_prefix),
                                                  _ptr(K_tree), _ptr(V_tree), _ptr(parent), _ptr(O), _ptr(lse),
                                                  _ptr(chunk_score), _ptr(device_status), _stream())
    _check(rc, "specext_verify_attn_static_scratch")


def specext_select_chunks(chunk_score: torch.Tensor, row: int, prefix_len: int, chunk_size: int, k: int,
                          idx: torch.Tensor, n_selected: torch.Tensor, device_status: torch.Tensor,
                          n_sink_chunks: int = 0, n_recent_chunks: int = 0) -> None:
    """Enqueues SelectChunks for one row of chunk_score [n_tree][n_chunks]."""
    if chunk_score.dtype != torch.float32 or chunk_score.dim() != 2 or not chunk_score.is_contiguous():
        raise ValueError("chunk_score must be a contiguous fp32 [n_tree][n_chunks] tensor")
    if idx.dtype != torch.int32 or n_selected.dtype != torch.int32:
        raise ValueError("idx and n_selected must be int32")
    n_tree, n_chunks = chunk_score.shape
    if idx.numel() < min(k, n_chunks):
        raise ValueError("idx is too small")
    rc = lib().specext_select_chunks(_ptr(chunk_score), n_tree, n_chunks, int(row), int(prefix_len),
                                     int(chunk_size), int(k), int(n_sink_chunks), int(n_recent_chunks),
                                     _ptr(idx), _ptr(n_selected),
                                     _ptr(device_status), _stream())
    _check(rc, "specext_select_chunks")


def specext_gather_kv(draft_K: torch.Tensor, draft_V: torch.Tensor, prefix_len: int, chunk_size: int,
                      idx: torch.Tensor, n_selected: torch.Tensor, max_selected: int, K_out: torch.Tensor,
                      V_out: torch.Tensor, n_tokens_out: torch.Tensor, device_status: torch.Tensor) -> None:
    """Enqueues UpdateDraftCache: draft_K/V [n_layers][>=L][H][D] -> K_out/V_out [n_layers][k*C][H][D]."""
    for t in (draft_K, draft_V):
        if t.dtype != torch.bfloat16 or t.dim() != 4 or t.stride(3) != 1:
            raise ValueError("draft K/V must be bf16 [layers][tokens][heads][dim]")
    if draft_K.stride() != draft_V.stride():
        raise ValueError("draft K and V must share strides")
    nl, _, H, D = draft_K.shape
    need = nl * max_selected * chunk_size * H * D
    if not (K_out.is_contiguous() and V_out.is_contiguous()) or K_out.numel() < need or V_out.numel() < need:
        raise ValueError("K_out/V_out must be contiguous and hold [layers][max_selected*C][H][D]")
    rc = lib().specext_gather_kv(_ptr(draft_K), _ptr(draft_V), nl, H, D, int(prefix_len), int(chunk_size),
                                 draft_K.stride(0), draft_K.stride(1), draft_K.stride(2), _ptr(idx),
                                 _ptr(n_selected), int(max_selected), _ptr(K_out), _ptr(V_out),
                                 _ptr(n_tokens_out), _ptr(device_status), _stream())
    _check(rc, "specext_gather_kv")


def specext_select_gather(chunk_score: torch.Tensor, row: int, prefix_len: int, chunk_size: int, k: int,
                          draft_K: torch.Tensor, draft_V: torch.Tensor, idx: torch.Tensor,
                          n_selected: torch.Tensor, K_out: torch.Tensor, V_out: torch.Tensor,
                          n_tokens_out: torch.Tensor, device_status: torch.Tensor, n_sink_chunks: int = 0,
                          n_recent_chunks: int = 0) -> None:
    """Enqueues SelectChunks + UpdateDraftCache as one call (one kernel launch for the usual sizes)."""
    if chunk_score.dtype != torch.float32 or chunk_score.dim() != 2 or not chunk_score.is_contiguous():
        raise ValueError("chunk_score must be a contiguous fp32 [n_tree][n_chunks] tensor")
    if idx.dtype != torch.int32 or n_selected.dtype != torch.int32:
        raise ValueError("idx and n_selected must be int32")
    for t in (draft_K, draft_V):
        if t.dtype != torch.bfloat16 or t.dim() != 4 or t.stride(3) != 1:
            raise ValueError("draft K/V must be bf16 [layers][tokens][heads][dim]")
    if draft_K.stride() != draft_V.stride():
        raise ValueError("draft K and V must share strides")
    n_tree, n_chunks = chunk_score.shape
    nl, _, H, D = draft_K.shape
    need = nl * k * chunk_size * H * D
    if idx.numel() < min(k, n_chunks):
        raise ValueError("idx is too small")
    if not (K_out.is_contiguous() and V_out.is_contiguous()) or K_out.numel() < need or V_out.numel() < need:
        raise ValueError("K_out/V_out must be contiguous and hold [layers][k*C][H][D]")
    rc = lib().specext_select_gather(_ptr(chunk_score), n_tree, n_chunks, int(row), int(prefix_len),
                                     int(chunk_size), int(k), int(n_sink_chunks), int(n_recent_chunks),
                                     _ptr(draft_K), _ptr(draft_V), nl, H, D,
                                     draft_K.stride(0), draft_K.stride(1), draft_K.stride(2), _ptr(idx),
                                     _ptr(n_selected), _ptr(K_out), _ptr(V_out), _ptr(n_tokens_out),
                                     _ptr(device_status), _stream())
    _check(rc, "specext_select_gather")


def specext_read_status(device_status: torch.Tensor) -> int:
    """Synchronises the current stream and returns the device status bit set."""
    return int(lib().specext_read_status(_ptr(device_status), _stream()))


def specext_launch_count() -> int:
    return int(lib().specext_launch_count())


def status_bits(bits: int) -> Tuple[str, ...]:
    return tuple(n for c, n in STATUS_NAMES.items() if c and bits & (1 << c))
