"""Buffer management around the three C-ABI calls (allocation and marshalling only).

`HotPath` owns the device buffers one decoding sequence needs (attention outputs, workspace,
device status word, selected indices, compact draft cache) and issues the library calls in the
order of Algorithm 1: verification attention for every layer (the last one also producing chunk
scores), then SelectChunks for the accepted node's row, then UpdateDraftCache.
"""
from __future__ import annotations

from typing import Dict, Optional

import torch

from . import api


class HotPath:
    def __init__(self, n_q_heads: int, n_kv_heads: int, head_dim: int, n_tree: int, chunk_size: int,
                 top_k: int, max_prefix: int, draft_layers: int = 1, draft_kv_heads: Optional[int] = None,
                 draft_head_dim: Optional[int] = None, softmax_scale: float = 0.0, device="cuda:0"):
        self.Hq, self.Hkv, self.D, self.T = n_q_heads, n_kv_heads, head_dim, n_tree
        self.C, self.k, self.max_prefix = chunk_size, top_k, max_prefix
        self.scale = softmax_scale
        self.device = torch.device(device)
        self.O = self._alloc((n_tree, n_q_heads, head_dim), torch.bfloat16)
        self.lse = self._alloc((n_q_heads, n_tree), torch.float32)
        self.max_chunks = -(-max_prefix // chunk_size)
        self._score_flat = self._alloc((n_tree * max(1, self.max_chunks),), torch.float32)
        self.status = self._alloc((1,), torch.int32).zero_()
        self.idx = self._alloc((max(1, top_k),), torch.int32).fill_(-1)
        self.n_selected = self._alloc((1,), torch.int32).zero_()
        self.n_tokens = self._alloc((1,), torch.int32).zero_()
        self.dl = draft_layers
        self.dH = draft_kv_heads or n_kv_heads
        self.dD = draft_head_dim or head_dim
        shape = (draft_layers, top_k * chunk_size, self.dH, self.dD)
        self.K_compact = self._alloc(shape, torch.bfloat16).zero_()
        self.V_compact = self._alloc(shape, torch.bfloat16).zero_()
        self._ws = self._alloc((0,), torch.uint8)
        self._desc_cache: Dict[tuple, api.AttnDesc] = {}

    # -- helpers -------------------------------------------------------------------------------
    def _alloc(self, shape, dtype) -> torch.Tensor:
        """Every device buffer of the sequence comes from here (a subclass may place them differently)."""
        return torch.empty(shape, dtype=dtype, device=self.device)

    def n_chunks(self, prefix_len: int) -> int:
        return -(-prefix_len // self.C)

    def chunk_score(self, prefix_len: int) -> torch.Tensor:
        """View [T][ceil(L/C)] of the score buffer for a given prefix length."""
        nc = self.n_chunks(prefix_len)
        return self._score_flat[: self.T * nc].view(self.T, nc)

    def _desc(self, t: Dict[str, torch.Tensor], prefix_len: int, want_score: bool) -> api.AttnDesc:
        key = (prefix_len, want_score, t["Q"].stride(), t["K_prefix"].stride(), t["K_tree"].stride())
        d = self._desc_cache.get(key)
        if d is None:
            d = api.make_attn_desc(t["Q"], t["K_prefix"], t["K_tree"], self.O, prefix_len, self.C, self.scale,
                                   want_score)
            need = api.specext_verify_attn_workspace(d)
            if need == 0:
                raise api.SpecextError(2, "specext_verify_attn_workspace")
            if self._ws.numel() < need:
                self._ws = self._alloc((need,), torch.uint8)
            self._desc_cache[key] = d
        return d

    # -- the three steps -----------------------------------------------------------------------
    def verify_attn(self, t: Dict[str, torch.Tensor], parent: torch.Tensor, prefix_len: int,
                    want_score: bool) -> None:
        if prefix_len > self.max_prefix:
            raise ValueError("prefix_len exceeds max_prefix")
        d = self._desc(t, prefix_len, want_score)
        cs = self.chunk_score(prefix_len) if want_score else None
        api.specext_verify_attn(d, t["Q"], t["K_prefix"], t["V_prefix"], t["K_tree"], t["V_tree"], parent,
                                self.O, self.lse, cs, self._ws, self.status)

    def select_chunks(self, row: int, prefix_len: int, n_sink_chunks: int = 0, n_recent_chunks: int = 0) -> None:
        api.specext_select_chunks(self.chunk_score(prefix_len), row, prefix_len, self.C, self.k, self.idx,
                                  self.n_selected, self.status, n_sink_chunks, n_recent_chunks)

    def gather_kv(self, draft_K: torch.Tensor, draft_V: torch.Tensor, prefix_len: int) -> None:
        api.specext_gather_kv(draft_K, draft_V, prefix_len, self.C, self.idx, self.n_selected, self.k,
                              self.K_compact, self.V_compact, self.n_tokens, self.status)

    def select_gather(self, row: int, prefix_len: int, draft_K: torch.Tensor, draft_V: torch.Tensor,
                      n_sink_chunks: int = 0, n_recent_chunks: int = 0) -> None:
        """SelectChunks + UpdateDraftCache as one library call."""
        api.specext_select_gather(self.chunk_score(prefix_len), row, prefix_len, self.C, self.k, draft_K, draft_V,
                                  self.idx, self.n_selected, self.K_compact, self.V_compact, self.n_tokens,
                                  self.status, n_sink_chunks, n_recent_chunks)

    def read_status(self) -> int:
        return api.specext_read_status(self.status)
