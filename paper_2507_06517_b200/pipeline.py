"""Whole-prompt driver: one object that owns the device buffers of a SpindleKV reduction pass and
issues the four library calls for all layers (plan, evict deep layers, build CodeBooks for shallow
layers, compact).  No arithmetic happens here; this is buffer ownership and call order only.
"""
from __future__ import annotations

from typing import Dict, Optional, Sequence

import numpy as np
import torch

from . import binding as B


class SpindleKVPass:
    """Buffers and call sequence for one prompt batch.

    ``K`` and ``V`` are ``[n_layers, B, H_kv, N, d]`` (equal lengths) or packed
    ``[n_layers, total_tokens, H_kv, d]`` with ``cu_seqlens``; ``Q`` is
    ``[n_layers - n_shallow, B, H_q, w, d]`` (window queries of the evicting layers).
    Layers ``[0, n_shallow)`` get CodeBooks, the others are evicted.
    """

    def __init__(self, cfg: B.Config, seq_lens: Sequence[int], dtype: torch.dtype, device="cuda",
                 layers_per_codebook_call: Optional[int] = None, keep_adjacency: bool = False):
        self.cfg = cfg
        self.seq_lens = [int(x) for x in seq_lens]
        self.dtype = dtype
        self.device = torch.device(device)
        self.n_seqs = len(self.seq_lens)
        self.max_len = max(self.seq_lens)
        self.packed = len(set(self.seq_lens)) > 1
        self.total = sum(self.seq_lens) if self.packed else self.n_seqs * self.max_len
        self.n_deep = cfg.n_layers - cfg.n_shallow
        self.n_shallow = cfg.n_shallow
        dev = self.device
        self.cu = None
        if self.packed:
            cu = np.concatenate([[0], np.cumsum(self.seq_lens)]).astype(np.int32)
            self.cu = torch.from_numpy(cu).to(dev)
        self.mode, self.ratio, self.k_ctx_host = B.spindlekv_plan_layers(cfg, self.seq_lens)
        H, d, T = cfg.n_kv_heads, cfg.head_dim, self.total
        i32 = dict(dtype=torch.int32, device=dev)
        if self.n_deep:
            self.deep_batch = B.Batch(self.n_deep, self.n_seqs, self.max_len, T, self.cu)
            self.k_ctx = torch.from_numpy(np.ascontiguousarray(self.k_ctx_host[self.n_shallow:])).to(dev)
            self.keep_idx = torch.zeros((self.n_deep, H, T), **i32)
            self.keep_cnt = torch.zeros((self.n_deep, self.n_seqs, H), **i32)
            self.scores = torch.zeros((self.n_deep, H, T), dtype=torch.float32, device=dev)
            nb = B.spindlekv_workspace_bytes(cfg, self.deep_batch, B.WS_EVICT)
            self.ws_evict = torch.empty(nb, dtype=torch.uint8, device=dev)
            self.K_kept = self._alloc_like_input(self.n_deep, dtype)
            self.V_kept = self._alloc_like_input(self.n_deep, dtype)
        if self.n_shallow:
            per_call = layers_per_codebook_call or self.n_shallow
            self.cb_layers_per_call = min(per_call, self.n_shallow)
            self.cb_batch = B.Batch(self.cb_layers_per_call, self.n_seqs, self.max_len, T, self.cu)
            nb = B.spindlekv_workspace_bytes(cfg, self.cb_batch, B.WS_CODEBOOK)
            self.ws_codebook = torch.empty(nb, dtype=torch.uint8, device=dev)
            self.cb: Dict[str, Dict[str, torch.Tensor]] = {}
            for g in ("K", "V"):
                self.cb[g] = {
                    "mag": torch.zeros((self.n_shallow, H, T), dtype=torch.float32, device=dev),
                    "ref": torch.zeros((self.n_shallow, H, T), **i32),
                    "centre_idx": torch.zeros((self.n_shallow, H, T), **i32),
                    "n_entries": torch.zeros((self.n_shallow, self.n_seqs, H), **i32),
                    "C": self._alloc_like_input(self.n_shallow, dtype),
                }
            self.adj = None
            if keep_adjacency:
                units = self.cb_layers_per_call * self.n_seqs * H
                self.adj = torch.zeros((units, self.max_len, B.row_words(self.max_len)), **i32)

    def _alloc_like_input(self, n_layers: int, dtype: torch.dtype) -> torch.Tensor:
        H, d = self.cfg.n_kv_heads, self.cfg.head_dim
        if self.packed:
            return torch.zeros((n_layers, self.total, H, d), dtype=dtype, device=self.device)
        return torch.zeros((n_layers, self.n_seqs, H, self.max_len, d), dtype=dtype, device=self.device)

    def _desc(self, t: torch.Tensor):
        return B.desc_thd(t) if self.packed else B.desc_bhnd(t)

    # -- the four calls, in order ------------------------------------------------------------
    def evict(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, stream=None) -> None:
        """Deep layers: ``K``/``V`` hold only the evicting layers."""
        cfg = self.cfg
        B.spindlekv_evict_deep(cfg, self.deep_batch, self._desc(K), B.desc_bhnd(Q), self.k_ctx, self.keep_idx,
                               self.keep_cnt, self.scores, self.ws_evict, stream)
        for src, dst in ((K, self.K_kept), (V, self.V_kept)):
            B.spindlekv_compact(self.deep_batch, cfg.n_kv_heads, cfg.head_dim, self._desc(src), self.keep_idx,
                                self.keep_cnt, self._desc(dst), None, None, stream)

    def codebook(self, G: torch.Tensor, which: str, stream=None) -> None:
        """Shallow layers: ``G`` holds only the CodeBook layers of ``which`` in {"K", "V"}."""
        cfg = self.cfg
        theta = cfg.theta_k if which == "K" else cfg.theta_v
        out = self.cb[which]
        step = self.cb_layers_per_call
        for l0 in range(0, self.n_shallow, step):
            n = min(step, self.n_shallow - l0)
            batch = self.cb_batch if n == step else B.Batch(n, self.n_seqs, self.max_len, self.total, self.cu)
            sl = slice(l0, l0 + n)
            B.spindlekv_codebook_shallow(cfg, batch, self._desc(G[sl]), theta, out["mag"][sl], out["ref"][sl],
                                         out["centre_idx"][sl], out["n_entries"][sl], self.ws_codebook, self.adj,
                                         stream)
            B.spindlekv_compact(batch, cfg.n_kv_heads, cfg.head_dim, self._desc(G[sl]), out["centre_idx"][sl],
                                out["n_entries"][sl], self._desc(out["C"][sl]), out["mag"][sl], None, stream)

    def run(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, stream=None) -> None:
        """All layers of one prompt batch (``K``/``V`` hold every layer)."""
        ns = self.n_shallow
        if self.n_deep:
            self.evict(K[ns:], V[ns:], Q, stream)
        if ns:
            self.codebook(K[:ns], "K", stream)
            self.codebook(V[:ns], "V", stream)

    def device_status(self):
        """Status words of both workspaces (synchronises the device)."""
        torch.cuda.synchronize(self.device)
        out = {}
        if self.n_deep:
            out["evict"] = B.spindlekv_poll_status(self.ws_evict)
        if self.n_shallow:
            out["codebook"] = B.spindlekv_poll_status(self.ws_codebook)
        return out
