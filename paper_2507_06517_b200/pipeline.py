"""Whole-prompt driver: one object that owns the device buffers of a SpindleKV reduction pass and
issues the four library calls for all layers (plan, evict deep layers, build CodeBooks for shallow
layers, compact).  No arithmetic happens here; this is buffer ownership and call order only.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, Optional, Sequence

import numpy as np
import torch

from . import binding as B


def record_graph(fn, device="cuda") -> "torch.cuda.CUDAGraph":
    """Records what ``fn()`` enqueues (calls of this library on the current stream and on streams forked from it) as a
    CUDA graph; ``replay()`` on the result repeats it with one launch from the host.  ``fn`` runs once outside the
    recording first, so that whatever is set up on first use (kernel attributes, side streams, workspaces) exists
    before the recording starts; the tensors it uses must stay where they are."""
    dev = torch.device(device)
    warm = torch.cuda.Stream(dev)
    warm.wait_stream(torch.cuda.current_stream(dev))
    with torch.cuda.stream(warm):
        fn()
    torch.cuda.current_stream(dev).wait_stream(warm)
    torch.cuda.synchronize(dev)
    graph = torch.cuda.CUDAGraph()
    # only this thread's calls belong to the recording (a communication library's watchdog thread may poll its events meanwhile)
    with torch.cuda.graph(graph, capture_error_mode="thread_local"):
        fn()
    return graph


class SpindleKVPass:
    """Buffers and call sequence for one prompt batch.

    ``K`` and ``V`` are ``[n_layers, B, H_kv, N, d]`` (equal lengths) or packed
    ``[n_layers, total_tokens, H_kv, d]`` with ``cu_seqlens``; ``Q`` is
    ``[n_layers - n_shallow, B, H_q, w, d]`` (window queries of the evicting layers).
    Layers ``[0, n_shallow)`` get CodeBooks, the others are evicted.
    """

    def __init__(self, cfg: B.Config, seq_lens: Sequence[int], dtype: torch.dtype, device="cuda",
                 layers_per_codebook_call: Optional[int] = None, keep_adjacency: bool = False,
                 side_by_side: bool = True):
        self.cfg = cfg
        # run(): the K CodeBooks, the V CodeBooks and the eviction are independent; on three streams the short
        # kernels of one (norms, lists, cover, top-k, gathers: a block per unit, far from filling the device) run
        # beside those of the others.  Costs a second CodeBook workspace.  Off when the adjacency is kept (one
        # buffer for both calls).
        self.side_by_side = side_by_side and not keep_adjacency
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

    def _codebook_chunk(self, G: torch.Tensor, which: str, l0: int, stream=None) -> None:
        """CodeBooks of ``G.shape[0]`` consecutive shallow layers starting at layer ``l0``."""
        cfg = self.cfg
        n = G.shape[0]
        theta = cfg.theta_k if which == "K" else cfg.theta_v
        out = self.cb[which]
        batch = self.cb_batch if n == self.cb_layers_per_call else B.Batch(n, self.n_seqs, self.max_len, self.total, self.cu)
        sl = slice(l0, l0 + n)
        B.spindlekv_codebook_shallow(cfg, batch, self._desc(G), theta, out["mag"][sl], out["ref"][sl],
                                     out["centre_idx"][sl], out["n_entries"][sl], self.ws_codebook, self.adj, stream)
        B.spindlekv_compact(batch, cfg.n_kv_heads, cfg.head_dim, self._desc(G), out["centre_idx"][sl],
                            out["n_entries"][sl], self._desc(out["C"][sl]), out["mag"][sl], None, stream)

    def codebook(self, G: torch.Tensor, which: str, stream=None) -> None:
        """Shallow layers: ``G`` holds only the CodeBook layers of ``which`` in {"K", "V"}."""
        step = self.cb_layers_per_call
        for l0 in range(0, self.n_shallow, step):
            self._codebook_chunk(G[l0:l0 + min(step, self.n_shallow - l0)], which, l0, stream)

    def run(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, stream=None) -> None:
        """All layers of one prompt batch (``K``/``V`` hold every layer)."""
        ns = self.n_shallow
        if self.side_by_side and ns and (stream is None or isinstance(stream, torch.cuda.Stream)):
            return self._run_side_by_side(K, V, Q, stream)   # (a raw stream handle cannot be joined with: one stream then)
        if self.n_deep:
            self.evict(K[ns:], V[ns:], Q, stream)
        if ns:
            self.codebook(K[:ns], "K", stream)
            self.codebook(V[:ns], "V", stream)

    def capture(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor) -> "torch.cuda.CUDAGraph":
        """Records one ``run`` on these tensors (side streams included) as a CUDA graph and returns it; ``replay()``
        on the result repeats the pass on whatever the same tensors hold by then, with one launch from the host."""
        return record_graph(lambda: self.run(K, V, Q), self.device)

    def _run_side_by_side(self, K, V, Q, stream=None) -> None:
        """``run`` on three streams: K CodeBooks on the caller's stream, V CodeBooks and the eviction on two side
        streams that start after the work already queued on the caller's stream and are joined before returning."""
        dev, ns = self.device, self.n_shallow
        cur = stream if stream is not None else torch.cuda.current_stream(dev)
        if not hasattr(self, "_side"):
            self._side = [torch.cuda.Stream(dev) for _ in range(2)]
            self._ws_codebook_v = torch.empty_like(self.ws_codebook)
        sV, sE = self._side
        ev = torch.cuda.Event()
        ev.record(cur)
        sV.wait_event(ev)
        self.codebook(K[:ns], "K", cur)
        ws = self.ws_codebook
        self.ws_codebook = self._ws_codebook_v
        try:
            self.codebook(V[:ns], "V", sV)
        finally:
            self.ws_codebook = ws
        if self.n_deep:
            sE.wait_event(ev)
            self.evict(K[ns:], V[ns:], Q, sE)
            cur.wait_stream(sE)
        cur.wait_stream(sV)

    # -- the same pass fed from host memory ----------------------------------------------------
    def host_outputs(self) -> Dict[str, torch.Tensor]:
        """Pinned host tensors for everything ``run_from_host`` brings back: index maps, counts,
        magnitudes, kept rows (up to the largest ``k + w`` of any layer) and CodeBook rows."""
        out: Dict[str, torch.Tensor] = {}

        def pin(name, t):
            out[name] = torch.empty(t.shape, dtype=t.dtype, pin_memory=True)

        if self.n_deep:
            pin("keep_idx", self.keep_idx)
            pin("keep_cnt", self.keep_cnt)
            pin("K_kept", self._kept_view(self.K_kept))
            pin("V_kept", self._kept_view(self.V_kept))
        if self.n_shallow:
            for g in ("K", "V"):
                for k in ("ref", "mag", "n_entries", "C"):
                    pin(f"{g}.{k}", self.cb[g][k])
        return out

    def _kept_view(self, t: torch.Tensor) -> torch.Tensor:
        if self.packed:
            return t
        return t[:, :, :, : int(self.k_ctx_host[self.n_shallow:].max()) + self.cfg.window]

    def run_from_host(self, hK: torch.Tensor, hV: torch.Tensor, hQ: Optional[torch.Tensor],
                      host_out: Dict[str, torch.Tensor]) -> None:
        """All layers of one prompt batch whose K, V (every layer) and Q (evicting layers) sit in pinned
        host memory.  Uploads, kernels and downloads run on three streams: while the CodeBooks of one
        group of layers are built, the next group is on its way in and the previous results are on
        their way out.  Returns once everything is enqueued; work that follows on the current stream
        is ordered after the last download."""
        dev, cfg, ns = self.device, self.cfg, self.n_shallow
        cur = torch.cuda.current_stream(dev)
        if not hasattr(self, "_s_in"):
            self._s_in, self._s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
            c = self.cb_layers_per_call if ns else 0
            self._stage = [self._alloc_like_input(c, self.dtype) for _ in range(2)] if ns else []
            if self.n_deep:
                self._dK = self._alloc_like_input(self.n_deep, self.dtype)
                self._dV = self._alloc_like_input(self.n_deep, self.dtype)
                self._dQ = torch.empty(hQ.shape, dtype=hQ.dtype, device=dev)
        s_in, s_out = self._s_in, self._s_out
        s_in.wait_stream(cur)
        s_out.wait_stream(cur)
        free = [None, None]   # event after the kernels that last read a staging buffer

        def send(dst, src, after=None):
            with torch.cuda.stream(s_in):
                if after is not None:
                    s_in.wait_event(after)
                dst.copy_(src, non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(s_in)
            return ev

        def fetch(pairs):
            ev = torch.cuda.Event()
            ev.record(cur)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev)
                for h, d in pairs:
                    h.copy_(d, non_blocking=True)

        slot = 0
        step = self.cb_layers_per_call if ns else 1
        for l0 in range(0, ns, step):
            n = min(step, ns - l0)
            for which, h in (("K", hK), ("V", hV)):
                buf = self._stage[slot & 1][:n]
                cur.wait_event(send(buf, h[l0:l0 + n], free[slot & 1]))
                self._codebook_chunk(buf, which, l0)
                free[slot & 1] = torch.cuda.Event()
                free[slot & 1].record(cur)
                o = self.cb[which]
                fetch([(host_out[f"{which}.{k}"][l0:l0 + n], o[k][l0:l0 + n]) for k in ("ref", "mag", "n_entries", "C")])
                slot += 1
        if self.n_deep:
            ev_k = send(self._dK, hK[ns:])
            ev_q = send(self._dQ, hQ)
            ev_v = send(self._dV, hV[ns:])
            cur.wait_event(ev_k)
            cur.wait_event(ev_q)
            B.spindlekv_evict_deep(cfg, self.deep_batch, self._desc(self._dK), B.desc_bhnd(self._dQ), self.k_ctx,
                                   self.keep_idx, self.keep_cnt, self.scores, self.ws_evict)
            B.spindlekv_compact(self.deep_batch, cfg.n_kv_heads, cfg.head_dim, self._desc(self._dK), self.keep_idx,
                                self.keep_cnt, self._desc(self.K_kept), None, None)
            fetch([(host_out["keep_idx"], self.keep_idx), (host_out["keep_cnt"], self.keep_cnt),
                   (host_out["K_kept"], self._kept_view(self.K_kept))])
            cur.wait_event(ev_v)
            B.spindlekv_compact(self.deep_batch, cfg.n_kv_heads, cfg.head_dim, self._desc(self._dV), self.keep_idx,
                                self.keep_cnt, self._desc(self.V_kept), None, None)
            fetch([(host_out["V_kept"], self._kept_view(self.V_kept))])
        cur.wait_stream(s_out)

    def device_status(self):
        """Status words of both workspaces (synchronises the device)."""
        torch.cuda.synchronize(self.device)
        out = {}
        if self.n_deep:
            out["evict"] = B.spindlekv_poll_status(self.ws_evict)
        if self.n_shallow:
            out["codebook"] = B.spindlekv_poll_status(self.ws_codebook)
            if hasattr(self, "_ws_codebook_v"):   # the V call of the last side-by-side run
                out["codebook_v"] = B.spindlekv_poll_status(self._ws_codebook_v)
        return out


class SpindleKVLiteralPass:
    """The composition of Section 3 as the paper writes it: every layer evicts under the pyramid of
    Eq. (5)(6) laid over all layers (Eq. (7)), then K and V CodeBooks are built from the tokens the layer
    kept (Algorithm 1), whose number differs from layer to layer.  ``cfg.n_shallow`` must be -1; all
    sequences have the same length.  ``K``, ``V``: ``[n_layers, B, H_kv, N, d]``; ``Q``:
    ``[n_layers, B, H_q, w, d]``.  No arithmetic happens here: buffers and call order only.
    """

    def __init__(self, cfg: B.Config, seq_lens: Sequence[int], dtype: torch.dtype, device="cuda",
                 keep_adjacency: bool = False):
        if cfg.n_shallow != -1:
            raise ValueError("SpindleKVLiteralPass needs cfg.n_shallow == -1")
        if len(set(int(x) for x in seq_lens)) != 1:
            raise ValueError("SpindleKVLiteralPass needs sequences of equal length")
        self.cfg = cfg
        self.device = torch.device(device)
        self.ev = SpindleKVPass(dataclasses.replace(cfg, n_shallow=0), seq_lens, dtype, device)
        self.mode, self.ratio, self.k_ctx_host = B.spindlekv_plan_layers(cfg, list(seq_lens))
        L, nB, H, d = cfg.n_layers, len(seq_lens), cfg.n_kv_heads, cfg.head_dim
        self.kept_host = (self.k_ctx_host + cfg.window).astype(np.int32)          # [L, B] tokens kept per head
        self.max_keep = int(self.kept_host.max())
        self.layer_lens = torch.from_numpy(np.ascontiguousarray(self.kept_host)).to(self.device)
        T = nB * self.max_keep
        self.cb_batch = B.Batch(L, nB, self.max_keep, T, None, self.layer_lens)
        nb = B.spindlekv_workspace_bytes(cfg, self.cb_batch, B.WS_CODEBOOK)
        self.ws_codebook = torch.empty(nb, dtype=torch.uint8, device=self.device)
        i32 = dict(dtype=torch.int32, device=self.device)
        self.cb: Dict[str, Dict[str, torch.Tensor]] = {}
        for g in ("K", "V"):
            self.cb[g] = {
                "mag": torch.zeros((L, H, T), dtype=torch.float32, device=self.device),
                "ref": torch.zeros((L, H, T), **i32),
                "centre_idx": torch.zeros((L, H, T), **i32),
                "n_entries": torch.zeros((L, nB, H), **i32),
                "C": torch.zeros((L, nB, H, self.max_keep, d), dtype=dtype, device=self.device),
            }
        self.adj = None
        if keep_adjacency:
            self.adj = torch.zeros((L * nB * H, self.max_keep, B.row_words(self.max_keep)), **i32)

    def _codebook(self, g: str, ws: torch.Tensor, stream) -> None:
        cfg = self.cfg
        kept = (self.ev.K_kept if g == "K" else self.ev.V_kept)[:, :, :, : self.max_keep]
        o = self.cb[g]
        B.spindlekv_codebook_shallow(cfg, self.cb_batch, B.desc_bhnd(kept), cfg.theta_k if g == "K" else cfg.theta_v,
                                     o["mag"], o["ref"], o["centre_idx"], o["n_entries"], ws, self.adj, stream)
        B.spindlekv_compact(self.cb_batch, cfg.n_kv_heads, cfg.head_dim, B.desc_bhnd(kept), o["centre_idx"],
                            o["n_entries"], B.desc_bhnd(o["C"]), o["mag"], None, stream)

    def run(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, which=("K", "V"), stream=None) -> None:
        self.ev.evict(K, V, Q, stream)
        if self.adj is None and tuple(which) == ("K", "V") and (stream is None or isinstance(stream, torch.cuda.Stream)):
            # the two CodeBook calls are independent: the V call runs on a side stream with a workspace of its own
            cur = stream if stream is not None else torch.cuda.current_stream(self.device)
            if not hasattr(self, "_side"):
                self._side = torch.cuda.Stream(self.device)
                self._ws_codebook_v = torch.empty_like(self.ws_codebook)
            ev = torch.cuda.Event()
            ev.record(cur)
            self._side.wait_event(ev)
            self._codebook("K", self.ws_codebook, cur)
            self._codebook("V", self._ws_codebook_v, self._side)
            cur.wait_stream(self._side)
            return
        for g in which:
            self._codebook(g, self.ws_codebook, stream)

    def entry_counts(self):
        """Host copies of the CodeBook sizes ``[L, B, H]`` for K and V (synchronises)."""
        return self.cb["K"]["n_entries"].cpu().numpy(), self.cb["V"]["n_entries"].cpu().numpy()

    def device_status(self):
        torch.cuda.synchronize(self.device)
        out = {"evict": B.spindlekv_poll_status(self.ev.ws_evict), "codebook": B.spindlekv_poll_status(self.ws_codebook)}
        if hasattr(self, "_ws_codebook_v"):
            out["codebook_v"] = B.spindlekv_poll_status(self._ws_codebook_v)
        return out


class SpindleKVRepeatPass:
    """The GQA "repeat" alternative of Section 3.3 inside the composition as written: the KV vectors of
    a group are taken once per query head, so every query head selects its own tokens (Eq. (2)(7) without
    the group mean of Eq. (3)); the K and V CodeBooks of a KV head are then built from the tokens all
    its query heads kept, listed one head after the other, where a token kept by several heads
    appears several times and collapses into one entry (cosine similarity 1).  ``cfg.n_shallow`` must
    be -1; equal-length sequences.  ``K``, ``V``: ``[L, B, H_kv, N, d]``; ``Q``: ``[L, B, H_q, w, d]``.
    One eviction call with ``per_query_head`` set serves all query heads.  Buffers and call order only.
    """

    def __init__(self, cfg: B.Config, seq_lens: Sequence[int], dtype: torch.dtype, device="cuda",
                 keep_adjacency: bool = False):
        if cfg.n_shallow != -1:
            raise ValueError("SpindleKVRepeatPass needs cfg.n_shallow == -1")
        if len(set(int(x) for x in seq_lens)) != 1:
            raise ValueError("SpindleKVRepeatPass needs sequences of equal length")
        self.cfg = cfg
        self.device = dev = torch.device(device)
        self.h_n = cfg.n_q_heads // cfg.n_kv_heads
        L, nB, H, Hq, d, N = cfg.n_layers, len(seq_lens), cfg.n_kv_heads, cfg.n_q_heads, cfg.head_dim, int(seq_lens[0])
        self.n_seqs, self.max_len = nB, N
        self.ecfg = dataclasses.replace(cfg, n_shallow=0, per_query_head=1)
        self.mode, self.ratio, self.k_ctx_host = B.spindlekv_plan_layers(cfg, list(seq_lens))
        self.k_ctx = torch.from_numpy(np.ascontiguousarray(self.k_ctx_host)).to(dev)
        self.ev_batch = B.Batch(L, nB, N, nB * N)
        i32 = dict(dtype=torch.int32, device=dev)
        self.keep_idx = torch.zeros((L, Hq, nB * N), **i32)              # per query head
        self.keep_cnt = torch.zeros((L, nB, Hq), **i32)
        self.scores = torch.zeros((L, Hq, nB * N), dtype=torch.float32, device=dev)
        self.ws_evict = torch.empty(B.spindlekv_workspace_bytes(self.ecfg, self.ev_batch, B.WS_EVICT), dtype=torch.uint8, device=dev)
        self.kept_host = (self.k_ctx_host + cfg.window).astype(np.int32)                     # per query head
        self.union_host = (self.h_n * self.kept_host).astype(np.int32)                       # per KV head
        self.max_union = int(self.union_host.max())
        self.layer_lens = torch.from_numpy(np.ascontiguousarray(self.union_host)).to(dev)
        T = nB * self.max_union
        self.union_idx = torch.zeros((L, H, T), **i32)
        self.union_cnt = torch.zeros((L, nB, H), **i32)
        self.cb_batch = B.Batch(L, nB, self.max_union, T, None, self.layer_lens)
        self.ws_codebook = torch.empty(B.spindlekv_workspace_bytes(cfg, self.cb_batch, B.WS_CODEBOOK), dtype=torch.uint8, device=dev)
        self.rep = {g: torch.zeros((L, nB, H, self.max_union, d), dtype=dtype, device=dev) for g in ("K", "V")}
        self.cb: Dict[str, Dict[str, torch.Tensor]] = {}
        for g in ("K", "V"):
            self.cb[g] = {
                "mag": torch.zeros((L, H, T), dtype=torch.float32, device=dev),
                "ref": torch.zeros((L, H, T), **i32),
                "centre_idx": torch.zeros((L, H, T), **i32),
                "n_entries": torch.zeros((L, nB, H), **i32),
                "C": torch.zeros((L, nB, H, self.max_union, d), dtype=dtype, device=dev),
            }
        self.adj = torch.zeros((L * nB * H, self.max_union, B.row_words(self.max_union)), **i32) if keep_adjacency else None

    def run(self, K: torch.Tensor, V: torch.Tensor, Q: torch.Tensor, which=("K", "V"), stream=None) -> None:
        cfg, H, d = self.cfg, self.cfg.n_kv_heads, self.cfg.head_dim
        B.spindlekv_evict_deep(self.ecfg, self.ev_batch, B.desc_bhnd(K), B.desc_bhnd(Q), self.k_ctx, self.keep_idx,
                               self.keep_cnt, self.scores, self.ws_evict, stream)
        # query head h_n*j + g is list g of KV head j: the per-query-head outputs are [L][H][h_n][...] as they stand
        L = cfg.n_layers
        B.spindlekv_union_lists(L, self.n_seqs, H, self.keep_idx.view(L, H, self.h_n, -1),
                                self.keep_cnt.view(L, self.n_seqs, H, self.h_n), self.max_len,
                                self.union_idx, self.union_cnt, self.max_union, stream, lists_inner=True)
        def codebook(g, ws, st):
            src, rep, o = (K if g == "K" else V), self.rep[g], self.cb[g]
            # rows of the union list, gathered from the KV head (the union list is laid out per max_union tokens,
            # the source per max_len tokens: two batches describe the two sides)
            self._gather(src, rep, st)
            B.spindlekv_codebook_shallow(cfg, self.cb_batch, B.desc_bhnd(rep), cfg.theta_k if g == "K" else cfg.theta_v,
                                         o["mag"], o["ref"], o["centre_idx"], o["n_entries"], ws, self.adj, st)
            B.spindlekv_compact(self.cb_batch, H, d, B.desc_bhnd(rep), o["centre_idx"], o["n_entries"],
                                B.desc_bhnd(o["C"]), o["mag"], None, st)

        if self.adj is None and tuple(which) == ("K", "V") and (stream is None or isinstance(stream, torch.cuda.Stream)):
            # the two CodeBook calls are independent: the V call runs on a side stream with a workspace of its own
            cur = stream if stream is not None else torch.cuda.current_stream(self.device)
            if not hasattr(self, "_side"):
                self._side = torch.cuda.Stream(self.device)
                self._ws_codebook_v = torch.empty_like(self.ws_codebook)
            ev = torch.cuda.Event()
            ev.record(cur)
            self._side.wait_event(ev)
            codebook("K", self.ws_codebook, cur)
            codebook("V", self._ws_codebook_v, self._side)
            cur.wait_stream(self._side)
            return
        for g in which:
            codebook(g, self.ws_codebook, stream)

    def _gather(self, src: torch.Tensor, rep: torch.Tensor, stream=None) -> None:
        # index rows are [L][H][B * max_union]; the compaction call addresses source rows through the batch's
        # max_len and index rows through total_len, so the batch carries the index layout and the source
        # tensor descriptor carries its own strides
        cfg = self.cfg
        B.spindlekv_compact(self.cb_batch, cfg.n_kv_heads, cfg.head_dim, B.desc_bhnd(src), self.union_idx, self.union_cnt,
                            B.desc_bhnd(rep), None, None, stream)

    def device_status(self):
        torch.cuda.synchronize(self.device)
        out = {"evict": B.spindlekv_poll_status(self.ws_evict), "codebook": B.spindlekv_poll_status(self.ws_codebook)}
        if hasattr(self, "_ws_codebook_v"):
            out["codebook_v"] = B.spindlekv_poll_status(self._ws_codebook_v)
        return out


class SpindleKVDecodeMerge:
    """Decode-time merging (Section 3.4, last paragraph) of ``t_new`` new tokens per (layer, sequence, head)
    into existing CodeBooks: match against the entries, build a CodeBook of the unmatched tokens, append
    it.  ``C``: ``[L, B, H, c_rows, d]`` with ``n_entries [L, B, H]`` (both updated in place); new tokens
    ``[L, B, H, t_new, d]``.  Results: ``ref_new``, ``mag_new`` ``[L, H, B * t_new]``.  Call order only.
    """

    def __init__(self, cfg: B.Config, n_layers: int, n_seqs: int, t_new: int, c_rows: int, dtype: torch.dtype,
                 device="cuda", keep_adjacency: bool = False):
        self.cfg, self.L, self.nB, self.t_new, self.c_rows = cfg, n_layers, n_seqs, t_new, c_rows
        self.device = dev = torch.device(device)
        H, d, T = cfg.n_kv_heads, cfg.head_dim, n_seqs * t_new
        i32 = dict(dtype=torch.int32, device=dev)
        self.batch = B.Batch(n_layers, n_seqs, t_new, T)
        self.ws_match = torch.empty(B.spindlekv_match_workspace_bytes(self.batch, H), dtype=torch.uint8, device=dev)
        self.ref_new = torch.zeros((n_layers, H, T), **i32)
        self.mag_new = torch.zeros((n_layers, H, T), dtype=torch.float32, device=dev)
        self.left_idx = torch.zeros((n_layers, H, T), **i32)
        self.left_cnt = torch.zeros((n_layers, n_seqs, H), **i32)
        self.left_rows = torch.zeros((n_layers, n_seqs, H, t_new, d), dtype=dtype, device=dev)
        self.left_batch = B.Batch(n_layers, n_seqs, t_new, T, None, self.left_cnt)   # lengths per head, on the device
        self.ws_codebook = torch.empty(B.spindlekv_workspace_bytes(cfg, self.left_batch, B.WS_CODEBOOK), dtype=torch.uint8, device=dev)
        self.left = {"mag": torch.zeros((n_layers, H, T), dtype=torch.float32, device=dev), "ref": torch.zeros((n_layers, H, T), **i32),
                     "centre_idx": torch.zeros((n_layers, H, T), **i32), "n_entries": torch.zeros((n_layers, n_seqs, H), **i32)}
        self.adj = torch.zeros((n_layers * n_seqs * H, t_new, B.row_words(t_new)), **i32) if keep_adjacency else None

    def run(self, G_new: torch.Tensor, C: torch.Tensor, n_entries: torch.Tensor, theta: float, stream=None) -> None:
        cfg, H, d = self.cfg, self.cfg.n_kv_heads, self.cfg.head_dim
        gd, cd, ld = B.desc_bhnd(G_new), B.desc_bhnd(C), B.desc_bhnd(self.left_rows)
        B.spindlekv_codebook_match(self.batch, H, d, gd, cd, n_entries, self.c_rows, theta, self.mag_new, self.ref_new,
                                   self.left_idx, self.left_cnt, self.ws_match, stream)
        B.spindlekv_compact(self.batch, H, d, gd, self.left_idx, self.left_cnt, ld, None, None, stream)
        o = self.left
        B.spindlekv_codebook_shallow(cfg, self.left_batch, ld, theta, o["mag"], o["ref"], o["centre_idx"], o["n_entries"],
                                     self.ws_codebook, self.adj, stream)
        B.spindlekv_codebook_append(self.batch, H, d, ld, o["mag"], o["ref"], o["centre_idx"], o["n_entries"],
                                    self.left_idx, self.left_cnt, cd, self.c_rows, n_entries, self.ref_new, stream)


class SpindleKVDecodeAttention:
    """Buffers for ``spindlekv_decode_attend``: the table of rotary cosines and sines, the scratch of the split
    pass and the output ``[L, B, H_q, d]`` (fp32).  ``batch`` describes the cached tokens.  Call order only."""

    def __init__(self, batch: B.Batch, n_q_heads: int, n_kv_heads: int, head_dim: int, n_positions: int,
                 rope_base: float = 10000.0, device="cuda"):
        self.batch, self.Hq, self.Hkv, self.d = batch, n_q_heads, n_kv_heads, head_dim
        dev = torch.device(device)
        self.table = torch.empty((n_positions, head_dim // 2, 2), dtype=torch.float32, device=dev)
        B.spindlekv_rope_table(head_dim, n_positions, rope_base, self.table)
        self.ws = torch.empty(B.spindlekv_decode_workspace_bytes(batch, n_q_heads, n_kv_heads, head_dim), dtype=torch.uint8, device=dev)
        self.out = torch.zeros((batch.n_layers, batch.n_seqs, n_q_heads, head_dim), dtype=torch.float32, device=dev)

    def run(self, q: torch.Tensor, pos_q: torch.Tensor, cb_k: Dict[str, torch.Tensor], cb_v: Dict[str, torch.Tensor],
            positions: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
        """``q``: ``[L, B, H_q, 1, d]`` pre-RoPE queries; ``cb_k`` / ``cb_v``: the ``C``, ``ref``, ``mag`` a CodeBook pass left."""
        B.spindlekv_decode_attend(self.batch, self.Hq, self.Hkv, self.d, B.desc_bhnd(q), pos_q, B.desc_bhnd(cb_k["C"]),
                                  cb_k["ref"], cb_k["mag"], B.desc_bhnd(cb_v["C"]), cb_v["ref"], cb_v["mag"], positions,
                                  self.table, self.out, self.ws, stream)
        return self.out
