"""Seeded synthetic inputs for the SpindleKV prefill reduction pass.

This module only draws random tensors; it holds none of the method's
arithmetic (no scores, no similarities, no budgets).  Both the CPU checker and
the CUDA path are fed from here so that they read the very same bytes.

Recipe (per layer and KV head, every draw from numpy's PCG64 seeded by
``[seed, layer, sequence, head, stream]``):

* ``n_clusters`` centroids for keys and, independently, for values, each
  ``N(0, I_d)``; a noise level ``sigma`` per cluster (a constant, or uniform in
  ``[lo, hi]``); a cluster id per token, uniform.
* ``k_t = c^K[z_t] + sigma[z_t] * eps``, ``v_t = c^V[z_t] + sigma[z_t] * eps'``.
* the first ``n_sink`` tokens are scaled by 5 ("sink" tokens with a large norm).
* window queries, one ``[w, d]`` block per query head:
  ``gauss``   : ``N(0, I_d)``;
  ``recency`` : ``eps + 2 * unit(k_t') + unit(k_s)`` with ``t'`` drawn with
  probability proportional to ``exp(-(l - 1 - t) / (l / 8))`` and ``s`` a
  uniformly drawn sink token, both taken from the KV head the query head reads.
* values are rounded once to the storage type (fp32 or bf16, round to nearest
  even) and returned as float32 arrays that hold exactly those values.

These tensors stand in for the long prompts (about 5k to 15k tokens) of the
evaluation suites the method was published with; none of those suites' items
are used or needed.
"""
from __future__ import annotations

import dataclasses
from typing import Optional, Sequence, Tuple, Union

import numpy as np

_STREAM_CENTROID_K = 0
_STREAM_CENTROID_V = 1
_STREAM_SIGMA = 2
_STREAM_ASSIGN = 3
_STREAM_NOISE_K = 4
_STREAM_NOISE_V = 5
_STREAM_QUERY = 6
_STREAM_LENGTHS = 7

SINK_SCALE = 5.0


@dataclasses.dataclass(frozen=True)
class Workload:
    """Shape and distribution of one synthetic KV-cache reduction problem."""

    name: str
    n_layers: int
    n_shallow: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    dtype: str  # "f32" or "bf16"
    window: int
    seq_lens: Tuple[int, ...]
    n_clusters: int
    sigma: Union[float, Tuple[float, float]]
    n_sink: int
    query: str  # "gauss" or "recency"
    budget_tokens: Optional[float] = None  # tokens kept per head, window included
    budget_frac: Optional[float] = None  # same, as a fraction of each length
    theta_k: float = 0.98
    theta_v: float = 0.95
    beta: float = 0.05
    seed: int = 20250706

    @property
    def batch(self) -> int:
        return len(self.seq_lens)

    @property
    def total_tokens(self) -> int:
        return int(sum(self.seq_lens))

    @property
    def max_len(self) -> int:
        return int(max(self.seq_lens))

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def packed(self) -> bool:
        return len(set(self.seq_lens)) > 1

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _varlen_lengths(seed: int, batch: int, lo: int, hi: int) -> Tuple[int, ...]:
    rng = np.random.Generator(np.random.PCG64([seed, _STREAM_LENGTHS]))
    return tuple(int(x) for x in rng.integers(lo, hi + 1, size=batch))


def workload(name: str, **overrides) -> Workload:
    """The five named configurations (tiny fp32 case, 8B shape at 4k and 16k,
    a packed variable-length batch, and a 70B shape at 32k)."""
    seed = overrides.get("seed", 20250706)
    if name == "C1":
        wl = Workload("C1", 2, 1, 4, 2, 64, "f32", 32, (512,), 32, 0.1, 4, "gauss",
                      budget_tokens=128.0, seed=seed)
    elif name == "C2":
        wl = Workload("C2", 32, 16, 32, 8, 128, "bf16", 32, (4096,), 256, 0.2, 8, "recency",
                      budget_tokens=512.0, seed=seed)
    elif name == "C3":
        wl = Workload("C3", 32, 16, 32, 8, 128, "bf16", 32, (16384,), 1024, (0.05, 0.4), 8,
                      "recency", budget_tokens=1024.0, seed=seed)
    elif name == "C4":
        wl = Workload("C4", 32, 16, 32, 8, 128, "bf16", 64, _varlen_lengths(seed, 8, 2048, 16384),
                      1024, (0.05, 0.4), 8, "recency", budget_frac=0.10, seed=seed)
    elif name == "C5":
        wl = Workload("C5", 80, 40, 64, 8, 128, "bf16", 32, (32768,), 4096, 0.25, 16, "recency",
                      budget_tokens=2048.0, seed=seed)
    else:
        raise KeyError(name)
    return wl.replace(**overrides) if overrides else wl


def round_to_dtype(x: np.ndarray, dtype: str) -> np.ndarray:
    """Round float32 values to the storage type and return them as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "f32":
        return x
    if dtype != "bf16":
        raise ValueError(dtype)
    u = x.view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    r = (u + bias) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def _rng(wl: Workload, layer: int, seq: int, head: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([wl.seed, layer, seq, head, stream]))


def unit_kv(wl: Workload, layer: int, seq: int, head: int) -> Tuple[np.ndarray, np.ndarray]:
    """Keys and values ``[l, d]`` of one (layer, sequence, KV head)."""
    l, d = wl.seq_lens[seq], wl.head_dim
    ck = _rng(wl, layer, seq, head, _STREAM_CENTROID_K).standard_normal((wl.n_clusters, d), dtype=np.float32)
    cv = _rng(wl, layer, seq, head, _STREAM_CENTROID_V).standard_normal((wl.n_clusters, d), dtype=np.float32)
    rs = _rng(wl, layer, seq, head, _STREAM_SIGMA)
    if isinstance(wl.sigma, tuple):
        sig = rs.uniform(wl.sigma[0], wl.sigma[1], size=wl.n_clusters).astype(np.float32)
    else:
        sig = np.full(wl.n_clusters, wl.sigma, dtype=np.float32)
    z = _rng(wl, layer, seq, head, _STREAM_ASSIGN).integers(0, wl.n_clusters, size=l)
    k = _rng(wl, layer, seq, head, _STREAM_NOISE_K).standard_normal((l, d), dtype=np.float32)
    v = _rng(wl, layer, seq, head, _STREAM_NOISE_V).standard_normal((l, d), dtype=np.float32)
    s = sig[z][:, None]
    k *= s
    v *= s
    k += ck[z]
    v += cv[z]
    ns = min(wl.n_sink, l)
    k[:ns] *= SINK_SCALE
    v[:ns] *= SINK_SCALE
    return round_to_dtype(k, wl.dtype), round_to_dtype(v, wl.dtype)


def window_queries(wl: Workload, layer: int, seq: int, k_heads: Sequence[np.ndarray]) -> np.ndarray:
    """Observation-window queries ``[H_q, w, d]`` of one (layer, sequence).

    ``k_heads[j]`` is the ``[l, d]`` key array of KV head ``j`` (used only by
    the ``recency`` recipe, to point the queries at recent tokens and sinks).
    """
    l, d, w = wl.seq_lens[seq], wl.head_dim, wl.window
    out = np.empty((wl.n_q_heads, w, d), dtype=np.float32)
    for i in range(wl.n_q_heads):
        rng = _rng(wl, layer, seq, i, _STREAM_QUERY)
        q = rng.standard_normal((w, d), dtype=np.float32)
        if wl.query == "recency":
            k = k_heads[i // wl.group]
            age = (l - 1 - np.arange(l, dtype=np.float64)) / (l / 8.0)
            p = np.exp(-age)
            p /= p.sum()
            t = rng.choice(l, size=w, p=p)
            s = rng.integers(0, max(1, min(wl.n_sink, l)), size=w)
            kt = k[t].astype(np.float32)
            ks = k[s].astype(np.float32)
            kt /= np.maximum(np.linalg.norm(kt, axis=1, keepdims=True), 1e-20)
            ks /= np.maximum(np.linalg.norm(ks, axis=1, keepdims=True), 1e-20)
            q += 2.0 * kt + ks
        elif wl.query != "gauss":
            raise ValueError(wl.query)
        out[i] = q
    return round_to_dtype(out, wl.dtype)


def layer_arrays(wl: Workload, layer: int, need_q: bool = True, layout: str = "auto"):
    """All sequences and heads of one layer as float32 numpy arrays.

    Returns ``(K, V, Q)``.  ``layout="bhnd"``: ``K, V`` are ``[B, H_kv, N, d]``
    (all sequences of equal length).  ``layout="thd"``: ``[total_tokens, H_kv,
    d]``, sequences packed back to back, token-major.  ``"auto"`` picks
    ``"thd"`` for ragged batches and ``"bhnd"`` otherwise.  ``Q`` is
    ``[B, H_q, w, d]`` (``None`` when ``need_q`` is false).
    """
    if layout == "auto":
        layout = "thd" if wl.packed else "bhnd"
    tot, hk, d = wl.total_tokens, wl.n_kv_heads, wl.head_dim
    if layout == "thd":
        K = np.empty((tot, hk, d), dtype=np.float32)
        V = np.empty((tot, hk, d), dtype=np.float32)
    elif layout == "bhnd":
        if wl.packed:
            raise ValueError("bhnd layout needs equal sequence lengths")
        K = np.empty((wl.batch, hk, wl.max_len, d), dtype=np.float32)
        V = np.empty((wl.batch, hk, wl.max_len, d), dtype=np.float32)
    else:
        raise ValueError(layout)
    Q = np.empty((wl.batch, wl.n_q_heads, wl.window, d), dtype=np.float32) if need_q else None
    off = 0
    for s, l in enumerate(wl.seq_lens):
        heads = []
        for j in range(hk):
            k, v = unit_kv(wl, layer, s, j)
            if layout == "thd":
                K[off:off + l, j] = k
                V[off:off + l, j] = v
            else:
                K[s, j] = k
                V[s, j] = v
            heads.append(k)
        if need_q:
            Q[s] = window_queries(wl, layer, s, heads)
        off += l
    return K, V, Q


def cu_seqlens(wl: Workload) -> np.ndarray:
    """Prefix sums of the sequence lengths, ``[B + 1]`` int32."""
    return np.concatenate([[0], np.cumsum(wl.seq_lens)]).astype(np.int32)
