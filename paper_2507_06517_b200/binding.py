"""Thin ctypes binding of ``libspindlekv.so``: same names as the C ABI, argument marshalling only.

Every step of the reduction pass runs in the library's CUDA kernels; torch is used for device
memory and streams.  Loading fails loudly when the library is missing and cannot be built.
"""
from __future__ import annotations

import ctypes as C
import dataclasses
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

OK, INVALID_ARG, BUDGET, WORKSPACE_TOO_SMALL, CAPACITY, UNSUPPORTED, CUDA_ERROR, TIMEOUT = range(8)
F32, BF16 = 0, 1
MODE_EVICT, MODE_CODEBOOK = 1, 2
WS_EVICT, WS_CODEBOOK = 0, 1
KERNEL_CLASSES = ("window_score", "topk", "norms", "similarity", "degree", "greedy", "finalise", "gather",
                  "similarity_fallback", "decode")


class SpindleKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.spindlekv_status_string(status).decode()} (status {status})")


class _Tensor(C.Structure):
    _fields_ = [("ptr", C.c_void_p), ("dtype", C.c_int32), ("stride_layer", C.c_int64),
                ("stride_seq", C.c_int64), ("stride_head", C.c_int64), ("stride_tok", C.c_int64)]


class _Config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("window", C.c_int32), ("n_shallow", C.c_int32),
                ("reserve_ratio", C.c_double), ("budget_tokens", C.c_double), ("beta", C.c_double),
                ("theta_k", C.c_float), ("theta_v", C.c_float), ("score_norm", C.c_int32),
                ("per_query_head", C.c_int32)]


class _Batch(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_seqs", C.c_int32), ("max_len", C.c_int32),
                ("total_len", C.c_int32), ("cu_seqlens", C.c_void_p), ("layer_lens", C.c_void_p), ("layer_lens_heads", C.c_int32)]


def _load() -> C.CDLL:
    path = _build.LIB
    if not os.path.exists(path):
        path = _build.build()
    lib = C.CDLL(path)
    lib.spindlekv_status_string.restype = C.c_char_p
    lib.spindlekv_status_string.argtypes = [C.c_int32]
    lib.spindlekv_plan_layers.restype = C.c_int32
    lib.spindlekv_plan_layers.argtypes = [C.POINTER(_Config), C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spindlekv_reserve_ratio.restype = C.c_int32
    lib.spindlekv_reserve_ratio.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spindlekv_workspace_bytes.restype = C.c_size_t
    lib.spindlekv_workspace_bytes.argtypes = [C.POINTER(_Config), C.POINTER(_Batch), C.c_int32]
    lib.spindlekv_evict_deep.restype = C.c_int32
    lib.spindlekv_evict_deep.argtypes = [C.POINTER(_Config), C.POINTER(_Batch), _Tensor, _Tensor, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.spindlekv_evict_deep_noalloc.restype = C.c_int32
    lib.spindlekv_evict_deep_noalloc.argtypes = [C.POINTER(_Config), C.POINTER(_Batch), _Tensor, _Tensor, C.c_void_p,
                                                 C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spindlekv_codebook_shallow.restype = C.c_int32
    lib.spindlekv_codebook_shallow.argtypes = [C.POINTER(_Config), C.POINTER(_Batch), _Tensor, C.c_float,
                                               C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_size_t, C.c_void_p]
    lib.spindlekv_compact.restype = C.c_int32
    lib.spindlekv_compact.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, _Tensor, C.c_void_p, C.c_void_p,
                                      C.c_void_p, _Tensor, C.c_void_p, C.c_void_p]
    lib.spindlekv_union_lists.restype = C.c_int32
    lib.spindlekv_union_lists.argtypes = [C.c_int32] * 7 + [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p,
                                                            C.c_void_p, C.c_void_p]
    lib.spindlekv_match_workspace_bytes.restype = C.c_size_t
    lib.spindlekv_match_workspace_bytes.argtypes = [C.POINTER(_Batch), C.c_int32]
    lib.spindlekv_codebook_match.restype = C.c_int32
    lib.spindlekv_codebook_match.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, _Tensor, _Tensor, C.c_void_p, C.c_int32,
                                             C.c_float, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                             C.c_size_t, C.c_void_p]
    lib.spindlekv_codebook_append.restype = C.c_int32
    lib.spindlekv_codebook_append.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, _Tensor] + [C.c_void_p] * 6 + \
                                             [_Tensor, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spindlekv_reconstruct.restype = C.c_int32
    lib.spindlekv_reconstruct.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, _Tensor, C.c_void_p, C.c_void_p,
                                          _Tensor, C.c_void_p]
    lib.spindlekv_rope_table_bytes.restype = C.c_size_t
    lib.spindlekv_rope_table_bytes.argtypes = [C.c_int32, C.c_int32]
    lib.spindlekv_rope_table.restype = C.c_int32
    lib.spindlekv_rope_table.argtypes = [C.c_int32, C.c_int32, C.c_double, C.c_void_p, C.c_void_p]
    lib.spindlekv_decode_workspace_bytes.restype = C.c_size_t
    lib.spindlekv_decode_workspace_bytes.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, C.c_int32]
    lib.spindlekv_decode_attend.restype = C.c_int32
    lib.spindlekv_decode_attend.argtypes = [C.POINTER(_Batch), C.c_int32, C.c_int32, C.c_int32, _Tensor, C.c_void_p,
                                            _Tensor, C.c_void_p, C.c_void_p, _Tensor, C.c_void_p, C.c_void_p,
                                            C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
    lib.spindlekv_poll_status.restype = C.c_int32
    lib.spindlekv_poll_status.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
    lib.spindlekv_set_tuning.restype = C.c_int32
    lib.spindlekv_set_tuning.argtypes = [C.c_int32, C.c_int64]
    lib.spindlekv_get_tuning.restype = C.c_int64
    lib.spindlekv_get_tuning.argtypes = [C.c_int32]
    lib.spindlekv_selftest_mbarrier_timeout.restype = C.c_int32
    lib.spindlekv_selftest_mbarrier_timeout.argtypes = [C.c_void_p, C.c_int64, C.c_void_p]
    lib.spindlekv_launch_count.restype = C.c_int64
    lib.spindlekv_launch_count.argtypes = [C.c_int32]
    lib.spindlekv_timing_enable.restype = None
    lib.spindlekv_timing_enable.argtypes = [C.c_int32]
    lib.spindlekv_timing_read.restype = C.c_int32
    lib.spindlekv_timing_read.argtypes = [C.c_int32, C.c_void_p, C.c_void_p]
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB


@dataclasses.dataclass
class Config:
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    window: int
    n_shallow: int
    reserve_ratio: float = -1.0
    budget_tokens: float = -1.0
    beta: float = 0.05
    theta_k: float = 0.98
    theta_v: float = 0.95
    score_norm: int = 0
    per_query_head: int = 0

    def c(self) -> _Config:
        return _Config(self.n_layers, self.n_q_heads, self.n_kv_heads, self.head_dim, self.window, self.n_shallow,
                       self.reserve_ratio, self.budget_tokens, self.beta, self.theta_k, self.theta_v, self.score_norm,
                       self.per_query_head)


@dataclasses.dataclass
class Batch:
    n_layers: int
    n_seqs: int
    max_len: int
    total_len: int
    cu_seqlens: Optional[torch.Tensor] = None  # device int32 [B+1]
    layer_lens: Optional[torch.Tensor] = None  # device int32 [n_layers, B] or [n_layers, B, H] (not with cu_seqlens)

    def c(self) -> _Batch:
        ptr = self.cu_seqlens.data_ptr() if self.cu_seqlens is not None else None
        ll = self.layer_lens.data_ptr() if self.layer_lens is not None else None
        heads = self.layer_lens.shape[2] if self.layer_lens is not None and self.layer_lens.dim() == 3 else 0
        return _Batch(self.n_layers, self.n_seqs, self.max_len, self.total_len, ptr, ll, heads)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def desc_bhnd(t: torch.Tensor) -> _Tensor:
    """Descriptor of a ``[layers, B, heads, rows, d]`` tensor (any strides, ``d`` contiguous)."""
    assert t.dim() == 5 and t.stride(4) == 1
    return _Tensor(t.data_ptr(), _dtype_code(t), t.stride(0), t.stride(1), t.stride(2), t.stride(3))


def desc_thd(t: torch.Tensor) -> _Tensor:
    """Descriptor of a packed ``[layers, total_tokens, heads, d]`` tensor (used with cu_seqlens)."""
    assert t.dim() == 4 and t.stride(3) == 1
    return _Tensor(t.data_ptr(), _dtype_code(t), t.stride(0), 0, t.stride(2), t.stride(1))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(status: int, where: str) -> None:
    if status != OK:
        raise SpindleKVError(status, where)


def spindlekv_plan_layers(cfg: Config, seq_lens: Sequence[int]):
    """Host planner: returns ``(layer_mode[m], r_c_layer[m, B], k_ctx[m, B])`` as numpy arrays."""
    B = len(seq_lens)
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    mode = np.zeros(cfg.n_layers, dtype=np.int32)
    ratio = np.zeros((cfg.n_layers, B), dtype=np.float64)
    k_ctx = np.zeros((cfg.n_layers, B), dtype=np.int32)
    cc = cfg.c()
    st = _lib.spindlekv_plan_layers(C.byref(cc), B, lens.ctypes.data, mode.ctypes.data, ratio.ctypes.data,
                                    k_ctx.ctypes.data)
    _check(st, "spindlekv_plan_layers")
    return mode, ratio, k_ctx


def spindlekv_reserve_ratio(seq_len: int, kept: int, entries_k: Sequence[int], entries_v: Sequence[int]):
    """Eq. (15)'s ``(r1, r2)`` of one layer from the CodeBook sizes per head (host arithmetic in the library)."""
    ek = np.ascontiguousarray(entries_k, dtype=np.int32)
    ev = np.ascontiguousarray(entries_v, dtype=np.int32)
    r1, r2 = C.c_double(0.0), C.c_double(0.0)
    st = _lib.spindlekv_reserve_ratio(int(ek.shape[0]), seq_len, kept, ek.ctypes.data, ev.ctypes.data, C.byref(r1), C.byref(r2))
    _check(st, "spindlekv_reserve_ratio")
    return float(r1.value), float(r2.value)


def spindlekv_workspace_bytes(cfg: Config, batch: Batch, which: int) -> int:
    cc, bb = cfg.c(), batch.c()
    return int(_lib.spindlekv_workspace_bytes(C.byref(cc), C.byref(bb), which))


def spindlekv_evict_deep(cfg: Config, batch: Batch, K: _Tensor, Qwin: _Tensor, k_ctx: torch.Tensor,
                         keep_idx: torch.Tensor, keep_cnt: torch.Tensor, scores: torch.Tensor,
                         ws: torch.Tensor, stream=None) -> None:
    cc, bb = cfg.c(), batch.c()
    st = _lib.spindlekv_evict_deep(C.byref(cc), C.byref(bb), K, Qwin, _ptr(k_ctx), _ptr(keep_idx), _ptr(keep_cnt),
                                   _ptr(scores), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "spindlekv_evict_deep")


NOALLOC_SCRATCH_BYTES = 8 * 1024 * 1024


def spindlekv_evict_deep_noalloc(cfg: Config, batch: Batch, K: _Tensor, Qwin: _Tensor, k_ctx: torch.Tensor,
                                 keep_idx: torch.Tensor, keep_cnt: torch.Tensor, scores: torch.Tensor,
                                 stream=None) -> None:
    """Eviction without a workspace, for callers that may not allocate device memory (a server whose
    pool owns the GPU, code under another allocator's lock): the kernels' scratch is a fixed 8 MiB
    array inside the library.  Raises ``WORKSPACE_TOO_SMALL`` when the call would use more than that
    (never on the tensor-core path, which keeps only a status block there).  Calls share the array, so
    calls that could overlap on the GPU must be ordered by the caller; ``spindlekv_poll_status(None)``
    reads the device status word of the last call."""
    cc, bb = cfg.c(), batch.c()
    st = _lib.spindlekv_evict_deep_noalloc(C.byref(cc), C.byref(bb), K, Qwin, _ptr(k_ctx), _ptr(keep_idx),
                                           _ptr(keep_cnt), _ptr(scores), _stream(stream))
    _check(st, "spindlekv_evict_deep_noalloc")


def spindlekv_codebook_shallow(cfg: Config, batch: Batch, Gamma: _Tensor, theta: float, mag: torch.Tensor,
                               ref: torch.Tensor, centre_idx: torch.Tensor, n_entries: torch.Tensor,
                               ws: torch.Tensor, adj_bits: Optional[torch.Tensor] = None, stream=None) -> None:
    cc, bb = cfg.c(), batch.c()
    st = _lib.spindlekv_codebook_shallow(C.byref(cc), C.byref(bb), Gamma, theta, _ptr(mag), _ptr(ref),
                                         _ptr(centre_idx), _ptr(n_entries), _ptr(adj_bits), _ptr(ws),
                                         ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "spindlekv_codebook_shallow")


def spindlekv_compact(batch: Batch, n_heads: int, head_dim: int, src: _Tensor, idx: torch.Tensor,
                      cnt: torch.Tensor, dst: _Tensor, divide_by: Optional[torch.Tensor] = None,
                      dst_cu_seqlens: Optional[torch.Tensor] = None, stream=None) -> None:
    bb = batch.c()
    st = _lib.spindlekv_compact(C.byref(bb), n_heads, head_dim, src, _ptr(idx), _ptr(cnt), _ptr(divide_by), dst,
                                _ptr(dst_cu_seqlens), _stream(stream))
    _check(st, "spindlekv_compact")


def spindlekv_union_lists(n_layers: int, n_seqs: int, n_heads: int, idx_in: torch.Tensor, cnt_in: torch.Tensor,
                          seq_in: int, idx_out: torch.Tensor, cnt_out: torch.Tensor, seq_out: int, stream=None,
                          lists_inner: bool = False) -> None:
    """``idx_in [n_lists, L, H, t_in]``, ``cnt_in [n_lists, L, B, H]`` (``lists_inner``: ``[L, H, n_lists, t_in]`` and
    ``[L, B, H, n_lists]``) -> ``idx_out [L, H, t_out]``, ``cnt_out [L, B, H]``."""
    n_lists = idx_in.shape[2] if lists_inner else idx_in.shape[0]
    st = _lib.spindlekv_union_lists(n_layers, n_seqs, n_heads, n_lists, 1 if lists_inner else 0, idx_in.shape[-1], seq_in,
                                    _ptr(idx_in), _ptr(cnt_in), idx_out.shape[-1], seq_out, _ptr(idx_out), _ptr(cnt_out),
                                    _stream(stream))
    _check(st, "spindlekv_union_lists")


def spindlekv_match_workspace_bytes(batch: Batch, n_heads: int) -> int:
    bb = batch.c()
    return int(_lib.spindlekv_match_workspace_bytes(C.byref(bb), n_heads))


def spindlekv_codebook_match(batch: Batch, n_heads: int, head_dim: int, G_new: _Tensor, Cb: _Tensor, n_entries: torch.Tensor,
                             c_rows: int, theta: float, mag_new: torch.Tensor, ref_new: torch.Tensor,
                             left_idx: torch.Tensor, left_cnt: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    bb = batch.c()
    st = _lib.spindlekv_codebook_match(C.byref(bb), n_heads, head_dim, G_new, Cb, _ptr(n_entries), c_rows, theta,
                                       _ptr(mag_new), _ptr(ref_new), _ptr(left_idx), _ptr(left_cnt), _ptr(ws),
                                       ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "spindlekv_codebook_match")


def spindlekv_codebook_append(batch: Batch, n_heads: int, head_dim: int, G_left: _Tensor, mag_left: torch.Tensor,
                              ref_left: torch.Tensor, centre_left: torch.Tensor, n_left_entries: torch.Tensor,
                              left_idx: torch.Tensor, left_cnt: torch.Tensor, Cb: _Tensor, c_rows: int,
                              n_entries: torch.Tensor, ref_new: torch.Tensor, stream=None) -> None:
    bb = batch.c()
    st = _lib.spindlekv_codebook_append(C.byref(bb), n_heads, head_dim, G_left, _ptr(mag_left), _ptr(ref_left),
                                        _ptr(centre_left), _ptr(n_left_entries), _ptr(left_idx), _ptr(left_cnt), Cb,
                                        c_rows, _ptr(n_entries), _ptr(ref_new), _stream(stream))
    _check(st, "spindlekv_codebook_append")


def spindlekv_reconstruct(batch: Batch, n_heads: int, head_dim: int, Cb: _Tensor, ref: torch.Tensor,
                          mag: torch.Tensor, dst: _Tensor, stream=None) -> None:
    bb = batch.c()
    st = _lib.spindlekv_reconstruct(C.byref(bb), n_heads, head_dim, Cb, _ptr(ref), _ptr(mag), dst, _stream(stream))
    _check(st, "spindlekv_reconstruct")


def spindlekv_rope_table_bytes(head_dim: int, n_positions: int) -> int:
    return int(_lib.spindlekv_rope_table_bytes(head_dim, n_positions))


def spindlekv_rope_table(head_dim: int, n_positions: int, base: float, table: torch.Tensor, stream=None) -> None:
    """Fills ``table`` (``[n_positions, head_dim/2, 2]`` fp32: cos, sin) for ``spindlekv_decode_attend``."""
    _check(_lib.spindlekv_rope_table(head_dim, n_positions, base, _ptr(table), _stream(stream)), "spindlekv_rope_table")


def spindlekv_decode_workspace_bytes(batch: Batch, n_q_heads: int, n_kv_heads: int, head_dim: int) -> int:
    bb = batch.c()
    return int(_lib.spindlekv_decode_workspace_bytes(C.byref(bb), n_q_heads, n_kv_heads, head_dim))


def spindlekv_decode_attend(batch: Batch, n_q_heads: int, n_kv_heads: int, head_dim: int, q: _Tensor, pos_q: torch.Tensor,
                            C_K: _Tensor, ref_K: torch.Tensor, mag_K: torch.Tensor, C_V: _Tensor, ref_V: torch.Tensor,
                            mag_V: torch.Tensor, positions: Optional[torch.Tensor], rope_table: torch.Tensor,
                            out: torch.Tensor, ws: torch.Tensor, stream=None) -> None:
    """One decode step over the replaced cache; ``rope_table`` is ``[n_positions, head_dim/2, 2]`` fp32."""
    bb = batch.c()
    st = _lib.spindlekv_decode_attend(C.byref(bb), n_q_heads, n_kv_heads, head_dim, q, _ptr(pos_q), C_K, _ptr(ref_K),
                                      _ptr(mag_K), C_V, _ptr(ref_V), _ptr(mag_V), _ptr(positions), _ptr(rope_table),
                                      rope_table.shape[0], _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream))
    _check(st, "spindlekv_decode_attend")


def spindlekv_poll_status(ws: Optional[torch.Tensor]):
    """Device status word of a workspace and ``[greedy rounds, live tokens left, units done as a bit matrix, list entries built from records]``.  ``None`` reads the
    built-in scratch of ``spindlekv_evict_deep_noalloc`` on the current device."""
    status = C.c_int32(0)
    detail = (C.c_int32 * 4)()
    st = _lib.spindlekv_poll_status(_ptr(ws), C.byref(status), detail)
    _check(st, "spindlekv_poll_status")
    return int(status.value), [int(x) for x in detail]


TUNE_RECORDS_PER_TILE, TUNE_GREEDY_ROUND_CAP, TUNE_MBAR_WAIT_CYCLES, TUNE_SIM_BLOCK_PAIRS = range(4)


def spindlekv_set_tuning(key: int, value: int) -> None:
    """Test hook: tightens one of the library's limits (``value < 0`` restores the default)."""
    _check(_lib.spindlekv_set_tuning(key, value), "spindlekv_set_tuning")


def spindlekv_get_tuning(key: int) -> int:
    return int(_lib.spindlekv_get_tuning(key))


def spindlekv_selftest_mbarrier_timeout(ws: torch.Tensor, limit: int, stream=None) -> None:
    """Test hook: a shared-memory barrier nobody arrives on; must leave TIMEOUT in the status word of ``ws``."""
    _check(_lib.spindlekv_selftest_mbarrier_timeout(_ptr(ws), limit, _stream(stream)), "spindlekv_selftest_mbarrier_timeout")


def spindlekv_launch_count(reset: bool = False) -> int:
    return int(_lib.spindlekv_launch_count(1 if reset else 0))


def spindlekv_timing_enable(on: bool) -> None:
    _lib.spindlekv_timing_enable(1 if on else 0)


def spindlekv_timing_read():
    """``{kernel class: (milliseconds, launches)}`` since timing was enabled."""
    out = {}
    for i, name in enumerate(KERNEL_CLASSES):
        ms, n = C.c_double(0.0), C.c_int64(0)
        _check(_lib.spindlekv_timing_read(i, C.byref(ms), C.byref(n)), "spindlekv_timing_read")
        out[name] = (float(ms.value), int(n.value))
    return out


def row_words(max_len: int) -> int:
    """Words per row of the adjacency bit matrix."""
    return 4 * ((max_len + 127) // 128)
