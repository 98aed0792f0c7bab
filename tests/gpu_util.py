"""Helpers shared by the GPU parity tests: build device tensors from the seeded generator and
compare library outputs with the CPU checker under the stated tolerances."""
from __future__ import annotations

import numpy as np
import torch

from oracle import spindlekv_oracle as O
from paper_2507_06517_b200 import binding as B
from paper_2507_06517_b200 import synth
from paper_2507_06517_b200.pipeline import SpindleKVPass

REL_MARGIN = 1e-4  # decisions closer than this (relative) to the k-th score / the threshold may differ


def torch_dtype(wl):
    return torch.float32 if wl.dtype == "f32" else torch.bfloat16


def to_device(x: np.ndarray, wl) -> torch.Tensor:
    return torch.from_numpy(x).to(torch_dtype(wl)).cuda()


def make_config(wl, **kw) -> B.Config:
    args = dict(n_layers=wl.n_layers, n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                window=wl.window, n_shallow=wl.n_shallow, beta=wl.beta, theta_k=wl.theta_k, theta_v=wl.theta_v)
    if wl.budget_tokens is not None:
        args["budget_tokens"] = wl.budget_tokens
    else:
        args["reserve_ratio"] = wl.budget_frac
    args.update(kw)
    return B.Config(**args)


def generate(wl, layers=None):
    """Host arrays for the listed layers: dict layer -> (K, V, Q) float32 numpy (Q None for shallow)."""
    layers = range(wl.n_layers) if layers is None else layers
    return {lam: synth.layer_arrays(wl, lam, need_q=lam >= wl.n_shallow) for lam in layers}


def stack_layers(wl, host, layers, what):
    idx = {"K": 0, "V": 1, "Q": 2}[what]
    return to_device(np.stack([host[lam][idx] for lam in layers]), wl)


def unit_rows(wl, arr, s, j):
    """Rows ``[l, d]`` of sequence ``s``, head ``j`` from a layer array in either layout."""
    if wl.packed:
        cu = synth.cu_seqlens(wl)
        return arr[cu[s]:cu[s + 1], j]
    return arr[s, j]


def tok_base(wl, s):
    return int(synth.cu_seqlens(wl)[s]) if wl.packed else s * wl.max_len


def unpack_adj(adj_unit: np.ndarray, l: int) -> np.ndarray:
    """``[max_len, row_words]`` int32 words -> boolean ``[l, l]``."""
    words = adj_unit[:l].view(np.uint32)
    bits = np.unpackbits(words.view(np.uint8), axis=1, bitorder="little")
    return bits[:, :l].astype(bool)


def check_evict_unit(wl, Qs, Ks, k_ctx, scores_gpu, keep_gpu, cnt_gpu, score_norm=0):
    """One (layer, sequence): ``Qs [H_q,w,d]``, ``Ks [H_kv,l,d]`` float arrays; GPU rows per KV head.

    Returns the number of kept positions that differ inside the allowed margin.
    """
    l = Ks.shape[1]
    w = wl.window
    l_c = l - w
    res = O.evict_deep(Qs.astype(np.float64), Ks.astype(np.float64), k_ctx, divide_by_distance=(score_norm == 0))
    n_margin = 0
    for j in range(Ks.shape[0]):
        want = res["scores"][j]
        got = scores_gpu[j][:l_c].astype(np.float64)
        np.testing.assert_allclose(got, want, rtol=1e-4, atol=1e-30)
        assert cnt_gpu[j] == k_ctx + w
        kg = keep_gpu[j][: k_ctx + w]
        assert np.all(np.diff(kg) > 0)
        assert list(kg[k_ctx:]) == list(range(l_c, l))  # the window is always reserved
        ko = res["keep"][j]
        if not np.array_equal(kg, ko):
            near = O.topk_margin_mask(want, k_ctx, REL_MARGIN)
            diff = np.setxor1d(kg[:k_ctx], ko[:k_ctx])
            assert np.all(near[diff]), "kept set differs outside the 1e-4 margin"
            n_margin += diff.size
    return n_margin


def check_codebook_unit(gamma, theta, adj_gpu, mag_gpu, ref_gpu, centre_gpu, n_gpu, C_gpu, val_tol):
    """One (layer, sequence, head, Gamma).  Returns the number of adjacency bits decided differently
    inside the allowed margin."""
    l = gamma.shape[0]
    r = O.codebook_shallow(gamma.astype(np.float64), theta)
    np.testing.assert_allclose(mag_gpu[:l], r["mag"], rtol=2e-6)
    n_flip = 0
    if adj_gpu is not None:
        G_gpu = unpack_adj(adj_gpu, l)
        assert np.array_equal(G_gpu, G_gpu.T) and np.all(np.diag(G_gpu))
        diff = G_gpu != r["G"]
        n_flip = int(diff.sum()) // 2
        if n_flip:
            near = O.threshold_margin_mask(r["S"], theta, REL_MARGIN)
            assert not np.any(diff & ~near), "adjacency differs outside the 1e-4 margin"
            r = O.codebook_shallow(gamma.astype(np.float64), theta, G_override=G_gpu)
    n = len(r["centres"])
    assert n_gpu == n
    assert np.array_equal(centre_gpu[:n], r["centres"])
    assert np.array_equal(ref_gpu[:l], r["ref"])
    if C_gpu is not None:
        np.testing.assert_allclose(C_gpu[:n].astype(np.float64), r["C"], rtol=val_tol, atol=val_tol)
    return n_flip


def value_tol(wl):
    return 1e-5 if wl.dtype == "f32" else 1e-2
