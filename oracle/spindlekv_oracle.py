"""CPU checker for the SpindleKV prefill KV-cache reduction pass.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of what
the paper defines, in numpy float64.  It shares no code with the CUDA library
and must never be imported by it; only the tests, the smoke check and the
benchmark's CPU-baseline leg may call it.

Every function names the passage it follows.  Equations are numbered in print
order: (1) masked softmax attention, (2) accumulated attention score, (3) GQA
group mean, (4) cosine similarity, (5) first/last-layer retain ratios,
(6) per-layer interpolation, (7) argTopK selection, (8) magnitudes,
(9) thresholded adjacency, (10) node degree, (11) greedy centre pick,
(12) reference assignment, (13) graph clean-up, (14) reconstruction.
"Algorithm 1" is the CodeBook-generation listing.

Readings taken where the text is silent, garbled or inconsistent:

* Eq. (2): ``A[i, a, b]`` is the weight query ``b`` puts on key ``a``; the
  denominator is ``l - a`` exactly as printed.
* Eq. (3): the sum runs over ``g = 0 .. h_n - 1`` and the printed ``n - a`` is
  ``l - a``.
* Eq. (1): causal mask; each window query ``b`` is normalised over keys
  ``0..b`` (window keys included); scale ``1 / sqrt(d_h)``.
* Eq. (5): the printed ``0.05`` is ``beta`` and the last case is
  ``2 r_c - 1`` (this is the only reading that is continuous at ``alpha`` and
  keeps the mean over layers equal to ``r_c``).
* Eq. (7): ties go to the lower index; the kept indices are returned in
  ascending position followed by the window positions.
* Eq. (9): strict ``>``; the diagonal of ``G`` is 1 (a token is similar to
  itself, which is what lets the loop end and gives isolated tokens an entry).
* Eq. (10) / Algorithm 1: the degree is the row sum of ``G`` (the listing
  prints ``S``).
* Eq. (11): ``argmax`` ties go to the lower index; a CodeBook entry is the
  unit vector of the centre token (no averaging).
* Zero vectors get ``gamma_hat = 0`` and therefore an entry of their own.
* Rotary position embedding (the matrix R of Eq. (1), which the paper does not spell out): the
  convention of the LLaMA / Mistral models the paper evaluates, i.e. element ``i < d_h/2`` is paired
  with element ``i + d_h/2`` and the pair is rotated by the angle ``p * base**(-2 i / d_h)`` at
  position ``p``.
* Attention over the replaced cache at decode time (Section 3.4, after Eq. (14)): K is rebuilt as
  ``C_K[r_K] (x) m_K`` from CodeBooks of pre-RoPE keys, rotated at each token's original position,
  and scored against the rotated query; V is rebuilt as ``C_V[r_V] (x) m_V``; every cached token is
  visible to the new query.
* The shallow/deep split is an argument: layers ``< n_shallow`` build
  CodeBooks over all tokens, layers ``>= n_shallow`` evict, with the pyramid
  of Eq. (5)(6) laid over the evicting layers only.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

MODE_EVICT = 1
MODE_CODEBOOK = 2


class BudgetError(ValueError):
    """The context reserve ratio falls outside ``(beta, 1]`` where Eq. (5) is defined."""


# --------------------------------------------------------------------------
# Budget planner: the unnumbered r_c definition, Eq. (5), Eq. (6), Eq. (7)'s k
# --------------------------------------------------------------------------

def context_reserve_ratio(reserved_tokens: float, l: int, l_w: int) -> float:
    """``r_c = (r*l - l_w) / l_c`` with ``l_c = l - l_w`` (Section 3.3).

    ``reserved_tokens`` is the product ``r * l``: tokens kept per head, the
    observation window included.
    """
    l_c = l - l_w
    if l_c <= 0:
        raise BudgetError("sequence not longer than the observation window")
    return (float(reserved_tokens) - float(l_w)) / float(l_c)


def pyramid_endpoints(r_c: float, beta: float) -> Tuple[float, float]:
    """Retain ratios of the first and last evicting layer, Eq. (5)."""
    alpha = 0.5 * (1.0 + beta)
    if beta < r_c <= alpha:
        return 2.0 * r_c - beta, beta
    if alpha < r_c <= 1.0:
        return 1.0, 2.0 * r_c - 1.0
    raise BudgetError(f"r_c={r_c} outside (beta, 1]")


def layer_ratio(r_first: float, r_last: float, m: int, lam: int, r_c: float) -> float:
    """Eq. (6): linear interpolation over ``m`` evicting layers (``m == 1``: flat ``r_c``)."""
    if m == 1:
        return r_c
    return r_first + (r_last - r_first) / float(m - 1) * float(lam)


def plan_layers(n_layers: int, n_shallow: int, seq_lens: Sequence[int], l_w: int, beta: float,
                reserve_ratio: Optional[float] = None, budget_tokens: Optional[float] = None):
    """Per-layer mode, retain ratio and top-k size for every sequence.

    Returns ``(mode[m], r_c_layer[m, B], k_ctx[m, B])``; shallow layers carry
    ratio 1 and ``k = l_c`` (nothing is evicted there).  ``k`` follows Eq. (7):
    ``floor(r_c(lambda) * l_c)``.  ``n_shallow = -1`` is the paper's own
    composition: all layers evict (pyramid over all ``m`` layers) and all build
    CodeBooks of the kept tokens.
    """
    B = len(seq_lens)
    if n_shallow == -1:
        # Section 3 as written: every layer evicts under the pyramid laid over all layers and then
        # builds CodeBooks of what it kept
        mode, ratio, k_ctx = plan_layers(n_layers, 0, seq_lens, l_w, beta, reserve_ratio, budget_tokens)
        return np.full(n_layers, MODE_EVICT | MODE_CODEBOOK, dtype=np.int32), ratio, k_ctx
    m_deep = n_layers - n_shallow
    mode = np.array([MODE_CODEBOOK if lam < n_shallow else MODE_EVICT for lam in range(n_layers)],
                    dtype=np.int32)
    ratio = np.ones((n_layers, B), dtype=np.float64)
    k_ctx = np.zeros((n_layers, B), dtype=np.int32)
    for s, l in enumerate(seq_lens):
        l_c = l - l_w
        if l_c <= 0:
            raise BudgetError("sequence not longer than the observation window")
        k_ctx[:n_shallow, s] = l_c
        if m_deep == 0:
            continue
        rl = float(budget_tokens) if budget_tokens is not None else float(reserve_ratio) * float(l)
        r_c = context_reserve_ratio(rl, l, l_w)
        r0, r1 = pyramid_endpoints(r_c, beta)
        for lam in range(m_deep):
            r = layer_ratio(r0, r1, m_deep, lam, r_c)
            ratio[n_shallow + lam, s] = r
            k_ctx[n_shallow + lam, s] = min(l_c, int(math.floor(r * float(l_c))))
    return mode, ratio, k_ctx


# --------------------------------------------------------------------------
# Deep layers: Eq. (1), (2), (3), (7)
# --------------------------------------------------------------------------

def window_attention(q_win: np.ndarray, k: np.ndarray) -> np.ndarray:
    """Eq. (1) restricted to the last ``w`` queries of one head.

    ``q_win`` is ``[w, d]`` (queries at positions ``l-w .. l-1``), ``k`` is
    ``[l, d]``.  Returns ``A[t, a]``: the weight window query ``t`` (position
    ``b = l - w + t``) puts on key ``a``; zero where ``a > b``.
    """
    q_win = np.asarray(q_win, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    w, d = q_win.shape
    l = k.shape[0]
    s = (q_win @ k.T) / math.sqrt(d)
    pos_b = (l - w) + np.arange(w)[:, None]
    allowed = np.arange(l)[None, :] <= pos_b
    s = np.where(allowed, s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


def accumulated_scores(q_win: np.ndarray, k: np.ndarray, divide_by_distance: bool = True) -> np.ndarray:
    """Eq. (2): ``ac[a] = sum_b A[b, a] / (l - a)`` over the window queries, for all ``a < l``.

    With ``divide_by_distance=False`` the raw window sum is returned (an
    extension outside the paper, used only to pin the tie-break).
    """
    A = window_attention(q_win, k)
    l = k.shape[0]
    ac = A.sum(axis=0)
    if divide_by_distance:
        ac = ac / (l - np.arange(l, dtype=np.float64))
    return ac


def group_scores(q_win_heads: np.ndarray, k_heads: np.ndarray, divide_by_distance: bool = True) -> np.ndarray:
    """Eq. (3): mean of Eq. (2) over the ``h_n`` query heads that share each KV head.

    ``q_win_heads`` is ``[H_q, w, d]``, ``k_heads`` is ``[H_kv, l, d]``;
    query head ``h_n * j + g`` reads KV head ``j``.  Returns ``[H_kv, l]``.
    """
    H_q, H_kv = q_win_heads.shape[0], k_heads.shape[0]
    h_n = H_q // H_kv
    l = k_heads.shape[1]
    out = np.zeros((H_kv, l), dtype=np.float64)
    for j in range(H_kv):
        for g in range(h_n):
            out[j] += accumulated_scores(q_win_heads[h_n * j + g], k_heads[j], divide_by_distance)
        out[j] /= float(h_n)
    return out


def arg_topk(scores: np.ndarray, k: int) -> np.ndarray:
    """Eq. (7): indices of the ``k`` largest scores, ties to the lower index, ascending."""
    scores = np.asarray(scores, dtype=np.float64)
    idx = np.arange(scores.shape[0])
    order = np.lexsort((idx, -scores))  # primary: score descending; secondary: index ascending
    return np.sort(order[:k]).astype(np.int32)


def evict_deep(q_win_heads: np.ndarray, k_heads: np.ndarray, k_ctx: int,
               divide_by_distance: bool = True) -> Dict[str, np.ndarray]:
    """Eq. (1)(2)(3)(7) for one (layer, sequence).

    Returns ``keep[H_kv, k_ctx + w]`` (selected context positions ascending,
    then the window positions, which are always reserved) and the context
    scores ``[H_kv, l_c]``.
    """
    w = q_win_heads.shape[1]
    H_kv, l, _ = k_heads.shape
    l_c = l - w
    sc = group_scores(q_win_heads, k_heads, divide_by_distance)[:, :l_c]
    keep = np.empty((H_kv, k_ctx + w), dtype=np.int32)
    for j in range(H_kv):
        keep[j, :k_ctx] = arg_topk(sc[j], k_ctx)
        keep[j, k_ctx:] = np.arange(l_c, l)
    return {"keep": keep, "scores": sc}


def topk_margin_mask(scores: np.ndarray, k: int, rel: float = 1e-4) -> np.ndarray:
    """Positions whose score lies within ``rel`` (relative) of the k-th largest score.

    Membership of such positions in the kept set may legitimately differ
    between two correct implementations that round differently.
    """
    scores = np.asarray(scores, dtype=np.float64)
    if k <= 0 or k >= scores.shape[0]:
        return np.zeros(scores.shape[0], dtype=bool)
    kth = np.sort(scores)[::-1][k - 1]
    return np.abs(scores - kth) < rel * abs(kth)


# --------------------------------------------------------------------------
# Shallow layers: Eq. (4), (8)-(13), Algorithm 1
# --------------------------------------------------------------------------

def magnitudes(gamma: np.ndarray) -> np.ndarray:
    """Eq. (8): ``m_a = sqrt(gamma_a . gamma_a)``."""
    gamma = np.asarray(gamma, dtype=np.float64)
    return np.sqrt((gamma * gamma).sum(axis=1))


def normalise(gamma: np.ndarray, m: np.ndarray) -> np.ndarray:
    """Eq. (8): ``gamma_hat = gamma / m``; a zero vector stays zero."""
    gamma = np.asarray(gamma, dtype=np.float64)
    safe = np.where(m > 0.0, m, 1.0)
    return np.where(m[:, None] > 0.0, gamma / safe[:, None], 0.0)


def cosine_similarity(gamma: np.ndarray) -> np.ndarray:
    """Eq. (4): ``S[a, b] = gamma_a . gamma_b / (|gamma_a| |gamma_b|)`` for all pairs of one head."""
    g = normalise(gamma, magnitudes(gamma))
    return g @ g.T


def adjacency(S: np.ndarray, theta: float) -> np.ndarray:
    """Eq. (9): ``G = where(S > theta, 1, 0)`` as a symmetric boolean matrix with unit diagonal.

    The pair ``(a, b)`` with ``a < b`` is decided once, from ``S[a, b]``, and
    mirrored, so that ``G`` is an undirected graph whatever the rounding of
    the two triangles of ``S``.
    """
    up = np.triu(S > theta, k=1)
    G = up | up.T
    np.fill_diagonal(G, True)
    return G


def codebook_cover_small(G: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. (10)-(13) written out on explicit node lists, for small ``N`` only.

    Nothing is kept between picks: for every pick the degree of each remaining node is counted
    afresh by going through all remaining nodes (Eq. (10), the node itself included because the
    diagonal of ``G`` is 1); the remaining node with the largest count, the lowest index among
    equals, becomes a centre (Eq. (11)); the remaining nodes similar to it, itself among them, take
    the new entry's number (Eq. (12)) and leave the graph (Eq. (13)).  Work per pick is quadratic in
    the number of remaining nodes.  This form shares no bookkeeping with ``codebook_greedy`` and
    serves as its cross-check.  Returns ``(centres, ref)``.
    """
    G = np.asarray(G, dtype=bool)
    n = G.shape[0]
    remaining = list(range(n))
    ref = [-1] * n
    centres: List[int] = []
    while remaining:
        chosen, chosen_degree = -1, -1
        for a in remaining:                      # ascending: the first largest count is the lowest index
            count = 0
            for b in remaining:
                if a == b or G[a, b]:
                    count += 1
            if count > chosen_degree:
                chosen, chosen_degree = a, count
        members = [b for b in remaining if b == chosen or G[chosen, b]]
        for b in members:
            ref[b] = len(centres)
        centres.append(chosen)
        gone = set(members)
        remaining = [b for b in remaining if b not in gone]
    return np.array(centres, dtype=np.int32), np.array(ref, dtype=np.int32)


def codebook_greedy(G: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Eq. (10)-(13) on a set of live nodes, usable at full sequence length.

    The steps of Eq. (10)-(13) in their order; what differs from the small-N form above is
    bookkeeping only: removed nodes leave a ``live`` set instead of having their
    rows and columns zeroed, and the degree vector of Eq. (10) is kept current
    by subtracting, for every removed node, its row of ``G`` (``G`` is
    symmetric, so that row is exactly what the node contributed to the other
    degrees).  Returns ``(centres, ref, pick_degree)``.
    """
    G = np.asarray(G, dtype=bool)
    n = G.shape[0]
    live = np.ones(n, dtype=bool)
    s = G.sum(axis=1).astype(np.int64)
    ref = -np.ones(n, dtype=np.int32)
    centres: List[int] = []
    degs: List[int] = []
    n_live = n
    while n_live > 0:
        iota = int(np.argmax(np.where(live, s, -1)))
        eta = np.flatnonzero(G[iota] & live)
        ref[eta] = len(centres)
        centres.append(iota)
        degs.append(int(s[iota]))
        live[eta] = False
        n_live -= eta.shape[0]
        s -= G[eta].sum(axis=0)
    return np.array(centres, dtype=np.int32), ref, np.array(degs, dtype=np.int64)


def codebook_shallow(gamma: np.ndarray, theta: float, G_override: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """Algorithm 1 for one (layer, sequence, KV head, Gamma in {K, V}).

    Returns magnitudes ``mag[N]``, references ``ref[N]``, centre token indices
    ``centres[|C|]``, the CodeBook ``C[|C|, d]`` (unit vectors of the centres)
    and the similarity matrix ``S``.  ``G_override`` replaces the adjacency
    (used by tests to settle pairs that sit on the threshold).
    """
    gamma = np.asarray(gamma, dtype=np.float64)
    mag = magnitudes(gamma)
    ghat = normalise(gamma, mag)
    S = ghat @ ghat.T
    G = adjacency(S, theta) if G_override is None else np.asarray(G_override, dtype=bool)
    centres, ref, degs = codebook_greedy(G)
    return {"mag": mag, "ref": ref, "centres": centres, "C": ghat[centres], "S": S, "G": G,
            "pick_degree": degs}


def threshold_margin_mask(S: np.ndarray, theta: float, rel: float = 1e-4) -> np.ndarray:
    """Pairs whose similarity lies within ``rel`` (relative) of the threshold."""
    return np.abs(S - theta) < rel * abs(theta)


def reconstruct(C: np.ndarray, ref: np.ndarray, mag: np.ndarray) -> np.ndarray:
    """Eq. (14): ``Gamma_r = C[r] (x) m``."""
    return np.asarray(C, dtype=np.float64)[ref] * np.asarray(mag, dtype=np.float64)[:, None]


def gather_rows(gamma: np.ndarray, idx: np.ndarray) -> np.ndarray:
    """Eq. (7), second line: ``Gamma_r = Gamma[eta]``."""
    return np.asarray(gamma)[np.asarray(idx, dtype=np.int64)]


# --------------------------------------------------------------------------
# The composition of Section 3 as written, and the reserve ratio of Eq. (15)
# --------------------------------------------------------------------------

def spindle_layer(q_win_heads: np.ndarray, k_heads: np.ndarray, v_heads: np.ndarray, k_ctx: int,
                  theta_k: float, theta_v: float) -> Dict[str, object]:
    """One layer of one sequence as Section 3 composes it: Eq. (1)(2)(3)(7) pick the tokens to keep
    per KV head; Algorithm 1 then builds a K and a V CodeBook from the kept rows of each head.

    Returns the kept positions ``keep[H_kv, k + w]`` and, per head, the CodeBook results of
    ``K[keep]`` and ``V[keep]`` (lists ``cb_k``, ``cb_v`` of ``codebook_shallow`` dictionaries).
    """
    ev = evict_deep(q_win_heads, k_heads, k_ctx)
    cb_k, cb_v = [], []
    for j in range(k_heads.shape[0]):
        cb_k.append(codebook_shallow(gather_rows(k_heads[j], ev["keep"][j]), theta_k))
        cb_v.append(codebook_shallow(gather_rows(v_heads[j], ev["keep"][j]), theta_v))
    return {"keep": ev["keep"], "scores": ev["scores"], "cb_k": cb_k, "cb_v": cb_v}


def spindle_layer_repeat(q_win_heads: np.ndarray, k_heads: np.ndarray, v_heads: np.ndarray, k_ctx: int,
                         theta_k: float, theta_v: float) -> Dict[str, object]:
    """The GQA "repeat" alternative of Section 3.3: the KV vectors are repeated ``h_n`` times, so that
    every query head ``i`` selects by its own ``ac_i`` of Eq. (2) (no group mean), and the CodeBooks of KV
    head ``j`` are built (Section 3.4) from the rows kept by its query heads ``h_n*j .. h_n*j + h_n - 1``,
    one head after the other; a token kept by several heads appears several times (cosine 1).

    Reading (the paper does not say over which tokens the CodeBook of a repeated cache is built): per KV
    head, over the concatenation above.  Returns ``keep[H_q, k + w]``, ``union[H_kv, h_n (k + w)]`` and the
    per-KV-head CodeBook results.
    """
    H_q, w = q_win_heads.shape[0], q_win_heads.shape[1]
    H_kv, l, _ = k_heads.shape
    h_n = H_q // H_kv
    keep = np.empty((H_q, k_ctx + w), dtype=np.int32)
    scores = np.empty((H_q, l - w), dtype=np.float64)
    for i in range(H_q):
        ev = evict_deep(q_win_heads[i:i + 1], k_heads[i // h_n:i // h_n + 1], k_ctx)
        keep[i], scores[i] = ev["keep"][0], ev["scores"][0]
    union = keep.reshape(H_kv, h_n * (k_ctx + w))
    cb_k = [codebook_shallow(gather_rows(k_heads[j], union[j]), theta_k) for j in range(H_kv)]
    cb_v = [codebook_shallow(gather_rows(v_heads[j], union[j]), theta_v) for j in range(H_kv)]
    return {"keep": keep, "scores": scores, "union": union, "cb_k": cb_k, "cb_v": cb_v}


def reserve_ratio_layer(l: int, kept: int, entries_k: Sequence[int], entries_v: Sequence[int]) -> Tuple[float, float]:
    """Eq. (15) for one layer: ``r1`` = kept K and V tokens over all K and V tokens (summed over the
    KV heads), ``r2`` = CodeBook entries of K and V over kept K and V tokens.  The dtype factor
    ``r3`` is left to the caller."""
    h = len(entries_k)
    r1 = (2.0 * h * kept) / (2.0 * h * l)
    r2 = (float(sum(entries_k)) + float(sum(entries_v))) / (2.0 * h * kept)
    return r1, r2


# --------------------------------------------------------------------------
# Decode-time merging of new tokens into a CodeBook (Section 3.4, last paragraph)
# --------------------------------------------------------------------------

def match_entries(C: np.ndarray, gamma_new: np.ndarray, theta: float) -> Tuple[np.ndarray, np.ndarray]:
    """For every new token the existing entry it is merged into, or -1.

    "Suitable" entries are those whose cosine similarity with the token exceeds ``theta`` (strictly).
    Reading: among several, the most similar one, the lower entry number on ties.  The cosine is taken
    with the entries as stored (their own norm divides, although it is 1 up to the rounding of the
    storage type).  Returns ``(ref, S)`` with ``S[t, j]`` the similarities.
    """
    C = np.asarray(C, dtype=np.float64)
    g = normalise(gamma_new, magnitudes(gamma_new))
    S = g @ normalise(C, magnitudes(C)).T if C.shape[0] else np.zeros((g.shape[0], 0))
    ref = -np.ones(g.shape[0], dtype=np.int32)
    for t in range(g.shape[0]):
        if S.shape[1] and S[t].max() > theta:
            ref[t] = int(np.argmax(S[t]))      # first maximum: lower entry number on ties
    return ref, S


def codebook_extend(C: np.ndarray, gamma_new: np.ndarray, theta: float,
                    ref_override: Optional[np.ndarray] = None, G_override: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """New tokens are merged into suitable entries; for the remaining ones the CodeBook construction is
    repeated (Algorithm 1 on the unmatched tokens, in their order) and its entries are appended.

    ``ref_override`` replaces the matching decisions and ``G_override`` the adjacency of the unmatched
    tokens (tests use both to settle decisions that sit on the threshold).  Returns ``ref`` (entry of
    every new token in the extended CodeBook), ``mag``, the extended ``C``, the similarities ``S`` and
    the unmatched positions ``left``.
    """
    C = np.asarray(C, dtype=np.float64)
    gamma_new = np.asarray(gamma_new, dtype=np.float64)
    ref, S = match_entries(C, gamma_new, theta)
    if ref_override is not None:
        ref = np.asarray(ref_override, dtype=np.int32).copy()
    left = np.flatnonzero(ref < 0)
    out_ref = ref.copy()
    C_ext = C
    sub = None
    if left.size:
        sub = codebook_shallow(gamma_new[left], theta, G_override=G_override)
        out_ref[left] = C.shape[0] + sub["ref"]
        C_ext = np.concatenate([C, sub["C"]], axis=0)
    return {"ref": out_ref, "mag": magnitudes(gamma_new), "C": C_ext, "S": S, "left": left, "sub": sub}


# --------------------------------------------------------------------------
# Decode-time attention over the replaced cache (Eq. (14), Eq. (1), Section 3.4 last paragraph)
# --------------------------------------------------------------------------

def rope_frequencies(d: int, base: float = 10000.0) -> np.ndarray:
    """Angular steps ``omega_i = base**(-2 i / d)`` for ``i = 0 .. d/2 - 1``."""
    return np.asarray(base, dtype=np.float64) ** (-2.0 * np.arange(d // 2, dtype=np.float64) / float(d))


def rope(x: np.ndarray, positions: np.ndarray, base: float = 10000.0) -> np.ndarray:
    """Rotary position embedding (the matrix R of Eq. (1)) of rows ``x[t]`` at positions ``positions[t]``.

    Element ``i`` and element ``i + d/2`` form a pair that is rotated by ``positions[t] * omega_i``:
    ``(a, b) -> (a cos - b sin, b cos + a sin)``.
    """
    x = np.asarray(x, dtype=np.float64)
    d = x.shape[-1]
    h = d // 2
    ang = np.asarray(positions, dtype=np.float64)[..., None] * rope_frequencies(d, base)
    c, s_ = np.cos(ang), np.sin(ang)
    a, b = x[..., :h], x[..., h:]
    return np.concatenate([a * c - b * s_, b * c + a * s_], axis=-1)


def decode_attention(q: np.ndarray, pos_q: int, C_K: np.ndarray, r_K: np.ndarray, m_K: np.ndarray,
                     C_V: np.ndarray, r_V: np.ndarray, m_V: np.ndarray, positions: Optional[np.ndarray] = None,
                     base: float = 10000.0) -> Dict[str, np.ndarray]:
    """One decode step of the query heads of a GQA group over the replaced cache of their KV head.

    ``q`` is ``[h_n, d]``: the pre-RoPE queries of the new token at position ``pos_q``.  The CodeBooks were
    built from pre-RoPE keys (Section 3.4), so: ``K = C_K[r_K] (x) m_K`` (Eq. (14)), rotated at each cached
    token's own position (``positions[t]``, default ``t``); the query is rotated at ``pos_q``;
    ``A = softmax(q K^T / sqrt(d))`` over all cached tokens (Eq. (1); every cached token precedes the
    query); ``V = C_V[r_V] (x) m_V``; output ``A V``.  Returns ``out [h_n, d]`` and ``A [h_n, n]``.
    """
    q = np.asarray(q, dtype=np.float64)
    n = np.asarray(r_K).shape[0]
    d = q.shape[1]
    positions = np.arange(n) if positions is None else np.asarray(positions)
    K = rope(reconstruct(C_K, r_K, m_K), positions, base)
    V = reconstruct(C_V, r_V, m_V)
    qr = rope(q, np.full(q.shape[0], pos_q), base)
    s = (qr @ K.T) / math.sqrt(d)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    A = e / e.sum(axis=1, keepdims=True)
    return {"out": A @ V, "A": A}
