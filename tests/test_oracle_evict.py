"""Pins for the checker's eviction path (Eq. (1)(2)(3)(7)): closed forms, invariants,
brute force on tiny inputs, and library softmax on small cases."""
import itertools
import math

import numpy as np
import pytest
import torch

from oracle import spindlekv_oracle as O


def _brute_scores(q, k, h_n):
    """Eq. (1)(2)(3) with python loops and math.exp, one scalar at a time."""
    H_q, w, d = q.shape
    H_kv, l, _ = k.shape
    out = [[0.0] * l for _ in range(H_kv)]
    for j in range(H_kv):
        for g in range(h_n):
            i = h_n * j + g
            for t in range(w):
                b = l - w + t
                logits = []
                for a in range(b + 1):
                    dot = 0.0
                    for c in range(d):
                        dot += float(q[i, t, c]) * float(k[j, a, c])
                    logits.append(dot / math.sqrt(d))
                mx = max(logits)
                den = sum(math.exp(x - mx) for x in logits)
                for a in range(b + 1):
                    out[j][a] += math.exp(logits[a] - mx) / den / (l - a) / h_n
    return np.array(out)


def test_scores_against_scalar_brute_force():
    rng = np.random.default_rng(0)
    q = rng.standard_normal((4, 3, 5))
    k = rng.standard_normal((2, 9, 5))
    got = O.group_scores(q, k)
    want = _brute_scores(q, k, 2)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-15)


def test_attention_rows_against_torch_softmax():
    rng = np.random.default_rng(1)
    q = rng.standard_normal((6, 16))
    k = rng.standard_normal((40, 16))
    A = O.window_attention(q, k)
    l, w = 40, 6
    for t in range(w):
        b = l - w + t
        logits = torch.tensor(k[: b + 1] @ q[t]) / math.sqrt(16)
        want = torch.softmax(logits, dim=0).numpy()
        np.testing.assert_allclose(A[t, : b + 1], want, rtol=1e-12)
        assert np.all(A[t, b + 1:] == 0.0)  # causal: later keys are invisible
    np.testing.assert_allclose(A.sum(axis=1), 1.0, rtol=1e-13)


def test_scale_is_inverse_sqrt_head_dim():
    # one query, two visible keys with dot products 4 and 0, d = 4 -> logits 2 and 0
    q = np.array([[2.0, 0.0, 0.0, 0.0]])
    k = np.array([[2.0, 0, 0, 0], [0.0, 1.0, 0, 0]])
    # window = 1 query at position 1 sees both keys
    A = O.window_attention(q, k)
    assert A[0, 0] == pytest.approx(math.exp(2.0) / (math.exp(2.0) + 1.0), rel=1e-14)


def test_mass_identity():
    # softmax rows sum to one, so sum_a (l - a) * ac[a] equals the number of window queries
    rng = np.random.default_rng(2)
    for l, w, d in [(50, 8, 8), (129, 32, 16)]:
        q = rng.standard_normal((w, d)) * 3
        k = rng.standard_normal((l, d))
        ac = O.accumulated_scores(q, k)
        assert np.sum((l - np.arange(l)) * ac) == pytest.approx(w, rel=1e-12)
        raw = O.accumulated_scores(q, k, divide_by_distance=False)
        assert raw.sum() == pytest.approx(w, rel=1e-12)


def test_zero_queries_closed_form_and_tie_break():
    # Q = 0: every visible key gets 1/(b+1); ac[a] = c / (l - a) rises with a, so the last k context
    # tokens are kept; without the distance division all context scores tie and the first k win.
    l, w, d, k_ctx = 64, 8, 4, 10
    l_c = l - w
    rng = np.random.default_rng(3)
    q = np.zeros((2, w, d))
    k = rng.standard_normal((1, l, d))
    c = sum(1.0 / (b + 1) for b in range(l_c, l))
    sc = O.group_scores(q, k)[0]
    np.testing.assert_allclose(sc[:l_c], c / (l - np.arange(l_c)), rtol=1e-13)
    res = O.evict_deep(q, k, k_ctx)
    assert list(res["keep"][0]) == list(range(l_c - k_ctx, l_c)) + list(range(l_c, l))
    res = O.evict_deep(q, k, k_ctx, divide_by_distance=False)
    assert list(res["keep"][0]) == list(range(k_ctx)) + list(range(l_c, l))


def test_single_head_group_equals_eq2_and_mean_over_group():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((4, 5, 8))
    k = rng.standard_normal((1, 30, 8))
    per_head = np.stack([O.accumulated_scores(q[i], k[0]) for i in range(4)])
    np.testing.assert_allclose(O.group_scores(q, k)[0], per_head.mean(axis=0), rtol=1e-13)
    np.testing.assert_array_equal(O.group_scores(q[:1], k)[0], per_head[0])  # h_n = 1
    # two KV heads: query heads 0,1 read KV head 0; 2,3 read KV head 1
    k2 = rng.standard_normal((2, 30, 8))
    g = O.group_scores(q, k2)
    want1 = 0.5 * (O.accumulated_scores(q[2], k2[1]) + O.accumulated_scores(q[3], k2[1]))
    np.testing.assert_allclose(g[1], want1, rtol=1e-13)


def test_dominant_key_takes_the_window_mass():
    # one context key aligned with every query at a huge scale: it receives ~all the weight
    l, w, d = 40, 4, 8
    rng = np.random.default_rng(5)
    k = rng.standard_normal((l, d)) * 0.01
    k[7] = 100.0 * np.ones(d)
    q = np.ones((w, d))
    ac = O.accumulated_scores(q, k)
    assert ac[7] == pytest.approx(w / (l - 7), rel=1e-9)


def test_topk_against_subset_enumeration():
    rng = np.random.default_rng(6)
    for n, k in [(6, 2), (9, 4), (12, 5), (12, 11), (5, 5), (7, 0)]:
        s = rng.random(n)
        got = O.arg_topk(s, k)
        best = max(itertools.combinations(range(n), k), key=lambda c: sum(s[list(c)]))
        assert list(got) == sorted(best)


def test_topk_ties_go_to_lower_index():
    assert list(O.arg_topk(np.array([1.0, 3.0, 3.0, 2.0, 3.0]), 2)) == [1, 2]
    assert list(O.arg_topk(np.array([5.0, 5.0, 5.0, 5.0]), 3)) == [0, 1, 2]
    assert list(O.arg_topk(np.array([0.0, 1.0, 0.0, 1.0, 0.0]), 3)) == [0, 1, 3]


def test_window_always_reserved_and_exact_budget():
    rng = np.random.default_rng(8)
    q = rng.standard_normal((4, 8, 16))
    k = rng.standard_normal((2, 100, 16))
    res = O.evict_deep(q, k, 17)
    keep = res["keep"]
    assert keep.shape == (2, 17 + 8)
    for j in range(2):
        assert list(keep[j, 17:]) == list(range(92, 100))
        assert np.all(np.diff(keep[j]) > 0)
        assert keep[j, 16] < 92
        kept_min = res["scores"][j][keep[j, :17]].min()
        dropped = np.setdiff1d(np.arange(92), keep[j, :17])
        assert kept_min >= res["scores"][j][dropped].max()


def test_margin_mask_marks_the_boundary_only():
    s = np.array([10.0, 5.0, 5.0 * (1 + 5e-5), 1.0, 0.5])
    m = O.topk_margin_mask(s, 2)
    assert list(m) == [False, True, True, False, False]
