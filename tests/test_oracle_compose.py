"""Pins for the checker's composition of Section 3 (every layer evicts, then builds CodeBooks of what it
kept) and for the reserve ratio of Eq. (15): closed forms and special cases whose answer does not
depend on the checker's own code."""
import math

import numpy as np
import pytest

from oracle import spindlekv_oracle as O


def test_literal_plan_is_the_pyramid_over_all_layers():
    for m, lens, w, budget in ((32, [16384], 32, 1024.0), (5, [600, 900], 16, 200.0)):
        mode, ratio, k = O.plan_layers(m, -1, lens, w, 0.05, budget_tokens=budget)
        assert np.all(mode == (O.MODE_EVICT | O.MODE_CODEBOOK))
        for s, l in enumerate(lens):
            r_c = (budget - w) / (l - w)
            assert abs(ratio[:, s].mean() - r_c) < 1e-12            # the pyramid keeps the mean (Eq. (5)(6))
            assert np.all(np.diff(ratio[:, s]) <= 0) and ratio[-1, s] >= 0.05 - 1e-12
            assert np.array_equal(k[:, s], np.floor(ratio[:, s] * (l - w)).astype(np.int32))   # Eq. (7)


def test_dominant_keys_are_kept_and_their_duplicates_share_entries():
    # Four context keys are 6x longer copies of one direction that every window query points at: they
    # take nearly all attention mass, so with k = 4 exactly they are kept (plus the window).  Among the
    # kept keys those four are parallel (cosine 1) and the window keys are random: K needs 1 + w entries.
    rng = np.random.default_rng(5)
    l, w, d, H = 120, 8, 32, 2
    k = rng.standard_normal((H, l, d)) * 0.1
    v = rng.standard_normal((H, l, d))
    dirn = rng.standard_normal(d)
    dirn /= np.linalg.norm(dirn)
    hot = [7, 40, 41, 99]
    for j in range(H):
        k[j, hot] = 6.0 * dirn * np.array([1.0, 1.5, 2.0, 2.5])[:, None]
        v[j, hot] = v[j, hot[0]]                                   # identical values: one V entry for the four
    q = np.tile(8.0 * dirn, (2 * H, w, 1))
    out = O.spindle_layer(q, k, v, 4, 0.98, 0.95)
    for j in range(H):
        assert list(out["keep"][j]) == hot + list(range(l - w, l))
        ck, cv = out["cb_k"][j], out["cb_v"][j]
        assert len(ck["centres"]) == 1 + w and len(cv["centres"]) == 1 + w
        assert len(set(ck["ref"][:4])) == 1 and len(set(cv["ref"][:4])) == 1
        # the entry is the unit vector of the centre; magnitudes are those of the kept rows (Eq. (8))
        np.testing.assert_allclose(np.abs(ck["C"][ck["ref"][0]] @ dirn), 1.0, atol=1e-12)
        np.testing.assert_allclose(ck["mag"][:4], 6.0 * np.array([1.0, 1.5, 2.0, 2.5]), rtol=1e-12)


def test_no_merging_and_total_merging():
    rng = np.random.default_rng(6)
    l, w, d, H = 90, 6, 16, 2
    k, v = rng.standard_normal((H, l, d)), rng.standard_normal((H, l, d))
    q = rng.standard_normal((2 * H, w, d))
    none = O.spindle_layer(q, k, v, 20, 1.0, 1.0)      # nothing is similar enough: one entry per kept token
    every = O.spindle_layer(q, k, v, 20, -1.5, -1.5)   # everything is: one entry per head
    for j in range(H):
        assert len(none["cb_k"][j]["centres"]) == 26 and list(none["cb_k"][j]["ref"]) == list(range(26))
        assert len(every["cb_v"][j]["centres"]) == 1 and np.all(every["cb_v"][j]["ref"] == 0)
    assert np.array_equal(none["keep"], every["keep"])  # eviction does not depend on the thresholds
    # Eq. (15): r1 = kept / l; r2 = entries / kept tokens
    r1, r2 = O.reserve_ratio_layer(l, 26, [26] * H, [26] * H)
    assert r1 == pytest.approx(26 / 90) and r2 == 1.0
    r1, r2 = O.reserve_ratio_layer(l, 26, [1] * H, [1] * H)
    assert r2 == pytest.approx(1 / 26)
    r1, r2 = O.reserve_ratio_layer(100, 40, [10, 30], [20, 20])
    assert r1 == pytest.approx(0.4) and r2 == pytest.approx(80 / 160)


def test_each_cache_uses_its_own_threshold():
    # one threshold merges everything, the other nothing: which cache got which shows in the entry counts
    rng = np.random.default_rng(16)
    l, w, d, H = 70, 5, 12, 2
    k, v = rng.standard_normal((H, l, d)), rng.standard_normal((H, l, d))
    q = rng.standard_normal((2 * H, w, d))
    out = O.spindle_layer(q, k, v, 15, 0.999999, -1.5)
    rep = O.spindle_layer_repeat(q, k, v, 15, 0.999999, -1.5)
    for j in range(H):
        assert len(out["cb_k"][j]["centres"]) == 20 and len(out["cb_v"][j]["centres"]) == 1
        assert len(rep["cb_v"][j]["centres"]) == 1 and len(rep["cb_k"][j]["centres"]) == len(set(rep["union"][j]))


def test_repeat_variant_selects_per_query_head_and_collapses_repeats():
    rng = np.random.default_rng(7)
    l, w, d, H, h_n = 100, 6, 16, 2, 3
    k, v = rng.standard_normal((H, l, d)), rng.standard_normal((H, l, d))
    q = rng.standard_normal((H * h_n, w, d))
    out = O.spindle_layer_repeat(q, k, v, 10, 0.999, 0.999)
    for i in range(H * h_n):
        # a query head's selection is what the group formula gives for a group of one (Eq. (3) with h_n = 1)
        alone = O.evict_deep(q[i:i + 1], k[i // h_n:i // h_n + 1], 10)
        assert np.array_equal(out["keep"][i], alone["keep"][0])
    for j in range(H):
        u = out["union"][j]
        assert np.array_equal(u, np.concatenate([out["keep"][h_n * j + g] for g in range(h_n)]))
        cb = out["cb_k"][j]
        # random directions: nothing merges except copies of the same token, so entries = distinct tokens,
        # and copies (the window, kept by every head, among them) share their entry
        assert len(cb["centres"]) == len(set(u.tolist()))
        first = {}
        for pos, tok in enumerate(u):
            first.setdefault(int(tok), cb["ref"][pos])
            assert cb["ref"][pos] == first[int(tok)]
    # identical query heads in a group select identical tokens: the union is h_n copies, entries as without repeat
    q_same = np.repeat(q[::h_n], h_n, axis=0)
    rep = O.spindle_layer_repeat(q_same, k, v, 10, 0.999, 0.999)
    base = O.spindle_layer(q_same, k, v, 10, 0.999, 0.999)   # group mean of equal scores = the score itself
    for j in range(H):
        assert np.array_equal(rep["keep"][h_n * j], base["keep"][j])
        assert len(rep["cb_k"][j]["centres"]) == len(base["cb_k"][j]["centres"])


def test_decode_time_merge_of_new_tokens():
    rng = np.random.default_rng(8)
    d = 24
    C = rng.standard_normal((5, d))
    C /= np.linalg.norm(C, axis=1, keepdims=True)
    far = rng.standard_normal((3, d))
    far -= (far @ C.T) @ np.linalg.pinv(C.T)            # orthogonal to every entry: cosine 0 with all of them
    new = np.stack([3.0 * C[2],                          # a copy of entry 2, three times as long
                    0.5 * (C[0] + 1e-3 * rng.standard_normal(d)),   # entry 0 with a little noise
                    far[0], 2.0 * far[0],                # two parallel strangers: one new entry for both
                    far[1],                              # another stranger: its own entry
                    C[4] + C[3]])                        # 45 degrees from two entries: cos = 0.707.. < theta
    out = O.codebook_extend(C, new, 0.9)
    assert list(out["ref"][:2]) == [2, 0] and list(out["left"]) == [2, 3, 4, 5]
    assert out["ref"][2] == out["ref"][3] and len({out["ref"][2], out["ref"][4], out["ref"][5]}) == 3
    assert out["C"].shape[0] == 5 + 3 and sorted(out["ref"][2:]) == sorted([5, 5, 6, 7])
    np.testing.assert_allclose(out["mag"][:2], [3.0, np.linalg.norm(new[1])], rtol=1e-12)
    # the same answer by brute force: scalar cosines, first maximum
    for t in range(new.shape[0]):
        cos = [float(new[t] @ C[j]) / (np.linalg.norm(new[t]) * np.linalg.norm(C[j])) for j in range(5)]
        best = max(range(5), key=lambda j: (cos[j], -j))
        assert (out["ref"][t] == best) if cos[best] > 0.9 else (out["ref"][t] >= 5)
    # every new token's reconstruction points within the threshold of the token (Eq. (14))
    rec = O.reconstruct(out["C"], out["ref"], out["mag"])
    cosr = (rec * new).sum(1) / (np.linalg.norm(rec, axis=1) * np.linalg.norm(new, axis=1))
    assert np.all(cosr > 0.9 - 1e-12)
    # with the 45-degree threshold lowered, the last token merges: two equally similar entries, lower number wins
    assert O.codebook_extend(C, new, 0.7)["ref"][5] == 3
    # nothing is suitable at theta >= 1: the result is the old CodeBook followed by the new tokens' own CodeBook
    alone = O.codebook_shallow(new, 1.0)
    ext = O.codebook_extend(C, new, 1.0)
    assert np.array_equal(ext["ref"], 5 + alone["ref"]) and np.allclose(ext["C"][5:], alone["C"])
    # an empty CodeBook: plain Algorithm 1
    assert np.array_equal(O.codebook_extend(np.zeros((0, d)), new, 0.9)["ref"], O.codebook_shallow(new, 0.9)["ref"])


def test_merge_takes_the_most_similar_entry_and_the_lower_number_on_exact_ties():
    # unit entries in the plane at 0, 30 and 0 degrees (entries 0 and 2 are the same vector), one at 90 degrees
    ang = np.deg2rad([0.0, 30.0, 0.0, 90.0])
    C = np.stack([np.cos(ang), np.sin(ang)], axis=1)
    deg = np.deg2rad([25.0, 0.0, 12.0, 50.0])
    new = np.stack([np.cos(deg), np.sin(deg)], axis=1) * np.array([2.0, 0.5, 1.0, 3.0])[:, None]
    ref, S = O.match_entries(C, new, math.cos(math.radians(28.0)))
    # 25 degrees: entries 0/2 (25 away) and 1 (5 away) are all suitable, the nearest wins
    # 0 degrees: entries 0 and 2 tie exactly, the lower number wins
    # 12 degrees: 12 from entries 0/2, 18 from entry 1: entry 0 again
    # 50 degrees: 20 from entry 1, suitable; 40 from entry 3, not suitable
    assert list(ref) == [1, 0, 0, 1]
    np.testing.assert_allclose(S[0], np.cos(np.deg2rad([25.0, 5.0, 25.0, 65.0])), atol=1e-15)
    # at a 4-degree threshold only the exact copy is suitable; the others open entries of their own
    out = O.codebook_extend(C, new, math.cos(math.radians(4.0)))
    assert list(out["ref"]) == [4, 0, 5, 6] and list(out["left"]) == [0, 2, 3]
