"""Pins for the checker's CodeBook path (Eq. (4), (8)-(14), Algorithm 1): hand-worked graphs,
an independent set-based greedy, exhaustive enumeration of small graphs, invariants,
degenerate thresholds and closed forms."""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import spindlekv_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _hand_graphs():
    out = []
    with open(os.path.join(GOLDEN, "hand_graphs.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, n, edges, centres, ref = [x.strip() for x in line.split("|")]
            n = int(n)
            G = np.eye(n, dtype=bool)
            for e in edges.split():
                a, b = map(int, e.split("-"))
                G[a, b] = G[b, a] = True
            out.append((name, G, [int(x) for x in centres.split()], [int(x) for x in ref.split()]))
    return out


@pytest.mark.parametrize("name,G,centres,ref", _hand_graphs(), ids=[g[0] for g in _hand_graphs()])
def test_hand_worked_graphs(name, G, centres, ref):
    for fn in (O.codebook_cover_small, O.codebook_greedy):
        res = fn(G)
        assert list(res[0]) == centres
        assert list(res[1]) == ref


def _set_greedy(adj):
    """Greedy cover on python sets: written independently of the numpy forms."""
    live = set(range(len(adj)))
    centres, ref = [], [-1] * len(adj)
    while live:
        best = min(live, key=lambda u: (-len(adj[u] & live), u))
        covered = adj[best] & live
        for b in covered:
            ref[b] = len(centres)
        centres.append(best)
        live -= covered
    return centres, ref


def _adj_sets(G):
    return [set(np.flatnonzero(G[a]).tolist()) for a in range(G.shape[0])]


def _check_invariants(G, centres, ref, degs=None):
    n = G.shape[0]
    assert np.all(ref >= 0) and np.all(ref < len(centres))  # nobody keeps -1
    for j, c in enumerate(centres):
        assert ref[c] == j  # a centre refers to itself
    for a, b in itertools.combinations(centres, 2):
        assert not G[a, b]  # centres are pairwise non-adjacent
    for b in range(n):
        first = min(j for j, c in enumerate(centres) if G[c, b])
        assert ref[b] == first  # the earliest-picked adjacent centre owns the token
    if degs is not None:
        assert np.all(np.diff(degs) <= 0)  # pick-time degrees never increase


def test_all_graphs_up_to_five_nodes():
    for n in range(1, 6):
        pairs = list(itertools.combinations(range(n), 2))
        for bits in range(1 << len(pairs)):
            G = np.eye(n, dtype=bool)
            for e, (a, b) in enumerate(pairs):
                if bits >> e & 1:
                    G[a, b] = G[b, a] = True
            want = _set_greedy(_adj_sets(G))
            c1, r1 = O.codebook_cover_small(G)
            c2, r2, d2 = O.codebook_greedy(G)
            assert list(c1) == want[0] and list(r1) == want[1]
            assert list(c2) == want[0] and list(r2) == want[1]
            _check_invariants(G, c2, r2, d2)


@pytest.mark.parametrize("n,p", [(12, 0.1), (30, 0.05), (30, 0.3), (48, 0.5), (64, 0.02), (64, 0.9)])
def test_random_graphs_three_ways(n, p):
    rng = np.random.default_rng(n * 1000 + int(p * 100))
    for _ in range(10):
        up = np.triu(rng.random((n, n)) < p, k=1)
        G = up | up.T | np.eye(n, dtype=bool)
        want = _set_greedy(_adj_sets(G))
        c1, r1 = O.codebook_cover_small(G)
        c2, r2, d2 = O.codebook_greedy(G)
        assert list(c1) == want[0] and list(r1) == want[1]
        assert list(c2) == want[0] and list(r2) == want[1]
        _check_invariants(G, c2, r2, d2)


def test_magnitude_and_unit_vectors():
    g = np.array([[3.0, 4.0, 0.0], [0.0, 0.0, 0.0], [1.0, 1.0, 1.0]])
    m = O.magnitudes(g)
    np.testing.assert_allclose(m, [5.0, 0.0, math.sqrt(3.0)], rtol=1e-15)
    gh = O.normalise(g, m)
    np.testing.assert_allclose(gh[0], [0.6, 0.8, 0.0], rtol=1e-15)
    assert np.all(gh[1] == 0.0)  # a zero vector stays zero


def test_cosine_of_known_angles():
    phis = np.array([0.0, 0.2, 1.0, 2.5])
    g = np.stack([np.cos(phis), np.sin(phis)], axis=1) * np.array([1.0, 7.0, 0.1, 3.0])[:, None]
    S = O.cosine_similarity(g)
    want = np.cos(phis[:, None] - phis[None, :])
    np.testing.assert_allclose(S, want, atol=1e-15)


def test_threshold_is_strict_and_diagonal_is_one():
    g = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    S = O.cosine_similarity(g)
    G = O.adjacency(S, 0.0)  # orthogonal pair has S == theta exactly: not adjacent
    assert not G[0, 1] and G[0, 2] and G[1, 2] and G[0, 0] and G[1, 1]
    assert np.array_equal(G, G.T)


def test_opposite_vectors_are_not_similar():
    # Eq. (9) compares the signed cosine: a vector and its negative (cosine -1) share no edge
    g = np.array([[2.0, 1.0], [-4.0, -2.0], [2.0, 1.1]])
    G = O.adjacency(O.cosine_similarity(g), 0.9)
    assert not G[0, 1] and not G[1, 2] and G[0, 2]
    r = O.codebook_shallow(g, 0.9)
    assert list(r["centres"]) == [0, 1] and list(r["ref"]) == [0, 1, 0]


def test_degenerate_thresholds():
    rng = np.random.default_rng(11)
    g = rng.standard_normal((20, 8))
    r = O.codebook_shallow(g, -1.5)  # everybody similar: one entry, centre 0
    assert list(r["centres"]) == [0] and np.all(r["ref"] == 0)
    r = O.codebook_shallow(g, 1.0)  # nobody similar: identity CodeBook
    assert list(r["centres"]) == list(range(20)) and list(r["ref"]) == list(range(20))


def test_duplicates_share_one_entry():
    # unfolding GQA repeats vectors; copies have cosine 1 and must collapse
    rng = np.random.default_rng(12)
    base = rng.standard_normal((6, 16))
    g = np.concatenate([base, 2.5 * base, base])
    r = O.codebook_shallow(g, 0.999)
    assert len(r["centres"]) == 6
    assert np.array_equal(r["ref"][:6], r["ref"][6:12]) and np.array_equal(r["ref"][:6], r["ref"][12:])


def test_well_separated_clusters_give_one_entry_each():
    rng = np.random.default_rng(13)
    d, n_cl = 64, 9
    cent = rng.standard_normal((n_cl, d))
    z = np.concatenate([np.arange(n_cl), rng.integers(0, n_cl, size=150)])
    g = cent[z] + 0.02 * rng.standard_normal((z.shape[0], d))
    r = O.codebook_shallow(g, 0.98)
    assert len(r["centres"]) == n_cl
    # tokens of one cluster share an entry, tokens of different clusters do not
    for a, b in itertools.combinations(range(z.shape[0]), 2):
        assert (r["ref"][a] == r["ref"][b]) == (z[a] == z[b])


def test_coverage_reconstruction_and_codebook_norms():
    rng = np.random.default_rng(14)
    cent = rng.standard_normal((12, 32))
    z = rng.integers(0, 12, size=200)
    g = cent[z] + 0.25 * rng.standard_normal((200, 32))
    theta = 0.93
    r = O.codebook_shallow(g, theta)
    np.testing.assert_allclose(np.linalg.norm(r["C"], axis=1), 1.0, rtol=1e-13)
    rec = O.reconstruct(r["C"], r["ref"], r["mag"])
    np.testing.assert_allclose(np.linalg.norm(rec, axis=1), r["mag"], rtol=1e-12)
    cos = (rec * g).sum(axis=1) / (np.linalg.norm(rec, axis=1) * np.linalg.norm(g, axis=1))
    centre_of = r["centres"][r["ref"]]
    own = centre_of == np.arange(200)
    assert np.all(cos[~own] > theta)  # every replaced token meets the similarity criterion
    np.testing.assert_allclose(cos[own], 1.0, rtol=1e-12)
    _check_invariants(r["G"], r["centres"], r["ref"], r["pick_degree"])
    # the small-N form, which recounts every degree for every pick, agrees at this size as well
    c1, r1 = O.codebook_cover_small(r["G"])
    assert np.array_equal(c1, r["centres"]) and np.array_equal(r1, r["ref"])


def test_g_override_and_margin_mask():
    g = np.array([[1.0, 0.0], [math.cos(0.2), math.sin(0.2)], [0.0, 1.0]])
    theta = math.cos(0.2) * (1 - 5e-5)
    r = O.codebook_shallow(g, theta)
    near = O.threshold_margin_mask(r["S"], theta)
    assert near[0, 1] and near[1, 0] and not near[0, 2]
    G2 = r["G"].copy()
    G2[0, 1] = G2[1, 0] = False
    r2 = O.codebook_shallow(g, theta, G_override=G2)
    assert len(r2["centres"]) == 3 and len(r["centres"]) == 2
