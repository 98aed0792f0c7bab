"""Pins for the checker's decode-time attention over the replaced cache (Eq. (14) with the rotary embedding of
Eq. (1) re-applied, Section 3.4): the identities of the rotation, a scalar brute force, an independent
complex-number formulation, the identity CodeBook (theta >= 1) against plain attention, and closed forms."""
import cmath
import math

import numpy as np
import torch

from oracle import spindlekv_oracle as O


def test_rotation_keeps_norms_is_the_identity_at_position_zero_and_composes():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((7, 16))
    pos = np.array([0, 1, 5, 100, 4095, 16383, 3])
    y = O.rope(x, pos)
    np.testing.assert_allclose(np.linalg.norm(y, axis=1), np.linalg.norm(x, axis=1), rtol=1e-12)
    np.testing.assert_allclose(y[0], x[0], rtol=0, atol=0)                        # angle 0
    np.testing.assert_allclose(O.rope(O.rope(x, pos), 2 * pos + 7), O.rope(x, 3 * pos + 7), atol=1e-9)


def test_score_depends_on_the_distance_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal(32), rng.standard_normal(32)
    want = float(O.rope(q[None], [10])[0] @ O.rope(k[None], [3])[0])
    for shift in (1, 50, 9000):
        got = float(O.rope(q[None], [10 + shift])[0] @ O.rope(k[None], [3 + shift])[0])
        assert abs(got - want) < 1e-9
    assert abs(float(O.rope(q[None], [11])[0] @ O.rope(k[None], [3])[0]) - want) > 1e-3   # and it does depend on it


def test_pairing_and_direction_of_the_rotation():
    # d = 4, base 10000: omega = [1, 0.01].  The unit vector along element 0 at position p turns into
    # (cos p, 0, sin p, 0): element 0 is paired with element 2 (= 0 + d/2), counter-clockwise.
    p = 0.5
    y = O.rope(np.array([[1.0, 0.0, 0.0, 0.0]]), [p])[0]
    np.testing.assert_allclose(y, [math.cos(p), 0.0, math.sin(p), 0.0], atol=1e-15)
    y = O.rope(np.array([[0.0, 1.0, 0.0, 0.0]]), [p])[0]
    np.testing.assert_allclose(y, [0.0, math.cos(0.01 * p), 0.0, math.sin(0.01 * p)], atol=1e-15)
    np.testing.assert_allclose(O.rope_frequencies(8, 10000.0), [1.0, 0.1, 0.01, 0.001], rtol=1e-14)


def test_rotation_as_complex_multiplication():
    # an independent formulation: the pair (x_i, x_{i+d/2}) as a complex number times exp(i p omega_i)
    rng = np.random.default_rng(3)
    d = 12
    x = rng.standard_normal((5, d))
    pos = [0, 2, 17, 333, 8191]
    y = O.rope(x, pos, base=500000.0)
    for t, p in enumerate(pos):
        for i in range(d // 2):
            z = complex(x[t, i], x[t, i + d // 2]) * cmath.exp(1j * p * 500000.0 ** (-2.0 * i / d))
            assert abs(z.real - y[t, i]) < 1e-9 and abs(z.imag - y[t, i + d // 2]) < 1e-9


def _plain_attention(q, pos_q, K, V, positions, base):
    """Plain attention of rotated queries over rotated keys, scalar loops, written without the checker."""
    h_n, d = q.shape
    n = K.shape[0]
    half = d // 2
    def rot(x, p):
        out = [0.0] * d
        for i in range(half):
            a = p * base ** (-2.0 * i / d)
            out[i] = x[i] * math.cos(a) - x[i + half] * math.sin(a)
            out[i + half] = x[i + half] * math.cos(a) + x[i] * math.sin(a)
        return out
    Kr = [rot(K[t], positions[t]) for t in range(n)]
    out = np.zeros((h_n, d))
    for g in range(h_n):
        qr = rot(q[g], pos_q)
        s = [sum(qr[i] * Kr[t][i] for i in range(d)) / math.sqrt(d) for t in range(n)]
        mx = max(s)
        e = [math.exp(v - mx) for v in s]
        z = sum(e)
        for t in range(n):
            for i in range(d):
                out[g, i] += e[t] / z * V[t][i]
    return out


def test_identity_codebook_gives_plain_attention_scalar_brute_force():
    # theta >= 1: nobody is merged, C = unit rows, r = identity, m = norms; Eq. (14) then returns the cache itself
    rng = np.random.default_rng(4)
    n, d, h_n = 9, 8, 3
    K, V, q = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal((h_n, d))
    ck, cv = O.codebook_shallow(K, 1.0), O.codebook_shallow(V, 1.0)
    assert list(ck["ref"]) == list(range(n))
    positions = np.array([0, 1, 2, 5, 6, 9, 10, 11, 40])          # kept tokens keep their original positions
    got = O.decode_attention(q, 41, ck["C"], ck["ref"], ck["mag"], cv["C"], cv["ref"], cv["mag"], positions, base=100.0)
    want = _plain_attention(q, 41, K, V, positions, 100.0)
    np.testing.assert_allclose(got["out"], want, rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(got["A"].sum(axis=1), 1.0, rtol=1e-13)


def test_against_torch_softmax_on_a_merged_cache():
    rng = np.random.default_rng(5)
    n, d, h_n = 60, 16, 4
    cent = rng.standard_normal((6, d))
    z = rng.integers(0, 6, size=n)
    K = cent[z] + 0.05 * rng.standard_normal((n, d))
    V = cent[z][:, ::-1] + 0.05 * rng.standard_normal((n, d))
    q = rng.standard_normal((h_n, d))
    ck, cv = O.codebook_shallow(K, 0.98), O.codebook_shallow(V, 0.95)
    assert len(ck["centres"]) < n                                   # something was merged
    got = O.decode_attention(q, n, ck["C"], ck["ref"], ck["mag"], cv["C"], cv["ref"], cv["mag"])
    Kr = torch.from_numpy(O.rope(O.reconstruct(ck["C"], ck["ref"], ck["mag"]), np.arange(n)))
    qr = torch.from_numpy(O.rope(q, np.full(h_n, n)))
    A = torch.softmax(qr @ Kr.T / math.sqrt(d), dim=1)
    want = A @ torch.from_numpy(O.reconstruct(cv["C"], cv["ref"], cv["mag"]))
    np.testing.assert_allclose(got["out"], want.numpy(), rtol=1e-10, atol=1e-12)
    # the replaced cache is close to the real one: so is the output (cosine above theta bounds the error loosely)
    plain = _plain_attention(q, n, K, V, np.arange(n), 10000.0)
    assert np.abs(got["out"] - plain).max() < 0.5 * np.abs(plain).max()


def test_closed_forms():
    rng = np.random.default_rng(6)
    d, n = 8, 5
    # a zero query weighs every cached token equally: the output is the mean of the rebuilt values
    C_K, C_V = np.eye(d)[:3], np.eye(d)[:2]
    r_K, m_K = np.array([0, 1, 2, 1, 0]), rng.uniform(0.5, 2.0, n)
    r_V, m_V = np.array([0, 1, 1, 0, 0]), rng.uniform(0.5, 2.0, n)
    out = O.decode_attention(np.zeros((2, d)), 7, C_K, r_K, m_K, C_V, r_V, m_V)
    np.testing.assert_allclose(out["A"], 1.0 / n, rtol=1e-14)
    np.testing.assert_allclose(out["out"][0], (C_V[r_V] * m_V[:, None]).mean(axis=0), rtol=1e-13)
    # value magnitudes scale the output linearly, key magnitudes do not
    q = rng.standard_normal((2, d))
    a = O.decode_attention(q, 7, C_K, r_K, m_K, C_V, r_V, m_V)["out"]
    b = O.decode_attention(q, 7, C_K, r_K, m_K, C_V, r_V, 3.0 * m_V)["out"]
    c = O.decode_attention(q, 7, C_K, r_K, 3.0 * m_K, C_V, r_V, m_V)["out"]
    np.testing.assert_allclose(b, 3.0 * a, rtol=1e-12)
    assert np.abs(c - a).max() > 1e-3
    # one key far ahead of the rest takes all the weight: the output is that token's rebuilt value
    m_big = m_K.copy()
    m_big[3] = 400.0
    q1 = np.zeros((1, d))
    q1[0, 1] = 1.0                                     # along entry 1 at distance 0: rotate the query to the key's position
    o = O.decode_attention(q1, 3, C_K, r_K, m_big, C_V, r_V, m_V)
    assert o["A"][0, 3] > 1 - 1e-12
    np.testing.assert_allclose(o["out"][0], C_V[r_V[3]] * m_V[3], rtol=1e-10, atol=1e-12)
