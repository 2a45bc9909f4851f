"""Pins for the oracle's counter-based noise: published SplitMix64 vector, a double-precision
Box-Muller from libm, distribution tests and the special words of the normal map."""
import math
import os

import numpy as np
import pytest
from scipy import stats

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
M64 = (1 << 64) - 1


def _golden_vector():
    with open(os.path.join(GOLDEN, "splitmix64_seed1234567.txt")) as f:
        return [int(l) for l in f if l.strip() and not l.startswith("#")]


def test_splitmix64_published_vector():
    # the j-th word of a stream with key K is the j-th output of SplitMix64 seeded with K
    want = _golden_vector()
    got = [oracle.lib().oracle_stream_word(1234567, j) for j in range(len(want))]
    assert got == want


def test_mix64_is_a_bijection_on_a_sample():
    # xor-shift and odd multiplication are invertible; distinct inputs give distinct outputs
    xs = np.arange(1 << 16, dtype=np.uint64)
    ys = {oracle.lib().oracle_mix64(int(x)) for x in xs}
    assert len(ys) == xs.size


def test_stream_key_separates_every_field():
    L = oracle.lib()
    base = L.oracle_stream_key(3, 0, 0, 0, 0)
    keys = {base}
    for args in [(1, 0, 0, 0, 0), (3, 1, 0, 0, 0), (3, 0, 1, 0, 0), (3, 0, 0, 1, 0), (3, 0, 0, 0, 1),
                 (3, 0, 1, 0, 1), (3, 0, 0, 1, 1), (3, 0, 1, 1, 0), (3, 0, 2**40, 0, 0)]:
        keys.add(L.oracle_stream_key(*args))
    assert len(keys) == 10
    # field order matters: (t=1,k=0) and (t=0,k=1) differ, checked above; and it is a pure function
    assert base == L.oracle_stream_key(3, 0, 0, 0, 0)


def test_stream_key_is_five_absorptions():
    # consistency of the C integer arithmetic with unbounded-integer arithmetic (catches a
    # 32-bit truncation of t or j); the construction itself is this project's, not the paper's
    G = 0x9E3779B97F4A7C15

    def fin(s):
        s ^= s >> 30
        s = (s * 0xBF58476D1CE4E5B9) & M64
        s ^= s >> 27
        s = (s * 0x94D049BB133111EB) & M64
        return s ^ (s >> 31)

    def key(tag, seed, t, k, w):
        s = seed
        for v in (tag, t, k, w, 0):
            s = fin((s + G * (v + 1)) & M64)
        return s

    L = oracle.lib()
    for args in [(3, 0, 0, 0, 0), (5, 2**63 + 11, 2**40 + 3, 47, 31), (2, 7, 0, 0, 15)]:
        assert L.oracle_stream_key(*args) == key(*args)
    K = key(3, 0, 2, 5, 1)
    for j in (0, 1, 2**32 - 1, 2**32, 2**33 + 5):
        assert L.oracle_stream_word(K, j) == fin((K + G * (j + 1)) & M64)


def test_export_matches_single_word_calls_beyond_2_pow_32():
    j0 = (1 << 32) - 3
    words, z = oracle.stream(3, 9, 4, 2, 1, j0, 8)
    L = oracle.lib()
    K = L.oracle_stream_key(3, 9, 4, 2, 1)
    assert [int(w) for w in words] == [L.oracle_stream_word(K, j0 + i) for i in range(8)]
    # coordinate j takes output j & 1 of the pair made from word j >> 1
    for i in range(8):
        j = j0 + i
        pair = oracle.normal_pair(L.oracle_stream_word(K, j >> 1))
        assert z[i] == np.float32(pair[j & 1])
        assert z[i] == np.float32(L.oracle_stream_normal(K, j))


def _libm_box_muller(words):
    """Both Box-Muller outputs of each word in double precision: shape [n, 2]."""
    k1 = (words >> np.uint64(40)).astype(np.float64)
    k2 = ((words >> np.uint64(16)) & np.uint64(0xFFFFFF)).astype(np.float64)
    radius = np.sqrt(-2.0 * np.log((k1 + 1.0) / 2.0**24))
    angle = 2.0 * np.pi * k2 / 2.0**24
    return np.stack([radius * np.cos(angle), radius * np.sin(angle)], axis=1)


def test_normal_map_against_double_precision_box_muller():
    n = 1 << 20
    words, z = oracle.stream(3, 0, 0, 0, 0, 0, n)
    # coordinates 0..n-1 use words 0..n/2-1, cosine output first
    ref = _libm_box_muller(words[: n // 2]).reshape(-1)
    err = np.abs(z.astype(np.float64) - ref)
    # binary32 evaluation: a few ulp of a value below 6, plus series truncation < 1e-8
    assert err.max() < 2e-6, err.max()
    assert np.abs(z).max() <= math.sqrt(2 * 24 * math.log(2)) + 1e-5


def test_normal_map_against_libm_for_every_radius_field_and_every_angle_field():
    # exhaustive in each 24-bit field of the word (the other one fixed)
    all24 = np.arange(1 << 24, dtype=np.uint64)
    for words in (all24 << np.uint64(40), (np.uint64(0x000100) << np.uint64(40)) | (all24 << np.uint64(16))):
        got = oracle.words_to_normals(words).astype(np.float64)
        ref = _libm_box_muller(words)
        assert np.abs(got - ref).max() < 2e-6


def test_normal_map_special_words():
    def word(k1, k2):
        return (k1 << 40) | (k2 << 16)

    pair = oracle.normal_pair
    top = (1 << 24) - 1
    r_max = math.sqrt(2 * 24 * math.log(2))
    assert pair(word(top, 12345)) == (0.0, 0.0)                           # u1 = 1: radius 0
    for k2, c, s in ((0, 1, 0), (1 << 22, 0, 1), (1 << 23, -1, 0), (3 << 22, 0, -1)):
        got = pair(word(0, k2))                                           # u1 = 2^-24, axis angles
        assert abs(got[0] - c * r_max) < 1e-6 and abs(got[1] - s * r_max) < 1e-6, (k2, got)
    # odd multiples of pi/4: both outputs have magnitude r_max / sqrt(2)
    d = r_max * math.sqrt(0.5)
    for q, (c, s) in enumerate(((1, 1), (-1, 1), (-1, -1), (1, -1))):
        got = pair(word(0, (q << 22) + (1 << 21)))
        assert abs(got[0] - c * d) < 2e-6 and abs(got[1] - s * d) < 2e-6, (q, got)
    # just past pi/4 (reflected evaluation) in every quadrant
    for q in range(4):
        k2 = (q << 22) + (1 << 21) + 12345
        ang = 2 * math.pi * k2 / 2**24
        got = pair(word(0, k2))
        assert abs(got[0] - r_max * math.cos(ang)) < 2e-6 and abs(got[1] - r_max * math.sin(ang)) < 2e-6
    # low 16 bits of the word are unused
    assert pair(word(77, 99) | 0xFFFF) == pair(word(77, 99))


def test_pair_outputs_are_uncorrelated_and_jointly_normal():
    n = 1 << 20
    _, z = oracle.stream(3, 5, 1, 2, 0, 0, n)
    zc, zs = z[0::2].astype(np.float64), z[1::2].astype(np.float64)
    bound = 5.0 / math.sqrt(n // 2)
    assert abs(np.corrcoef(zc, zs)[0, 1]) < bound
    assert abs(np.corrcoef(zc**2, zs**2)[0, 1]) < bound   # independent, not merely uncorrelated
    # z_c^2 + z_s^2 = -2 ln u1 is exponential with mean 2
    r2 = zc**2 + zs**2
    assert stats.kstest(r2[: 1 << 17], "expon", args=(0, 2.0)).pvalue > 1e-3


def test_normal_and_uniform_distribution():
    n = 1 << 21
    words, z = oracle.stream(2, 0, 0, 0, 3, 0, n)
    z = z.astype(np.float64)
    assert abs(z.mean()) < 4.0 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 5.0 * math.sqrt(2.0 / n)
    assert stats.kstest(z[: 1 << 18], "norm").pvalue > 1e-3
    U = np.array([oracle.lib().oracle_word_to_unit(int(w)) for w in words[:4096]])
    top = (words[:4096] >> np.uint64(40)).astype(np.float64) / 2.0**24
    assert np.array_equal(U.astype(np.float64), top)          # exact 24-bit grid
    k1 = (words >> np.uint64(40)).astype(np.float64) / 2.0**24
    assert 0.0 <= k1.min() and k1.max() < 1.0
    assert abs(k1.mean() - 0.5) < 4.0 / math.sqrt(12 * n)
    assert stats.kstest(k1[: 1 << 18], "uniform").pvalue > 1e-3


def test_streams_are_uncorrelated_across_step_worker_and_coordinate():
    n = 1 << 18
    _, z0 = oracle.stream(3, 0, 0, 0, 0, 0, n)
    bound = 5.0 / math.sqrt(n)
    for args in [(3, 0, 0, 1, 0), (3, 0, 1, 0, 0), (3, 0, 0, 0, 1), (3, 1, 0, 0, 0), (2, 0, 0, 0, 0)]:
        _, z1 = oracle.stream(*args, 0, n)
        assert abs(np.corrcoef(z0, z1)[0, 1]) < bound, args
    assert abs(np.corrcoef(z0[:-1], z0[1:])[0, 1]) < bound   # neighbouring coordinates


def test_problem_data_generators():
    cfg = oracle.make_config(m=3, tau=1, T=1, a_lo=0.1, a_hi=1.0, c_std=0.05, sigma=0.25, seed=4)
    j = np.arange(20000)
    a = oracle.curvature(cfg, j).astype(np.float64)
    assert a.min() >= 0.1 - 1e-7 and a.max() < 1.0
    assert abs(a.mean() - 0.55) < 0.01
    # a_j = a_lo + (a_hi - a_lo) U with U the 24-bit uniform of the curvature stream
    words, _ = oracle.stream(oracle.TAG_CURVATURE, 4, 0, 0, 0, 0, 64)
    U = (words >> np.uint64(40)).astype(np.float64) / 2.0**24
    assert np.abs(a[:64] - (0.1 + 0.9 * U)).max() < 1e-7
    for w in range(3):
        c = oracle.centre(cfg, w, j[:4096]).astype(np.float64)
        _, z = oracle.stream(oracle.TAG_CENTRE, 4, 0, 0, w, 0, 4096)
        assert np.abs(c - 0.05 * z.astype(np.float64)).max() < 1e-8
        g = oracle.supplied_gradient(cfg, w, j[:4096]).astype(np.float64)
        _, z5 = oracle.stream(oracle.TAG_SUPPLIED, 4, 0, 0, w, 0, 4096)
        assert np.abs(g - 0.25 * z5.astype(np.float64)).max() < 1e-7
