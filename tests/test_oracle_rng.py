"""Pins for the oracle's random numbers and log-sum-exp (CPU only)."""
import math

import numpy as np
import scipy.special
import scipy.stats

import oracle


def test_philox_known_answers():
    # Known-answer vectors of Philox4x32-10 as published with the generator
    # (Salmon et al., SC'11, reference test vectors): counter, key -> output.
    kat = [
        ([0, 0, 0, 0], [0, 0], [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]),
        ([0xFFFFFFFF] * 4, [0xFFFFFFFF] * 2, [0x408F276D, 0x41C83B0E, 0xA20BC7C6, 0x6D5451FD]),
        ([0x243F6A88, 0x85A308D3, 0x13198A2E, 0x03707344], [0xA4093822, 0x299F31D0],
         [0xD16CFE09, 0x94FDCCEB, 0x5001E420, 0x24126EA1]),
    ]
    for ctr, key, want in kat:
        assert oracle.philox4x32_10(ctr, key) == want


def test_philox_is_a_bijection_on_a_sample():
    outs = {tuple(oracle.philox4x32_10([i, 7, 3, 1], [5, 9])) for i in range(4096)}
    assert len(outs) == 4096


def test_uniform_lattice_and_law():
    u = np.array([oracle.uniform(11, s, b, j) for s in range(40) for b in range(40) for j in range(1, 8)])
    assert u.min() >= 0.0 and u.max() <= 1.0 - 2.0 ** -24
    k = u * 2.0 ** 24
    assert np.all(k == np.round(k))           # on the 2^-24 lattice
    assert scipy.stats.kstest(u, "uniform").pvalue > 1e-3
    # distinct counters give distinct draws (no reuse across slot / step / position)
    assert len(np.unique(u)) > 0.999 * len(u)


def test_uniform_depends_on_every_counter_field():
    base = oracle.uniform(1, 2, 3, 4)
    assert base != oracle.uniform(2, 2, 3, 4)
    assert base != oracle.uniform(1, 3, 3, 4)
    assert base != oracle.uniform(1, 2, 4, 4)
    assert base != oracle.uniform(1, 2, 3, 5)
    assert base != oracle.uniform(1 + (1 << 32), 2, 3, 4)   # high key word is used


def test_gumbel_law_and_streams():
    g = np.array([oracle.gumbel(3, 1, 0, oracle.TAG_PROPOSE, 2, i) for i in range(20000)])
    assert scipy.stats.kstest(g, "gumbel_r").pvalue > 1e-3
    assert abs(g.mean() - 0.5772156649) < 0.03
    # range implied by u' in [2^-25, 1 - 2^-25]
    assert g.min() > -math.log(-math.log(2.0 ** -25)) - 1e-9
    assert g.max() < -math.log(-math.log1p(-2.0 ** -25)) + 1e-9
    # different tags / positions are different streams
    a = [oracle.gumbel(3, 1, 0, oracle.TAG_FINAL, 2, i) for i in range(64)]
    b = [oracle.gumbel(3, 1, 0, oracle.TAG_PROPOSE, 2, i) for i in range(64)]
    c = [oracle.gumbel(3, 1, 0, oracle.TAG_PROPOSE, 3, i) for i in range(64)]
    assert a != b and b != c


def test_gumbel_uses_four_words_per_counter():
    # indices 4k..4k+3 share a Philox counter (lane = i // 4), word = i % 4
    key = [3, 0]
    for i in (0, 5, 1023):
        words = oracle.philox4x32_10([i // 4, 9, 2, (oracle.TAG_PROPOSE << 16) | 1], key)
        u = ((words[i % 4] >> 8) + 0.5) * 2.0 ** -24
        assert oracle.gumbel(3, 9, 2, oracle.TAG_PROPOSE, 1, i) == -math.log(-math.log(u))


def test_logsumexp_against_scipy():
    rng = np.random.default_rng(0)
    for scale in (0.1, 3.0, 50.0, 700.0):
        row = rng.normal(0, scale, 5000)
        assert math.isclose(oracle.logsumexp(row), scipy.special.logsumexp(row), rel_tol=1e-13, abs_tol=1e-12)
    row = np.array([-np.inf, 0.0, -np.inf, 1.0])
    assert math.isclose(oracle.logsumexp(row), math.log(1 + math.e), rel_tol=1e-14)
    assert oracle.logsumexp(np.full(7, -np.inf)) == -np.inf
