"""Pins of the oracle's counter-based generator and Gumbel-max sampler."""
import math

import numpy as np
import pytest
import scipy.stats

import oracle


def _kat(golden_dir):
    rows = []
    for line in open(golden_dir + "/philox4x32_10_kat.txt"):
        if line.strip() and not line.startswith("#"):
            v = [int(t, 16) for t in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


def _philox_py(ctr, key):
    """Second, independent write-up in Python integers."""
    c, k = list(ctr), list(key)
    for r in range(10):
        p0, p1 = 0xD2511F53 * c[0], 0xCD9E8D57 * c[2]
        c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
        k = [(k[0] + 0x9E3779B9) & 0xFFFFFFFF, (k[1] + 0xBB67AE85) & 0xFFFFFFFF]
    return c


def test_philox_known_answers(golden_dir):
    rows = _kat(golden_dir)
    assert len(rows) == 3
    for ctr, key, want in rows:
        assert list(oracle.philox(ctr, key)) == want
        assert _philox_py(ctr, key) == want


def test_philox_matches_python_writeup_on_random_counters():
    rng = np.random.default_rng(0)
    for _ in range(200):
        ctr = [int(v) for v in rng.integers(0, 2**32, 4)]
        key = [int(v) for v in rng.integers(0, 2**32, 2)]
        assert list(oracle.philox(ctr, key)) == _philox_py(ctr, key)


def test_gumbel_map():
    for r in (0, 1, 12345, 2**31, 2**32 - 1):
        u = (r + 0.5) / 2**32
        assert oracle.gumbel_of(r) == pytest.approx(-math.log(-math.log(u)), rel=1e-15)
    assert math.isfinite(oracle.gumbel_of(0)) and math.isfinite(oracle.gumbel_of(2**32 - 1))
    # range of the variate for 32-bit words
    assert oracle.gumbel_of(0) == pytest.approx(-math.log(32 * math.log(2) - math.log(0.5)), rel=1e-12)
    assert oracle.gumbel_of(2**32 - 1) == pytest.approx(33 * math.log(2), abs=1e-6)


@pytest.mark.parametrize("V", [40, 96])
def test_sampler_distribution_chi_square(V):
    # V = 96: three full groups; V = 40: one full group and a short tail group
    rng = np.random.default_rng(V)
    x = (rng.standard_normal((1, V)) * 1.5).astype(np.float32)
    x[0, 3] += 2.0
    x[0, V - 1] += 1.0
    p = oracle.softmax_row(x, 0)
    N = 60000
    counts = np.zeros(V)
    for s in range(N // 4):
        for j in range(4):                      # the four draws of one counter are independent
            counts[oracle.sample_row(x, 0, 1234, 0, s, 1, j)] += 1
    chi2 = ((counts - N * p) ** 2 / (N * p)).sum()
    # 99.9% quantile; a wrong group weight or a dropped element shifts chi2 by thousands
    assert chi2 < scipy.stats.chi2.ppf(0.999, V - 1)


def test_sampler_determinism_and_streams():
    rng = np.random.default_rng(5)
    x = (rng.standard_normal((4, 64)) * 2).astype(np.float32)
    a = [oracle.sample_row(x, r, 7, r, 3, 1, 0) for r in range(4) for _ in range(2)]
    assert a[0::2] == a[1::2]
    base = [oracle.sample_row(x, 0, 7, 0, s, 1, 0) for s in range(64)]
    assert len(set(base)) > 8                                    # steps give fresh draws
    assert base != [oracle.sample_row(x, 0, 8, 0, s, 1, 0) for s in range(64)]   # seed matters
    assert base != [oracle.sample_row(x, 0, 7, 1, s, 1, 0) for s in range(64)]   # row matters
    assert base != [oracle.sample_row(x, 0, 7, 0, s, 0, 0) for s in range(64)]   # domain matters


def test_sampler_respects_masked_tokens_and_peaks():
    x = np.full((1, 70), -np.inf, np.float32)
    x[0, [2, 40, 69]] = [0.0, 1.0, 0.5]
    seen = {oracle.sample_row(x, 0, 1, 0, s, 1, 0) for s in range(400)}
    assert seen == {2, 40, 69}
    x = np.zeros((1, 70), np.float32)
    x[0, 33] = 60.0
    assert {oracle.sample_row(x, 0, 1, 0, s, 1, 0) for s in range(200)} == {33}


def test_strict_sampled_equals_plain_sampled_decoding():
    # sample-and-match: the accepted prefix is exactly where the drafts equal the tokens a
    # plain sampled decode of the same rows (same seed, step, row) would emit
    rng = np.random.default_rng(9)
    V, L, C = 48, 5, 12
    x = (rng.standard_normal((C * L, V)) * 0.7).astype(np.float32)
    x[np.arange(C * L), rng.integers(0, V, C * L)] += 4.0
    own = np.array([oracle.sample_row(x, r, 42, r, 6, 1, 0) for r in range(C * L)])
    d = np.where(rng.random(C * L) < 0.7, own, rng.integers(0, V, C * L))
    out = oracle.verify(x, d, np.arange(0, C * L + 1, L), mode=oracle.VERIFY_STRICT_SAMPLED,
                        seed=42, step=6)
    assert np.array_equal(out["sampled"], own)
    for c in range(C):
        a = 0
        while a < L and d[c * L + a] == own[c * L + a]:
            a += 1
        assert out["accept_len"][c] == a
        assert out["next_token"][c] == (own[c * L + a] if a < L else -1)
