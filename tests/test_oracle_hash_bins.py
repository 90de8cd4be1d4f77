"""Pins for the oracle's jitter hash, tick conversion and histogram bins."""
import numpy as np
import pytest

from oracle import lib, NBINS
from helpers import read_golden

L = lib()
M32 = 0xFFFFFFFF


def test_hash_golden_vectors():
    for seed, i, j, h, d6000, d2500 in read_golden("hash_vectors.txt"):
        hv = L.orc_hash(int(seed, 16), int(i), int(j))
        assert hv == int(h, 16)
        assert L.orc_jitter(hv, 6000) == int(d6000)
        assert L.orc_jitter(hv, 2500) == int(d2500)


def _unxorshift(x, s):
    y = x
    for _ in range(32 // s + 1):
        y = x ^ (y >> s)
    return y & M32


def test_mix_is_the_stated_bijection():
    # invert the finaliser step by step: if any shift or multiplier in the oracle were different
    # from the written definition, this inverse would not undo it
    inv1, inv2 = pow(0xA54FF53B, -1, 1 << 32), pow(0x510E527F, -1, 1 << 32)
    rng = np.random.default_rng(7)
    for x in [0, 1, M32, 0x80000000] + [int(v) for v in rng.integers(0, 1 << 32, size=2000)]:
        y = L.orc_mix(x)
        y = _unxorshift(y, 16); y = (y * inv2) & M32
        y = _unxorshift(y, 15); y = (y * inv1) & M32
        y = _unxorshift(y, 16)
        assert y == x
    assert L.orc_mix(0) == 0 and L.orc_mix(1) == 0x9A6B0037 and L.orc_mix(M32) == 0x5037B341


def test_hash_statistics():
    n = 100_000
    h = np.array([L.orc_hash(3, 5, j) for j in range(n)], dtype=np.uint64)
    u = h / 2.0 ** 32
    assert abs(u.mean() - 0.5) < 0.005
    counts = np.bincount((h >> 24).astype(np.int64), minlength=256)
    chi2 = ((counts - n / 256) ** 2 / (n / 256)).sum()
    assert chi2 < 330          # chi-square(255): mean 255, sd 22.6
    assert abs(np.corrcoef(u[:-1], u[1:])[0, 1]) < 0.01
    # token, request and seed each change the stream
    a = [L.orc_hash(0, 0, j) for j in range(64)]
    assert a != [L.orc_hash(0, 1, j) for j in range(64)]
    assert a != [L.orc_hash(1, 0, j) for j in range(64)]
    assert a != [L.orc_hash(1 << 32, 0, j) for j in range(64)]
    assert len(set(a)) == 64


def test_hash_avalanche():
    rng = np.random.default_rng(11)
    flips = []
    for _ in range(300):
        i, j = int(rng.integers(0, 1 << 24)), int(rng.integers(1, 8192))
        b = int(rng.integers(0, 13))
        flips.append(bin(L.orc_hash(9, i, j) ^ L.orc_hash(9, i, j ^ (1 << b))).count("1"))
    assert 14.5 < np.mean(flips) < 17.5


@pytest.mark.parametrize("J", [0, 1, 2, 2500, 6000, 100000])
def test_jitter_range(J):
    rng = np.random.default_rng(J)
    hs = [0, M32, 0x7FFFFFFF, 0x80000000] + [int(v) for v in rng.integers(0, 1 << 32, size=20000)]
    d = np.array([L.orc_jitter(h, J) for h in hs])
    assert d.min() >= -J and d.max() <= J
    assert L.orc_jitter(0, J) == -J and L.orc_jitter(M32, J) == J
    if J == 0:
        assert (d == 0).all()
    if J == 2:                       # all 5 values occur about equally often
        c = np.bincount(d[4:] + 2, minlength=5)
        assert c.min() > 0.18 * 20000 and c.max() < 0.22 * 20000
    if J >= 2500:
        assert abs(d[4:].mean()) < 0.03 * J


def test_tick_table_of_the_workloads():
    f = np.float32
    assert L.orc_seconds_to_ticks(f(0.030)) == 30000
    assert L.orc_seconds_to_ticks(f(1.0)) == 1_000_000
    assert L.orc_rate_to_ticks(f(500.0)) == 2000 and L.orc_rate_to_ticks(f(20.0)) == 50000
    assert L.orc_rate_to_ticks(f(1500.0)) == 667 and L.orc_rate_to_ticks(f(40.0)) == 25000
    assert L.orc_rate_to_ticks(f(200.0)) == 5000 and L.orc_rate_to_ticks(f(10.0)) == 100000
    assert L.orc_rate_to_ticks(f(5.0)) == 200000
    # halves round to even
    assert L.orc_rate_to_ticks(f(400000.0)) == 2      # 2.5
    assert L.orc_rate_to_ticks(f(4000000.0 / 7.0)) in (1, 2) and L.orc_rate_to_ticks(f(2.0e6 / 11.0)) in (5, 6)
    assert L.orc_seconds_to_ticks(f(0.5e-6)) == 0 and L.orc_seconds_to_ticks(f(1.5e-6)) == 2


def test_bins_partition_the_axis():
    assert NBINS == 864
    prev = -1
    for b in range(NBINS):
        lo = L.orc_bin_lower_edge(b)
        assert lo > prev
        prev = lo
        assert L.orc_bin(lo) == b
        if b + 1 < NBINS:
            hi = L.orc_bin_lower_edge(b + 1)
            assert L.orc_bin(hi - 1) == b
            if b >= 32:
                assert (hi - lo) * 32 <= lo          # 32 bins per octave: width <= lo/32
    assert L.orc_bin(0) == 0 and L.orc_bin(31) == 31 and L.orc_bin(32) == 32 and L.orc_bin(64) == 64
    assert L.orc_bin(1 << 30) == 832 and L.orc_bin((1 << 31) - 1) == 863 and L.orc_bin(1 << 40) == 863
    assert L.orc_bin(200000) == L.orc_bin(196608) and L.orc_bin_lower_edge(L.orc_bin(200000)) == 196608


def test_bins_monotone_exhaustive():
    t = np.arange(0, 1 << 20, dtype=np.int64)
    b = np.array([L.orc_bin(int(v)) for v in t[::7]])
    assert (np.diff(b) >= 0).all()
    for e in range(5, 31):           # every power of two opens an octave of 32 bins
        assert L.orc_bin(1 << e) == 32 * (e - 4)
        assert L.orc_bin((1 << e) - 1) == 32 * (e - 4) - 1
