"""Pins for the oracle's counter-based random numbers."""
import ctypes
import os

import numpy as np
import pytest

from oracle import rd_oracle as orc


def _load_kat():
    path = os.path.join(os.path.dirname(__file__), "golden", "philox4x32_10_kat.txt")
    rows = []
    for line in open(path):
        line = line.split("#")[0].strip()
        if not line:
            continue
        w = [int(t, 16) for t in line.split()]
        rows.append((w[0:4], w[4:6], w[6:10]))
    return rows


def test_philox_known_answers():
    rows = _load_kat()
    assert len(rows) >= 3
    for ctr, key, want in rows:
        got = orc.philox4x32_10(np.array(ctr, dtype=np.uint32), key)
        assert [int(x) for x in got] == want


def test_philox_vectorised_equals_scalar():
    rng = np.random.default_rng(1)
    ctr = rng.integers(0, 2**32, size=(17, 4), dtype=np.uint64).astype(np.uint32)
    key = (0x12345678, 0x9ABCDEF0)
    batch = orc.philox4x32_10(ctr, key)
    for i in range(17):
        assert np.array_equal(batch[i], orc.philox4x32_10(ctr[i], key))


def test_philox_matches_curand_host_generator():
    """cuRAND's host Philox4_32_10 generator (CPU only, no device) starts its stream at counter 0
    with the seed as key: its first four words are the block philox(ctr=0, key=seed)."""
    try:
        lib = ctypes.CDLL("libcurand.so.10")
    except OSError:
        try:
            lib = ctypes.CDLL("/usr/local/cuda/lib64/libcurand.so.10")
        except OSError:
            pytest.skip("libcurand not present")
    gen = ctypes.c_void_p()
    CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) != 0:
        pytest.skip("curand host generator unavailable")
    seed = 0x0123456789ABCDEF
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    out = (ctypes.c_uint32 * 4)()
    assert lib.curandGenerate(gen, out, ctypes.c_size_t(4)) == 0
    lib.curandDestroyGenerator(gen)
    want = orc.philox4x32_10(np.zeros(4, dtype=np.uint32), (seed & 0xFFFFFFFF, seed >> 32))
    assert sorted(int(x) for x in out) == sorted(int(x) for x in want)


def test_unit_interval_open_and_exact_in_float32():
    w = np.array([0, 1, 511, 512, 2**32 - 1], dtype=np.uint32)
    u = orc._unit_interval(w)
    assert u.min() > 0 and u.max() < 1
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)
    assert u[0] == 2.0 ** -24 and u[-1] == 1 - 2.0 ** -24


def test_init_state_moments_and_keys():
    z = orc.init_state(7, 0, 5, 40000, 1.0, np.float64)
    assert abs(z.mean()) < 0.02 and abs(z.std() - 1) < 0.02
    assert abs(np.mean(z ** 3)) < 0.05 and abs(np.mean(z ** 4) - 3) < 0.15
    # consecutive elements uncorrelated (catches a cos/cos or shared-angle slip)
    assert abs(np.corrcoef(z[0::2], z[1::2])[0, 1]) < 0.02
    assert abs(np.corrcoef(z[0::4], z[2::4])[0, 1]) < 0.03
    # a function of (seed, seq, pos) only; sigma scales
    assert np.array_equal(z[:64], orc.init_state(7, 0, 5, 64, 1.0, np.float64))
    assert not np.array_equal(z[:64], orc.init_state(7, 0, 6, 64, 1.0, np.float64))
    assert not np.array_equal(z[:64], orc.init_state(7, 1, 5, 64, 1.0, np.float64))
    assert not np.array_equal(z[:64], orc.init_state(8, 0, 5, 64, 1.0, np.float64))
    assert np.allclose(orc.init_state(7, 0, 5, 64, 0.5, np.float64), 0.5 * z[:64])


def test_gumbel_max_samples_the_softmax():
    """Gumbel-max is an exact sampler: empirical frequencies over many positions match softmax."""
    logits = np.array([0.0, 1.0, 2.0, -1.0, 0.5], dtype=np.float32)
    p = np.exp(logits - logits.max()); p /= p.sum()
    n = 20000
    counts = np.zeros(5)
    for t in range(n):
        counts[orc.sample_token(logits, 1.0, 3, 0, t)] += 1
    assert np.abs(counts / n - p).max() < 0.012
    # temperature sharpens
    c2 = np.zeros(5)
    for t in range(4000):
        c2[orc.sample_token(logits, 0.25, 3, 0, t)] += 1
    p2 = np.exp(4 * (logits - logits.max())); p2 /= p2.sum()
    assert np.abs(c2 / 4000 - p2).max() < 0.03


def test_greedy_lowest_index_on_ties():
    assert orc.sample_token(np.array([1.0, 3.0, 3.0, 2.0]), 0.0, 0, 0, 0) == 1
