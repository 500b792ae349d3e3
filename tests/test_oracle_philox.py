"""Pins for the oracle's sample-index stream (not GPU).

The stream is Philox4x32-10 (Salmon et al., SC'11). It is pinned to (a) the published
known-answer vectors and (b) an independent library implementation: cuRAND's *host*
generator of the same algorithm, which runs on the CPU. Then the index mapping
floor(u * m / 2^32) is checked by range, by an exact integer re-derivation with Python
big integers, by chunking independence and by a chi-square uniformity test.
"""
import ctypes
import os

import numpy as np
import pytest

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def _kat():
    rows = []
    with open(os.path.join(HERE, "golden", "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            v = [int(t, 16) for t in line.split()]
            rows.append((v[0:4], v[4:6], v[6:10]))
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) == 3
    for ctr, key, out in rows:
        got = oracle.philox4x32_10(ctr, key)
        assert [int(x) for x in got] == out


def _curand_host(seed, n):
    try:
        lib = ctypes.CDLL("libcurand.so.10")
    except OSError:
        try:
            lib = ctypes.CDLL("/usr/local/cuda/lib64/libcurand.so.10")
        except OSError:
            pytest.skip("cuRAND not found")
    g = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(g), 161) != 0:  # CURAND_RNG_PSEUDO_PHILOX4_32_10
        pytest.skip("cuRAND host generator unavailable")
    assert lib.curandSetPseudoRandomGeneratorSeed(g, ctypes.c_ulonglong(seed)) == 0
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(g, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
    lib.curandDestroyGenerator(g)
    return out


@pytest.mark.parametrize("seed", [0, 1, 0x123456789ABCDEF1])
def test_philox_matches_curand_host_generator(seed):
    """cuRAND's host Philox4_32_10 emits, for stream position p, output word p%4 of the block
    with counter (p / (4*65536), 0, (p/4) % 65536, 0) and key = the 64-bit seed. That exercises
    counter words 0 and 2 and both key words, the ones the sample stream uses."""
    S = 65536
    o = _curand_host(seed, 4 * S * 2 + 64)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for ctr0, node in [(0, 0), (0, 1), (0, 2), (0, 777), (0, 65535), (1, 0), (1, 3), (1, 40000), (2, 0), (2, 15)]:
        p = 4 * (ctr0 * S + node)
        want = o[p:p + 4]
        got = oracle.philox4x32_10([ctr0, 0, node, 0], key)
        assert np.array_equal(got, want), (ctr0, node)
    # and through the index function itself: with m = 2^32 the index is the raw word
    m = 1 << 32
    for node in (0, 5, 1023):
        idx = oracle.sample_indices(seed, node, m - 1, 0, 8)
        raw = np.concatenate([o[4 * node:4 * node + 4], o[4 * (S + node):4 * (S + node) + 4]]).astype(np.uint64)
        assert np.array_equal(idx.astype(np.uint64), (raw * np.uint64(m - 1)) >> np.uint64(32))


def test_index_mapping_exact_and_in_range():
    seed, node = 0xDEADBEEFCAFE, 11
    for m in (1, 2, 3, 1000, 4096, 65537, (1 << 32) - 1):
        idx = oracle.sample_indices(seed, node, m, 0, 1000)
        assert idx.max() < m
        for n in (1, 2, 3, 4, 5, 8, 9, 1000):
            q = (n - 1) >> 2
            word = int(oracle.philox4x32_10([q & 0xFFFFFFFF, q >> 32, node, 0],
                                            [seed & 0xFFFFFFFF, seed >> 32])[(n - 1) & 3])
            assert int(idx[n - 1]) == (word * m) >> 32


def test_index_stream_is_chunking_independent():
    a = oracle.sample_indices(7, 3, 8192, 0, 5000)
    b = np.concatenate([oracle.sample_indices(7, 3, 8192, 0, 1), oracle.sample_indices(7, 3, 8192, 1, 2),
                        oracle.sample_indices(7, 3, 8192, 3, 1234), oracle.sample_indices(7, 3, 8192, 1237, 3763)])
    assert np.array_equal(a, b)
    # different nodes and seeds give different streams
    assert not np.array_equal(a, oracle.sample_indices(7, 4, 8192, 0, 5000))
    assert not np.array_equal(a, oracle.sample_indices(8, 3, 8192, 0, 5000))


def test_index_stream_uniform_chi_square():
    m, n = 64, 256000
    idx = oracle.sample_indices(0, 0, m, 0, n)
    counts = np.bincount(idx, minlength=m).astype(np.float64)
    chi2 = ((counts - n / m) ** 2 / (n / m)).sum()
    # 63 degrees of freedom: mean 63, sd ~11.2; 130 is ~6 sd
    assert chi2 < 130.0
    # serial correlation of consecutive draws
    a = idx[:-1].astype(np.float64) - idx.mean()
    b = idx[1:].astype(np.float64) - idx.mean()
    assert abs((a * b).mean() / idx.var()) < 0.01


def test_invalid_arguments_rejected():
    with pytest.raises(ValueError):
        oracle.sample_indices(0, 0, 0, 0, 4)
    with pytest.raises(ValueError):
        oracle.sample_indices(0, 0, 1 << 33, 0, 4)
