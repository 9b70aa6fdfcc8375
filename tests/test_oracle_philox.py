"""Pins for the oracle's random stream (no GPU needed).

The Philox words are checked against an implementation that is not ours: the cuRAND
host generator (CURAND_RNG_PSEUDO_PHILOX4_32_10), which runs on the CPU.  With generator
offset 0 its output word 4*t + k is word k of Philox4x32-10 on counter (0, 0, t, 0)
keyed by the 64-bit seed (observed from the library's output, not from its code).
"""
import ctypes
import ctypes.util

import numpy as np
import pytest

from oracle import cos_oracle as orc


def _curand():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so",
                 ctypes.util.find_library("curand")):
        if not name:
            continue
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


def _curand_words(lib, seed, count):
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0
    try:
        assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        out = np.zeros(count, dtype=np.uint32)
        assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(count)) == 0
    finally:
        lib.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFEDCBA9876543210, 0xFFFFFFFFFFFFFFFF])
def test_philox_words_match_curand_host_generator(seed):
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not present")
    T = 4096
    theirs = _curand_words(lib, seed, 4 * T)
    t = np.arange(T)
    zero = np.zeros(T, dtype=np.uint64)
    w = orc.philox4x32_10(zero, zero, t, zero, seed & 0xFFFFFFFF, seed >> 32)
    mine = np.stack(w, axis=1).reshape(-1)
    assert np.array_equal(mine, theirs)


def test_philox_is_a_bijection_on_small_counter_sets_and_key_sensitive():
    c = np.arange(1 << 14)
    z = np.zeros_like(c)
    a = np.stack(orc.philox4x32_10(c, z, z, z, 7, 9), axis=1)
    assert len({tuple(x) for x in a.tolist()}) == len(c)          # distinct counters, distinct blocks
    for args in ((z, c, z, z, 7, 9), (z, z, c, z, 7, 9), (z, z, z, c, 7, 9)):
        b = np.stack(orc.philox4x32_10(*args), axis=1)
        assert not np.array_equal(a[1:], b[1:])                    # each counter lane matters
    b = np.stack(orc.philox4x32_10(c, z, z, z, 8, 9), axis=1)
    d = np.stack(orc.philox4x32_10(c, z, z, z, 7, 10), axis=1)
    assert not np.array_equal(a, b) and not np.array_equal(a, d)   # each key word matters


def test_uniform_mapping_is_open_interval_lattice():
    w = np.array([0, 1, 511, 512, 0xFFFFFFFF, 0x80000000], dtype=np.uint32)
    u = orc.word_to_uniform(w)
    assert u[0] == 2.0 ** -24 and u[1] == 2.0 ** -24 and u[2] == 2.0 ** -24
    assert u[3] == 3 * 2.0 ** -24
    assert u[4] == 1.0 - 2.0 ** -24
    assert u[5] == 0.5 + 2.0 ** -24
    assert np.all(u > 0) and np.all(u < 1)
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)   # exact in fp32


def test_position_uniforms_counter_layout_and_sharding():
    seed, off = 0xA5A5A5A55A5A5A5A, (3 << 32) | 17
    ua, us = orc.position_uniforms(seed, off, rows=6, positions=4)
    # element (b, j) must be the words of counter (b, j, off_lo, off_hi)
    for b in range(6):
        for j in range(4):
            w = orc.philox4x32_10([b], [j], [off & 0xFFFFFFFF], [off >> 32], seed & 0xFFFFFFFF, seed >> 32)
            assert ua[b, j] == orc.word_to_uniform(w[0])[0]
            assert us[b, j] == orc.word_to_uniform(w[1])[0]
    # a shard that starts at global row 2 sees the same numbers as rows 2.. of the full batch
    ua2, us2 = orc.position_uniforms(seed, off, rows=4, positions=4, row_base=2)
    assert np.array_equal(ua2, ua[2:]) and np.array_equal(us2, us[2:])
    # a different offset gives a different stream
    ub, _ = orc.position_uniforms(seed, off + 1, rows=6, positions=4)
    assert not np.array_equal(ua, ub)


def test_uniforms_are_uniform_chi_squared():
    ua, us = orc.position_uniforms(1234567, 0, rows=125000, positions=8)     # 1e6 draws each
    for u in (ua.ravel(), us.ravel()):
        counts, _ = np.histogram(u, bins=256, range=(0.0, 1.0))
        expected = len(u) / 256
        chi2 = float(np.sum((counts - expected) ** 2 / expected))
        # 255 d.o.f.: mean 255, sd ~22.6; 6 sd window
        assert 255 - 6 * 22.6 < chi2 < 255 + 6 * 22.6
        assert abs(u.mean() - 0.5) < 5 * (1 / np.sqrt(12 * len(u)))
    # the two words are not the same stream
    assert abs(np.corrcoef(ua.ravel(), us.ravel())[0, 1]) < 0.01
