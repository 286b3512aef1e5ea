"""Pins for the oracle's counter-based generator."""
import ctypes as C
import glob
import site

import numpy as np
import pytest

import oracle


def test_published_known_answers(golden):
    for row in golden("philox4x32_10_kat.txt")["kat"]:
        v = [int(x, 16) for x in row]
        c, k, want = v[0:4], v[4:6], v[6:10]
        got = oracle.philox(k[0], k[1], *c)
        assert [int(x) for x in got] == want


def test_counter_sensitivity():
    # every counter word and every key word changes the output
    base = oracle.philox(1, 2, 3, 4, 5, 6)
    for pos in range(6):
        args = [1, 2, 3, 4, 5, 6]
        args[pos] += 1
        assert not np.array_equal(base, oracle.philox(*args))


def _curand():
    for sp in site.getsitepackages():
        hits = glob.glob(sp + "/nvidia/curand/lib/libcurand.so*")
        if hits:
            return hits[0]
    return None


@pytest.mark.skipif(_curand() is None, reason="libcurand not present")
def test_against_curand_host_generator_first_block():
    # cuRAND's host PHILOX4_32_10 generator uses the 64-bit seed as the key and starts at
    # counter zero: its first four outputs are Philox(key = seed; counter = 0).
    L = C.CDLL(_curand())
    for seed in (0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, 160608495):
        gen = C.c_void_p()
        if L.curandCreateGeneratorHost(C.byref(gen), 161) != 0:
            pytest.skip("cuRAND host generator unavailable")
        assert L.curandSetPseudoRandomGeneratorSeed(gen, C.c_ulonglong(seed)) == 0
        out = np.zeros(4, dtype=np.uint32)
        assert L.curandGenerate(gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(4)) == 0
        L.curandDestroyGenerator(gen)
        mine = oracle.philox(seed & 0xFFFFFFFF, seed >> 32, 0, 0, 0, 0)
        assert np.array_equal(out, mine)


def test_uniformity_of_words():
    # 2^16 counters: each output word's top byte is uniform within 5 sigma
    n = 1 << 16
    top = np.zeros((4, 256), dtype=np.int64)
    for i in range(n):
        r = oracle.philox(7, 9, i, 0, 3, 0)
        for e in range(4):
            top[e, int(r[e]) >> 24] += 1
    exp = n / 256
    assert np.all(np.abs(top - exp) < 5 * np.sqrt(exp))
