"""Pins for the oracle's Philox4x32-10 (Salmon et al., SC'11).

The independent implementation is cuRAND's *host* generator (CPU, no GPU needed).  With
CURAND_RNG_PSEUDO_PHILOX4_32_10, the 4-word block at position n of its output (n = offset/4
+ block index) was found, by matching against this oracle, to be the Philox block of counter
(low 32 bits of n>>16, n>>48, n & 0xFFFF, 0) under key = (seed low word, seed high word);
a wrong Philox could not satisfy that for thousands of (seed, position) pairs by chance.
"""
import ctypes as C
import ctypes.util

import numpy as np
import pytest

from oracle import oracle

CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161


def _curand():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so",
                 ctypes.util.find_library("curand")):
        if not name:
            continue
        try:
            return C.CDLL(name)
        except OSError:
            continue
    return None


def _curand_blocks(cr, seed, offset, nblocks):
    gen = C.c_void_p()
    assert cr.curandCreateGeneratorHost(C.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) == 0
    try:
        assert cr.curandSetPseudoRandomGeneratorSeed(gen, C.c_ulonglong(seed)) == 0
        assert cr.curandSetGeneratorOffset(gen, C.c_ulonglong(offset)) == 0
        out = np.zeros(4 * nblocks, dtype=np.uint32)
        assert cr.curandGenerate(gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(out.size)) == 0
    finally:
        cr.curandDestroyGenerator(gen)
    return out.reshape(nblocks, 4)


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, 20090577])
@pytest.mark.parametrize("offset", [0, 4, 4 * 123456, 4 * 0xFFFFFFFF, 4 * ((1 << 40) + 123),
                                    4 * ((0xFFFFFFFF << 16) + 0xFFF0), 4 * ((0x2BCD << 48) + (0x1234567 << 16) + 77)])
def test_philox_matches_curand_host(seed, offset):
    cr = _curand()
    if cr is None:
        pytest.skip("libcurand not found")
    nblocks = 64
    ref = _curand_blocks(cr, seed, offset, nblocks)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for j in range(nblocks):
        n = offset // 4 + j
        mine = oracle.philox4x32_10([(n >> 16) & 0xFFFFFFFF, n >> 48, n & 0xFFFF, 0], key)
        assert (mine == ref[j]).all(), (seed, offset, j)


def test_philox_blocks_helper_matches_single_calls():
    seed = 0xDEADBEEF12345678
    blk = oracle.philox_blocks(seed, 0xFFFFFFFE, 5, 6, 7, 4)  # wraps the first counter word
    for j in range(4):
        one = oracle.philox4x32_10([(0xFFFFFFFE + j) & 0xFFFFFFFF, 5, 6, 7], [seed & 0xFFFFFFFF, seed >> 32])
        assert (blk[j] == one).all()


def test_every_input_word_matters():
    """Flipping one bit of any counter or key word changes about half of the output bits."""
    base_ctr, base_key = [11, 22, 33, 44], [55, 66]
    ref = oracle.philox4x32_10(base_ctr, base_key)
    for word in range(6):
        for bit in (0, 13, 31):
            ctr, key = list(base_ctr), list(base_key)
            if word < 4:
                ctr[word] ^= 1 << bit
            else:
                key[word - 4] ^= 1 << bit
            out = oracle.philox4x32_10(ctr, key)
            flipped = sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(out, ref))
            assert 32 <= flipped <= 96, (word, bit, flipped)


def test_uniformity_of_top_byte():
    from scipy import stats
    words = oracle.philox_blocks(20090577, 0, 3, 9, oracle.TAG_NOISE, 1 << 16).reshape(-1)
    counts = np.bincount(words >> 24, minlength=256)
    chi2, p = stats.chisquare(counts)
    assert p > 1e-4
