"""Pins for the oracle's Philox4x32-10 and the minibatch index sampler (Algorithm 1, step 2)."""
import ctypes
import ctypes.util
import os

import numpy as np
import pytest

from oracle import dpsgd_oracle as orc

M0, M1 = 0xD2511F53, 0xCD9E8D57
MASK = 0xFFFFFFFF


def _load_curand():
    for name in ("/usr/local/cuda/lib64/libcurand.so", ctypes.util.find_library("curand")):
        if name and (os.path.exists(name) or "/" not in name):
            try:
                return ctypes.CDLL(name)
            except OSError:
                pass
    return None


def _curand_quads(lib, seed, offset, count):
    """`count` 32-bit outputs of cuRAND's HOST Philox4_32_10 generator, as rows of four."""
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0   # PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    buf = (ctypes.c_uint32 * count)()
    assert lib.curandGenerate(gen, buf, ctypes.c_size_t(count)) == 0
    lib.curandDestroyGenerator(gen)
    return np.frombuffer(buf, dtype=np.uint32).reshape(-1, 4).copy()


def test_philox_matches_curand_host_generator():
    """Library pin.  cuRAND's host generator emits, as its q-th group of four outputs, the
    Philox4x32-10 block with counter (q div 65536, 0, q mod 65536, 0) and key = seed."""
    lib = _load_curand()
    if lib is None:
        pytest.skip("libcurand not present")
    rng = np.random.default_rng(7)
    for seed in (0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, int(rng.integers(1, 2 ** 63))):
        quads = _curand_quads(lib, seed, 0, 4 * 65536 * 2)
        q = np.concatenate([np.arange(0, 300), rng.integers(0, 2 * 65536, 500)])
        mine = np.stack(orc.philox4x32_10(q // 65536, 0, q % 65536, 0,
                                          seed & MASK, seed >> 32), axis=-1)
        assert np.array_equal(mine, quads[q])
    # far-away low counter word through the generator offset (offset counts single outputs)
    seed = 0xFEDCBA9876543210
    for c0, s in ((3, 9), (0x00FFFFF1, 77), (0x7FFFFFF0, 65535)):
        quad = _curand_quads(lib, seed, 4 * (65536 * c0 + s), 4)[0]
        mine = np.array([int(v) for v in orc.philox4x32_10(c0, 0, s, 0, seed & MASK, seed >> 32)])
        assert np.array_equal(mine, quad)


def test_philox_round_is_a_bijection():
    """For a fixed key the round maps counters one-to-one: undo it with the inverses of the
    odd multipliers modulo 2^32."""
    inv0, inv1 = pow(M0, -1, 2 ** 32), pow(M1, -1, 2 ** 32)
    assert (inv0 * M0) & MASK == 1 and (inv1 * M1) & MASK == 1
    rng = np.random.default_rng(11)
    c = [rng.integers(0, 2 ** 32, 2000, dtype=np.uint64) for _ in range(4)]
    k = [np.uint64(0xDEADBEEF), np.uint64(0x12345678)]
    out = orc.philox_round(c, k)
    for t in range(2000):
        o = [int(v[t]) for v in out]
        c2 = (o[1] * inv1) & MASK
        c0 = (o[3] * inv0) & MASK
        hi1 = (M1 * c2) >> 32
        hi0 = (M0 * c0) >> 32
        c1 = o[0] ^ hi1 ^ int(k[0])
        c3 = o[2] ^ hi0 ^ int(k[1])
        assert [c0, c1, c2, c3] == [int(v[t]) for v in c]


def test_philox_every_input_word_matters():
    base = np.array([int(v) for v in orc.philox4x32_10(1, 2, 3, 4, 5, 6)])
    for pos in range(6):
        args = [1, 2, 3, 4, 5, 6]
        args[pos] ^= 1
        other = np.array([int(v) for v in orc.philox4x32_10(*args)])
        flipped = sum(bin(int(a) ^ int(b)).count("1") for a, b in zip(base, other))
        assert 32 < flipped < 96          # avalanche: about half of 128 bits


def test_sample_indices_layout_and_mapping():
    """Draw b of node i at iteration k is word b mod 4 of the block with counter
    (b div 4, i, k_lo, k_hi); the index is floor(u*m / 2^32), checked with Python integers."""
    seed, k, n, B, m = 0xABCDEF0123456789, (5 << 32) | 17, 5, 11, 1000
    idx = orc.sample_indices(seed, k, n, B, m)
    assert idx.shape == (n, B) and idx.dtype == np.int32
    for i in range(n):
        for b in range(B):
            w = orc.philox4x32_10(b // 4, i, k & MASK, k >> 32, seed & MASK, seed >> 32)
            u = int(w[b % 4])
            assert idx[i, b] == (u * m) // 2 ** 32


def test_sample_indices_range_and_streams():
    seed = 42
    a = orc.sample_indices(seed, 3, 16, 128, 65536)
    assert a.min() >= 0 and a.max() < 65536
    assert np.array_equal(a, orc.sample_indices(seed, 3, 16, 128, 65536))     # stateless
    assert not np.array_equal(a, orc.sample_indices(seed, 4, 16, 128, 65536))  # k matters
    assert not np.array_equal(a, orc.sample_indices(seed + 1, 3, 16, 128, 65536))
    assert len({tuple(r) for r in a}) == 16                                    # node matters
    one = orc.sample_indices(seed, 0, 4, 9, 1)
    assert np.all(one == 0)                                                    # m = 1
    big = orc.sample_indices(seed, 0, 64, 64, 2 ** 31 - 1)
    assert big.min() >= 0 and big.max() > 2 ** 29


def test_sample_indices_uniform_chi_square():
    m, bins = 1024, 64
    draws = np.concatenate([orc.sample_indices(9, k, 32, 64, m).ravel() for k in range(64)])
    counts = np.bincount(draws * bins // m, minlength=bins)
    expected = len(draws) / bins
    chi2 = float(np.sum((counts - expected) ** 2 / expected))
    # 63 degrees of freedom: mean 63, sd 11.2; 130 is six sigma
    assert chi2 < 130.0
    # with replacement: a minibatch of 128 out of 64 must repeat
    assert len(set(orc.sample_indices(1, 0, 1, 128, 64)[0])) <= 64
