"""Pins for oracle/rng.py: none of them re-uses the oracle's own formula."""
import ctypes
import math
import os

import numpy as np
import pytest

from oracle import rng


# ---- Philox: scalar big-integer re-derivation of the round function -----------------
def philox_bigint(ctr, key):
    """Philox4x32-10 on Python integers, written from the S-P network description:
    two multiplications by fixed odd constants, high halves mixed with the key into
    the neighbouring words, low halves permuted; Weyl-sequence key schedule."""
    c = list(ctr)
    k = list(key)
    for rnd in range(10):
        if rnd:
            k = [(k[0] + 0x9E3779B9) % 2 ** 32, (k[1] + 0xBB67AE85) % 2 ** 32]
        prod_a = 0xD2511F53 * c[0]
        prod_b = 0xCD9E8D57 * c[2]
        c = [(prod_b // 2 ** 32) ^ c[1] ^ k[0], prod_b % 2 ** 32,
             (prod_a // 2 ** 32) ^ c[3] ^ k[1], prod_a % 2 ** 32]
    return c


def test_philox_matches_bigint_scalar():
    g = np.random.default_rng(123)
    ctrs = g.integers(0, 2 ** 32, size=(200, 4), dtype=np.uint64)
    keys = g.integers(0, 2 ** 32, size=(200, 2), dtype=np.uint64)
    for c, k in zip(ctrs, keys):
        got = rng.philox4x32_10(c[0:1], c[1:2], c[2:3], c[3:4], int(k[0]), int(k[1]))
        want = philox_bigint([int(v) for v in c], [int(v) for v in k])
        assert [int(w[0]) for w in got] == want


def test_philox_is_a_bijection_on_a_counter_range():
    # a keyed permutation never maps two counters to the same block
    q = np.arange(1 << 16, dtype=np.uint64)
    w = rng.philox4x32_10(q, 0 * q, 0 * q + 7, 0 * q, 99, 1)
    blocks = np.stack(w, axis=1)
    assert len(np.unique(blocks, axis=0)) == len(q)


def _curand_host():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    return None


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFEDCBA9876543210])
def test_philox_matches_curand_host_generator(seed):
    """The cuRAND *host* generator PHILOX4_32_10 runs on the CPU.  Its i-th block of
    four outputs (i < 4096) is the Philox block with key = seed and counter (0, 0, i, 0)."""
    lib = _curand_host()
    if lib is None:
        pytest.skip("libcurand not present")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:
        pytest.skip("cuRAND host generator unavailable")
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    n = 4 * 4096
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    i = np.arange(4096, dtype=np.uint64)
    w = rng.philox4x32_10(0 * i, 0 * i, i, 0 * i, seed & 0xFFFFFFFF, seed >> 32)
    assert np.array_equal(np.stack(w, axis=1).reshape(-1).astype(np.uint32), out)


def test_stream_words_layout():
    # element e comes from block e div 4, word e mod 4, counter words (q, 0, segment, 4*layer+tag)
    seed, seg, layer, tag = 0xABCDEF0123, 3, 2, rng.TAG_WEIGHT
    w = rng.stream_words(seed, seg, layer, tag, 23)
    for e in (0, 1, 6, 22):
        blk = philox_bigint([e // 4, 0, seg, 4 * layer + tag], [seed % 2 ** 32, seed // 2 ** 32])
        assert int(w[e]) == blk[e % 4]
    # prefix property: a longer stream starts with the shorter one
    assert np.array_equal(rng.stream_words(seed, seg, layer, tag, 1000)[:23], w)


# ---- uniforms ------------------------------------------------------------------------
def test_uniform_open_interval_and_exactness():
    words = np.array([0, 1, 511, 512, 2 ** 31, 2 ** 32 - 1], dtype=np.uint64)
    u = rng.uniform_open01(words)
    assert u.dtype == np.float32
    assert float(u.min()) == 2.0 ** -24 and float(u.max()) == 1.0 - 2.0 ** -24
    for r, v in zip(words, u):
        assert float(v) == (2 * (int(r) >> 9) + 1) / 2 ** 24      # exact rational value


def test_uniform_kappa_labels_shape_range_moments():
    # Section 3: SIL is 60 x 47 with kappa = 10 (stored here class-major: 47 rows of 60)
    sil = rng.gen_labels(1, 0, 47, 60, rng.DIST_UNIFORM_KAPPA, 10.0)
    assert sil.shape == (47, 60) and sil.dtype == np.float32
    assert sil.min() > 0.0 and sil.max() < 10.0
    big = rng.gen_labels(1, 0, 1000, 1000, rng.DIST_UNIFORM_KAPPA, 10.0).astype(np.float64)
    n = big.size
    assert abs(big.mean() - 5.0) < 4 * (10 / math.sqrt(12)) / math.sqrt(n)       # mean kappa/2
    assert abs(big.var() - 100.0 / 12.0) < 0.05                                   # var kappa^2/12
    # kappa scales linearly (Eq. 1): kappa=1 values times 10 equal kappa=10 values up to 1 rounding
    one = rng.gen_labels(1, 0, 47, 60, rng.DIST_UNIFORM_KAPPA, 1.0)
    assert np.allclose(one * 10.0, sil, rtol=2 ** -23, atol=0)


def test_labels_deterministic_and_seed_sensitive():
    a = rng.gen_labels(1, 0, 47, 64, rng.DIST_NORMAL)
    assert np.array_equal(a.view(np.uint32), rng.gen_labels(1, 0, 47, 64, rng.DIST_NORMAL).view(np.uint32))
    assert not np.array_equal(a, rng.gen_labels(2, 0, 47, 64, rng.DIST_NORMAL))
    assert not np.array_equal(a, rng.gen_labels(1, 1, 47, 64, rng.DIST_NORMAL))
    # element (class j, i) depends only on its flat index: a taller matrix has the same first rows
    tall = rng.gen_labels(1, 0, 62, 64, rng.DIST_NORMAL)
    assert np.array_equal(tall[:47], a)


# ---- the normal sampler against libm and the exact distribution --------------------------
def test_spec_log_matches_libm():
    n = np.concatenate([np.arange(1, 20001, 2), np.arange(2 ** 24 - 20001, 2 ** 24, 2),
                        np.random.default_rng(0).integers(0, 2 ** 23, 200000) * 2 + 1])
    got = rng.spec_log_u(n)
    want = np.log(n.astype(np.float64) / 2.0 ** 24)        # the division is exact
    assert np.max(np.abs(got - want) / np.maximum(np.abs(want), 1e-300)) < 1e-13
    assert np.all(got < 0.0)


def test_spec_sincos_matches_libm():
    j = np.concatenate([np.arange(0, 2 ** 24, 4099), np.array([0, 2 ** 21 - 1, 2 ** 21, 2 ** 22 - 1, 2 ** 22,
                                                                 2 ** 23, 3 * 2 ** 22, 2 ** 24 - 1])])
    c, s = rng.spec_sincos(j)
    theta = (j.astype(np.float64) + 0.5) * (2.0 * math.pi / 2 ** 24)
    assert np.max(np.abs(c - np.cos(theta))) < 1e-14
    assert np.max(np.abs(s - np.sin(theta))) < 1e-14


def test_normals_equal_libm_box_muller_after_rounding():
    words = rng.stream_words(5, 0, 0, 0, 400000).reshape(-1, 2)
    z0, z1 = rng.normal_pairs(words[:, 0], words[:, 1])
    u1 = (2.0 * (words[:, 0] >> np.uint64(9)).astype(np.float64) + 1.0) / 2 ** 24
    theta = ((words[:, 1] >> np.uint64(8)).astype(np.float64) + 0.5) * (2.0 * math.pi / 2 ** 24)
    rad = np.sqrt(-2.0 * np.log(u1))
    e0 = (rad * np.cos(theta)).astype(np.float32)
    e1 = (rad * np.sin(theta)).astype(np.float32)
    for got, want in ((z0, e0), (z1, e1)):
        ulp = np.abs(got.view(np.int32).astype(np.int64) - want.view(np.int32).astype(np.int64))
        assert ulp.max() <= 1                       # at most a rounding-boundary flip
        assert np.mean(ulp == 0) > 0.9999


def test_normal_labels_moments_and_ks():
    z = rng.gen_labels(1, 0, 1000, 1000, rng.DIST_NORMAL).astype(np.float64).ravel()
    n = z.size
    assert abs(z.mean()) < 4.0 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 4.0 * math.sqrt(2.0 / n)
    assert abs(np.mean(z ** 4) - 3.0) < 0.05                   # kurtosis of a normal
    zs = np.sort(z)
    cdf = 0.5 * (1.0 + np.vectorize(math.erf)(zs[::10] / math.sqrt(2.0)))
    emp = (np.arange(n)[::10] + 0.5) / n
    assert np.max(np.abs(cdf - emp)) < 1.63 / math.sqrt(n) + 1e-5     # KS, alpha = 0.01
    # the two members of a Box-Muller pair are uncorrelated
    assert abs(np.mean(z[0::2] * z[1::2])) < 4.0 / math.sqrt(n / 2)


# ---- weight initialisation (Section 2: framework default for Linear) ---------------------
def test_init_linear_bounds_and_moments():
    W, b = rng.init_linear(2, 0, 1, 784, 512)
    bound = 1.0 / math.sqrt(784.0)
    assert W.shape == (512, 784) and b.shape == (512,)
    assert np.abs(W).max() < bound * (1 + 1e-6) and np.abs(b).max() < bound * (1 + 1e-6)
    assert abs(float(W.mean())) < 4 * bound / math.sqrt(3 * W.size)
    assert abs(float(W.astype(np.float64).var()) - bound ** 2 / 3.0) < 0.02 * bound ** 2
    W2, _ = rng.init_linear(2, 0, 2, 784, 512)
    assert not np.array_equal(W, W2)                 # layers use distinct streams
