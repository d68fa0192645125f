"""Pins for the oracle's random-number chain: Philox4x32-10 -> uniform -> Gumbel.

Philox is pinned to NVIDIA's cuRAND *host* generator (runs on the CPU, no GPU
needed), an implementation independent of ours.  The fixed fp32 logarithm is
pinned to libm's double log; the Gumbel variates to the distribution's closed
forms (mean = Euler-Mascheroni, variance = pi^2/6, CDF exp(-exp(-x))).
"""
import ctypes as C
import ctypes.util
import math
import os

import numpy as np
import pytest

import oracle


def _curand():
    for p in ("/usr/local/cuda/lib64/libcurand.so", ctypes.util.find_library("curand")):
        if p and (os.path.exists(p) or "/" not in p):
            try:
                return C.CDLL(p)
            except OSError:
                pass
    return None


CURAND_RNG_PSEUDO_PHILOX4_32_10 = 161
SUBSEQ = 65536  # cuRAND's host ordering interleaves this many subsequences (counter word 2)


@pytest.mark.parametrize("seed", [0, 1, 0x0123456789ABCDEF, 0xFFFFFFFFFFFFFFFF, 0xDEADBEEF00000001])
def test_philox_matches_curand_host(seed):
    cr = _curand()
    if cr is None:
        pytest.skip("libcurand not found")
    gen = C.c_void_p()
    assert cr.curandCreateGeneratorHost(C.byref(gen), CURAND_RNG_PSEUDO_PHILOX4_32_10) == 0
    assert cr.curandSetPseudoRandomGeneratorSeed(gen, C.c_ulonglong(seed)) == 0
    n_blocks = SUBSEQ * 2 + 64          # reaches counter word 0 in {0, 1, 2}
    out = np.zeros(4 * n_blocks, np.uint32)
    assert cr.curandGenerate(gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(out.size)) == 0
    key = [seed & 0xFFFFFFFF, seed >> 32]
    rng = np.random.default_rng(7)
    blocks = list(range(0, 40)) + [SUBSEQ - 1, SUBSEQ, SUBSEQ + 1, 2 * SUBSEQ + 5] + \
        [int(x) for x in rng.integers(0, n_blocks, 200)]
    for j in blocks:
        # block j of the host stream = counter (j // SUBSEQ, 0, j % SUBSEQ, 0)
        got = oracle.philox4x32_10([j // SUBSEQ, 0, j % SUBSEQ, 0], key)
        assert list(got) == list(out[4 * j:4 * j + 4]), (seed, j)
    # a large stream offset reaches counter word 1
    c0, c1, c2 = 7, 3, 11
    off = 4 * (SUBSEQ * (c0 + (c1 << 32)) + c2)
    assert cr.curandSetGeneratorOffset(gen, C.c_ulonglong(off)) == 0
    o4 = np.zeros(4, np.uint32)
    assert cr.curandGenerate(gen, o4.ctypes.data_as(C.c_void_p), C.c_size_t(4)) == 0
    assert list(oracle.philox4x32_10([c0, c1, c2, 0], key)) == list(o4)
    cr.curandDestroyGenerator(gen)


def test_philox_counter_words_all_matter():
    base = oracle.philox4x32_10([1, 2, 3, 4], [5, 6])
    for pos in range(4):
        c = [1, 2, 3, 4]
        c[pos] ^= 1
        assert list(oracle.philox4x32_10(c, [5, 6])) != list(base)
    assert list(oracle.philox4x32_10([1, 2, 3, 4], [5, 7])) != list(base)


def test_uniform_is_exact_odd_multiple():
    assert oracle.uniform(0) == 2.0 ** -24
    assert oracle.uniform(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    assert oracle.uniform(0x1FF) == 2.0 ** -24          # low 9 bits are dropped
    assert oracle.uniform(0x200) == 3 * 2.0 ** -24
    rng = np.random.default_rng(0)
    for x in rng.integers(0, 2 ** 32, 2000):
        x = int(x)
        assert oracle.uniform(x) == (2 * (x >> 9) + 1) * 2.0 ** -24


def test_dlog_close_to_libm():
    rng = np.random.default_rng(1)
    xs = np.concatenate([
        np.float32(2.0) ** rng.uniform(-24, 5, 20000).astype(np.float32),
        np.float32(1.0) + rng.uniform(-1e-3, 1e-3, 2000).astype(np.float32),
        np.array([2.0 ** -24, 1 - 2.0 ** -24, 0.5, 1.0, 2.0, 1.41421354, 1.41421342, 0.70710678, 16.635532], np.float32),
    ]).astype(np.float32)
    for x in xs:
        got = oracle.dlog(float(x))
        ref = math.log(float(x))
        assert abs(got - ref) <= 2.5e-7 * max(1.0, abs(ref)) + 1e-7 * abs(ref) + 1e-14, (x, got, ref)
    assert oracle.dlog(1.0) == 0.0


def test_dlog_range_of_gumbel_chain_is_safe():
    # -dlog(u) must stay a positive normal float for the extreme uniforms
    for x in (0, 0xFFFFFFFF):
        u = oracle.uniform(x)
        t = -oracle.dlog(u)
        assert t > 2.0 ** -126 and math.isfinite(t)
        assert math.isfinite(oracle.gumbel(x))


def test_gumbel_matches_closed_form_pointwise():
    rng = np.random.default_rng(2)
    for x in rng.integers(0, 2 ** 32, 5000):
        x = int(x)
        u = (2 * (x >> 9) + 1) * 2.0 ** -24
        ref = -math.log(-math.log(u))
        got = oracle.gumbel(x)
        # the inner log's rounding error is amplified by 1/(-log u) when u -> 1
        amp = 1.0 + 1.0 / (-math.log(u))
        assert abs(got - ref) <= 4e-7 * amp + 2e-6, (x, got, ref)


def test_gumbel_moments_and_cdf():
    rng = np.random.default_rng(3)
    xs = rng.integers(0, 2 ** 32, 400000)
    g = np.array([oracle.gumbel(int(x)) for x in xs], np.float64)
    n = g.size
    assert abs(g.mean() - 0.5772156649) < 5 * math.sqrt(math.pi ** 2 / 6 / n)
    assert abs(g.var() - math.pi ** 2 / 6) < 0.02
    # Kolmogorov-Smirnov against F(x) = exp(-exp(-x))
    gs = np.sort(g)
    F = np.exp(-np.exp(-gs))
    dmax = np.max(np.abs(F - (np.arange(n) + 0.5) / n))
    assert dmax < 1.63 / math.sqrt(n)       # 1% critical value


def test_perturbed_key_layout():
    # unit i of list l uses word i&3 of Philox(counter=(i>>2, l, round_lo, round_hi), key=seed)
    seed, rnd, lst = 0x1122334455667788, 0x0000000300000009, 41
    for i in (0, 1, 2, 3, 4, 5, 1023, 16383):
        w = oracle.philox4x32_10([i >> 2, lst, rnd & 0xFFFFFFFF, rnd >> 32], [seed & 0xFFFFFFFF, seed >> 32])
        g = oracle.gumbel(int(w[i & 3]))
        want = np.float32(np.float32(0.25) + np.float32(g))
        assert oracle.perturbed_key(0.25, seed, rnd, lst, i) == float(want)
    assert oracle.perturbed_key(0.25, seed, rnd, lst, 5, greedy=1) == 0.25
