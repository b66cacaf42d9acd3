"""Pins for the oracle's decision stream (Algorithm 1: "b ~ U[0,1]; if b <= p").

The Philox4x32-10 words are compared with an independent implementation:
cuRAND's host-side CURAND_RNG_PHILOX4_32_10 generator, driven through its
public API.  Observed through that API, the host generator's 4-word block
number n (= offset / 4) uses key = (seed_lo, seed_hi) and counter
(lo32(n >> 16), hi32(n >> 16), n & 0xFFFF, 0).  The oracle's counter layout
(t_lo, t_hi, k, 0) therefore makes the whole decision stream reachable:
block n = t * 65536 + k.
"""
import ctypes as C
import glob
import math

import numpy as np
import pytest

import oracle


def _curand():
    paths = sorted(glob.glob("/usr/local/cuda/lib64/libcurand.so*"))
    if not paths:
        import torch, os  # the wheel may carry its own copy
        base = os.path.dirname(os.path.dirname(torch.__file__))
        paths = sorted(glob.glob(os.path.join(base, "nvidia", "curand", "lib", "libcurand.so*")))
    if not paths:
        pytest.skip("libcurand not found")
    return C.CDLL(paths[0])


class _HostPhilox:
    def __init__(self):
        self.lib = _curand()
        self.gen = C.c_void_p()
        rc = self.lib.curandCreateGeneratorHost(C.byref(self.gen), 161)  # PHILOX4_32_10
        if rc != 0:
            pytest.skip(f"curandCreateGeneratorHost -> {rc}")

    def words(self, seed, offset, n):
        assert self.lib.curandSetPseudoRandomGeneratorSeed(self.gen, C.c_ulonglong(seed)) == 0
        assert self.lib.curandSetGeneratorOffset(self.gen, C.c_ulonglong(offset)) == 0
        out = np.zeros(n, dtype=np.uint32)
        assert self.lib.curandGenerate(self.gen, out.ctypes.data_as(C.c_void_p), C.c_size_t(n)) == 0
        return out

    def __del__(self):
        try:
            self.lib.curandDestroyGenerator(self.gen)
        except Exception:
            pass


def test_philox_words_match_curand_host_generator():
    ref = _HostPhilox()
    rng = np.random.default_rng(7)
    seeds = [0, 1, 2025, 0xDEADBEEF, 0x0123456789ABCDEF, 2**64 - 1]
    blocks = [0, 1, 2, 3, 65535, 65536, 65537, 2**32 - 1, 2**32, 2**48 + 5, 2**61 + 12345] + \
             [int(v) for v in rng.integers(0, 2**62, size=24)]
    for seed in seeds:
        for n in blocks:
            want = ref.words(seed, 4 * n, 4)
            hi = n >> 16
            got = oracle.philox4x32_10([hi & 0xFFFFFFFF, hi >> 32, n & 0xFFFF, 0],
                                       [seed & 0xFFFFFFFF, seed >> 32])
            assert np.array_equal(got, want), (hex(seed), n, got, want)


def test_philox_consecutive_counters_match_one_curand_sequence():
    ref = _HostPhilox()
    want = ref.words(99, 4 * 65500, 4 * 64)      # crosses the 65536-block boundary
    got = np.concatenate([oracle.philox4x32_10([n >> 16, 0, n & 0xFFFF, 0], [99, 0])
                          for n in range(65500, 65564)])
    assert np.array_equal(got, want)


def test_draw_word_is_the_curand_stream_at_offset_t_k():
    ref = _HostPhilox()
    rng = np.random.default_rng(11)
    for seed in (2025, 0xFEEDFACECAFEBEEF):
        for _ in range(40):
            t = int(rng.integers(0, 2**44))
            k = int(rng.integers(0, 65536))
            want = ref.words(seed, 4 * ((t << 16) | k), 1)[0]
            assert oracle.draw_word(seed, t, k) == int(want)
        for t in range(4):
            for k in range(8):
                want = ref.words(seed, 4 * ((t << 16) | k), 1)[0]
                assert oracle.draw_word(seed, t, k) == int(want)


def test_threshold_values():
    assert oracle.threshold(0.0) == 0
    assert oracle.threshold(1.0) == 2**32
    assert oracle.threshold(0.25) == 2**30
    assert oracle.threshold(0.5) == 2**31
    assert oracle.threshold(0.1) == math.floor(0.1 * 2**32)


def test_decision_is_word_below_threshold_and_extremes():
    for t in range(50):
        for k in range(8):
            r = oracle.draw_word(5, t, k)
            for p in (0.0, 0.1, 0.25, 0.5, 0.9, 1.0):
                assert oracle.decision(5, t, k, p) == int(r < math.floor(p * 2**32))
            assert oracle.decision(5, t, k, 0.0) == 0     # p = 0: never pull
            assert oracle.decision(5, t, k, 1.0) == 1     # p = 1: always pull


@pytest.mark.parametrize("p", [0.02, 0.1, 0.25, 0.5, 0.9])
def test_decision_frequency_within_four_sigma(p):
    K, T = 32, 2000
    b = np.array([[oracle.decision(2025, t, k, p) for k in range(K)] for t in range(T)])
    n = K * T
    sigma = math.sqrt(p * (1 - p) / n)
    assert abs(b.mean() - p) < 4 * sigma
    # per-worker and per-step marginals too (independence over k and t)
    assert np.all(np.abs(b.mean(axis=0) - p) < 5 * math.sqrt(p * (1 - p) / T))
    # lag-1 autocorrelation over t and cross-correlation between neighbours in k
    c = b - p
    assert abs((c[1:] * c[:-1]).mean()) < 5 * p * (1 - p) / math.sqrt(n)
    assert abs((c[:, 1:] * c[:, :-1]).mean()) < 5 * p * (1 - p) / math.sqrt(n)


def test_decisions_depend_on_seed_step_and_worker():
    base = [oracle.draw_word(1, t, k) for t in range(16) for k in range(16)]
    assert len(set(base)) == len(base)
    assert base != [oracle.draw_word(2, t, k) for t in range(16) for k in range(16)]
    # high halves of seed and t are used
    assert oracle.draw_word(1, 3, 0) != oracle.draw_word(1 + 2**32, 3, 0)
    assert oracle.draw_word(1, 3, 0) != oracle.draw_word(1, 3 + 2**32, 0)
    # (t, k) are not interchangeable
    assert oracle.draw_word(1, 2, 5) != oracle.draw_word(1, 5, 2)
