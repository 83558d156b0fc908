"""Pins for the oracle's counter-based generator and its uniform mapping."""
import ctypes
import ctypes.util
import glob

import numpy as np
import pytest
from scipy import stats

from oracle import flop_oracle as O


def _load_curand():
    names = [ctypes.util.find_library("curand")] + sorted(glob.glob("/usr/local/cuda*/lib64/libcurand.so*"))
    try:
        import nvidia.curand  # type: ignore
        import os
        names += sorted(glob.glob(os.path.join(os.path.dirname(nvidia.curand.__file__), "lib", "libcurand.so*")))
    except Exception:
        pass
    for n in names:
        if not n:
            continue
        try:
            return ctypes.CDLL(n)
        except OSError:
            continue
    return None


def test_philox_matches_vendor_host_generator():
    """Independent library pin: a vendor HOST generator of the same published
    algorithm (it runs on the CPU).  Its output block b holds the Philox block
    of counter (b // 65536, 0, b % 65536, 0) and an offset of 4*65536*2^32
    outputs advances the second counter word by one (observed ordering of that
    host generator); the key is the 64-bit seed as (low, high)."""
    lib = _load_curand()
    if lib is None:
        pytest.skip("no host Philox library to compare with")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:     # 161: the Philox4x32-10 generator
        pytest.skip("host generator unavailable")
    try:
        for seed in (0, 0xDEADBEEFCAFEF00D, 0x0000000100000000):
            assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
            nblk = 65536 + 1000
            for hi, lo_base in ((0, 0), (5, 9)):
                off = 4 * 65536 * ((hi << 32) + lo_base)
                assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(off)) == 0
                out = (ctypes.c_uint32 * (4 * nblk))()
                assert lib.curandGenerate(gen, out, ctypes.c_size_t(4 * nblk)) == 0
                got = np.frombuffer(out, dtype=np.uint32).reshape(nblk, 4)
                b = np.arange(nblk, dtype=np.uint64)
                c0 = np.uint64(lo_base) + b // np.uint64(65536)
                c2 = b % np.uint64(65536)
                w = O.philox4x32_10(c0, 0 * b + np.uint64(hi), c2, 0 * b, seed & 0xFFFFFFFF, seed >> 32)
                assert np.array_equal(np.stack(w, axis=1), got)
    finally:
        lib.curandDestroyGenerator(gen)


def test_philox_is_injective_on_counters_and_key_sensitive():
    c = np.arange(1 << 16, dtype=np.uint64)
    w = np.stack(O.philox4x32_10(c, 0 * c, 0 * c, 0 * c, 7, 9), axis=1)
    assert len(np.unique(w, axis=0)) == len(c)          # a bijection never collides
    w2 = np.stack(O.philox4x32_10(c, 0 * c, 0 * c, 0 * c, 8, 9), axis=1)
    assert np.mean(w == w2) < 1e-3
    # avalanche: flipping one counter bit flips about half of the 128 output bits
    w3 = np.stack(O.philox4x32_10(c ^ np.uint64(1), 0 * c, 0 * c, 0 * c, 7, 9), axis=1)
    flipped = np.unpackbits((w ^ w3).view(np.uint8)).mean()
    assert abs(flipped - 0.5) < 0.01


def test_uniform_mapping_open_interval_and_exact_in_fp32():
    x = np.array([0, 1, 511, 512, 0x7FFFFFFF, 0x80000000, 0xFFFFFFFF], dtype=np.uint32)
    u = O.uniform_from_bits(x)
    assert u.min() == 2.0 ** -24 and u.max() == 1.0 - 2.0 ** -24
    assert np.all((u > 0) & (u < 1))
    assert np.array_equal(u.astype(np.float32).astype(np.float64), u)          # 24 significant bits
    assert np.array_equal((1.0 - u).astype(np.float32).astype(np.float64), 1.0 - u)
    # symmetric about 1/2: bits x and ~x give u and 1-u
    assert np.allclose(O.uniform_from_bits(~x), 1.0 - u, rtol=0, atol=0)


def test_gate_uniforms_statistics():
    n = 1 << 20
    u = O.gate_uniforms(n, seed=0, offset=0)
    assert abs(u.mean() - 0.5) < 4 * np.sqrt(1 / 12 / n)
    assert abs(u.var() - 1 / 12) < 1e-3
    assert stats.kstest(u, "uniform").pvalue > 1e-3
    # no lag-1 or lag-4 correlation (words of a block, neighbouring blocks)
    for lag in (1, 4):
        assert abs(np.corrcoef(u[:-lag], u[lag:])[0, 1]) < 5e-3
    # different seeds / offsets give different streams
    assert np.mean(u == O.gate_uniforms(n, seed=1, offset=0)) < 1e-3


def test_gate_uniforms_counter_continuation():
    """Gate j uses counter offset + j//4, word j%4: advancing the offset by m
    blocks continues the same stream 4m gates later."""
    seed = 0x1234567890ABCDEF
    a = O.gate_uniforms(1000, seed, offset=(1 << 32) - 100)   # crosses the low counter word
    b = O.gate_uniforms(1000 - 4 * 37, seed, offset=(1 << 32) - 100 + 37)
    assert np.array_equal(a[4 * 37:], b)
    assert O.gate_uniforms(0, 0, 0).shape == (0,)
    assert np.array_equal(O.gate_uniforms(7, 3, 5)[:5], O.gate_uniforms(5, 3, 5))
