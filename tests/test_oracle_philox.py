"""Pins for the oracle's mask generator (Eq. 1): Philox4x32-10 and the Bernoulli threshold.

The oracle is checked against things other than itself:
  * NVIDIA's cuRAND *host* generator CURAND_RNG_PSEUDO_PHILOX4_32_10 (a library routine that
    runs on the CPU): its stream, quad q of one generate call, is Philox4x32-10 at counter
    (q >> 16, 0, q & 0xffff, 0) under key = the 64-bit seed;
  * a second Philox written independently with numpy integers (tests/philox_ref.py);
  * the closed form P(drop) = floor(p * 2^32) / 2^32 evaluated in exact rational arithmetic;
  * binomial confidence bounds on keep rates and on independence across paths and elements.
"""
import ctypes
import glob
import os
from fractions import Fraction

import numpy as np
import pytest

import oracle
from philox_ref import keep_bits, philox4x32_10 as philox_np


def _load_curand():
    pats = ["/usr/local/cuda/lib64/libcurand.so*"]
    try:
        import nvidia.curand as nc
        pats.append(os.path.join(os.path.dirname(nc.__file__), "lib", "libcurand.so*"))
    except Exception:
        pass
    for pat in pats:
        for path in sorted(glob.glob(pat)):
            try:
                return ctypes.CDLL(path)
            except OSError:
                continue
    return None


def _curand_host_stream(cr, seed, n_words):
    gen = ctypes.c_void_p()
    assert cr.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0  # PHILOX4_32_10
    try:
        assert cr.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
        out = np.zeros(n_words, dtype=np.uint32)
        assert cr.curandGenerate(gen, out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)),
                                 ctypes.c_size_t(n_words)) == 0
    finally:
        cr.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 0x0123456789ABCDEF, 0xD509A7C4, 2**64 - 1])
def test_philox_matches_curand_host_generator(seed):
    cr = _load_curand()
    if cr is None:
        pytest.skip("libcurand not found")
    n_quads = 65536 * 2 + 64  # crosses two steps of counter word 0
    stream = _curand_host_stream(cr, seed, 4 * n_quads).reshape(n_quads, 4)
    q = np.arange(n_quads, dtype=np.uint64)
    ctr = np.stack([q >> np.uint64(16), np.zeros_like(q), q & np.uint64(0xFFFF), np.zeros_like(q)], -1)
    key = np.broadcast_to(np.array([seed & 0xFFFFFFFF, seed >> 32], dtype=np.uint64), (n_quads, 2))
    assert np.array_equal(philox_np(ctr, key), stream)
    # the oracle's C routine, directly against the library, on a spread of quads
    for qq in list(range(0, 300)) + [65535, 65536, 65537, 131071, 131072, n_quads - 1]:
        got = oracle.philox4x32_10([qq >> 16, 0, qq & 0xFFFF, 0], [seed & 0xFFFFFFFF, seed >> 32])
        assert np.array_equal(got, stream[qq]), qq


def test_oracle_philox_matches_independent_implementation():
    rng = np.random.default_rng(7)
    ctr = rng.integers(0, 2**32, size=(4000, 4), dtype=np.uint64)
    key = rng.integers(0, 2**32, size=(4000, 2), dtype=np.uint64)
    # edge words too
    ctr[:8] = [[0, 0, 0, 0], [2**32 - 1] * 4, [1, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 0], [0, 0, 0, 1],
               [2**32 - 1, 0, 0, 0], [0, 0, 0, 2**32 - 1]]
    ref = philox_np(ctr, key)
    for n in range(ctr.shape[0]):
        assert np.array_equal(oracle.philox4x32_10(ctr[n], key[n]), ref[n]), n
    # every counter and key word matters
    base = oracle.philox4x32_10([5, 6, 7, 8], [9, 10])
    for w in range(4):
        c = [5, 6, 7, 8]
        c[w] += 1
        assert not np.array_equal(oracle.philox4x32_10(c, [9, 10]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 6, 7, 8], [10, 10]), base)
    assert not np.array_equal(oracle.philox4x32_10([5, 6, 7, 8], [9, 11]), base)


@pytest.mark.parametrize("p", [0.0, 0.05, 0.1, 0.2, 0.3, 0.5, 0.75, 0.999])
def test_drop_threshold_closed_form(p):
    p32 = np.float32(p)
    exact = Fraction(float(p32)) * 2**32          # exact rational value of the float times 2^32
    assert oracle.drop_threshold(p) == exact.numerator // exact.denominator
    if p == 0.0:
        assert oracle.drop_threshold(p) == 0
    if p == 0.5:
        assert oracle.drop_threshold(p) == 2**31


def test_mask_keying_and_packing():
    """masks() packs keep bits of counter (j>>2, i, t, seq_base+b), word j&3, keep iff word >= thr."""
    B, T, K, d, p, seed, seq_base = 2, 3, 4, 200, 0.3, 0xABCDEF0123456789, 11
    thr = oracle.drop_threshold(p)
    bits = oracle.masks(B, T, K, d, p, seed, seq_base)
    assert bits.shape == (B, T, K, 7)
    for b in range(B):
        for t in range(T):
            for i in range(K):
                ref = keep_bits(seed, seq_base + b, t, i, d, thr)
                got = (bits[b, t, i][np.arange(d) // 32] >> (np.arange(d) % 32).astype(np.uint32)) & 1
                assert np.array_equal(got.astype(bool), ref)
                assert all(oracle.mask_keep(seed, seq_base + b, t, i, j, thr) == int(ref[j])
                           for j in range(0, d, 17))
    # bits past d stay clear
    assert not (bits[..., 6] >> np.uint32(200 - 192)).any()
    # sequence id enters truncated to 32 bits
    a = oracle.masks(1, 1, 1, 64, 0.5, 1, 3)
    b_ = oracle.masks(1, 1, 1, 64, 0.5, 1, 3 + 2**32)
    assert np.array_equal(a, b_)


def test_p_zero_keeps_everything_and_masks_are_nested_in_p():
    d = 4096
    assert oracle.masks(1, 2, 3, d, 0.0, 99).view(np.uint8).sum() == 255 * (2 * 3 * d // 8)
    lo = oracle.masks(1, 2, 3, d, 0.1, 99)
    hi = oracle.masks(1, 2, 3, d, 0.3, 99)
    assert not (hi & ~lo).any()  # whatever p=0.1 drops, p=0.3 drops too (same word, higher bar)


def _unpack(bits, d):
    j = np.arange(d)
    return ((bits[..., j // 32] >> (j % 32).astype(np.uint32)) & 1).astype(np.float64)


@pytest.mark.parametrize("p", [0.05, 0.1, 0.3, 0.5])
def test_keep_rate_and_independence(p):
    """Eq. 1: entries are iid Bernoulli(1-p): rate within 5 sigma; paths and neighbours uncorrelated."""
    B, T, K, d = 2, 4, 16, 4096
    m = _unpack(oracle.masks(B, T, K, d, p, 0x5EED, 0), d)      # [B,T,K,d]
    n = m.size
    q = 1.0 - oracle.drop_threshold(p) / 2**32
    assert abs(m.mean() - q) < 5 * np.sqrt(q * (1 - q) / n)
    # per-word-slot rate (each of the four Philox output words is used)
    for w in range(4):
        mw = m[..., w::4]
        assert abs(mw.mean() - q) < 5 * np.sqrt(q * (1 - q) / mw.size)
    z = (m - q) / np.sqrt(q * (1 - q))
    def corr_ok(a, b):
        c = (a * b).mean()
        return abs(c) < 5 / np.sqrt(a.size)
    assert corr_ok(z[:, :, :-1], z[:, :, 1:])        # path i vs i+1
    assert corr_ok(z[:, :-1], z[:, 1:])              # position t vs t+1
    assert corr_ok(z[:-1], z[1:])                    # sequence b vs b+1
    assert corr_ok(z[..., :-1], z[..., 1:])          # element j vs j+1
    assert corr_ok(z[..., :-4], z[..., 4:])          # same word slot, next counter
    # different seeds give different, uncorrelated masks
    z2 = (_unpack(oracle.masks(B, T, K, d, p, 0x5EEE, 0), d) - q) / np.sqrt(q * (1 - q))
    assert corr_ok(z, z2)
