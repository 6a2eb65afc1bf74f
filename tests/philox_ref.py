"""A second, independent Philox4x32-10 written with numpy uint64 arithmetic.

Used only by the tests, to cross-check the oracle's C implementation and the CUDA
kernels' masks.  Vectorised over leading axes: ctr[...,4], key[...,2] -> out[...,4].
"""
import numpy as np

_MUL = (np.uint64(0xD2511F53), np.uint64(0xCD9E8D57))
_WEYL = (0x9E3779B9, 0xBB67AE85)
_LO = np.uint64(0xFFFFFFFF)
_S32 = np.uint64(32)


def philox4x32_10(ctr, key):
    c = [np.asarray(ctr)[..., n].astype(np.uint64) for n in range(4)]
    k = [np.asarray(key)[..., n].astype(np.uint64) for n in range(2)]
    for rnd in range(10):
        kr = [(k[n] + np.uint64((rnd * _WEYL[n]) & 0xFFFFFFFF)) & _LO for n in range(2)]
        prod0 = _MUL[0] * c[0]
        prod2 = _MUL[1] * c[2]
        c = [(prod2 >> _S32) ^ c[1] ^ kr[0], prod2 & _LO, (prod0 >> _S32) ^ c[3] ^ kr[1], prod0 & _LO]
    return np.stack(c, axis=-1).astype(np.uint32)


def keep_bits(seed, s, t, i, d, thr):
    """bool[d]: keep flags of (sequence s, position t, path i) under the mask keying rule."""
    j = np.arange(d, dtype=np.uint64)
    ctr = np.stack([j >> np.uint64(2), np.full(d, i, np.uint64), np.full(d, t, np.uint64),
                    np.full(d, s & 0xFFFFFFFF, np.uint64)], axis=-1)
    key = np.array([seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF], dtype=np.uint64)
    words = philox4x32_10(ctr, np.broadcast_to(key, (d, 2)))
    picked = words[np.arange(d), (j & np.uint64(3)).astype(np.int64)]
    return picked >= np.uint32(thr)
