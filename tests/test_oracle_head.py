"""Pins for the oracle's dropout head (Eq. 2, Eq. 3) and per-path decoding (Sec. 3.2).

Anchors: numpy fp64 GEMV (a library routine) at p = 0 and on explicitly masked inputs, the
independent numpy Philox for the masks, E[h^(i)] = h (stated after Eq. 2), the linearity of Eq. 3,
and a brute-force enumeration of all 16 masks of a d = 4 head with their exact probabilities.
"""
import itertools
from collections import Counter

import numpy as np
import pytest
import torch

import oracle
from philox_ref import keep_bits

SEED = 0xD509A7C4


def _bf16_bits(x):
    return torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16).view(torch.uint16).numpy()


def _bf16_to_f64(bits):
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _head(V, d, seed, dtype):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((V, d)) / np.sqrt(d)).astype(np.float32)
    h = rng.standard_normal(d).astype(np.float32)
    if dtype == oracle.BF16:
        Wb, hb = _bf16_bits(W), _bf16_bits(h)
        return Wb, hb, _bf16_to_f64(Wb), _bf16_to_f64(hb)
    return W, h, W.astype(np.float64), h.astype(np.float64)


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
def test_p_zero_is_a_plain_gemv(dtype):
    V, d = 37, 24  # V != d so a transposed operand cannot pass
    W, h, W64, h64 = _head(V, d, 1, dtype)
    got = oracle.logits_row(W, dtype, h, 0.0, SEED, 0, 0, 0)
    ref = W64 @ h64
    assert np.allclose(got, ref, rtol=1e-13, atol=1e-15)
    tok, gap = oracle.argmax(got)
    assert tok == int(np.argmax(ref))
    srt = np.sort(ref)
    assert gap == pytest.approx(srt[-1] - srt[-2], rel=1e-9)


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.BF16])
@pytest.mark.parametrize("p", [0.1, 0.3, 0.5])
def test_masked_logits_against_explicit_mask_and_linearity(dtype, p):
    V, d = 53, 40
    W, h, W64, h64 = _head(V, d, 2, dtype)
    thr = oracle.drop_threshold(p)
    p64 = float(np.float32(p))
    for (s, t, i) in [(0, 0, 0), (3, 2, 5), (2**32 + 3, 2, 5), (7, 60, 31)]:
        keep = keep_bits(SEED, s, t, i, d, thr)
        hm = oracle.masked_hidden(h, dtype, p, SEED, s, t, i)
        assert np.array_equal(hm, np.where(keep, h64, 0.0))        # Eq. 2 numerator, exact
        got = oracle.logits_row(W, dtype, h, p, SEED, s, t, i)
        ref = (W64 @ np.where(keep, h64, 0.0)) / (1.0 - p64)        # Eq. 2 + Eq. 3
        assert np.allclose(got, ref, rtol=1e-12, atol=1e-14)
        # linearity: W(h*m) = Wh - W(h*(1-m))
        lin = (W64 @ h64 - W64 @ np.where(keep, 0.0, h64)) / (1.0 - p64)
        assert np.allclose(got, lin, rtol=1e-10, atol=1e-12)
        # the positive scale cannot change the decoded token
        assert oracle.argmax(got)[0] == int(np.argmax(W64 @ np.where(keep, h64, 0.0)))
    # sequence ids that agree mod 2^32 share masks
    a = oracle.logits_row(W, dtype, h, p, SEED, 3, 2, 5)
    b = oracle.logits_row(W, dtype, h, p, SEED, 2**32 + 3, 2, 5)
    assert np.array_equal(a, b)


def test_expectation_of_dropout_is_identity():
    """E[h^(i)] = h: the sample mean of masked/rescaled copies approaches h at the CLT rate."""
    d, p, n = 64, 0.3, 4000
    rng = np.random.default_rng(5)
    h = (rng.standard_normal(d) + 2.0).astype(np.float32)
    p64 = float(np.float32(p))
    acc = np.zeros(d)
    for i in range(n):
        acc += oracle.masked_hidden(h, oracle.F32, p, SEED, 1, i // 32, i % 32) / (1.0 - p64)
    mean = acc / n
    sigma = np.abs(h) * np.sqrt(p64 / (1 - p64) / n)
    assert np.all(np.abs(mean - h) < 5 * sigma)


def test_argmax_first_index_on_ties():
    assert oracle.argmax([1.0, 3.0, 3.0, 2.0]) == (1, 0.0)
    assert oracle.argmax([0.0, 0.0, 0.0]) == (0, 0.0)
    tok, gap = oracle.argmax([-1.0, -5.0, -0.5])
    assert tok == 2 and gap == 0.5
    assert oracle.argmax([4.0])[0] == 0


def test_bruteforce_all_masks_d4():
    """d = 4: the token of every sample equals table[its mask]; the empirical distribution over
    many paths matches the exact mixture sum_mask P(mask) [table[mask] = y] (chi-square)."""
    d, V, p = 4, 6, 0.3
    rng = np.random.default_rng(11)
    W = rng.standard_normal((V, d)).astype(np.float32)
    h = rng.standard_normal(d).astype(np.float32)
    W64, h64 = W.astype(np.float64), h.astype(np.float64)
    q_drop = oracle.drop_threshold(p) / 2**32
    table, prob = {}, Counter()
    for mask in itertools.product([0, 1], repeat=d):
        tok = int(np.argmax(W64 @ (h64 * np.array(mask))))
        table[mask] = tok
        keep = sum(mask)
        prob[tok] += (1 - q_drop) ** keep * q_drop ** (d - keep)
    assert table[(0, 0, 0, 0)] == 0          # all dropped: all logits 0, first index wins
    assert abs(sum(prob.values()) - 1) < 1e-12
    thr = oracle.drop_threshold(p)
    T, K = 8, 32
    H = np.broadcast_to(h, (1, T, d)).copy()
    out = oracle.verify_batched(W, oracle.F32, H, np.zeros((1, T), np.int32), K, p, SEED)
    seen = Counter()
    masks_seen = set()
    for t in range(T):
        for i in range(K):
            mask = tuple(int(x) for x in keep_bits(SEED, 0, t, i, d, thr))
            masks_seen.add(mask)
            assert out["tokens"][0, t, i] == table[mask]
            seen[table[mask]] += 1
    assert len(masks_seen) >= 8              # the sample exercises many masks
    n = T * K
    cells = [(y, pr) for y, pr in prob.items() if pr * n >= 5]
    rest_p = 1.0 - sum(pr for _, pr in cells)
    chi2 = sum((seen[y] - n * pr) ** 2 / (n * pr) for y, pr in cells)
    if rest_p * n >= 1:
        rest_seen = n - sum(seen[y] for y, _ in cells)
        chi2 += (rest_seen - n * rest_p) ** 2 / (n * rest_p)
    assert chi2 < 30.0, (chi2, seen, prob)   # far beyond the 99.9 % point for <= 6 cells


def test_p_zero_is_greedy_verification_and_k1_is_single_path():
    V, d, T, K = 97, 32, 6, 5
    rng = np.random.default_rng(3)
    W = rng.standard_normal((V, d)).astype(np.float32)
    H = rng.standard_normal((2, T, d)).astype(np.float32)
    greedy = np.argmax(H.astype(np.float64) @ W.astype(np.float64).T, axis=-1).astype(np.int32)
    draft = greedy.copy()
    draft[0, 3] = (draft[0, 3] + 1) % V          # first mismatch of sequence 0 at t = 3
    draft[1, 0] = (draft[1, 0] + 1) % V          # sequence 1 rejected at once
    out = oracle.verify_batched(W, oracle.F32, H, draft, K, 0.0, SEED)
    assert np.array_equal(out["tokens"], np.broadcast_to(greedy[..., None], (2, T, K)))
    assert np.all(out["counts"] == K)
    assert out["accept_len"].tolist() == [3, 0]
    assert np.array_equal(out["hits"], np.where(draft == greedy, K, 0))
    # K = 1: one path; accepted exactly while draft == that path's token
    out1 = oracle.verify_batched(W, oracle.F32, H, draft, 1, 0.4, SEED)
    tok = out1["tokens"][..., 0]
    for b in range(2):
        exp = 0
        while exp < T and draft[b, exp] == tok[b, exp]:
            exp += 1
        assert out1["accept_len"][b] == exp
        for t in range(T):
            l = oracle.logits_row(W, oracle.F32, H[b, t], 0.4, SEED, b, t, 0)
            assert tok[b, t] == int(np.argmax(l))
    assert np.all(out1["counts"] == 1)
