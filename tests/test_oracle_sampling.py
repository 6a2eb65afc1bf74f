"""Pins of the oracle's sampling decode rule (Sec. 3.2 names nucleus sampling as the alternative
to the top-1 token; the paper gives no parameters, so the reading is: temperature tau, nucleus
mass top_p, a draw from the renormalised nucleus of Softmax(l / tau) made by the Gumbel-max
construction with counter-based noise).

Nothing here re-types the oracle's own code path: the uniform variates are checked against the
Python-integer Philox, the nucleus against a numpy sort-and-cut, the draw against a numpy
Gumbel-max, and -- the pin that fixes the distribution itself -- token frequencies over many
paths against the textbook nucleus probabilities with a chi-square bound."""
import numpy as np
import pytest
from scipy import special, stats

import oracle
from philox_ref import philox4x32_10

SEED = 0xD509A7C4


def _uniform_ref(seed, s, t, i, v):
    ctr = np.array([v >> 2, i | 0x80000000, t, s & 0xFFFFFFFF], dtype=np.uint64)
    key = np.array([seed & 0xFFFFFFFF, seed >> 32], dtype=np.uint64)
    w = int(philox4x32_10(ctr, key)[v & 3])
    return ((w >> 9) + 0.5) / 2.0 ** 23


def test_uniform_variates_follow_the_keying_rule_and_stay_inside_the_unit_interval():
    rng = np.random.default_rng(1)
    for _ in range(300):
        seed = int(rng.integers(0, 2 ** 63))
        s, t, i, v = (int(rng.integers(0, 2 ** 32)), int(rng.integers(0, 64)), int(rng.integers(0, 1024)),
                      int(rng.integers(0, 200000)))
        u = oracle.sample_uniform(seed, s, t, i, v)
        assert u == _uniform_ref(seed, s, t, i, v)
        assert 0.0 < u < 1.0 and np.float32(u) == u           # exact in fp32 too
    # the four words of one Philox call serve four consecutive vocabulary entries
    us = [oracle.sample_uniform(SEED, 3, 2, 1, v) for v in range(8)]
    assert len(set(us)) == 8


def test_noise_counters_are_disjoint_from_mask_counters():
    # same (s, t, i, index): the mask word and the noise word come from different Philox counters
    thr = oracle.drop_threshold(0.5)
    agree = 0
    for v in range(2000):
        keep = oracle.mask_keep(SEED, 5, 1, 7, v, thr)
        u = oracle.sample_uniform(SEED, 5, 1, 7, v)
        agree += int(keep == (u >= 0.5))
    assert 800 < agree < 1200          # independent fair coins agree about half of the time


def test_gumbel_transform():
    for u in (1e-7, 0.1, 0.5, 0.9, 1 - 1e-7):
        assert abs(oracle.gumbel(u) - (-np.log(-np.log(u)))) < 1e-12
    assert abs(oracle.gumbel(np.exp(-1.0))) < 1e-12        # closed form: u = 1/e gives g = 0
    # a Gumbel variate has mean = Euler's constant and variance pi^2 / 6
    g = np.array([oracle.gumbel(oracle.sample_uniform(SEED, 0, 0, 0, v)) for v in range(40000)])
    assert abs(g.mean() - np.euler_gamma) < 0.03 and abs(g.var() - np.pi ** 2 / 6) < 0.08


def _nucleus_ref(logits, tau, top_p):
    p = special.softmax(np.asarray(logits, dtype=np.float64) / tau)
    if top_p >= 1.0:
        return np.ones(len(p), dtype=bool), p
    order = sorted(range(len(p)), key=lambda v: (-p[v], v))
    keep = np.zeros(len(p), dtype=bool)
    cum = 0.0
    for v in order:
        keep[v] = True
        cum += p[v]
        if cum >= top_p:
            break
    return keep, p


@pytest.mark.parametrize("tau", [0.5, 1.0, 2.0])
@pytest.mark.parametrize("top_p", [0.05, 0.5, 0.9, 0.999, 1.0])
def test_nucleus_is_the_sort_and_cut_definition(tau, top_p):
    rng = np.random.default_rng(int(tau * 10 + top_p * 1000))
    for V in (1, 2, 7, 50, 1000):
        logits = rng.normal(0, 2.0, V)
        logits[rng.integers(0, V)] = logits.max()          # an exact tie at the top
        keep, _ = _nucleus_ref(logits, tau, top_p)
        assert np.array_equal(oracle.nucleus(logits, tau, top_p), keep)
    # a worked case: probabilities 0.5, 0.3, 0.2 -> top_p 0.5 keeps one token, 0.51 two, 0.81 all three
    l = np.log(np.array([0.3, 0.5, 0.2]))
    assert oracle.nucleus(l, 1.0, 0.5).tolist() == [False, True, False]
    assert oracle.nucleus(l, 1.0, 0.51).tolist() == [True, True, False]
    assert oracle.nucleus(l, 1.0, 0.81).tolist() == [True, True, True]


def test_draw_is_the_gumbel_max_over_the_nucleus():
    rng = np.random.default_rng(7)
    for case in range(40):
        V = int(rng.integers(2, 300))
        logits = rng.normal(0, 1.5, V)
        tau, top_p = float(rng.choice([0.7, 1.0, 1.3])), float(rng.choice([0.3, 0.8, 1.0]))
        s, t, i = int(rng.integers(0, 1000)), int(rng.integers(0, 8)), int(rng.integers(0, 32))
        keep, _ = _nucleus_ref(logits, tau, top_p)
        keys = np.array([logits[v] / tau - np.log(-np.log(_uniform_ref(SEED, s, t, i, v))) if keep[v] else -np.inf
                         for v in range(V)])
        tok, gap = oracle.sample_row(logits, tau, top_p, SEED, s, t, i)
        assert tok == int(np.argmax(keys))
        top2 = np.sort(keys)[-2:] if V > 1 else [-np.inf, keys[0]]
        assert gap == pytest.approx(top2[1] - top2[0], rel=1e-9, abs=1e-12) or (np.isinf(gap) and np.isinf(top2[0]))


@pytest.mark.parametrize("tau,top_p", [(1.0, 1.0), (0.6, 1.0), (1.0, 0.7), (1.5, 0.9)])
def test_token_frequencies_match_the_nucleus_distribution(tau, top_p):
    """The pin that fixes the law of the draw: over many paths the tokens must be distributed as
    Softmax(l / tau) restricted to the nucleus and renormalised (what nucleus sampling means)."""
    logits = np.array([1.2, 0.3, -0.5, 2.0, 0.0, 1.9, -2.0, 0.8])
    keep, p = _nucleus_ref(logits, tau, top_p)
    q = np.where(keep, p, 0.0)
    q /= q.sum()
    n = 20000
    toks = np.array([oracle.sample_row(logits, tau, top_p, SEED, 11, 3, i)[0] for i in range(n)])
    counts = np.bincount(toks, minlength=len(logits))
    assert counts[~keep].sum() == 0                      # nothing outside the nucleus is ever drawn
    chi2 = ((counts[keep] - n * q[keep]) ** 2 / (n * q[keep])).sum()
    assert chi2 < stats.chi2.ppf(1 - 1e-6, df=max(1, int(keep.sum()) - 1))


def test_limits_reduce_to_the_argmax():
    rng = np.random.default_rng(3)
    logits = rng.normal(0, 1, 500)
    top = int(np.argmax(logits))
    for i in range(50):
        assert oracle.sample_row(logits, 1e-6, 1.0, SEED, 0, 0, i)[0] == top     # temperature -> 0
        assert oracle.sample_row(logits, 1.0, 1e-9, SEED, 0, 0, i)[0] == top     # nucleus of one token
    draws = {oracle.sample_row(logits, 1.0, 1.0, SEED, 0, 0, i)[0] for i in range(50)}
    assert len(draws) > 10                                                        # ... and otherwise it really samples


def test_whole_call_with_sampling_decode():
    rng = np.random.default_rng(5)
    V, d, B, T, K, p = 300, 64, 2, 3, 6, 0.2
    W = rng.normal(0, 0.3, (V, d)).astype(np.float32)
    H = rng.normal(0, 1.0, (B, T, d)).astype(np.float32)
    draft = rng.integers(0, V, (B, T)).astype(np.int32)
    out = oracle.verify_batched_sampled(W, oracle.F32, H, draft, K, p, SEED, temperature=0.8, top_p=0.9, seq_base=4)
    for b in range(B):
        for t in range(T):
            for i in range(K):
                l = oracle.logits_row(W, oracle.F32, H[b, t], p, SEED, 4 + b, t, i)
                assert out["tokens"][b, t, i] == oracle.sample_row(l, 0.8, 0.9, SEED, 4 + b, t, i)[0]
            cnt, hits = oracle.counts(out["tokens"][b, t], int(draft[b, t]))
            assert np.array_equal(out["counts"][b, t], cnt) and out["hits"][b, t] == hits
        assert out["accept_len"][b] == oracle.accept_chain(out["tokens"][b], draft[b])
    # temperature -> 0 gives back the argmax call
    cold = oracle.verify_batched_sampled(W, oracle.F32, H, draft, K, p, SEED, temperature=1e-7, top_p=1.0, seq_base=4)
    plain = oracle.verify_batched(W, oracle.F32, H, draft, K, p, SEED, seq_base=4)
    assert np.array_equal(cold["tokens"], plain["tokens"]) and np.array_equal(cold["accept_len"], plain["accept_len"])
