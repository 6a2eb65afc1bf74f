"""Pins for the oracle's JS-divergence criterion (Sec. 3.2: Eq. 4, Eq. 5, Algorithm 1).

Checked against things other than the oracle itself: scipy's Jensen-Shannon distance and
softmax (library routines), closed forms (identical and disjoint distributions, the ln 2 bound),
a brute-force restatement of Algorithm 1 with scipy on small vocabularies, and special cases of
the whole path (p = 0 makes every head equal to the centroid)."""
import numpy as np
import pytest
from scipy.spatial.distance import jensenshannon
from scipy.special import rel_entr, softmax

import oracle


def test_js_closed_forms():
    P = np.array([0.2, 0.3, 0.5])
    assert oracle.js_divergence(P, P) == 0.0
    assert abs(oracle.js_divergence([1, 0, 0], [0, 0.5, 0.5]) - np.log(2)) < 1e-15      # disjoint supports
    # two-point example by hand: P=(1,0), Q=(1/2,1/2): M=(3/4,1/4)
    want = 0.5 * np.log(1 / 0.75) + 0.5 * (0.5 * np.log(0.5 / 0.75) + 0.5 * np.log(0.5 / 0.25))
    assert abs(oracle.js_divergence([1, 0], [0.5, 0.5]) - want) < 1e-15


def test_js_matches_scipy_and_is_symmetric_and_bounded():
    rng = np.random.default_rng(0)
    for V in (2, 7, 100, 5000):
        for _ in range(5):
            P = rng.dirichlet(np.full(V, 0.3))
            Q = rng.dirichlet(np.full(V, 0.3))
            got = oracle.js_divergence(P, Q)
            assert abs(got - jensenshannon(P, Q) ** 2) < 1e-12       # scipy returns the square root
            assert abs(got - oracle.js_divergence(Q, P)) < 1e-15
            assert 0.0 <= got <= np.log(2) + 1e-15


def _js(P, Q):
    """JS from scipy's elementwise relative entropy; the inputs are taken as given (scipy's
    jensenshannon would renormalise a draft distribution whose fp32 entries do not sum to 1)."""
    M = 0.5 * (P + Q)
    return 0.5 * rel_entr(P, M).sum() + 0.5 * rel_entr(Q, M).sum()


def _algorithm1_bruteforce(logits, draft_prob):
    K = logits.shape[0]
    pbar = softmax(logits.mean(axis=0))
    heads = [_js(softmax(logits[i]), pbar) for i in range(K)]
    d = _js(np.asarray(draft_prob, dtype=np.float64), pbar)
    return np.array(heads + [d]), d <= max(heads)


def test_eq4_eq5_against_scipy_restatement():
    rng = np.random.default_rng(1)
    seen = set()
    for trial in range(60):
        K, V = int(rng.integers(1, 9)), int(rng.integers(2, 400))
        logits = rng.normal(0, rng.choice([0.3, 1.5, 4.0]), size=(K, V))
        # drafts near the centroid (Eq. 5 tends to hold) and far from it (it tends to fail)
        base = logits.mean(axis=0) + rng.normal(0, rng.choice([0.05, 0.5, 3.0]), size=V)
        dp = softmax(base)
        js, ok = oracle.js_from_logits(logits, dp)
        want_js, want_ok = _algorithm1_bruteforce(logits, dp)
        assert np.abs(js - want_js).max() < 1e-12
        assert ok == bool(want_ok)
        seen.add(ok)
    assert seen == {True, False}


def test_identical_heads_have_zero_divergence_and_k1_rejects_any_other_draft():
    rng = np.random.default_rng(2)
    row = rng.normal(size=50)
    logits = np.tile(row, (4, 1))
    js, ok = oracle.js_from_logits(logits, softmax(row))
    assert np.all(js[:4] == 0.0) and js[4] < 1e-15                  # the draft IS the centroid (up to rounding)
    js, ok = oracle.js_from_logits(logits, softmax(row + rng.normal(0, 0.5, size=50)))
    assert js[4] > 0 and not ok                                     # concentrated heads: Eq. 5 alone rejects
    js, ok = oracle.js_from_logits(row[None, :], softmax(row))      # K = 1: the head is the centroid
    assert js[0] == 0.0 and js[1] < 1e-15                           # Eq. 5 holds only if js[1] is exactly 0


def _toy(rng, V=300, d=64, B=2, T=3):
    W = (rng.normal(size=(V, d)) * d ** -0.5 * 3).astype(np.float32)
    H = rng.normal(size=(B, T, d)).astype(np.float32)
    return W, H


def test_verify_js_is_algorithm_1_on_the_masked_heads():
    rng = np.random.default_rng(3)
    W, H = _toy(rng)
    B, T, K, p, seed = 2, 3, 5, 0.3, 99
    V = W.shape[0]
    und = np.einsum("btd,vd->btv", H.astype(np.float64), W.astype(np.float64))
    dp = softmax(und + rng.normal(0, 0.8, size=und.shape), axis=-1).astype(np.float32)
    draft = und.argmax(-1).astype(np.int32)
    draft[1, 1] = 7                                                  # an implausible draft token
    out = oracle.verify_js(W, oracle.F32, H, draft, dp, K, p, seed, seq_base=4)
    plain = oracle.verify_batched(W, oracle.F32, H, draft, K, p, seed, seq_base=4, rule=oracle.RULE_MAJORITY)
    assert np.array_equal(out["tokens"], plain["tokens"]) and np.array_equal(out["counts"], plain["counts"])
    for b in range(B):
        run, open_ = 0, True
        for t in range(T):
            logits = np.stack([oracle.logits_row(W, oracle.F32, H[b, t], p, seed, 4 + b, t, i) for i in range(K)])
            js, ok5 = _algorithm1_bruteforce(logits, dp[b, t].astype(np.float64))
            assert np.abs(out["js"][b, t] - js).max() < 1e-12
            assert out["js_ok"][b, t] == int(ok5)
            ok = ok5 or oracle.majority_token(out["tokens"][b, t]) == draft[b, t]
            if open_ and ok:
                run += 1
            else:
                open_ = False
        assert out["accept_len"][b] == run
    # Algorithm 1 accepts at least what the majority rule alone accepts
    assert (out["accept_len"] >= plain["accept_len"]).all()


def test_p_zero_collapses_heads_onto_the_centroid():
    rng = np.random.default_rng(4)
    W, H = _toy(rng)
    und = np.einsum("btd,vd->btv", H.astype(np.float64), W.astype(np.float64))
    dp = softmax(und, axis=-1).astype(np.float32)                    # the draft distribution is the target's
    draft = und.argmax(-1).astype(np.int32)
    out = oracle.verify_js(W, oracle.F32, H, draft, dp, 4, 0.0, 1)
    assert np.all(out["js"][..., :4] == 0.0)                         # no dropout: every head equals the centroid
    assert np.all(out["js"][..., 4] < 1e-12)                         # and so does this draft (up to fp32 rounding of dp)
    assert (out["accept_len"] == H.shape[1]).all()                   # accepted by Eq. 5 or, failing that, by majority
