"""Pins for the oracle's histogram and acceptance steps (Sec. 3.2 Eq. 3' and Eq. 6, the
left-to-right rule, tree drafts of Sec. 4.4), checked against brute force with Python
containers, invariants that hold for any input, and a hand-worked tree fixture."""
import json
from collections import Counter
from pathlib import Path

import numpy as np
import pytest

import oracle

SEED = 0xD509A7C4
GOLDEN = Path(__file__).parent / "golden"


def _toy(V=211, d=48, B=3, T=6, seed=0):
    rng = np.random.default_rng(seed)
    W = rng.standard_normal((V, d)).astype(np.float32)
    H = rng.standard_normal((B, T, d)).astype(np.float32)
    return W, H


def test_counts_hits_and_majority_bruteforce():
    rng = np.random.default_rng(1)
    for _ in range(300):
        K = int(rng.integers(1, 33))
        toks = rng.integers(0, 6, size=K).astype(np.int32)
        draft = int(rng.integers(0, 7))
        cnt, hits = oracle.counts(toks, draft)
        c = Counter(toks.tolist())
        assert cnt.tolist() == [c[x] for x in toks.tolist()]
        assert hits == c.get(draft, 0)
        best = max(c.values())
        assert oracle.majority_token(toks) == min(x for x, n in c.items() if n == best)
        assert oracle.accept_chain(toks[None, :], [draft], oracle.RULE_NAIVE) == int(draft in c)


def test_majority_is_plurality_with_smallest_id_tiebreak():
    assert oracle.majority_token([9, 4, 4, 9, 7]) == 4
    assert oracle.majority_token([3, 2, 1]) == 1
    assert oracle.majority_token([8]) == 8
    assert oracle.majority_token([5, 6, 6, 5, 6]) == 6


@pytest.mark.parametrize("rule", [oracle.RULE_NAIVE, oracle.RULE_MAJORITY])
def test_chain_scan_bruteforce_and_first_reject_stops(rule):
    rng = np.random.default_rng(2)
    for _ in range(200):
        T, K = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        toks = rng.integers(0, 4, size=(T, K)).astype(np.int32)
        draft = rng.integers(0, 4, size=T).astype(np.int32)
        L = oracle.accept_chain(toks, draft, rule)
        ok = []
        for t in range(T):
            c = Counter(toks[t].tolist())
            if rule == oracle.RULE_NAIVE:
                ok.append(draft[t] in c)
            else:
                best = max(c.values())
                ok.append(draft[t] == min(x for x, n in c.items() if n == best))
        exp = next((t for t, o in enumerate(ok) if not o), T)
        assert L == exp and 0 <= L <= T
        # whatever follows the first rejection cannot matter
        if L < T - 1:
            d2 = draft.copy()
            d2[L + 1:] = rng.integers(0, 4, size=T - L - 1)
            assert oracle.accept_chain(toks, d2, rule) == L


def test_tree_golden_fixture():
    g = json.loads((GOLDEN / "tree_case.json").read_text())
    for name, rule in (("naive", oracle.RULE_NAIVE), ("majority", oracle.RULE_MAJORITY)):
        L, best, ok = oracle.accept_tree(g["tokens"], g["node_token"], g["node_parent"], g["node_hrow"], rule)
        assert ok.tolist() == g[name]["node_ok"]
        assert L == g[name]["accept_len"]
        assert best == g[name]["best_node"]
    # nothing accepted
    L, best, ok = oracle.accept_tree([[1, 1, 1]], [2, 3], [-1, 0], [0, 0], oracle.RULE_NAIVE)
    assert (L, best, ok.tolist()) == (0, -1, [0, 0])


@pytest.mark.parametrize("rule", [oracle.RULE_NAIVE, oracle.RULE_MAJORITY])
def test_tree_bruteforce_paths(rule):
    """Enumerate root-to-node paths explicitly; accepted length = longest fully accepted path."""
    rng = np.random.default_rng(4)
    for _ in range(100):
        N, K, R = int(rng.integers(1, 20)), int(rng.integers(1, 6)), int(rng.integers(1, 6))
        toks = rng.integers(0, 3, size=(R, K)).astype(np.int32)
        parent = np.array([int(rng.integers(-1, n)) for n in range(N)], dtype=np.int32)
        hrow = rng.integers(0, R, size=N).astype(np.int32)
        ntok = rng.integers(0, 3, size=N).astype(np.int32)
        L, best, ok = oracle.accept_tree(toks, ntok, parent, hrow, rule)

        def node_test(n):
            c = Counter(toks[hrow[n]].tolist())
            if rule == oracle.RULE_NAIVE:
                return ntok[n] in c
            m = max(c.values())
            return ntok[n] == min(x for x, k in c.items() if k == m)

        exp_len, exp_best = 0, -1
        for n in range(N):
            path, m = [], n
            while m >= 0:
                path.append(m)
                m = parent[m]
            good = all(node_test(x) for x in path)
            assert bool(ok[n]) == good
            if good and len(path) > exp_len:
                exp_len, exp_best = len(path), n
        assert (L, best) == (exp_len, exp_best)


def test_chain_equals_path_shaped_tree_and_batched_equals_singles():
    W, H = _toy()
    B, T, _ = H.shape
    K, p = 6, 0.25
    rng = np.random.default_rng(9)
    greedy = np.argmax(H.astype(np.float64) @ W.astype(np.float64).T, -1).astype(np.int32)
    draft = np.where(rng.random((B, T)) < 0.8, greedy, rng.integers(0, W.shape[0], (B, T))).astype(np.int32)
    for rule in (oracle.RULE_NAIVE, oracle.RULE_MAJORITY):
        full = oracle.verify_batched(W, oracle.F32, H, draft, K, p, SEED, seq_base=5, rule=rule)
        for b in range(B):
            one = oracle.verify_batched(W, oracle.F32, H[b:b + 1], draft[b:b + 1], K, p, SEED,
                                        seq_base=5 + b, rule=rule)
            for key in ("tokens", "counts", "hits", "accept_len", "gap"):
                assert np.array_equal(one[key][0], full[key][b]), key
        parent = np.tile(np.arange(-1, T - 1, dtype=np.int32), (B, 1))
        hrow = np.tile(np.arange(T, dtype=np.int32), (B, 1))
        tree = oracle.verify_tree(W, oracle.F32, H, draft, parent, hrow, K, p, SEED, seq_base=5, rule=rule)
        assert np.array_equal(tree["tokens"], full["tokens"])
        assert np.array_equal(tree["counts"], full["counts"])
        assert np.array_equal(tree["accept_len"], full["accept_len"])
        for b in range(B):
            L = full["accept_len"][b]
            assert tree["best_node"][b] == L - 1
            assert tree["node_ok"][b].tolist() == [1] * L + [0] * (T - L)


def test_nested_paths_make_acceptance_monotone_in_K():
    """Counter-based masks: the first K paths are the same for any larger K, so under the naive
    rule the token set only grows and the accepted length cannot shrink."""
    W, H = _toy(seed=3)
    B, T, _ = H.shape
    rng = np.random.default_rng(10)
    greedy = np.argmax(H.astype(np.float64) @ W.astype(np.float64).T, -1).astype(np.int32)
    draft = greedy.copy()
    prev = None
    for K in (1, 2, 4, 8, 16):
        out = oracle.verify_batched(W, oracle.F32, H, draft, K, 0.5, SEED)
        if prev is not None:
            assert np.array_equal(out["tokens"][..., :prev["tokens"].shape[-1]], prev["tokens"])
            assert np.all(out["accept_len"] >= prev["accept_len"])
        assert np.all(out["accept_len"] <= T)
        assert np.all(out["counts"].max(-1) <= K) and np.all(out["counts"] >= 1)
        prev = out


def test_shared_masks_make_paths_persistent_heads():
    """Other reading of Eq. 1 (no position index on m^(i)): with shared masks a path applies one
    mask at every position, so equal hidden rows decode to equal tokens path by path, and the
    tokens of position t equal those of a single-position call on that row (which has t = 0)."""
    rng = np.random.default_rng(21)
    V, d, T, K, p, seed = 200, 48, 4, 6, 0.4, 77
    W = (rng.normal(size=(V, d)) * 0.4).astype(np.float32)
    row = rng.normal(size=d).astype(np.float32)
    H = np.tile(row, (1, T, 1))                                  # the same hidden row at every position
    draft = np.zeros((1, T), dtype=np.int32)
    sh = oracle.verify_batched(W, oracle.F32, H, draft, K, p, seed, seq_base=5, shared_masks=True)
    ind = oracle.verify_batched(W, oracle.F32, H, draft, K, p, seed, seq_base=5)
    assert (sh["tokens"] == sh["tokens"][:, :1]).all()           # identical across positions, path by path
    assert not (ind["tokens"] == ind["tokens"][:, :1]).all()     # independent masks: they differ somewhere
    assert np.array_equal(sh["tokens"][0, 0], ind["tokens"][0, 0])   # position 0 is keyed alike in both readings
    H2 = rng.normal(size=(1, T, d)).astype(np.float32)
    sh2 = oracle.verify_batched(W, oracle.F32, H2, draft, K, p, seed, seq_base=5, shared_masks=True)
    for t in range(T):                                           # position t under shared masks == that row alone
        one = oracle.verify_batched(W, oracle.F32, H2[:, t:t + 1], draft[:, :1], K, p, seed, seq_base=5)
        assert np.array_equal(sh2["tokens"][0, t], one["tokens"][0, 0])


@pytest.mark.parametrize("bonus", [0, 1])
def test_next_token_is_the_plain_greedy_token_at_the_first_unaccepted_position(bonus):
    """Pins for oracle.verify_batched_next: the plain tokens are a library fp64 GEMV argmax; the
    dropout part equals verify_batched on the same rows; next[b] follows from a brute-force scan."""
    rng = np.random.default_rng(31 + bonus)
    V, d, B, T, K, p, seed = 150, 40, 3, 4, 5, 0.3, 1234
    T_h = T + bonus
    W = (rng.normal(size=(V, d)) * 0.5).astype(np.float32)
    H = rng.normal(size=(B, T_h, d)).astype(np.float32)
    und = np.einsum("bqd,vd->bqv", H.astype(np.float64), W.astype(np.float64))
    greedy = und.argmax(-1).astype(np.int32)
    draft = greedy[:, :T].copy()
    draft[0, 2] = (draft[0, 2] + 1) % V            # sequence 0: a wrong draft at position 2
    draft[1, 0] = (draft[1, 0] + 1) % V            # sequence 1: wrong at once; sequence 2: all plausible
    out = oracle.verify_batched_next(W, oracle.F32, H, draft, K, p, seed, seq_base=9)
    assert np.array_equal(out["plain"], greedy)
    if bonus == 0:                                  # same rows, same keys: the dropout part is the plain call's
        ref = oracle.verify_batched(W, oracle.F32, H, draft, K, p, seed, seq_base=9)
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(out[key], ref[key]), key
    for b in range(B):
        n = 0
        while n < T and draft[b, n] in out["tokens"][b, n]:
            n += 1
        assert out["accept_len"][b] == n
        assert out["next"][b] == (greedy[b, n] if n < T_h else -1)
    # p = 0: every dropout path is the plain token, everything plausible is accepted
    out0 = oracle.verify_batched_next(W, oracle.F32, H, greedy[:, :T].copy(), K, 0.0, seed)
    assert (out0["tokens"] == out0["plain"][..., None]).all()
    assert (out0["accept_len"] == T).all()
    assert np.array_equal(out0["next"], greedy[:, T] if bonus else np.full(B, -1))
