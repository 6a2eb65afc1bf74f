"""Comparison policy of the GPU parity tests.

Masks, histograms and accepted lengths are integer results and must match the oracle bit for
bit.  Decoded tokens must be identical except where the oracle's own top-2 logit gap is below
NEAR_TIE (fp32 accumulation on the GPU vs fp64 in the oracle may then pick the other
candidate); such rows are counted and returned.  Where a token did differ, the integer stages
are still checked exactly, by feeding the GPU's tokens to the oracle's integer routines.
"""
import numpy as np

import oracle

NEAR_TIE = 2e-2          # oracle top-2 gap below which a token may differ
TOL_LOGIT_BF16 = 2e-2    # max abs error of debug logits, bf16 storage
TOL_LOGIT_F32 = 1e-4     # max abs error of debug logits, fp32 storage
# bf16 heads with d <= 1024: the products of two bf16 values are exact in fp32, so the only error is
# the fp32 accumulation of d terms, at most d * 2^-23 * sum|w_j h_j| even if every add truncates:
# 1024 * 1.2e-7 * (1024 * 0.02 * 0.8) ~ 2e-3 in the worst case, a few 1e-5 in practice.  One wrong
# mask bit moves a logit by |w_j h_j| / (1-p) ~ 2e-2, which this bound no longer hides.
TOL_LOGIT_BF16_SMALL_D = 1e-3


def check_chain(got, ref, draft, rule=oracle.RULE_NAIVE):
    """got: dict of numpy arrays from the CUDA path; ref: oracle.verify_batched output."""
    tok, rtok = got["tokens"], ref["tokens"]
    B, T, K = rtok.shape
    assert tok.shape == rtok.shape
    differ = tok != rtok
    bad = differ & (ref["gap"] >= NEAR_TIE)
    assert not bad.any(), f"{int(bad.sum())} token mismatches outside near-ties, e.g. {np.argwhere(bad)[:4].tolist()}"
    # integer stages, exact, on the GPU's own tokens
    for b in range(B):
        for t in range(T):
            cnt, hits = oracle.counts(tok[b, t], int(draft[b, t]))
            assert np.array_equal(got["counts"][b, t], cnt)
            if got.get("hits") is not None:
                assert got["hits"][b, t] == hits
        assert got["accept_len"][b] == oracle.accept_chain(tok[b], draft[b], rule)
    # and against the oracle's end-to-end values wherever no token differed
    same_pos = ~differ.any(axis=2)
    assert np.array_equal(got["counts"][same_pos], ref["counts"][same_pos])
    same_seq = same_pos.all(axis=1)
    assert np.array_equal(got["accept_len"][same_seq], ref["accept_len"][same_seq])
    return int(differ.sum())


def check_tree(got, ref, node_token, node_parent, node_hrow, rule=oracle.RULE_NAIVE):
    tok, rtok = got["tokens"], ref["tokens"]
    B = rtok.shape[0]
    differ = tok != rtok
    bad = differ & (ref["gap"] >= NEAR_TIE)
    assert not bad.any(), f"{int(bad.sum())} token mismatches outside near-ties"
    for b in range(B):
        L, best, ok = oracle.accept_tree(tok[b], node_token[b], node_parent[b], node_hrow[b], rule)
        assert got["accept_len"][b] == L and got["best_node"][b] == best
        assert np.array_equal(got["node_ok"][b], ok)
        for q in range(tok.shape[1]):
            assert np.array_equal(got["counts"][b, q], oracle.counts(tok[b, q], -1)[0])
    same_seq = ~differ.any(axis=(1, 2))
    for key in ("accept_len", "best_node", "node_ok", "counts"):
        assert np.array_equal(got[key][same_seq], ref[key][same_seq]), key
    return int(differ.sum())


def to_np(d):
    return {k: (v.cpu().numpy() if v is not None else None) for k, v in d.items()}
