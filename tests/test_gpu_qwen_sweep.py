"""The Qwen3-8B-shaped head sweep (d=4096, V=151936, T=7): K in {4,8,16,32} x p in {0.05,0.1,0.2} at
B=1, and K=8, p=0.1 at B=8 and B=32, each at full size in the bench launch configuration.

One head is built once for the module.  Per point: integer stages (counts, hits, accepted
lengths) are checked in full from the GPU's own tokens with the oracle's integer routines, the
tokens must lie in the vocabulary, and eight paths spread evenly over the call's rows are compared
one by one with the oracle (token outside near-ties, full logit row within the bf16 bound)."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import NEAR_TIE, TOL_LOGIT_BF16, to_np

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"
BASE = wl.CONFIGS["qwen8b"]
POINTS = [(1, K, p) for K in (4, 8, 16, 32) for p in (0.05, 0.1, 0.2)] + [(8, 8, 0.1), (32, 8, 0.1)]


@pytest.fixture(scope="module")
def head():
    W = wl.make_head(BASE.V, BASE.d, BASE.dtype, seed=1, device=DEV)
    ctx = pk.Context(0)
    ctx.set_head(W, max_rows=32 * BASE.T * 8, max_hidden_rows=32 * BASE.T)
    yield W, wl.to_numpy_storage(W), ctx
    ctx.close()


@pytest.mark.parametrize("B,K,p", POINTS)
def test_qwen_sweep_point(head, B, K, p):
    W, Wn, ctx = head
    cfg = BASE.with_(B=B, K=K, p=p)
    work = wl.make_workload(cfg, device=DEV, W=W)
    got = to_np(ctx.verify_batched(work.H, work.draft, K, p, SEED, seq_base=11))
    assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05
    draft = work.draft.cpu().numpy()
    assert (got["tokens"] >= 0).all() and (got["tokens"] < cfg.V).all()
    for b in range(B):
        for t in range(cfg.T):
            cnt, hits = oracle.counts(got["tokens"][b, t], int(draft[b, t]))
            assert np.array_equal(got["counts"][b, t], cnt) and got["hits"][b, t] == hits
        assert got["accept_len"][b] == oracle.accept_chain(got["tokens"][b], draft[b], oracle.RULE_NAIVE)
    rng = np.random.default_rng(1000 * B + 10 * K + int(100 * p))
    # eight paths, one from each eighth of the call's rows (every launch and row block is hit)
    rows = [min(cfg.rows - 1, int((k + rng.random()) * cfg.rows / 8)) for k in range(8)]
    paths = sorted({(r // (cfg.T * K), (r // K) % cfg.T, r % K) for r in rows})
    Hn = wl.to_numpy_storage(work.H)
    sel = torch.tensor(paths, dtype=torch.int32, device=DEV)
    logits = ctx.debug_logits(work.H, sel, p, SEED, seq_base=11).cpu().numpy()
    for n, (b, t, i) in enumerate(paths):
        exp = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], p, SEED, 11 + b, t, i)
        assert np.abs(logits[n] - exp).max() < TOL_LOGIT_BF16
        tok, gap = oracle.argmax(exp)
        assert got["tokens"][b, t, i] == tok or gap < NEAR_TIE
