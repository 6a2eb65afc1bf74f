"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The oracle needs V*d fp64 multiply-adds per path (half a second at the Llama-3-8B head).  The
benchmarked call (Llama-3-8B head, 40 paths) is compared with it in full.  The larger calls are
compared on a sample of paths spread evenly over the call's rows, so that every kernel launch
and both row blocks of a two-block launch are hit: decoded tokens (outside near-ties) and full
logit rows, one by one.  Everything that is integer work is checked in full from the GPU's own
tokens with the oracle's integer routines: multiplicities, hits, accepted lengths, tree walks;
masks are compared bit for bit on sampled paths."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import NEAR_TIE, TOL_LOGIT_BF16, check_chain, to_np

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"


def _sample_paths(cfg, n, rng):
    """n paths (b, t, i), one from each of n equal stretches of the call's rows (row = (b*T+t)*K+i):
    every launch of up to 256 (or 2 x 256) rows gets its share."""
    rows = cfg.rows
    n = min(n, rows)
    picks = sorted({min(rows - 1, int((k + rng.random()) * rows / n)) for k in range(n)})
    return [(r // (cfg.T * cfg.K), (r // cfg.K) % cfg.T, r % cfg.K) for r in picks]


def _check_sampled_paths(ctx, cfg, work, got_tokens, paths, seq_base=0):
    Wn, Hn = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H)
    sel = torch.tensor(paths, dtype=torch.int32, device=DEV)
    logits = ctx.debug_logits(work.H, sel, cfg.p, SEED, seq_base=seq_base).cpu().numpy()
    assert ctx.device_error() == 0
    near = 0
    for n, (b, t, i) in enumerate(paths):
        exp = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, seq_base + b, t, i)
        assert np.abs(logits[n] - exp).max() < TOL_LOGIT_BF16, (b, t, i)
        tok, gap = oracle.argmax(exp)
        if got_tokens[b, t, i] != tok:
            assert gap < NEAR_TIE, f"path {(b, t, i)}: token {got_tokens[b, t, i]} vs {tok}, gap {gap}"
            near += 1
    return near


def _check_masks(ctx, cfg, paths, seq_base=0):
    got = ctx.debug_masks(cfg.B, cfg.T, cfg.K, cfg.d, cfg.p, SEED, seq_base=seq_base).cpu().numpy().view(np.uint32)
    thr = oracle.drop_threshold(cfg.p)
    for (b, t, i) in paths[:4]:
        bits = np.array([oracle.mask_keep(SEED, seq_base + b, t, i, j, thr) for j in range(0, cfg.d, 7)], dtype=np.uint32)
        js = np.arange(0, cfg.d, 7)
        assert np.array_equal((got[b, t, i, js // 32] >> (js % 32)) & 1, bits)


def test_bench_workload_every_path():
    """The call bench.py times (Llama-3-8B head, B=1, T=5, K=8: 40 paths; the mask pass and the head
    kernel, which finishes the call itself) against the oracle's whole call: all 40 tokens, counts,
    hits and the accepted length."""
    cfg = wl.CONFIGS["llama8b"]
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05 and ctx.last_launches() == 2
        draft = work.draft.cpu().numpy()
        ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft,
                                    cfg.K, cfg.p, SEED)
        n_diff = check_chain(got, ref, draft)
        near = int((ref["gap"] < NEAR_TIE).sum())
        print(f"llama8b: {n_diff} of {cfg.rows} tokens differ, all inside the {near} near-tie rows")
        assert n_diff <= near
    finally:
        ctx.close()


@pytest.mark.parametrize("name,overrides,n_paths", [
    ("llama8b", dict(K=32, T=8), 16),                 # 256 rows: staged operand, CTA pairs
    ("qwen8b", dict(K=16), 8),                        # 112 rows: staged operand, three groups
    ("qwen8b", dict(K=32, p=0.2), 8),                 # 224 rows: two accumulator slots, exposed epilogue
])
def test_chain_configs_at_full_size(name, overrides, n_paths):
    cfg = wl.CONFIGS[name].with_(**overrides)
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05
        draft = work.draft.cpu().numpy()
        for b in range(cfg.B):                        # integer stages, in full, from the GPU's tokens
            for t in range(cfg.T):
                cnt, hits = oracle.counts(got["tokens"][b, t], int(draft[b, t]))
                assert np.array_equal(got["counts"][b, t], cnt) and got["hits"][b, t] == hits
            assert got["accept_len"][b] == oracle.accept_chain(got["tokens"][b], draft[b], oracle.RULE_NAIVE)
        assert (got["tokens"] >= 0).all() and (got["tokens"] < cfg.V).all()
        paths = _sample_paths(cfg, n_paths, np.random.default_rng(11))
        _check_masks(ctx, cfg, paths)
        _check_sampled_paths(ctx, cfg, work, got["tokens"], paths)
        # the accepted drafts of this recipe are plausible ones: something is accepted somewhere
        assert got["hits"].sum() > 0
    finally:
        ctx.close()


def test_tree_config_at_full_size():
    cfg0 = wl.CONFIGS["tree"]
    work = wl.make_workload(cfg0, device=DEV)
    cfg = work.cfg                                    # T = hidden rows per sequence of the drawn trees
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        got = to_np(ctx.verify_tree(work.H, work.node_token, work.node_parent, work.node_hrow, cfg.K, cfg.p, SEED))
        assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05
        nt, npar, nh = (x.cpu().numpy() for x in (work.node_token, work.node_parent, work.node_hrow))
        for b in range(cfg.B):
            L, best, ok = oracle.accept_tree(got["tokens"][b], nt[b], npar[b], nh[b], oracle.RULE_NAIVE)
            assert got["accept_len"][b] == L and got["best_node"][b] == best
            assert np.array_equal(got["node_ok"][b], ok)
            assert 0 <= L <= 7
            for q in range(cfg.T):
                assert np.array_equal(got["counts"][b, q], oracle.counts(got["tokens"][b, q], -1)[0])
        paths = _sample_paths(cfg, 32, np.random.default_rng(12))   # several paths in every launch and row block
        _check_sampled_paths(ctx, cfg, work, got["tokens"], paths)
    finally:
        ctx.close()


def test_llama70b_config_sampled():
    cfg = wl.CONFIGS["llama70b"]
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        assert ctx.device_error() == 0
        draft = work.draft.cpu().numpy()
        for b in range(cfg.B):
            assert got["accept_len"][b] == oracle.accept_chain(got["tokens"][b], draft[b], oracle.RULE_NAIVE)
        paths = _sample_paths(cfg, 32, np.random.default_rng(13))   # 2048 rows: four two-block launches, eight paths each
        _check_sampled_paths(ctx, cfg, work, got["tokens"], paths)
    finally:
        ctx.close()


@pytest.mark.parametrize("name,reps", [("llama8b", 300), ("llama8b_k32", 100), ("llama8b_b2k32", 60)])
def test_full_size_runs_are_deterministic(name, reps):
    """The same call repeated back to back (one launch; CTA pairs; two row blocks per launch) must
    give the same bytes every time, also when other seeds run in between: a missed barrier or a
    stale partial would show up here long before it shows up in a parity sample."""
    cfg = wl.CONFIGS[name]
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        first = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        scratch = ctx.alloc_outputs(cfg.B, cfg.T, cfg.K)
        for n in range(reps):
            ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED + 1 + n, out=scratch)   # another seed in between
            again = ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED)
            if n % 20 == 19 or n == reps - 1:
                got = to_np(again)
                for key in first:
                    assert np.array_equal(first[key], got[key]), (n, key)
        assert ctx.device_error() == 0
    finally:
        ctx.close()
