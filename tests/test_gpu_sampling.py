"""GPU parity of the sampling decode rule (dropmatch_verify_batched_sampled) against the oracle:
the drawn tokens must be identical except where the oracle's two best perturbed keys
(logit / temperature + Gumbel noise) are closer than the near-tie bound; counts, hits and accepted
lengths are integer work on the tokens and must match exactly.  With a nucleus (top_p < 1) the
GPU sums fp32 probabilities where the oracle sums fp64 ones: where the running mass passes top_p
within 1e-4 the boundary token may differ, so a token may also equal the oracle's draw at
top_p * (1 -+ 1e-4); such rows are counted and must stay rare."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import check_chain, to_np

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"

CASES = [
    (wl.CONFIGS["toy"], 1.0),                                                           # fp32 head, CUDA cores
    (wl.Config("s_bf16", d=512, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1), 0.7),     # one group, one launch
    (wl.Config("s_staged", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1), 1.3),  # staged operand, pairs
    (wl.Config("s_two_blocks", d=64, V=20000, dtype=wl.BF16, B=3, T=8, K=25, p=0.1), 1.0),  # 600 paths
    (wl.Config("s_odd_d", d=136, V=999, dtype=wl.BF16, B=1, T=3, K=4, p=0.1), 2.0),      # CUDA cores, bf16
]


@pytest.mark.parametrize("cfg,tau", CASES, ids=lambda c: getattr(c, "name", str(c)))
def test_sampled_tokens_match_the_oracle(cfg, tau):
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        got = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=tau, seq_base=3))
        assert ctx.device_error() == 0
        draft = work.draft.cpu().numpy()
        ref = oracle.verify_batched_sampled(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft,
                                            cfg.K, cfg.p, SEED, temperature=tau, top_p=1.0, seq_base=3)
        n_diff = check_chain(got, ref, draft)
        assert n_diff <= max(2, cfg.rows // 10)
        # it does sample: with noise of the size of the logits' spread the paths of a position disagree
        plain = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=3))
        assert (got["tokens"] != plain["tokens"]).mean() > 0.5
        # reproducible from the indices alone
        again = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=tau, seq_base=3))
        assert np.array_equal(again["tokens"], got["tokens"])
    finally:
        ctx.close()


def test_cold_temperature_is_the_argmax_call_and_top_p_is_refused():
    cfg = wl.Config("s_cold", d=256, V=2000, dtype=wl.BF16, B=2, T=4, K=6, p=0.2)
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        cold = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=1e-6))
        plain = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(cold[key], plain[key]), key
        with pytest.raises(pk.DropMatchError) as e:     # the nucleus needs the logits buffer of dm_enable_js
            ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=1.0, top_p=0.9)
        assert e.value.status == binding.EWORKSPACE
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=0.0)
        assert e.value.status == binding.EINVAL
    finally:
        ctx.close()


NUCLEUS_CASES = [
    (wl.CONFIGS["toy"], 1.0, 0.9),
    (wl.Config("n_bf16", d=512, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1), 0.7, 0.5),
    (wl.Config("n_flat", d=256, V=20000, dtype=wl.BF16, B=1, T=2, K=16, p=0.2), 3.0, 0.95),   # flat: a nucleus of thousands
    (wl.Config("n_peaked", d=256, V=5000, dtype=wl.BF16, B=2, T=2, K=8, p=0.1), 0.05, 0.3),    # peaked: one or two tokens
    (wl.Config("n_staged", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1), 1.0, 0.8),   # staged head kernel, 192 paths
    (wl.Config("n_tiny", d=64, V=37, dtype=wl.BF16, B=1, T=2, K=4, p=0.3), 1.0, 0.6),
    (wl.Config("n_cluster8", d=128, V=60000, dtype=wl.BF16, B=1, T=1, K=8, p=0.1), 1.5, 0.9),   # eight CTAs per path
    (wl.Config("n_cluster2", d=64, V=9000, dtype=wl.BF16, B=1, T=8, K=8, p=0.1), 1.0, 0.7),     # 64 paths: two CTAs per path
]


@pytest.mark.parametrize("cfg,tau,top_p", NUCLEUS_CASES, ids=lambda c: getattr(c, "name", str(c)))
def test_nucleus_sampling_matches_the_oracle(cfg, tau, top_p):
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        ctx.enable_js(cfg.rows, cfg.B * cfg.T)
        got = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=tau, top_p=top_p,
                                               seq_base=2))
        assert ctx.device_error() == 0
        Wn, Hn, draft = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H), work.draft.cpu().numpy()
        p32 = float(np.float32(top_p))
        ref = oracle.verify_batched_sampled(Wn, cfg.dtype, Hn, draft, cfg.K, cfg.p, SEED, temperature=tau, top_p=p32,
                                            seq_base=2)
        differ = got["tokens"] != ref["tokens"]
        boundary_cases = 0
        for b, t, i in np.argwhere(differ & (ref["gap"] >= 2e-2)):
            logits = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, 2 + b, t, i)
            alts = {oracle.sample_row(logits, tau, p32 * f, SEED, 2 + b, t, i)[0] for f in (1 - 1e-4, 1 + 1e-4)}
            assert got["tokens"][b, t, i] in alts, (b, t, i)
            boundary_cases += 1
        assert boundary_cases <= max(1, cfg.rows // 50)
        # every drawn token lies in the oracle's nucleus at a slightly larger mass
        for b in range(cfg.B):
            for t in range(cfg.T):
                for i in range(0, cfg.K, max(1, cfg.K // 2)):
                    logits = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, 2 + b, t, i)
                    assert oracle.nucleus(logits, tau, min(1.0, p32 * (1 + 1e-3)))[got["tokens"][b, t, i]]
                cnt, hits = oracle.counts(got["tokens"][b, t], int(draft[b, t]))
                assert np.array_equal(got["counts"][b, t], cnt) and got["hits"][b, t] == hits
            assert got["accept_len"][b] == oracle.accept_chain(got["tokens"][b], draft[b])
        again = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=tau, top_p=top_p,
                                                 seq_base=2))
        assert np.array_equal(again["tokens"], got["tokens"])       # reproducible bit for bit
    finally:
        ctx.close()


@pytest.mark.parametrize("top_p", [1.0, 0.9])
def test_sampling_on_the_llama8b_head(top_p):
    """Full-size head (V=128256, d=4096), 16 paths: temperature sampling in the fused epilogue and
    nucleus sampling through the logits buffer, each against the oracle."""
    cfg = wl.CONFIGS["llama8b"].with_(T=2)
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        if top_p < 1.0:
            ctx.enable_js(cfg.rows, cfg.B * cfg.T)
        got = to_np(ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=0.8, top_p=top_p))
        assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05
        Wn, Hn, draft = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H), work.draft.cpu().numpy()
        p32 = float(np.float32(top_p))
        ref = oracle.verify_batched_sampled(Wn, cfg.dtype, Hn, draft, cfg.K, cfg.p, SEED, temperature=0.8, top_p=p32)
        for b, t, i in np.argwhere((got["tokens"] != ref["tokens"]) & (ref["gap"] >= 2e-2)):
            assert top_p < 1.0
            logits = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, b, t, i)
            alts = {oracle.sample_row(logits, 0.8, p32 * f, SEED, b, t, i)[0] for f in (1 - 1e-4, 1 + 1e-4)}
            assert got["tokens"][b, t, i] in alts
        for t in range(cfg.T):
            cnt, hits = oracle.counts(got["tokens"][0, t], int(draft[0, t]))
            assert np.array_equal(got["counts"][0, t], cnt) and got["hits"][0, t] == hits
        assert got["accept_len"][0] == oracle.accept_chain(got["tokens"][0], draft[0])
    finally:
        ctx.close()
