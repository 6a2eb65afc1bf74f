"""GPU parity of the sampling decode rule (dropmatch_verify_batched_sampled) against the oracle:
the drawn tokens must be identical except where the oracle's two best perturbed keys
(logit / temperature + Gumbel noise) are closer than the near-tie bound; counts, hits and accepted
lengths are integer work on the tokens and must match exactly."""
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
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=1.0, top_p=0.9)
        assert e.value.status == binding.EUNSUPPORTED
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_batched_sampled(work.H, work.draft, cfg.K, cfg.p, SEED, temperature=0.0)
        assert e.value.status == binding.EINVAL
    finally:
        ctx.close()
