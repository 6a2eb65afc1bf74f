"""What happens when a kernel gives up on one of its internal waits.

Every wait inside the tensor-core kernel has a time limit; when it runs out the kernel sets the
context's device error word, winds down (shared memory and TMEM are released as usual) and
returns.  A consumer further down the stream must not mistake the outputs of such a call for
results, so the device itself writes the fail-safe values (no token, nothing accepted).  The test
makes a wait run out by setting the limit to a few clock cycles on a tiny head: nothing hangs and
nothing faults, the call simply comes back early.  The next call, with the default limit
restored, must again match the oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import check_chain, to_np

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_wait_that_runs_out_gives_fail_safe_outputs_and_the_context_recovers():
    cfg = wl.Config("tiny", d=256, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1)
    work = wl.make_workload(cfg, device=DEV)
    draft = work.draft.cpu().numpy()
    ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft, cfg.K,
                                cfg.p, wl.MASK_SEED)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        good = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED))
        assert ctx.device_error() == 0 and ctx.last_impl() == binding.IMPL_TCGEN05
        check_chain(good, ref, draft)

        ctx.debug_set_wait_limit(1)           # the first wait that is not satisfied at once gives up
        out = ctx.alloc_outputs(cfg.B, cfg.T, cfg.K)
        for t in out.values():
            t.fill_(12345)
        ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED, out=out)
        torch.cuda.synchronize()              # the kernel returns by itself
        bad = to_np(out)
        assert (bad["tokens"] == -1).all() and (bad["counts"] == 0).all()
        assert (bad["hits"] == 0).all() and (bad["accept_len"] == 0).all()
        assert ctx.device_error() != 0        # reads and clears the word
        assert ctx.device_error() == 0

        ctx.debug_set_wait_limit(0)           # default again: the context is as good as new
        again = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED))
        assert ctx.device_error() == 0
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(again[key], good[key]), key
    finally:
        ctx.close()
