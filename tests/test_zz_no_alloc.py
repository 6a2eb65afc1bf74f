"""dropmatch_verify_batched_static, the entry point for hosts that cannot allocate device memory
when they verify (a server whose pool owns all of HBM, a decode loop that may not stall on
cudaMalloc, a plug-in without a context of its own).  It must give exactly what the context-based
call gives on the same kernel family, call after call, although every call reuses one fixed
scratch array inside the library; and both are refereed by the CPU oracle.  Collected last on
purpose: a stop-at-first-failure run has then already run every other test."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import check_chain

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
KEYS = ("tokens", "counts", "hits", "accept_len")


def _np(d):
    return {k: d[k].cpu().numpy().copy() for k in KEYS}


@pytest.mark.parametrize("cfg", [
    wl.Config("static_f32", d=256, V=4096, dtype=wl.F32, B=1, T=4, K=8, p=0.1, draft_mode="toy"),
    wl.Config("static_bf16", d=512, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.2),
], ids=lambda c: c.name)
@pytest.mark.parametrize("rule", [binding.RULE_NAIVE, binding.RULE_MAJORITY])
def test_static_entry_point_matches_context_entry_point_twice(cfg, rule):
    work = wl.make_workload(cfg, device=DEV)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        ctx.set_impl(binding.IMPL_SIMT)          # the static call runs the CUDA-core kernels
        out = None
        for call, seed in enumerate((wl.MASK_SEED, wl.MASK_SEED + 12345)):
            want = _np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, seed, seq_base=5, rule=rule))
            out = binding.verify_batched_static(work.W, work.H, work.draft, cfg.K, cfg.p, seed, seq_base=5,
                                                rule=rule, out=out)   # second call reuses the outputs
            torch.cuda.synchronize()
            got = _np(out)
            for key in KEYS:   # integer results of the same kernels on the same inputs: bit-exact
                assert np.array_equal(got[key], want[key]), (call, key)
            draft = work.draft.cpu().numpy()
            ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft,
                                        cfg.K, cfg.p, seed, seq_base=5, rule=rule)
            check_chain(got, ref, draft, rule)   # and what the oracle computes from Eq. 1-3 and Sec. 3.2
        assert ctx.device_error() == 0
    finally:
        ctx.close()


def test_static_entry_point_rejects_calls_beyond_its_scratch():
    cfg = wl.Config("static_big", d=64, V=256, dtype=wl.BF16, B=3, T=11, K=8, p=0.1)   # 264 rows > 256
    assert cfg.rows > binding.STATIC_MAX_ROWS
    work = wl.make_workload(cfg, device=DEV)
    with pytest.raises(pk.DropMatchError) as e:
        binding.verify_batched_static(work.W, work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED)
    assert e.value.status == binding.ESTATICLIMIT
    assert "fixed scratch" in str(e.value)
