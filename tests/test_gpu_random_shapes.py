"""Seeded random shapes through every kernel family against the oracle: small heads with odd
sizes, and wide-vocabulary heads with few hidden elements so that the staged, CTA-pair and
two-row-block launches are reached while the oracle still finishes in a second or two."""
import numpy as np
import pytest

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import check_chain, to_np

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"


def _random_configs():
    rng = np.random.default_rng(20260401)
    cfgs = []
    for n in range(10):                                   # small heads, odd sizes
        bf16 = bool(rng.integers(2))
        d = int(rng.choice([64, 128, 192, 320, 512]) if bf16 and rng.random() < 0.7 else 8 * rng.integers(1, 40))
        cfgs.append(wl.Config(f"rand_small{n}", d=d, V=int(rng.integers(3, 3000)), dtype=wl.BF16 if bf16 else wl.F32,
                              B=int(rng.integers(1, 4)), T=int(rng.integers(1, 6)), K=int(rng.integers(1, 20)),
                              p=float(rng.choice([0.0, 0.05, 0.1, 0.3, 0.6])), draft_mode="toy"))
    for n in range(8):                                    # wide vocabularies: several tiles per CTA
        cfgs.append(wl.Config(f"rand_wide{n}", d=int(rng.choice([64, 128])), V=int(rng.integers(20000, 90000)),
                              dtype=wl.BF16, B=int(rng.integers(1, 5)), T=int(rng.integers(2, 9)),
                              K=int(rng.choice([4, 8, 16, 24, 32])), p=float(rng.choice([0.1, 0.2, 0.4]))))
    return cfgs


@pytest.mark.parametrize("cfg", _random_configs(), ids=lambda c: f"{c.name}-d{c.d}-V{c.V}-r{c.rows}")
def test_random_shape(cfg):
    if cfg.V < 5:
        pytest.skip("the draft recipe needs five vocabulary entries")
    work = wl.make_workload(cfg, device=DEV)
    ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                                work.draft.cpu().numpy(), cfg.K, cfg.p, SEED, seq_base=7, rule=oracle.RULE_MAJORITY)
    impls = [binding.IMPL_SIMT] + ([binding.IMPL_TCGEN05] if cfg.dtype == wl.BF16 and cfg.d % 64 == 0 else [])
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
        for impl in impls:
            ctx.set_impl(impl)
            got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=7,
                                           rule=binding.RULE_MAJORITY))
            assert ctx.device_error() == 0 and ctx.last_impl() == impl
            n_diff = check_chain(got, ref, work.draft.cpu().numpy(), oracle.RULE_MAJORITY)
            assert n_diff <= max(2, cfg.rows // 10)
    finally:
        ctx.close()
