"""GPU parity of the JS-divergence criterion (Algorithm 1) against the oracle, through the C ABI.

Tokens and counts follow the policy of the other parity tests.  Divergences are fp32 sums over
the vocabulary of fp32 logits: |gpu - oracle| <= JS_ABS + JS_REL * oracle.  Eq. 5 compares two
such numbers, so its outcome must match the oracle's except where the oracle's own margin
|JS(draft) - max JS(heads)| is inside that error band (counted).  The accepted length is integer
work and must equal Algorithm 1 re-run on the GPU's own tokens and Eq. 5 outcomes."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import NEAR_TIE, to_np

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"
JS_ABS, JS_REL = 2e-5, 2e-3
LAUNCHES = {}     # kernels of the latest verify_js call of each configuration
# head kernel(s) (+ the mask pass of staged operands) + the sweeps: one cooperative kernel where the
# call's logits fit the shared memory of the GPU, else two, else (K > 32) three
EXPECT_LAUNCHES = {"js_bf16_a": 1 + 1, "js_bf16_staged": 2 + 2, "js_rows288": 4 + 2, "js_k24": 1 + 1, "js_k40": 1 + 3,
                   "llama8b": 2 + 1}


def _run(cfg, impl=binding.IMPL_AUTO, seq_base=0, noise=None):
    work = wl.make_workload(cfg, device=DEV)
    n_pos = cfg.B * cfg.T
    if noise is None:   # some positions with a draft close to the target, some far from it
        noise = np.linspace(0.02, 1.2, n_pos)
    dp = wl.make_draft_probs(work.W, work.H.reshape(n_pos, cfg.d), noise).view(cfg.B, cfg.T, cfg.V)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=max(cfg.rows, 16), max_hidden_rows=n_pos)
        ctx.enable_js(cfg.rows, n_pos)
        ctx.set_impl(impl)
        got = to_np(ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED, seq_base=seq_base))
        assert ctx.device_error() == 0
        LAUNCHES[cfg.name] = ctx.last_launches()
        again = to_np(ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED, seq_base=seq_base))
        for key in got:      # the counters the sweeps leave behind are ready for the next call
            assert np.array_equal(got[key], again[key], equal_nan=got[key].dtype.kind == "f"), key
    finally:
        ctx.close()
    ref = oracle.verify_js(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                           work.draft.cpu().numpy(), dp.cpu().numpy(), cfg.K, cfg.p, SEED, seq_base=seq_base)
    return got, ref, work.draft.cpu().numpy()


def _check(got, ref, draft, cfg):
    B, T, K = cfg.B, cfg.T, cfg.K
    differ = got["tokens"] != ref["tokens"]
    # a near-tie that flips a token is allowed (the oracle's verify_js does not report gaps, so the
    # plain call's policy is applied by the caller where it matters); here tokens must simply agree
    assert not differ.any(), f"{int(differ.sum())} token mismatches"
    assert np.array_equal(got["counts"], ref["counts"])
    err = np.abs(got["js"].astype(np.float64) - ref["js"])
    assert (err <= JS_ABS + JS_REL * ref["js"]).all(), f"max JS error {err.max()} at {np.unravel_index(err.argmax(), err.shape)}"
    margin = np.abs(ref["js"][..., K] - ref["js"][..., :K].max(axis=-1))
    band = 2 * (JS_ABS + JS_REL * ref["js"].max(axis=-1))
    flips = got["js_ok"] != ref["js_ok"]
    assert not (flips & (margin > band)).any(), "Eq. 5 outcome differs outside the error band"
    for b in range(B):          # Algorithm 1 + scan, re-run on the GPU's own integers
        run, open_ = 0, True
        for t in range(T):
            ok = bool(got["js_ok"][b, t]) or oracle.majority_token(got["tokens"][b, t]) == draft[b, t]
            if open_ and ok:
                run += 1
            else:
                open_ = False
        assert got["accept_len"][b] == run
    same = ~flips.any(axis=1)
    assert np.array_equal(got["accept_len"][same], ref["accept_len"][same])
    return int(flips.sum())


SMALL = [
    wl.Config("js_bf16_a", d=512, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1),          # one group, in-kernel masks
    wl.Config("js_bf16_b", d=256, V=9000, dtype=wl.BF16, B=1, T=4, K=5, p=0.3),          # K that does not divide 16
    wl.Config("js_bf16_staged", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1),   # staged operand, CTA pairs
    wl.Config("js_f32", d=100, V=517, dtype=wl.F32, B=2, T=3, K=7, p=0.2, draft_mode="toy"),   # CUDA-core family
    wl.Config("js_k1", d=256, V=700, dtype=wl.BF16, B=1, T=2, K=1, p=0.2),
    wl.Config("js_rows288", d=128, V=40000, dtype=wl.BF16, B=3, T=6, K=16, p=0.1),       # two head launches with logits
    wl.Config("js_k24", d=128, V=5000, dtype=wl.BF16, B=1, T=3, K=24, p=0.2),            # 17..32 paths in registers
    wl.Config("js_k40", d=128, V=2000, dtype=wl.BF16, B=1, T=2, K=40, p=0.2),            # more than fit: series by series
    # many positions on a tiny vocabulary: the shares of the call do not fit the last block's scratch
    wl.Config("js_many_pos", d=64, V=50, dtype=wl.BF16, B=2, T=50, K=2, p=0.2, draft_mode="toy"),
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
def test_js_small_heads(cfg):
    got, ref, draft = _run(cfg, seq_base=3)
    _check(got, ref, draft, cfg)
    if cfg.name in EXPECT_LAUNCHES:
        assert LAUNCHES[cfg.name] == EXPECT_LAUNCHES[cfg.name]
    if cfg.K > 1:
        assert ref["js_ok"].any() or ref["js"][..., cfg.K].min() > 0      # the workload is not degenerate


def test_js_eq5_takes_both_outcomes_somewhere():
    cfg = wl.Config("js_both", d=512, V=4000, dtype=wl.BF16, B=4, T=4, K=8, p=0.3)
    got, ref, draft = _run(cfg, noise=np.tile([0.01, 0.05, 0.6, 1.5], 4))
    _check(got, ref, draft, cfg)
    assert ref["js_ok"].any() and not ref["js_ok"].all()


def test_js_needs_its_buffers():
    cfg = wl.Config("js_err", d=256, V=1000, dtype=wl.BF16, B=1, T=2, K=4, p=0.1)
    work = wl.make_workload(cfg, device=DEV)
    dp = wl.make_draft_probs(work.W, work.H.reshape(2, cfg.d), 0.1).view(1, 2, cfg.V)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=cfg.rows)
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED)
        assert e.value.status == binding.EWORKSPACE
        ctx.enable_js(cfg.rows, 2)
        ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED)
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_js(work.H, work.draft, dp, 2 * cfg.K, cfg.p, SEED)    # more rows than reserved
        assert e.value.status == binding.EWORKSPACE
        with pytest.raises(pk.DropMatchError):
            ctx.enable_js(cfg.rows + 1, 2)                                   # beyond dm_set_head's max_rows
    finally:
        ctx.close()


def test_js_llama8b_full_size():
    cfg = wl.CONFIGS["llama8b"]
    got, ref, draft = _run(cfg)
    assert LAUNCHES[cfg.name] == EXPECT_LAUNCHES[cfg.name]
    tok_diff = got["tokens"] != ref["tokens"]
    if tok_diff.any():      # full size: allow near-tie flips, judged by the plain oracle's gaps
        work = wl.make_workload(cfg, device="cpu")
        plain = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                                      draft, cfg.K, cfg.p, SEED)
        assert not (tok_diff & (plain["gap"] >= NEAR_TIE)).any()
        pytest.skip("a near-tie flipped a token; divergences are checked by the other tests")
    _check(got, ref, draft, cfg)


@pytest.mark.parametrize("cfg", [
    wl.Config("js_graph_one", d=256, V=9000, dtype=wl.BF16, B=1, T=4, K=8, p=0.2),        # sweeps in one cooperative launch
    wl.Config("js_graph_two", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1),      # sweeps in two launches
], ids=lambda c: c.name)
def test_js_call_in_a_cuda_graph(cfg):
    """dropmatch_verify_js only enqueues work: captured into a CUDA graph and replayed it gives the
    eager call's results (the oracle referees the eager call in the tests above)."""
    work = wl.make_workload(cfg, device=DEV)
    n_pos = cfg.B * cfg.T
    dp = wl.make_draft_probs(work.W, work.H.reshape(n_pos, cfg.d), np.linspace(0.02, 1.2, n_pos)).view(cfg.B, cfg.T, cfg.V)
    ctx = pk.Context(0)
    try:
        ctx.set_head(work.W, max_rows=max(cfg.rows, 16), max_hidden_rows=n_pos)
        ctx.enable_js(cfg.rows, n_pos)
        want = to_np(ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED, seq_base=2))
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            out = ctx.verify_js(work.H, work.draft, dp, cfg.K, cfg.p, SEED, seq_base=2)
        for _ in range(3):
            for t in out.values():
                t.zero_()
            graph.replay()
            torch.cuda.synchronize()
            got = to_np(out)
            for key in want:
                assert np.array_equal(got[key], want[key], equal_nan=want[key].dtype.kind == "f"), key
        assert ctx.device_error() == 0
    finally:
        ctx.close()
