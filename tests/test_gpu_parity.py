"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle, element by
element, on the same seeded inputs."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import binding, workloads as wl
from parity_util import (NEAR_TIE, TOL_LOGIT_BF16, TOL_LOGIT_BF16_SMALL_D, TOL_LOGIT_F32, check_chain, check_tree,
                         to_np)

pytestmark = pytest.mark.gpu
SEED = wl.MASK_SEED
DEV = "cuda:0"


@pytest.fixture(scope="module")
def ctx():
    c = pk.Context(0)
    yield c
    c.close()


def _impls(ctx, cfg):
    """Kernel families that can serve this head: always the CUDA-core one, plus tcgen05 for bf16, d % 64 == 0."""
    out = [binding.IMPL_SIMT]
    if cfg.dtype == wl.BF16 and cfg.d % 64 == 0:
        out.append(binding.IMPL_TCGEN05)
    return out


def _run_chain(ctx, cfg, impl, rule=oracle.RULE_NAIVE, seq_base=0, work=None):
    work = work or wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=max(cfg.rows, 16), max_hidden_rows=cfg.B * cfg.T)
    ctx.set_impl(impl)
    try:
        got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=seq_base, rule=rule))
        assert ctx.device_error() == 0
        assert ctx.last_impl() == impl
    finally:
        ctx.set_impl(binding.IMPL_AUTO)
    ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                                work.draft.cpu().numpy(), cfg.K, cfg.p, SEED, seq_base=seq_base, rule=rule)
    n_diff = check_chain(got, ref, work.draft.cpu().numpy(), rule)
    return got, ref, n_diff, work


@pytest.mark.parametrize("shape", [(1, 4, 8, 256), (2, 3, 5, 200), (1, 1, 1, 4), (3, 2, 32, 4096), (1, 2, 3, 33)])
@pytest.mark.parametrize("p", [0.0, 0.1, 0.5])
def test_masks_bit_exact(ctx, shape, p):
    B, T, K, d = shape
    got = ctx.debug_masks(B, T, K, d, p, SEED, seq_base=7).cpu().numpy().view(np.uint32)
    assert np.array_equal(got, oracle.masks(B, T, K, d, p, SEED, 7))


@pytest.mark.parametrize("shape,p", [((2, 3, 16, 256), 0.1), ((1, 9, 16, 192), 0.3), ((3, 8, 25, 64), 0.5),
                                     ((1, 2, 8, 4096), 0.1)])
def test_staged_masked_operand_elementwise(ctx, shape, p):
    """The masked hidden rows that the tensor-core kernel stages for wide calls (Eq. 1, and Eq. 2
    without its scale): every element equals the oracle's, so the zero pattern is the mask bit for
    bit and the kept values are the stored hidden-state values unchanged."""
    B, T, K, d = shape
    H = wl.make_hidden(B * T, d, wl.BF16, seed=2, device=DEV).view(B, T, d)
    W = wl.make_head(64, d, wl.BF16, seed=1, device=DEV)
    ctx.set_head(W, max_rows=B * T * K)
    got = ctx.debug_masked_operand(H, K, p, SEED, seq_base=9).float().cpu().numpy()
    assert ctx.device_error() == 0
    Hn = wl.to_numpy_storage(H)
    for b in range(B):
        for t in range(T):
            for i in range(K):
                exp = oracle.masked_hidden(Hn[b, t], wl.BF16, p, SEED, 9 + b, t, i)
                assert np.array_equal(got[(b * T + t) * K + i].astype(np.float64), exp), (b, t, i)


def test_toy_config_fp32(ctx):
    cfg = wl.CONFIGS["toy"]
    got, ref, n_diff, work = _run_chain(ctx, cfg, binding.IMPL_SIMT)
    assert n_diff == 0   # fp32 head: no near-tie is expected to flip at this size
    sel = torch.tensor([[0, t, i] for t in range(cfg.T) for i in (0, 3, 7)], dtype=torch.int32, device=DEV)
    logits = ctx.debug_logits(work.H, sel, cfg.p, SEED).cpu().numpy()
    Wn, Hn = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H)
    for n, (b, t, i) in enumerate(sel.cpu().tolist()):
        exp = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, b, t, i)
        assert np.abs(logits[n] - exp).max() < TOL_LOGIT_F32


SMALL = [
    # several vocabulary tiles with a ragged tail, several k-blocks, rows not a multiple of 16
    wl.Config("bf16_a", d=512, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1),
    wl.Config("bf16_b", d=192, V=1111, dtype=wl.BF16, B=1, T=5, K=5, p=0.3),
    wl.Config("bf16_c", d=1024, V=20000, dtype=wl.BF16, B=3, T=2, K=16, p=0.05),
    wl.Config("bf16_k1", d=256, V=700, dtype=wl.BF16, B=1, T=1, K=1, p=0.2),
    wl.Config("bf16_wide", d=64, V=130, dtype=wl.BF16, B=1, T=2, K=32, p=0.5),
    wl.Config("bf16_odd_d", d=136, V=999, dtype=wl.BF16, B=1, T=3, K=4, p=0.1),      # CUDA-core only
    wl.Config("f32_b", d=100, V=517, dtype=wl.F32, B=2, T=3, K=7, p=0.2, draft_mode="toy"),
    wl.Config("bf16_rows200", d=256, V=2500, dtype=wl.BF16, B=5, T=5, K=8, p=0.1),
    wl.Config("bf16_rows300", d=128, V=1500, dtype=wl.BF16, B=3, T=10, K=10, p=0.1),
    # vocabulary slices of several tiles per CTA whose accumulators do not all fit in TMEM at once
    # (staged masked operand): four groups of one tile, two groups of two tiles, three groups
    wl.Config("bf16_groups4", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1),
    wl.Config("bf16_groups2", d=256, V=61111, dtype=wl.BF16, B=2, T=4, K=16, p=0.2),
    wl.Config("bf16_groups_nocache", d=192, V=50000, dtype=wl.BF16, B=1, T=9, K=16, p=0.1),
    # 600 paths: one launch that takes two blocks of 256 side by side, then one of 88
    wl.Config("bf16_two_blocks", d=64, V=40000, dtype=wl.BF16, B=3, T=8, K=25, p=0.1),
    wl.Config("bf16_two_blocks_exact", d=128, V=30000, dtype=wl.BF16, B=2, T=8, K=32, p=0.2),   # exactly 512
]


@pytest.mark.parametrize("cfg", SMALL, ids=lambda c: c.name)
@pytest.mark.parametrize("rule", [oracle.RULE_NAIVE, oracle.RULE_MAJORITY])
def test_small_heads_all_impls(ctx, cfg, rule):
    for impl in _impls(ctx, cfg):
        got, ref, n_diff, work = _run_chain(ctx, cfg, impl, rule=rule, seq_base=3)
        assert n_diff <= max(2, cfg.rows // 10)
        sel_l = [[b, t, i] for b in range(cfg.B) for t in range(cfg.T) for i in (0, cfg.K - 1)][:12]
        sel = torch.tensor(sel_l, dtype=torch.int32, device=DEV)
        ctx.set_impl(impl)
        logits = ctx.debug_logits(work.H, sel, cfg.p, SEED, seq_base=3).cpu().numpy()
        ctx.set_impl(binding.IMPL_AUTO)
        assert ctx.device_error() == 0
        Wn, Hn = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H)
        tol = TOL_LOGIT_F32 if cfg.dtype == wl.F32 else (TOL_LOGIT_BF16_SMALL_D if cfg.d <= 1024 else TOL_LOGIT_BF16)
        for n, (b, t, i) in enumerate(sel_l):
            exp = oracle.logits_row(Wn, cfg.dtype, Hn[b, t], cfg.p, SEED, 3 + b, t, i)
            assert np.abs(logits[n] - exp).max() < tol, (impl, b, t, i)


def test_p_zero_is_greedy_verification(ctx):
    cfg = wl.Config("p0", d=256, V=2000, dtype=wl.BF16, B=2, T=4, K=6, p=0.0)
    for impl in _impls(ctx, cfg):
        got, ref, n_diff, work = _run_chain(ctx, cfg, impl)
        assert (got["tokens"] == got["tokens"][..., :1]).all()      # every path decodes the same token
        assert (got["counts"] == cfg.K).all()


def test_batched_equals_singles_and_chain_equals_path_tree(ctx):
    cfg = wl.Config("bs", d=256, V=3000, dtype=wl.BF16, B=3, T=4, K=8, p=0.2)
    work = wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=cfg.rows)
    for impl in _impls(ctx, cfg):
        ctx.set_impl(impl)
        full = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=10))
        for b in range(cfg.B):
            one = to_np(ctx.verify_batched(work.H[b:b + 1].contiguous(), work.draft[b:b + 1].contiguous(),
                                           cfg.K, cfg.p, SEED, seq_base=10 + b))
            for key in ("tokens", "counts", "hits", "accept_len"):
                assert np.array_equal(one[key][0], full[key][b]), key
        single = to_np(ctx.verify(work.H[0].contiguous(), work.draft[0].contiguous(), cfg.K, cfg.p, SEED))
        ref0 = to_np(ctx.verify_batched(work.H[:1].contiguous(), work.draft[:1].contiguous(), cfg.K, cfg.p, SEED))
        assert np.array_equal(single["tokens"], ref0["tokens"][0])
        assert single["accept_len"][0] == ref0["accept_len"][0]
        parent = torch.arange(-1, cfg.T - 1, dtype=torch.int32, device=DEV).repeat(cfg.B, 1).contiguous()
        hrow = torch.arange(cfg.T, dtype=torch.int32, device=DEV).repeat(cfg.B, 1).contiguous()
        tree = to_np(ctx.verify_tree(work.H, work.draft, parent, hrow, cfg.K, cfg.p, SEED, seq_base=10))
        assert np.array_equal(tree["tokens"], full["tokens"])
        assert np.array_equal(tree["accept_len"], full["accept_len"])
        assert np.array_equal(tree["best_node"], full["accept_len"] - 1)
        ctx.set_impl(binding.IMPL_AUTO)
    assert ctx.device_error() == 0


@pytest.mark.parametrize("rule", [oracle.RULE_NAIVE, oracle.RULE_MAJORITY])
def test_tree_against_oracle(ctx, rule):
    cfg = wl.Config("tree_s", d=256, V=4000, dtype=wl.BF16, B=3, T=0, K=8, p=0.15, kind="tree", N=25)
    work = wl.make_workload(cfg, device=DEV)
    cfg = work.cfg
    ctx.set_head(work.W, max_rows=cfg.rows)
    Wn, Hn = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H)
    nt, npar, nh = (x.cpu().numpy() for x in (work.node_token, work.node_parent, work.node_hrow))
    ref = oracle.verify_tree(Wn, cfg.dtype, Hn, nt, npar, nh, cfg.K, cfg.p, SEED, seq_base=2, rule=rule)
    assert ref["accept_len"].max() >= 1          # the workload exercises accepted paths
    for impl in _impls(ctx, cfg):
        ctx.set_impl(impl)
        got = to_np(ctx.verify_tree(work.H, work.node_token, work.node_parent, work.node_hrow, cfg.K, cfg.p,
                                    SEED, seq_base=2, rule=rule))
        ctx.set_impl(binding.IMPL_AUTO)
        assert ctx.device_error() == 0
        check_tree(got, ref, nt, npar, nh, rule)


HOST_CASES = [
    wl.Config("host", d=256, V=3000, dtype=wl.BF16, B=2, T=5, K=8, p=0.1),      # mask pass reads the pinned H in place
    wl.Config("host_24", d=256, V=3000, dtype=wl.BF16, B=1, T=3, K=8, p=0.1),   # in-kernel masks: copy kernel first
    wl.Config("host_f32", d=96, V=1500, dtype=wl.F32, B=2, T=3, K=4, p=0.2),    # CUDA-core head, one finalize block per sequence
    wl.Config("host_600", d=128, V=2000, dtype=wl.BF16, B=1, T=75, K=8, p=0.1), # several launches, one finalize block
    wl.Config("host_3x200", d=128, V=2000, dtype=wl.BF16, B=3, T=25, K=8, p=0.1),   # ... and three: the host waits for the stream
]


@pytest.mark.parametrize("cfg", HOST_CASES, ids=lambda c: c.name)
def test_host_entry_point_equals_device_entry_point(ctx, cfg):
    work = wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=cfg.rows, max_hidden_rows=cfg.B * cfg.T)
    dev = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=1))
    Hh, dh = work.H.cpu().pin_memory(), work.draft.cpu().pin_memory()
    for _ in range(2):        # pinned inputs and outputs: the device reads and writes them in place
        host = ctx.verify_batched_host(Hh, dh, cfg.K, cfg.p, SEED, seq_base=1)
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(host[key].numpy(), dev[key]), key
    Hp, dp = work.H.cpu().clone(), work.draft.cpu().clone()      # pageable inputs and outputs: staged by the library
    for _ in range(2):
        out = ctx.alloc_host_outputs(cfg.B, cfg.T, cfg.K, pin=False)
        host = ctx.verify_batched_host(Hp, dp, cfg.K, cfg.p, SEED, seq_base=1, out=out)
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(host[key].numpy(), dev[key]), key
    mixed = ctx.alloc_host_outputs(cfg.B, cfg.T, cfg.K, pin=False)   # pinned inputs, pageable outputs
    host = ctx.verify_batched_host(Hh, dh, cfg.K, cfg.p, SEED, seq_base=1, out=mixed)
    for key in ("tokens", "counts", "hits", "accept_len"):
        assert np.array_equal(host[key].numpy(), dev[key]), key
    with pytest.raises(pk.DropMatchError) as e:
        big = torch.zeros((cfg.B + 1, cfg.T, cfg.d), dtype=work.H.dtype)
        ctx.verify_batched_host(big, torch.zeros((cfg.B + 1, cfg.T), dtype=torch.int32), cfg.K, cfg.p, SEED)
    assert e.value.status == binding.EWORKSPACE


def test_run_to_run_determinism(ctx):
    cfg = wl.Config("det", d=512, V=5000, dtype=wl.BF16, B=2, T=4, K=8, p=0.1)
    work = wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=cfg.rows)
    first = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
    for _ in range(20):
        again = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))
        for key in first:
            assert np.array_equal(first[key], again[key])


def test_argument_errors(ctx):
    cfg = wl.Config("err", d=256, V=1000, dtype=wl.BF16, B=1, T=2, K=4, p=0.1)
    work = wl.make_workload(cfg, device=DEV)
    fresh = pk.Context(0)
    with pytest.raises(pk.DropMatchError) as e:
        fresh.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED)
    assert e.value.status == binding.ENOHEAD
    fresh.close()
    ctx.set_head(work.W, max_rows=cfg.rows)
    for kw, status in ((dict(K=0), binding.EINVAL), (dict(K=2000), binding.EINVAL), (dict(p=1.0), binding.EINVAL),
                       (dict(p=-0.1), binding.EINVAL), (dict(p=float("nan")), binding.EINVAL),
                       (dict(rule=5), binding.EINVAL), (dict(K=16), binding.EWORKSPACE)):
        args = dict(K=cfg.K, p=cfg.p, rule=0)
        args.update(kw)
        with pytest.raises(pk.DropMatchError) as e:
            ctx.verify_batched(work.H, work.draft, args["K"], args["p"], SEED, rule=args["rule"])
        assert e.value.status == status, kw
    L = binding.lib()
    assert L.dm_set_head(ctx._h, work.W.data_ptr(), 1000, 252, binding.BF16, 8, 8) == binding.EUNSUPPORTED
    assert L.dm_set_head(ctx._h, work.W.data_ptr() + 2, 1000, 256, binding.BF16, 8, 8) == binding.EINVAL
    # refused dm_set_head calls leave the previous head in place
    assert ctx.workspace_bytes() > 0
    # the context still works after the refused calls
    ok = ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED)
    assert int(ok["accept_len"][0]) <= cfg.T


def test_shared_mask_mode(ctx):
    """DM_MASK_PER_PATH: masks, tokens, counts and accepted lengths against the oracle's shared-mask
    reading; the masks of every position equal those of position 0."""
    cfg = wl.Config("shared", d=256, V=3000, dtype=wl.BF16, B=2, T=4, K=8, p=0.3)
    work = wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=cfg.rows)
    ctx.set_mask_mode(binding.MASK_PER_PATH)
    try:
        bits = ctx.debug_masks(cfg.B, cfg.T, cfg.K, cfg.d, cfg.p, SEED, seq_base=2).cpu().numpy().view(np.uint32)
        ref_bits = oracle.masks(cfg.B, 1, cfg.K, cfg.d, cfg.p, SEED, 2)          # position 0 of each sequence
        for t in range(cfg.T):
            assert np.array_equal(bits[:, t], ref_bits[:, 0])
        ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                                    work.draft.cpu().numpy(), cfg.K, cfg.p, SEED, seq_base=2, shared_masks=True)
        for impl in _impls(ctx, cfg):
            ctx.set_impl(impl)
            got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=2))
            ctx.set_impl(binding.IMPL_AUTO)
            assert ctx.device_error() == 0
            check_chain(got, ref, work.draft.cpu().numpy())
    finally:
        ctx.set_mask_mode(binding.MASK_PER_POSITION)
    with pytest.raises(pk.DropMatchError):
        ctx.set_mask_mode(7)


EDGE = [
    # one position whose 300 paths straddle two launches of the tensor-core kernel
    wl.Config("edge_k300", d=128, V=2000, dtype=wl.BF16, B=1, T=1, K=300, p=0.2),
    # almost everything dropped: many all-zero masked rows, all-zero logits, ties resolved to token 0
    wl.Config("edge_p_high", d=64, V=300, dtype=wl.BF16, B=2, T=3, K=16, p=0.97),
    # a one-word vocabulary and a two-word one
    wl.Config("edge_v1", d=64, V=1, dtype=wl.BF16, B=1, T=2, K=4, p=0.1, draft_mode="toy"),
    wl.Config("edge_v2", d=128, V=2, dtype=wl.BF16, B=1, T=3, K=8, p=0.5, draft_mode="toy"),
    # widest single launch exactly (256 paths) and one more (257)
    wl.Config("edge_rows256", d=64, V=40000, dtype=wl.BF16, B=1, T=8, K=32, p=0.1),
    wl.Config("edge_rows257", d=64, V=1000, dtype=wl.BF16, B=1, T=1, K=257, p=0.1),
    # a vocabulary so large that a slice has 16 tiles even at 24 paths (staged operand, many groups)
    wl.Config("edge_big_v", d=64, V=300000, dtype=wl.BF16, B=1, T=3, K=8, p=0.1),
    # 1, 8 and 24 paths on a head whose slices have several tiles: CTA pairs padded to 64 accumulator
    # columns, with a staging buffer sized for nothing wider
    wl.Config("edge_pad_r1", d=128, V=60000, dtype=wl.BF16, B=1, T=1, K=1, p=0.2),
    wl.Config("edge_pad_r8", d=128, V=60000, dtype=wl.BF16, B=1, T=1, K=8, p=0.2),
    wl.Config("edge_pad_r24", d=192, V=50000, dtype=wl.BF16, B=1, T=3, K=8, p=0.1),
    # a long hidden size (256 blocks of 64) on a small vocabulary
    wl.Config("edge_long_d", d=16384, V=700, dtype=wl.BF16, B=1, T=2, K=8, p=0.1),
    # fp32 head whose hidden size is the minimum the CUDA-core kernel takes
    wl.Config("edge_f32_d4", d=4, V=50, dtype=wl.F32, B=1, T=2, K=16, p=0.5, draft_mode="toy"),
]


@pytest.mark.parametrize("cfg", EDGE, ids=lambda c: c.name)
def test_edge_shapes(ctx, cfg):
    if cfg.V < 5:   # the workload recipe draws drafts from a top-5: build the few inputs by hand
        W = wl.make_head(cfg.V, cfg.d, cfg.dtype, seed=1, device=DEV)
        H = wl.make_hidden(cfg.B * cfg.T, cfg.d, cfg.dtype, seed=2, device=DEV).view(cfg.B, cfg.T, cfg.d)
        draft = torch.zeros((cfg.B, cfg.T), dtype=torch.int32, device=DEV)
        work = wl.Workload(cfg, W, H, draft, None, None, None)
    else:
        work = wl.make_workload(cfg, device=DEV)
    for impl in _impls(ctx, cfg):
        got, ref, n_diff, _ = _run_chain(ctx, cfg, impl, work=work)
        assert n_diff <= max(2, cfg.rows // 10)
    if cfg.name == "edge_p_high":
        zero_rows = (oracle.masks(cfg.B, cfg.T, cfg.K, cfg.d, cfg.p, SEED, 0) == 0).all(axis=-1)
        assert zero_rows.any()                                   # some paths really dropped everything ...
        assert (ref["tokens"][zero_rows] == 0).all()             # ... and decode to token 0 on both sides
        assert (got["tokens"][zero_rows] == 0).all()


@pytest.mark.parametrize("bonus", [0, 1])
@pytest.mark.parametrize("cfg", [
    wl.Config("next_bf16", d=256, V=3000, dtype=wl.BF16, B=3, T=4, K=8, p=0.2),          # one launch, finished in-kernel
    wl.Config("next_bf16_wide", d=128, V=60000, dtype=wl.BF16, B=2, T=5, K=31, p=0.1),   # staged, several launches
    wl.Config("next_f32", d=100, V=517, dtype=wl.F32, B=2, T=3, K=7, p=0.2, draft_mode="toy"),
], ids=lambda c: c.name)
def test_next_token_call(ctx, cfg, bonus):
    T_h = cfg.T + bonus
    work = wl.make_workload(cfg.with_(T=T_h), device=DEV)              # T_h hidden rows; drafts for the first T
    draft = work.draft[:, :cfg.T].contiguous()
    ctx.set_head(work.W, max_rows=cfg.B * T_h * (cfg.K + 1))
    ref = oracle.verify_batched_next(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H),
                                     draft.cpu().numpy(), cfg.K, cfg.p, SEED, seq_base=4)
    for impl in _impls(ctx, cfg):
        ctx.set_impl(impl)
        got = to_np(ctx.verify_batched_next(work.H, draft, cfg.K, cfg.p, SEED, seq_base=4))
        ctx.set_impl(binding.IMPL_AUTO)
        assert ctx.device_error() == 0
        bad = (got["tokens"] != ref["tokens"]) & (ref["gap"] >= NEAR_TIE)
        assert not bad.any()
        bad_plain = (got["plain"] != ref["plain"]) & (ref["plain_gap"] >= NEAR_TIE)
        assert not bad_plain.any()
        d_np = draft.cpu().numpy()
        for b in range(cfg.B):                                          # integer stages from the GPU's own tokens
            n = oracle.accept_chain(got["tokens"][b, :cfg.T], d_np[b], oracle.RULE_NAIVE)
            assert got["accept_len"][b] == n
            assert got["next"][b] == (got["plain"][b, n] if n < T_h else -1)
            for t in range(T_h):
                cnt, hits = oracle.counts(got["tokens"][b, t], int(d_np[b, t]) if t < cfg.T else -1)
                assert np.array_equal(got["counts"][b, t], cnt)
                if t < cfg.T:
                    assert got["hits"][b, t] == hits
        if not (got["tokens"] != ref["tokens"]).any() and not (got["plain"] != ref["plain"]).any():
            for key in ("counts", "hits", "accept_len", "next"):
                assert np.array_equal(got[key], ref[key]), key


def test_side_stream_and_head_swaps(ctx):
    """Calls issued on a non-default stream, and a context that is pointed at one head after another
    (fp32 -> bf16 tensor-core -> bf16 staged -> back), give what a fresh context gives."""
    cfgs = [wl.CONFIGS["toy"],
            wl.Config("swap_a", d=256, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1),
            wl.Config("swap_b", d=128, V=60000, dtype=wl.BF16, B=2, T=6, K=16, p=0.1),
            wl.Config("swap_a", d=256, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1)]
    side = torch.cuda.Stream(device=DEV)
    for cfg in cfgs:
        work = wl.make_workload(cfg, device=DEV)
        torch.cuda.synchronize()
        ctx.set_head(work.W, max_rows=cfg.rows)
        with torch.cuda.stream(side):
            got = ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=1)
            again = ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=1)
        side.synchronize()
        assert ctx.device_error() == 0
        fresh = pk.Context(0)
        fresh.set_head(work.W, max_rows=cfg.rows)
        want = to_np(fresh.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=1))
        fresh.close()
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(got[key].cpu().numpy(), want[key]), (cfg.name, key)
            assert np.array_equal(again[key].cpu().numpy(), want[key]), (cfg.name, key)


@pytest.mark.parametrize("cfg", [
    wl.Config("graph_a", d=256, V=3000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1),            # one launch per call
    wl.Config("graph_b", d=128, V=60000, dtype=wl.BF16, B=2, T=8, K=25, p=0.1),          # 400 paths: staged, two row blocks
], ids=lambda c: c.name)
def test_verify_call_in_a_cuda_graph(ctx, cfg):
    """The device-pointer entry points only enqueue work (no allocation, no synchronisation), so a
    call can be captured into a CUDA graph and replayed; every replay gives the eager result."""
    work = wl.make_workload(cfg, device=DEV)
    ctx.set_head(work.W, max_rows=cfg.rows)
    want = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=6))
    out = ctx.alloc_outputs(cfg.B, cfg.T, cfg.K)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED, seq_base=6, out=out)
    for _ in range(3):
        for t in out.values():
            t.zero_()
        graph.replay()
        torch.cuda.synchronize()
        got = to_np(out)
        for key in ("tokens", "counts", "hits", "accept_len"):
            assert np.array_equal(got[key], want[key]), key
    assert ctx.device_error() == 0


def test_tree_with_plain_tokens(ctx):
    """dropmatch_verify_tree_next: the tree results equal dropmatch_verify_tree's, and the extra
    unmasked path of every hidden row is the oracle's plain greedy token (outside near-ties)."""
    cfg = wl.Config("tree_next", d=256, V=4000, dtype=wl.BF16, B=3, T=0, K=8, p=0.15, kind="tree", N=25)
    work = wl.make_workload(cfg, device=DEV)
    cfg = work.cfg
    ctx.set_head(work.W, max_rows=cfg.B * cfg.T * (cfg.K + 1))
    Wn, Hn = wl.to_numpy_storage(work.W), wl.to_numpy_storage(work.H)
    dummy = np.zeros((cfg.B, cfg.T), dtype=np.int32)
    plain_ref = oracle.verify_batched_next(Wn, cfg.dtype, Hn, dummy, 1, 0.0, SEED)     # only its plain tokens are used
    for impl in _impls(ctx, cfg):
        ctx.set_impl(impl)
        base = to_np(ctx.verify_tree(work.H, work.node_token, work.node_parent, work.node_hrow, cfg.K, cfg.p, SEED,
                                     seq_base=2))
        got = to_np(ctx.verify_tree_next(work.H, work.node_token, work.node_parent, work.node_hrow, cfg.K, cfg.p,
                                         SEED, seq_base=2))
        ctx.set_impl(binding.IMPL_AUTO)
        assert ctx.device_error() == 0
        for key in ("tokens", "counts", "node_ok", "best_node", "accept_len"):
            assert np.array_equal(got[key], base[key]), key
        bad = (got["plain"] != plain_ref["plain"]) & (plain_ref["plain_gap"] >= NEAR_TIE)
        assert not bad.any()


def test_head_rewritten_in_stream_order_with_pdl_off(ctx):
    """A caller that refreshes W on the stream right before it verifies (a weight reload, a
    dequantisation into the head buffer) switches programmatic stream serialization off: the
    verify kernel then starts only after the write has completed.  Refereed by the oracle on the
    new head."""
    cfg = wl.Config("reload", d=512, V=30000, dtype=wl.BF16, B=2, T=3, K=8, p=0.1)
    work = wl.make_workload(cfg, device=DEV)
    W_new = wl.make_head(cfg.V, cfg.d, cfg.dtype, seed=77, device=DEV)
    W_buf = work.W.clone()
    ctx.set_head(W_buf, max_rows=cfg.rows)
    ctx.set_pdl(False)
    try:
        ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED)       # a call on the old head is in flight
        W_buf.copy_(W_new)                                               # ... the head is rewritten on the same stream
        got = to_np(ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, SEED))   # ... and used right behind it
        assert ctx.device_error() == 0
    finally:
        ctx.set_pdl(True)
    draft = work.draft.cpu().numpy()
    ref = oracle.verify_batched(wl.to_numpy_storage(W_new), cfg.dtype, wl.to_numpy_storage(work.H), draft, cfg.K,
                                cfg.p, SEED)
    check_chain(got, ref, draft)
