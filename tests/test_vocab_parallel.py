"""Vocabulary-parallel verification (each rank holds a slice of the LM head, one all-gather of
packed per-path maxima, then histogram and acceptance on every rank).

CPU part (no GPU): the host plumbing of VocabParallelVerifier under two gloo ranks with a stand-in
context, and the shard arithmetic.  GPU part: shards run one after the other on one GPU, and two
processes that share the GPU (their kernels never wait on each other) and all-gather host copies
over gloo, are both refereed by the CPU oracle on the whole head (tokens outside near-ties, counts,
hits, accepted lengths) and must equal the unsharded CUDA call bit for bit."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2603_03333_b200 import vocab_parallel as vp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(worker_src, world=2, extra_env=None, timeout=300):
    port = _free_port()
    procs = []
    for rank in range(world):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), **(extra_env or {}))
        procs.append(subprocess.Popen([sys.executable, "-c", worker_src.format(root=str(ROOT))], env=env,
                                      stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for pr in procs:
        out, err = pr.communicate(timeout=timeout)
        assert pr.returncode == 0, err[-3000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    return outs


def test_shard_rows_cover_the_vocabulary_once():
    for V, world in ((128256, 4), (151936, 8), (1000, 3), (7, 4), (64, 1)):
        spans = [vp.shard_rows(V, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == V
        for (a0, a1), (b0, b1) in zip(spans, spans[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(b % 8 == 0 for b, _ in spans if b < V)      # shard starts keep W rows 16-byte aligned


FAKE_WORKER = r"""
import json, sys
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
from paper_2603_03333_b200 import vocab_parallel as vp
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()

class FakeCtx:                       # records what the verifier hands to the library
    def set_head(self, W, max_rows): self.rows = W.shape[0]
    def set_vocab_offset(self, off): self.off = off
    def partial_best(self, H, K, p, seed, seq_base):
        return torch.arange(6, dtype=torch.int64) * 10 + rank      # each rank's own words
    def finalize_packed(self, packed, draft, K, rule):
        return packed

ctx = FakeCtx()
b, e = vp.shard_rows(40, world, rank)
v = vp.VocabParallelVerifier(ctx, torch.zeros((e - b, 8)), b, max_rows=6, gather_on_cpu=True)
got = v.verify_batched(torch.zeros((1, 2, 8)), torch.zeros((1, 2), dtype=torch.int32), 3, 0.1, 1)
print(json.dumps(dict(rank=rank, off=ctx.off, rows=ctx.rows, gathered=got.tolist())), flush=True)
dist.destroy_process_group()
"""


def test_two_gloo_ranks_gather_their_words_in_rank_order():
    outs = _spawn(FAKE_WORKER)
    want = [[i * 10 + r for i in range(6)] for r in range(2)]
    for o in outs:
        assert o["gathered"] == want            # [n_parts][rows], rank r's words in row r, on every rank
    assert [o["off"] for o in sorted(outs, key=lambda o: o["rank"])] == [0, 24]
    assert sum(o["rows"] for o in outs) == 40


@pytest.mark.gpu
@pytest.mark.parametrize("cfg_kw", [
    dict(d=256, V=3000, B=2, T=3, K=8, p=0.1),            # small head: one accumulator group
    dict(d=128, V=60000, B=2, T=6, K=16, p=0.1),          # staged operand, CTA pairs on the full head
    dict(d=64, V=300, B=2, T=3, K=16, p=0.97),            # many all-dropped paths: ties across shards -> token 0
])
@pytest.mark.parametrize("world", [2, 3])
def test_shards_run_in_turn_equal_the_whole_head(cfg_kw, world):
    import oracle
    import paper_2603_03333_b200 as pk
    from paper_2603_03333_b200 import binding, workloads as wl
    from parity_util import check_chain, to_np
    cfg = wl.Config("vp", dtype=wl.BF16, **cfg_kw)
    work = wl.make_workload(cfg, device="cuda:0")
    full = pk.Context(0)
    full.set_head(work.W, max_rows=cfg.rows)
    want = full.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED, seq_base=2)
    whole = full.partial_best(work.H, cfg.K, cfg.p, wl.MASK_SEED, seq_base=2)
    parts = []
    for rank in range(world):
        b, e = vp.shard_rows(cfg.V, world, rank)
        if b == e:
            parts.append(torch.zeros_like(whole))
            continue
        ctx = pk.Context(0)
        ctx.set_head(work.W[b:e], max_rows=cfg.rows)
        ctx.set_vocab_offset(b)
        parts.append(ctx.partial_best(work.H, cfg.K, cfg.p, wl.MASK_SEED, seq_base=2))
        assert ctx.device_error() == 0
        if ctx.last_impl() == binding.IMPL_TCGEN05 and cfg.rows <= 256:
            assert ctx.last_launches() <= 2     # the head kernel reduces into the caller's words (+ the mask pass)
        ctx.close()
    gathered = torch.stack(parts)
    # unsigned maximum of the packed words == the unsharded head's words
    merged = gathered.cpu().numpy().view(np.uint64).max(axis=0)
    assert np.array_equal(merged, whole.cpu().numpy().view(np.uint64))
    got = full.finalize_packed(gathered, work.draft, cfg.K)
    for key in ("tokens", "counts", "hits", "accept_len"):
        assert torch.equal(got[key], want[key]), key
    full.close()
    # the referee: the oracle on the whole, unsharded head
    draft = work.draft.cpu().numpy()
    ref = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft, cfg.K,
                                cfg.p, wl.MASK_SEED, seq_base=2)
    check_chain(to_np(got), ref, draft)


GPU_WORKER = r"""
import json, sys
sys.path.insert(0, {root!r})
sys.path.insert(0, {root!r} + "/tests")
import torch, torch.distributed as dist
import oracle
import paper_2603_03333_b200 as pk
from paper_2603_03333_b200 import workloads as wl, vocab_parallel as vp
from parity_util import check_chain, to_np
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
cfg = wl.Config("vp2", d=256, V=5000, dtype=wl.BF16, B=2, T=4, K=8, p=0.2)
work = wl.make_workload(cfg, device="cuda:0")            # same seeds on every rank: same W, H, drafts
b, e = vp.shard_rows(cfg.V, world, rank)
ctx = pk.Context(0)
ver = vp.VocabParallelVerifier(ctx, work.W[b:e].contiguous(), b, max_rows=cfg.rows, gather_on_cpu=True)
got = ver.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED, seq_base=1)
torch.cuda.synchronize()
ref_ctx = pk.Context(0)
ref_ctx.set_head(work.W, max_rows=cfg.rows)
ref = ref_ctx.verify_batched(work.H, work.draft, cfg.K, cfg.p, wl.MASK_SEED, seq_base=1)
same = all(bool(torch.equal(got[k], ref[k])) for k in ("tokens", "counts", "hits", "accept_len"))
draft = work.draft.cpu().numpy()                          # the referee: the oracle on the whole head
want = oracle.verify_batched(wl.to_numpy_storage(work.W), cfg.dtype, wl.to_numpy_storage(work.H), draft, cfg.K,
                             cfg.p, wl.MASK_SEED, seq_base=1)
check_chain(to_np(got), want, draft)
print(json.dumps(dict(rank=rank, same=same, accept=got["accept_len"].tolist())), flush=True)
dist.barrier()                                            # nobody leaves while a peer still gathers
dist.destroy_process_group()
"""


@pytest.mark.gpu
def test_two_processes_on_one_gpu_all_gather_over_gloo():
    outs = _spawn(GPU_WORKER, timeout=600)
    assert all(o["same"] for o in outs)
    assert outs[0]["accept"] == outs[1]["accept"]
