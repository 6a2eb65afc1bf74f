"""Seeded synthetic inputs for the DropMatch verification path.

This module holds no part of the method (no masks, no dropout paths, no
acceptance): it only draws LM-head weights, hidden states, draft tokens and
draft trees with the shapes and value distributions of the benchmark
configurations, so that the CUDA path and the CPU oracle can be fed the very
same tensors.  The one piece of arithmetic here is the plain undropped head
``H @ W^T`` (a library matmul) whose top-k tokens are used to *draw drafts*
that a target model would plausibly accept; it stands in for a draft model.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

F32, BF16 = 0, 1

MASK_SEED = 0xD509A7C4  # Philox key used by tests and the benchmark


@dataclass(frozen=True)
class Config:
    name: str
    d: int
    V: int
    dtype: int          # F32 or BF16 (storage type of W and H)
    B: int
    T: int              # chain length, or hidden rows per sequence for a tree
    K: int
    p: float
    kind: str = "chain"  # "chain" or "tree"
    N: int = 0           # tree nodes per sequence
    draft_mode: str = "top5"  # "toy": top-1 at t<2 then uniform; "top5": 70 % top-1 / 30 % top-5

    @property
    def rows(self) -> int:
        return self.B * self.T * self.K

    def with_(self, **kw) -> "Config":
        return replace(self, **kw)


CONFIGS = {
    # the five benchmark configurations (toy, Llama-3-8B head, Qwen3-8B head, tree, Llama-3-70B head)
    "toy": Config("toy", d=256, V=4096, dtype=F32, B=1, T=4, K=8, p=0.1, draft_mode="toy"),
    "llama8b": Config("llama8b", d=4096, V=128256, dtype=BF16, B=1, T=5, K=8, p=0.1),
    "qwen8b": Config("qwen8b", d=4096, V=151936, dtype=BF16, B=1, T=7, K=8, p=0.1),
    "tree": Config("tree", d=4096, V=128256, dtype=BF16, B=4, T=61, K=8, p=0.1, kind="tree", N=60),
    "llama70b": Config("llama70b", d=8192, V=128256, dtype=BF16, B=16, T=8, K=16, p=0.1),
    # the Llama-3-8B head at the upper end of the HBM-bound range (256 paths: staged operand, CTA pairs)
    "llama8b_k32": Config("llama8b_k32", d=4096, V=128256, dtype=BF16, B=1, T=8, K=32, p=0.1),
    # ... and a tensor-bound call on the same head (512 paths: two row blocks per launch)
    "llama8b_b2k32": Config("llama8b_b2k32", d=4096, V=128256, dtype=BF16, B=2, T=8, K=32, p=0.1),
}


def torch_dtype(dtype: int) -> torch.dtype:
    return torch.float32 if dtype == F32 else torch.bfloat16


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def make_head(V: int, d: int, dtype: int, seed: int = 1, device="cpu") -> torch.Tensor:
    """W[V,d]: fp32 ~ N(0, 1/d) for the toy head, bf16 ~ N(0, 0.02^2) for the LLM-shaped heads."""
    g = _gen(seed, device)
    std = d ** -0.5 if dtype == F32 else 0.02
    W = torch.empty((V, d), dtype=torch_dtype(dtype), device=device)
    step = max(1, (1 << 26) // d)  # draw in fp32 slabs so the fp32 copy never exceeds 256 MB
    for v0 in range(0, V, step):
        v1 = min(V, v0 + step)
        W[v0:v1] = (torch.randn((v1 - v0, d), generator=g, device=device, dtype=torch.float32) * std
                    ).to(W.dtype)
    return W


def make_hidden(n_rows: int, d: int, dtype: int, seed: int = 2, device="cpu") -> torch.Tensor:
    """H[n_rows,d]: toy ~ N(0, 1/d); otherwise N(0,1) with every row rescaled to RMS 1 (what a
    final RMSNorm with unit gain would hand to the LM head), rounded to bf16."""
    g = _gen(seed, device)
    x = torch.randn((n_rows, d), generator=g, device=device, dtype=torch.float32)
    if dtype == F32:
        return x * d ** -0.5
    x = x / x.pow(2).mean(dim=1, keepdim=True).sqrt()
    return x.to(torch.bfloat16)


def undropped_topk(W: torch.Tensor, H: torch.Tensor, k: int) -> torch.Tensor:
    """Top-k token ids of the plain head H @ W^T, fp32 accumulation, as int64 [n_rows,k]."""
    n = H.shape[0]
    V = W.shape[0]
    Hf = H.to(torch.float32)
    best_val = torch.full((n, 0), 0.0, device=H.device)
    best_idx = torch.zeros((n, 0), dtype=torch.int64, device=H.device)
    step = 16384
    for v0 in range(0, V, step):
        v1 = min(V, v0 + step)
        logits = Hf @ W[v0:v1].to(torch.float32).T
        val, idx = logits.topk(min(k, v1 - v0), dim=1)
        best_val = torch.cat([best_val, val], dim=1)
        best_idx = torch.cat([best_idx, idx + v0], dim=1)
        val, sel = best_val.topk(min(k, best_val.shape[1]), dim=1)
        best_val, best_idx = val, best_idx.gather(1, sel)
    return best_idx


def make_chain_draft(topk: torch.Tensor, B: int, T: int, V: int, mode: str, seed: int = 3) -> torch.Tensor:
    """draft[B,T] int32 on CPU.  ``topk`` is undropped_topk(...)[B*T, >=5] (any device)."""
    rng = np.random.default_rng(seed)
    top = topk.cpu().numpy().reshape(B, T, -1)
    draft = np.zeros((B, T), dtype=np.int32)
    for b in range(B):
        for t in range(T):
            if mode == "toy":
                draft[b, t] = top[b, t, 0] if t < 2 else rng.integers(0, V)
            else:
                draft[b, t] = top[b, t, 0] if rng.random() < 0.7 else top[b, t, rng.integers(0, 5)]
    return torch.from_numpy(draft)


def make_draft_probs(W: torch.Tensor, H: torch.Tensor, noise, seed: int = 6) -> torch.Tensor:
    """draft_prob[n_rows,V] float32: a stand-in for the draft model's distribution, the softmax of
    the plain (undropped) head applied to H + noise * N(0,1); ``noise`` is a float or one value per
    row (small: the draft agrees with the target; large: it does not).  Library matmul/softmax."""
    g = _gen(seed, H.device)
    Hf = H.to(torch.float32)
    n = torch.as_tensor(noise, dtype=torch.float32, device=H.device).reshape(-1, 1)
    Hn = Hf + n * torch.randn(Hf.shape, generator=g, device=H.device, dtype=torch.float32)
    out = torch.empty((H.shape[0], W.shape[0]), dtype=torch.float32, device=H.device)
    step = 32
    for r0 in range(0, H.shape[0], step):
        out[r0:r0 + step] = torch.softmax(Hn[r0:r0 + step] @ W.to(torch.float32).T, dim=1)
    return out


def make_tree_shape(B: int, N: int, max_depth: int = 7, max_branch: int = 4, seed: int = 4):
    """Random draft trees in topological order.

    Returns (node_parent[B,N], node_hrow[B,N], n_hidden) as numpy int32 arrays.  parent -1 means
    the node hangs off the committed prefix, whose hidden state is hidden row 0; every node that
    has children owns one further hidden row (numbered in node order), and all children of one
    parent share that row.  ``n_hidden`` is the largest row count over the batch.
    """
    rng = np.random.default_rng(seed)
    parent = np.zeros((B, N), dtype=np.int32)
    hrow = np.zeros((B, N), dtype=np.int32)
    n_hidden = 1
    for b in range(B):
        depth, nchild = [], []
        root_children = 0
        for n in range(N):
            cands = [m for m in range(n) if depth[m] < max_depth and nchild[m] < max_branch]
            if root_children < max_branch and (n == 0 or rng.random() < 0.15 or not cands):
                parent[b, n] = -1
                depth.append(1)
                root_children += 1
            else:
                m = int(cands[rng.integers(0, len(cands))])
                parent[b, n] = m
                depth.append(depth[m] + 1)
                nchild[m] += 1
            nchild.append(0)
        row_of = {-1: 0}
        for n in range(N):
            par = int(parent[b, n])
            if par not in row_of:
                row_of[par] = len(row_of)
            hrow[b, n] = row_of[par]
        n_hidden = max(n_hidden, len(row_of))
    return parent, hrow, n_hidden


def make_tree_tokens(top4: torch.Tensor, parent: np.ndarray, hrow: np.ndarray, n_hidden: int,
                     seed: int = 5) -> np.ndarray:
    """node_token[B,N]: siblings draw distinct tokens from their shared hidden row's undropped
    top-4.  ``top4`` is undropped_topk(...)[B*n_hidden, 4]."""
    rng = np.random.default_rng(seed)
    B, N = parent.shape
    top = top4.cpu().numpy().reshape(B, n_hidden, -1)
    tok = np.zeros((B, N), dtype=np.int32)
    for b in range(B):
        used: dict[int, list[int]] = {}
        for n in range(N):
            r = int(hrow[b, n])
            free = [c for c in range(top.shape[2]) if c not in used.setdefault(r, [])]
            c = free[rng.integers(0, len(free))]
            used[r].append(c)
            tok[b, n] = top[b, r, c]
    return tok


def to_numpy_storage(x: torch.Tensor) -> np.ndarray:
    """CPU numpy view in the layout the oracle reads: float32, or uint16 bit patterns for bf16."""
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.uint16).numpy()
    return x.numpy()


@dataclass
class Workload:
    cfg: Config
    W: torch.Tensor            # [V,d] on `device`
    H: torch.Tensor            # [B,T,d] on `device` (T = hidden rows per sequence)
    draft: torch.Tensor | None        # [B,T] int32 (chain)
    node_token: torch.Tensor | None   # [B,N] int32 (tree)
    node_parent: torch.Tensor | None
    node_hrow: torch.Tensor | None


def make_workload(cfg: Config, device="cpu", W: torch.Tensor | None = None) -> Workload:
    """All inputs of one verify call for ``cfg``; pass ``W`` to reuse a head already built."""
    if W is None:
        W = make_head(cfg.V, cfg.d, cfg.dtype, seed=1, device=device)
    if cfg.kind == "chain":
        H = make_hidden(cfg.B * cfg.T, cfg.d, cfg.dtype, seed=2, device=device)
        top = undropped_topk(W, H, 5)
        draft = make_chain_draft(top, cfg.B, cfg.T, cfg.V, cfg.draft_mode, seed=3).to(device)
        return Workload(cfg, W, H.view(cfg.B, cfg.T, cfg.d), draft, None, None, None)
    parent, hrow, n_hidden = make_tree_shape(cfg.B, cfg.N, seed=4)
    cfg = cfg.with_(T=n_hidden)
    H = make_hidden(cfg.B * n_hidden, cfg.d, cfg.dtype, seed=2, device=device)
    top4 = undropped_topk(W, H, 4)
    tok = make_tree_tokens(top4, parent, hrow, n_hidden, seed=5)
    as_t = lambda a: torch.from_numpy(a).to(device)
    return Workload(cfg, W, H.view(cfg.B, n_hidden, cfg.d), None, as_t(tok), as_t(parent), as_t(hrow))
