"""Thin ctypes binding of libdropmatch's C ABI (include/dropmatch.h).

Argument marshalling only: torch tensors give device pointers and the current stream; every
step of the verification path runs inside the library's CUDA kernels.  There is no CPU
fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

OK, EINVAL, EUNSUPPORTED, ECUDA, EWORKSPACE, EDEVICE, ENOHEAD, ESTATICLIMIT = 0, -1, -2, -3, -4, -5, -6, -7
STATIC_MAX_ROWS = 256
F32, BF16 = 0, 1
RULE_NAIVE, RULE_MAJORITY = 0, 1
IMPL_AUTO, IMPL_SIMT, IMPL_TCGEN05 = 0, 1, 2
MASK_PER_POSITION, MASK_PER_PATH = 0, 1

_LIB_PATH = Path(__file__).resolve().parent / "libdropmatch.so"
_lib = None

_vp, _ci, _cf, _u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint64

# name -> (restype, argtypes); mirrors include/dropmatch.h declaration by declaration
SIGNATURES = {
    "dm_create": (_ci, [ctypes.POINTER(_vp), _ci]),
    "dm_destroy": (_ci, [_vp]),
    "dm_set_head": (_ci, [_vp, _vp, _ci, _ci, _ci, _ci, _ci]),
    "dm_set_impl": (_ci, [_vp, _ci]),
    "dm_set_pdl": (_ci, [_vp, _ci]),
    "dm_set_mask_mode": (_ci, [_vp, _ci]),
    "dm_set_vocab_offset": (_ci, [_vp, _ci]),
    "dropmatch_partial_best": (_ci, [_vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _vp, _vp]),
    "dropmatch_finalize_packed": (_ci, [_vp, _vp, _ci, _vp, _ci, _ci, _ci, _ci, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify": (_ci, [_vp, _vp, _vp, _ci, _ci, _cf, _u64, _ci, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_batched": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _ci, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_batched_sampled": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _ci, _cf, _cf,
                                               _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_batched_next": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _ci, _cf, _u64, _u64, _ci,
                                            _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_batched_host": (_ci, [_vp, _vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _ci, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_batched_static": (_ci, [_ci, _vp, _ci, _ci, _ci, _vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _ci,
                                              _vp, _vp, _vp, _vp, _vp]),
    "dm_enable_js": (_ci, [_vp, _ci, _ci]),
    "dropmatch_verify_js": (_ci, [_vp, _vp, _vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_tree": (_ci, [_vp, _vp, _vp, _vp, _vp, _ci, _ci, _ci, _ci, _cf, _u64, _u64, _ci,
                                    _vp, _vp, _vp, _vp, _vp, _vp]),
    "dropmatch_verify_tree_next": (_ci, [_vp, _vp, _vp, _vp, _vp, _ci, _ci, _ci, _ci, _cf, _u64, _u64, _ci,
                                         _vp, _vp, _vp, _vp, _vp, _vp, _vp]),
    "dm_debug_logits": (_ci, [_vp, _vp, _ci, _ci, _vp, _ci, _cf, _u64, _u64, _vp, _vp]),
    "dm_debug_masks": (_ci, [_vp, _ci, _ci, _ci, _ci, _cf, _u64, _u64, _vp, _vp]),
    "dm_debug_masked_operand": (_ci, [_vp, _vp, _ci, _ci, _ci, _cf, _u64, _u64, _vp, _vp]),
    "dm_debug_read_stream": (_ci, [_vp, _vp, ctypes.c_size_t, _vp]),
    "dm_device_error": (_ci, [_vp, _vp, ctypes.POINTER(ctypes.c_uint32)]),
    "dm_debug_set_wait_limit": (_ci, [_vp, _u64]),
    "dm_profile_head": (_ci, [_vp, _ci]),
    "dm_profile_read": (_ci, [_vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(_ci)]),
    "dm_workspace_bytes": (ctypes.c_size_t, [_vp]),
    "dm_last_impl": (_ci, [_vp]),
    "dm_last_launches": (_ci, [_vp]),
    "dm_strerror": (ctypes.c_char_p, [_ci]),
}


class DropMatchError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {strerror(status)} (status {status})")


def lib() -> ctypes.CDLL:
    """Load libdropmatch.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise ImportError(f"{_LIB_PATH} is missing: run `python -c 'import __graft_entry__ as g; g.build()'`")
        L = ctypes.CDLL(str(_LIB_PATH))
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().dm_strerror(status).decode()


def _check(status: int, where: str):
    if status != OK:
        raise DropMatchError(status, where)


def _ptr(t):
    # the address as a plain int: ctypes converts it for pointer parameters, and building a
    # c_void_p object per argument would cost more than the rest of the marshalling together
    return None if t is None else t.data_ptr()


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream(device) -> int:
    # the handle of torch's current stream on `device` (the short way where this torch has it)
    if _raw_stream is not None:
        index = device if isinstance(device, int) else torch.device(device).index
        if index is not None:
            return _raw_stream(index)
    return torch.cuda.current_stream(device).cuda_stream


def _dev(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{what} must be a contiguous CUDA tensor of {dtype}")
    return t


def verify_batched_static(W, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE, out=None):
    """dropmatch_verify_batched_static: chain verification without a context and without any
    device allocation inside the library (the output tensors are the caller's; pass `out` to
    reuse them).  B*T*K may not exceed STATIC_MAX_ROWS."""
    if W.dtype not in (torch.float32, torch.bfloat16) or not W.is_cuda or not W.is_contiguous() or W.dim() != 2:
        raise TypeError("W must be a contiguous 2-D CUDA tensor of float32 or bfloat16")
    dtype = F32 if W.dtype == torch.float32 else BF16
    _dev(H, W.dtype, "H"); _dev(draft, torch.int32, "draft")
    B, T, _ = H.shape
    V, d = W.shape
    if out is None:
        i32 = dict(dtype=torch.int32, device=W.device)
        out = dict(tokens=torch.empty((B, T, K), **i32), counts=torch.empty((B, T, K), **i32),
                   hits=torch.empty((B, T), **i32), accept_len=torch.empty((B,), **i32))
    _check(lib().dropmatch_verify_batched_static(W.device.index, _ptr(W), V, d, dtype, _ptr(H), _ptr(draft), B, T, K,
                                                 p, seed, seq_base, rule, _ptr(out["tokens"]), _ptr(out["counts"]),
                                                 _ptr(out["hits"]), _ptr(out["accept_len"]), _stream(W.device)),
           "dropmatch_verify_batched_static")
    return out


class Context:
    """One dm_ctx: a device, an LM head, and the library-owned workspace."""

    def __init__(self, device: int = 0):
        self._h = ctypes.c_void_p()
        self.device = torch.device("cuda", device)
        _check(lib().dm_create(ctypes.byref(self._h), device), "dm_create")
        self._W = None
        self.dtype = None

    def close(self):
        if self._h:
            lib().dm_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _tdtype(self):
        return torch.float32 if self.dtype == F32 else torch.bfloat16

    # -- dm_set_head / dm_set_impl
    def set_head(self, W: torch.Tensor, max_rows: int, max_hidden_rows: int | None = None):
        """W must be complete before a verify call is enqueued and must not be written by work that
        is still in flight on the stream (see set_pdl)."""
        if W.dtype not in (torch.float32, torch.bfloat16) or not W.is_cuda or not W.is_contiguous() or W.dim() != 2:
            raise TypeError("W must be a contiguous 2-D CUDA tensor of float32 or bfloat16")
        dtype = F32 if W.dtype == torch.float32 else BF16
        V, d = W.shape
        _check(lib().dm_set_head(self._h, _ptr(W), V, d, dtype, max_rows, max_hidden_rows or max_rows), "dm_set_head")
        self._W, self.dtype, self.V, self.d = W, dtype, V, d   # keep W alive

    def set_impl(self, impl: int):
        _check(lib().dm_set_impl(self._h, impl), "dm_set_impl")

    def set_pdl(self, enable: bool):
        """Off: verify kernels never start before earlier work of the stream has completed (needed when
        that work writes W; by default the kernel streams W while the kernel ahead is still finishing)."""
        _check(lib().dm_set_pdl(self._h, int(enable)), "dm_set_pdl")

    def set_mask_mode(self, mode: int):
        _check(lib().dm_set_mask_mode(self._h, mode), "dm_set_mask_mode")

    # -- vocabulary-sharded heads
    def set_vocab_offset(self, offset: int):
        _check(lib().dm_set_vocab_offset(self._h, offset), "dm_set_vocab_offset")

    def partial_best(self, H, K, p, seed, seq_base=0):
        """-> int64 tensor [B*T*K] holding the packed (key, inverted token id) words bit for bit."""
        B, T, _ = H.shape
        _dev(H, self._tdtype(), "H")
        out = torch.empty((B * T * K,), dtype=torch.int64, device=self.device)
        _check(lib().dropmatch_partial_best(self._h, _ptr(H), B, T, K, p, seed, seq_base, _ptr(out),
                                            _stream(self.device)), "dropmatch_partial_best")
        return out

    def finalize_packed(self, packed, draft, K, rule=RULE_NAIVE):
        """packed: int64 [n_parts, B*T*K] (or [B*T*K]); draft[B,T] -> the outputs of verify_batched."""
        _dev(draft, torch.int32, "draft")
        B, T = draft.shape
        if packed.dim() == 1:
            packed = packed.unsqueeze(0)
        _dev(packed, torch.int64, "packed")
        if packed.shape[1] != B * T * K:
            raise TypeError("packed must have B*T*K words per part")
        out = self.alloc_outputs(B, T, K)
        _check(lib().dropmatch_finalize_packed(self._h, _ptr(packed), packed.shape[0], _ptr(draft), B, T, K, rule,
                                               _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["hits"]),
                                               _ptr(out["accept_len"]), _stream(self.device)),
               "dropmatch_finalize_packed")
        return out

    # -- dropmatch_verify
    def verify(self, H, draft, K, p, seed, rule=RULE_NAIVE):
        T = H.shape[0]
        _dev(H, self._tdtype(), "H"); _dev(draft, torch.int32, "draft")
        tokens = torch.empty((T, K), dtype=torch.int32, device=self.device)
        counts = torch.empty_like(tokens)
        alen = torch.empty((1,), dtype=torch.int32, device=self.device)
        _check(lib().dropmatch_verify(self._h, _ptr(H), _ptr(draft), T, K, p, seed, rule, _ptr(tokens),
                                      _ptr(counts), _ptr(alen), _stream(self.device)), "dropmatch_verify")
        return dict(tokens=tokens, counts=counts, accept_len=alen)

    # -- dropmatch_verify_batched
    def verify_batched(self, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE, out=None):
        B, T, _ = H.shape
        _dev(H, self._tdtype(), "H"); _dev(draft, torch.int32, "draft")
        if out is None:
            out = self.alloc_outputs(B, T, K)
        _check(lib().dropmatch_verify_batched(self._h, _ptr(H), _ptr(draft), B, T, K, p, seed, seq_base, rule,
                                              _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["hits"]),
                                              _ptr(out["accept_len"]), _stream(self.device)),
               "dropmatch_verify_batched")
        return out

    # -- dropmatch_verify_batched_sampled
    def verify_batched_sampled(self, H, draft, K, p, seed, temperature=1.0, top_p=1.0, seq_base=0, rule=RULE_NAIVE,
                               out=None):
        B, T, _ = H.shape
        _dev(H, self._tdtype(), "H"); _dev(draft, torch.int32, "draft")
        if out is None:
            out = self.alloc_outputs(B, T, K)
        _check(lib().dropmatch_verify_batched_sampled(self._h, _ptr(H), _ptr(draft), B, T, K, p, seed, seq_base, rule,
                                                      temperature, top_p, _ptr(out["tokens"]), _ptr(out["counts"]),
                                                      _ptr(out["hits"]), _ptr(out["accept_len"]),
                                                      _stream(self.device)), "dropmatch_verify_batched_sampled")
        return out

    # -- dropmatch_verify_batched_next
    def verify_batched_next(self, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE):
        """H[B,T_h,d] with T_h = T or T+1 (bonus row), draft[B,T].  Adds plain[B,T_h], next[B]."""
        B, T_h, _ = H.shape
        T = draft.shape[1]
        if T_h - T not in (0, 1):
            raise TypeError("H must have T or T+1 hidden rows per sequence")
        _dev(H, self._tdtype(), "H"); _dev(draft, torch.int32, "draft")
        i32 = dict(dtype=torch.int32, device=self.device)
        out = dict(tokens=torch.empty((B, T_h, K), **i32), counts=torch.empty((B, T_h, K), **i32),
                   hits=torch.empty((B, T), **i32), accept_len=torch.empty((B,), **i32),
                   plain=torch.empty((B, T_h), **i32), next=torch.empty((B,), **i32))
        _check(lib().dropmatch_verify_batched_next(self._h, _ptr(H), _ptr(draft), B, T, T_h - T, K, p, seed, seq_base,
                                                   rule, _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["hits"]),
                                                   _ptr(out["accept_len"]), _ptr(out["plain"]), _ptr(out["next"]),
                                                   _stream(self.device)), "dropmatch_verify_batched_next")
        return out

    def alloc_outputs(self, B, T, K):
        i32 = dict(dtype=torch.int32, device=self.device)
        return dict(tokens=torch.empty((B, T, K), **i32), counts=torch.empty((B, T, K), **i32),
                    hits=torch.empty((B, T), **i32), accept_len=torch.empty((B,), **i32))

    # -- dropmatch_verify_batched_host
    def verify_batched_host(self, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE, out=None):
        """H, draft and outputs are CPU tensors (pinned for speed); returns after the results are on the host."""
        B, T, _ = H.shape
        if H.is_cuda or draft.is_cuda or not H.is_contiguous() or not draft.is_contiguous():
            raise TypeError("host entry point takes contiguous CPU tensors")
        if H.dtype != self._tdtype() or draft.dtype != torch.int32:
            raise TypeError("H must have the head's dtype and draft must be int32")
        if out is None:
            out = self.alloc_host_outputs(B, T, K)
        _check(lib().dropmatch_verify_batched_host(self._h, _ptr(H), _ptr(draft), B, T, K, p, seed, seq_base, rule,
                                                   _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["hits"]),
                                                   _ptr(out["accept_len"]), _stream(self.device)),
               "dropmatch_verify_batched_host")
        return out

    @staticmethod
    def alloc_host_outputs(B, T, K, pin=True):
        mk = lambda *s: torch.empty(s, dtype=torch.int32, pin_memory=pin)
        return dict(tokens=mk(B, T, K), counts=mk(B, T, K), hits=mk(B, T), accept_len=mk(B))

    # -- dm_enable_js / dropmatch_verify_js
    def enable_js(self, max_rows: int, max_hidden_rows: int):
        _check(lib().dm_enable_js(self._h, max_rows, max_hidden_rows), "dm_enable_js")

    def verify_js(self, H, draft, draft_prob, K, p, seed, seq_base=0):
        """Algorithm 1 (JS test, else majority).  draft_prob[B,T,V] float32 on the device."""
        B, T, _ = H.shape
        _dev(H, self._tdtype(), "H"); _dev(draft, torch.int32, "draft"); _dev(draft_prob, torch.float32, "draft_prob")
        if tuple(draft_prob.shape) != (B, T, self.V):
            raise TypeError("draft_prob must have shape [B, T, V]")
        i32 = dict(dtype=torch.int32, device=self.device)
        out = dict(tokens=torch.empty((B, T, K), **i32), counts=torch.empty((B, T, K), **i32),
                   js=torch.empty((B, T, K + 1), dtype=torch.float32, device=self.device),
                   js_ok=torch.empty((B, T), **i32), accept_len=torch.empty((B,), **i32))
        _check(lib().dropmatch_verify_js(self._h, _ptr(H), _ptr(draft), _ptr(draft_prob), B, T, K, p, seed, seq_base,
                                         _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["js"]), _ptr(out["js_ok"]),
                                         _ptr(out["accept_len"]), _stream(self.device)), "dropmatch_verify_js")
        return out

    # -- dropmatch_verify_tree
    def verify_tree(self, H, node_token, node_parent, node_hrow, K, p, seed, seq_base=0, rule=RULE_NAIVE):
        B, N_h, _ = H.shape
        N = node_token.shape[1]
        _dev(H, self._tdtype(), "H")
        for name, t in (("node_token", node_token), ("node_parent", node_parent), ("node_hrow", node_hrow)):
            _dev(t, torch.int32, name)
        i32 = dict(dtype=torch.int32, device=self.device)
        out = dict(tokens=torch.empty((B, N_h, K), **i32), counts=torch.empty((B, N_h, K), **i32),
                   node_ok=torch.empty((B, N), **i32), best_node=torch.empty((B,), **i32),
                   accept_len=torch.empty((B,), **i32))
        _check(lib().dropmatch_verify_tree(self._h, _ptr(H), _ptr(node_token), _ptr(node_parent), _ptr(node_hrow),
                                           B, N_h, N, K, p, seed, seq_base, rule, _ptr(out["tokens"]),
                                           _ptr(out["counts"]), _ptr(out["node_ok"]), _ptr(out["best_node"]),
                                           _ptr(out["accept_len"]), _stream(self.device)), "dropmatch_verify_tree")
        return out

    def verify_tree_next(self, H, node_token, node_parent, node_hrow, K, p, seed, seq_base=0, rule=RULE_NAIVE):
        """verify_tree plus plain[B,N_h]: the undropped greedy token of every hidden row."""
        B, N_h, _ = H.shape
        N = node_token.shape[1]
        _dev(H, self._tdtype(), "H")
        for name, t in (("node_token", node_token), ("node_parent", node_parent), ("node_hrow", node_hrow)):
            _dev(t, torch.int32, name)
        i32 = dict(dtype=torch.int32, device=self.device)
        out = dict(tokens=torch.empty((B, N_h, K), **i32), counts=torch.empty((B, N_h, K), **i32),
                   node_ok=torch.empty((B, N), **i32), best_node=torch.empty((B,), **i32),
                   accept_len=torch.empty((B,), **i32), plain=torch.empty((B, N_h), **i32))
        _check(lib().dropmatch_verify_tree_next(self._h, _ptr(H), _ptr(node_token), _ptr(node_parent),
                                                _ptr(node_hrow), B, N_h, N, K, p, seed, seq_base, rule,
                                                _ptr(out["tokens"]), _ptr(out["counts"]), _ptr(out["node_ok"]),
                                                _ptr(out["best_node"]), _ptr(out["accept_len"]), _ptr(out["plain"]),
                                                _stream(self.device)), "dropmatch_verify_tree_next")
        return out

    # -- debug
    def debug_logits(self, H, row_sel, p, seed, seq_base=0):
        B, T, _ = H.shape
        _dev(H, self._tdtype(), "H"); _dev(row_sel, torch.int32, "row_sel")
        n = row_sel.shape[0]
        out = torch.empty((n, self.V), dtype=torch.float32, device=self.device)
        _check(lib().dm_debug_logits(self._h, _ptr(H), B, T, _ptr(row_sel), n, p, seed, seq_base, _ptr(out),
                                     _stream(self.device)), "dm_debug_logits")
        return out

    def debug_masks(self, B, T, K, d, p, seed, seq_base=0):
        out = torch.empty((B, T, K, (d + 31) // 32), dtype=torch.int32, device=self.device)
        _check(lib().dm_debug_masks(self._h, B, T, K, d, p, seed, seq_base, _ptr(out), _stream(self.device)),
               "dm_debug_masks")
        return out

    def debug_masked_operand(self, H, K, p, seed, seq_base=0):
        """-> [B*T*K, d] tensor of the head's dtype: every path's hidden row with its dropped elements zeroed."""
        B, T, d = H.shape
        _dev(H, self._tdtype(), "H")
        out = torch.empty((B * T * K, d), dtype=H.dtype, device=self.device)
        _check(lib().dm_debug_masked_operand(self._h, _ptr(H), B, T, K, p, seed, seq_base, _ptr(out),
                                             _stream(self.device)), "dm_debug_masked_operand")
        return out

    def debug_read_stream(self, t: torch.Tensor):
        """One read-only pass over a CUDA tensor's bytes (for measuring the read-only HBM rate)."""
        _check(lib().dm_debug_read_stream(self._h, _ptr(t), t.numel() * t.element_size(), _stream(self.device)),
               "dm_debug_read_stream")

    def device_error(self) -> int:
        code = ctypes.c_uint32()
        _check(lib().dm_device_error(self._h, _stream(self.device), ctypes.byref(code)), "dm_device_error")
        return code.value

    def debug_set_wait_limit(self, cycles: int):
        _check(lib().dm_debug_set_wait_limit(self._h, cycles), "dm_debug_set_wait_limit")

    def profile_head(self, enable: bool):
        _check(lib().dm_profile_head(self._h, int(enable)), "dm_profile_head")

    def profile_read(self):
        """-> (summed head-kernel milliseconds, number of calls) since the last read."""
        ms, n = ctypes.c_double(), ctypes.c_int()
        _check(lib().dm_profile_read(self._h, ctypes.byref(ms), ctypes.byref(n)), "dm_profile_read")
        return ms.value, n.value

    def workspace_bytes(self) -> int:
        return lib().dm_workspace_bytes(self._h)

    def last_impl(self) -> int:
        return lib().dm_last_impl(self._h)

    def last_launches(self) -> int:
        return lib().dm_last_launches(self._h)
