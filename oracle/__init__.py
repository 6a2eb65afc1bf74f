"""ctypes access to the DropMatch CPU oracle (TEST INFRASTRUCTURE, not the product).

The arithmetic lives in ``dropmatch_oracle.c`` (plain C, fp64).  This module only
marshals numpy arrays.  Tests, the smoke check and the benchmark's cpu-baseline
leg may import it; the CUDA package never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

F32, BF16 = 0, 1
RULE_NAIVE, RULE_MAJORITY = 0, 1

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "dropmatch_oracle.c"
_LIB = _HERE / "liboracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP over vocabulary rows only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.run(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-Wall", "-Wextra",
             str(_SRC), "-o", str(tmp), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        u32p = ctypes.POINTER(ctypes.c_uint32)
        i32p = ctypes.POINTER(ctypes.c_int32)
        f64p = ctypes.POINTER(ctypes.c_double)
        vp, ci, cf, u64 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint64
        L.oracle_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.oracle_philox4x32_10.restype = None
        L.oracle_drop_threshold.argtypes = [cf]
        L.oracle_drop_threshold.restype = ctypes.c_uint32
        L.oracle_mask_keep.argtypes = [u64, u64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32,
                                       ctypes.c_uint32]
        L.oracle_mask_keep.restype = ci
        L.oracle_masks.argtypes = [ci, ci, ci, ci, cf, u64, u64, u32p]
        L.oracle_masks.restype = None
        L.oracle_masked_hidden.argtypes = [vp, ci, ci, cf, u64, u64, ci, ci, f64p]
        L.oracle_masked_hidden.restype = None
        L.oracle_logits_row.argtypes = [vp, ci, ci, ci, vp, cf, u64, u64, ci, ci, f64p]
        L.oracle_logits_row.restype = None
        L.oracle_argmax.argtypes = [f64p, ci, f64p]
        L.oracle_argmax.restype = ci
        L.oracle_counts.argtypes = [i32p, ci, ctypes.c_int32, i32p]
        L.oracle_counts.restype = ci
        L.oracle_majority_token.argtypes = [i32p, ci]
        L.oracle_majority_token.restype = ctypes.c_int32
        L.oracle_position_ok.argtypes = [i32p, ci, ctypes.c_int32, ci]
        L.oracle_position_ok.restype = ci
        L.oracle_accept_chain.argtypes = [i32p, i32p, ci, ci, ci]
        L.oracle_accept_chain.restype = ci
        L.oracle_accept_tree.argtypes = [i32p, i32p, i32p, i32p, ci, ci, ci, i32p, i32p]
        L.oracle_accept_tree.restype = ci
        L.oracle_verify_batched.argtypes = [vp, ci, ci, ci, vp, i32p, ci, ci, ci, cf, u64, u64, ci,
                                            i32p, f64p, i32p, i32p, i32p]
        L.oracle_verify_batched.restype = None
        L.oracle_verify_batched_ex.argtypes = [vp, ci, ci, ci, vp, i32p, ci, ci, ci, cf, u64, u64, ci, ci,
                                               i32p, f64p, i32p, i32p, i32p]
        L.oracle_verify_batched_ex.restype = None
        L.oracle_verify_tree.argtypes = [vp, ci, ci, ci, vp, i32p, i32p, i32p, ci, ci, ci, ci, cf,
                                         u64, u64, ci, i32p, f64p, i32p, i32p, i32p, i32p]
        L.oracle_verify_tree.restype = None
        L.oracle_verify_batched_next.argtypes = [vp, ci, ci, ci, vp, i32p, ci, ci, ci, ci, cf, u64, u64, ci,
                                                 i32p, f64p, i32p, i32p, i32p, i32p, f64p, i32p]
        L.oracle_verify_batched_next.restype = None
        L.oracle_js_divergence.argtypes = [f64p, f64p, ci]
        L.oracle_js_divergence.restype = ctypes.c_double
        L.oracle_js_from_logits.argtypes = [f64p, ci, ci, f64p, f64p]
        L.oracle_js_from_logits.restype = ci
        L.oracle_verify_js.argtypes = [vp, ci, ci, ci, vp, i32p, ctypes.POINTER(ctypes.c_float), ci, ci, ci, cf,
                                       u64, u64, i32p, i32p, f64p, i32p, i32p]
        L.oracle_verify_js.restype = None
        cd = ctypes.c_double
        L.oracle_sample_uniform.argtypes = [u64, u64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
        L.oracle_sample_uniform.restype = cd
        L.oracle_gumbel.argtypes = [cd]
        L.oracle_gumbel.restype = cd
        L.oracle_nucleus.argtypes = [f64p, ci, cd, cd, ctypes.POINTER(ctypes.c_ubyte)]
        L.oracle_nucleus.restype = ci
        L.oracle_sample_row.argtypes = [f64p, ci, cd, cd, u64, u64, ctypes.c_uint32, ctypes.c_uint32, f64p]
        L.oracle_sample_row.restype = ci
        L.oracle_verify_batched_sampled.argtypes = [vp, ci, ci, ci, vp, i32p, ci, ci, ci, cf, u64, u64, ci, cd, cd,
                                                    i32p, f64p, i32p, i32p, i32p]
        L.oracle_verify_batched_sampled.restype = None
        _lib = L
    return _lib


def threads() -> int:
    """Threads the OpenMP loop over the vocabulary will use."""
    env = os.environ.get("OMP_NUM_THREADS")
    if env and env.isdigit() and int(env) > 0:
        return int(env)
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# --------------------------------------------------------------------------- helpers
def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _store(a, dtype: int) -> np.ndarray:
    """Storage view the C code reads: float32 for F32, raw uint16 bit patterns for BF16."""
    a = np.ascontiguousarray(a)
    if dtype == F32:
        if a.dtype != np.float32:
            raise TypeError("F32 arrays must be float32")
    else:
        if a.dtype != np.uint16:
            raise TypeError("BF16 arrays must be passed as uint16 bit patterns")
    return a


def _f64p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


# --------------------------------------------------------------------------- wrappers
def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.asarray(ctr, dtype=np.uint32).copy()
    k = np.asarray(key, dtype=np.uint32).copy()
    o = np.zeros(4, dtype=np.uint32)
    u32p = ctypes.POINTER(ctypes.c_uint32)
    lib().oracle_philox4x32_10(c.ctypes.data_as(u32p), k.ctypes.data_as(u32p), o.ctypes.data_as(u32p))
    return o


def drop_threshold(p: float) -> int:
    return int(lib().oracle_drop_threshold(float(np.float32(p))))


def mask_keep(seed: int, s: int, t: int, i: int, j: int, thr: int) -> int:
    return int(lib().oracle_mask_keep(seed, s, t, i, j, thr))


def masks(B, T, K, d, p, seed, seq_base=0) -> np.ndarray:
    """uint32[B,T,K,ceil(d/32)]; bit j%32 of word j//32 set iff element j is kept."""
    out = np.zeros((B, T, K, (d + 31) // 32), dtype=np.uint32)
    lib().oracle_masks(B, T, K, d, float(np.float32(p)), seed, seq_base,
                       out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint32)))
    return out


def masked_hidden(h_row, dtype, p, seed, s, t, i) -> np.ndarray:
    h = _store(h_row, dtype)
    out = np.zeros(h.shape[0], dtype=np.float64)
    lib().oracle_masked_hidden(h.ctypes.data, dtype, h.shape[0], float(np.float32(p)), seed, s, t, i,
                               _f64p(out))
    return out


def logits_row(W, dtype, h_row, p, seed, s, t, i) -> np.ndarray:
    Ws, h = _store(W, dtype), _store(h_row, dtype)
    V, d = Ws.shape
    assert h.shape == (d,)
    out = np.zeros(V, dtype=np.float64)
    lib().oracle_logits_row(Ws.ctypes.data, dtype, V, d, h.ctypes.data, float(np.float32(p)), seed,
                            s, t, i, _f64p(out))
    return out


def argmax(logits):
    l = np.ascontiguousarray(logits, dtype=np.float64)
    gap = ctypes.c_double()
    tok = lib().oracle_argmax(_f64p(l), l.shape[0], ctypes.byref(gap))
    return int(tok), float(gap.value)


def counts(tokens, draft: int):
    t, tp = _i32(tokens)
    c = np.zeros_like(t)
    hits = lib().oracle_counts(tp, t.shape[0], int(draft), c.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
    return c, int(hits)


def majority_token(tokens) -> int:
    t, tp = _i32(tokens)
    return int(lib().oracle_majority_token(tp, t.shape[0]))


def accept_chain(tokens, draft, rule=RULE_NAIVE) -> int:
    t, tp = _i32(tokens)
    d, dp = _i32(draft)
    T, K = t.shape
    assert d.shape == (T,)
    return int(lib().oracle_accept_chain(tp, dp, T, K, rule))


def accept_tree(tokens, node_token, node_parent, node_hrow, rule=RULE_NAIVE):
    """-> (accept_len, best_node, node_ok[N])"""
    t, tp = _i32(tokens)
    nt, ntp = _i32(node_token)
    npar, nparp = _i32(node_parent)
    nh, nhp = _i32(node_hrow)
    N = nt.shape[0]
    ok = np.zeros(max(N, 1), dtype=np.int32)
    best = ctypes.c_int32(-1)
    L = lib().oracle_accept_tree(tp, ntp, nparp, nhp, N, t.shape[1], rule,
                                 ok.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), ctypes.byref(best))
    return int(L), int(best.value), ok[:N]


def verify_batched(W, dtype, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE, shared_masks=False):
    """H[B,T,d], draft[B,T] -> dict(tokens[B,T,K], gap, counts, hits[B,T], accept_len[B]).
    shared_masks: one mask per (sequence, path) for all positions instead of one per position."""
    Ws, Hs = _store(W, dtype), _store(H, dtype)
    V, d = Ws.shape
    B, T, d2 = Hs.shape
    assert d2 == d
    dr, drp = _i32(draft)
    assert dr.shape == (B, T)
    i32p = ctypes.POINTER(ctypes.c_int32)
    tokens = np.zeros((B, T, K), dtype=np.int32)
    gap = np.zeros((B, T, K), dtype=np.float64)
    cnt = np.zeros((B, T, K), dtype=np.int32)
    hits = np.zeros((B, T), dtype=np.int32)
    alen = np.zeros((B,), dtype=np.int32)
    lib().oracle_verify_batched_ex(Ws.ctypes.data, dtype, V, d, Hs.ctypes.data, drp, B, T, K,
                                   float(np.float32(p)), seed, seq_base, rule, int(bool(shared_masks)),
                                   tokens.ctypes.data_as(i32p), _f64p(gap), cnt.ctypes.data_as(i32p),
                                hits.ctypes.data_as(i32p), alen.ctypes.data_as(i32p))
    return dict(tokens=tokens, gap=gap, counts=cnt, hits=hits, accept_len=alen)


def verify_tree(W, dtype, H, node_token, node_parent, node_hrow, K, p, seed, seq_base=0,
                rule=RULE_NAIVE):
    """H[B,N_h,d]; node arrays [B,N] -> dict(tokens[B,N_h,K], gap, counts, node_ok[B,N],
    best_node[B], accept_len[B])."""
    Ws, Hs = _store(W, dtype), _store(H, dtype)
    V, d = Ws.shape
    B, N_h, d2 = Hs.shape
    assert d2 == d
    nt, ntp = _i32(node_token)
    npar, nparp = _i32(node_parent)
    nh, nhp = _i32(node_hrow)
    N = nt.shape[1]
    i32p = ctypes.POINTER(ctypes.c_int32)
    tokens = np.zeros((B, N_h, K), dtype=np.int32)
    gap = np.zeros((B, N_h, K), dtype=np.float64)
    cnt = np.zeros((B, N_h, K), dtype=np.int32)
    ok = np.zeros((B, N), dtype=np.int32)
    best = np.zeros((B,), dtype=np.int32)
    alen = np.zeros((B,), dtype=np.int32)
    lib().oracle_verify_tree(Ws.ctypes.data, dtype, V, d, Hs.ctypes.data, ntp, nparp, nhp, B, N_h, N,
                             K, float(np.float32(p)), seed, seq_base, rule,
                             tokens.ctypes.data_as(i32p), _f64p(gap), cnt.ctypes.data_as(i32p),
                             ok.ctypes.data_as(i32p), best.ctypes.data_as(i32p),
                             alen.ctypes.data_as(i32p))
    return dict(tokens=tokens, gap=gap, counts=cnt, node_ok=ok, best_node=best, accept_len=alen)


def js_divergence(P, Q) -> float:
    """Jensen-Shannon divergence (natural logarithm) of two probability vectors."""
    P = np.ascontiguousarray(P, dtype=np.float64)
    Q = np.ascontiguousarray(Q, dtype=np.float64)
    assert P.shape == Q.shape and P.ndim == 1
    return float(lib().oracle_js_divergence(_f64p(P), _f64p(Q), P.shape[0]))


def js_from_logits(logits, draft_prob):
    """logits[K,V], draft_prob[V] -> (js[K+1], eq5_holds): JS of each head and of the draft to the
    centroid of Eq. 4."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    dp = np.ascontiguousarray(draft_prob, dtype=np.float64)
    K, V = l.shape
    assert dp.shape == (V,)
    out = np.zeros(K + 1, dtype=np.float64)
    ok = lib().oracle_js_from_logits(_f64p(l), K, V, _f64p(dp), _f64p(out))
    return out, bool(ok)


def verify_js(W, dtype, H, draft, draft_prob, K, p, seed, seq_base=0):
    """Algorithm 1 on B chains.  draft_prob[B,T,V] float32.
    -> dict(tokens[B,T,K], counts, js[B,T,K+1], js_ok[B,T], accept_len[B])."""
    Ws, Hs = _store(W, dtype), _store(H, dtype)
    V, d = Ws.shape
    B, T, d2 = Hs.shape
    assert d2 == d
    dr, drp = _i32(draft)
    dp = np.ascontiguousarray(draft_prob, dtype=np.float32)
    assert dr.shape == (B, T) and dp.shape == (B, T, V)
    i32p = ctypes.POINTER(ctypes.c_int32)
    tokens = np.zeros((B, T, K), dtype=np.int32)
    cnt = np.zeros((B, T, K), dtype=np.int32)
    js = np.zeros((B, T, K + 1), dtype=np.float64)
    js_ok = np.zeros((B, T), dtype=np.int32)
    alen = np.zeros((B,), dtype=np.int32)
    lib().oracle_verify_js(Ws.ctypes.data, dtype, V, d, Hs.ctypes.data, drp,
                           dp.ctypes.data_as(ctypes.POINTER(ctypes.c_float)), B, T, K, float(np.float32(p)), seed,
                           seq_base, tokens.ctypes.data_as(i32p), cnt.ctypes.data_as(i32p), _f64p(js),
                           js_ok.ctypes.data_as(i32p), alen.ctypes.data_as(i32p))
    return dict(tokens=tokens, counts=cnt, js=js, js_ok=js_ok, accept_len=alen)


def verify_batched_next(W, dtype, H, draft, K, p, seed, seq_base=0, rule=RULE_NAIVE):
    """H[B,T_h,d] with T_h = T or T+1, draft[B,T] -> verify_batched's outputs (tokens/counts over
    T_h rows) plus plain[B,T_h], plain_gap, next[B]."""
    Ws, Hs = _store(W, dtype), _store(H, dtype)
    V, d = Ws.shape
    B, T_h, d2 = Hs.shape
    dr, drp = _i32(draft)
    T = dr.shape[1]
    assert d2 == d and dr.shape[0] == B and T_h - T in (0, 1)
    i32p = ctypes.POINTER(ctypes.c_int32)
    tokens = np.zeros((B, T_h, K), dtype=np.int32)
    gap = np.zeros((B, T_h, K), dtype=np.float64)
    cnt = np.zeros((B, T_h, K), dtype=np.int32)
    hits = np.zeros((B, T), dtype=np.int32)
    alen = np.zeros((B,), dtype=np.int32)
    plain = np.zeros((B, T_h), dtype=np.int32)
    pgap = np.zeros((B, T_h), dtype=np.float64)
    nxt = np.zeros((B,), dtype=np.int32)
    lib().oracle_verify_batched_next(Ws.ctypes.data, dtype, V, d, Hs.ctypes.data, drp, B, T, T_h - T, K,
                                     float(np.float32(p)), seed, seq_base, rule, tokens.ctypes.data_as(i32p),
                                     _f64p(gap), cnt.ctypes.data_as(i32p), hits.ctypes.data_as(i32p),
                                     alen.ctypes.data_as(i32p), plain.ctypes.data_as(i32p), _f64p(pgap),
                                     nxt.ctypes.data_as(i32p))
    return dict(tokens=tokens, gap=gap, counts=cnt, hits=hits, accept_len=alen, plain=plain, plain_gap=pgap,
                next=nxt)


def sample_uniform(seed: int, s: int, t: int, i: int, v: int) -> float:
    """The uniform variate in (0,1) behind the Gumbel noise of vocabulary entry v."""
    return float(lib().oracle_sample_uniform(seed, s, t, i, v))


def gumbel(u: float) -> float:
    return float(lib().oracle_gumbel(float(u)))


def nucleus(logits, temperature: float, top_p: float) -> np.ndarray:
    """bool[V]: the tokens nucleus sampling may draw from Softmax(logits / temperature)."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    out = np.zeros(l.shape[0], dtype=np.uint8)
    lib().oracle_nucleus(_f64p(l), l.shape[0], float(temperature), float(top_p),
                         out.ctypes.data_as(ctypes.POINTER(ctypes.c_ubyte)))
    return out.astype(bool)


def sample_row(logits, temperature, top_p, seed, s, t, i):
    """-> (token, gap): one draw of the sampling decode rule from a row of logits."""
    l = np.ascontiguousarray(logits, dtype=np.float64)
    gap = ctypes.c_double()
    tok = lib().oracle_sample_row(_f64p(l), l.shape[0], float(temperature), float(top_p), seed, s, t, i,
                                  ctypes.byref(gap))
    return int(tok), float(gap.value)


def verify_batched_sampled(W, dtype, H, draft, K, p, seed, temperature=1.0, top_p=1.0, seq_base=0, rule=RULE_NAIVE):
    """verify_batched with every path's token drawn by the sampling decode rule instead of the argmax."""
    Ws, Hs = _store(W, dtype), _store(H, dtype)
    V, d = Ws.shape
    B, T, d2 = Hs.shape
    assert d2 == d
    dr, drp = _i32(draft)
    assert dr.shape == (B, T)
    i32p = ctypes.POINTER(ctypes.c_int32)
    tokens = np.zeros((B, T, K), dtype=np.int32)
    gap = np.zeros((B, T, K), dtype=np.float64)
    cnt = np.zeros((B, T, K), dtype=np.int32)
    hits = np.zeros((B, T), dtype=np.int32)
    alen = np.zeros((B,), dtype=np.int32)
    lib().oracle_verify_batched_sampled(Ws.ctypes.data, dtype, V, d, Hs.ctypes.data, drp, B, T, K,
                                        float(np.float32(p)), seed, seq_base, rule, float(temperature), float(top_p),
                                        tokens.ctypes.data_as(i32p), _f64p(gap), cnt.ctypes.data_as(i32p),
                                        hits.ctypes.data_as(i32p), alen.ctypes.data_as(i32p))
    return dict(tokens=tokens, gap=gap, counts=cnt, hits=hits, accept_len=alen)
