"""ctypes front end of the fp64 CPU oracle (`fasa_oracle.c`).

TEST INFRASTRUCTURE ONLY.  Tests, the smoke check and the benchmark's CPU-baseline
leg import this module; nothing on the product path does, and this module never
imports the CUDA package.  It compiles the C file with gcc on first use.

Each wrapper passes numpy arrays to one C function and cites the passage that
function follows (arxiv 2602.03152).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "fasa_oracle.c")
_LIB = os.path.join(_HERE, "libfasa_oracle.so")
_lock = threading.Lock()
_lib = None

_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)
_u16p = ctypes.POINTER(ctypes.c_uint16)


def build(force: bool = False) -> str:
    """Compile the oracle into a shared object next to its source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["gcc", "-O2", "-std=c99", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
            )
            os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.fasa_oracle_bf16_to_f64.restype = ctypes.c_double
        _lib.fasa_oracle_bf16_to_f64.argtypes = [ctypes.c_uint16]
        _lib.fasa_oracle_f32_to_bf16.restype = ctypes.c_uint16
        _lib.fasa_oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.fasa_oracle_theta.restype = ctypes.c_double
        _lib.fasa_oracle_theta.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_double]
        _lib.fasa_oracle_select.restype = ctypes.c_int
        _lib.fasa_oracle_decode_bf16.restype = ctypes.c_int
    return _lib


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _ptr(a, t):
    return a.ctypes.data_as(t) if a is not None else None


def bf16_bits_to_f64(bits) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float64."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    out = np.empty(bits.shape, dtype=np.float64)
    _load().fasa_oracle_widen_bf16(_ptr(bits, _u16p), ctypes.c_int64(bits.size), _ptr(out, _f64p))
    return out


def f32_to_bf16_bits(x: float) -> int:
    """Round-to-nearest-even binary32 -> bf16 bits."""
    return int(_load().fasa_oracle_f32_to_bf16(ctypes.c_float(x)))


def theta(i: int, d: int, base: float) -> float:
    """theta_i = B^(-2i/d), 0-based FC index (Sec. 3.1)."""
    return float(_load().fasa_oracle_theta(i, d, ctypes.c_double(base)))


def rope(x, pos: float, base: float, pairing: int = 0) -> np.ndarray:
    """Rotate every FC of one d-vector to position `pos` (Sec. 3.1, Eq. 1)."""
    x = _f64(x)
    assert x.ndim == 1 and x.size % 2 == 0
    out = np.empty_like(x)
    _load().fasa_oracle_rope(_ptr(x, _f64p), ctypes.c_int(x.size), ctypes.c_double(pos),
                             ctypes.c_double(base), ctypes.c_int(pairing), _ptr(out, _f64p))
    return out


def fc_partial_logits(q, K, pairing: int = 0) -> np.ndarray:
    """Single-FC raw scores alpha^(i)[j] for all i, shape [d/2, L] (Sec. 3.3, Eq. 3)."""
    q, K = _f64(q), _f64(K)
    L, d = K.shape
    a = np.empty((d // 2, L), dtype=np.float64)
    _load().fasa_oracle_fc_partial_logits(_ptr(q, _f64p), _ptr(K, _f64p), ctypes.c_int(L),
                                          ctypes.c_int(d), ctypes.c_int(pairing), _ptr(a, _f64p))
    return a


def fc_score(q, K, dom, pairing: int = 0, group_reduce: int = 0) -> np.ndarray:
    """Importance scores S_t[j] of one KV head from its G query heads (Sec. 4.1, TIP)."""
    q, K = _f64(q), _f64(K)
    if q.ndim == 1:
        q = q[None, :]
    G, d = q.shape
    L = K.shape[0]
    dom = np.ascontiguousarray(dom, dtype=np.int32)
    S = np.empty(L, dtype=np.float64)
    _load().fasa_oracle_fc_score(_ptr(q, _f64p), ctypes.c_int(G), _ptr(K, _f64p), ctypes.c_int(L),
                                 ctypes.c_int(d), ctypes.c_int(pairing), _ptr(dom, _i32p),
                                 ctypes.c_int(dom.size), ctypes.c_int(group_reduce), _ptr(S, _f64p))
    return S


def select(S, k: int, n_sink: int = 0, n_recent: int = 0, tie_rel: float = 1e-3):
    """T_t = forced U TopK-I(S_t, k), ascending; also the boundary record (Sec. 4.1)."""
    S = _f64(S)
    L = S.size
    idx = np.empty(max(L, 1), dtype=np.int32)
    band = np.zeros(4, dtype=np.float64)
    n = _load().fasa_oracle_select(_ptr(S, _f64p), ctypes.c_int(L), ctypes.c_int(k),
                                   ctypes.c_int(n_sink), ctypes.c_int(n_recent),
                                   ctypes.c_double(tie_rel), _ptr(idx, _i32p), _ptr(band, _f64p))
    info = {"has_boundary": bool(band[0]), "s_k": band[1], "s_k1": band[2], "tie": bool(band[3])}
    return idx[:n].copy(), info


def attn_subset(q, K, V, idx, scale: float):
    """FAC on the selected rows: (O [G,d], lse [G]) (Sec. 4.2, Eq. 6-7)."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    if q.ndim == 1:
        q = q[None, :]
    G, d = q.shape
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    O = np.empty((G, d), dtype=np.float64)
    lse = np.empty(G, dtype=np.float64)
    _load().fasa_oracle_attn_subset(_ptr(q, _f64p), ctypes.c_int(G), _ptr(K, _f64p), _ptr(V, _f64p),
                                    ctypes.c_int(d), _ptr(idx, _i32p), ctypes.c_int(idx.size),
                                    ctypes.c_double(scale), _ptr(O, _f64p), _ptr(lse, _f64p))
    return O, lse


def attn_dense(q, K, V, L: int, scale: float):
    """Full-KV attention over rows 0..L-1 (FKV, Sec. 5.1)."""
    q, K, V = _f64(q), _f64(K), _f64(V)
    if q.ndim == 1:
        q = q[None, :]
    G, d = q.shape
    O = np.empty((G, d), dtype=np.float64)
    lse = np.empty(G, dtype=np.float64)
    _load().fasa_oracle_attn_dense(_ptr(q, _f64p), ctypes.c_int(G), _ptr(K, _f64p), _ptr(V, _f64p),
                                   ctypes.c_int(d), ctypes.c_int(L), ctypes.c_double(scale),
                                   _ptr(O, _f64p), _ptr(lse, _f64p))
    return O, lse


def ca_counts(q, K, top_k: int, pairing: int = 0, f32: bool = False) -> np.ndarray:
    """top_k * CA of every FC for one query head (Sec. 3.3, Eq. 4): sizes of the
    intersections of the full-head and single-FC top-k index sets."""
    q, K = _f64(q), _f64(K)
    L, d = K.shape
    c = np.zeros(d // 2, dtype=np.int32)
    _load().fasa_oracle_ca_counts(_ptr(q, _f64p), _ptr(K, _f64p), ctypes.c_int(L), ctypes.c_int(d),
                                  ctypes.c_int(pairing), ctypes.c_int(top_k), ctypes.c_int(int(f32)),
                                  _ptr(c, _i32p))
    return c


def calibrate_bf16(q_bits, K_bits, seq_lens, top_k: int, *, pairing=0, f32=True, n_threads=0,
                   counts=None, n_used=None):
    """Stage 1 of Algorithm 1 on bf16 bit patterns: adds every (sequence, query head) sample's
    intersection counts to counts [Hq, d/2] and the sample count to n_used [Hq] (int64)."""
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    K_bits = np.ascontiguousarray(K_bits, dtype=np.uint16)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, Hq, d = q_bits.shape
    _, Hkv, Lmax, _ = K_bits.shape
    counts = np.zeros((Hq, d // 2), dtype=np.int64) if counts is None else counts
    n_used = np.zeros(Hq, dtype=np.int64) if n_used is None else n_used
    i64p = ctypes.POINTER(ctypes.c_int64)
    _load().fasa_oracle_calibrate_bf16(
        _ptr(q_bits, _u16p), _ptr(K_bits, _u16p), _ptr(seq_lens, _i32p), ctypes.c_int(B), ctypes.c_int(Hq),
        ctypes.c_int(Hkv), ctypes.c_int(d), ctypes.c_int(Lmax), ctypes.c_int(pairing), ctypes.c_int(top_k),
        ctypes.c_int(int(f32)), ctypes.c_int(n_threads), _ptr(counts, i64p), _ptr(n_used, i64p))
    return counts, n_used


def select_dominant(counts, n_used, n_kv_heads: int, top_k: int, n_dom: int):
    """Stage 2 of Algorithm 1: (I_dom [Hkv, n_dom] ascending, mean CA [Hkv, d/2])."""
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    n_used = np.ascontiguousarray(n_used, dtype=np.int64)
    Hq, n_fc = counts.shape
    dom = np.zeros((n_kv_heads, n_dom), dtype=np.int32)
    mean = np.zeros((n_kv_heads, n_fc), dtype=np.float64)
    i64p = ctypes.POINTER(ctypes.c_int64)
    _load().fasa_oracle_select_dominant(_ptr(counts, i64p), _ptr(n_used, i64p), ctypes.c_int(Hq),
                                        ctypes.c_int(n_kv_heads), ctypes.c_int(n_fc), ctypes.c_int(top_k),
                                        ctypes.c_int(n_dom), _ptr(dom, _i32p), _ptr(mean, _f64p))
    return dom, mean


def decode_bf16(q_bits, K_bits, V_bits, seq_lens, dom, *, pairing=0, group_reduce=0, n_sink=0,
                n_recent=0, budget=256, n_sel_max=None, scale=None, tie_rel=1e-3, n_threads=0,
                sel_heads=0, want_scores=True, want_sparse=True, want_dense=True):
    """One whole decode step on bf16 bit patterns, unit by unit in the paper's order.

    q_bits [B,Hq,d], K_bits/V_bits [B,Hkv,Lmax,d] (uint16), seq_lens [B], dom [Hkv,F].
    sel_heads query heads share one index set (0 = all heads of a KV head, 1 = one set per
    query head, the per-head reading of Sec. 4.1); scores, idx, n_sel and band then have
    Hs = Hq / sel_heads rows per sequence instead of Hkv.
    Returns a dict with scores, idx, n_sel, band, out, lse, dense_out, dense_lse, threads.
    """
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    K_bits = np.ascontiguousarray(K_bits, dtype=np.uint16)
    V_bits = np.ascontiguousarray(V_bits, dtype=np.uint16)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    dom = np.ascontiguousarray(dom, dtype=np.int32)
    B, Hq, d = q_bits.shape
    _, Hkv, Lmax, _ = K_bits.shape
    F = dom.shape[1]
    if scale is None:
        scale = 1.0 / np.sqrt(float(d))
    if n_sel_max is None:
        n_sel_max = Lmax
    group = Hq // Hkv
    per = sel_heads if sel_heads > 0 else group
    if per <= 0 or group % per != 0:
        raise ValueError("sel_heads must divide the group")
    Hs = Hq // per
    scores = np.full((B, Hs, Lmax), np.nan, dtype=np.float64) if want_scores else None
    idx = np.full((B, Hs, n_sel_max), -1, dtype=np.int32)
    n_sel = np.zeros((B, Hs), dtype=np.int32)
    band = np.zeros((B, Hs, 4), dtype=np.float64)
    out = np.zeros((B, Hq, d), dtype=np.float64) if want_sparse else None
    lse = np.zeros((B, Hq), dtype=np.float64) if want_sparse else None
    dout = np.zeros((B, Hq, d), dtype=np.float64) if want_dense else None
    dlse = np.zeros((B, Hq), dtype=np.float64) if want_dense else None
    used = _load().fasa_oracle_decode_bf16(
        _ptr(q_bits, _u16p), _ptr(K_bits, _u16p), _ptr(V_bits, _u16p), _ptr(seq_lens, _i32p),
        _ptr(dom, _i32p), ctypes.c_int(B), ctypes.c_int(Hq), ctypes.c_int(Hkv), ctypes.c_int(d),
        ctypes.c_int(Lmax), ctypes.c_int(F), ctypes.c_int(pairing), ctypes.c_int(group_reduce),
        ctypes.c_int(n_sink), ctypes.c_int(n_recent), ctypes.c_int(budget),
        ctypes.c_int(n_sel_max), ctypes.c_double(scale), ctypes.c_double(tie_rel),
        ctypes.c_int(n_threads), ctypes.c_int(sel_heads), _ptr(scores, _f64p), _ptr(idx, _i32p), _ptr(n_sel, _i32p),
        _ptr(band, _f64p), _ptr(out, _f64p), _ptr(lse, _f64p), _ptr(dout, _f64p), _ptr(dlse, _f64p))
    if used < 0:
        raise ValueError("sel_heads must divide the group")
    return {"scores": scores, "idx": idx, "n_sel": n_sel, "band": band, "out": out, "lse": lse,
            "dense_out": dout, "dense_lse": dlse, "threads": int(used)}


def decode_batched_bf16(q_bits, K_bits, V_bits, seq_lens, dom, **kw):
    """A block of T query tokens per sequence (speculative / multi-token decoding).

    The method defines token importance prediction and focused attention for ONE query q_t
    (Sec. 4.1-4.2: S_t, T_t and Eq. 6-7 all carry the index t).  A block of T queries is
    therefore T decode steps, nothing else: query t of the block (0 <= t < T) is the query of
    the cache position L - T + t, where L = seq_lens[b] counts the rows cached INCLUDING the
    block's own T keys; it sees the rows at positions <= its own (rows j < L - (T - 1 - t)),
    and has its own scores, its own index set and its own output.  Written out as exactly that:
    T calls of decode_bf16 on the shortened caches.

    q_bits [B,T,Hq,d]; K_bits, V_bits, seq_lens, dom and the keyword arguments as decode_bf16.
    Returns the dict of decode_bf16 with a token axis after the batch axis ([B,T,...]).
    """
    q_bits = np.ascontiguousarray(q_bits, dtype=np.uint16)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, T = q_bits.shape[:2]
    steps = []
    for t in range(T):
        lens_t = np.maximum(seq_lens - (T - 1 - t), 0).astype(np.int32)
        steps.append(decode_bf16(q_bits[:, t], K_bits, V_bits, lens_t, dom, **kw))
    out = {"threads": steps[0]["threads"]}
    for key in ("scores", "idx", "n_sel", "band", "out", "lse", "dense_out", "dense_lse"):
        out[key] = None if steps[0][key] is None else np.stack([s_[key] for s_ in steps], axis=1)
    return out

