"""Parity rules between a candidate result and the fp64 oracle.

TEST INFRASTRUCTURE ONLY (used by tests/, the smoke check and the benchmark's
self-check).  Takes plain numpy arrays; knows nothing about the CUDA library.

Rules
  scores     |S - S_oracle| <= 1e-5 * sum_g sum_{dominant channels} |q_c k_c|
             (fp32 accumulation of exact bf16 products).
  selection  bit-exact sets wherever the oracle's k-th and (k+1)-th ranked scores
             differ by more than 1e-3 relative; otherwise the sets may differ only
             inside the tie band around the k-th score, sizes equal.
  attention  max-abs <= 2e-3 against the oracle run on the candidate's own index
             set (which is the oracle's set whenever the sets agree).
"""
from __future__ import annotations

import numpy as np

from . import fasa_oracle as O

SCORE_REL = 1e-5
TIE_REL = 1e-3
ATTN_ABS = 2e-3


def dominant_channels(dom, pairing: int, d: int = 128) -> np.ndarray:
    dom = np.asarray(dom, dtype=np.int64)
    return np.concatenate([dom, dom + d // 2]) if pairing == 0 else np.concatenate([2 * dom, 2 * dom + 1])


def score_bound(q64, k64, ch) -> np.ndarray:
    """sum_g sum_c |q_gc k_jc| per row j (q64 [G,d], k64 [L,d])."""
    return np.abs(k64[:, ch]) @ np.abs(q64[:, ch]).sum(axis=0)


def check_scores(s_gpu, s_or, bound, what=""):
    err = np.abs(np.asarray(s_gpu, dtype=np.float64) - s_or)
    lim = SCORE_REL * bound + 1e-30
    worst = int(np.argmax(err / lim))
    assert np.all(err <= lim), f"{what}: score {worst} off by {err[worst]:.3e} > {lim[worst]:.3e}"


def check_selection(idx_gpu, s_or, L, k, n_sink, n_recent, what=""):
    """Applies the selection rule; returns True when the sets are identical."""
    idx_or, info = O.select(s_or[:L], k, n_sink, n_recent, TIE_REL)
    idx_gpu = np.asarray(idx_gpu)
    assert idx_gpu.size == idx_or.size, f"{what}: n_sel {idx_gpu.size} != {idx_or.size}"
    assert np.all(np.diff(idx_gpu) > 0), f"{what}: indices not strictly ascending"
    if idx_gpu.size:
        assert idx_gpu[0] >= 0 and idx_gpu[-1] < L, f"{what}: index out of range"
    if np.array_equal(idx_gpu, idx_or):
        return True
    assert info["tie"], f"{what}: sets differ although the boundary scores are {info['s_k']} / {info['s_k1']}"
    tol = TIE_REL * max(abs(info["s_k"]), abs(info["s_k1"]))
    diff = np.setxor1d(idx_gpu, idx_or)
    forced = (diff < n_sink) | (diff >= L - n_recent)
    assert not forced.any(), f"{what}: a forced position is missing"
    off = np.abs(s_or[diff] - info["s_k"])
    assert np.all(off <= tol), f"{what}: sets differ outside the tie band ({off.max():.3e} > {tol:.3e})"
    return False


def check_attention(out_gpu, out_or, what="", tol=ATTN_ABS):
    err = np.abs(np.asarray(out_gpu, dtype=np.float64) - out_or)
    assert np.all(np.isfinite(out_gpu)), f"{what}: non-finite output"
    assert err.max() <= tol, f"{what}: attention max-abs error {err.max():.3e} > {tol}"
    return float(err.max())


def check_step(q, k, v, seq_lens, dom, *, pairing, group_reduce, n_sink, n_recent, budget, scale,
               scores=None, idx=None, n_sel=None, out=None, dense_out=None, units=None, sel_heads=0, what=""):
    """Checks whatever parts of one decode step are given (numpy arrays in the library's
    layouts; q/k/v as float64 widenings of the bf16 inputs) against the oracle, unit by unit.
    A unit is (b, hs): sel_heads query heads sharing one index set (0 = all heads of a KV
    head).  `units` limits the check to some (b, hs) pairs.  Returns a small report dict."""
    B, Hq, d = q.shape
    Hkv = k.shape[1]
    group = Hq // Hkv
    G = sel_heads if sel_heads > 0 else group
    Hs = Hq // G
    rep = {"units": 0, "sets_identical": 0, "attn_err": 0.0, "dense_err": 0.0}
    todo = units if units is not None else [(b, hs) for b in range(B) for hs in range(Hs)]
    for (b, hs) in todo:
        h = hs * G // group                      # the KV head this unit attends
        L = int(min(max(int(seq_lens[b]), 0), k.shape[2]))
        tag = f"{what}[b={b},unit={hs},kv={h},L={L}]"
        qs, ks, vs = q[b, hs * G:(hs + 1) * G], k[b, h, :L], v[b, h, :L]
        s_or = O.fc_score(qs, ks, dom[h], pairing, group_reduce) if L > 0 else np.zeros(0)
        kk = budget if budget > 0 else (-budget * L + 999) // 1000
        rep["units"] += 1
        if scores is not None and L > 0:
            bound = score_bound(qs, ks, dominant_channels(dom[h], pairing, d))
            check_scores(scores[b, hs, :L], s_or, bound, tag)
        sel = None
        if idx is not None:
            n = int(n_sel[b, hs])
            sel = np.asarray(idx[b, hs, :n])
            rep["sets_identical"] += bool(check_selection(sel, s_or, L, kk, n_sink, n_recent, tag))
        if out is not None:
            if sel is None:
                sel, _ = O.select(s_or, kk, n_sink, n_recent, TIE_REL)
            o_or, _ = O.attn_subset(qs, ks, vs, sel, scale)
            rep["attn_err"] = max(rep["attn_err"], check_attention(out[b, hs * G:(hs + 1) * G], o_or, tag + " sparse"))
        if dense_out is not None:
            o_or, _ = O.attn_dense(qs, ks, vs, L, scale)
            rep["dense_err"] = max(rep["dense_err"], check_attention(dense_out[b, hs * G:(hs + 1) * G], o_or, tag + " dense"))
    return rep
