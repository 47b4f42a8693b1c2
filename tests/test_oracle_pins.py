"""Pins of the fp64 CPU oracle against what the paper and the mathematics fix.

None of these tests re-types an oracle formula: each compares an oracle function
with hand-worked numbers (tests/golden/worked_example_d4.json), a closed form, an
invariant the paper states, a library routine (numpy matmul, torch.topk, torch
SDPA in fp64), an independent complex-number / brute-force formulation, or the
separately written input generator.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import fasa_oracle as O
from paper_2602_03152_b200 import synth

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "worked_example_d4.json")))
RNG = np.random.default_rng(1234)


# ----------------------------------------------------------------- bf16 ----

def test_bf16_widening_matches_torch():
    bits = np.arange(0, 65536, dtype=np.uint32).astype(np.uint16)
    mine = O.bf16_bits_to_f64(bits)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    both_nan = np.isnan(mine) & np.isnan(ref)
    assert np.array_equal(mine[~both_nan], ref[~both_nan])


def test_bf16_rounding_matches_torch():
    xs = np.concatenate([RNG.standard_normal(4000) * 10.0 ** RNG.integers(-6, 6, 4000),
                         [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, np.inf, -np.inf]])
    xs = xs.astype(np.float32)
    ref = torch.from_numpy(xs).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    mine = np.array([O.f32_to_bf16_bits(float(x)) for x in xs], dtype=np.uint16)
    assert np.array_equal(mine, ref)


# ----------------------------------------------------------------- RoPE ----

def test_theta_closed_forms():
    # Sec. 3.1: theta_i = B^(-2i/d); FC 0 turns one radian per position, the last
    # FC turns slowest.
    assert O.theta(0, 128, 500000.0) == 1.0
    assert math.isclose(O.theta(63, 128, 500000.0), 500000.0 ** (-126.0 / 128.0), rel_tol=1e-15)
    assert math.isclose(O.theta(32, 128, 10000.0), 0.01, rel_tol=1e-14)
    th = [O.theta(i, 128, 500000.0) for i in range(64)]
    assert all(a > b for a, b in zip(th, th[1:]))
    assert GOLD["rope"]["theta"] == pytest.approx([O.theta(0, 4, 100.0), O.theta(1, 4, 100.0)], rel=1e-15)


def test_rope_hand_worked():
    g = GOLD["rope"]
    assert O.rope(g["x"], g["pos"], g["base"], 0) == pytest.approx(g["rotate_half"], abs=1e-14)
    assert O.rope(g["x"], g["pos"], g["base"], 1) == pytest.approx(g["interleaved"], abs=1e-14)


def test_rope_quarter_turn_and_norm():
    # FC 0 has theta = 1: position pi/2 maps (1, 0) to (0, 1) (counter-clockwise, Eq. 1).
    x = np.zeros(128); x[0] = 1.0
    y = O.rope(x, math.pi / 2, 500000.0, 0)
    assert abs(y[0]) < 1e-15 and abs(y[64] - 1.0) < 1e-15
    y = O.rope(x, math.pi / 2, 500000.0, 1)
    assert abs(y[0]) < 1e-15 and abs(y[1] - 1.0) < 1e-15
    v = RNG.standard_normal(128)
    for pairing in (0, 1):
        r = O.rope(v, 12345.0, 500000.0, pairing)
        assert math.isclose(np.linalg.norm(r), np.linalg.norm(v), rel_tol=1e-13)
        assert np.allclose(O.rope(v, 0.0, 500000.0, pairing), v, atol=0)


@pytest.mark.parametrize("pairing", [0, 1])
def test_rope_is_complex_multiplication(pairing):
    # Textbook form: FC i as the complex number x0 + i x1 is multiplied by e^{i m theta_i}.
    d, base, m = 128, 500000.0, 4097.0
    v = RNG.standard_normal(d)
    c0 = np.arange(64) if pairing == 0 else 2 * np.arange(64)
    c1 = c0 + 64 if pairing == 0 else c0 + 1
    z = (v[c0] + 1j * v[c1]) * np.exp(1j * m * base ** (-2.0 * np.arange(64) / d))
    r = O.rope(v, m, base, pairing)
    assert np.allclose(r[c0], z.real, atol=1e-12) and np.allclose(r[c1], z.imag, atol=1e-12)


@pytest.mark.parametrize("pairing", [0, 1])
def test_relative_position_identity(pairing):
    # Sec. 3.1: (q R_t1)(k R_t2)^T depends on t1 - t2 only, FC by FC.
    d, base = 128, 500000.0
    q, k = RNG.standard_normal(d), RNG.standard_normal(d)
    a = O.fc_partial_logits(O.rope(q, 4096, base, pairing), O.rope(k, 1000, base, pairing)[None], pairing)
    b = O.fc_partial_logits(O.rope(q, 4096 + 777, base, pairing), O.rope(k, 1777, base, pairing)[None], pairing)
    c = O.fc_partial_logits(O.rope(q, 3096, base, pairing), k[None], pairing)
    assert np.allclose(a, b, atol=1e-9) and np.allclose(a, c, atol=1e-9)
    # closed form per FC: |q_i||k_i| cos(phi_q - phi_k + dt * theta_i)
    c0 = np.arange(64) if pairing == 0 else 2 * np.arange(64)
    c1 = c0 + 64 if pairing == 0 else c0 + 1
    zq, zk = q[c0] + 1j * q[c1], k[c0] + 1j * k[c1]
    th = base ** (-2.0 * np.arange(64) / d)
    closed = np.abs(zq) * np.abs(zk) * np.cos(np.angle(zq) - np.angle(zk) + 3096 * th)
    assert np.allclose(a[:, 0], closed, atol=1e-9)


@pytest.mark.parametrize("pairing", [0, 1])
def test_generator_rope_agrees_with_oracle(pairing):
    # The input generator has its own (torch, vectorised) rotation.
    x = torch.from_numpy(RNG.standard_normal((5, 128)))
    pos = torch.tensor([0.0, 1.0, 17.0, 4096.0, 131071.0], dtype=torch.float64)
    got = synth.rope_rotate(x, pos, 500000.0, pairing).numpy()
    for r in range(5):
        assert np.allclose(got[r], O.rope(x[r].numpy(), float(pos[r]), 500000.0, pairing), atol=1e-9)


# --------------------------------------------------------------- scores ----

def test_scores_hand_worked():
    g = GOLD["scores"]
    assert np.array_equal(O.fc_partial_logits(g["q"], g["K"], 0), np.array(g["alpha_fc_rotate_half"]))
    assert np.array_equal(O.fc_partial_logits(g["q"], g["K"], 1), np.array(g["alpha_fc_interleaved"]))
    assert np.array_equal(O.fc_score(g["q"], g["K"], [0, 1], 0), np.array(g["alpha_full"]))
    assert np.array_equal(O.fc_score(g["q"], g["K"], GOLD["select"]["dom"], 0), np.array(GOLD["select"]["S"]))


@pytest.mark.parametrize("pairing", [0, 1])
def test_partial_logits_sum_to_full_dot(pairing):
    # Sec. 4.1: alpha = sum over all d/2 FCs of alpha^(i).
    q, K = RNG.standard_normal(128), RNG.standard_normal((300, 128))
    a = O.fc_partial_logits(q, K, pairing)
    assert a.shape == (64, 300)
    full = K @ q
    assert np.allclose(a.sum(axis=0), full, atol=1e-12 * np.abs(K * q).sum(axis=1).max())
    # each FC touches exactly its two channels: zeroing them kills that FC only
    i = 37
    c0, c1 = (i, i + 64) if pairing == 0 else (2 * i, 2 * i + 1)
    q2 = q.copy(); q2[[c0, c1]] = 0.0
    a2 = O.fc_partial_logits(q2, K, pairing)
    assert np.all(a2[i] == 0.0) and np.array_equal(np.delete(a2, i, 0), np.delete(a, i, 0))


@pytest.mark.parametrize("pairing", [0, 1])
def test_fc_score_is_subset_sum_and_group_sum(pairing):
    G, L = 4, 257
    q, K = RNG.standard_normal((G, 128)), RNG.standard_normal((L, 128))
    dom = np.array([5, 60, 33, 2, 17, 48, 63, 0])
    per_head = np.stack([O.fc_partial_logits(q[g], K, pairing)[dom].sum(axis=0) for g in range(G)])
    assert np.allclose(O.fc_score(q, K, dom, pairing, 0), per_head.sum(axis=0), atol=1e-12)
    assert np.allclose(O.fc_score(q, K, dom, pairing, 1), per_head.max(axis=0), atol=1e-12)
    # order of the dominant list does not matter; all 64 FCs give sum_g q_g . k (library matmul)
    assert np.allclose(O.fc_score(q, K, dom[::-1].copy(), pairing, 0), O.fc_score(q, K, dom, pairing, 0), atol=1e-12)
    assert np.allclose(O.fc_score(q, K, np.arange(64), pairing, 0), (K @ q.T).sum(axis=1), atol=1e-11)
    # brute force with explicit channel lists
    ch = np.concatenate([dom, dom + 64]) if pairing == 0 else np.concatenate([2 * dom, 2 * dom + 1])
    brute = np.zeros(L)
    for j in range(L):
        for g in range(G):
            for c in ch:
                brute[j] += q[g, c] * K[j, c]
    assert np.allclose(O.fc_score(q, K, dom, pairing, 0), brute, atol=1e-12)


# ------------------------------------------------------------ selection ----

def _brute_select(S, k, n_sink, n_recent):
    L = len(S)
    forced = [j for j in range(L) if j < n_sink or j >= L - n_recent]
    rest = [j for j in range(L) if j not in set(forced)]
    # j is kept iff fewer than k others outrank it (higher score, or equal score and lower index)
    kept = [j for j in rest if sum(1 for i in rest if S[i] > S[j] or (S[i] == S[j] and i < j)) < k]
    return sorted(forced + kept)


def test_select_hand_worked():
    g = GOLD["select"]
    idx, info = O.select(g["S"], g["k"])
    assert idx.tolist() == g["T"]
    assert info["has_boundary"] and info["s_k"] == 0.0 and info["s_k1"] == 0.0 and info["tie"]


def test_select_matches_torch_topk_untied():
    S = RNG.standard_normal(5000)
    for k in (1, 7, 256, 4999, 5000, 6000):
        idx, info = O.select(S, k)
        ref = torch.topk(torch.from_numpy(S), min(k, 5000)).indices.sort().values.numpy()
        assert np.array_equal(idx, ref)
        if k < 5000:
            srt = np.sort(S)[::-1]
            assert info["s_k"] == srt[k - 1] and info["s_k1"] == srt[k]
    idx, info = O.select(S, 0)
    assert idx.size == 0 and not info["has_boundary"]


def test_select_ties_and_forced_vs_brute_force():
    for trial in range(30):
        L = int(RNG.integers(1, 60))
        S = RNG.integers(-3, 4, L).astype(np.float64)      # many equal values
        k = int(RNG.integers(0, L + 3))
        ns, nr = int(RNG.integers(0, 5)), int(RNG.integers(0, 5))
        idx, _ = O.select(S, k, ns, nr)
        assert idx.tolist() == _brute_select(S, k, ns, nr), (L, k, ns, nr)
    idx, _ = O.select(np.ones(100), 10)
    assert idx.tolist() == list(range(10))                 # all equal: lowest indices
    idx, _ = O.select(np.arange(100.0), 5, 4, 6)
    assert idx.tolist() == [0, 1, 2, 3] + [89, 90, 91, 92, 93] + [94, 95, 96, 97, 98, 99]
    idx, _ = O.select(np.arange(10.0), 3, 8, 8)             # overlapping forced ranges
    assert idx.tolist() == list(range(10))


def test_select_tie_band_flag():
    S = np.array([10.0, 9.0, 5.0, 4.9999, 1.0])
    assert O.select(S, 3)[1]["tie"]            # 5.0 vs 4.9999: within 1e-3 relative
    assert not O.select(S, 2)[1]["tie"]        # 9.0 vs 5.0
    assert not O.select(S, 4)[1]["tie"]


# ------------------------------------------------------------ attention ----

def test_fac_hand_worked():
    s, f = GOLD["scores"], GOLD["fac"]
    out, lse = O.attn_subset(s["q"], s["K"], f["V"], GOLD["select"]["T"], f["scale"])
    assert out[0] == pytest.approx(f["O"], abs=1e-15)
    assert lse[0] == pytest.approx(f["lse"], abs=1e-15)


def test_dense_matches_torch_sdpa_fp64():
    G, L, d = 4, 777, 128
    q, K, V = RNG.standard_normal((G, d)), RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    out, lse = O.attn_dense(q, K, V, L, 1 / math.sqrt(d))
    tq, tk, tv = (torch.from_numpy(a) for a in (q, K, V))
    ref = torch.nn.functional.scaled_dot_product_attention(tq[None, :, None, :], tk[None, None].expand(1, G, L, d),
                                                           tv[None, None].expand(1, G, L, d))
    assert np.allclose(out, ref[0, :, 0].numpy(), atol=1e-13)
    assert np.allclose(lse, torch.logsumexp(tq @ tk.T / math.sqrt(d), dim=1).numpy(), atol=1e-12)
    # only the first L rows count
    out2, _ = O.attn_dense(q, K, V, 100, 1 / math.sqrt(d))
    ref2 = torch.softmax(tq @ tk[:100].T / math.sqrt(d), dim=1) @ tv[:100]
    assert np.allclose(out2, ref2.numpy(), atol=1e-13)


def test_subset_properties():
    G, L, d = 3, 400, 128
    q, K, V = RNG.standard_normal((G, d)), RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    sc = 1 / math.sqrt(d)
    idx = np.sort(RNG.choice(L, 50, replace=False)).astype(np.int32)
    out, lse = O.attn_subset(q, K, V, idx, sc)
    tq, tk, tv = torch.from_numpy(q), torch.from_numpy(K[idx]), torch.from_numpy(V[idx])
    assert np.allclose(out, (torch.softmax(tq @ tk.T * sc, 1) @ tv).numpy(), atol=1e-13)   # gather, then library
    perm = RNG.permutation(50)
    out_p, lse_p = O.attn_subset(q, K, V, idx[perm], sc)                                    # order-free
    assert np.allclose(out, out_p, atol=1e-13) and np.allclose(lse, lse_p, atol=1e-13)
    one, lse1 = O.attn_subset(q, K, V, [123], sc)                                           # one token: its value row
    assert np.array_equal(one, np.tile(V[123], (G, 1))) and np.allclose(lse1, q @ K[123] * sc)
    flat, _ = O.attn_subset(np.zeros((G, d)), K, V, idx, sc)                                # q = 0: plain mean
    assert np.allclose(flat, np.tile(V[idx].mean(0), (G, 1)), atol=1e-13)
    allrows, _ = O.attn_subset(q, K, V, np.arange(L), sc)                                   # whole cache = dense
    dense, _ = O.attn_dense(q, K, V, L, sc)
    assert np.array_equal(allrows, dense)
    empty, lse0 = O.attn_subset(q, K, V, np.zeros(0, np.int32), sc)
    assert np.all(empty == 0) and np.all(np.isneginf(lse0))
    big, _ = O.attn_subset(q * 300, K, V, idx, sc)                                          # no overflow
    assert np.all(np.isfinite(big))


def test_lse_merge_identity():
    # Any split of the selection, merged with the log-sum-exp weights, gives the whole.
    G, L, d = 2, 300, 128
    q, K, V = RNG.standard_normal((G, d)), RNG.standard_normal((L, d)), RNG.standard_normal((L, d))
    sc = 1 / math.sqrt(d)
    idx = RNG.permutation(L)[:120]
    whole, lse = O.attn_subset(q, K, V, idx, sc)
    parts = [O.attn_subset(q, K, V, idx[a:b], sc) for a, b in ((0, 1), (1, 50), (50, 120))]
    m = np.max([p[1] for p in parts], axis=0)
    w = [np.exp(p[1] - m) for p in parts]
    merged = sum(wi[:, None] * p[0] for wi, p in zip(w, parts)) / sum(w)[:, None]
    assert np.allclose(merged, whole, atol=1e-13)
    assert np.allclose(m + np.log(sum(w)), lse, atol=1e-13)


# ----------------------------------------------------------- whole step ----

def _small_workload(**kw):
    kw.setdefault("budget", 40)
    w = synth.CONFIGS["c1"].replace(batch=2, max_len=600, len_lo=300, len_hi=600, **kw)
    return w, synth.make_inputs(w, "cpu")


def test_decode_step_composes_the_parts():
    w, t = _small_workload()
    qb, kb, vb = synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"])
    r = O.decode_bf16(qb, kb, vb, t["seq_lens"].numpy(), t["dom"].numpy(), n_sink=w.n_sink,
                      n_recent=w.n_recent, budget=w.budget, n_threads=2)
    q64, k64, v64 = t["q"].double().numpy(), t["k"].double().numpy(), t["v"].double().numpy()
    G, sc = w.group, 1 / math.sqrt(128)
    for b in range(w.batch):
        L = int(t["seq_lens"][b])
        for h in range(w.n_kv_heads):
            dom = t["dom"][h].numpy()
            ch = np.concatenate([dom, dom + 64])
            qs = q64[b, h * G:(h + 1) * G]
            S = (k64[b, h, :L][:, ch] @ qs[:, ch].T).sum(axis=1)                # library matmul
            assert np.allclose(r["scores"][b, h, :L], S, atol=1e-11)
            assert np.all(np.isnan(r["scores"][b, h, L:]))                       # rows past L untouched
            n = int(r["n_sel"][b, h])
            assert n == min(L, w.budget + w.n_sink + w.n_recent)
            idx = r["idx"][b, h, :n]
            ref_idx, _ = O.select(r["scores"][b, h, :L], w.budget, w.n_sink, w.n_recent)
            assert np.array_equal(idx, ref_idx)
            p = torch.softmax(torch.from_numpy(qs @ k64[b, h, idx].T * sc), 1).numpy()
            assert np.allclose(r["out"][b, h * G:(h + 1) * G], p @ v64[b, h, idx], atol=1e-12)
            pd = torch.softmax(torch.from_numpy(qs @ k64[b, h, :L].T * sc), 1).numpy()
            assert np.allclose(r["dense_out"][b, h * G:(h + 1) * G], pd @ v64[b, h, :L], atol=1e-12)


def test_all_fcs_reproduce_dense_topk():
    # With every FC dominant the selection is the paper's "Oracle" baseline: top-k of the full logits.
    w, t = _small_workload(n_dom=64, n_sink=0, n_recent=0)
    r = O.decode_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"]),
                      t["seq_lens"].numpy(), t["dom"].numpy(), budget=w.budget, want_dense=False)
    G = w.group
    for b in range(w.batch):
        L = int(t["seq_lens"][b])
        for h in range(w.n_kv_heads):
            full = (t["k"][b, h, :L].double() @ t["q"][b, h * G:(h + 1) * G].double().T).sum(1)
            ref = torch.topk(full, w.budget).indices.sort().values.numpy()
            assert np.array_equal(r["idx"][b, h, :w.budget], ref)


def test_budget_covering_context_reproduces_dense():
    w, t = _small_workload()
    r = O.decode_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"]),
                      t["seq_lens"].numpy(), t["dom"].numpy(), n_sink=w.n_sink, n_recent=w.n_recent,
                      budget=w.max_len)
    assert np.array_equal(r["n_sel"], np.repeat(t["seq_lens"].numpy()[:, None], w.n_kv_heads, 1))
    assert np.allclose(r["out"], r["dense_out"], atol=1e-14)
    # permille budget: ceil(0.189 L) in integers
    r2 = O.decode_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"]),
                       t["seq_lens"].numpy(), t["dom"].numpy(), budget=-189, want_dense=False)
    for b in range(w.batch):
        L = int(t["seq_lens"][b])
        assert int(r2["n_sel"][b, 0]) == math.ceil(189 * L / 1000)


# --------------------------------------------- index sets per query head ----

def _decode(w, t, **kw):
    return O.decode_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"]),
                         t["seq_lens"].numpy(), t["dom"].numpy(), n_sink=w.n_sink, n_recent=w.n_recent,
                         budget=w.budget, **kw)


@pytest.mark.parametrize("sel_heads", [1, 2])
def test_sets_per_query_head_equal_the_model_with_repeated_kv_heads(sel_heads):
    # Sec. 4.1 keeps one index set per head.  Sets shared by sel_heads query heads of a
    # grouped-query model must be what the default path (one set per KV head, pinned above)
    # gives on the same model with every K/V head repeated once per set: this fixes which
    # cache a unit reads, which query heads it covers and where its rows land.
    w, t = _small_workload()
    rep = w.group // sel_heads
    r = _decode(w, t, sel_heads=sel_heads)
    x = O.decode_bf16(synth.bf16_bits(t["q"]), np.repeat(synth.bf16_bits(t["k"]), rep, axis=1),
                      np.repeat(synth.bf16_bits(t["v"]), rep, axis=1), t["seq_lens"].numpy(),
                      np.repeat(t["dom"].numpy(), rep, axis=0), n_sink=w.n_sink, n_recent=w.n_recent,
                      budget=w.budget)
    assert r["idx"].shape == (w.batch, w.n_q_heads // sel_heads, w.max_len)
    for key in ("scores", "idx", "n_sel", "band", "out", "lse", "dense_out", "dense_lse"):
        assert np.array_equal(r[key], x[key], equal_nan=True), key
    # the dense output does not depend on how sets are shared; the sparse one does
    d = _decode(w, t)
    assert np.array_equal(r["dense_out"], d["dense_out"])
    assert not np.array_equal(r["out"], d["out"])


def test_sets_per_query_head_all_fcs_reproduce_each_heads_dense_topk():
    w, t = _small_workload(n_dom=64, n_sink=0, n_recent=0)
    r = _decode(w, t, sel_heads=1, want_dense=False)
    G = w.group
    for b in range(w.batch):
        L = int(t["seq_lens"][b])
        for g in range(w.n_q_heads):
            full = t["k"][b, g // G, :L].double() @ t["q"][b, g].double()
            ref = torch.topk(full, w.budget).indices.sort().values.numpy()
            assert np.array_equal(r["idx"][b, g, :w.budget], ref)
            p = torch.softmax(full[ref] / math.sqrt(128), 0)
            assert np.allclose(r["out"][b, g], (p[:, None] * t["v"][b, g // G, ref].double()).sum(0).numpy(), atol=1e-12)


def test_sets_per_query_head_budget_covering_context_reproduces_dense():
    w, t = _small_workload(budget=600)
    r = _decode(w, t, sel_heads=1)
    assert np.array_equal(r["n_sel"], np.repeat(t["seq_lens"].numpy()[:, None], w.n_q_heads, 1))
    assert np.allclose(r["out"], r["dense_out"], atol=1e-14)


def test_set_sharing_must_divide_the_group():
    w, t = _small_workload()
    with pytest.raises(ValueError):
        _decode(w, t, sel_heads=3)
    assert np.array_equal(_decode(w, t, sel_heads=w.group)["idx"], _decode(w, t)["idx"])


# --------------------------------- offline calibration (Algorithm 1, Eq. 4) ----

def test_ca_hand_worked():
    g = GOLD["scores"]
    q, K = np.array(g["q"]), np.array(g["K"])
    for f32 in (False, True):
        assert O.ca_counts(q, K, 2, f32=f32).tolist() == GOLD["ca"]["top2_common"]
        assert O.ca_counts(q, K, 1, f32=f32).tolist() == GOLD["ca"]["top1_common"]


@pytest.mark.parametrize("pairing", [0, 1])
def test_ca_matches_library_topk_and_python_sets(pairing):
    rng = np.random.default_rng(77 + pairing)
    L, d, k = 300, 128, 24
    q, K = rng.standard_normal(d), rng.standard_normal((L, d))
    got = O.ca_counts(q, K, k, pairing)
    full = set(torch.topk(torch.from_numpy(K @ q), k).indices.tolist())
    for i in range(d // 2):
        c0, c1 = (i, i + d // 2) if pairing == 0 else (2 * i, 2 * i + 1)
        a_i = torch.from_numpy(q[c0] * K[:, c0] + q[c1] * K[:, c1])
        assert got[i] == len(full & set(torch.topk(a_i, k).indices.tolist())), i


def test_ca_of_a_query_living_in_one_fc():
    # q is zero outside FC 5: alpha equals alpha^(5) (CA = 1), every other alpha^(i) is all
    # zeros, whose top-k is the first k positions by the tie rule
    rng = np.random.default_rng(5)
    L, d, k = 200, 128, 16
    K = rng.standard_normal((L, d))
    q = np.zeros(d)
    q[5], q[5 + 64] = 1.5, -0.75
    got = O.ca_counts(q, K, k)
    assert got[5] == k
    first = set(range(k))
    top = set(torch.topk(torch.from_numpy(K @ q), k).indices.tolist())
    assert all(got[i] == len(first & top) for i in range(64) if i != 5)


def test_ca_binary32_path_equals_fp64_where_binary32_is_exact():
    # small integers: every product and sum is exact in binary32, so both paths rank alike;
    # many equal scores exercise the tie rule in both
    rng = np.random.default_rng(9)
    q = rng.integers(-3, 4, 128).astype(np.float64)
    K = rng.integers(-3, 4, (150, 128)).astype(np.float64)
    assert np.array_equal(O.ca_counts(q, K, 20, f32=True), O.ca_counts(q, K, 20, f32=False))


def test_calibration_batch_accumulates_samples_and_skips_short_sequences():
    w = synth.CONFIGS["c1"].replace(batch=3, max_len=400, len_lo=100, len_hi=400)
    t = synth.make_inputs(w, "cpu")
    t["seq_lens"] = torch.tensor([400, 32, 257], dtype=torch.int32)          # the middle one is too short for top-32
    qb, kb = synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"])
    counts, used = O.calibrate_bf16(qb, kb, t["seq_lens"].numpy(), 32, f32=False, n_threads=2)
    assert used.tolist() == [2] * w.n_q_heads
    q64, k64 = t["q"].double().numpy(), t["k"].double().numpy()
    for g in (0, 13, 31):
        want = sum(O.ca_counts(q64[b, g], k64[b, g // w.group, :L], 32) for b, L in ((0, 400), (2, 257)))
        assert np.array_equal(counts[g], want)
    # a second call adds to the same arrays
    O.calibrate_bf16(qb, kb, t["seq_lens"].numpy(), 32, f32=False, counts=counts, n_used=used)
    assert used.tolist() == [4] * w.n_q_heads and np.array_equal(counts[13] // 2, counts[13] - counts[13] // 2)
    assert counts.max() <= 4 * 32 and counts.min() >= 0


def test_select_dominant_ranks_group_means_with_lower_index_first():
    counts = np.zeros((4, 64), dtype=np.int64)                # 2 KV heads x 2 query heads
    used = np.array([3, 1, 2, 2], dtype=np.int64)
    counts[0, [7, 9, 20]] = [30, 10, 12]
    counts[1, [9, 20, 40]] = [20, 18, 5]                      # KV head 0 sums: FC 7: 30, 9: 30, 20: 30, 40: 5
    counts[2, 63] = 8
    counts[3, [0, 63]] = [8, 1]                               # KV head 1 sums: FC 63: 9, 0: 8
    dom, mean = O.select_dominant(counts, used, 2, top_k=10, n_dom=2)
    assert dom.tolist() == [[7, 9], [0, 63]]                  # three-way tie keeps the two lowest indices
    assert math.isclose(mean[0, 7], 30 / (4 * 10)) and math.isclose(mean[1, 63], 9 / (4 * 10)) and mean[0, 1] == 0.0
    order = np.argsort(-counts[:2].sum(0), kind="stable")[:3]
    assert sorted(order.tolist()) == O.select_dominant(counts, used, 2, 10, 3)[0][0].tolist()


def test_calibration_recovers_planted_dominant_fcs():
    # keys and queries whose energy sits in three FCs: those FCs decide the ranking, so their
    # CA is the highest and Algorithm 1 returns exactly them
    rng = np.random.default_rng(11)
    B, Hq, Hkv, L, d = 2, 4, 2, 500, 128
    planted = [3, 17, 40]
    scale = np.ones(d)
    for i in planted:
        scale[[i, i + 64]] = 12.0
    q = torch.from_numpy(rng.standard_normal((B, Hq, d)) * scale).to(torch.bfloat16)
    K = torch.from_numpy(rng.standard_normal((B, Hkv, L, d)) * scale).to(torch.bfloat16)
    counts, used = O.calibrate_bf16(synth.bf16_bits(q), synth.bf16_bits(K), np.array([L, L - 37], dtype=np.int32), 50)
    dom, mean = O.select_dominant(counts, used, Hkv, 50, 3)
    assert dom.tolist() == [planted, planted]
    assert mean[:, planted].min() > 1.5 * np.delete(mean, planted, axis=1).max()


def _batched_case(seed, B=2, T=4, Hq=4, Hkv=2, L=90, F=6, budget=11, n_sink=1, n_recent=3):
    rng = np.random.default_rng(seed)
    q = torch.from_numpy(rng.standard_normal((B, T, Hq, 128))).to(torch.bfloat16)
    k = torch.from_numpy(rng.standard_normal((B, Hkv, L, 128))).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((B, Hkv, L, 128))).to(torch.bfloat16)
    lens = np.array([L, L - 17][:B], dtype=np.int32)
    dom = np.stack([np.sort(rng.choice(64, F, replace=False)) for _ in range(Hkv)]).astype(np.int32)
    return q, k, v, lens, dom, dict(budget=budget, n_sink=n_sink, n_recent=n_recent)


def test_batched_queries_with_one_token_are_the_decode_step():
    from paper_2602_03152_b200 import synth
    q, k, v, lens, dom, kw = _batched_case(3, T=1)
    a = O.decode_batched_bf16(synth.bf16_bits(q), synth.bf16_bits(k), synth.bf16_bits(v), lens, dom, **kw)
    b = O.decode_bf16(synth.bf16_bits(q[:, 0]), synth.bf16_bits(k), synth.bf16_bits(v), lens, dom, **kw)
    for key in ("scores", "idx", "n_sel", "out", "lse", "dense_out"):
        assert np.array_equal(a[key][:, 0], b[key], equal_nan=True), key


def test_batched_queries_against_the_masked_dense_formulation():
    # The same block computed the way a dense framework would: ONE matrix product of all T queries
    # against the dominant channels of the keys, a causal mask over the block (the query whose own
    # key sits at cache row L - T + t sees rows <= that one), library top-k on the masked scores,
    # then ONE masked scaled-dot-product attention over all rows with a boolean mask holding the T
    # index sets.  Sink and recent positions are relative to each query's own visible range.
    from paper_2602_03152_b200 import synth
    q, k, v, lens, dom, kw = _batched_case(4)
    B, T, Hq = q.shape[:3]
    Hkv, G = k.shape[1], q.shape[2] // k.shape[1]
    r = O.decode_batched_bf16(synth.bf16_bits(q), synth.bf16_bits(k), synth.bf16_bits(v), lens, dom, **kw)
    q64, k64, v64 = q.double(), k.double(), v.double()
    for b in range(B):
        L = int(lens[b])
        for h in range(Hkv):
            ch = np.concatenate([dom[h], dom[h] + 64])
            qsum = q64[b, :, h * G:(h + 1) * G].sum(dim=1)                         # [T,128]: sum over the group
            S = qsum[:, ch] @ k64[b, h, :L][:, ch].T                               # [T,L]
            own = torch.arange(T) + (L - T)                                         # cache row of each query's own key
            visible = torch.arange(L)[None, :] <= own[:, None]
            mask = torch.zeros((T, L), dtype=torch.bool)
            for t in range(T):
                Lt = int(own[t]) + 1
                assert np.allclose(r["scores"][b, t, h, :Lt], S[t, :Lt].numpy(), rtol=1e-12, atol=1e-12)
                forced = torch.zeros(L, dtype=torch.bool)
                forced[:kw["n_sink"]] = True
                forced[Lt - kw["n_recent"]:Lt] = True
                cand = S[t].clone()
                cand[~visible[t] | forced] = -float("inf")
                top = torch.topk(cand, kw["budget"]).indices
                sel = torch.sort(torch.cat([torch.nonzero(forced).flatten(), top])).values
                n = int(r["n_sel"][b, t, h])
                assert n == kw["budget"] + kw["n_sink"] + kw["n_recent"]
                assert np.array_equal(r["idx"][b, t, h, :n], sel.numpy()), (b, h, t)
                mask[t, sel] = True
            for g in range(G):
                hq = h * G + g
                o = torch.nn.functional.scaled_dot_product_attention(q64[b, :, hq][None], k64[b, h, :L][None], v64[b, h, :L][None],
                                                                     attn_mask=mask[None])[0]
                assert np.allclose(r["out"][b, :, hq], o.numpy(), rtol=1e-11, atol=1e-12)
            # the last query of the block is the ordinary decode step on the whole cache
    last = O.decode_bf16(synth.bf16_bits(q[:, -1]), synth.bf16_bits(k), synth.bf16_bits(v), lens, dom, **kw)
    assert np.array_equal(r["idx"][:, -1], last["idx"]) and np.array_equal(r["out"][:, -1], last["out"])


def test_batched_queries_do_not_see_later_keys_of_their_block():
    # planting a huge key at the block's last position changes the last query's result only
    from paper_2602_03152_b200 import synth
    q, k, v, lens, dom, kw = _batched_case(5, B=1, T=3, n_recent=0)
    base = O.decode_batched_bf16(synth.bf16_bits(q), synth.bf16_bits(k), synth.bf16_bits(v), lens, dom, **kw)
    k2, v2 = k.clone(), v.clone()
    k2[0, :, int(lens[0]) - 1] *= 50.0
    v2[0, :, int(lens[0]) - 1] += 7.0
    moved = O.decode_batched_bf16(synth.bf16_bits(q), synth.bf16_bits(k2), synth.bf16_bits(v2), lens, dom, **kw)
    assert np.array_equal(base["out"][:, :2], moved["out"][:, :2]) and np.array_equal(base["idx"][:, :2], moved["idx"][:, :2])
    assert not np.array_equal(base["out"][:, 2], moved["out"][:, 2])


def test_byte_model_of_the_benchmark():
    # bench.step_bytes is the denominator of every reported roofline fraction.  Sec. 4.4: the
    # fraction of the KV cache that a step loads is N_tip/d + N_fac/t (N_tip counted in FCs of
    # two channels each, d = 128 channels); q and out are the only other terms.  Checked
    # against that closed form and against the configuration's byte counts worked by hand.
    import bench
    from paper_2602_03152_b200 import synth
    for name, lens, n_sel_unit in (("c1", [32768], 324), ("c4", [65536] * 8, 256), ("c2", [65536 + 977 * b for b in range(16)], 1024),
                                   ("c3", [16384] * 32, 3097)):
        w = synth.CONFIGS[name]
        units = w.batch * w.n_kv_heads
        by = bench.step_bytes(w, lens, n_sel_unit * units)
        qo = w.batch * w.n_q_heads * 128 * (2 + 4)                  # bf16 query in, fp32 output back
        assert by["qo"] == qo and by["fasa"] == by["proxy"] + by["gathered"] + qo
        t_mean = sum(lens) / len(lens)
        frac = (by["fasa"] - qo) / (by["dense"] - qo)
        assert math.isclose(frac, w.n_dom / 128 + n_sel_unit / t_mean, rel_tol=1e-12), name
        assert by["dense"] - qo == sum(lens) * w.n_kv_heads * 2 * 128 * 2       # every K and V row, bf16
    # configuration 1 by hand: 8 units x 32768 tokens x 16 FCs x 4 bytes of proxy, 8 x 324 rows of 512 bytes, q + out
    by = bench.step_bytes(synth.CONFIGS["c1"], [32768], 8 * 324)
    assert (by["proxy"], by["gathered"], by["qo"], by["fasa"]) == (16777216, 1327104, 24576, 18128896)
    assert by["dense"] == 134217728 + 24576
    # index sets per query head gather more rows but stream the proxy once per KV head
    w1 = synth.CONFIGS["c4"].replace(sel_heads=1)
    b1 = bench.step_bytes(w1, [65536] * 8, 256 * 8 * 32)
    assert b1["proxy"] == bench.step_bytes(synth.CONFIGS["c4"], [65536] * 8, 0)["proxy"] and b1["gathered"] == 256 * 256 * 512
