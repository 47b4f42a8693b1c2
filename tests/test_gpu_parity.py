"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle, element by
element on the same seeded bf16 inputs.  Index sets are bit-exact outside a 1e-3-relative
tie band; attention is within max-abs 2e-3; scores within 1e-5 of sum |q_c k_c|."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import fasa_oracle as O
from oracle import parity
from paper_2602_03152_b200 import binding, synth

from gpu_harness import SENTINEL, Run

pytestmark = pytest.mark.gpu

C = synth.CONFIGS


def _full_check(r: Run, budget=None, dense=True):
    """Checks the three separate calls against the oracle, then the one-launch step (where the
    configuration has one) against the oracle and against the separate calls."""
    r.build_proxy()
    if dense:
        r.dense_step()
    first = None
    for fused in (False, True):
        assert r.fasa.step_cluster_size() > 0
        r.reset_outputs()
        r.step(budget, fused=fused)
        h = r.host()
        rep = parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                                n_sel=h["n_sel"], out=h["out"], dense_out=h["dense"] if dense and not fused else None,
                                what=r.w.name + (" fused" if fused else ""), **r.oracle_kwargs(budget))
        # rows at and past the sequence length are never written
        for b in range(r.w.batch):
            L = int(h["seq_lens"][b])
            assert np.all(h["scores"][b, :, L:] == SENTINEL)
            for hh in range(r.w.n_sets):
                assert np.all(h["idx"][b, hh, int(h["n_sel"][b, hh]):] == -7)
        assert r.fasa.device_status() == 0
        if not fused:
            first = (rep, h)
        else:
            h0 = first[1]
            assert np.array_equal(h["scores"], h0["scores"]) and np.array_equal(h["idx"], h0["idx"])
            assert np.array_equal(h["n_sel"], h0["n_sel"])
            assert np.abs(h["out"] - h0["out"]).max() <= 1e-4
            fin = np.isfinite(h0["lse"])
            assert np.array_equal(np.isfinite(h["lse"]), fin) and np.abs(h["lse"][fin] - h0["lse"][fin]).max() <= 1e-4
    return first


def test_config0_full_size():
    rep, h = _full_check(Run(C["c0"]))
    assert rep["units"] == 1 and int(h["n_sel"][0, 0]) == 256


def test_config1_shape_scaled_ragged_tail():
    w = C["c1"].replace(max_len=3001, len_lo=2999, len_hi=2999)
    rep, h = _full_check(Run(w))
    assert rep["units"] == 8 and np.all(h["n_sel"] == 256 + 68)


def test_config2_shape_scaled_ragged_batch():
    w = C["c2"].replace(batch=3, max_len=2100, len_lo=500, len_hi=2100, budget=100)
    rep, _ = _full_check(Run(w))
    assert rep["units"] == 24


def test_config3_shape_group_of_7_permille_budget():
    w = C["c3"].replace(batch=2, max_len=1500, len_lo=900, len_hi=1400)
    r = Run(w)
    rep, h = _full_check(r)
    for b in range(2):
        assert np.all(h["n_sel"][b] == math.ceil(189 * int(h["seq_lens"][b]) / 1000))


@pytest.mark.parametrize("F", [1, 3, 4, 5, 8, 13, 32, 64])
def test_dominant_fc_counts(F):
    w = C["c4"].replace(batch=1, max_len=777, len_lo=700, len_hi=700, n_dom=F, budget=64)
    _full_check(Run(w), dense=False)


def test_all_fcs_equal_dense_topk_on_gpu():
    # F = 64: the GPU selection must be the top-k of the full logits (the "Oracle" baseline).
    w = C["c4"].replace(batch=1, max_len=2048, len_lo=2048, len_hi=2048, n_dom=64, budget=128)
    r = Run(w)
    _, h = _full_check(r, dense=False)
    G = w.group
    for hh in range(w.n_kv_heads):
        full = (h["k"][0, hh] @ h["q"][0, hh * G:(hh + 1) * G].T).sum(1)
        ref = np.sort(np.argsort(-full, kind="stable")[:128])
        got = h["idx"][0, hh, :128]
        if not np.array_equal(got, ref):
            parity.check_selection(got, full, 2048, 128, 0, 0, "F=64")


@pytest.mark.parametrize("G,Hkv", [(1, 2), (2, 2), (3, 1), (4, 2), (5, 1), (6, 1), (7, 2), (8, 1)])
def test_group_sizes(G, Hkv):
    w = C["c1"].replace(n_q_heads=G * Hkv, n_kv_heads=Hkv, max_len=900, len_lo=850, len_hi=850, budget=77)
    _full_check(Run(w))


def test_interleaved_pairing_and_max_reduce():
    w = C["c1"].replace(max_len=1000, len_lo=1000, len_hi=1000, pairing=1, budget=50)
    _full_check(Run(w), dense=False)
    w = C["c1"].replace(max_len=1000, len_lo=1000, len_hi=1000, group_reduce=1, budget=50)
    _full_check(Run(w), dense=False)
    w = C["c3"].replace(batch=1, max_len=600, len_lo=600, len_hi=600, group_reduce=1, budget=50)
    _full_check(Run(w), dense=False)


@pytest.mark.parametrize("L,budget,sink,recent", [
    (1, 256, 0, 0), (1, 256, 4, 64), (2, 1, 0, 0), (100, 256, 0, 0), (256, 256, 0, 0), (257, 256, 0, 0),
    (50, 8, 30, 30), (300, 10, 4, 64), (68, 256, 4, 64), (69, 1, 4, 64), (1000, 1, 0, 0), (1000, 999, 0, 0),
])
def test_length_and_budget_edges(L, budget, sink, recent):
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=1024, len_lo=L, len_hi=L, budget=budget,
                        n_sink=sink, n_recent=recent)
    _, h = _full_check(Run(w, n_sel_max=1024))
    assert np.all(h["n_sel"] == min(L, budget + min(L, sink) + min(recent, L - min(L, sink))))


def test_budget_covering_context_equals_dense():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=1500, len_lo=1234, len_hi=1234, budget=1500)
    r = Run(w, n_sel_max=1500)
    _, h = _full_check(r)
    assert np.all(h["n_sel"] == 1234)
    assert np.array_equal(h["idx"][0, 0, :1234], np.arange(1234))
    assert np.abs(h["out"] - h["dense"]).max() <= 2e-5
    assert np.abs(h["lse"] - h["dense_lse"]).max() <= 1e-4


def test_empty_sequence_gives_zero_output():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, batch=2, max_len=256, len_lo=256, len_hi=256, budget=16)
    t = synth.make_inputs(w, "cpu")
    t["seq_lens"] = torch.tensor([0, 200], dtype=torch.int32)
    r = Run(w, t)
    _, h = _full_check(r)
    assert np.all(h["n_sel"][0] == 0) and np.all(h["out"][0] == 0) and np.all(h["dense"][0] == 0)
    assert np.all(np.isneginf(h["lse"][0])) and np.all(np.isneginf(h["dense_lse"][0]))


def test_zero_query_ties_resolve_to_lowest_indices():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=500, len_lo=500, len_hi=500, budget=20, n_sink=0,
                        n_recent=0)
    t = synth.make_inputs(w, "cpu")
    t["q"] = torch.zeros_like(t["q"])
    r = Run(w, t)
    _, h = _full_check(r)
    assert np.array_equal(h["idx"][0, 0, :20], np.arange(20))
    # q = 0: attention is the plain mean of the selected value rows
    assert np.abs(h["out"][0, 0] - h["v"][0, 0, :20].mean(0)).max() <= 2e-3


def test_lse_matches_oracle():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=700, len_lo=700, len_hi=700, budget=90)
    r = Run(w)
    _, h = _full_check(r)
    G = w.group
    for hh in range(2):
        n = int(h["n_sel"][0, hh])
        _, lse = O.attn_subset(h["q"][0, hh * G:(hh + 1) * G], h["k"][0, hh], h["v"][0, hh], h["idx"][0, hh, :n],
                               1 / math.sqrt(128))
        assert np.abs(h["lse"][0, hh * G:(hh + 1) * G] - lse).max() <= 1e-3
        _, dlse = O.attn_dense(h["q"][0, hh * G:(hh + 1) * G], h["k"][0, hh], h["v"][0, hh], 700, 1 / math.sqrt(128))
        assert np.abs(h["dense_lse"][0, hh * G:(hh + 1) * G] - dlse).max() <= 1e-3


def test_results_are_deterministic():
    w = C["c2"].replace(batch=2, max_len=5000, len_lo=3000, len_hi=5000, budget=300)
    r = Run(w)
    r.build_proxy()
    for fused in (False, True):
        r.step(fused=fused); r.dense_step()
        a = [x.clone() for x in (r.scores, r.idx, r.n_sel, r.out, r.dense)]
        r.reset_outputs()
        r.step(fused=fused); r.dense_step()
        for x, y in zip(a, (r.scores, r.idx, r.n_sel, r.out, r.dense)):
            assert torch.equal(x, y)


def test_decode_step_equals_separate_calls_and_host_variant():
    w = C["c1"].replace(max_len=2000, len_lo=1500, len_hi=1500, budget=128)
    r = Run(w)
    r.build_proxy()
    r.step()
    ref = [x.clone() for x in (r.scores, r.idx, r.n_sel, r.out)]
    for x in (r.scores, r.out):
        x.fill_(SENTINEL)
    r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, r.ws)
    torch.cuda.synchronize()
    for x, y in zip(ref[:3], (r.scores, r.idx, r.n_sel)):
        assert torch.equal(x, y)
    assert float((ref[3] - r.out).abs().max()) <= 1e-4      # another split of the rows: fp32 rounding only
    r.fasa.set_step_mode(0)                                  # mode 0 is the three calls themselves
    r.step()
    ref0 = [x.clone() for x in (r.scores, r.idx, r.n_sel, r.out)]
    assert torch.equal(ref0[1], ref[1]) and float((ref0[3] - ref[3]).abs().max()) <= 1e-4
    r.out.fill_(SENTINEL)
    r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, r.ws)
    torch.cuda.synchronize()
    for x, y in zip(ref0, (r.scores, r.idx, r.n_sel, r.out)):
        assert torch.equal(x, y)
    r.fasa.set_step_mode(1)
    # host variant: append one token, then the same step; compare with the oracle on the grown cache
    s = synth.make_step_inputs(w, 0, "cpu")
    stage = torch.empty(r.fasa.stage_bytes(), dtype=torch.uint8, device="cuda")
    out_host = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32).pin_memory()
    r.fasa.decode_step_host(s["q"].pin_memory(), s["k_new"].pin_memory(), s["v_new"].pin_memory(), stage, r.k, r.v,
                            r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, out_host, r.ws)
    assert r.seq_lens.cpu().tolist() == [1501]
    kc, vc = r.k.cpu(), r.v.cpu()
    assert torch.equal(kc[:, :, 1500], s["k_new"][:, :, 0]) and torch.equal(vc[:, :, 1500], s["v_new"][:, :, 0])
    rep = parity.check_step(s["q"].double().numpy(), kc.double().numpy(), vc.double().numpy(), [1501],
                            np.sort(r.dom.numpy(), axis=1), scores=r.scores.cpu().numpy(), idx=r.idx.cpu().numpy(),
                            n_sel=r.n_sel.cpu().numpy(), out=out_host.numpy(), what="host step", **r.oracle_kwargs())
    assert rep["units"] == 8
    assert torch.equal(out_host, r.out.cpu())
    # pageable inputs take the staging copies instead of being read in place: same contract
    s2 = synth.make_step_inputs(w, 1, "cpu")
    out2 = torch.empty((w.batch, w.n_q_heads, 128), dtype=torch.float32)
    r.fasa.decode_step_host(s2["q"], s2["k_new"], s2["v_new"], stage, r.k, r.v, r.proxy, r.seq_lens, w.budget,
                            r.scores, r.idx, r.n_sel, r.out, out2, r.ws)
    assert r.seq_lens.cpu().tolist() == [1502]
    kc, vc = r.k.cpu(), r.v.cpu()
    assert torch.equal(kc[:, :, 1501], s2["k_new"][:, :, 0])
    parity.check_step(s2["q"].double().numpy(), kc.double().numpy(), vc.double().numpy(), [1502],
                      np.sort(r.dom.numpy(), axis=1), scores=r.scores.cpu().numpy(), idx=r.idx.cpu().numpy(),
                      n_sel=r.n_sel.cpu().numpy(), out=out2.numpy(), what="host step, pageable", **r.oracle_kwargs())


@pytest.mark.parametrize("mode", [1, 0])
def test_append_decode_step_equals_append_then_step(mode):
    # ragged batch, group of 7, permille budget; several steps in a row so the per-sequence
    # arrival counter of the one-launch form is reused
    w = C["c3"].replace(batch=3, max_len=1300, len_lo=700, len_hi=1297)
    t = synth.make_inputs(w, "cpu")
    t["seq_lens"] = torch.tensor([700, 1297, 1001], dtype=torch.int32)
    a, b = Run(w, t), Run(w, {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in t.items()})
    for r in (a, b):
        r.fasa.set_step_mode(mode)
        r.build_proxy()
    for step in range(5):
        s = synth.make_step_inputs(w, step, "cuda")
        a.fasa.kv_append(a.k, a.v, a.proxy, a.seq_lens, s["k_new"], s["v_new"])
        a.fasa.decode_step(s["q"], a.k, a.v, a.proxy, a.seq_lens, w.budget, a.scores, a.idx, a.n_sel, a.out, a.ws)
        n0 = b.fasa.launch_count()
        b.fasa.append_decode_step(s["q"], s["k_new"], s["v_new"], b.k, b.v, b.proxy, b.seq_lens, w.budget, b.scores,
                                  b.idx, b.n_sel, b.out, b.ws)
        torch.cuda.synchronize()
        assert b.fasa.launch_count() - n0 == (1 if mode == 1 else 5)
        for x, y in ((a.k, b.k), (a.v, b.v), (a.proxy, b.proxy), (a.seq_lens, b.seq_lens), (a.scores, b.scores),
                     (a.idx, b.idx), (a.n_sel, b.n_sel)):
            assert torch.equal(x, y)
        assert float((a.out - b.out).abs().max()) <= 1e-5
    # sequence 1 filled up after 3 steps: later tokens are dropped and flagged, on both routes
    assert a.seq_lens.cpu().tolist() == [705, 1300, 1006]
    assert a.fasa.device_status() & binding.DEV_APPEND_FULL and b.fasa.device_status() & binding.DEV_APPEND_FULL
    # and the result of the last step agrees with the oracle on the grown cache
    kc, vc = b.k.cpu(), b.v.cpu()
    parity.check_step(s["q"].cpu().double().numpy(), kc.double().numpy(), vc.double().numpy(), [705, 1300, 1006],
                      np.sort(b.dom.numpy(), axis=1), scores=b.scores.cpu().numpy(), idx=b.idx.cpu().numpy(),
                      n_sel=b.n_sel.cpu().numpy(), out=b.out.cpu().numpy(), what="append+step", **b.oracle_kwargs())


def test_select_step_gives_the_index_sets_of_the_separate_calls():
    w = C["c2"].replace(batch=3, max_len=9000, len_lo=4000, len_hi=8999, budget=300, n_sink=2, n_recent=9)
    r = Run(w)
    r.build_proxy()
    r.step()                                                   # fasa_fc_score + fasa_topk + attention
    ref = (r.scores.clone(), r.idx.clone(), r.n_sel.clone())
    r.reset_outputs()
    n0 = r.fasa.launch_count()
    r.fasa.select_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel)
    torch.cuda.synchronize()
    assert r.fasa.launch_count() == n0 + 1
    assert torch.equal(r.scores, ref[0]) and torch.equal(r.idx, ref[1]) and torch.equal(r.n_sel, ref[2])
    assert torch.all(r.out == SENTINEL)                        # no attention ran
    # appending form: the cache's own next row appended again, lengths grow by one
    lens0 = r.seq_lens.clone()
    bi = torch.arange(w.batch, device="cuda")
    k_new = r.k[bi, :, lens0.long()].unsqueeze(2).contiguous()
    v_new = r.v[bi, :, lens0.long()].unsqueeze(2).contiguous()
    r.fasa.select_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, None, r.idx, r.n_sel, k_new, v_new)
    torch.cuda.synchronize()
    assert torch.equal(r.seq_lens, lens0 + 1)
    idx_a, n_a = r.idx.clone(), r.n_sel.clone()
    r.fasa.fc_score(r.q, r.proxy, r.seq_lens, r.scores)
    r.fasa.topk(r.scores, r.seq_lens, w.budget, r.idx, r.n_sel, r.ws)
    torch.cuda.synchronize()
    assert torch.equal(r.idx, idx_a) and torch.equal(r.n_sel, n_a)
    assert r.fasa.device_status() == 0
    with pytest.raises(binding.FasaError):                     # k_new without v_new
        r.fasa.select_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, None, r.idx, r.n_sel, k_new, None)


# ------------------------------------------------------------------ blocks of queries ----

def _batched_run(w, T, budget=None, seed=0):
    """Runs fasa_decode_step_batched on a block of T queries per sequence and checks every (sequence,
    query) pair against the oracle: query t sees the rows up to its own position."""
    r = Run(w)
    r.build_proxy()
    budget = w.budget if budget is None else budget
    B, Hq, Hs, Lm = w.batch, w.n_q_heads, w.n_sets, w.max_len
    q = torch.stack([synth.make_step_inputs(w.replace(index=w.index + seed), 40 + t, "cuda")["q"] for t in range(T)], dim=1).contiguous()
    scores = torch.full((B, T, Hs, Lm), SENTINEL, dtype=torch.float32, device="cuda")
    idx = torch.full((B, T, Hs, r.n_sel_max), -7, dtype=torch.int32, device="cuda")
    n_sel = torch.full((B, T, Hs), -7, dtype=torch.int32, device="cuda")
    out = torch.full((B, T, Hq, 128), SENTINEL, dtype=torch.float32, device="cuda")
    lse = torch.full((B, T, Hq), SENTINEL, dtype=torch.float32, device="cuda")
    r.fasa.decode_step_batched(q, r.k, r.v, r.proxy, r.seq_lens, budget, scores, idx, n_sel, out, r.ws, lse)
    torch.cuda.synchronize()
    assert r.fasa.device_status() == 0
    h = r.host()
    qh = q.cpu().double().numpy()
    for t in range(T):
        lens_t = np.maximum(h["seq_lens"] - (T - 1 - t), 0)
        parity.check_step(qh[:, t], h["k"], h["v"], lens_t, h["dom"], scores=scores[:, t].cpu().numpy(), idx=idx[:, t].cpu().numpy(),
                          n_sel=n_sel[:, t].cpu().numpy(), out=out[:, t].cpu().numpy(), what=f"{w.name} query {t} of {T}",
                          **r.oracle_kwargs(budget))
        for b in range(B):                       # rows at and past what the query sees are never written
            assert torch.all(scores[b, t, :, int(lens_t[b]):] == SENTINEL)
    return r, q, scores, idx, n_sel, out, lse


@pytest.mark.parametrize("T", [1, 2, 4, 8])
def test_batched_queries_match_the_oracle(T):
    w = C["c1"].replace(batch=2, max_len=3000, len_lo=1500, len_hi=2999, budget=100, n_sink=2, n_recent=5)
    r, q, scores, idx, n_sel, out, lse = _batched_run(w, T)
    if T == 1:
        # one query per block: the single-query calls on the same inputs (scores up to the
        # rounding order of the fp32 accumulation, everything after them the same kernels)
        r.q = q[:, 0].contiguous()
        r.step()
        assert torch.allclose(scores[:, 0], r.scores, rtol=0, atol=2e-4 * float(r.scores[r.scores != SENTINEL].abs().max()))
        assert float((out[:, 0] - r.out).abs().max()) <= 1e-3


@pytest.mark.parametrize("cfg,kw,T", [
    ("c3", dict(batch=2, max_len=2000, len_lo=900, len_hi=1999, budget=-150), 8),          # group of 7 x 8 queries = 56 columns, no RoPE
    ("c1", dict(batch=1, n_q_heads=8, n_kv_heads=1, max_len=1500, len_lo=1500, len_hi=1500, budget=64), 8),   # 8 x 8 = 64 columns
    ("c1", dict(batch=2, max_len=1000, len_lo=3, len_hi=999, n_dom=3, budget=40), 3),     # one 8-channel block, padded K
    ("c1", dict(batch=1, max_len=2500, len_lo=2400, len_hi=2400, n_dom=5, budget=40, pairing=1), 5),   # odd chunk count
    ("c1", dict(batch=1, max_len=2100, len_lo=2100, len_hi=2100, n_dom=64, budget=77), 2),  # all FCs: 8 blocks of 16 channels
    ("c1", dict(batch=2, max_len=1300, len_lo=600, len_hi=1300, n_dom=13, budget=50, group_reduce=1), 4),   # max over the group
    ("c4", dict(batch=2, n_q_heads=8, n_kv_heads=2, max_len=1800, len_lo=700, len_hi=1800, budget=33, sel_heads=1), 6),   # a set per head
])
def test_batched_queries_shapes(cfg, kw, T):
    _batched_run(C[cfg].replace(**kw), T)


def test_batched_queries_on_paged_caches_equal_the_contiguous_results():
    # a block of 4 queries after a 4-token append, page pools in random order: the batched calls read
    # the proxy and the K/V rows through the block table and must give the contiguous bits
    w = C["c1"].replace(batch=2, max_len=2000, len_lo=700, len_hi=1900, budget=60, n_sink=1, n_recent=4)
    t = synth.make_inputs(w, "cpu")
    P, T = 64, 4
    r, f, kp, vp, tab, table, need = _paged_twin(w, t, P, extra_tokens=T)
    proxy_p, lens_p = f.alloc_proxy(), r.seq_lens.clone()
    r.build_proxy()
    f.proxy_build(kp, proxy_p, lens_p)
    g = torch.Generator().manual_seed(4)
    kn = torch.randn((w.batch, w.n_kv_heads, T, 128), generator=g).to(torch.bfloat16).cuda()
    vn = torch.randn((w.batch, w.n_kv_heads, T, 128), generator=g).to(torch.bfloat16).cuda()
    r.fasa.kv_append(r.k, r.v, r.proxy, r.seq_lens, kn, vn)
    f.kv_append(kp, vp, proxy_p, lens_p, kn, vn)
    q = torch.stack([synth.make_step_inputs(w, 70 + j, "cuda")["q"] for j in range(T)], dim=1).contiguous()
    B, Hq, Hs, Lm = w.batch, w.n_q_heads, w.n_sets, w.max_len
    res = []
    for fa, k, v, px, ln in ((r.fasa, r.k, r.v, r.proxy, r.seq_lens), (f, kp, vp, proxy_p, lens_p)):
        scores = torch.full((B, T, Hs, Lm), SENTINEL, dtype=torch.float32, device="cuda")
        idx = torch.full((B, T, Hs, r.n_sel_max), -7, dtype=torch.int32, device="cuda")
        n_sel = torch.full((B, T, Hs), -7, dtype=torch.int32, device="cuda")
        out = torch.full((B, T, Hq, 128), SENTINEL, dtype=torch.float32, device="cuda")
        fa.decode_step_batched(q, k, v, px, ln, w.budget, scores, idx, n_sel, out, r.ws)
        torch.cuda.synchronize()
        assert fa.device_status() == 0
        res.append((scores, idx, n_sel, out))
    for x, y in zip(*res):
        assert torch.equal(x, y)
    # and the contiguous run against the oracle, on the grown caches
    kh, vh = r.k.cpu().double().numpy(), r.v.cpu().double().numpy()
    lens = r.seq_lens.cpu().numpy()
    for tq in range(T):
        parity.check_step(q[:, tq].cpu().double().numpy(), kh, vh, np.maximum(lens - (T - 1 - tq), 0), np.sort(r.dom.numpy(), axis=1),
                          scores=res[0][0][:, tq].cpu().numpy(), idx=res[0][1][:, tq].cpu().numpy(), n_sel=res[0][2][:, tq].cpu().numpy(),
                          out=res[0][3][:, tq].cpu().numpy(), what=f"paged block, query {tq}", **r.oracle_kwargs())


def test_batched_queries_reject_what_they_cannot_take():
    w = C["c1"].replace(batch=1, n_q_heads=16, n_kv_heads=1, max_len=600, len_lo=600, len_hi=600)   # 16 heads per set? no: group 16 > 8
    w = C["c3"].replace(batch=1, max_len=600, len_lo=600, len_hi=600)
    r = Run(w)
    r.build_proxy()
    for T in (9, 0):
        q = torch.zeros((1, max(T, 1), w.n_q_heads, 128), dtype=torch.bfloat16, device="cuda")
        st = r.fasa._lib.fasa_fc_score_batched(r.fasa._h, q.data_ptr(), r.proxy.data_ptr(), r.seq_lens.data_ptr(), T,
                                               r.scores.data_ptr(), None)
        assert st == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert r.fasa.device_status() == 0


def test_large_selection_is_attended_by_the_split_k_kernel():
    # n_sel_max * ceil(G / 4) >= 2048 and a workspace: cluster kernel without its attention
    # phase, then the split-K tensor-core attention whose splits merge inside their own cluster
    # (2 launches); same results as one launch
    w = C["c3"].replace(batch=2, max_len=6000, len_lo=5000, len_hi=6000, budget=-300)
    r = Run(w)
    r.build_proxy()
    r.step(fused=True)                       # no workspace: one launch
    one = [x.clone() for x in (r.scores, r.idx, r.n_sel, r.out, r.lse)]
    r.reset_outputs()
    n0 = r.fasa.launch_count()
    r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, r.ws, r.lse)
    torch.cuda.synchronize()
    assert r.fasa.launch_count() - n0 == 2
    for x, y in zip(one[:3], (r.scores, r.idx, r.n_sel)):
        assert torch.equal(x, y)
    assert float((one[3] - r.out).abs().max()) <= 1e-4 and float((one[4] - r.lse).abs().max()) <= 1e-4
    h = r.host()
    parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                      n_sel=h["n_sel"], out=h["out"], what="split attention", **r.oracle_kwargs())
    assert r.fasa.device_status() == 0


# ---- index sets shared by fewer query heads than a KV head serves (Sec. 4.1: a set per head) ----

@pytest.mark.parametrize("cfg,sel,kw", [
    ("c1", 1, dict(max_len=3001, len_lo=2999, len_hi=2999)),                        # 32 sets of one head
    ("c1", 2, dict(batch=2, max_len=2100, len_lo=900, len_hi=2100)),                # 16 sets of two heads
    ("c3", 1, dict(batch=2, max_len=1500, len_lo=900, len_hi=1400)),                # group of 7, permille budget
    ("c0", 1, dict()),                                                              # config 0 at full size
    ("c1", 1, dict(max_len=1200, len_lo=1100, len_hi=1200, group_reduce=1, pairing=1, n_dom=5)),
])
def test_index_sets_per_query_head(cfg, sel, kw):
    w = C[cfg].replace(sel_heads=sel, **kw)
    rep, h = _full_check(Run(w))
    assert rep["units"] == w.batch * w.n_q_heads // sel
    assert h["idx"].shape[1] == w.n_q_heads // sel


def test_index_sets_per_query_head_equal_the_model_with_repeated_kv_heads():
    # the same statement as the oracle's pin, on the GPU: bit-exact scores and sets, both routes
    w = C["c1"].replace(batch=2, max_len=2000, len_lo=1500, len_hi=2000, sel_heads=1)
    t = synth.make_inputs(w, "cpu")
    x = dict(t)
    x["k"], x["v"] = t["k"].repeat_interleave(w.group, dim=1), t["v"].repeat_interleave(w.group, dim=1)
    x["dom"] = t["dom"].repeat_interleave(w.group, dim=0)
    a, b = Run(w, t), Run(w.replace(n_kv_heads=w.n_q_heads, sel_heads=0), x)
    for fused in (False, True):
        for r in (a, b):
            r.build_proxy()
            r.reset_outputs()
            r.step(fused=fused)
        for u, v in ((a.scores, b.scores), (a.idx, b.idx), (a.n_sel, b.n_sel), (a.out, b.out), (a.lse, b.lse)):
            assert torch.equal(u, v)


@pytest.mark.parametrize("mode", [1, 0])
def test_index_sets_per_query_head_append_form(mode):
    # several sets share a KV head: each cluster of the one-launch form writes the new rows itself
    w = C["c3"].replace(batch=3, max_len=1300, len_lo=700, len_hi=1297, sel_heads=1)
    t = synth.make_inputs(w, "cpu")
    t["seq_lens"] = torch.tensor([700, 1299, 1001], dtype=torch.int32)
    a, b = Run(w, t), Run(w, {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in t.items()})
    for r in (a, b):
        r.fasa.set_step_mode(mode)
        r.build_proxy()
    for step in range(3):
        s = synth.make_step_inputs(w, step, "cuda")
        a.fasa.kv_append(a.k, a.v, a.proxy, a.seq_lens, s["k_new"], s["v_new"])
        a.fasa.decode_step(s["q"], a.k, a.v, a.proxy, a.seq_lens, w.budget, a.scores, a.idx, a.n_sel, a.out, a.ws)
        n0 = b.fasa.launch_count()
        b.fasa.append_decode_step(s["q"], s["k_new"], s["v_new"], b.k, b.v, b.proxy, b.seq_lens, w.budget, b.scores,
                                  b.idx, b.n_sel, b.out, b.ws)
        torch.cuda.synchronize()
        assert b.fasa.launch_count() - n0 == (1 if mode == 1 else 5)
        for u, v in ((a.k, b.k), (a.v, b.v), (a.proxy, b.proxy), (a.seq_lens, b.seq_lens), (a.scores, b.scores),
                     (a.idx, b.idx), (a.n_sel, b.n_sel)):
            assert torch.equal(u, v)
        assert float((a.out - b.out).abs().max()) <= 1e-5
    assert a.seq_lens.cpu().tolist() == [703, 1300, 1004]
    parity.check_step(s["q"].cpu().double().numpy(), b.k.cpu().double().numpy(), b.v.cpu().double().numpy(),
                      [703, 1300, 1004], np.sort(b.dom.numpy(), axis=1), scores=b.scores.cpu().numpy(),
                      idx=b.idx.cpu().numpy(), n_sel=b.n_sel.cpu().numpy(), out=b.out.cpu().numpy(),
                      what="append+step, sets per head", **b.oracle_kwargs())


def test_index_sets_per_query_head_large_selection_and_static_scratch():
    # one head per set: the split route starts at n_sel_max >= 2048; the no-workspace variant agrees
    w = C["c1"].replace(batch=1, n_q_heads=8, n_kv_heads=2, max_len=6000, len_lo=5000, len_hi=6000, budget=2500,
                        sel_heads=1)
    r = Run(w)
    r.build_proxy()
    n0 = r.fasa.launch_count()
    r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, r.ws, r.lse)
    torch.cuda.synchronize()
    assert r.fasa.launch_count() - n0 == 2
    h = r.host()
    parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                      n_sel=h["n_sel"], out=h["out"], what="split attention, sets per head", **r.oracle_kwargs())
    out2 = torch.full_like(r.out, SENTINEL)
    r.fasa.sparse_decode_attn_static(r.q, r.k, r.v, r.idx, r.n_sel, out2)
    torch.cuda.synchronize()
    assert torch.equal(out2, r.out)
    assert r.fasa.device_status() == 0


# ---- offline calibration (Algorithm 1; CA of Eq. 4): integer counts, bit-exact ----

def _calib(w, t, top_k, calls=1):
    f = binding.Fasa.from_workload(w, t["dom"])
    q, k, lens = t["q"].cuda(), t["k"].cuda(), t["seq_lens"].cuda()
    counts = torch.zeros((w.n_q_heads, 64), dtype=torch.int64, device="cuda")
    used = torch.zeros(w.n_q_heads, dtype=torch.int64, device="cuda")
    ws = torch.empty(f.calib_workspace_bytes(top_k), dtype=torch.uint8, device="cuda")
    for _ in range(calls):
        n0 = f.launch_count()
        f.calib_accumulate(q, k, lens, top_k, counts, used, ws)
        assert f.launch_count() == n0 + 3
    torch.cuda.synchronize()
    assert f.device_status() == 0
    c_or, u_or = O.calibrate_bf16(synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), t["seq_lens"].numpy(), top_k,
                                  pairing=w.pairing, f32=True)
    return counts.cpu().numpy(), used.cpu().numpy(), c_or, u_or


@pytest.mark.parametrize("cfg,kw,top_k", [
    ("c0", dict(), 256),                                                            # config 0 at full size
    ("c1", dict(batch=2, max_len=3001, len_lo=1500, len_hi=3001), 100),            # ragged, tail tile
    ("c3", dict(batch=2, max_len=1500, len_lo=900, len_hi=1400), 33),              # group of 7, no RoPE
    ("c1", dict(batch=1, max_len=2048, len_lo=2048, len_hi=2048, pairing=1), 1),   # interleaved pairing, top-1
    ("c1", dict(batch=1, n_q_heads=4, n_kv_heads=1, max_len=20000, len_lo=20000, len_hi=20000), 4096),
])
def test_calibration_counts_match_the_oracle(cfg, kw, top_k):
    w = C[cfg].replace(**kw)
    t = synth.make_inputs(w, "cpu")
    counts, used, c_or, u_or = _calib(w, t, top_k)
    assert np.array_equal(used, u_or) and used.min() >= 1
    assert np.array_equal(counts, c_or)
    assert counts.max() <= used.max() * top_k


def test_calibration_counts_against_the_fp64_statement_of_eq4():
    # The bit-exact test above decides set membership in binary32, as the kernel does.  Against the
    # plain fp64 statement of Eq. 4 the count of a (query head, FC) pair may differ only through
    # positions whose score lies within 1e-3 (relative) of the K-th score of the full-score list or
    # of that FC's list: those are the only memberships a rounding can flip.
    w = C["c1"].replace(batch=1, n_q_heads=8, n_kv_heads=2, max_len=3000, len_lo=3000, len_hi=3000)
    t = synth.make_inputs(w, "cpu")
    top_k = 100
    counts, used, _, _ = _calib(w, t, top_k)
    q64, k64 = t["q"].double().numpy(), t["k"].double().numpy()

    def band(s):
        o = np.sort(s)[::-1]
        tol = 1e-3 * max(abs(o[top_k - 1]), abs(o[top_k]))
        return int(np.sum(np.abs(s - o[top_k - 1]) <= tol)) - 1          # the K-th position itself cannot flip alone

    worst = 0
    for hq in range(w.n_q_heads):
        K = k64[0, hq // w.group, :3000]
        c64 = O.ca_counts(q64[0, hq], K, top_k, w.pairing, f32=False)
        a = O.fc_partial_logits(q64[0, hq], K, w.pairing)                 # [64][L]
        b_full = band(a.sum(axis=0))
        for i in range(64):
            slack = b_full + band(a[i])
            assert abs(int(counts[hq, i]) - int(c64[i])) <= slack, (hq, i, counts[hq, i], c64[i], slack)
            worst = max(worst, abs(int(counts[hq, i]) - int(c64[i])))
    assert used.tolist() == [1] * w.n_q_heads and worst <= 3


def test_calibration_accumulates_and_skips_short_sequences():
    w = C["c1"].replace(batch=3, n_q_heads=8, n_kv_heads=2, max_len=700, len_lo=100, len_hi=700)
    t = synth.make_inputs(w, "cpu")
    t["seq_lens"] = torch.tensor([700, 64, 0], dtype=torch.int32)      # 64 == top_k and 0: not samples
    counts, used, c_or, u_or = _calib(w, t, 64, calls=2)
    assert used.tolist() == [2] * 8 and np.array_equal(counts, 2 * c_or) and np.array_equal(u_or, [1] * 8)


def test_calibration_end_to_end_recovers_planted_fcs_and_feeds_create():
    # the planted-energy case of the oracle's pin, on the GPU, through Stage 2 into fasa_create
    rng = np.random.default_rng(11)
    w = C["c1"].replace(batch=2, n_q_heads=4, n_kv_heads=2, max_len=500, len_lo=500, len_hi=500, n_dom=3)
    planted = [3, 17, 40]
    scale = np.ones(128)
    for i in planted:
        scale[[i, i + 64]] = 12.0
    t = {"q": torch.from_numpy(rng.standard_normal((2, 4, 128)) * scale).to(torch.bfloat16),
         "k": torch.from_numpy(rng.standard_normal((2, 2, 500, 128)) * scale).to(torch.bfloat16),
         "seq_lens": torch.tensor([500, 463], dtype=torch.int32), "dom": torch.tensor([[0, 1, 2], [0, 1, 2]], dtype=torch.int32)}
    counts, used, c_or, u_or = _calib(w, t, 50)
    assert np.array_equal(counts, c_or) and np.array_equal(used, u_or)
    dom, mean = binding.calib_select(torch.from_numpy(counts), torch.from_numpy(used), 2, 50, 3)
    assert dom.tolist() == [planted, planted]
    assert np.array_equal(dom.numpy(), O.select_dominant(c_or, u_or, 2, 50, 3)[0])
    binding.Fasa.from_workload(w, dom).close()


def test_calibration_rejects_what_it_cannot_take():
    w = C["c1"].replace(batch=32, max_len=512, len_lo=512, len_hi=512)           # 32 * 32 * 65 > 65535 grid rows
    f = binding.Fasa.from_workload(w, synth.dominant_fcs(w))
    with pytest.raises(binding.FasaError) as e:
        f.calib_workspace_bytes(16)
    assert e.value.status == binding.ERR_UNSUPPORTED
    g = binding.Fasa.from_workload(w.replace(batch=1), synth.dominant_fcs(w))
    for bad in (0, 513, -3):
        with pytest.raises(binding.FasaError):
            g.calib_workspace_bytes(bad)


def test_decode_loop_replays_from_a_cuda_graph():
    # a serving loop captures its steps once and replays them: three append+step calls (one
    # launch each) and a dense call in one graph; nothing in a call allocates or synchronises,
    # and the lengths advance on the device, so a replay continues where the last one ended
    w = C["c1"].replace(batch=2, max_len=1200, len_lo=700, len_hi=1100)
    t = synth.make_inputs(w, "cpu")
    eager, graphed = Run(w, t), Run(w, {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in t.items()})
    steps = [synth.make_step_inputs(w, i, "cuda") for i in range(3)]
    outs_e = [torch.zeros_like(eager.out) for _ in steps]
    outs_g = [torch.zeros_like(eager.out) for _ in steps]
    for r in (eager, graphed):
        r.build_proxy()
    torch.cuda.synchronize()

    def run(r, outs):
        for s_, o in zip(steps, outs):
            r.fasa.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], r.k, r.v, r.proxy, r.seq_lens, w.budget,
                                      None, r.idx, r.n_sel, o, None)
        r.fasa.full_decode_attn(steps[-1]["q"], r.k, r.v, r.seq_lens, r.dense, r.ws)

    g = torch.cuda.CUDAGraph()
    n0 = graphed.fasa.launch_count()
    with torch.cuda.graph(g):
        run(graphed, outs_g)
    assert graphed.fasa.launch_count() - n0 == 3 + 1          # (the dense pass of this size merges inside its clusters)
    for rounds in range(2):
        g.replay()
        run(eager, outs_e)
        torch.cuda.synchronize()
        for x, y in ((eager.k, graphed.k), (eager.v, graphed.v), (eager.proxy, graphed.proxy),
                     (eager.seq_lens, graphed.seq_lens), (eager.idx, graphed.idx), (eager.n_sel, graphed.n_sel),
                     (eager.dense, graphed.dense)):
            assert torch.equal(x, y)
        for x, y in zip(outs_e, outs_g):
            assert torch.equal(x, y)
    assert graphed.seq_lens.cpu().tolist() == [int(l) + 6 for l in t["seq_lens"].tolist()]
    assert graphed.fasa.device_status() == 0


def test_fasa_m_caches_in_pinned_host_memory():
    # Algorithm 2 (the memory-optimised variant): only the dominant part of the key cache - the
    # proxy - lives on the GPU; K and V sit in page-locked host memory, the attention kernels
    # fetch the selected rows over the host link and the append calls store new rows there.
    # Same kernels, same bits: every result must equal the device-resident run exactly.
    w = C["c3"].replace(batch=2, max_len=3000, len_lo=1400, len_hi=2900)
    t = synth.make_inputs(w, "cpu")
    dev = Run(w, t, n_sel_max=1300)
    host = Run(w, {k_: (v_.clone() if torch.is_tensor(v_) else v_) for k_, v_ in t.items()}, n_sel_max=1300)
    kh, vh = host.fasa.alloc_host_cache(), host.fasa.alloc_host_cache()
    assert kh.is_pinned() and not kh.is_cuda
    kh.copy_(t["k"]); vh.copy_(t["v"])
    host.k, host.v = kh, vh
    for r in (dev, host):
        r.build_proxy()                                        # Split of the whole cache, read over the link
    assert torch.equal(dev.proxy, host.proxy)
    bulk = synth.make_step_inputs(w.replace(index=w.index + 5), 0, "cuda")
    kb, vb = bulk["k_new"].repeat(1, 1, 3, 1).contiguous(), bulk["v_new"].repeat(1, 1, 3, 1).contiguous()
    for r in (dev, host):
        r.fasa.kv_append(r.k, r.v, r.proxy, r.seq_lens, kb, vb)           # three rows at once
    for step, ws in enumerate((None, "ws", None)):             # one launch / split-K route / one launch
        s = synth.make_step_inputs(w, step, "cuda")
        for r in (dev, host):
            r.fasa.append_decode_step(s["q"], s["k_new"], s["v_new"], r.k, r.v, r.proxy, r.seq_lens, -400 if ws else w.budget,
                                      r.scores, r.idx, r.n_sel, r.out, r.ws if ws else None, r.lse)
        torch.cuda.synchronize()
        for x, y in ((dev.proxy, host.proxy), (dev.seq_lens, host.seq_lens), (dev.scores, host.scores),
                     (dev.idx, host.idx), (dev.n_sel, host.n_sel), (dev.out, host.out), (dev.lse, host.lse)):
            assert torch.equal(x, y)
    host.dense_step(); dev.dense_step()
    assert torch.equal(dev.dense, host.dense)
    # the host tensors themselves now hold the appended rows
    assert torch.equal(dev.k.cpu(), kh) and torch.equal(dev.v.cpu(), vh)
    lens = dev.seq_lens.cpu().tolist()
    assert lens == [int(l) + 6 for l in t["seq_lens"].tolist()]
    parity.check_step(s["q"].cpu().double().numpy(), kh.double().numpy(), vh.double().numpy(), lens,
                      np.sort(host.dom.numpy(), axis=1), scores=host.scores.cpu().numpy(), idx=host.idx.cpu().numpy(),
                      n_sel=host.n_sel.cpu().numpy(), out=host.out.cpu().numpy(),
                      what="caches in host memory", **host.oracle_kwargs())
    assert host.fasa.device_status() == 0


@pytest.mark.parametrize("cfg,kw,budget", [
    ("c3", dict(batch=2, max_len=3000, len_lo=1400, len_hi=2900), -150),                     # group of 7: one pass over the link
    ("c1", dict(batch=2, max_len=2500, len_lo=900, len_hi=2400, n_dom=8, pairing=1), 200),  # sinks and recent rows, 8 FCs
    ("c4", dict(batch=1, n_q_heads=8, n_kv_heads=2, max_len=1900, len_lo=1890, len_hi=1890, n_dom=32), 64),
])
def test_fasa_m_split_key_cache(cfg, kw, budget):
    # Algorithm 2 as stated: the dominant channels of the keys stay on the GPU (the proxy), the other
    # channels and the values live in page-locked host memory; Split on append, Combine in the
    # attention kernel.  Layout bit for bit, index sets equal to the whole-row path, outputs against
    # the oracle and within fp32 rounding of the whole-row path (same products, another order).
    w = C[cfg].replace(**kw)
    r = Run(w)
    r.build_proxy()
    f = r.fasa
    knd, vh = f.alloc_host_nondom(), f.alloc_host_cache()
    assert knd.is_pinned() and knd.shape[-1] == 128 - 2 * w.n_dom
    vh.copy_(r.t["v"])
    f.m_split(r.k, knd, r.seq_lens)
    torch.cuda.synchronize()
    dom = np.sort(r.dom.numpy(), axis=1)
    lens = r.t["seq_lens"].tolist()
    for b in range(w.batch):
        for h in range(w.n_kv_heads):
            d = np.concatenate([dom[h], dom[h] + 64]) if w.pairing == 0 else np.concatenate([2 * dom[h], 2 * dom[h] + 1])
            rest = np.setdiff1d(np.arange(128), d)                     # ascending
            L = lens[b]
            assert torch.equal(knd[b, h, :L], r.t["k"][b, h, :L][:, torch.from_numpy(rest)])
            assert torch.all(knd[b, h, L:] == 0)
    # one appended token through Split + UpdateCache, against the whole-row append
    s = synth.make_step_inputs(w, 2, "cuda")
    proxy2, lens2 = r.proxy.clone(), r.seq_lens.clone()
    f.m_kv_append(knd, vh, proxy2, lens2, s["k_new"], s["v_new"])
    f.kv_append(r.k, r.v, r.proxy, r.seq_lens, s["k_new"], s["v_new"])
    torch.cuda.synchronize()
    assert torch.equal(proxy2, r.proxy) and torch.equal(lens2, r.seq_lens) and torch.equal(vh, r.v.cpu())
    knd_ref = f.alloc_host_nondom()
    f.m_split(r.k, knd_ref, r.seq_lens)
    torch.cuda.synchronize()
    assert torch.equal(knd, knd_ref)
    # the step: whole-row path on the device, split path over the link
    r.reset_outputs()
    r.fasa.decode_step(s["q"], r.k, r.v, r.proxy, r.seq_lens, budget, r.scores, r.idx, r.n_sel, r.out, None, r.lse)
    ref = [x.clone() for x in (r.scores, r.idx, r.n_sel, r.out, r.lse)]
    r.reset_outputs()
    n0 = f.launch_count()
    f.m_decode_step(s["q"], knd, vh, proxy2, lens2, budget, r.scores, r.idx, r.n_sel, r.out, r.ws, r.lse)
    torch.cuda.synchronize()
    assert f.launch_count() - n0 == 2 and f.device_status() == 0
    assert torch.equal(r.scores, ref[0]) and torch.equal(r.idx, ref[1]) and torch.equal(r.n_sel, ref[2])
    assert float((r.out - ref[3]).abs().max()) <= 1e-4
    h = r.host()
    parity.check_step(s["q"].cpu().double().numpy(), r.k.cpu().double().numpy(), r.v.cpu().double().numpy(), r.seq_lens.cpu().numpy(),
                      h["dom"], idx=h["idx"], n_sel=h["n_sel"], out=h["out"], what="split key cache", **r.oracle_kwargs(budget))
    # appending form of the step (Algorithm 2's loop body): equals append + step
    s3 = synth.make_step_inputs(w, 3, "cuda")
    f.kv_append(r.k, r.v, r.proxy, r.seq_lens, s3["k_new"], s3["v_new"])
    f.decode_step(s3["q"], r.k, r.v, r.proxy, r.seq_lens, budget, None, r.idx, r.n_sel, r.out, None)
    ref_idx, ref_out = r.idx.clone(), r.out.clone()
    f.m_decode_step(s3["q"], knd, vh, proxy2, lens2, budget, None, r.idx, r.n_sel, r.out, r.ws, None, s3["k_new"], s3["v_new"])
    torch.cuda.synchronize()
    assert torch.equal(lens2, r.seq_lens) and torch.equal(r.idx, ref_idx) and float((r.out - ref_out).abs().max()) <= 1e-4


def _resident_expect(w, dom_sorted_h, k_rows, v_rows):
    """Rows of the resident buffer for the given K / V rows [n][128] of one KV head."""
    if w.pairing == 0:
        c0, c1 = dom_sorted_h, dom_sorted_h + 64
    else:
        c0, c1 = 2 * dom_sorted_h, 2 * dom_sorted_h + 1
    rest = np.setdiff1d(np.arange(128), np.concatenate([c0, c1]))
    pairs = np.stack([c0, c1], axis=1).reshape(-1)                    # proxy order: (c0, c1) per dominant FC, ascending
    kk = torch.cat([k_rows[:, torch.from_numpy(rest)], k_rows[:, torch.from_numpy(pairs)]], dim=1)
    return torch.stack([kk, v_rows], dim=1)                            # [n][2][128]


def _check_resident(w, f, buf, dom, k_dev, v_dev, lens):
    S, Sp = w.n_sink + w.n_recent, (w.n_sink + w.n_recent + 3) & ~3
    units = w.batch * w.n_kv_heads
    tags = buf[:units * Sp * 4].view(torch.int32).view(units, Sp).cpu()
    rows = buf[units * Sp * 4:].view(torch.bfloat16).view(units, S, 2, 128).cpu()
    dom_sorted = np.sort(dom.numpy(), axis=1)
    for b in range(w.batch):
        L = int(lens[b])
        want = sorted(set(range(min(w.n_sink, L))) | set(range(max(w.n_sink, L - w.n_recent), L)))
        for h in range(w.n_kv_heads):
            u = b * w.n_kv_heads + h
            held = sorted(int(x) for x in tags[u, :S] if x >= 0)
            assert held == want, (b, h, L)
            for s_ in range(S):
                pos = int(tags[u, s_])
                if pos < 0:
                    continue
                assert s_ == (pos if pos < w.n_sink else w.n_sink + (pos - w.n_sink) % w.n_recent)
                exp = _resident_expect(w, dom_sorted[h], k_dev[b, h, pos:pos + 1].cpu(), v_dev[b, h, pos:pos + 1].cpu())[0]
                assert torch.equal(rows[u, s_], exp), (b, h, s_, pos)


@pytest.mark.parametrize("kw,budget", [
    (dict(batch=2, max_len=2500, len_lo=900, len_hi=2400), 200),                          # 16 FCs, 4 sinks + 64 recent
    (dict(batch=3, max_len=700, len_lo=20, len_hi=640, n_dom=8, pairing=1, n_sink=3, n_recent=30), 40),   # a sequence shorter than the window
])
def test_fasa_m_resident_forced_rows(kw, budget):
    # The sink positions and the recent window are part of every selection: with a resident buffer
    # they stay on the GPU (a slot per position, tagged) and never cross the host link.  The buffer
    # holds exactly those rows after a build, after single appends and after a bulk append; the
    # step's results do not change bit for bit; and they still do not change when the host copies
    # of those rows are overwritten with garbage, which shows where the kernel reads them.
    w = C["c1"].replace(**kw)
    r = Run(w)
    r.build_proxy()
    f = r.fasa
    knd, vh = f.alloc_host_nondom(), f.alloc_host_cache()
    vh.copy_(r.t["v"])
    f.m_split(r.k, knd, r.seq_lens)
    s = synth.make_step_inputs(w, 5, "cuda")
    r.reset_outputs()
    f.m_decode_step(s["q"], knd, vh, r.proxy, r.seq_lens, budget, None, r.idx, r.n_sel, r.out, r.ws, r.lse)
    ref = [x.clone() for x in (r.idx, r.n_sel, r.out, r.lse)]
    assert f._lib.fasa_m_resident_bytes(f._h) == w.batch * w.n_kv_heads * (((w.n_sink + w.n_recent + 3) & ~3) * 4 + (w.n_sink + w.n_recent) * 512)
    buf = f.alloc_resident()
    f.m_resident_build(knd, vh, r.proxy, r.seq_lens)
    torch.cuda.synchronize()
    _check_resident(w, f, buf, r.dom, r.k, r.v, r.seq_lens.tolist())

    def poison_host(lens):
        for b in range(w.batch):
            L = int(lens[b])
            for lo, hi in ((0, min(w.n_sink, L)), (max(w.n_sink, L - w.n_recent), L)):
                knd[b, :, lo:hi] = float("nan")
                vh[b, :, lo:hi] = float("nan")

    for poisoned in (False, True):
        if poisoned:
            poison_host(r.seq_lens.tolist())
        r.reset_outputs()
        f.m_decode_step(s["q"], knd, vh, r.proxy, r.seq_lens, budget, None, r.idx, r.n_sel, r.out, r.ws, r.lse)
        torch.cuda.synchronize()
        assert f.device_status() == 0
        for x, y in zip((r.idx, r.n_sel, r.out, r.lse), ref):
            assert torch.equal(x, y), poisoned
    vh.copy_(r.v)                                  # (the host copies whole again: those rows leave the window below)
    f.m_split(r.k, knd, r.seq_lens)
    torch.cuda.synchronize()
    # three single appends through the step, then a bulk append longer than the window; the whole-row
    # device caches follow with the ordinary calls and give the reference
    lens2 = r.seq_lens.clone()
    for i in range(3):
        si = synth.make_step_inputs(w, 10 + i, "cuda")
        f.kv_append(r.k, r.v, r.proxy.clone(), r.seq_lens, si["k_new"], si["v_new"])          # (device caches + lengths)
        f.m_decode_step(si["q"], knd, vh, r.proxy, lens2, budget, None, r.idx, r.n_sel, r.out, r.ws, None, si["k_new"], si["v_new"])
        torch.cuda.synchronize()
        assert torch.equal(lens2, r.seq_lens)
        _check_resident(w, f, buf, r.dom, r.k, r.v, lens2.tolist())
    room = w.max_len - int(r.seq_lens.max())
    n_bulk = min(room, w.n_recent + 37)
    if n_bulk > 0:
        g = torch.Generator(device="cuda").manual_seed(77)
        kb = torch.randn(w.batch, w.n_kv_heads, n_bulk, 128, device="cuda", generator=g).to(torch.bfloat16)
        vb = torch.randn(w.batch, w.n_kv_heads, n_bulk, 128, device="cuda", generator=g).to(torch.bfloat16)
        f.kv_append(r.k, r.v, r.proxy.clone(), r.seq_lens, kb, vb)
        f.m_kv_append(knd, vh, r.proxy, lens2, kb, vb)
        torch.cuda.synchronize()
        assert torch.equal(lens2, r.seq_lens)
        _check_resident(w, f, buf, r.dom, r.k, r.v, lens2.tolist())
    poison_host(lens2.tolist())
    s9 = synth.make_step_inputs(w, 9, "cuda")
    r.reset_outputs()
    f.decode_step(s9["q"], r.k, r.v, r.proxy, r.seq_lens, budget, None, r.idx, r.n_sel, r.out, None)
    ref_idx, ref_out = r.idx.clone(), r.out.clone()
    r.reset_outputs()
    f.m_decode_step(s9["q"], knd, vh, r.proxy, lens2, budget, None, r.idx, r.n_sel, r.out, r.ws, None)
    torch.cuda.synchronize()
    assert f.device_status() == 0 and torch.equal(r.idx, ref_idx)
    assert bool(torch.isfinite(r.out).all()) and float((r.out - ref_out).abs().max()) <= 1e-4
    # switched off again: the poisoned host rows are read, which the outputs show
    f.m_set_resident(None)
    f.m_decode_step(s9["q"], knd, vh, r.proxy, lens2, budget, None, r.idx, r.n_sel, r.out, r.ws, None)
    torch.cuda.synchronize()
    assert not float((r.out - ref_out).abs().max()) <= 1e-2     # (NaN logits: the kernel writes zeros, or NaN)


def test_fasa_m_resident_needs_forced_positions():
    w = C["c4"].replace(batch=1, n_q_heads=8, n_kv_heads=2, max_len=600, len_lo=600, len_hi=600)
    r = Run(w)
    assert w.n_sink + w.n_recent == 0 and r.fasa._lib.fasa_m_resident_bytes(r.fasa._h) == 0
    buf = torch.zeros(1 << 12, dtype=torch.uint8, device="cuda")
    assert r.fasa._lib.fasa_m_set_resident(r.fasa._h, buf.data_ptr(), None) == binding.ERR_UNSUPPORTED


def test_fasa_m_split_needs_whole_chunks():
    w = C["c1"].replace(batch=1, max_len=600, len_lo=600, len_hi=600, n_dom=6)
    r = Run(w)
    assert r.fasa._lib.fasa_m_nondom_row_elems(6) == 0 and r.fasa._lib.fasa_m_nondom_row_elems(16) == 96
    buf = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    st = r.fasa._lib.fasa_m_split(r.fasa._h, r.k.data_ptr(), buf.data_ptr(), r.seq_lens.data_ptr(), None)
    assert st == binding.ERR_UNSUPPORTED


def _random_workloads(n, seed):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        hkv = int(rng.integers(1, 4))
        g = int(rng.choice([1, 2, 3, 4, 6, 7, 8]))
        sel = int(rng.choice([d for d in range(1, g + 1) if g % d == 0]))
        lm = int(rng.integers(40, 5000))
        lo = int(rng.integers(1, lm + 1))
        budget = int(rng.integers(1, lm + 50)) if rng.random() < 0.7 else -int(rng.integers(1, 1001))
        out.append(C["c1"].replace(index=100 + i, batch=int(rng.integers(1, 4)), n_q_heads=hkv * g, n_kv_heads=hkv,
                                   max_len=lm, len_lo=lo, len_hi=lm, n_dom=int(rng.integers(1, 65)), budget=budget,
                                   n_sink=int(rng.integers(0, 9)), n_recent=int(rng.integers(0, 70)),
                                   pairing=int(rng.integers(0, 2)), group_reduce=int(rng.integers(0, 2)),
                                   sel_heads=0 if sel == g else sel, rope=bool(rng.integers(0, 2))))
    return out


@pytest.mark.parametrize("w", _random_workloads(int(os.environ.get("FASA_RANDOM_CASES", "24")), 20260203),
                         ids=lambda w: f"i{w.index}")
def test_seeded_random_configurations(w):
    # shapes nobody picked by hand: heads, group, set sharing, lengths, F, budget form, forced
    # positions, pairing and reduction all drawn at random (seeded)
    rep, h = _full_check(Run(w))
    assert rep["units"] == w.batch * w.n_sets


# ---- paged caches: page pools + a block table; every call must give the contiguous results ----

def _paged_twin(w, t, P, spare=3, seed=0, extra_tokens=0):
    """A contiguous Run and a paged context over the same logical caches, pages in random order;
    logical pages past what a sequence needs (its length + extra_tokens) stay unmapped (-1)."""
    r = Run(w, t)
    B, Hkv, Lm = w.batch, w.n_kv_heads, w.max_len
    pps = (Lm + P - 1) // P
    need = [min(pps, (int(l) + extra_tokens + P - 1) // P) for l in t["seq_lens"].tolist()]
    n_pages = sum(need) + spare
    perm = torch.randperm(n_pages, generator=torch.Generator().manual_seed(seed)).tolist()
    table = torch.full((B, pps), -1, dtype=torch.int32)
    it = iter(perm)
    for b in range(B):
        for lp in range(need[b]):
            table[b, lp] = next(it)
    f = binding.Fasa(B, w.n_q_heads, Hkv, Lm, t["dom"], rope_pairing=w.pairing, group_reduce=w.group_reduce,
                     n_sink=w.n_sink, n_recent=w.n_recent, select_heads=w.sel_heads, page_size=P, n_pages=n_pages)
    assert f.step_cluster_size() == r.fasa.step_cluster_size() > 0
    kp, vp = f.alloc_paged_cache(), f.alloc_paged_cache()
    pad = pps * P - Lm
    kl = torch.nn.functional.pad(t["k"], (0, 0, 0, pad)).view(B, Hkv, pps, P, 128)
    vl = torch.nn.functional.pad(t["v"], (0, 0, 0, pad)).view(B, Hkv, pps, P, 128)
    for b in range(B):
        for lp in range(need[b]):
            kp[table[b, lp]] = kl[b, :, lp].cuda()
            vp[table[b, lp]] = vl[b, :, lp].cuda()
    tab = table.cuda()
    f.set_block_table(tab)
    return r, f, kp, vp, tab, table, need


def _logical(pool, table, need, P, Lm):
    """[B, Hkv, Lm, ...] view of a page pool through the block table (unmapped pages read as zero)."""
    B, pps = table.shape
    out = torch.zeros((B, pool.shape[1], pps * P) + tuple(pool.shape[3:]), dtype=pool.dtype, device=pool.device)
    for b in range(B):
        for lp in range(need[b]):
            out[b, :, lp * P:(lp + 1) * P] = pool[table[b, lp]]
    return out[:, :, :Lm]


@pytest.mark.parametrize("P,cfg,kw", [
    (16, "c1", dict(batch=2, max_len=1000, len_lo=300, len_hi=990)),
    (64, "c3", dict(batch=3, max_len=2100, len_lo=500, len_hi=2000)),
    (256, "c1", dict(batch=2, max_len=3001, len_lo=1500, len_hi=2990, n_dom=5, pairing=1, sel_heads=1)),
])
def test_paged_caches_give_the_contiguous_results(P, cfg, kw):
    w = C[cfg].replace(**kw)
    t = synth.make_inputs(w, "cpu")
    r, f, kp, vp, tab, table, need = _paged_twin(w, t, P, extra_tokens=45)
    Lm = w.max_len
    proxy_p = f.alloc_proxy()
    lens_p = r.seq_lens.clone()
    # Split of the whole cache
    r.build_proxy()
    f.proxy_build(kp, proxy_p, lens_p)
    tiles = (Lm + 15) // 16
    lp_proxy = _logical(proxy_p.view(f.n_pages, w.n_kv_heads, P // 16, -1), table, need, P // 16, tiles)
    assert torch.equal(lp_proxy, r.proxy)
    # a bulk append (40 rows) and single-token appends that cross page boundaries
    g = torch.Generator().manual_seed(9)
    kn = torch.randn((w.batch, w.n_kv_heads, 40, 128), generator=g).to(torch.bfloat16).cuda()
    vn = torch.randn((w.batch, w.n_kv_heads, 40, 128), generator=g).to(torch.bfloat16).cuda()
    r.fasa.kv_append(r.k, r.v, r.proxy, r.seq_lens, kn, vn)
    f.kv_append(kp, vp, proxy_p, lens_p, kn, vn)
    for i in range(5):
        r.fasa.kv_append(r.k, r.v, r.proxy, r.seq_lens, kn[:, :, i:i + 1].contiguous(), vn[:, :, i:i + 1].contiguous())
        f.kv_append(kp, vp, proxy_p, lens_p, kn[:, :, i:i + 1].contiguous(), vn[:, :, i:i + 1].contiguous())
    torch.cuda.synchronize()
    assert torch.equal(lens_p, r.seq_lens)
    lens = r.seq_lens.cpu().tolist()
    kl, vl = _logical(kp, table, need, P, Lm), _logical(vp, table, need, P, Lm)
    for b, L in enumerate(lens):
        assert torch.equal(kl[b, :, :L], r.k[b, :, :L]) and torch.equal(vl[b, :, :L], r.v[b, :, :L])
    lp_proxy = _logical(proxy_p.view(f.n_pages, w.n_kv_heads, P // 16, -1), table, need, P // 16, tiles)
    for b, L in enumerate(lens):
        assert torch.equal(lp_proxy[b, :, :L // 16], r.proxy[b, :, :L // 16])
    # the three calls, the composite step, the dense path, the append form and the calibration
    out_p, lse_p = torch.zeros_like(r.out), torch.zeros_like(r.lse)
    scores_p, idx_p, n_sel_p = torch.full_like(r.scores, SENTINEL), torch.full_like(r.idx, -7), torch.zeros_like(r.n_sel)
    r.step()
    f.fc_score(r.q, proxy_p, lens_p, scores_p)
    f.topk(scores_p, lens_p, w.budget, idx_p, n_sel_p, r.ws)
    f.sparse_decode_attn(r.q, kp, vp, idx_p, n_sel_p, out_p, r.ws, lse_p)
    torch.cuda.synchronize()
    for x, y in ((scores_p, r.scores), (idx_p, r.idx), (n_sel_p, r.n_sel), (out_p, r.out), (lse_p, r.lse)):
        assert torch.equal(x, y)
    out3 = torch.zeros_like(out_p)
    f.sparse_decode_attn_static(r.q, kp, vp, idx_p, n_sel_p, out3)
    r.dense_step()
    dense_p = torch.zeros_like(r.dense)
    f.full_decode_attn(r.q, kp, vp, lens_p, dense_p, r.ws)
    torch.cuda.synchronize()
    assert torch.equal(out3, out_p) and torch.equal(dense_p, r.dense)
    # the one-launch step (no workspace) and the select + split-K route (large bound, workspace)
    out2 = torch.zeros_like(out_p)
    for ws_, launches in ((None, 1), (r.ws, None)):
        r.reset_outputs()
        scores_p.fill_(SENTINEL); idx_p.fill_(-7)
        n0, m0 = f.launch_count(), r.fasa.launch_count()
        f.decode_step(r.q, kp, vp, proxy_p, lens_p, w.budget, scores_p, idx_p, n_sel_p, out2, ws_)
        r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, ws_)
        torch.cuda.synchronize()
        assert f.launch_count() - n0 == r.fasa.launch_count() - m0 == (launches or f.launch_count() - n0)
        for x, y in ((scores_p, r.scores), (idx_p, r.idx), (n_sel_p, r.n_sel), (out2, r.out)):
            assert torch.equal(x, y)
    # the append form, one launch on both sides, then once more as separate kernels (mode 0)
    for mode in (1, 0):
        s_ = synth.make_step_inputs(w, 1 + mode, "cuda")
        for ff in (r.fasa, f):
            ff.set_step_mode(mode)
        n0 = f.launch_count()
        r.fasa.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores,
                                  r.idx, r.n_sel, r.out, r.ws if mode == 0 else None)
        f.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], kp, vp, proxy_p, lens_p, w.budget, scores_p, idx_p,
                             n_sel_p, out2, r.ws if mode == 0 else None)
        torch.cuda.synchronize()
        assert f.launch_count() - n0 == (1 if mode == 1 else 5)
        for x, y in ((lens_p, r.seq_lens), (scores_p, r.scores), (idx_p, r.idx), (n_sel_p, r.n_sel), (out2, r.out)):
            assert torch.equal(x, y)
    for ff in (r.fasa, f):
        ff.set_step_mode(1)
    if w.batch * w.n_q_heads * 65 <= 65535:
        top_k = 64
        cc = [torch.zeros((w.n_q_heads, 64), dtype=torch.int64, device="cuda") for _ in range(2)]
        uu = [torch.zeros(w.n_q_heads, dtype=torch.int64, device="cuda") for _ in range(2)]
        ws_c = torch.empty(f.calib_workspace_bytes(top_k), dtype=torch.uint8, device="cuda")
        r.fasa.calib_accumulate(r.q, r.k, r.seq_lens, top_k, cc[0], uu[0], ws_c)
        f.calib_accumulate(r.q, kp, lens_p, top_k, cc[1], uu[1], ws_c)
        torch.cuda.synchronize()
        assert torch.equal(cc[0], cc[1]) and torch.equal(uu[0], uu[1]) and int(uu[0].min()) >= 1
    assert f.device_status() == 0 and r.fasa.device_status() == 0
    # and against the oracle, on the logical view of the pools
    h = r.host()
    kl, vl = _logical(kp, table, need, P, Lm), _logical(vp, table, need, P, Lm)
    parity.check_step(s_["q"].cpu().double().numpy(), kl.cpu().double().numpy(), vl.cpu().double().numpy(),
                      lens_p.cpu().numpy(), h["dom"], scores=scores_p.cpu().numpy(), idx=idx_p.cpu().numpy(),
                      n_sel=n_sel_p.cpu().numpy(), out=out2.cpu().numpy(), what="paged", **r.oracle_kwargs())


@pytest.mark.parametrize("w", _random_workloads(int(os.environ.get("FASA_RANDOM_CASES", "24")), 777),
                         ids=lambda w: f"i{w.index}")
def test_seeded_random_configurations_paged(w):
    # the random shapes again, on page pools of a random page size: the one-launch step (with
    # and without a workspace), the three calls and the dense path must equal the contiguous run
    P = [16, 32, 64, 128][w.index % 4]
    t = synth.make_inputs(w, "cpu")
    r, f, kp, vp, tab, table, need = _paged_twin(w, t, P, seed=w.index, extra_tokens=2)     # two appends below
    proxy_p = f.alloc_proxy()
    lens_p = r.seq_lens.clone()
    r.build_proxy()
    f.proxy_build(kp, proxy_p, lens_p)
    s_ = synth.make_step_inputs(w, 0, "cuda")
    scores_p, idx_p, n_sel_p = torch.full_like(r.scores, SENTINEL), torch.full_like(r.idx, -7), torch.zeros_like(r.n_sel)
    out_p, dense_p = torch.zeros_like(r.out), torch.zeros_like(r.dense)
    for ws_ in (None, r.ws):
        r.fasa.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], r.k, r.v, r.proxy, r.seq_lens, w.budget, r.scores, r.idx,
                                  r.n_sel, r.out, ws_)
        f.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], kp, vp, proxy_p, lens_p, w.budget, scores_p, idx_p, n_sel_p,
                             out_p, ws_)
        torch.cuda.synchronize()
        for x, y in ((lens_p, r.seq_lens), (scores_p, r.scores), (idx_p, r.idx), (n_sel_p, r.n_sel), (out_p, r.out)):
            assert torch.equal(x, y)
    r.q = s_["q"]
    r.step()
    f.fc_score(r.q, proxy_p, lens_p, scores_p)
    f.topk(scores_p, lens_p, w.budget, idx_p, n_sel_p, r.ws)
    f.sparse_decode_attn(r.q, kp, vp, idx_p, n_sel_p, out_p, r.ws)
    r.dense_step()
    f.full_decode_attn(r.q, kp, vp, lens_p, dense_p, r.ws)
    torch.cuda.synchronize()
    for x, y in ((scores_p, r.scores), (idx_p, r.idx), (n_sel_p, r.n_sel), (out_p, r.out), (dense_p, r.dense)):
        assert torch.equal(x, y)
    assert f.device_status() == r.fasa.device_status()       # (a full cache flags the dropped token on both sides)


def test_paged_cache_table_errors_are_flagged_not_followed():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=256, len_lo=200, len_hi=200, budget=32)
    t = synth.make_inputs(w, "cpu")
    r, f, kp, vp, tab, table, need = _paged_twin(w, t, 64)
    proxy_p = f.alloc_proxy()
    lens = r.seq_lens.clone()
    f.proxy_build(kp, proxy_p, lens)
    assert f.device_status() == 0
    # a block table must be set before a paged context touches a cache
    g = binding.Fasa(1, 8, 2, 256, t["dom"], page_size=64, n_pages=8)
    with pytest.raises(binding.FasaError):
        g.proxy_build(kp, proxy_p, lens)
    # reads through a bad entry use page 0 and raise the bit; the result stays finite
    tab[0, 1] = 10 ** 6
    f.full_decode_attn(r.q, kp, vp, lens, r.dense, r.ws)
    assert f.device_status() == binding.DEV_PAGE_CLAMPED and torch.isfinite(r.dense).all()
    tab[0, 1] = -1
    f.fc_score(r.q, proxy_p, lens, r.scores)
    assert f.device_status() == binding.DEV_PAGE_CLAMPED
    # writes through a bad entry are dropped: the pools do not change
    lens.fill_(64)
    before = (kp.clone(), vp.clone(), proxy_p.clone())
    s_ = synth.make_step_inputs(w, 0, "cuda")
    f.kv_append(kp, vp, proxy_p, lens, s_["k_new"], s_["v_new"])
    assert f.device_status() == binding.DEV_PAGE_CLAMPED
    assert torch.equal(kp, before[0]) and torch.equal(vp, before[1]) and torch.equal(proxy_p, before[2])
    assert lens.cpu().tolist() == [65]
    # the same through the one-launch append form
    lens.fill_(64)
    f.append_decode_step(s_["q"], s_["k_new"], s_["v_new"], kp, vp, proxy_p, lens, w.budget, None, r.idx, r.n_sel, r.out, None)
    assert f.device_status() & binding.DEV_PAGE_CLAMPED
    assert torch.equal(kp, before[0]) and torch.equal(vp, before[1]) and torch.equal(proxy_p, before[2])
    assert lens.cpu().tolist() == [65] and torch.isfinite(r.out).all()


def test_strided_token_major_cache():
    # K/V stored [B][L][Hkv][128] (token-major), addressed through the stride fields.
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, batch=2, max_len=640, len_lo=400, len_hi=640, budget=40)
    t = synth.make_inputs(w, "cpu")
    r = Run(w, t)
    kt = r.k.permute(0, 2, 1, 3).contiguous()   # [B][L][H][d]
    vt = r.v.permute(0, 2, 1, 3).contiguous()
    st = (640 * 2 * 128, 128, 2 * 128)          # stride_b, stride_h, stride_t in elements
    f = binding.Fasa(w.batch, w.n_q_heads, w.n_kv_heads, w.max_len, r.dom, n_sink=w.n_sink, n_recent=w.n_recent,
                     k_strides=st, v_strides=st)
    proxy = f.alloc_proxy()
    f.proxy_build(kt, proxy, r.seq_lens)
    r.build_proxy()
    assert torch.equal(proxy, r.proxy)
    f.decode_step(r.q, kt, vt, proxy, r.seq_lens, w.budget, r.scores, r.idx, r.n_sel, r.out, r.ws)
    f.full_decode_attn(r.q, kt, vt, r.seq_lens, r.dense, r.ws)
    torch.cuda.synchronize()
    h = r.host()
    parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                      n_sel=h["n_sel"], out=h["out"], dense_out=h["dense"], what="strided", **r.oracle_kwargs())


# ------------------------------------------------------------------ cache update ----

def _expected_proxy(k_bits_cpu, dom_sorted, pairing, row_elems, lens):
    """The documented proxy layout by plain indexing.  Logical row j of a head = the pairs
    (K[j][c0], K[j][c1]) of its sorted dominant FCs, zero padded; tiles of 16 rows; inside a tile
    blocks of 16 channels in tensor-core operand order (lane 4g+t: P[g][2t..2t+1], P[g+8][2t..2t+1],
    P[g][2t+8..2t+9], P[g+8][2t+8..2t+9]), then one block of 8 channels if the chunk count is odd."""
    B, H, Lm, _ = k_bits_cpu.shape
    tiles = (Lm + 15) // 16
    logical = torch.zeros((B, H, tiles * 16, row_elems), dtype=torch.int16)
    for h in range(H):
        for r, i in enumerate(dom_sorted[h].tolist()):
            c0, c1 = (i, i + 64) if pairing == 0 else (2 * i, 2 * i + 1)
            logical[:, h, :Lm, 2 * r] = k_bits_cpu[:, h, :, c0]
            logical[:, h, :Lm, 2 * r + 1] = k_bits_cpu[:, h, :, c1]
    for b in range(B):
        logical[b, :, int(lens[b]):] = 0
    chunks = row_elems // 8
    n16, n8 = chunks // 2, chunks % 2
    out = torch.zeros((B, H, tiles, 16 * row_elems), dtype=torch.int16)
    lg = logical.view(B, H, tiles, 16, row_elems)
    for kb in range(n16):
        for g in range(8):
            for t in range(4):
                base = kb * 256 + (g * 4 + t) * 8                  # in 2-byte elements
                for e, (rr, cc) in enumerate([(g, 2 * t), (g, 2 * t + 1), (g + 8, 2 * t), (g + 8, 2 * t + 1),
                                              (g, 2 * t + 8), (g, 2 * t + 9), (g + 8, 2 * t + 8), (g + 8, 2 * t + 9)]):
                    out[:, :, :, base + e] = lg[:, :, :, rr, kb * 16 + cc]
    if n8:
        for g in range(8):
            for t in range(4):
                base = n16 * 256 + (g * 4 + t) * 4
                for e, (rr, cc) in enumerate([(g, 2 * t), (g, 2 * t + 1), (g + 8, 2 * t), (g + 8, 2 * t + 1)]):
                    out[:, :, :, base + e] = lg[:, :, :, rr, n16 * 16 + cc]
    return out


@pytest.mark.parametrize("F,pairing", [(16, 0), (5, 0), (16, 1), (64, 0), (1, 1), (12, 0), (40, 1)])
def test_proxy_build_layout_is_bit_exact(F, pairing):
    w = C["c2"].replace(batch=2, max_len=300, len_lo=100, len_hi=300, n_dom=F, pairing=pairing)
    r = Run(w)
    r.build_proxy()
    torch.cuda.synchronize()
    exp = _expected_proxy(r.t["k"].view(torch.int16), torch.sort(r.dom, dim=1).values, pairing, r.fasa.row_elems,
                          r.t["seq_lens"])
    assert torch.equal(r.proxy.cpu().view(torch.int16), exp)


def test_kv_append_bulk_then_stepwise():
    w = C["c3"].replace(batch=3, max_len=200, len_lo=0, len_hi=0)
    t = synth.make_inputs(w, "cpu")
    r = Run(w, t)
    src_k, src_v = r.k.clone(), r.v.clone()
    r.k.zero_(); r.v.zero_()
    lens = torch.zeros(3, dtype=torch.int32, device="cuda")
    # bulk prefill of 150 rows, then 20 single-token appends
    r.fasa.kv_append(r.k, r.v, r.proxy, lens, src_k[:, :, :150].contiguous(), src_v[:, :, :150].contiguous())
    for s in range(150, 170):
        r.fasa.kv_append(r.k, r.v, r.proxy, lens, src_k[:, :, s:s + 1].contiguous(), src_v[:, :, s:s + 1].contiguous())
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [170, 170, 170]
    assert torch.equal(r.k[:, :, :170], src_k[:, :, :170]) and torch.equal(r.v[:, :, :170], src_v[:, :, :170])
    assert torch.count_nonzero(r.k[:, :, 170:].view(torch.int16)) == 0
    exp = _expected_proxy(src_k.cpu().view(torch.int16), torch.sort(r.dom, dim=1).values, 0, r.fasa.row_elems,
                          [170, 170, 170])
    assert torch.equal(r.proxy.cpu().view(torch.int16), exp)
    assert r.fasa.device_status() == 0
    # attention over the appended cache agrees with the oracle
    r.seq_lens = lens
    r.t["seq_lens"] = lens.cpu()
    r.t["k"], r.t["v"] = r.k.cpu(), r.v.cpu()
    r.step(); r.dense_step()
    h = r.host()
    parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                      n_sel=h["n_sel"], out=h["out"], dense_out=h["dense"], what="appended", **r.oracle_kwargs())


def test_kv_append_bulk_from_ragged_lengths_and_into_a_full_cache():
    # 40 rows at once onto sequences of different, unaligned lengths; one of them runs out of rows
    w = C["c1"].replace(batch=3, n_q_heads=8, n_kv_heads=2, max_len=120, len_lo=0, len_hi=0, n_dom=13)
    t = synth.make_inputs(w.replace(len_lo=120, len_hi=120), "cpu")
    r = Run(w, t)
    start = [7, 95, 50]
    lens = torch.tensor(start, dtype=torch.int32, device="cuda")
    r.fasa.proxy_build(r.k, r.proxy, lens)
    g = torch.Generator().manual_seed(3)
    kn = torch.randn((3, 2, 40, 128), generator=g).to(torch.bfloat16).cuda()
    vn = torch.randn((3, 2, 40, 128), generator=g).to(torch.bfloat16).cuda()
    k_ref, v_ref = r.k.clone(), r.v.clone()
    r.fasa.kv_append(r.k, r.v, r.proxy, lens, kn, vn)
    torch.cuda.synchronize()
    assert lens.cpu().tolist() == [47, 120, 90]
    assert r.fasa.device_status() == binding.DEV_APPEND_FULL
    for b, (l0, l1) in enumerate(zip(start, [47, 120, 90])):
        k_ref[b, :, l0:l1] = kn[b, :, :l1 - l0]
        v_ref[b, :, l0:l1] = vn[b, :, :l1 - l0]
    assert torch.equal(r.k, k_ref) and torch.equal(r.v, v_ref)
    exp = _expected_proxy(k_ref.cpu().view(torch.int16), torch.sort(r.dom, dim=1).values, 0, r.fasa.row_elems, [47, 120, 90])
    got = r.proxy.cpu().view(torch.int16)
    # rows past the new lengths may hold what the first build left there: compare the live rows
    live = _expected_proxy(torch.ones_like(k_ref.cpu().view(torch.int16)), torch.sort(r.dom, dim=1).values, 0,
                           r.fasa.row_elems, [47, 120, 90]) != 0
    assert torch.equal(got[live], exp[live])


def test_device_status_bits_instead_of_faults():
    w = C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=128, len_lo=128, len_hi=128, budget=16)
    r = Run(w)
    r.build_proxy()
    # cache full: the appended row is dropped, the length stays at max_len
    s = synth.make_step_inputs(w, 0, "cuda")
    r.fasa.kv_append(r.k, r.v, r.proxy, r.seq_lens, s["k_new"], s["v_new"])
    assert r.fasa.device_status() & binding.DEV_APPEND_FULL
    assert r.seq_lens.cpu().tolist() == [128]
    # a length beyond max_len is clamped
    r.seq_lens.fill_(100000)
    for fused in (False, True):
        r.reset_outputs()
        r.step(fused=fused)
        assert r.fasa.device_status() & binding.DEV_LEN_CLAMPED
        assert int(r.n_sel[0, 0]) == 16 + 68
    # an out-of-range index is clamped to row 0, n_sel beyond the list to its capacity
    r.seq_lens.fill_(128)
    r.idx.fill_(10 ** 6)
    r.n_sel.fill_(10 ** 6)
    r.fasa.sparse_decode_attn(r.q, r.k, r.v, r.idx, r.n_sel, r.out, r.ws)
    st = r.fasa.device_status()
    assert st & binding.DEV_IDX_CLAMPED and st & binding.DEV_NSEL_CLAMPED
    assert torch.isfinite(r.out).all()
    # selection larger than the index list: cut to the best n_sel_max
    small = torch.empty((1, 2, 10), dtype=torch.int32, device="cuda")
    r.fasa.topk(r.scores, r.seq_lens, 50, small, r.n_sel, r.ws)
    assert r.fasa.device_status() & binding.DEV_NSEL_CLAMPED
    assert r.n_sel.cpu().tolist() == [[10, 10]]
    assert r.fasa.device_status() == 0
    r.fasa.decode_step(r.q, r.k, r.v, r.proxy, r.seq_lens, 50, None, small, r.n_sel, r.out)
    assert r.fasa.device_status() & binding.DEV_NSEL_CLAMPED
    assert r.n_sel.cpu().tolist() == [[10, 10]]


# ------------------------------------------------------------------ top-k alone ----

def _topk_only(scores_cpu, lens, budget, n_sink, n_recent, n_sel_max, mode=1):
    """mode 1: the cluster kernel's selection phases; mode 0: the register-resident kernel; mode 2: one CTA per row."""
    B, H, Lm = scores_cpu.shape
    dom = torch.arange(4, dtype=torch.int32).repeat(H, 1)
    f = binding.Fasa(B, H, H, Lm, dom, n_sink=n_sink, n_recent=n_recent)
    f.set_step_mode(mode)
    sc = scores_cpu.cuda()
    ln = torch.tensor(lens, dtype=torch.int32, device="cuda")
    idx = torch.full((B, H, n_sel_max), -7, dtype=torch.int32, device="cuda")
    ns = torch.full((B, H), -7, dtype=torch.int32, device="cuda")
    f.topk(sc, ln, budget, idx, ns)
    torch.cuda.synchronize()
    assert f.device_status() == 0
    return idx.cpu().numpy(), ns.cpu().numpy()


def _assert_topk_exact(scores_cpu, lens, budget, n_sink=0, n_recent=0, n_sel_max=None):
    """Given the same fp32 scores, the GPU set equals the oracle's bit for bit, ties included."""
    B, H, Lm = scores_cpu.shape
    n_sel_max = n_sel_max or Lm
    idx, ns = _topk_only(scores_cpu, lens, budget, n_sink, n_recent, n_sel_max, 1)
    for other in (0, 2):                                               # all three kernels, bit for bit
        idx0, ns0 = _topk_only(scores_cpu, lens, budget, n_sink, n_recent, n_sel_max, other)
        assert np.array_equal(idx, idx0) and np.array_equal(ns, ns0), other
    for b in range(B):
        L = lens[b]
        k = budget if budget > 0 else (-budget * L + 999) // 1000
        for h in range(H):
            ref, _ = O.select(scores_cpu[b, h, :L].double().numpy(), k, n_sink, n_recent)
            assert int(ns[b, h]) == ref.size
            assert np.array_equal(idx[b, h, :ref.size], ref), (b, h)


def test_topk_exact_on_heavy_ties():
    g = torch.Generator().manual_seed(5)
    # few distinct values: the k-th rank always falls inside a run of equal scores
    sc = torch.randint(-3, 4, (2, 3, 5000), generator=g).float()
    for budget in (1, 100, 2500, 4999):
        _assert_topk_exact(sc, [5000, 4321], budget)
    _assert_topk_exact(sc, [5000, 4321], 64, n_sink=4, n_recent=64)
    _assert_topk_exact(torch.zeros(1, 2, 3000), [3000], 17)
    _assert_topk_exact(torch.full((1, 2, 3000), -1.5), [2999], -189)


def test_topk_exact_on_crowded_bins():
    # The select phase finishes on the candidates of the k-th key's bin when that bin holds at most
    # 4096 keys cluster-wide.  Scores crowded into one bin of the first pass (same sign, exponent and
    # two leading mantissa bits) take a second cluster pass before the candidates are few enough;
    # scores crowded into one bin of the second pass as well take all three.
    g = torch.Generator().manual_seed(12)
    sc1 = 1.0 + 0.2 * torch.rand((2, 2, 20000), generator=g)                  # one 11-bit bin, ~12 keys per 22-bit bin
    sc2 = 1.0 + 1e-4 * torch.rand((1, 2, 20000), generator=g)                 # one 22-bit bin: every radix pass runs
    sc3 = torch.cat([sc1[:1, :, :10000], -sc1[:1, :, 10000:]], dim=2)         # the crowd split over a positive and a negative bin
    for sc in (sc1, sc2, sc3):
        lens = [20000 - 37 * b for b in range(sc.shape[0])]
        for budget in (1, 300, 4096, 9000, 19990):
            _assert_topk_exact(sc, lens, budget)
        _assert_topk_exact(sc, lens, 500, n_sink=3, n_recent=100)
        _assert_topk_exact(sc, lens, -189)
    # exactly 4096 / 4097 keys in the bin (the capacity of the cluster kernel's candidate area), and
    # 8192 / 8193 (that of the one-CTA-per-row kernel's list), the rest far below
    for n_in in (4096, 4097, 8192, 8193):
        sc = torch.full((1, 1, 30000), -5.0)
        sc[0, 0, torch.randperm(30000, generator=g)[:n_in]] = 1.0 + 0.2 * torch.rand(n_in, generator=g)
        for budget in (1, 2048, n_in - 1, n_in, n_in + 5):
            _assert_topk_exact(sc, [30000], budget)


def test_topk_exact_on_special_values():
    g = torch.Generator().manual_seed(6)
    sc = torch.randn(1, 4, 4096, generator=g)
    sc[0, 0, ::7] = float("inf")
    sc[0, 1, ::5] = float("-inf")
    sc[0, 2, 100:300] = 0.0             # (+0 only: fc_score never emits -0, which would rank below +0)
    sc[0, 3] = sc[0, 3].abs() * 1e-40   # subnormals
    for budget in (10, 600, 3000):
        _assert_topk_exact(sc, [4096], budget)


@pytest.mark.parametrize("L,B,H", [(32768, 1, 8), (131072, 2, 2), (140001, 1, 2), (20000, 3, 5)])
def test_topk_exact_at_scale(L, B, H):
    # 131072 fills the register-resident capacity of an 8-CTA cluster; 140001 takes the
    # streaming fallback; 20000 x 15 units uses small clusters.
    g = torch.Generator().manual_seed(L)
    sc = torch.randn(B, H, L, generator=g) * 40.0
    lens = [L - 13 * b for b in range(B)]
    for budget in (256, 4096):
        _assert_topk_exact(sc, lens, budget, n_sink=4, n_recent=64, n_sel_max=4096 + 68)
    _assert_topk_exact(sc, lens, -189, n_sel_max=(189 * L + 999) // 1000)


# ------------------------------------------------------------------ full sizes ----

def test_config1_full_size():
    rep, h = _full_check(Run(C["c1"]))
    assert rep["units"] == 8 and np.all(h["n_sel"] == 324)


def test_config4_point_full_length_sampled_units():
    # One sweep point at the full 65536 context, batch reduced to keep host memory modest.
    w = C["c4"].replace(batch=2, n_q_heads=16, n_kv_heads=4, budget=2048, n_dom=32)
    r = Run(w)
    r.build_proxy()
    r.dense_step()
    for fused in (False, True):
        r.reset_outputs()
        r.step(fused=fused)
        h = r.host()
        parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], scores=h["scores"], idx=h["idx"],
                          n_sel=h["n_sel"], out=h["out"], dense_out=h["dense"], units=[(0, 0), (1, 3), (1, 1)],
                          what="c4", **r.oracle_kwargs())


def _full_size_sampled(w, units, budget=None, append=False, keep=None):
    """A benchmark workload at its full size, inputs drawn on the device, run as bench.py runs
    it (one fasa_append_decode_step / fasa_decode_step call) and checked against the oracle on
    a few (batch, KV head) units whose K/V are copied to the host."""
    from gpu_harness import ensure_built
    ensure_built()
    t = synth.make_inputs(w, "cuda")
    f = binding.Fasa.from_workload(w, t["dom"])
    B, Hq, Hkv, Lm = w.batch, w.n_q_heads, w.n_kv_heads, w.max_len
    n_sel_max = w.n_sel_max()
    proxy = f.alloc_proxy()
    ws = f.alloc_workspace(n_sel_max)
    idx = torch.full((B, Hkv, n_sel_max), -7, dtype=torch.int32, device="cuda")
    n_sel = torch.full((B, Hkv), -7, dtype=torch.int32, device="cuda")
    out = torch.full((B, Hq, 128), SENTINEL, dtype=torch.float32, device="cuda")
    scores = torch.full((B, Hkv, Lm), SENTINEL, dtype=torch.float32, device="cuda")
    lens = t["seq_lens"].clone()
    q, k, v = t["q"], t["k"], t["v"]
    if append:
        lens -= 1                                    # the step appends the cache's own last row again
        bi = torch.arange(B, device="cuda")
        k_new = k[bi, :, lens.long()].unsqueeze(2).contiguous()
        v_new = v[bi, :, lens.long()].unsqueeze(2).contiguous()
        f.proxy_build(k, proxy, lens)
        f.append_decode_step(q, k_new, v_new, k, v, proxy, lens, w.budget, scores, idx, n_sel, out, ws)
    else:
        f.proxy_build(k, proxy, lens)
        f.decode_step(q, k, v, proxy, lens, w.budget, scores, idx, n_sel, out, ws)
    torch.cuda.synchronize()
    assert f.device_status() == 0
    assert torch.equal(lens, t["seq_lens"])
    G = w.group
    dom = np.sort(t["dom"].numpy(), axis=1)
    for (b, h) in units:
        L = int(t["seq_lens"][b])
        # one-unit views in the layouts check_step expects: [1][G][d], [1][1][L][d]
        rep = parity.check_step(q[b:b + 1, h * G:(h + 1) * G].cpu().double().numpy(), k[b:b + 1, h:h + 1, :L].cpu().double().numpy(),
                                v[b:b + 1, h:h + 1, :L].cpu().double().numpy(), [L], dom[h:h + 1], pairing=w.pairing,
                                group_reduce=w.group_reduce, n_sink=w.n_sink, n_recent=w.n_recent, budget=w.budget,
                                scale=1.0 / math.sqrt(128.0), scores=scores[b:b + 1, h:h + 1, :L].cpu().numpy(),
                                idx=idx[b:b + 1, h:h + 1].cpu().numpy(), n_sel=n_sel[b:b + 1, h:h + 1].cpu().numpy(),
                                out=out[b:b + 1, h * G:(h + 1) * G].cpu().numpy(), what=f"{w.name} unit ({b},{h})")
        assert rep["units"] == 1
        if keep is not None:
            keep.setdefault("q", {})[(b, h)] = q[b, h * G:(h + 1) * G].cpu().double().numpy()
            keep.setdefault("k", {})[(b, h)] = k[b, h, :L].cpu().double().numpy()
            keep.setdefault("idx", {})[(b, h)] = idx[b, h].cpu().numpy()
            keep.setdefault("n_sel", {})[(b, h)] = int(n_sel[b, h])
    if keep is not None:
        keep.update(t=t, proxy=proxy, idx_dev=idx, n_sel_dev=n_sel, out_dev=out)
    return f


def test_config2_full_size_sampled_units():
    # batch 16, ragged 64K-128K contexts, 8 GiB of K/V on the device: the cluster kernel in its wide
    # form (clusters of 4 CTAs of 1024 threads, up to 32768 keys each), several rounds of CTAs
    f = _full_size_sampled(C["c2"], [(0, 0), (7, 5), (15, 7)])
    assert f.step_cluster_size() == 4


@pytest.mark.parametrize("layer", [0, 1])
@pytest.mark.parametrize("step", [1, 512, 4096, 15360])
def test_config3_full_size_sampled_units_with_append(step, layer):
    # long-CoT shape: batch 32, G = 7, prompt 1024 + `step` generated tokens, budget 18.9 % of the
    # current length; two layers = two contexts with their own dominant-FC tables and caches.  Small
    # selections are attended inside the cluster kernel, large ones by the split-K kernel.
    L = 1024 + step
    w = C["c3"].replace(len_lo=L, len_hi=L, index=C["c3"].index + 1000 * layer)
    _full_size_sampled(w, [(0, 0), (31, 3), (13, 2)], append=True)


@pytest.mark.parametrize("budget", [256, 4096])
def test_config4_full_size_in_the_launch_shape_of_the_benchmark(budget):
    # batch 8 x 8 KV heads = 64 units, clusters of 4 with 16384 keys per CTA, the appending form:
    # budget 256 is one launch, budget 4096 the select-only cluster kernel + the split-K kernel
    # (64 units x clusters of 4 would put one 512-thread CTA on some SMs and two on others: the plan
    # takes the wide form, clusters of 2 CTAs of 1024 threads with 32768 keys each)
    f = _full_size_sampled(C["c4"].replace(budget=budget), [(0, 0), (3, 5), (7, 7)], append=True)
    assert f.step_cluster_size() == 2


@pytest.mark.parametrize("F,budget", [(4, 64), (64, 4096)])
def test_config4_sweep_corners_at_full_length(F, budget):
    # the corners of the budget x dominant-FC grid at the full 65536 context; with all 64 FCs the
    # score is the full logit, so the selection must also be the dense top-k (the "Oracle"
    # baseline of Sec. 5.1), taken here from a plain fp64 matrix product
    w = C["c4"].replace(n_dom=F, budget=budget)
    units = [(1, 2), (6, 0)]
    got = {}
    f = _full_size_sampled(w, units, keep=got)
    if F == 64:
        G = w.group
        for (b, h) in units:
            full = got["k"][(b, h)] @ got["q"][(b, h)].sum(axis=0)                  # sum over the group of q_g . k_j
            n = int(got["n_sel"][(b, h)])
            assert n == budget
            parity.check_selection(got["idx"][(b, h)][:n], full, 65536, budget, 0, 0, f"dense top-k ({b},{h})")


def test_config4_full_size_paged_and_host_resident_caches():
    # the benchmark's c4 point (budget 256) once more with (a) 64-token pages in random order and
    # (b) K and V in page-locked host memory (FASA-M): both must give the bits of the contiguous,
    # device-resident run, which is checked against the oracle on sampled units
    w = C["c4"]
    got = {}
    f = _full_size_sampled(w, [(2, 3), (5, 6)], keep=got)
    t = got["t"]
    B, Hq, Hkv, Lm, P = w.batch, w.n_q_heads, w.n_kv_heads, w.max_len, 64
    n_sel_max = w.n_sel_max()

    def fresh():
        return (torch.full((B, Hkv, n_sel_max), -7, dtype=torch.int32, device="cuda"), torch.full((B, Hkv), -7, dtype=torch.int32, device="cuda"),
                torch.full((B, Hq, 128), SENTINEL, dtype=torch.float32, device="cuda"))

    # (a) paged
    pps = Lm // P
    n_pages = B * pps
    table = torch.randperm(n_pages, generator=torch.Generator().manual_seed(3)).to(torch.int32).view(B, pps).cuda()
    fp = binding.Fasa(B, Hq, Hkv, Lm, t["dom"], rope_pairing=w.pairing, group_reduce=w.group_reduce, n_sink=w.n_sink,
                      n_recent=w.n_recent, page_size=P, n_pages=n_pages)
    fp.set_block_table(table)
    kp, vp = fp.alloc_paged_cache(), fp.alloc_paged_cache()
    for src, dst in ((t["k"], kp), (t["v"], vp)):
        dst[table.long().view(-1)] = src.view(B, Hkv, pps, P, 128).permute(0, 2, 1, 3, 4).reshape(n_pages, Hkv, P, 128)
    proxy = fp.alloc_proxy()
    fp.proxy_build(kp, proxy, t["seq_lens"])
    idx, n_sel, out = fresh()
    fp.decode_step(t["q"], kp, vp, proxy, t["seq_lens"], w.budget, None, idx, n_sel, out, None)
    torch.cuda.synchronize()
    assert fp.device_status() == 0
    assert torch.equal(idx, got["idx_dev"]) and torch.equal(n_sel, got["n_sel_dev"]) and torch.equal(out, got["out_dev"])
    del kp, vp, proxy, fp
    # (b) host-resident K and V, the proxy on the GPU
    kh, vh = f.alloc_host_cache(), f.alloc_host_cache()
    kh.copy_(t["k"]); vh.copy_(t["v"])
    idx, n_sel, out = fresh()
    f.decode_step(t["q"], kh, vh, got["proxy"], t["seq_lens"], w.budget, None, idx, n_sel, out, None)
    torch.cuda.synchronize()
    assert f.device_status() == 0
    assert torch.equal(idx, got["idx_dev"]) and torch.equal(n_sel, got["n_sel_dev"]) and torch.equal(out, got["out_dev"])


def test_contexts_of_different_sizes_coexist():
    # a large context, then a small one, then the large one again: per-kernel launch limits are
    # process-wide and must cover every live context
    big = Run(C["c4"].replace(batch=1, n_q_heads=8, n_kv_heads=2, max_len=30000, len_lo=30000, len_hi=30000, budget=64))
    small = Run(C["c1"].replace(n_q_heads=8, n_kv_heads=2, max_len=600, len_lo=600, len_hi=600, budget=32))
    for r in (big, small, big):
        r.build_proxy()
        r.reset_outputs()
        r.step(fused=True)
        h = r.host()
        parity.check_step(h["q"], h["k"], h["v"], h["seq_lens"], h["dom"], idx=h["idx"], n_sel=h["n_sel"], out=h["out"],
                          what=r.w.name, **r.oracle_kwargs())
        assert r.fasa.device_status() == 0
