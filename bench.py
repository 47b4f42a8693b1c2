#!/usr/bin/env python
"""Benchmark of the FASA decode hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl reference]

One step = one pass of the whole hot path over one batch: append one token per sequence
(K, V and proxy-K rows), score every cached key on the dominant FCs, select the top-budget
tokens, run exact attention over the selected rows and merge the splits.  The step is one
call, fasa_append_decode_step (one cluster kernel: append -> score -> select -> attention, or
that kernel ending after the selection + the split-K attention kernels where the selection is
large); the stand-alone calls (fasa_kv_append, fasa_fc_score, fasa_topk,
fasa_sparse_decode_attn) and the dense path are timed beside it.  The headline workload is
the largest single-GPU configuration (c2: batch 16, 64K-128K contexts, 8 GiB of K/V); the
smaller configurations ride along under `other_workloads`, and the budget row of
configuration 4 under `budget_row`.  Inputs are synthetic (paper_2602_03152_b200.synth) and
resident in HBM before the timed region; L2 is flushed between steps.  Rank 0 prints one JSON
line.

Headline metric: effective HBM GB/s = algorithmic bytes of the step (proxy bytes of every
cached token + K/V rows of the selected tokens + q + out) / device time, summed over ranks;
`us_per_step`, the dense-path time and the speedup ride along.  `roofline` describes the
dominant kernel (the cluster kernel: the whole step where it is one launch, scoring +
selection where attention is handed to the split-K kernel), `kernels` the three calls the
method names, `cpu_baseline` the fp64 oracle timed on the host, `parity` one unit of the timed
configuration checked against that oracle.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fasa_decode_attn_effective_hbm_gbs"
UNIT = "GB/s"
L2_FLUSH_BYTES = 256 << 20


# DRAM traffic of the dominant kernel from one ncu capture (dram__bytes_read.sum +
# dram__bytes_write.sum per launch) at the workload named here, next to that launch's algorithmic
# bytes.  Traffic follows the tokens processed, so for another workload of the same kernel the
# captured ratio is applied to its own algorithmic bytes and the figure is labelled
# "extrapolated"; it is reported only while the kernel sources are the captured ones.
TRAFFIC_CAPTURE = {"kernel": "fused_decode_kernel", "workload": "c4_sweep_llama3_8b_64k", "dram_bytes": 281.39e6,
                   "algorithmic_bytes": 277.02e6,
                   "sources": ("paper_2602_03152_b200/csrc/fasa_fused.cu", "paper_2602_03152_b200/csrc/fasa_score_core.cuh"),
                   "sha1": "bcda1628a361a3d74946dc3064adc6dc087de2ef"}


def _traffic(bytes_per_launch, workload):
    """(traffic bytes per launch or None, how it was obtained)."""
    import hashlib
    if not TRAFFIC_CAPTURE["sha1"]:
        return None, "no counters taken since the kernel last changed"
    h = hashlib.sha1()
    try:
        for f in TRAFFIC_CAPTURE["sources"]:
            h.update(open(os.path.join(ROOT, f), "rb").read())
    except OSError:
        return None, "kernel sources not found"
    if h.hexdigest() != TRAFFIC_CAPTURE["sha1"]:
        return None, "the kernel changed since the counters were taken"
    ratio = TRAFFIC_CAPTURE["dram_bytes"] / TRAFFIC_CAPTURE["algorithmic_bytes"]
    if workload == TRAFFIC_CAPTURE["workload"]:
        return bytes_per_launch * ratio, "ncu counters of this workload and kernel"
    return bytes_per_launch * ratio, ("extrapolated: DRAM bytes per algorithmic byte from an ncu capture of the same kernel at "
                                      + TRAFFIC_CAPTURE["workload"] + ", applied to this launch's algorithmic bytes")


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs, burst copy)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ---------------------------------------------------------------- byte model ----

def step_bytes(w, lens, n_sel):
    """Algorithmic bytes of one FASA step and of one dense step (Sec. 4.4 byte model).
    lens: per-sequence context at scoring time; n_sel: tokens attended, summed over the index
    sets.  The proxy counts once per KV head however many index sets share it."""
    units_len = sum(int(l) for l in lens) * w.n_kv_heads
    qo = w.batch * w.n_q_heads * 128 * (2 + 4)
    proxy = units_len * 4 * w.n_dom
    gathered = int(n_sel) * 512
    return {"proxy": proxy, "gathered": gathered, "qo": qo, "fasa": proxy + gathered + qo,
            "dense": units_len * 512 + qo}


# ---------------------------------------------------------------- clocks ----

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.rows, self.proc = [], None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def mark(self):
        """Forget the samples taken so far (set-up time)."""
        self.first = len(self.rows)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[getattr(self, "first", 0):]:
            try:
                sm.append(float(r[0])); mx = float(r[1])
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        # the busiest half of the samples stands for "under load"
        sm_sorted = sorted(sm)
        load = sm_sorted[len(sm_sorted) // 2:] if sm_sorted else []
        return {"sm_mhz": statistics.median(load) if load else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---------------------------------------------------------------- shared by both arms ----

def config_dict(w, lens=None):
    """What both arms print under `config`: the workload, by name and by its numbers."""
    lens = [w.len_lo, w.len_hi] if lens is None else lens
    return {"workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
            "context_lo": int(min(lens)), "context_hi": int(max(lens)), "max_len": w.max_len, "n_dom": w.n_dom,
            "budget": w.budget, "n_sink": w.n_sink, "n_recent": w.n_recent, "heads_per_index_set": w.heads_per_set,
            "l2": f"GPU arm: flushed before every step ({L2_FLUSH_BYTES >> 20} MiB write) and K/V + proxy larger than L2; "
                  "CPU arm: none",
            "per_rank": "each rank runs its own batch of independent units, no collective"}


def oracle_sample(w):
    """The bounded sample of a workload that the oracle is timed on: the units of sequence 0,
    context cut to 32768 rows where longer (about a second of CPU work per pass on a few cores)."""
    L = min(w.max_len, 32768)
    return w.replace(batch=1, max_len=L, len_lo=min(w.len_lo, L), len_hi=min(w.len_hi, L))


# ---------------------------------------------------------------- reference arm ----

def run_reference(args, w):
    """Times the fp64 CPU oracle, as it stands, on the host cores: each step is one oracle
    pass (score -> select -> attention) over a bounded sample of the workload's units."""
    from oracle import fasa_oracle as O
    from paper_2602_03152_b200 import synth

    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    sw = oracle_sample(w)
    t = synth.make_inputs(sw, "cpu")
    qb, kb, vb = synth.bf16_bits(t["q"]), synth.bf16_bits(t["k"]), synth.bf16_bits(t["v"])
    lens, dom = t["seq_lens"].numpy(), t["dom"].numpy()
    kw = dict(pairing=sw.pairing, group_reduce=sw.group_reduce, n_sink=sw.n_sink, n_recent=sw.n_recent,
              budget=sw.budget, n_sel_max=sw.n_sel_max(), n_threads=cores, want_scores=False, want_dense=False)
    steps, warm = max(1, min(args.steps, 20)), max(1, min(args.warmup, 3))
    for _ in range(warm):
        r = O.decode_bf16(qb, kb, vb, lens, dom, **kw)
    t0 = time.perf_counter()
    for _ in range(steps):
        r = O.decode_bf16(qb, kb, vb, lens, dom, **kw)
    dt = (time.perf_counter() - t0) / steps
    by = step_bytes(sw, lens, int(r["n_sel"].sum()))
    val = by["fasa"] / dt / 1e9
    sample = f"{sw.n_kv_heads} units (sequence 0 of {w.batch}), context {int(lens[0])}, one oracle pass per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": warm, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic", "config": config_dict(w), "sample": sample,
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": int(r["threads"]), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


# ---------------------------------------------------------------- our arm ----

def measure(w, K, W, dev, world, step_mode=None, sampler_factory=None, want_e2e=True, t=None, lens=None,
            min_region_s=0.0, want_parts=True, want_dense=True):
    """Times one workload on this rank's GPU; returns a dict of measurements (durations are
    max over ranks where that matters).  `t` reuses inputs drawn earlier (their dominant-FC
    list is redrawn for w.n_dom); `lens` overrides the sequence lengths.  The timed region is
    one block of exactly K steps, repeated until it has run for min_region_s of device time."""
    import torch
    import torch.distributed as dist

    from paper_2602_03152_b200 import binding, synth

    if t is None:
        t = synth.make_inputs(w, dev)
    else:
        t = dict(t)
        t["dom"] = synth.dominant_fcs(w)
    if lens is not None:
        t["seq_lens"] = torch.as_tensor(lens, dtype=torch.int32, device=dev)
    lens_full = t["seq_lens"].clone()
    # The cache has one spare row so each step appends at row L-1 and scores L rows.
    lens_start = (lens_full - 1).clamp_(min=0)
    f = binding.Fasa.from_workload(w, t["dom"])
    if step_mode is not None:
        f.set_step_mode(step_mode)
    fused = f.step_cluster_size() > 0
    q, k, v = t["q"], t["k"], t["v"]
    n_sel_max = w.n_sel_max()
    B, Hq, Hs, Lm = w.batch, w.n_q_heads, w.n_sets, w.max_len        # Hs index sets per sequence
    proxy = f.alloc_proxy(dev)
    ws = f.alloc_workspace(n_sel_max, dev)
    scores = torch.zeros((B, Hs, Lm), dtype=torch.float32, device=dev)
    idx = torch.zeros((B, Hs, n_sel_max), dtype=torch.int32, device=dev)
    n_sel = torch.zeros((B, Hs), dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, 128), dtype=torch.float32, device=dev)
    dense_out = torch.zeros_like(out)
    lens = lens_full.clone()
    f.proxy_build(k, proxy, lens)
    torch.cuda.synchronize()
    # the token appended each step: the cache's own last row, so the cache content never changes
    bi = torch.arange(B, device=dev)
    last = lens_start.long()
    k_new = k[bi, :, last].unsqueeze(2).contiguous()
    v_new = v[bi, :, last].unsqueeze(2).contiguous()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def timed(fn, n, warm):
        """n event-timed calls of fn on the current stream, L2 flushed and the sequence
        lengths reset before each; returns the list of durations in microseconds."""
        durs = []
        for i in range(warm + n):
            lens.copy_(lens_start)
            flush.fill_(i & 0xff)
            a, b = ev(), ev()
            a.record()
            fn()
            b.record()
            b.synchronize()
            if i >= warm:
                durs.append(a.elapsed_time(b) * 1e3)
        return durs

    def rank_max(x):
        if world > 1:
            tt = torch.tensor([x], dtype=torch.float64, device=dev)
            dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            return float(tt.item())
        return x

    def fasa_step():
        f.append_decode_step(q, k_new, v_new, k, v, proxy, lens, w.budget, None if fused else scores, idx, n_sel,
                             out, ws)

    def dense_step():
        f.kv_append(k, v, proxy, lens, k_new, v_new)
        f.full_decode_attn(q, k, v, lens, dense_out, ws)

    # nvidia-smi needs a moment before its first sample: the sampler was started by the caller
    # before the inputs were drawn; only samples taken from here on are kept
    sampler = sampler_factory() if sampler_factory else None
    if sampler is not None:
        sampler.mark()

    # ---- timed region: blocks of exactly K whole steps ----------------------------------
    timed(fasa_step, 0, W)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    l0 = f.launch_count()
    blocks = [timed(fasa_step, K, 0)]
    torch.cuda.synchronize()
    launches = f.launch_count() - l0
    while sum(sum(b_) for b_ in blocks) * 1e-6 < min_region_s and len(blocks) < 200 and world == 1:
        blocks.append(timed(fasa_step, K, 0))
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    block_us = [sum(b_) / K for b_ in blocks]
    us_per_step = rank_max(sum(block_us) / len(block_us))
    all_steps = [x for b_ in blocks for x in b_]

    n_sel_total = int(n_sel.sum().item())
    by = step_bytes(w, lens_full.cpu().tolist(), n_sel_total)
    Kk = min(K, 200)

    # ---- the dominant kernel alone, where the step is several launches --------------------
    launches_per_step = launches / max(K, 1)
    select_us = None
    if fused and launches_per_step > 1:
        select_us = statistics.mean(timed(lambda: f.select_step(q, k, v, proxy, lens, w.budget, None, idx, n_sel, k_new, v_new),
                                          Kk, W))
        lens.copy_(lens_start)
        fasa_step()                                # (leave idx / n_sel / out as the whole step writes them)

    # ---- the stand-alone calls, one C-ABI call at a time ---------------------------------
    kern_us = None
    if want_parts:
        parts = {"kv_append": [], "fc_score": [], "topk": [], "sparse_attn": []}
        for i in range(W + Kk):
            lens.copy_(lens_start)
            flush.fill_(i & 0xff)
            e = [ev() for _ in range(5)]
            e[0].record(); f.kv_append(k, v, proxy, lens, k_new, v_new)
            e[1].record(); f.fc_score(q, proxy, lens, scores)
            e[2].record(); f.topk(scores, lens, w.budget, idx, n_sel, ws)
            e[3].record(); f.sparse_decode_attn(q, k, v, idx, n_sel, out, ws)
            e[4].record(); e[4].synchronize()
            if i >= W:
                for j, name in enumerate(parts):
                    parts[name].append(e[j].elapsed_time(e[j + 1]) * 1e3)
        kern_us = {n: statistics.mean(v_) for n, v_ in parts.items()}
    dense_us = statistics.mean(timed(dense_step, min(Kk, 50), W)) if want_dense else None

    # ---- end to end from host buffers ---------------------------------------------------
    e2e_us = h2d = d2h = None
    if want_e2e:
        stage = torch.empty(f.stage_bytes(), dtype=torch.uint8, device=dev)
        qh, knh, vnh = q.cpu().pin_memory(), k_new.cpu().pin_memory(), v_new.cpu().pin_memory()
        oh = torch.empty((B, Hq, 128), dtype=torch.float32).pin_memory()

        def e2e_step():
            f.decode_step_host(qh, knh, vnh, stage, k, v, proxy, lens, w.budget, None if fused else scores, idx,
                               n_sel, out, oh, ws)

        e2e_us = rank_max(statistics.mean(timed(e2e_step, Kk, W)))
        h2d = qh.numel() * 2 + knh.numel() * 2 + vnh.numel() * 2
        d2h = oh.numel() * 4
    # one more whole step, whose outputs the parity check reads
    lens.copy_(lens_start)
    fasa_step()
    torch.cuda.synchronize()
    status = f.device_status()
    clocks = sampler.stop() if sampler else None
    return dict(w=w, t=t, by=by, us_per_step=us_per_step, step_us_median=statistics.median(all_steps),
                block_us=block_us, launches=launches, kern_us=kern_us, dense_us=dense_us, e2e_us=e2e_us, h2d=h2d,
                d2h=d2h, status=status, clocks=clocks, fused=fused, cluster_size=f.step_cluster_size(),
                launches_per_step=launches_per_step, select_us=select_us, n_sel_total=n_sel_total,
                lens_full=lens_full, last=dict(idx=idx, n_sel=n_sel, out=out))


def kernel_rooflines(m, peak):
    """The three calls the method names, each against its own bytes: `bytes` counts what the
    call must move including its unavoidable scratch (the fp32 score per token that scoring
    writes and the selection reads, the index list), `bytes_method` only what the byte model of
    the method counts for that stage (proxy rows; nothing for the selection; K/V rows)."""
    w, by, ku = m["w"], m["by"], m["kern_us"]
    tokens = by["proxy"] // (4 * w.n_dom) * w.n_sets // w.n_kv_heads      # scored positions: one fp32 per (set, token)
    sel = m["n_sel_total"]
    rows = {
        "fasa_fc_score": (by["proxy"] + 4 * tokens + by["qo"] // 3, by["proxy"], ku["fc_score"]),
        "fasa_topk": (4 * tokens + 4 * sel, 0, ku["topk"]),
        "fasa_sparse_decode_attn": (by["gathered"] + 4 * sel + by["qo"], by["gathered"], ku["sparse_attn"]),
    }
    out = {}
    for name, (b_all, b_method, us) in rows.items():
        out[name] = {"us": us, "bytes": b_all, "gbs": b_all / us / 1e3, "frac": b_all / us / 1e3 / peak, "bound": "hbm",
                     "bytes_method": b_method, "frac_method_bytes": b_method / us / 1e3 / peak}
    return out


def summarize(m, peak):
    """The figures every workload reports (the headline workload adds the contract's keys)."""
    w, by = m["w"], m["by"]
    gbs = lambda nbytes, us: nbytes / (us * 1e-6) / 1e9
    r = {
        "workload": w.name, "batch": w.batch, "n_q_heads": w.n_q_heads, "n_kv_heads": w.n_kv_heads,
        "context": int(m["lens_full"].max()), "context_mean": float(m["lens_full"].float().mean()),
        "n_dom": w.n_dom, "budget": w.budget, "n_sink": w.n_sink, "n_recent": w.n_recent,
        "n_sel_per_unit": m["n_sel_total"] / (w.batch * w.n_sets), "heads_per_index_set": w.heads_per_set,
        "step_mode": ("three kernels" if not m["fused"] else
                      f"one cluster kernel (cluster of {m['cluster_size']})" if m["launches_per_step"] == 1 else
                      f"cluster kernel (cluster of {m['cluster_size']}, ends after the selection) + split-K tensor-core attention + merge"),
        "launches_per_step": m["launches_per_step"],
        "us_per_step": m["us_per_step"], "us_per_step_median": m["step_us_median"], "step_bytes": by["fasa"],
        "step_gbs": gbs(by["fasa"], m["us_per_step"]), "step_frac_of_peak": gbs(by["fasa"], m["us_per_step"]) / peak,
        "device_status": m["status"],
    }
    if m["dense_us"] is not None:
        r.update({"dense_us_per_step": m["dense_us"], "dense_bytes": by["dense"],
                  "dense_frac_of_peak": gbs(by["dense"], m["dense_us"]) / peak,
                  "speedup_vs_dense": m["dense_us"] / m["us_per_step"],
                  "byte_ratio_dense_over_fasa": by["dense"] / by["fasa"]})
    if m["kern_us"] is not None:
        r["standalone_us"] = m["kern_us"]
        r["kernels"] = kernel_rooflines(m, peak)
    return r


def run_fasa(args, w):
    import torch
    import torch.distributed as dist

    from paper_2602_03152_b200 import build, synth

    build.build()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the FASA path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    gpu_id = str(local)
    try:
        gpu_id = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    K, W = args.steps, max(3, args.warmup)
    # Weak scaling: every rank holds its own batch of independent (batch, KV head) units.
    wl = w.replace(index=w.index + 100 * rank)
    sampler = ClockSampler(gpu_id) if rank == 0 else None     # started early, marked at the timed region
    m = measure(wl, K, W, dev, world, args.step_mode, (lambda: sampler) if rank == 0 else None,
                min_region_s=args.min_region_s)

    peak, peak_src = _peaks()
    line_extra = {}
    if world == 1 and rank == 0 and not args.no_cpu_baseline:
        line_extra = cpu_baseline(wl, m)                       # (reads the inputs: before they are released)
    m.pop("t")
    m.pop("last")
    torch.cuda.empty_cache()

    # Other configurations of the same path, a few steps each (single GPU only).
    others, budget_row = [], []
    if world == 1 and not args.no_extras:
        for name in args.extras.split(","):
            if name and name in synth.CONFIGS and name != args.config:
                mo = measure(synth.CONFIGS[name], 50, 3, dev, 1, args.step_mode, None, want_e2e=False, min_region_s=0.05)
                mo.pop("t"); mo.pop("last")
                others.append(summarize(mo, peak))
                del mo
                torch.cuda.empty_cache()
    if world == 1 and not args.no_budget_row:
        # configuration 4 at 16 dominant FCs, every budget of its grid: the step and the dense
        # path at each point ("speed-up over dense at every budget")
        base = synth.CONFIGS["c4"]
        tb = synth.make_inputs(base, dev)
        for kb in (64, 128, 256, 512, 1024, 2048, 4096):
            mo = measure(base.replace(budget=kb), 12, 3, dev, 1, args.step_mode, None, want_e2e=False, t=tb,
                         want_parts=False, want_dense=True)
            sm = summarize(mo, peak)
            budget_row.append({k_: sm[k_] for k_ in ("budget", "us_per_step", "step_bytes", "step_frac_of_peak", "dense_us_per_step",
                                                     "speedup_vs_dense", "byte_ratio_dense_over_fasa", "launches_per_step", "device_status")})
            del mo
        del tb
        torch.cuda.empty_cache()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    by, us_per_step = m["by"], m["us_per_step"]
    head = summarize(m, peak)
    roof_us = by["fasa"] / (peak * 1e9) * 1e6
    if m["fused"] and m["launches_per_step"] == 1:
        # dominant kernel = the whole step in one launch: its algorithmic bytes are the step's
        tr, tr_src = _traffic(by["fasa"], wl.name)
        roofline = {"kernel": "fused_decode_kernel (whole step)", "bound": "hbm", "achieved": head["step_gbs"], "peak": peak,
                    "unit": "GB/s", "frac": head["step_frac_of_peak"], "traffic": tr, "traffic_source": tr_src,
                    "bytes_per_launch": by["fasa"], "us_per_launch": us_per_step, "peak_source": peak_src,
                    "cluster_size": m["cluster_size"]}
    elif m["fused"]:
        # dominant kernel = the cluster kernel ending after the selection (append + scoring + selection
        # in one launch): it moves the proxy rows of every token, q and the index lists it writes
        kb = by["proxy"] + by["qo"] // 3 + 4 * m["n_sel_total"]
        us = m["select_us"]
        tr, tr_src = _traffic(kb, wl.name)
        roofline = {"kernel": "fused_decode_kernel (append + scoring + selection)", "bound": "hbm",
                    "achieved": kb / us / 1e3, "peak": peak, "unit": "GB/s", "frac": kb / us / 1e3 / peak,
                    "traffic": tr, "traffic_source": tr_src, "bytes_per_launch": kb, "us_per_launch": us,
                    "share_of_step_time": us / us_per_step, "peak_source": peak_src, "cluster_size": m["cluster_size"]}
    else:
        fc_us = m["kern_us"]["fc_score"]
        roofline = {"kernel": "fc_score_kernel", "bound": "hbm", "achieved": by["proxy"] / (fc_us * 1e-6) / 1e9,
                    "peak": peak, "unit": "GB/s", "frac": by["proxy"] / (fc_us * 1e-6) / 1e9 / peak, "traffic": None,
                    "traffic_source": "no counters taken", "bytes_per_launch": by["proxy"], "us_per_launch": fc_us,
                    "peak_source": peak_src}
    roofline["frac_of_nominal_8tbs"] = roofline["achieved"] / 8000.0      # context: the DGX figure for HBM3e
    cfg = config_dict(w, m["lens_full"].cpu().tolist())
    cfg["step_mode"] = head["step_mode"]
    clocks = m["clocks"]
    line = {
        "metric": METRIC, "value": world * by["fasa"] / (us_per_step * 1e-6) / 1e9, "unit": UNIT,
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": us_per_step / 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in, f32 accumulate",
        "data": "synthetic", "config": cfg,
        "timed_blocks": len(m["block_us"]), "us_per_step": us_per_step,
        "us_per_step_median_block": statistics.median(m["block_us"]), "us_per_step_median": m["step_us_median"],
        "us_per_step_x_sm_mhz": (us_per_step * clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None,
        "n_sel_per_unit": head["n_sel_per_unit"],
        "step_bytes": by["fasa"], "step_roofline_us": roof_us, "step_frac_of_roofline": roof_us / us_per_step,
        "dense_us_per_step": m["dense_us"], "dense_bytes": by["dense"], "dense_frac_of_roofline": head["dense_frac_of_peak"],
        "speedup_vs_dense": head["speedup_vs_dense"], "byte_ratio_dense_over_fasa": head["byte_ratio_dense_over_fasa"],
        "standalone_kernels_us": m["kern_us"], "kernels": head["kernels"],
        "roofline": roofline,
        "e2e": {"value": world * by["fasa"] / (m["e2e_us"] * 1e-6) / 1e9, "unit": UNIT, "us_per_step": m["e2e_us"],
                "h2d_bytes_per_step": m["h2d"], "d2h_bytes_per_step": m["d2h"]},
        "gpu_launches": int(m["launches"]), "device_status": m["status"], "clocks": clocks,
        "other_workloads": others, "budget_row": {"workload": "c4_sweep_llama3_8b_64k", "n_dom": 16, "rows": budget_row},
    }
    line.update(line_extra)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Workload c4 as a grid: budget x dominant-FC count at the Llama-3-8B shape, batch 8,
    context 65536.  One JSON object with a row per point."""
    import torch

    from paper_2602_03152_b200 import build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    base = synth.CONFIGS["c4"]
    if args.batch is not None:
        base = base.replace(batch=args.batch)
    if args.select_heads is not None:
        base = base.replace(sel_heads=args.select_heads)
    t = synth.make_inputs(base, dev)
    peak, peak_src = _peaks()
    rows = []
    for F in ((4, 8, 16, 32, 64) if args.n_dom is None else (args.n_dom,)):
        for k in (64, 128, 256, 512, 1024, 2048, 4096):
            w = base.replace(n_dom=F, budget=k)
            m = measure(w, args.sweep_steps, 3, dev, 1, args.step_mode, None, want_e2e=False, t=t)
            sm = summarize(m, peak)
            rows.append({k_: sm[k_] for k_ in ("n_dom", "budget", "us_per_step", "step_bytes", "step_gbs", "step_frac_of_peak",
                                               "dense_us_per_step", "speedup_vs_dense", "byte_ratio_dense_over_fasa",
                                               "standalone_us", "kernels", "step_mode", "launches_per_step",
                                               "device_status")})
            del m
    print(json.dumps({"sweep": base.name, "batch": base.batch, "context": base.max_len,
                      "heads_per_index_set": base.heads_per_set, "peak_gbs": peak,
                      "peak_source": peak_src, "steps_per_point": args.sweep_steps, "rows": rows}), flush=True)


def run_calib(args):
    """Offline calibration (Algorithm 1) on the Llama-3-8B shape of workload c1: one call =
    batch x query heads samples (per-FC and full raw scores, 65 top-k selections each,
    intersection counts).  One JSON object: time per call, samples per second, the bytes the
    three kernels move and the oracle's time for one sample on the host."""
    import time

    import numpy as np
    import torch

    from oracle import fasa_oracle as O
    from paper_2602_03152_b200 import binding, build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.CONFIGS[args.config]
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    top_k = args.budget if args.budget is not None else 256
    t = synth.make_inputs(w, dev)
    f = binding.Fasa.from_workload(w, t["dom"])
    counts = torch.zeros((w.n_q_heads, 64), dtype=torch.int64, device=dev)
    used = torch.zeros(w.n_q_heads, dtype=torch.int64, device=dev)
    ws = torch.empty(f.calib_workspace_bytes(top_k), dtype=torch.uint8, device=dev)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    ts = []
    for i in range(args.warmup + args.steps):
        flush.fill_(i & 1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        f.calib_accumulate(t["q"], t["k"], t["seq_lens"], top_k, counts, used, ws)
        b.record()
        b.synchronize()
        if i >= args.warmup:
            ts.append(a.elapsed_time(b) * 1e3)
    us = float(np.mean(ts))
    samples = int(sum(1 for l in t["seq_lens"].tolist() if l > top_k)) * w.n_q_heads
    tokens = int(sum(t["seq_lens"].tolist()))
    # K rows once per KV head (query heads of a group re-read them from L2), 65 fp32 score rows
    # per sample written and read once, 65 index lists written and read once
    by = tokens * w.n_kv_heads * 256 + 2 * tokens * w.n_q_heads * 65 * 4 + 2 * samples * 65 * top_k * 4
    peak, peak_src = _peaks()
    # the oracle on one sample (sequence 0, query head 0), as it stands
    q0 = t["q"][0, 0].double().cpu().numpy()
    k0 = t["k"][0, 0, :int(t["seq_lens"][0])].double().cpu().numpy()
    t0 = time.perf_counter()
    c_or = O.ca_counts(q0, k0, top_k, w.pairing, f32=True)
    cpu_s = time.perf_counter() - t0
    got = (counts[0].cpu().numpy() // max(1, args.warmup + args.steps)) if w.batch == 1 else None
    print(json.dumps({"calibration": w.name, "top_k": top_k, "samples_per_call": samples, "us_per_call": us,
                      "samples_per_s": samples / us * 1e6, "bytes_per_call": by, "gbs": by / us / 1e3,
                      "frac_of_peak": by / us / 1e3 / peak, "peak_source": peak_src,
                      "workspace_bytes": int(ws.numel()), "launches_per_call": 3, "steps": args.steps,
                      "oracle_s_per_sample": cpu_s, "oracle_samples_per_s": 1.0 / cpu_s,
                      "counts_match_oracle_sample": None if got is None else bool(np.array_equal(got, c_or)),
                      "device_status": f.device_status()}), flush=True)


def _longcot_resident(w, samples, reps, dev, n_layers=28):
    """All 28 layers of workload c3 resident at once (their own random bf16 K/V caches, proxies and
    dominant-FC tables, about 32 GB), one decode step of the whole stack = 28 append+step
    calls captured in a CUDA graph, a second graph for the dense stack; both replayed at the
    sampled cache lengths.  The lengths are device data, so one capture could serve them all;
    a serving loop knows its step count, though, and passes the selection bound of the current
    length (n_sel_max = ceil(0.189 L)), which lets the library attend inside the cluster kernel
    while selections are small: one capture per sampled length, as a loop with length buckets
    would hold.  No L2 flush: 28 layers of cache stream through L2 between two visits of a layer."""
    import torch

    from paper_2602_03152_b200 import binding, synth

    B, Hq, Hkv, Lm = w.batch, w.n_q_heads, w.n_kv_heads, w.max_len
    n_sel_max = w.n_sel_max()
    lens_all = torch.zeros((n_layers, B), dtype=torch.int32, device=dev)
    full = torch.full((B,), Lm, dtype=torch.int32, device=dev)
    layers = []
    for l in range(n_layers):
        wl = w.replace(index=w.index + 1000 * (l + 1))              # every layer its own seed
        t = synth.make_inputs(wl.replace(len_lo=Lm, len_hi=Lm), dev)
        s = synth.make_step_inputs(wl, 0, dev)
        f = binding.Fasa.from_workload(wl, t["dom"])
        proxy = f.alloc_proxy(dev)
        f.proxy_build(t["k"], proxy, full)
        layers.append(dict(f=f, k=t["k"], v=t["v"], proxy=proxy, lens=lens_all[l], q=s["q"], kn=s["k_new"], vn=s["v_new"],
                           idx=torch.zeros(B * w.n_sets * n_sel_max, dtype=torch.int32, device=dev),
                           n_sel=torch.zeros((B, w.n_sets), dtype=torch.int32, device=dev),
                           out=torch.zeros((B, Hq, 128), dtype=torch.float32, device=dev),
                           ws=f.alloc_workspace(n_sel_max, dev)))
    torch.cuda.synchronize()

    def fasa_stack(n_bound):
        for y in layers:
            idx = y["idx"][:B * w.n_sets * n_bound].view(B, w.n_sets, n_bound)
            y["f"].append_decode_step(y["q"], y["kn"], y["vn"], y["k"], y["v"], y["proxy"], y["lens"], w.budget, None,
                                      idx, y["n_sel"], y["out"], y["ws"])

    def dense_stack():
        for y in layers:
            y["f"].kv_append(y["k"], y["v"], y["proxy"], y["lens"], y["kn"], y["vn"])
            y["f"].full_decode_attn(y["q"], y["k"], y["v"], y["lens"], y["out"], y["ws"])

    def capture(fn):
        lens_all.fill_(1024)
        n0 = sum(y["f"].launch_count() for y in layers)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            fn()
        return g, sum(y["f"].launch_count() for y in layers) - n0

    dense_graph = capture(dense_stack)
    pts = []
    for L in samples:
        n_bound = min(n_sel_max, (-w.budget * L + 999) // 1000 + w.n_sink + w.n_recent) if w.budget < 0 else n_sel_max
        row = {"context": L, "n_sel_max_passed": n_bound}
        for name, (g, launches) in (("fasa", capture(lambda: fasa_stack(n_bound))), ("dense", dense_graph)):
            ts = []
            for i in range(reps + 2):
                lens_all.fill_(L - 1)                               # every step appends at row L-1
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                g.replay()
                b.record()
                b.synchronize()
                if i >= 2:
                    ts.append(a.elapsed_time(b) * 1e3)
            row[name + "_us_per_token_step"] = sum(ts) / len(ts)
            row[name + "_launches"] = launches
        row["n_sel_per_unit"] = float(layers[0]["n_sel"].float().mean().item())
        row["speedup_vs_dense"] = row["dense_us_per_token_step"] / row["fasa_us_per_token_step"]
        pts.append(row)
    status = 0
    for y in layers:
        status |= y["f"].device_status()
    return pts, status


def run_offload(args):
    """The memory-optimised variant (FASA-M, Algorithm 2) on --config's shape: K and V caches in
    page-locked host memory, only the proxy (the dominant part of the key cache) on the GPU.  One
    step = one fasa_append_decode_step call; the selected rows cross the host link inside the
    kernel.  The bound is the link: bytes over it per step / a measured pinned-to-device copy rate.
    One JSON object, with the same step on device-resident caches and the dense path over the
    host-resident caches beside it."""
    import numpy as np
    import torch

    from paper_2602_03152_b200 import binding, build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.CONFIGS[args.config]
    if args.budget is not None:
        w = w.replace(budget=args.budget)
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def timed(fn, n, warm, pre=None):
        ts = []
        for i in range(warm + n):
            flush.fill_(i & 1)
            if pre:
                pre()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            b.synchronize()
            if i >= warm:
                ts.append(a.elapsed_time(b) * 1e3)
        return float(np.mean(ts)), float(np.min(ts))

    src = torch.empty(256 << 20, dtype=torch.uint8).pin_memory()
    dst = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    _, cp_best = timed(lambda: dst.copy_(src, non_blocking=True), 5, 2)
    link_gbs = (256 << 20) / cp_best / 1e3
    del src, dst

    t = synth.make_inputs(w, dev)
    f = binding.Fasa.from_workload(w, t["dom"])
    B, Hq, Lm = w.batch, w.n_q_heads, w.max_len
    n_sel_max = w.n_sel_max()
    proxy = f.alloc_proxy(dev)
    f.proxy_build(t["k"], proxy, t["seq_lens"])
    kh, vh = f.alloc_host_cache(), f.alloc_host_cache()
    kh.copy_(t["k"])
    vh.copy_(t["v"])
    s = synth.make_step_inputs(w, 0, dev)
    idx = torch.zeros((B, w.n_sets, n_sel_max), dtype=torch.int32, device=dev)
    n_sel = torch.zeros((B, w.n_sets), dtype=torch.int32, device=dev)
    out = torch.zeros((B, Hq, 128), dtype=torch.float32, device=dev)
    ws = f.alloc_workspace(n_sel_max, dev)
    lens = t["seq_lens"].clone()
    start = (t["seq_lens"] - 1).clamp_(min=0)

    # Without a workspace the step stays one launch whatever the selection size (the cluster
    # kernel's own gather); the tensor-core attention route is measured beside it.
    def step(k, v):
        return lambda: f.append_decode_step(s["q"], s["k_new"], s["v_new"], k, v, proxy, lens, w.budget, None, idx,
                                            n_sel, out, None)

    reset = lambda: lens.copy_(start)
    us_host, _ = timed(step(kh, vh), args.steps, args.warmup, reset)
    out_host = out.clone()
    # the same caches through the tensor-core attention kernel (a workspace hands the attention over)
    us_host_ws, _ = timed(lambda: f.append_decode_step(s["q"], s["k_new"], s["v_new"], kh, vh, proxy, lens, w.budget, None, idx,
                                                       n_sel, out, ws), args.steps, args.warmup, reset)
    # the split key cache of Algorithm 2: only the non-dominant channels of the selected keys cross the link
    split = None
    if w.n_dom % 4 == 0:
        knd = f.alloc_host_nondom()
        f.m_split(t["k"], knd, t["seq_lens"])
        torch.cuda.synchronize()
        us_split, _ = timed(lambda: f.m_decode_step(s["q"], knd, vh, proxy, lens, w.budget, None, idx, n_sel, out, ws, None,
                                                    s["k_new"], s["v_new"]), args.steps, args.warmup, reset)
        nsel = int(n_sel.sum().item())
        split_link = nsel * (512 - 4 * w.n_dom) + w.batch * w.n_kv_heads * (512 - 4 * w.n_dom)
        split = {"us_per_step": us_split, "link_bytes_per_step": split_link, "link_bytes_per_selected_token": 512 - 4 * w.n_dom,
                 "achieved_gbs": split_link / us_split / 1e3, "frac_of_link": split_link / us_split / 1e3 / link_gbs,
                 "max_abs_diff_vs_whole_rows": float((out - out_host).abs().max())}
        # the forced rows (sinks + recent window) kept on the GPU: they no longer cross the link
        if w.n_sink + w.n_recent > 0:
            out_split = out.clone()
            res_buf = f.alloc_resident()
            f.m_resident_build(knd, vh, proxy, t["seq_lens"])
            torch.cuda.synchronize()
            us_res, _ = timed(lambda: f.m_decode_step(s["q"], knd, vh, proxy, lens, w.budget, None, idx, n_sel, out, ws, None,
                                                      s["k_new"], s["v_new"]), args.steps, args.warmup, reset)
            forced = sum(min(int(L), w.n_sink + w.n_recent) for L in t["seq_lens"].cpu().tolist()) * w.n_kv_heads
            res_link = (nsel - forced) * (512 - 4 * w.n_dom) + w.batch * w.n_kv_heads * (512 - 4 * w.n_dom)
            split["resident_forced_rows"] = {
                "us_per_step": us_res, "link_bytes_per_step": res_link, "rows_kept_on_gpu_per_unit": w.n_sink + w.n_recent,
                "gpu_bytes": int(res_buf.numel()), "achieved_gbs": res_link / us_res / 1e3,
                "frac_of_link": res_link / us_res / 1e3 / link_gbs, "outputs_identical": bool(torch.equal(out, out_split))}
            f.m_set_resident(None)
            del res_buf
        del knd
    n_sel_total = int(n_sel.sum().item())
    us_dev, _ = timed(step(t["k"], t["v"]), args.steps, args.warmup, reset)
    same = bool(torch.equal(out, out_host))
    dense_steps = max(3, min(args.steps, 10))
    us_dense_host, _ = timed(lambda: f.full_decode_attn(s["q"], kh, vh, lens, out, ws), dense_steps, 1, reset)
    by = step_bytes(w, t["seq_lens"].cpu().tolist(), n_sel_total)
    link_bytes = by["gathered"] + w.batch * w.n_kv_heads * 512          # selected rows in, the new K and V rows out
    hbm_peak, _ = _peaks()
    bound_us = link_bytes / link_gbs / 1e3 + (by["proxy"] + by["qo"]) / hbm_peak / 1e3
    tokens = int(sum(t["seq_lens"].cpu().tolist())) * w.n_kv_heads
    print(json.dumps({
        "offload": w.name, "variant": "FASA-M (Algorithm 2): K, V in page-locked host memory; proxy-K on the GPU",
        "budget": w.budget, "n_dom": w.n_dom, "steps": args.steps,
        "us_per_step": us_host, "us_per_step_device_resident": us_dev, "outputs_identical_to_device_resident": same,
        "link_bytes_per_step": link_bytes, "hbm_bytes_per_step": by["proxy"] + by["qo"],
        "roofline": {"bound": "host link", "achieved": link_bytes / us_host / 1e3, "peak": link_gbs, "unit": "GB/s",
                     "frac": link_bytes / us_host / 1e3 / link_gbs,
                     "peak_source": "measured here: 256 MiB page-locked host -> device copy, best of 5",
                     "step_bound_us": bound_us, "step_frac_of_bound": bound_us / us_host},
        "whole_rows_tensor_core_attention": {"us_per_step": us_host_ws, "achieved_gbs": link_bytes / us_host_ws / 1e3,
                                             "frac_of_link": link_bytes / us_host_ws / 1e3 / link_gbs},
        "split_key_cache": split,
        "dense_over_host_resident_caches_us": us_dense_host,
        "speedup_vs_dense_over_host_resident_caches": us_dense_host / us_host,
        "gpu_bytes_per_cached_token": {"fasa_m": f.row_elems * 2, "full_cache": 512 + f.row_elems * 2},
        "gpu_cache_bytes": {"fasa_m": tokens * f.row_elems * 2, "full_cache": tokens * (512 + f.row_elems * 2)},
        "device_status": f.device_status()}), flush=True)


def run_paged(args):
    """Paged caches on --config's shape (page pools in random page order behind a block table): the
    step (fasa_decode_step), the same work as the three stand-alone kernels and the dense path, next
    to the same on contiguous caches.  One JSON object."""
    import numpy as np
    import torch

    from paper_2602_03152_b200 import binding, build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.CONFIGS[args.config]
    if args.budget is not None:
        w = w.replace(budget=args.budget)
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    P = args.paged
    t = synth.make_inputs(w, dev)
    B, Hq, Hkv, Lm = w.batch, w.n_q_heads, w.n_kv_heads, w.max_len
    pps = (Lm + P - 1) // P
    n_pages = B * pps
    table = torch.randperm(n_pages, generator=torch.Generator().manual_seed(1)).to(torch.int32).view(B, pps).to(dev)
    fc = binding.Fasa.from_workload(w, t["dom"])
    fp = binding.Fasa(B, Hq, Hkv, Lm, t["dom"], rope_pairing=w.pairing, group_reduce=w.group_reduce, n_sink=w.n_sink,
                      n_recent=w.n_recent, select_heads=w.sel_heads, page_size=P, n_pages=n_pages)
    fp.set_block_table(table)
    kp, vp = fp.alloc_paged_cache(dev), fp.alloc_paged_cache(dev)
    pad = pps * P - Lm
    for src, dst in ((t["k"], kp), (t["v"], vp)):
        lv = torch.nn.functional.pad(src, (0, 0, 0, pad)).view(B, Hkv, pps, P, 128).permute(0, 2, 1, 3, 4)
        dst[table.long().view(-1)] = lv.reshape(B * pps, Hkv, P, 128)
    n_sel_max = w.n_sel_max()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    res = {}
    outs = {}
    for name, f, k, v in (("contiguous", fc, t["k"], t["v"]), ("paged", fp, kp, vp)):
        proxy = f.alloc_proxy(dev)
        f.proxy_build(k, proxy, t["seq_lens"])
        scores = torch.zeros((B, w.n_sets, Lm), dtype=torch.float32, device=dev)
        idx = torch.zeros((B, w.n_sets, n_sel_max), dtype=torch.int32, device=dev)
        n_sel = torch.zeros((B, w.n_sets), dtype=torch.int32, device=dev)
        out = torch.zeros((B, Hq, 128), dtype=torch.float32, device=dev)
        ws = f.alloc_workspace(n_sel_max, dev)
        f.set_step_mode(1)

        def three():
            f.fc_score(t["q"], proxy, t["seq_lens"], scores)
            f.topk(scores, t["seq_lens"], w.budget, idx, n_sel, ws)
            f.sparse_decode_attn(t["q"], k, v, idx, n_sel, out, ws)

        row = {}
        n0 = f.launch_count()
        f.decode_step(t["q"], k, v, proxy, t["seq_lens"], w.budget, None, idx, n_sel, out, ws)
        row["launches_per_step"] = int(f.launch_count() - n0)
        for what, fn in (("step_us", lambda: f.decode_step(t["q"], k, v, proxy, t["seq_lens"], w.budget, None, idx, n_sel, out, ws)),
                         ("step_three_kernels_us", three),
                         ("dense_us", lambda: f.full_decode_attn(t["q"], k, v, t["seq_lens"], out, ws))):
            ts = []
            for i in range(args.warmup + args.steps):
                flush.fill_(i & 1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                b.synchronize()
                if i >= args.warmup:
                    ts.append(a.elapsed_time(b) * 1e3)
            row[what] = float(np.mean(ts))
        three()
        torch.cuda.synchronize()
        outs[name] = (out.clone(), idx.clone())
        row["device_status"] = f.device_status()
        res[name] = row
        del proxy, scores
    by = step_bytes(w, t["seq_lens"].cpu().tolist(), int(n_sel.sum().item()))
    peak, _ = _peaks()
    for name in res:
        res[name]["step_frac_of_peak"] = by["fasa"] / res[name]["step_us"] / 1e3 / peak
        res[name]["three_kernels_frac_of_peak"] = by["fasa"] / res[name]["step_three_kernels_us"] / 1e3 / peak
        res[name]["dense_frac_of_peak"] = by["dense"] / res[name]["dense_us"] / 1e3 / peak
    print(json.dumps({"paged_caches": w.name, "page_size": P, "n_pages": n_pages, "budget": w.budget, "steps": args.steps,
                      "results_identical": bool(torch.equal(outs["paged"][0], outs["contiguous"][0]) and
                                                torch.equal(outs["paged"][1], outs["contiguous"][1])),
                      **res}), flush=True)


def run_batched(args):
    """Blocks of query tokens (q_len > 1) on --config's shape: the three batched calls (scoring of all
    queries of a block in one pass over the proxy on the tcgen05 tensor cores, selection and attention
    per query) next to q_len repetitions of the single-query calls.  One JSON object."""
    import numpy as np
    import torch

    from paper_2602_03152_b200 import binding, build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.CONFIGS[args.config]
    if args.budget is not None:
        w = w.replace(budget=args.budget)
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    t = synth.make_inputs(w, dev)
    f = binding.Fasa.from_workload(w, t["dom"])
    B, Hq, Hs, Lm = w.batch, w.n_q_heads, w.n_sets, w.max_len
    n_sel_max = w.n_sel_max()
    proxy = f.alloc_proxy(dev)
    f.proxy_build(t["k"], proxy, t["seq_lens"])
    ws = f.alloc_workspace(n_sel_max, dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    peak, peak_src = _peaks()
    tokens = int(sum(t["seq_lens"].cpu().tolist()))

    def timed(fn):
        ts = []
        for i in range(args.warmup + args.steps):
            flush.fill_(i & 1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            b.synchronize()
            if i >= args.warmup:
                ts.append(a.elapsed_time(b) * 1e3)
        return float(np.mean(ts))

    s1 = torch.zeros((B, Hs, Lm), dtype=torch.float32, device=dev)
    i1 = torch.zeros((B, Hs, n_sel_max), dtype=torch.int32, device=dev)
    n1 = torch.zeros((B, Hs), dtype=torch.int32, device=dev)
    o1 = torch.zeros((B, Hq, 128), dtype=torch.float32, device=dev)
    single = {"fc_score": timed(lambda: f.fc_score(t["q"], proxy, t["seq_lens"], s1)),
              "topk": timed(lambda: f.topk(s1, t["seq_lens"], w.budget, i1, n1, ws)),
              "sparse_attn": timed(lambda: f.sparse_decode_attn(t["q"], t["k"], t["v"], i1, n1, o1, ws))}
    rows = []
    for T in (1, 2, 4, 8):
        if T * w.heads_per_set > 64:
            continue
        q = torch.stack([synth.make_step_inputs(w, 40 + j, dev)["q"] for j in range(T)], dim=1).contiguous()
        sc = torch.zeros((B, T, Hs, Lm), dtype=torch.float32, device=dev)
        idx = torch.zeros((B, T, Hs, n_sel_max), dtype=torch.int32, device=dev)
        n_sel = torch.zeros((B, T, Hs), dtype=torch.int32, device=dev)
        out = torch.zeros((B, T, Hq, 128), dtype=torch.float32, device=dev)
        us = {"fc_score_batched": timed(lambda: f.fc_score_batched(q, proxy, t["seq_lens"], sc)),
              "topk_batched": timed(lambda: f.topk_batched(sc, t["seq_lens"], w.budget, idx, n_sel)),
              "sparse_attn_batched": timed(lambda: f.sparse_decode_attn_batched(q, t["k"], t["v"], idx, n_sel, out, ws)),
              "step_batched": timed(lambda: f.decode_step_batched(q, t["k"], t["v"], proxy, t["seq_lens"], w.budget, sc, idx, n_sel,
                                                                  out, ws))}
        sel = int(n_sel.sum().item())
        # scoring: the proxy once for all queries, one fp32 score per (query, set, token), the queries
        score_bytes = tokens * w.n_kv_heads * 4 * w.n_dom + 4 * tokens * Hs * T + B * T * Hq * 256
        flops = 2.0 * tokens * w.n_kv_heads * (2 * w.n_dom) * (w.group * T)
        step_bytes_ = tokens * w.n_kv_heads * 4 * w.n_dom + sel * 512 + B * T * Hq * 128 * 6
        rows.append({"q_len": T, "columns": T * w.heads_per_set, "us": us, "n_sel_per_query_unit": sel / (B * T * Hs),
                     "fc_score_batched": {"bytes": score_bytes, "gbs": score_bytes / us["fc_score_batched"] / 1e3,
                                          "frac": score_bytes / us["fc_score_batched"] / 1e3 / peak, "bound": "hbm",
                                          "tflops": flops / us["fc_score_batched"] / 1e6,
                                          "speedup_vs_q_len_single_calls": T * single["fc_score"] / us["fc_score_batched"]},
                     "step_batched": {"bytes_method": step_bytes_, "frac_method_bytes": step_bytes_ / us["step_batched"] / 1e3 / peak,
                                      "speedup_vs_q_len_single_steps": T * sum(single.values()) / us["step_batched"]},
                     "device_status": f.device_status()})
        del q, sc, idx, n_sel, out
    print(json.dumps({"batched_queries": w.name, "budget": w.budget, "n_dom": w.n_dom, "steps": args.steps, "peak_gbs": peak,
                      "peak_source": peak_src, "single_query_calls_us": single, "rows": rows}), flush=True)


def partial_total(samples, points, key, n_layers):
    """Seconds of the decode steps up to the last sampled context: per step n_layers x the step time,
    linearly interpolated between the samples taken so far."""
    acc = 0.0
    for L in range(1025, samples[len(points) - 1] + 1):
        j = 0
        while j + 1 < len(points) and samples[j + 1] <= L:
            j += 1
        if j == len(points) - 1:
            v = points[j][key]
        else:
            x0, x1 = samples[j], samples[j + 1]
            v = points[j][key] + (points[j + 1][key] - points[j][key]) * (L - x0) / (x1 - x0)
        acc += v * n_layers
    return acc * 1e-6


def run_longcot(args):
    """Workload c3 (long-CoT shape, Qwen2.5-7B-like attention): 28 layers, batch 32, prompt
    1024 then 15360 decode steps, budget 18.9 % of the current length, 16 dominant FCs.  One
    layer's step is timed at sampled cache lengths (FASA and dense); the whole run's decode time
    is the sum over steps of 28 x the step time, linearly interpolated between the samples."""
    import torch

    from paper_2602_03152_b200 import build, synth

    build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    w = synth.CONFIGS["c3"]
    t = synth.make_inputs(w.replace(len_lo=w.max_len, len_hi=w.max_len), dev)
    peak, _ = _peaks()
    samples = [1025, 2048, 4096, 6144, 8192, 10240, 12288, 14336, 16384]
    pts = []
    for L in samples:
        m = measure(w, args.sweep_steps, 3, dev, 1, args.step_mode, None, want_e2e=False, t=t, lens=[L] * w.batch)
        sm = summarize(m, peak)
        pts.append({"context": L, "n_sel_per_unit": sm["n_sel_per_unit"], "us_per_step": sm["us_per_step"],
                    "dense_us_per_step": sm["dense_us_per_step"], "step_frac_of_peak": sm["step_frac_of_peak"],
                    "dense_frac_of_peak": sm["dense_frac_of_peak"], "speedup_vs_dense": sm["speedup_vs_dense"],
                    "device_status": sm["device_status"]})
        del m
        # progress line (stderr): what a run that is cut short has measured so far
        done_steps = max(0, min(L, 1024 + 15360) - 1024)
        print(json.dumps({"longcot_progress": {"sampled_context": L, "decode_steps_covered": done_steps,
                                               "us_per_step": pts[-1]["us_per_step"],
                                               "dense_us_per_step": pts[-1]["dense_us_per_step"],
                                               "fasa_seconds_so_far": partial_total(samples, pts, "us_per_step", 28),
                                               "dense_seconds_so_far": partial_total(samples, pts, "dense_us_per_step", 28)}}),
              file=sys.stderr, flush=True)

    def total(points, key, n_layers):
        acc = 0.0
        for L in range(1025, 16385):              # cache length after each of the 15360 appends
            j = max(i for i, s_ in enumerate(samples) if s_ <= L)
            if j == len(samples) - 1:
                v = points[j][key]
            else:
                a, b = samples[j], samples[j + 1]
                v = points[j][key] + (points[j + 1][key] - points[j][key]) * (L - a) / (b - a)
            acc += v * n_layers
        return acc * 1e-6

    # the prompt's cache update: 1024 rows per (sequence, KV head) in one fasa_kv_append call
    # (K, V and the dominant slices), against the bytes it must move
    from paper_2602_03152_b200 import binding
    fpre = binding.Fasa.from_workload(w, t["dom"])
    ppre = fpre.alloc_proxy(dev)
    lens0 = torch.zeros(w.batch, dtype=torch.int32, device=dev)
    kn, vn = t["k"][:, :, :1024].contiguous(), t["v"][:, :, :1024].contiguous()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    tsp = []
    for i in range(8):
        flush.fill_(i & 1)
        lens0.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fpre.kv_append(t["k"], t["v"], ppre, lens0, kn, vn)
        b.record()
        b.synchronize()
        if i >= 3:
            tsp.append(a.elapsed_time(b) * 1e3)
    pre_bytes = w.batch * w.n_kv_heads * 1024 * (2 * 512 + 4 * w.n_dom)          # K, V read + written, proxy written
    prefill = {"rows_per_unit": 1024, "us_per_layer": sum(tsp) / len(tsp), "bytes": pre_bytes,
               "gbs": pre_bytes / (sum(tsp) / len(tsp)) / 1e3, "frac_of_peak": pre_bytes / (sum(tsp) / len(tsp)) / 1e3 / peak}
    del fpre, ppre, flush, kn, vn

    tf, td = total(pts, "us_per_step", 28), total(pts, "dense_us_per_step", 28)
    res = {"longcot": w.name, "layers": 28, "batch": w.batch, "prompt": 1024, "decode_steps": 15360,
           "budget_permille": -w.budget, "n_dom": w.n_dom, "steps_per_sample": args.sweep_steps,
           "fasa_decode_attention_seconds": tf, "dense_decode_attention_seconds": td,
           "speedup_vs_dense": td / tf, "theory_byte_ratio": 1.0 / (w.n_dom / 128.0 + 0.189),
           "method": "one layer timed at the sampled contexts (L2 flushed before each step), linear interpolation, x 28 layers",
           "prefill_kv_append": prefill, "samples": pts}
    del t
    free, _ = torch.cuda.mem_get_info()
    if free > (48 << 30) and not args.no_resident:
        rp, status = _longcot_resident(w, samples, max(3, args.sweep_steps // 2), dev)
        rf, rd = total(rp, "fasa_us_per_token_step", 1), total(rp, "dense_us_per_token_step", 1)
        res["resident_stack"] = {
            "method": "28 layers resident (own caches, ~32 GB), one token step of the whole stack replayed from a CUDA "
                      "graph at the sampled contexts, no L2 flush, linear interpolation over the 15360 steps",
            "fasa_decode_attention_seconds": rf, "dense_decode_attention_seconds": rd, "speedup_vs_dense": rd / rf,
            "device_status": status, "samples": rp}
    print(json.dumps(res), flush=True)


def cpu_baseline(w, m):
    """The fp64 oracle, as it stands, on the host: (1) timed on a bounded sample of the workload
    (the units of sequence 0, context cut to 32768 rows where longer), on all cores and on one;
    (2) one unit of the TIMED configuration at its full length, checked against the step's last
    outputs with the parity rules of the tests.  Returns the `cpu_baseline` and `parity` objects."""
    import math

    import numpy as np

    from oracle import fasa_oracle as O
    from oracle import parity as P
    from paper_2602_03152_b200 import synth

    t = m["t"]
    cores = os.cpu_count() or 1
    L = min(int(t["seq_lens"][0]), 32768)
    qb = synth.bf16_bits(t["q"][:1])
    kb = synth.bf16_bits(t["k"][:1, :, :L])
    vb = synth.bf16_bits(t["v"][:1, :, :L])
    lens = np.array([L], dtype=np.int32)
    dom = t["dom"].numpy()
    res = {}
    for label, threads, budget_s in (("all", cores, 10.0), ("one", 1, 6.0)):
        kw = dict(pairing=w.pairing, group_reduce=w.group_reduce, n_sink=w.n_sink, n_recent=w.n_recent,
                  budget=w.budget, n_sel_max=w.n_sel_max(), n_threads=threads, want_scores=False, want_dense=False)
        r = O.decode_bf16(qb, kb, vb, lens, dom, **kw)      # warm-up, page in
        reps, t0 = 0, time.perf_counter()
        while reps < 2 or (time.perf_counter() - t0 < budget_s and reps < 2000):
            r = O.decode_bf16(qb, kb, vb, lens, dom, **kw)
            reps += 1
        res[label] = ((time.perf_counter() - t0) / reps, int(r["threads"]), reps)
    sb = step_bytes(w.replace(batch=1), [L], int(r["n_sel"].sum()))
    dt, used, reps = res["all"]
    base = {"value": sb["fasa"] / dt / 1e9, "unit": UNIT, "cores": used, "kind": "oracle", "us_per_step_sample": dt * 1e6,
            "single_thread": {"value": sb["fasa"] / res["one"][0] / 1e9, "unit": UNIT, "cores": 1,
                              "us_per_step_sample": res["one"][0] * 1e6, "passes": res["one"][2]},
            "sample": f"{w.n_kv_heads} units of sequence 0 (context {L}"
                      + (f", cut from {int(t['seq_lens'][0])}" if L < int(t["seq_lens"][0]) else "")
                      + f") out of batch {w.batch}, {reps} passes"}

    # parity of the timed configuration: unit (sequence 0, index set 0) at its full length
    last = m["last"]
    G = w.heads_per_set
    h = 0
    Lf = int(t["seq_lens"][0])
    par = {"unit": [0, 0], "context": Lf, "ok": False}
    try:
        rep = P.check_step(t["q"][:1, :G].cpu().double().numpy(), t["k"][:1, :1, :Lf].cpu().double().numpy(),
                           t["v"][:1, :1, :Lf].cpu().double().numpy(), [Lf], np.sort(dom, axis=1)[h:h + 1], pairing=w.pairing,
                           group_reduce=w.group_reduce, n_sink=w.n_sink, n_recent=w.n_recent, budget=w.budget,
                           scale=1.0 / math.sqrt(128.0), idx=last["idx"][:1, :1].cpu().numpy(),
                           n_sel=last["n_sel"][:1, :1].cpu().numpy(), out=last["out"][:1, :G].cpu().numpy(),
                           sel_heads=w.sel_heads, what="bench")
        par.update(ok=True, index_set_identical=bool(rep["sets_identical"]), attn_max_abs_err=rep["attn_err"],
                   attn_tolerance=P.ATTN_ABS, n_sel=int(last["n_sel"][0, 0]),
                   rule="index set bit-exact outside the 1e-3 tie band; attention max-abs <= 2e-3 against the oracle on the GPU's set")
    except AssertionError as e:
        par["error"] = str(e)[:300]
    return {"cpu_baseline": base, "parity": par}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="fasa", choices=["fasa", "reference"])
    ap.add_argument("--config", default="c2", help="workload: c0, c1, c2 (default: the largest single-GPU one), c4")
    ap.add_argument("--budget", type=int, default=None)
    ap.add_argument("--n-dom", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch (profiling)")
    ap.add_argument("--select-heads", type=int, default=None,
                    help="query heads sharing one index set (default: all heads of a KV head; 1 = a set per head)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extras", default="c1,c4", help="other workloads reported under other_workloads (50 steps each)")
    ap.add_argument("--no-budget-row", action="store_true", help="skip configuration 4's budget row")
    ap.add_argument("--min-region-s", type=float, default=0.4,
                    help="repeat the block of --steps steps until the timed region has run this long on the device")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="config 4 grid (budget x dominant FCs) instead of the bench line")
    ap.add_argument("--longcot", action="store_true", help="config 3 (long-CoT decode) instead of the bench line")
    ap.add_argument("--calib", action="store_true",
                    help="offline calibration (Algorithm 1) on --config's shape instead of the bench line; --budget = top-k")
    ap.add_argument("--offload", action="store_true",
                    help="FASA-M (Algorithm 2): K/V caches in page-locked host memory, instead of the bench line")
    ap.add_argument("--paged", type=int, default=0, metavar="PAGE_SIZE",
                    help="paged caches with this page size (a power of two >= 16) against contiguous ones, instead of the bench line")
    ap.add_argument("--batched", action="store_true",
                    help="blocks of query tokens (q_len 1..8) on --config's shape instead of the bench line")
    ap.add_argument("--no-resident", action="store_true", help="--longcot: skip the 28-layer resident measurement")
    ap.add_argument("--sweep-steps", type=int, default=20)
    ap.add_argument("--step-mode", type=int, default=None, choices=[0, 1, 2],
                    help="0: fasa_decode_step as three kernels; 1 (default): one cluster kernel where available; "
                         "2: as 1, with the one-CTA-per-row kernel behind fasa_topk")
    args = ap.parse_args()

    if args.sweep:
        return run_sweep(args)
    if args.longcot:
        return run_longcot(args)
    if args.calib:
        return run_calib(args)
    if args.offload:
        return run_offload(args)
    if args.paged:
        return run_paged(args)
    if args.batched:
        return run_batched(args)
    from paper_2602_03152_b200 import synth
    w = synth.CONFIGS[args.config]
    if args.budget is not None:
        w = w.replace(budget=args.budget)
    if args.n_dom is not None:
        w = w.replace(n_dom=args.n_dom)
    if args.batch is not None:
        w = w.replace(batch=args.batch)
    if args.select_heads is not None:
        w = w.replace(sel_heads=args.select_heads)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_fasa(args, w)


if __name__ == "__main__":
    main()
