"""Shared helper of the GPU parity tests: run the CUDA path on one workload through the
Python binding (hence the C ABI) and hand numpy copies to the oracle-side checks."""
import math

import numpy as np
import torch

from paper_2602_03152_b200 import binding, build, synth

SENTINEL = 12345.0


def ensure_built():
    build.build()
    return binding.load_library()


class Run:
    """Device state for one workload, with every output buffer pre-filled by sentinels."""

    def __init__(self, w: synth.Workload, t=None, n_sel_max=None, dev="cuda"):
        ensure_built()
        self.w = w
        self.t = t if t is not None else synth.make_inputs(w, "cpu")
        self.q = self.t["q"].to(dev)
        self.k = self.t["k"].to(dev)
        self.v = self.t["v"].to(dev)
        self.seq_lens = self.t["seq_lens"].to(dev)
        self.dom = self.t["dom"]
        self.fasa = binding.Fasa.from_workload(w, self.dom)
        self.n_sel_max = n_sel_max if n_sel_max is not None else w.n_sel_max()
        B, Hq, Hs, Lm = w.batch, w.n_q_heads, w.n_sets, w.max_len      # Hs index sets per sequence
        assert self.fasa.n_sets == Hs
        self.proxy = self.fasa.alloc_proxy(dev)
        self.scores = torch.full((B, Hs, Lm), SENTINEL, dtype=torch.float32, device=dev)
        self.idx = torch.full((B, Hs, self.n_sel_max), -7, dtype=torch.int32, device=dev)
        self.n_sel = torch.full((B, Hs), -7, dtype=torch.int32, device=dev)
        self.out = torch.full((B, Hq, 128), SENTINEL, dtype=torch.float32, device=dev)
        self.lse = torch.full((B, Hq), SENTINEL, dtype=torch.float32, device=dev)
        self.dense = torch.full((B, Hq, 128), SENTINEL, dtype=torch.float32, device=dev)
        self.dense_lse = torch.full((B, Hq), SENTINEL, dtype=torch.float32, device=dev)
        self.ws = self.fasa.alloc_workspace(self.n_sel_max, dev)

    def build_proxy(self):
        self.fasa.proxy_build(self.k, self.proxy, self.seq_lens)

    def reset_outputs(self):
        self.scores.fill_(SENTINEL)
        self.idx.fill_(-7)
        self.n_sel.fill_(-7)
        self.out.fill_(SENTINEL)
        self.lse.fill_(SENTINEL)

    def step(self, budget=None, fused=False):
        """The three calls one after another, or fasa_decode_step as one cluster kernel."""
        budget = self.w.budget if budget is None else budget
        f = self.fasa
        if fused:
            assert f.step_cluster_size() > 0, "the one-launch step is not available for this configuration"
            n0 = f.launch_count()
            f.decode_step(self.q, self.k, self.v, self.proxy, self.seq_lens, budget, self.scores, self.idx,
                          self.n_sel, self.out, None, self.lse)
            assert f.launch_count() == n0 + 1
        else:
            f.fc_score(self.q, self.proxy, self.seq_lens, self.scores)
            f.topk(self.scores, self.seq_lens, budget, self.idx, self.n_sel, self.ws)
            f.sparse_decode_attn(self.q, self.k, self.v, self.idx, self.n_sel, self.out, self.ws, self.lse)
        torch.cuda.synchronize()

    def dense_step(self):
        self.fasa.full_decode_attn(self.q, self.k, self.v, self.seq_lens, self.dense, self.ws, self.dense_lse)
        torch.cuda.synchronize()

    def host(self):
        """float64 widenings of the inputs plus numpy copies of the outputs."""
        return dict(
            q=self.t["q"].double().numpy(), k=self.t["k"].double().numpy(), v=self.t["v"].double().numpy(),
            seq_lens=self.t["seq_lens"].numpy(), dom=np.sort(self.dom.numpy(), axis=1),
            scores=self.scores.cpu().numpy(), idx=self.idx.cpu().numpy(), n_sel=self.n_sel.cpu().numpy(),
            out=self.out.cpu().numpy(), lse=self.lse.cpu().numpy(), dense=self.dense.cpu().numpy(),
            dense_lse=self.dense_lse.cpu().numpy())

    def oracle_kwargs(self, budget=None):
        w = self.w
        return dict(pairing=w.pairing, group_reduce=w.group_reduce, n_sink=w.n_sink, n_recent=w.n_recent,
                    budget=w.budget if budget is None else budget, scale=1.0 / math.sqrt(128.0),
                    sel_heads=w.sel_heads)
