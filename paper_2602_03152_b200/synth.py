"""Seeded synthetic inputs for the FASA decode path.

This module only draws inputs (shapes, value distributions, RoPE'd keys and
queries, dominant-FC lists, ragged lengths).  It holds none of the method's
arithmetic (no scoring, selection or attention) and imports neither the CUDA
binding nor the CPU oracle; both sides read the tensors it returns.

The tensors stand in for real model activations: shapes follow the model
families the paper evaluates (Llama-3-8B-like 32/8 heads, Qwen2.5-7B-like 28/4
heads, head_dim 128, N_tip = 16, long-CoT decode lengths), values follow a
recipe that gives keys a per-channel scale spread and a few outlier channels.

Recipe (per workload, seed = 20260203 + workload index):
  * channel scales s_c = exp(N(0, 0.5^2)), one vector for K and Q, one for V;
  * K pre-RoPE = N(0,1) * s_c, two seeded outlier channels multiplied by 8
    (independently for V); Q pre-RoPE = N(0,1) * s_c;
  * RoPE (theta_i = base^(-2i/d)) in fp64 at positions 0..L_max-1 for K and at
    position L_b for the query of sequence b, then round to bf16;
  * workloads marked `rope=False` use N(0,1) bf16 tensors as they are;
  * dominant FCs: F distinct indices per KV head, sampled without replacement
    with weight (i+1)^2 (biased to slow-turning FCs) or uniformly.
Rows at and beyond L_b hold ordinary random data: a reader that runs past the
sequence length produces wrong results instead of zeros.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import torch

BASE_SEED = 20260203


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    index: int                 # seed offset
    batch: int
    n_q_heads: int
    n_kv_heads: int
    max_len: int               # rows allocated per (b, kv head)
    len_lo: int                # sequence lengths are uniform in [len_lo, len_hi]
    len_hi: int
    n_dom: int                 # F = N_tip, dominant FCs per KV head
    budget: int                # N_fac (>0 absolute, <0 = -permille of the length)
    n_sink: int = 0
    n_recent: int = 0
    head_dim: int = 128
    rope_base: float = 500000.0
    pairing: int = 0           # 0 rotate-half (i, i+d/2); 1 interleaved (2i, 2i+1)
    rope: bool = True
    dom_bias: bool = True      # weight (i+1)^2 when True, uniform otherwise
    group_reduce: int = 0
    sel_heads: int = 0         # query heads sharing one index set; 0 = all heads of a KV head

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    @property
    def heads_per_set(self) -> int:
        return self.sel_heads if self.sel_heads > 0 else self.group

    @property
    def n_sets(self) -> int:
        """Index sets (selection units) per sequence."""
        return self.n_q_heads // self.heads_per_set

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)

    def n_sel_max(self) -> int:
        k = self.budget if self.budget > 0 else (-self.budget * self.max_len + 999) // 1000
        return min(self.max_len, k + self.n_sink + self.n_recent)


# The five benchmark shapes.  c3 describes one layer of the long-CoT run; the
# driver loop appends a token per step.
CONFIGS: Dict[str, Workload] = {
    "c0": Workload("c0_single_head_4k", 0, 1, 4, 1, 4096, 4096, 4096, 8, 256, dom_bias=False),
    "c1": Workload("c1_llama3_8b_32k", 1, 1, 32, 8, 32768, 32768, 32768, 16, 256, 4, 64),
    "c2": Workload("c2_batch16_ragged_128k", 2, 16, 32, 8, 131072, 65536, 131072, 16, 1024),
    "c3": Workload("c3_longcot_qwen7b_layer", 3, 32, 28, 4, 16384, 1024, 1024, 16, -189,
                   rope=False),
    "c4": Workload("c4_sweep_llama3_8b_64k", 4, 8, 32, 8, 65536, 65536, 65536, 16, 256),
}


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def dominant_fcs(w: Workload) -> torch.Tensor:
    """int32 [n_kv_heads, n_dom]: distinct FC indices per KV head (unsorted, CPU)."""
    g = _gen(BASE_SEED + w.index + 7919, "cpu")
    n_fc = w.head_dim // 2
    if w.n_dom >= n_fc:
        return torch.arange(n_fc, dtype=torch.int32).repeat(w.n_kv_heads, 1)
    i = torch.arange(n_fc, dtype=torch.float64)
    wt = (i + 1.0) ** 2 if w.dom_bias else torch.ones(n_fc, dtype=torch.float64)
    rows = [torch.multinomial(wt, w.n_dom, replacement=False, generator=g) for _ in range(w.n_kv_heads)]
    return torch.stack(rows).to(torch.int32)


def seq_lens(w: Workload) -> torch.Tensor:
    """int32 [batch] lengths, uniform in [len_lo, len_hi] (CPU)."""
    g = _gen(BASE_SEED + w.index + 104729, "cpu")
    if w.len_lo == w.len_hi:
        return torch.full((w.batch,), w.len_lo, dtype=torch.int32)
    return torch.randint(w.len_lo, w.len_hi + 1, (w.batch,), generator=g, dtype=torch.int64).to(torch.int32)


def rope_rotate(x: torch.Tensor, pos: torch.Tensor, base: float, pairing: int) -> torch.Tensor:
    """Rotate FC i of x[..., d] (fp64) by pos * base^(-2i/d); pos broadcasts over x[..., 0]."""
    d = x.shape[-1]
    i = torch.arange(d // 2, dtype=torch.float64, device=x.device)
    theta = torch.exp(-2.0 * i / d * math.log(base))
    ang = pos.to(torch.float64).unsqueeze(-1) * theta
    c, s = torch.cos(ang), torch.sin(ang)
    if pairing == 0:
        x0, x1 = x[..., : d // 2], x[..., d // 2:]
        return torch.cat([x0 * c - x1 * s, x0 * s + x1 * c], dim=-1)
    x0, x1 = x[..., 0::2], x[..., 1::2]
    out = torch.empty_like(x)
    out[..., 0::2] = x0 * c - x1 * s
    out[..., 1::2] = x0 * s + x1 * c
    return out


def channel_profile(w: Workload):
    """(s_k [d], s_v [d]) fp64 per-channel scales incl. the x8 outlier channels (CPU)."""
    g = _gen(BASE_SEED + w.index, "cpu")
    d = w.head_dim
    s_k = torch.exp(0.5 * torch.randn(d, generator=g, dtype=torch.float64))
    s_v = torch.exp(0.5 * torch.randn(d, generator=g, dtype=torch.float64))
    out_k = torch.randperm(d, generator=g)[:2]
    out_v = torch.randperm(d, generator=g)[:2]
    s_q = s_k.clone()
    s_k = s_k.clone()
    s_k[out_k] *= 8.0
    s_v[out_v] *= 8.0
    return s_q, s_k, s_v


def make_inputs(w: Workload, device="cpu", lens: Optional[torch.Tensor] = None) -> Dict[str, torch.Tensor]:
    """Draw one workload.

    Returns q bf16 [B,Hq,d], k/v bf16 [B,Hkv,max_len,d] (post-RoPE keys), seq_lens
    int32 [B], dom int32 [Hkv,F] (all on `device` except `dom`, which stays on the
    CPU for the context constructor).  Values depend on the device kind because
    CPU and CUDA generators differ: a comparison copies one draw to both sides.
    """
    dev = torch.device(device)
    B, Hq, Hkv, d, Lm = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.max_len
    lens = seq_lens(w) if lens is None else lens.to(torch.int32).cpu()
    s_q, s_k, s_v = (t.to(dev) for t in channel_profile(w))
    g = _gen(BASE_SEED + w.index + 15485863, dev)

    k = torch.empty((B, Hkv, Lm, d), dtype=torch.bfloat16, device=dev)
    v = torch.empty((B, Hkv, Lm, d), dtype=torch.bfloat16, device=dev)
    q = torch.empty((B, Hq, d), dtype=torch.bfloat16, device=dev)
    pos = torch.arange(Lm, dtype=torch.float64, device=dev)
    # Chunk the fp64 work so the largest workload stays within a few GB of scratch.
    rows = max(1, min(Lm, (1 << 24) // d))
    for b in range(B):
        for h in range(Hkv):
            for r0 in range(0, Lm, rows):
                r1 = min(Lm, r0 + rows)
                kk = torch.randn((r1 - r0, d), generator=g, dtype=torch.float32, device=dev).to(torch.float64)
                vv = torch.randn((r1 - r0, d), generator=g, dtype=torch.float32, device=dev).to(torch.float64)
                if w.rope:
                    kk = rope_rotate(kk * s_k, pos[r0:r1], w.rope_base, w.pairing)
                    vv = vv * s_v
                k[b, h, r0:r1] = kk.to(torch.bfloat16)
                v[b, h, r0:r1] = vv.to(torch.bfloat16)
        qq = torch.randn((Hq, d), generator=g, dtype=torch.float32, device=dev).to(torch.float64)
        if w.rope:
            qpos = torch.full((Hq,), float(lens[b]), dtype=torch.float64, device=dev)
            qq = rope_rotate(qq * s_q, qpos, w.rope_base, w.pairing)
        q[b] = qq.to(torch.bfloat16)
    return {"q": q, "k": k, "v": v, "seq_lens": lens.to(dev), "dom": dominant_fcs(w)}


def make_step_inputs(w: Workload, step: int, device="cpu") -> Dict[str, torch.Tensor]:
    """New-token tensors for one decode step: q [B,Hq,d], k_new/v_new [B,Hkv,1,d] (bf16)."""
    dev = torch.device(device)
    g = _gen(BASE_SEED + w.index + 32452843 + 1000003 * (step + 1), dev)
    B, Hq, Hkv, d = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    q = torch.randn((B, Hq, d), generator=g, dtype=torch.float32, device=dev).to(torch.bfloat16)
    kn = torch.randn((B, Hkv, 1, d), generator=g, dtype=torch.float32, device=dev).to(torch.bfloat16)
    vn = torch.randn((B, Hkv, 1, d), generator=g, dtype=torch.float32, device=dev).to(torch.bfloat16)
    return {"q": q, "k_new": kn, "v_new": vn}


def bf16_bits(t: torch.Tensor):
    """uint16 numpy view of a bf16 tensor's bit patterns (copied to the host)."""
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view("uint16")


def shard_units(n_units: int, rank: int, world: int) -> List[int]:
    """Contiguous, balanced slice of independent (batch, KV head) units for one rank."""
    base, rem = divmod(n_units, world)
    lo = rank * base + min(rank, rem)
    hi = lo + base + (1 if rank < rem else 0)
    return list(range(lo, hi))
