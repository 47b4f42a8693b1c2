"""fasa_sparse_decode_attn_static: the sparse-attention call for callers that cannot give the
library a workspace (no cudaMalloc available to them), whose split-K partials live in a fixed
array inside the library.  Called through the C ABI twice in a row and compared with
fasa_sparse_decode_attn on the same inputs.  Collected last on purpose (file name)."""
import numpy as np
import pytest
import torch

from paper_2602_03152_b200 import binding, synth

from gpu_harness import SENTINEL, Run

pytestmark = pytest.mark.gpu

ATTN_ABS = 2e-3   # the attention tolerance of the parity tests


def test_static_scratch_variant_matches_workspace_variant_twice():
    w = synth.CONFIGS["c1"].replace(max_len=6000, len_lo=5000, len_hi=5000, budget=700)
    r = Run(w)
    r.build_proxy()
    r.step()                                   # fills idx / n_sel and the reference out / lse
    ref_out, ref_lse = r.out.clone(), r.lse.clone()
    assert torch.isfinite(ref_out).all()
    for call in range(2):
        if call == 1:
            # a different query and selection for the second call: the array keeps the first
            # call's contents and nothing of them may leak into this result
            s = synth.make_step_inputs(w, 3, "cuda")
            r.q = s["q"]
            r.step(budget=300)
            ref_out, ref_lse = r.out.clone(), r.lse.clone()
        out = torch.full_like(r.out, SENTINEL)
        lse = torch.full_like(r.lse, SENTINEL)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        r.fasa.sparse_decode_attn_static(r.q, r.k, r.v, r.idx, r.n_sel, out, lse)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert r.fasa.device_status() == 0
        if call == 1:
            # (the first call on a device may load the library's module, which is where the
            # array lives; from the second call on nothing on the device may change size)
            assert free_after == free_before
        assert float((out - ref_out).abs().max()) <= ATTN_ABS
        assert float((lse - ref_lse).abs().max()) <= ATTN_ABS
        # both variants run the same kernels with the same split plan: anything of the first
        # call's partials leaking into the second would show as a difference in the bits
        assert torch.equal(out, ref_out) and torch.equal(lse, ref_lse)


def test_static_scratch_variant_rejects_what_does_not_fit():
    # 64 sequences x 64 query heads x many splits: more partials than the fixed array holds
    dom = torch.arange(4, dtype=torch.int32).repeat(8, 1)
    f = binding.Fasa(64, 64, 8, 65536, dom)
    n_sel_max = 65536
    q = torch.zeros((64, 64, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(16, dtype=torch.bfloat16, device="cuda")       # never read: the call must refuse first
    idx = torch.zeros(16, dtype=torch.int32, device="cuda")
    out = torch.zeros((64, 64, 128), dtype=torch.float32, device="cuda")
    st = f._lib.fasa_sparse_decode_attn_static(f._h, q.data_ptr(), kv.data_ptr(), kv.data_ptr(), idx.data_ptr(),
                                               idx.data_ptr(), n_sel_max, out.data_ptr(), None, None)
    assert st == binding.ERR_WORKSPACE
    torch.cuda.synchronize()
