"""CPU-only checks of the C-ABI boundary: the library builds, loads and exports every
symbol include/fasa.h declares, and argument validation answers before any GPU work."""
import ctypes
import os
import re

import pytest

from paper_2602_03152_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load_library()


def test_header_and_binding_list_the_same_entry_points(lib):
    header = open(os.path.join(ROOT, "include", "fasa.h")).read()
    declared = set(re.findall(r"\b(fasa_[a-z_0-9]+)\s*\(", header))
    declared -= {"fasa_ctx_t", "fasa_config_t"}
    assert declared == set(binding.SYMBOLS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings_and_row_elems(lib):
    assert lib.fasa_status_string(0) == b"ok"
    for st in (-1, -2, -3, -4, -5):
        assert lib.fasa_status_string(st) not in (b"ok", b"unknown status")
    assert lib.fasa_status_string(99) == b"unknown status"
    assert [lib.fasa_proxy_row_elems(f) for f in (1, 4, 5, 8, 16, 17, 64)] == [8, 8, 16, 16, 32, 40, 128]
    assert lib.fasa_proxy_row_elems(0) == 0 and lib.fasa_proxy_row_elems(65) == 0


def _cfg(**kw):
    base = dict(batch=1, n_q_heads=4, n_kv_heads=1, head_dim=128, max_len=64, n_dom=2, rope_pairing=0,
                group_reduce=0, select_heads=0, n_sink=0, n_recent=0, softmax_scale=0.0, page_size=0, n_pages=0)
    base.update(kw)
    return binding.FasaConfig(base["batch"], base["n_q_heads"], base["n_kv_heads"], base["head_dim"],
                              base["max_len"], base["n_dom"], base["rope_pairing"], base["group_reduce"],
                              base["select_heads"], base["n_sink"], base["n_recent"], base["softmax_scale"], 0, 0, 0, 0, 0, 0,
                              base["page_size"], base["n_pages"])


@pytest.mark.parametrize("kw,expect", [
    (dict(batch=0), binding.ERR_INVALID_ARG),
    (dict(max_len=-5), binding.ERR_INVALID_ARG),
    (dict(n_sink=-1), binding.ERR_INVALID_ARG),
    (dict(head_dim=64), binding.ERR_UNSUPPORTED),
    (dict(n_dom=0), binding.ERR_UNSUPPORTED),
    (dict(n_dom=65), binding.ERR_UNSUPPORTED),
    (dict(n_q_heads=5, n_kv_heads=2), binding.ERR_UNSUPPORTED),
    (dict(n_q_heads=9, n_kv_heads=1), binding.ERR_UNSUPPORTED),
    (dict(rope_pairing=2), binding.ERR_UNSUPPORTED),
    (dict(group_reduce=3), binding.ERR_UNSUPPORTED),
    (dict(select_heads=3), binding.ERR_UNSUPPORTED),      # does not divide the group of 4
    (dict(select_heads=-1), binding.ERR_UNSUPPORTED),
    (dict(page_size=24, n_pages=4), binding.ERR_UNSUPPORTED),   # not a power of two
    (dict(page_size=8, n_pages=4), binding.ERR_UNSUPPORTED),    # smaller than a 16-token proxy tile
    (dict(page_size=16, n_pages=0), binding.ERR_UNSUPPORTED),   # an empty pool
])
def test_create_rejects_bad_config_without_a_gpu(lib, kw, expect):
    cfg = _cfg(**kw)
    dom = (ctypes.c_int32 * 64)(*range(64))
    h = ctypes.c_void_p()
    assert lib.fasa_create(ctypes.byref(cfg), ctypes.cast(dom, ctypes.c_void_p), ctypes.byref(h)) == expect
    assert not h.value


def test_create_rejects_bad_fc_lists_and_nulls(lib):
    h = ctypes.c_void_p()
    cfg = _cfg()
    for bad in ([3, 3], [0, 64], [-1, 2]):
        dom = (ctypes.c_int32 * 2)(*bad)
        assert lib.fasa_create(ctypes.byref(cfg), ctypes.cast(dom, ctypes.c_void_p), ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.fasa_create(None, None, ctypes.byref(h)) == binding.ERR_INVALID_ARG
    assert lib.fasa_destroy(None) == binding.ERR_INVALID_ARG
    assert lib.fasa_fc_score(None, None, None, None, None, None) == binding.ERR_INVALID_ARG
    assert lib.fasa_topk(None, None, None, 1, 1, None, None, None, None) == binding.ERR_INVALID_ARG
    assert lib.fasa_launch_count(None) == 0


def test_calib_select_is_host_only_and_agrees_with_the_oracle(lib):
    # Stage 2 of Algorithm 1 runs on the host: random counts with many equal sums (ties keep
    # the lower FC), compared with the oracle's separate statement of the same rule
    import numpy as np
    import torch
    from oracle import fasa_oracle as O
    rng = np.random.default_rng(3)
    Hq, Hkv, top_k = 28, 4, 64
    counts = rng.integers(0, 6, (Hq, 64)).astype(np.int64) * 10
    used = rng.integers(1, 5, Hq).astype(np.int64)
    for n_dom in (1, 16, 63, 64):
        dom, mean = binding.calib_select(torch.from_numpy(counts), torch.from_numpy(used), Hkv, top_k, n_dom)
        dom_or, mean_or = O.select_dominant(counts, used, Hkv, top_k, n_dom)
        assert np.array_equal(dom.numpy(), dom_or)
        assert np.allclose(mean.numpy(), mean_or, rtol=1e-15, atol=0)
    with pytest.raises(binding.FasaError):
        binding.calib_select(torch.from_numpy(counts), torch.from_numpy(used), Hkv, top_k, 65)
    with pytest.raises(binding.FasaError):
        binding.calib_select(torch.from_numpy(counts), torch.from_numpy(used), 5, top_k, 4)
