"""Host-side checks of the CUDA library that need no GPU: it loads, exports what the header declares,
and its host-only entry points validate their arguments."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2503_05931_b200 import build_ext, binding
    build_ext.build()
    return binding.load_library()


def test_exports_every_declared_symbol(lib):
    from paper_2503_05931_b200 import binding
    header = open(os.path.join(ROOT, "include", "aed_dec.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(aed_dec_[a-z_]+)\s*\(", header))
    assert {"aed_dec_create", "aed_dec_precompute_cross_kv", "aed_dec_step", "aed_dec_greedy_decode",
            "aed_dec_destroy"} <= declared
    raw = C.CDLL(binding.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert declared == set(binding.EXPORTED_SYMBOLS)


def test_workspace_bytes_and_validation(lib):
    from paper_2503_05931_b200 import binding, workloads
    model = workloads.MODELS["canary24"]
    cfg = binding.make_config(model, "bf16", max_batch=64, max_total_enc_frames=9000, max_enc_len=500, max_dec_len=240)
    need = binding.workspace_bytes(cfg)
    # at least the two K/V stores: self 24*64*2*1024*240*2 B, cross 24*2*1024*9000*2 B
    assert need >= 24 * 64 * 2 * 1024 * 240 * 2 + 24 * 2 * 1024 * 9000 * 2
    assert need < 8e9
    cfg32 = binding.make_config(model, "fp32", max_batch=64, max_total_enc_frames=9000, max_enc_len=500, max_dec_len=240)
    assert binding.workspace_bytes(cfg32) > need
    bad = binding.make_config(dict(model, n_heads=10), "bf16", max_batch=1, max_total_enc_frames=10, max_enc_len=10, max_dec_len=4)
    assert binding.workspace_bytes(bad) == 0
    assert lib.aed_dec_workspace_bytes(None) == 0
    # argument validation happens before any CUDA call
    assert lib.aed_dec_create(None, None, None) == binding.AED_ERR_INVALID_ARG
    handle = C.c_void_p()
    w = binding.AedWeights()
    assert lib.aed_dec_create(C.byref(bad), C.byref(w), C.byref(handle)) == binding.AED_ERR_UNSUPPORTED
    assert b"head_dim" in lib.aed_dec_create_error()
    assert lib.aed_dec_create(C.byref(cfg), C.byref(w), C.byref(handle)) == binding.AED_ERR_INVALID_ARG   # no workspace
    assert lib.aed_dec_step(None, None, None, None, None) == binding.AED_ERR_INVALID_ARG
    assert lib.aed_dec_greedy_decode(None, None, None, None) == binding.AED_ERR_INVALID_ARG
    assert lib.aed_dec_launch_count(None) == 0
    lib.aed_dec_destroy(None)


def test_bucketing_reduces_padding():
    from paper_2503_05931_b200 import bucketing, workloads
    w = workloads.make_workload("cfg5", with_weights=False, with_enc=False)
    assert w.batch == 4096
    rng = np.random.default_rng(0)
    rand = bucketing.random_batches(w.batch, 128, rng)
    buck = bucketing.bucket_batches_2d(w.enc_lens, w.dec_lens)
    for batches in (rand, buck):
        seen = np.sort(np.concatenate(batches))
        assert np.array_equal(seen, np.arange(w.batch))
    pe_r, pd_r = bucketing.padding_fractions(w.enc_lens, w.dec_lens, rand)
    pe_b, pd_b = bucketing.padding_fractions(w.enc_lens, w.dec_lens, buck)
    # random batches pad well over half of both rectangles (the paper's fixed batches: 57 % / 59 %);
    # 8 x 4 quantile buckets remove most of it (the paper's finer 30 x 2 buckets: 4.5 % / 19 %)
    assert pe_r > 0.5 and pd_r > 0.5
    assert pe_b < 0.3 and pd_b < 0.3 and pe_b < pe_r / 2 and pd_b < pd_r / 2
    for b in buck:
        assert len(b) * (w.enc_lens[b].max() + w.dec_lens[b].max()) <= 65536 or len(b) == 1
