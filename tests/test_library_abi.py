"""CPU-side checks of the C-ABI library: it loads, exports every entry point
declared in include/deer.h, and rejects bad arguments on the host before any
launch.  No kernel runs here."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_15176_b200 import build
    build.build()
    from paper_2512_15176_b200 import binding
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "deer.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(deer_[a-z_]+)\s*\(", text))
    assert {"deer_block_attn", "deer_lmhead_select", "deer_accept", "deer_kv_commit"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} declared in deer.h but not exported"
    from paper_2512_15176_b200 import binding
    assert names == set(binding.EXPORTS)


def test_host_side_argument_validation(lib):
    from paper_2512_15176_b200 import binding as L
    kv = ctypes.c_void_p()
    desc = L.deer_kv_desc()
    assert lib.deer_kv_create(ctypes.byref(kv), ctypes.byref(desc)) == L.DEER_ERR_INVALID_ARG
    assert b"null" in lib.deer_last_error()
    fake = 0x1000          # never dereferenced on the host
    desc = L.deer_kv_desc(fake, fake, fake, fake, fake, fake, fake, fake, 4, 2, 96, 16, 1, 4)
    assert lib.deer_kv_create(ctypes.byref(kv), ctypes.byref(desc)) == L.DEER_ERR_UNSUPPORTED      # head_dim 96
    desc.head_dim = 128
    desc.page_size = 32
    assert lib.deer_kv_create(ctypes.byref(kv), ctypes.byref(desc)) == L.DEER_ERR_UNSUPPORTED      # page size
    desc.page_size = 16
    assert lib.deer_kv_create(ctypes.byref(kv), ctypes.byref(desc)) == L.DEER_OK
    try:
        # block larger than 32
        assert lib.deer_block_attn(kv, fake, fake, fake, fake, fake, 1, 33, 4, 0, 0, 1.0, 64, fake, 1 << 20, None) == L.DEER_ERR_UNSUPPORTED
        # Hq not a multiple of Hkv
        assert lib.deer_block_attn(kv, fake, fake, fake, fake, fake, 1, 8, 3, 0, 0, 1.0, 64, fake, 1 << 20, None) == L.DEER_ERR_INVALID_ARG
        # misaligned pointer
        assert lib.deer_block_attn(kv, fake, fake + 2, fake, fake, fake, 1, 8, 4, 0, 0, 1.0, 64, fake, 1 << 20, None) == L.DEER_ERR_INVALID_ARG
        # workspace too small
        need = lib.deer_block_attn_workspace_bytes(1, 8, 4, 2, 128, 64)
        assert need > 0
        assert lib.deer_block_attn(kv, fake, fake, fake, fake, fake, 1, 8, 4, 0, 0, 1.0, 64, fake, need - 1, None) == L.DEER_ERR_WORKSPACE
        # empty batch is a no-op
        assert lib.deer_block_attn(kv, fake, fake, fake, fake, fake, 0, 8, 4, 0, 0, 1.0, 64, None, 0, None) == L.DEER_OK
        assert lib.deer_kv_reserve(kv, fake, 0, 8, None) == L.DEER_OK
        assert lib.deer_kv_commit(kv, fake, fake, 0, 8, None) == L.DEER_OK
        # acceptance + commit in one launch: greedy only, empty batch is a no-op
        assert lib.deer_accept_commit(kv, fake, L.DEER_ACC_GREEDY, 0, 8, fake, fake, -1, fake, fake, fake, None) == L.DEER_OK
        assert lib.deer_accept_commit(kv, fake, L.DEER_ACC_SAMPLE, 4, 8, fake, fake, -1, fake, fake, fake, None) == L.DEER_ERR_UNSUPPORTED
        assert lib.deer_accept_commit(kv, fake, L.DEER_ACC_GREEDY, 4, 40, fake, fake, -1, fake, fake, fake, None) == L.DEER_ERR_UNSUPPORTED
        assert lib.deer_accept_commit(kv, None, L.DEER_ACC_GREEDY, 4, 8, fake, fake, -1, fake, fake, fake, None) == L.DEER_ERR_INVALID_ARG
        assert lib.deer_kv_reserve(kv, fake, 4, 40, None) == L.DEER_ERR_UNSUPPORTED
    finally:
        lib.deer_kv_destroy(kv)
    # LM head: hidden size not a multiple of 64, bad mode, missing outputs
    assert lib.deer_lmhead_select(fake, fake, 8, 100, 512, 0, 1.0, None, fake, None, None, None, None, fake, 1 << 20, None) == L.DEER_ERR_UNSUPPORTED
    assert lib.deer_lmhead_select(fake, fake, 8, 128, 512, 7, 1.0, None, fake, None, None, None, None, fake, 1 << 20, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_lmhead_select(fake, fake, 8, 128, 512, 2, 0.0, None, fake, None, fake, None, None, fake, 1 << 20, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_lmhead_select(fake, fake, 8, 128, 512, 1, 1.0, None, fake, None, None, None, None, fake, 1 << 20, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_lmhead_select(fake, fake, 0, 128, 512, 0, 1.0, None, fake, None, None, None, None, None, 0, None) == L.DEER_OK
    # acceptance: bad mode, k too large, sample mode without its inputs
    assert lib.deer_accept(5, 1, 8, 100, fake, fake, None, None, None, 1.0, None, None, None, -1, fake, fake, fake, None, 0, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_accept(0, 1, 64, 100, fake, fake, None, None, None, 1.0, None, None, None, -1, fake, fake, fake, None, 0, None) == L.DEER_ERR_UNSUPPORTED
    assert lib.deer_accept(1, 1, 8, 100, fake, None, None, None, None, 1.0, None, None, None, -1, fake, fake, fake, None, 0, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_accept(0, 0, 8, 100, fake, fake, None, None, None, 1.0, None, None, None, -1, fake, fake, fake, None, 0, None) == L.DEER_OK
    assert lib.deer_accept_workspace_bytes(0, 16, 32, 151936) == 0
    need = lib.deer_accept_workspace_bytes(1, 16, 32, 151936)
    assert 2 * 16 * 32 * 4 < need < (1 << 20)          # per-row statistics and per-slice sums; no copy of a vocabulary row
    # truncation: null outputs, non-positive temperature or top_p
    assert lib.deer_truncate(4, 100, fake, fake, 1.0, 5, 0.9, None, fake, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_truncate(4, 100, fake, fake, 0.0, 5, 0.9, fake, fake, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_truncate(4, 100, fake, fake, 1.0, 5, 0.0, fake, fake, None) == L.DEER_ERR_INVALID_ARG
    assert lib.deer_truncate(0, 100, fake, fake, 1.0, 5, 0.9, fake, fake, None) == L.DEER_OK


def test_workload_is_deterministic_and_shaped():
    import numpy as np
    from paper_2512_15176_b200 import workload as W
    c = W.config(0)
    a, b = W.hidden(c), W.hidden(c)
    assert a.shape == (8, 512) and (a == b).all()
    assert abs(float(a.float().std()) - 1.0) < 0.05
    c4 = W.config(3)
    n = W.seq_lengths(c4)
    assert n.shape == (16,) and n.min() >= 2048 and n.max() <= 16384 and len(set(n.tolist())) > 8
    L = W.planted_prefix_lengths(W.config(1).with_(B=4000))
    assert 6.0 < L.mean() < 10.0 and L.max() == 32 and (L == 32).mean() > 0.02      # decaying law with mass at the cap
    u = W.uniform_open(1, "u", (1000,)).numpy()
    assert u.min() > 0 and u.max() < 1 and u.dtype == np.float32
    s = W.sweep_config(4, 4096, 16, W.MASK_BIDIR)
    assert s.ctx == (2048, 4096) and s.growth == 64 * 16
