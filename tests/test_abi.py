"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, sizes workspaces, validates configurations and reports errors."""
import ctypes as C
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def im():
    from paper_2605_25475_b200 import buildlib
    buildlib.build()
    from paper_2605_25475_b200 import binding
    return binding


def declared_functions():
    src = open(os.path.join(ROOT, "include", "indexmem.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(im_[a-z_0-9]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(im):
    names = declared_functions()
    assert {"im_create", "im_prefill_chunk", "im_decode_step", "im_destroy"} <= set(names)
    lib = C.CDLL(im.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), f"{n} declared in indexmem.h but not exported"
    assert set(names) == set(im.EXPORTED)


def test_workspace_bytes_and_validation(im):
    cfg = im.Config(n_layers=2, max_seqs=3, n_q_heads=8, n_kv_heads=2, head_dim=64, budget=128, max_chunk=256)
    nbytes = im.im_workspace_bytes(cfg.to_c())
    # at least the K/V slabs: 2 * units * Hkv * cap * d * 2 bytes, cap = 128 + 256
    assert nbytes >= 2 * 6 * 2 * 384 * 64 * 2
    assert nbytes % 256 == 0
    bigger = im.im_workspace_bytes(im.Config(n_layers=2, max_seqs=3, n_q_heads=8, n_kv_heads=2, head_dim=64,
                                             budget=256, max_chunk=256).to_c())
    assert bigger > nbytes
    bad = [dict(n_q_heads=7), dict(head_dim=60), dict(budget=4, n_sink=4), dict(compress_interval=0),
           dict(n_layers=0), dict(act=2), dict(lambda_=1.5), dict(pending_slots=100)]
    for kw in bad:
        base = dict(n_layers=1, max_seqs=1, n_q_heads=8, n_kv_heads=2, head_dim=64, budget=128)
        base.update(kw)
        assert im.im_workspace_bytes(im.Config(**base).to_c()) == 0, kw


def test_config_struct_layout(im):
    # 19 int32, 6 float, padding to 8, one uint64
    assert C.sizeof(im.im_config) == 112
    assert im.im_config.seed.offset == 104 and im.im_config.score_share.offset == 68 and im.im_config.scorer.offset == 72


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device error path")
def test_create_without_device_fails_loudly(im):
    cfg = im.Config(n_layers=1, max_seqs=1, n_q_heads=4, n_kv_heads=1, head_dim=64, budget=16).to_c()
    h = C.c_void_p()
    rc = im._lib.im_create(C.byref(cfg), C.c_void_p(0x10000), 1 << 40, C.byref(h))
    assert rc == im.IM_ERR_CUDA and not h.value
    assert im._lib.im_last_error().decode() != ""
    rc = im._lib.im_create(C.byref(cfg), C.c_void_p(0x10001), 1 << 40, C.byref(h))
    assert rc == im.IM_ERR_ARG
