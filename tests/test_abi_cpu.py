"""The C-ABI library loads and exports every symbol include/kvs.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2609_35750_b200 import build, binding
    build.build()
    return binding.load()


def _declared():
    text = open(os.path.join(ROOT, "include", "kvs.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kvs_[a-z0-9_]+)\s*\(", text)))


def test_header_symbols_exported_and_bound(lib):
    from paper_2609_35750_b200 import binding
    names = _declared()
    assert "kvs_mask_meta" in names and "kvs_attn_fwd" in names and "kvs_attn_bwd" in names
    for n in names:
        assert hasattr(lib, n), n
        assert n in binding.SIGNATURES, f"{n} has no ctypes signature"
    assert sorted(binding.SIGNATURES) == names


def test_strerror_and_size_queries(lib):
    from paper_2609_35750_b200 import binding as B
    assert B.strerror(0) == "ok"
    for c in range(-8, 0):
        assert B.strerror(c) and "unknown" not in B.strerror(c)
    assert "unknown" in B.strerror(-99)
    assert B.kvs_mask_meta_bytes(-1, 10, 10) == 0
    a = B.kvs_mask_meta_bytes(1, 1024, 1024)
    b = B.kvs_mask_meta_bytes(2, 131072, 65536)
    assert 0 < a < b and a % 256 == 0
    # classes (1 B) + row lists (2 B) for 2 x 512^2 tiles dominate
    assert b >= 3 * 2 * 512 * 512
    # max_seqlen larger than the batch is clamped
    assert B.kvs_mask_meta_bytes(1, 1024, 10**6) == a
    w16 = B.kvs_attn_bwd_workspace_bytes(1024, 4, 4, 64, B.GRAD_BF16)
    w32 = B.kvs_attn_bwd_workspace_bytes(1024, 4, 4, 64, B.GRAD_FP32)
    assert w16 >= 1024 * 4 * 64 * 4 + 1024 * 4 * 4 and 0 < w32 < w16
    assert B.kvs_attn_bwd_workspace_bytes(1024, 4, 4, 64, 7) == 0
    assert B.kvs_host_arena_bytes(1, 1024, 1024, 4, 4, 64, B.GRAD_BF16) > w16


def test_host_side_argument_errors_need_no_gpu(lib):
    from paper_2609_35750_b200 import binding as B
    # null pointers / bad dims are rejected before any CUDA call
    assert lib.kvs_mask_meta(None, None, 1, 128, 128, None, 0, None) == B.KVS_ERR_INVALID_ARG
    assert lib.kvs_attn_fwd(None, None, None, None, 1, 128, 128, 4, 4, 96, 0.0, None, None, None) == B.KVS_ERR_UNSUPPORTED
    assert lib.kvs_attn_fwd(None, None, None, None, 1, 128, 128, 6, 4, 128, 0.0, None, None, None) == B.KVS_ERR_UNSUPPORTED
    assert lib.kvs_attn_fwd(None, None, None, None, 1, 128, 128, 4, 4, 128, 0.0, None, None, None) == B.KVS_ERR_INVALID_ARG
    assert lib.kvs_attn_fwd(None, None, None, None, 1, 0, 0, 4, 4, 128, 0.0, None, None, None) == B.KVS_OK   # empty batch
    assert lib.kvs_attn_bwd(None, None, None, None, None, None, None, 1, 128, 128, 4, 4, 128, 0.0, 5, None, None, None, None, 0,
                            None) == B.KVS_ERR_INVALID_ARG
    assert lib.kvs_device_status(None, None) == B.KVS_ERR_INVALID_ARG


def test_binding_refuses_cpu_tensors(lib):
    import torch
    from paper_2609_35750_b200 import binding as B
    ev = torch.zeros(128, dtype=torch.int32)
    cu = torch.tensor([0, 128], dtype=torch.int32)
    with pytest.raises(ValueError, match="CUDA tensor"):
        B.kvs_mask_meta(ev, cu, 128, meta_buf=torch.zeros(1 << 20, dtype=torch.uint8))
