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


def test_host_arena_and_decode_split_sizing(lib):
    from paper_2609_35750_b200 import binding as B
    # the host entry point keeps three chunks of (trace range, KV head) on the device: with 8 KV heads a chunk is one head
    # over all tokens, so the arena (three chunks with their fp32 dQ accumulators) is below the tensors; with one KV head the batch is cut into up to 8 trace ranges
    T, d = 131072, 128
    tensors = lambda Hq, Hkv: (2 * Hq + 2 * Hkv) * T * d * 2 * 2          # q, dout, out, dq + k, v, dk, dv in bf16
    a8 = B.kvs_host_arena_bytes(2, T, 65536, 32, 8, d, B.GRAD_BF16)
    assert 0 < a8 < 0.6 * tensors(32, 8)
    a1_one = B.kvs_host_arena_bytes(1, T, T, 8, 1, d, B.GRAD_BF16)         # one trace cannot be cut
    a1_many = B.kvs_host_arena_bytes(16, T, 8192, 8, 1, d, B.GRAD_BF16)    # 16 traces of 8192: 8 ranges, three chunks of
    assert a1_many < 0.6 * a1_one                                          # at most T / 8 + 8192 tokens resident
    assert B.kvs_host_arena_bytes(2, T, 65536, 32, 5, d, B.GRAD_BF16) == 0      # Hq % Hkv != 0
    assert B.kvs_host_arena_bytes(0, 0, 0, 32, 8, d, B.GRAD_BF16) == 256
    # split count of decode attention: at least one, never more than a split per 4 tiles of 128 tokens, and the last wave
    # of three CTAs per SM is at least 92 % full whenever some count in range allows it
    slots = 3 * 148
    for S, Hkv, n in [(32, 8, 12288), (64, 4, 7168), (16, 8, 16384), (8, 8, 32768), (256, 8, 2048), (1, 8, 100000), (1, 1, 300), (4, 2, 4096)]:
        k = lib.kvs_decode_num_splits(S, Hkv, n)
        cap = min(64, (n + 511) // 512)
        assert 1 <= k <= max(cap, 1), (S, Hkv, n, k)
        want = max(1, min(cap, -(-2 * slots // (S * Hkv))))
        eff = lambda m: S * Hkv * m / (-(-S * Hkv * m // slots) * slots)
        best = max(eff(m) for m in range(want, min(cap, 3 * want) + 1))
        assert eff(k) >= min(0.92, best) - 1e-9, (S, Hkv, n, k, eff(k), best)
    assert lib.kvs_decode_num_splits(0, 8, 100) == 1 and lib.kvs_decode_num_splits(4, 8, 0) == 1


def test_host_chunk_plan_properties(lib):
    """The trace ranges of the host-buffer entry point, on seeded random batches: contiguous and in order, every trace
    with tokens covered exactly once, no range without tokens, at most min(batch, ceil(8 / Hkv)) ranges, none larger
    than the slot the arena provides (total / ranges + the longest trace)."""
    import numpy as np
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(77)
    for case in range(300):
        batch = int(rng.integers(1, 40))
        Hkv = int(rng.choice([1, 2, 3, 4, 8, 16]))
        kind = case % 4
        if kind == 0:
            lens = rng.integers(0, 5000, size=batch)
        elif kind == 1:
            lens = np.where(rng.random(batch) < 0.4, 0, rng.integers(1, 300, size=batch))      # many empty traces
        elif kind == 2:
            lens = rng.integers(1, 50, size=batch); lens[int(rng.integers(0, batch))] = 100000     # one giant trace
        else:
            lens = np.full(batch, int(rng.integers(1, 4096)))
        if lens.sum() == 0:
            lens[0] = 1
        cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
        total, maxlen = int(cu[-1]), int(lens.max())
        plan = B.kvs_host_chunk_plan(cu, maxlen, Hkv)
        want = max(1, min(batch, -(-8 // Hkv)))
        assert 1 <= len(plan) <= want, (case, plan)
        covered = np.zeros(batch, dtype=bool)
        prev_end = 0
        for b0, b1 in plan:
            assert prev_end <= b0 < b1 <= batch
            assert lens[prev_end:b0].sum() == 0                       # only empty traces are skipped
            tokens = int(cu[b1] - cu[b0])
            assert 0 < tokens <= total // want + maxlen
            covered[b0:b1] = True
            prev_end = b1
        assert lens[prev_end:].sum() == 0 and lens[~covered].sum() == 0
    # malformed tables are refused
    with pytest.raises(B.KvsError):
        B.kvs_host_chunk_plan(np.array([0, 5, 3], dtype=np.int32), 10, 1)
    with pytest.raises(B.KvsError):
        B.kvs_host_chunk_plan(np.array([1, 5, 8], dtype=np.int32), 10, 1)
    with pytest.raises(B.KvsError):
        B.kvs_host_chunk_plan(np.array([0, 50, 80], dtype=np.int32), 10, 1)         # a trace longer than max_seqlen


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
