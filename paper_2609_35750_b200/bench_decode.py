"""Decode-attention throughput over a paged, fragmented KV cache (rollout side).

    python -m paper_2609_35750_b200.bench_decode [--seqs 64] [--live 7168] [--page-size 16]

One step = kvs_decode_attn for one new token of every sequence over its live cache.  The kernel
reads every live K and V row once, so it is bound by HBM: the JSON line reports algorithmic bytes
per second (live K and V rows of the sequences' KV heads; q, out and the block tables are noise)
against the measured copy bandwidth.  The block tables point at randomly permuted pages, the
state a cache is in after many evictions and re-allocations.
"""
from __future__ import annotations

import argparse
import json
import os

import numpy as np
import torch

from . import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seqs", type=int, default=64)
    ap.add_argument("--live", type=int, default=7168, help="live tokens per sequence (config 1's peak cache: prompt + summary + segment)")
    ap.add_argument("--page-size", type=int, default=16)
    ap.add_argument("--hq", type=int, default=28)
    ap.add_argument("--hkv", type=int, default=4)
    ap.add_argument("--head-dim", type=int, default=128)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--splits", type=int, default=0)
    a = ap.parse_args()
    dev = "cuda"
    S, n, ps = a.seqs, a.live, a.page_size
    pages_per_seq = (n + ps - 1) // ps
    num_pages = S * pages_per_seq + 8
    cache = B.PagedCache(num_pages, ps, S, pages_per_seq, a.hkv, a.head_dim, device=dev)
    g = torch.Generator(device=dev).manual_seed(0)
    cache.k_cache.copy_(torch.randn(cache.k_cache.shape, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16))
    cache.v_cache.copy_(torch.randn(cache.v_cache.shape, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16))
    perm = torch.randperm(num_pages, generator=g, device=dev)[: S * pages_per_seq].to(torch.int32)
    cache.block_table.copy_(perm.view(S, pages_per_seq))
    cache.n_tokens.fill_(n)
    q = torch.randn((S, a.hq, a.head_dim), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    splits = a.splits or int(B.load().kvs_decode_num_splits(S, a.hkv, n))
    ws = torch.empty(int(B.load().kvs_decode_workspace_bytes(S, a.hq, a.head_dim, splits)), dtype=torch.uint8, device=dev)
    out = torch.empty_like(q)
    lse = torch.empty((S, a.hq), dtype=torch.float32, device=dev)
    for _ in range(a.warmup):
        cache.decode(q, num_splits=splits, out=out, lse=lse, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.steps):
        cache.decode(q, num_splits=splits, out=out, lse=lse, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.steps
    algo = 2.0 * S * n * a.hkv * a.head_dim * 2          # K and V rows, bf16
    peak = 6650.0
    src = "fallback"
    mp = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(mp):
        peak = float(json.load(open(mp))["hbm_gbs"])
        src = "measured"
    gbs = algo / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "decode_attn_hbm_gbs", "value": gbs, "unit": "GB/s", "ms_per_step": ms, "steps": a.steps, "warmup": a.warmup,
        "config": {"workload": "decode over a fragmented paged cache", "seqs": S, "live_tokens": n, "page_size": ps, "Hq": a.hq,
                   "Hkv": a.hkv, "head_dim": a.head_dim, "splits": splits,
                   "l2": "K/V working set %.0f MB, larger than L2" % (algo / 1e6)},
        "tokens_per_s": S / (ms * 1e-3),
        "roofline": {"kernel": ("decode_tc_kernel (tcgen05)" if (a.head_dim == 128 and a.hq // a.hkv in (1, 2, 4, 7, 8) and (a.hq // a.hkv >= 4 or (a.page_size % 8 == 0 and 128 % a.page_size == 0))) else "decode_partial_kernel"), "bound": "hbm", "achieved": gbs, "peak": peak, "unit": "GB/s",
                     "frac": gbs / peak, "traffic": None, "peak_source": src + " copy bandwidth"},
        "dtype": "bf16", "data": "synthetic"}))


if __name__ == "__main__":
    main()
