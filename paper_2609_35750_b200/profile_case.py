"""A small, bounded run of the hot path for profilers (ncu) and quick timing.

    python -m paper_2609_35750_b200.profile_case --config 2 --shrink 4 --iters 2

Runs mask metadata + forward + backward `iters` times on a shrunk copy of a workload (inputs
still larger than L2, a few hundred MB on the device) and prints CUDA-event times.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as B
from . import workloads as W


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--variant", type=str, default="")
    ap.add_argument("--shrink", type=int, default=4)
    ap.add_argument("--iters", type=int, default=2)
    ap.add_argument("--hq", type=int, default=None)
    ap.add_argument("--hkv", type=int, default=None)
    ap.add_argument("--grad", type=str, default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--batch", type=int, default=None, help="number of traces (default: the config's own)")
    ap.add_argument("--meta-only", action="store_true",
                    help="run only the mask-metadata pass (no q/k/v tensors): lets the batch be large enough for its bandwidth to show")
    a = ap.parse_args()
    dev = "cuda"
    w = W.make_workload(a.config, seed=0, shrink=a.shrink, Hq=a.hq, Hkv=a.hkv, variant=a.variant, batch=a.batch)
    if a.meta_only:
        ev = torch.from_numpy(w.evict_at).to(dev)
        cu = torch.from_numpy(w.cu_seqlens).to(dev)
        nbytes = B.kvs_mask_meta_bytes(w.batch, w.total_tokens, w.max_seqlen)
        meta = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        ms = []
        for _ in range(max(a.iters, 3)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=meta)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        st = B.kvs_device_status(meta)
        nb = sum(-(-int(t) // 128) for t in (w.cu_seqlens[1:] - w.cu_seqlens[:-1]))
        tiles = sum((-(-int(t) // 128)) ** 2 for t in (w.cu_seqlens[1:] - w.cu_seqlens[:-1]))
        # algorithmic bytes: evict_at read once and copied once (4 + 4 B per token), one class byte and one
        # 2-byte list slot per tile of the per-trace square
        alg = 8 * w.total_tokens + 3 * tiles
        print(json.dumps({"workload": w.name, "traces": w.batch, "tokens": w.total_tokens, "key_blocks": nb, "tiles": tiles,
                          "meta_buffer_bytes": nbytes, "status": st, "ms": ms, "algorithmic_bytes": alg,
                          "gbs_last": alg / (ms[-1] * 1e-3) / 1e9}))
        if st != 0:
            raise SystemExit(1)
        return
    q, k, v, do = W.make_tensors(w, seed=0, device=dev)
    ev = torch.from_numpy(w.evict_at).to(dev)
    cu = torch.from_numpy(w.cu_seqlens).to(dev)
    grad = B.GRAD_BF16 if a.grad == "bf16" else B.GRAD_FP32
    meta = torch.empty(B.kvs_mask_meta_bytes(w.batch, w.total_tokens, w.max_seqlen), dtype=torch.uint8, device=dev)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(w.total_tokens, w.Hq, w.Hkv, w.d, grad), dtype=torch.uint8, device=dev)
    times = []
    for _ in range(a.iters):
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record()
        B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=meta)
        e[1].record()
        out, lse = B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale)
        e[2].record()
        B.kvs_attn_bwd(do, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, grad, workspace=ws)
        e[3].record()
        torch.cuda.synchronize()
        times.append([e[i].elapsed_time(e[i + 1]) for i in range(3)])
    st = (B.kvs_device_status(meta), B.kvs_device_status(ws))
    pairs = W.count_pairs(w)
    t = times[-1]
    print(json.dumps({"workload": w.name, "shrink": a.shrink, "tokens": w.total_tokens, "Hq": w.Hq, "Hkv": w.Hkv, "d": w.d,
                      "pairs": pairs, "status": st, "ms_meta_fwd_bwd": t,
                      "fwd_tflops": 4.0 * w.d * w.Hq * pairs / (t[1] * 1e-3) / 1e12,
                      "bwd_tflops": 10.0 * w.d * w.Hq * pairs / (t[2] * 1e-3) / 1e12}))
    if st != (0, 0):
        raise SystemExit(1)


if __name__ == "__main__":
    main()
