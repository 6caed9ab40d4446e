#!/usr/bin/env python
"""Benchmark of the eviction-masked attention hot path (mask metadata + forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = kvs_mask_meta + kvs_attn_fwd + kvs_attn_bwd (bf16 gradients, i.e. including the
row-sum pre-pass and the cast post-pass) over one synthetic batch resident in HBM.  Prints
ONE JSON line.  `value` = effective TFLOP/s counting only unmasked (query, key) pairs:
14 * head_dim * Hq * pairs per step.  With N > 1 every rank runs its own batch of the same
configuration (seed + rank): independent traces, no collective on the data path; started
without a launcher (`python bench.py --gpus N`, WORLD_SIZE unset) it starts the N ranks itself.

After the headline measurement of the default run (config 2, one GPU) the other configurations
are timed for a few steps each and reported under `per_config` in the same line.

Smaller runs for profilers and other paths, all through the same library calls:
    --shrink S [--hq H --hkv H --batch B]   a shrunk copy of the configuration
    --path meta                             the mask-metadata pass alone (large batches: its bandwidth)
    --path dual                             student + teacher forward in one pass against two separate forwards
    --path decode [--seqs --live --page-size --hq --hkv --head-dim --splits]
                                            rollout side: decode attention over a fragmented paged cache
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "masked_attn_fwd_bwd_effective_tflops"
UNIT = "TFLOP/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the backward main kernel: a small JSON
# file written beside the ncu summaries whenever that kernel is captured (absent or no entry: null)
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "bwd_kernel_traffic.json")
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_traffic(workload_name):
    try:
        with open(TRAFFIC_FILE) as f:
            return int(json.load(f)[workload_name]["dram_bytes_per_launch"])
    except Exception:
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


# ------------------------------------------------------------------------------------------
# CPU oracle timing (baseline leg and the reference arm).  Workers are spawned processes so
# that no CUDA state is forked; each evaluates whole query rows with the oracle as it stands.
# ------------------------------------------------------------------------------------------
def _oracle_rows_worker(args):
    cfg, variant, seed, trace_idx, rows, heads_per_row = args
    from threadpoolctl import threadpool_limits
    threadpool_limits(1)              # one BLAS thread per worker process: cores == processes
    from oracle import kvs_oracle as O
    from paper_2609_35750_b200 import workloads as W
    w = W.make_workload(cfg, seed=seed, variant=variant)
    ev = w.trace(trace_idx)
    T = ev.shape[0]
    r = np.random.default_rng(1234 + seed)
    # one KV head of one trace, drawn with the workload's distribution (bf16-rounded N(0,1))
    import torch
    k = torch.randn((T, w.d), generator=torch.Generator().manual_seed(seed + 1)).to(torch.bfloat16).float().numpy()
    v = torch.randn((T, w.d), generator=torch.Generator().manual_seed(seed + 2)).to(torch.bfloat16).float().numpy()
    t0 = time.perf_counter()
    pairs = 0
    for i in rows:
        for _ in range(heads_per_row):
            qi = (r.standard_normal(w.d) * w.q_prescale).astype(np.float32)
            do = r.standard_normal(w.d).astype(np.float32)
            o, lse, dq, vis, dkc, dvc = O.row_fwd_bwd(qi, k, v, do, ev, int(i), w.scale)
            pairs += int(vis.shape[0])
    dt = time.perf_counter() - t0
    return pairs, dt


def time_oracle(cfg: int, variant: str, seed: int, target_seconds: float, rows_per_worker: int | None = None):
    """Times the oracle on a bounded sample: random query rows of trace 0, one process per
    host core.  Returns dict(value TFLOP/s, cores, sample, seconds, pairs)."""
    import multiprocessing as mp
    from paper_2609_35750_b200 import workloads as W
    w = W.make_workload(cfg, seed=seed, variant=variant)
    try:
        cores = len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        cores = os.cpu_count() or 1
    cores = max(1, min(cores, 64))
    T = int(w.cu_seqlens[1])
    mean_live = W.count_pairs(w) / w.total_tokens
    # an fp64 row costs about 7 matrix-vector passes over its live keys
    est_row_s = max(2e-4, mean_live * w.d * 7 / 2.5e8)
    if rows_per_worker is None:
        rows_per_worker = max(4, int(target_seconds / est_row_s))
    rng = np.random.default_rng(99 + seed)
    jobs = [(cfg, variant, seed, 0, rng.integers(0, T, size=rows_per_worker).tolist(), 1) for _ in range(cores)]
    ctx = mp.get_context("spawn")
    t0 = time.perf_counter()
    with ctx.Pool(cores) as pool:
        res = pool.map(_oracle_rows_worker, jobs)
    wall = time.perf_counter() - t0
    pairs = sum(p for p, _ in res)
    busy = max(dt for _, dt in res)
    flops = 14.0 * w.d * pairs            # one head per evaluated row
    return {
        "value": flops / busy / 1e12,
        "unit": UNIT,
        "cores": cores,
        "kind": "oracle",
        "sample": f"{cores * rows_per_worker} random (query row, head) pairs of trace 0 of {w.name}, fp64 row-by-row oracle "
                  f"(out, lse, dq and the row's dk/dv contributions), {pairs} unmasked pairs, one process per core; "
                  f"value = 14*d*pairs / slowest worker's compute time ({busy:.1f} s; {wall:.1f} s wall with start-up)",
        "seconds": busy,
        "pairs": pairs,
        "rows_per_worker": rows_per_worker,
    }


# ------------------------------------------------------------------------------------------
# clocks
# ------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "100"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        try:
            for line in open(self.path):
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                    power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out = {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                   "samples": len(sm), "power_w_max": max(power) if power else None}
        return out


# ------------------------------------------------------------------------------------------
def run_reference(args):
    """`--impl reference`: the CPU oracle as it stands, each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2609_35750_b200 import workloads as W
    w = W.make_workload(args.config, seed=0, variant=args.variant)
    per_step = max(2.0, min(20.0, 90.0 / max(1, args.steps + args.warmup)))
    rows = None
    vals, secs = [], []
    for s in range(args.warmup + args.steps):
        r = time_oracle(args.config, args.variant, 0, per_step, rows)
        rows = r["rows_per_worker"]          # every step evaluates the same number of rows
        if s >= args.warmup:
            vals.append(r["value"])
            secs.append(r["seconds"])
    value = float(np.mean(vals))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": float(np.mean(secs) * 1e3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "tokens": w.total_tokens, "Hq": w.Hq, "Hkv": w.Hkv, "head_dim": w.d,
                   "note": "each step is a bounded sample of query rows, not the whole batch"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": r["cores"], "kind": "oracle", "sample": r["sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "tokens_per_s": value * 1e12 / (14.0 * w.d * w.Hq * W.count_pairs(w) / w.total_tokens),
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def time_train_steps(torch, B, W, w, seed, dev, steps, warmup, grad, barrier=None, sampler=None, reorder=0):
    """Mask metadata + forward + backward, `warmup` untimed and `steps` timed steps on the current stream.
    Returns a dict of per-phase mean times (ms), the total, and the device status.
    reorder > 0: the token-level path.  Every step also sorts the keys of each window of `reorder` keys by eviction step
    (kvs_reorder_keys), brings k and v into that slot order, builds the metadata for the slots, and returns dk, dv to token
    order; all of it inside the timed step (counted under the metadata time)."""
    q, k, v, do = W.make_tensors(w, seed=seed, device=str(dev))
    ev = torch.from_numpy(w.evict_at).to(dev)
    cu = torch.from_numpy(w.cu_seqlens).to(dev)
    Tt, Hq, Hkv, d = w.total_tokens, w.Hq, w.Hkv, w.d
    meta = torch.empty(B.kvs_mask_meta_bytes(w.batch, Tt, w.max_seqlen), dtype=torch.uint8, device=dev)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, Hq, Hkv, d, grad), dtype=torch.uint8, device=dev)
    gdt = torch.bfloat16 if grad == B.GRAD_BF16 else torch.float32
    out = torch.empty_like(q)
    lse = torch.empty((Hq, Tt), dtype=torch.float32, device=dev)
    dq, dk, dv = (torch.empty(t.shape, dtype=gdt, device=dev) for t in (q, k, v))
    if reorder:
        perm, kf, ke = (torch.empty(Tt, dtype=torch.int32, device=dev) for _ in range(3))
        kp, vp, dkp, dvp = torch.empty_like(k), torch.empty_like(v), torch.empty_like(dk), torch.empty_like(dv)
    stream = torch.cuda.current_stream()
    mk = lambda: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    ev_fwd, ev_bwd, ev_meta = mk(), mk(), mk()
    for pair in ev_bwd:              # create the handles before they are passed through the C ABI
        pair[0].record(stream)
        pair[1].record(stream)

    def step(i=None):
        if i is not None:
            ev_meta[i][0].record(stream)
        if reorder:
            B.kvs_reorder_keys(ev, cu, w.max_seqlen, reorder, perm=perm, key_first=kf, key_evict=ke)
            B.kvs_permute_rows(k, perm, kp)
            B.kvs_permute_rows(v, perm, vp)
            B.kvs_mask_meta_keys(kf, ke, cu, w.max_seqlen, meta_buf=meta)
        else:
            B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=meta)
        kk, vv, dkk, dvv = (kp, vp, dkp, dvp) if reorder else (k, v, dk, dv)
        if i is not None:
            ev_meta[i][1].record(stream)
            ev_fwd[i][0].record(stream)
        B.kvs_attn_fwd(q, kk, vv, meta, w.batch, w.max_seqlen, w.softmax_scale, out=out, lse=lse)
        if i is not None:
            ev_fwd[i][1].record(stream)
        B.kvs_attn_bwd(do, q, kk, vv, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, grad, dq=dq, dk=dkk, dv=dvv,
                       workspace=ws, main_events=(ev_bwd[i] if i is not None else None))
        if reorder:
            B.kvs_permute_rows(dkp, perm, dk, inverse=True)
            B.kvs_permute_rows(dvp, perm, dv, inverse=True)

    for _ in range(max(warmup, 0)):
        step()
    torch.cuda.synchronize()
    status = (B.kvs_device_status(meta), B.kvs_device_status(ws))
    if status != (0, 0):
        raise SystemExit(f"device status after warm-up: {status}")
    if sampler is not None:
        sampler.start()
        time.sleep(0.3)
    if barrier is not None:
        barrier()
    torch.cuda.synchronize()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for i in range(steps):
        step(i)
    t_end.record(stream)
    torch.cuda.synchronize()
    if barrier is not None:
        barrier()
    clocks = sampler.stop() if sampler is not None else None
    status = (B.kvs_device_status(meta), B.kvs_device_status(ws))
    if status != (0, 0):
        raise SystemExit(f"device status after the timed region: {status}")
    mean = lambda evs: float(np.mean([a.elapsed_time(b) for a, b in evs]))
    return {"ms_total": t_begin.elapsed_time(t_end), "ms_fwd": mean(ev_fwd), "ms_bwd_main": mean(ev_bwd), "ms_meta": mean(ev_meta),
            "clocks": clocks, "tensors": (q, k, v, do)}


def run_per_config(torch, B, W, dev, peaks, gpu_index):
    """The other configurations on the same clock as the headline: 1 warm-up + 3 timed steps each."""
    res = {}
    for key, cfg, variant, reorder in (("0", 0, "", 0), ("1", 1, "", 0), ("3", 3, "", 0), ("4", 4, "", 0),
                                       ("4_keys_reordered", 4, "", 4096), ("4_control", 4, "control", 0),
                                       ("4b", 4, "b", 0), ("4b_keys_reordered", 4, "b", 4096),
                                       ("5", 5, "", 0), ("6", 6, "", 0), ("7", 7, "", 0)):
        w = W.make_workload(cfg, seed=0, variant=variant)
        sampler = ClockSampler(gpu_index)
        r = time_train_steps(torch, B, W, w, 0, dev, steps=3, warmup=1, grad=B.GRAD_BF16, sampler=sampler, reorder=reorder)
        r.pop("tensors")
        torch.cuda.empty_cache()
        ms = r["ms_total"] / 3
        tf = W.fwd_bwd_flops(w) / (ms * 1e-3) / 1e12
        res[key] = {"workload": w.name, "tokens": w.total_tokens, "unmasked_pairs": W.count_pairs(w), "steps": 3, "warmup": 1,
                    "reorder_window": reorder, "ms_per_step": ms, "effective_tflops": tf, "frac_of_burst_peak": tf / float(peaks["bf16_tflops"]),
                    "tokens_per_s": w.total_tokens / (ms * 1e-3), "ms_fwd": r["ms_fwd"], "ms_bwd_main": r["ms_bwd_main"],
                    "sm_mhz_median": (r["clocks"] or {}).get("sm_mhz"), "reasons": (r["clocks"] or {}).get("reasons")}
    return res


def run_meta_only(args):
    """--path meta: the mask-metadata pass alone (no q/k/v), so that the batch can be large enough for its bandwidth to show."""
    import torch
    from paper_2609_35750_b200 import binding as B
    from paper_2609_35750_b200 import workloads as W
    dev = "cuda"
    w = W.make_workload(args.config, seed=0, shrink=args.shrink, Hq=args.hq, Hkv=args.hkv, variant=args.variant, batch=args.batch)
    ev = torch.from_numpy(w.evict_at).to(dev)
    cu = torch.from_numpy(w.cu_seqlens).to(dev)
    nbytes = B.kvs_mask_meta_bytes(w.batch, w.total_tokens, w.max_seqlen)
    meta = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    ms = []
    for _ in range(args.warmup + max(args.steps, 1)):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=meta)
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1))
    ms = ms[args.warmup:]
    st = B.kvs_device_status(meta)
    lens = (w.cu_seqlens[1:] - w.cu_seqlens[:-1]).astype(np.int64)
    nb = int(((lens + 127) // 128).sum())
    tiles = int((((lens + 127) // 128) ** 2).sum())
    # algorithmic bytes: evict_at read once and copied once (4 + 4 B per token), one class byte and one
    # 2-byte list slot per tile of the per-trace square
    alg = 8 * w.total_tokens + 3 * tiles
    peaks = load_peaks()
    gbs = alg / (float(np.median(ms)) * 1e-3) / 1e9
    print(json.dumps({"metric": "mask_meta_gbs", "value": gbs, "unit": "GB/s", "steps": len(ms), "warmup": args.warmup,
                      "ms_per_step": float(np.median(ms)), "config": {"workload": w.name, "traces": w.batch, "tokens": w.total_tokens,
                                                                       "key_blocks": nb, "tiles": tiles, "meta_buffer_bytes": nbytes},
                      "roofline": {"kernel": "mask metadata (4 launches)", "bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]),
                                   "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]), "traffic": None,
                                   "algorithmic_bytes": alg},
                      "status": st, "dtype": "int32", "data": "synthetic"}), flush=True)
    if st != 0:
        raise SystemExit(1)


def measure_decode(hq, hkv, S, n, ps, head_dim=128, splits=0, steps=50, warmup=3):
    """One step = kvs_decode_attn for one new token of every sequence over its live cache.  The kernel reads every live
    K and V row once, so it is bound by HBM: algorithmic bytes = live K and V rows of the sequences' KV heads.  The block
    tables point at randomly permuted pages, the state of a cache after many evictions."""
    import torch
    from paper_2609_35750_b200 import binding as B
    dev = "cuda"
    pages_per_seq = (n + ps - 1) // ps
    num_pages = S * pages_per_seq + 8
    cache = B.PagedCache(num_pages, ps, S, pages_per_seq, hkv, head_dim, device=dev)
    g = torch.Generator(device=dev).manual_seed(0)
    cache.k_cache.copy_(torch.randn(cache.k_cache.shape, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16))
    cache.v_cache.copy_(torch.randn(cache.v_cache.shape, generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16))
    perm = torch.randperm(num_pages, generator=g, device=dev)[: S * pages_per_seq].to(torch.int32)
    cache.block_table.copy_(perm.view(S, pages_per_seq))
    cache.n_tokens.fill_(n)
    q = torch.randn((S, hq, head_dim), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    splits = splits or int(B.load().kvs_decode_num_splits(S, hkv, n))
    ws = torch.empty(int(B.load().kvs_decode_workspace_bytes(S, hq, head_dim, splits)), dtype=torch.uint8, device=dev)
    out = torch.empty_like(q)
    lse = torch.empty((S, hq), dtype=torch.float32, device=dev)
    for _ in range(max(warmup, 1)):
        cache.decode(q, num_splits=splits, out=out, lse=lse, workspace=ws)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        cache.decode(q, num_splits=splits, out=out, lse=lse, workspace=ws)
    e1.record()
    torch.cuda.synchronize()
    if B.kvs_device_status(ws) != 0:
        raise SystemExit("device status after the timed region: %d" % B.kvs_device_status(ws))
    ms = e0.elapsed_time(e1) / steps
    algo = 2.0 * S * n * hkv * head_dim * 2          # K and V rows, bf16
    peaks = load_peaks()
    gbs = algo / (ms * 1e-3) / 1e9
    return {
        "metric": "decode_attn_hbm_gbs", "value": gbs, "unit": "GB/s", "ms_per_step": ms, "steps": steps, "warmup": warmup,
        "config": {"workload": "decode over a fragmented paged cache", "seqs": S, "live_tokens": n, "page_size": ps, "Hq": hq,
                   "Hkv": hkv, "head_dim": head_dim, "splits": splits,
                   "l2": "K/V working set %.0f MB, larger than L2" % (algo / 1e6)},
        "tokens_per_s": S / (ms * 1e-3),
        "roofline": {"kernel": "decode attention (partial + combine)", "bound": "hbm", "achieved": gbs, "peak": float(peaks["hbm_gbs"]),
                     "unit": "GB/s", "frac": gbs / float(peaks["hbm_gbs"]), "traffic": None,
                     "peak_source": peaks["_source"] + " copy bandwidth"},
        "dtype": "bf16", "data": "synthetic"}


def run_decode(args):
    """--path decode: the rollout-side decode step on one shape, one JSON line."""
    print(json.dumps(measure_decode(args.hq or 28, args.hkv or 4, args.seqs, args.live, args.page_size, args.head_dim, args.splits,
                                    args.steps, args.warmup)), flush=True)


def run_dual(args):
    """--path dual: the self-distillation forward (student under the eviction mask + full-context teacher; the teacher
    costs one more pass over the evicted keys only, then a merge) against the two plain forwards it replaces."""
    import torch
    from paper_2609_35750_b200 import binding as B
    from paper_2609_35750_b200 import workloads as W
    dev = "cuda"
    w = W.make_workload(args.config, seed=0, shrink=args.shrink, Hq=args.hq, Hkv=args.hkv, variant=args.variant, batch=args.batch)
    q, k, v, _ = W.make_tensors(w, seed=0, device=dev, with_dout=False)
    ev = torch.from_numpy(w.evict_at).to(dev)
    cu = torch.from_numpy(w.cu_seqlens).to(dev)
    meta = B.kvs_mask_meta(ev, cu, w.max_seqlen)
    meta_c = B.kvs_mask_meta(torch.full_like(ev, int(W.INF)), cu, w.max_seqlen)
    meta_e = B.kvs_mask_meta_evicted(ev, cu, w.max_seqlen)
    o = [torch.empty_like(q) for _ in range(2)]
    l = [torch.empty((w.Hq, w.total_tokens), dtype=torch.float32, device=dev) for _ in range(2)]

    def dual():
        B.kvs_attn_fwd_dual(q, k, v, meta, meta_e, w.batch, w.max_seqlen, w.softmax_scale, out_student=o[0], lse_student=l[0],
                            out_teacher=o[1], lse_teacher=l[1])

    def separate():
        B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale, out=o[0], lse=l[0])
        B.kvs_attn_fwd(q, k, v, meta_c, w.batch, w.max_seqlen, w.softmax_scale, out=o[1], lse=l[1])

    def timed(fn):
        for _ in range(max(args.warmup, 1)):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    ms_dual, ms_sep = timed(dual), timed(separate)
    if B.kvs_device_status(meta) != 0 or B.kvs_device_status(meta_c) != 0:
        raise SystemExit("device status set")
    pairs_s = W.count_pairs(w)
    lens = np.diff(w.cu_seqlens).astype(np.int64)
    pairs_t = int((lens * (lens + 1) // 2).sum())
    flops = 4.0 * w.d * w.Hq * (pairs_s + pairs_t)        # what two separate forwards compute (unmasked pairs of both masks)
    peaks = load_peaks()
    tf = flops / (ms_dual * 1e-3) / 1e12
    print(json.dumps({"metric": "dual_forward_effective_tflops", "value": tf, "unit": "TFLOP/s", "steps": args.steps, "warmup": args.warmup,
                      "ms_per_step": ms_dual, "ms_two_separate_forwards": ms_sep, "speedup_over_separate": ms_sep / ms_dual,
                      "config": {"workload": w.name, "tokens": w.total_tokens, "Hq": w.Hq, "Hkv": w.Hkv, "head_dim": w.d,
                                 "student_pairs": pairs_s, "teacher_pairs": pairs_t,
                                 "flops": "4*d*Hq*(student pairs + teacher pairs): the shared q k^T is counted once per stream"},
                      "roofline": {"kernel": "fwd_kernel x2 + dual_merge_kernel", "bound": "tensor", "achieved": tf, "peak": float(peaks["bf16_tflops"]),
                                   "unit": "TFLOP/s", "frac": tf / float(peaks["bf16_tflops"]), "traffic": None},
                      "dtype": "bf16", "data": "synthetic"}), flush=True)


def spawn_ranks(n):
    """`python bench.py --gpus N` without a launcher: start the N ranks here (one process per GPU, LOCAL_RANK = GPU
    index), pass rank 0's JSON line through, everything else the ranks print goes to stderr."""
    from paper_2609_35750_b200 import dist as D
    results = D.spawn_local(n, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:],
                            env_extra={"NCCL_DEBUG": os.environ.get("NCCL_DEBUG", "INFO"),
                                       "NCCL_DEBUG_SUBSYS": os.environ.get("NCCL_DEBUG_SUBSYS", "INIT")})
    line = None
    for rank, (rc, text) in enumerate(results):
        for ln in text.splitlines():
            if rank == 0 and ln.startswith("{") and '"metric"' in ln:
                line = ln
            else:
                print(f"[rank {rank}] {ln}", file=sys.stderr)
    bad = [(r, rc) for r, (rc, _) in enumerate(results) if rc != 0]
    if bad:
        raise SystemExit(f"bench.py --gpus {n}: ranks failed (rank, exit code): {bad}")
    if line is None:
        raise SystemExit(f"bench.py --gpus {n}: rank 0 printed no result line")
    print(line, flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload 0..7 (default 2: keep-last-4-turns, the target config)")
    ap.add_argument("--variant", type=str, default="")
    ap.add_argument("--impl", type=str, default="native", choices=["native", "reference"])
    ap.add_argument("--path", type=str, default="train", choices=["train", "meta", "decode", "dual"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e", action="store_true", help="measure the host-buffer entry point also when the case was reduced by a flag")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    ap.add_argument("--shrink", type=int, default=1, help="divide every length of the configuration (small cases for profilers)")
    ap.add_argument("--hq", type=int, default=None)
    ap.add_argument("--hkv", type=int, default=None)
    ap.add_argument("--batch", type=int, default=None, help="number of traces (default: the configuration's own)")
    ap.add_argument("--grad", type=str, default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--reorder", type=int, default=0,
                    help="token-level eviction: sort the keys of every window of this many keys by eviction step (0: off)")
    ap.add_argument("--seqs", type=int, default=64, help="--path decode: sequences")
    ap.add_argument("--live", type=int, default=7168, help="--path decode: live tokens per sequence")
    ap.add_argument("--page-size", type=int, default=16, help="--path decode: tokens per page")
    ap.add_argument("--head-dim", type=int, default=128, help="--path decode")
    ap.add_argument("--splits", type=int, default=0, help="--path decode: KV splits (0: chosen by the library)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return
    if args.path == "meta":
        run_meta_only(args)
        return
    if args.path == "decode":
        run_decode(args)
        return
    if args.path == "dual":
        run_dual(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_ranks(args.gpus)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    small = args.shrink != 1 or args.hq is not None or args.hkv is not None or args.batch is not None or args.reorder != 0

    # CPU baseline first (rank 0, N = 1 only), before this process touches CUDA
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not small:
        cpu_baseline = time_oracle(args.config, args.variant, 0, args.cpu_seconds)
        cpu_baseline = {k: cpu_baseline[k] for k in ("value", "unit", "cores", "kind", "sample")}

    import torch
    from paper_2609_35750_b200 import binding as B
    from paper_2609_35750_b200 import dist as D
    from paper_2609_35750_b200 import workloads as W

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU implementation")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    D.init_from_env(backend="nccl")
    B.load()

    w = W.make_workload(args.config, seed=rank, variant=args.variant, shrink=args.shrink, Hq=args.hq, Hkv=args.hkv, batch=args.batch)
    Tt, Hq, Hkv, d = w.total_tokens, w.Hq, w.Hkv, w.d
    grad = B.GRAD_BF16 if args.grad == "bf16" else B.GRAD_FP32
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local_rank) if rank == 0 else None
    r = time_train_steps(torch, B, W, w, rank, dev, args.steps, args.warmup, grad, barrier=D.barrier, sampler=sampler,
                         reorder=args.reorder)
    q, k, v, do = r.pop("tensors")
    clocks = r["clocks"]
    ms_total = r["ms_total"]
    ms_total_max, units_total = D.aggregate(ms_total, float(W.fwd_bwd_flops(w)) * args.steps, device=dev)
    _, tokens_total = D.aggregate(ms_total, float(Tt) * args.steps, device=dev)
    ms_fwd, ms_bwd_main, ms_meta = r["ms_fwd"], r["ms_bwd_main"], r["ms_meta"]
    pairs = W.count_pairs(w)
    torch.cuda.empty_cache()

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    e2e = None
    if not args.no_e2e and (not small or args.e2e):
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hq, hk, hv, hdo = pin(q), pin(k), pin(v), pin(do)
        hev, hcu = pin(torch.from_numpy(w.evict_at)), pin(torch.from_numpy(w.cu_seqlens))
        gdt = torch.bfloat16 if grad == B.GRAD_BF16 else torch.float32
        ho = torch.empty(hq.shape, dtype=torch.bfloat16).pin_memory()
        hl = torch.empty((Hq, Tt), dtype=torch.float32).pin_memory()
        hdq = torch.empty(hq.shape, dtype=gdt).pin_memory()
        hdk = torch.empty(hk.shape, dtype=gdt).pin_memory()
        hdv = torch.empty(hk.shape, dtype=gdt).pin_memory()
        del q, k, v, do
        torch.cuda.empty_cache()
        arena = torch.empty(B.kvs_host_arena_bytes(w.batch, Tt, w.max_seqlen, Hq, Hkv, d, grad), dtype=torch.uint8, device=dev)
        h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv, hdo, hev, hcu))
        d2h = sum(t.numel() * t.element_size() for t in (ho, hl, hdq, hdk, hdv))
        e_steps = max(1, min(args.steps, 5))

        def e2e_step():
            B.kvs_attn_fwd_bwd_host(hev, hcu, hq, hk, hv, hdo, w.max_seqlen, w.softmax_scale, grad, ho, hl, hdq, hdk, hdv, arena)

        e2e_step()
        D.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(e_steps):
            e2e_step()
        b.record(stream)
        torch.cuda.synchronize()
        D.barrier()
        ms_e2e, units_e2e = D.aggregate(a.elapsed_time(b), float(W.fwd_bwd_flops(w)) * e_steps, device=dev)
        e2e = {"value": units_e2e / (ms_e2e * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": ms_e2e / e_steps, "steps": e_steps,
               "api": "kvs_attn_fwd_bwd_host (pinned host buffers in, pinned host buffers out)"}
        del arena, hq, hk, hv, hdo, ho, hl, hdq, hdk, hdv
        torch.cuda.empty_cache()
    else:
        del q, k, v, do
        torch.cuda.empty_cache()

    if rank != 0:
        D.shutdown()
        return

    peaks = load_peaks()
    per_config = None
    rollout_decode = None
    if world == 1 and not small and args.config == 2 and args.variant == "" and not args.no_per_config:
        per_config = run_per_config(torch, B, W, dev, peaks, local_rank)
        # the rollout side on the same clock: one decode step over config 1's peak cache and over a wider one,
        # with 16-token and 1-token pages (fraction of the measured HBM copy bandwidth)
        rollout_decode = {}
        for name, (hq_, hkv_, S_, n_) in (("64x7168_Hq28_Hkv4", (28, 4, 64, 7168)), ("32x12288_Hq32_Hkv8", (32, 8, 32, 12288))):
            for ps_ in (16, 1):
                r = measure_decode(hq_, hkv_, S_, n_, ps_, steps=30, warmup=3)
                rollout_decode[f"{name}_pages{ps_}"] = {"ms_per_step": r["ms_per_step"], "gbs": r["value"], "frac_of_hbm": r["roofline"]["frac"],
                                                        "splits": r["config"]["splits"]}

    value = units_total / (ms_total_max * 1e-3) / 1e12
    flops_bwd_main = 10.0 * d * Hq * pairs
    achieved = flops_bwd_main / (ms_bwd_main * 1e-3) / 1e12
    peak = float(peaks["bf16_tflops_sustained"])      # the kernel is timed inside a long step
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "traces": w.batch, "tokens": Tt, "Hq": Hq, "Hkv": Hkv, "head_dim": d,
                   "unmasked_pairs": pairs, "flops_per_step": W.fwd_bwd_flops(w), "grad_dtype": args.grad,
                   "reorder_window": args.reorder,
                   "l2": "inputs larger than L2 (q, dout, out, dq are each %.2f GB)" % (Tt * Hq * d * 2 / 1e9),
                   "parallelism": f"independent batches x{world}" if world > 1 else "single GPU", "notes": w.notes},
        "tokens_per_s": tokens_total / (ms_total_max * 1e-3),
        "pct_of_bf16_peak": {"of_measured_burst": 100 * value / float(peaks["bf16_tflops"]),
                             "of_measured_sustained": 100 * value / float(peaks["bf16_tflops_sustained"]),
                             "of_nominal_2250": 100 * value / 2250.0, "peaks": peaks["_source"]},
        "breakdown_ms": {"mask_meta": ms_meta, "fwd": ms_fwd, "bwd_main": ms_bwd_main,
                         "bwd_pre_post": ms_total_max / args.steps - ms_meta - ms_fwd - ms_bwd_main,
                         "fwd_tflops": 4.0 * d * Hq * pairs / (ms_fwd * 1e-3) / 1e12, "bwd_main_tflops": achieved},
        "roofline": {"kernel": "bwd_kernel (dQ/dK/dV main)", "bound": "tensor", "achieved": achieved, "peak": peak,
                     "unit": "TFLOP/s", "frac": achieved / peak, "traffic": load_traffic(w.name),
                     "frac_of_burst_peak": achieved / float(peaks["bf16_tflops"]),
                     "peak_source": f"{peaks['_source']} cuBLAS bf16, sustained (kernel timed inside a long step)",
                     "flops_per_launch": flops_bwd_main},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": ((8 if grad == B.GRAD_BF16 else 7) + (5 if args.reorder else 0)) * args.steps,
        "cpu_baseline": cpu_baseline,
        "per_config": per_config,
        "rollout_decode": rollout_decode,
    }
    print(json.dumps(line), flush=True)
    D.shutdown()


if __name__ == "__main__":
    main()
