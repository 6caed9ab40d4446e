#!/usr/bin/env python
"""Benchmark of the eviction-masked attention hot path (mask metadata + forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl reference]

One step = kvs_mask_meta + kvs_attn_fwd + kvs_attn_bwd (bf16 gradients, i.e. including the
row-sum pre-pass and the cast post-pass) over one synthetic batch resident in HBM.  Prints
ONE JSON line.  `value` = effective TFLOP/s counting only unmasked (query, key) pairs:
14 * head_dim * Hq * pairs per step.  With N > 1 every rank runs its own batch of the same
configuration (seed + rank): independent traces, no collective on the data path.
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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the backward main kernel, from the
# ncu captures summarised under profiles/ (None until a capture of that workload exists)
NCU_DRAM_BYTES_PER_LAUNCH = {"cfg2_keep_last_4_turns": 20461770496}   # profiles/bwd_kernel_cfg2.md, full-size light pass
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2, help="workload 0..4 (default 2: keep-last-4-turns, the target config)")
    ap.add_argument("--variant", type=str, default="")
    ap.add_argument("--impl", type=str, default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=12.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)

    if args.impl == "reference":
        run_reference(args)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    # CPU baseline first (rank 0, N = 1 only), before this process touches CUDA
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
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

    w = W.make_workload(args.config, seed=rank, variant=args.variant)
    q, k, v, do = W.make_tensors(w, seed=rank, device=str(dev))
    ev = torch.from_numpy(w.evict_at).to(dev)
    cu = torch.from_numpy(w.cu_seqlens).to(dev)
    Tt, Hq, Hkv, d = w.total_tokens, w.Hq, w.Hkv, w.d
    grad = B.GRAD_BF16
    meta = torch.empty(B.kvs_mask_meta_bytes(w.batch, Tt, w.max_seqlen), dtype=torch.uint8, device=dev)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, Hq, Hkv, d, grad), dtype=torch.uint8, device=dev)
    out = torch.empty_like(q)
    lse = torch.empty((Hq, Tt), dtype=torch.float32, device=dev)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    stream = torch.cuda.current_stream()

    n_ev = args.steps
    ev_fwd = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
    ev_bwd = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
    ev_meta = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_ev)]
    for pair in ev_bwd:              # create the handles before they are passed through the C ABI
        pair[0].record(stream)
        pair[1].record(stream)

    def step(i=None):
        if i is not None:
            ev_meta[i][0].record(stream)
        B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=meta)
        if i is not None:
            ev_meta[i][1].record(stream)
            ev_fwd[i][0].record(stream)
        B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale, out=out, lse=lse)
        if i is not None:
            ev_fwd[i][1].record(stream)
        B.kvs_attn_bwd(do, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, grad, dq=dq, dk=dk, dv=dv,
                       workspace=ws, main_events=(ev_bwd[i] if i is not None else None))

    for _ in range(max(args.warmup, 0)):
        step()
    torch.cuda.synchronize()
    status = (B.kvs_device_status(meta), B.kvs_device_status(ws))
    if status != (0, 0):
        raise SystemExit(f"device status after warm-up: {status}")

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    D.barrier()
    torch.cuda.synchronize()
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for i in range(args.steps):
        step(i)
    t_end.record(stream)
    torch.cuda.synchronize()
    D.barrier()
    clocks = sampler.stop() if rank == 0 else None
    ms_total = t_begin.elapsed_time(t_end)
    ms_total_max, units_total = D.aggregate(ms_total, float(W.fwd_bwd_flops(w)) * args.steps, device=dev)
    _, tokens_total = D.aggregate(ms_total, float(Tt) * args.steps, device=dev)
    status = (B.kvs_device_status(meta), B.kvs_device_status(ws))
    if status != (0, 0):
        raise SystemExit(f"device status after the timed region: {status}")

    ms_fwd = float(np.mean([a.elapsed_time(b) for a, b in ev_fwd]))
    ms_bwd_main = float(np.mean([a.elapsed_time(b) for a, b in ev_bwd]))
    ms_meta = float(np.mean([a.elapsed_time(b) for a, b in ev_meta]))
    pairs = W.count_pairs(w)

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    e2e = None
    if not args.no_e2e:
        del out, lse, dq, dk, dv, ws, meta
        torch.cuda.empty_cache()
        pin = lambda t: t.cpu().contiguous().pin_memory()
        hq, hk, hv, hdo = pin(q), pin(k), pin(v), pin(do)
        hev, hcu = pin(torch.from_numpy(w.evict_at)), pin(torch.from_numpy(w.cu_seqlens))
        ho = torch.empty(hq.shape, dtype=torch.bfloat16).pin_memory()
        hl = torch.empty((Hq, Tt), dtype=torch.float32).pin_memory()
        hdq = torch.empty(hq.shape, dtype=torch.bfloat16).pin_memory()
        hdk = torch.empty(hk.shape, dtype=torch.bfloat16).pin_memory()
        hdv = torch.empty(hk.shape, dtype=torch.bfloat16).pin_memory()
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

    if rank != 0:
        D.shutdown()
        return

    peaks = load_peaks()
    value = units_total / (ms_total_max * 1e-3) / 1e12
    flops_bwd_main = 10.0 * d * Hq * pairs
    achieved = flops_bwd_main / (ms_bwd_main * 1e-3) / 1e12
    peak = float(peaks["bf16_tflops_sustained"])      # the kernel is timed inside a long step
    profile_traffic = NCU_DRAM_BYTES_PER_LAUNCH.get(w.name)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_total_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "traces": w.batch, "tokens": Tt, "Hq": Hq, "Hkv": Hkv, "head_dim": d,
                   "unmasked_pairs": pairs, "flops_per_step": W.fwd_bwd_flops(w), "grad_dtype": "bf16",
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
                     "unit": "TFLOP/s", "frac": achieved / peak, "traffic": profile_traffic,
                     "peak_source": f"{peaks['_source']} cuBLAS bf16, sustained (kernel timed inside a long step)",
                     "flops_per_launch": flops_bwd_main},
        "clocks": clocks,
        "e2e": e2e,
        "gpu_launches": 8 * args.steps,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line), flush=True)
    D.shutdown()


if __name__ == "__main__":
    main()
