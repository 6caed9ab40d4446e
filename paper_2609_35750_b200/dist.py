"""Process-group plumbing for runs with one process per GPU.

The path has no exchange step: every (trace, KV-head group) is independent in forward and
backward, so ranks take whole traces and never communicate tensors.  The only collectives
are a barrier around the timed region and two scalar reductions for the report (max of the
per-rank times, sum of the units processed).  Works on NCCL (GPU) and gloo (CPU tests).
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import numpy as np


def world() -> Tuple[int, int]:
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))


def init_from_env(backend: str = "nccl") -> bool:
    """Initialises torch.distributed from RANK / WORLD_SIZE / MASTER_* when WORLD_SIZE > 1."""
    import torch.distributed as dist
    rank, ws = world()
    if ws <= 1:
        return False
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend=backend, rank=rank, world_size=ws)
    return True


def active() -> bool:
    import torch.distributed as dist
    return dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1


def barrier() -> None:
    import torch.distributed as dist
    if active():
        dist.barrier()


def shutdown() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def aggregate(ms_local: float, units_local: float, device="cpu") -> Tuple[float, float]:
    """(max over ranks of the elapsed time, sum over ranks of the units processed)."""
    if not active():
        return float(ms_local), float(units_local)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    u = torch.tensor([units_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def partition_traces(costs: Sequence[float], world_size: int) -> List[List[int]]:
    """Assigns whole traces to ranks, longest-processing-time first, so that the summed cost
    (e.g. unmasked pairs per trace) is balanced.  Deterministic; returns per-rank sorted lists."""
    order = sorted(range(len(costs)), key=lambda i: (-float(costs[i]), i))
    load = [0.0] * world_size
    parts: List[List[int]] = [[] for _ in range(world_size)]
    for i in order:
        r = min(range(world_size), key=lambda x: (load[x], x))
        parts[r].append(i)
        load[r] += float(costs[i])
    return [sorted(p) for p in parts]


def shard_workload(w, rank: int, world_size: int):
    """The sub-batch of `w` (a workloads.Workload) that `rank` owns: whole traces, re-packed.
    Returns (sub_workload, token_index) where token_index maps its packed tokens back to w's."""
    from .workloads import Workload
    costs = []
    for b in range(w.batch):
        ev = w.trace(b).astype(np.int64)
        T = ev.shape[0]
        costs.append(float((np.minimum(ev, T) - np.arange(T)).sum()))
    mine = partition_traces(costs, world_size)[rank]
    lens = [int(w.cu_seqlens[b + 1] - w.cu_seqlens[b]) for b in mine]
    cu = np.zeros(len(mine) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    idx = np.concatenate([np.arange(w.cu_seqlens[b], w.cu_seqlens[b + 1]) for b in mine]) if mine else np.zeros(0, np.int64)
    ev = w.evict_at[idx] if mine else np.zeros(0, np.int32)
    sub = Workload(f"{w.name}[rank{rank}/{world_size}]", cu, ev.astype(np.int32), w.Hq, w.Hkv, w.d,
                   q_prescale=w.q_prescale, softmax_scale=w.softmax_scale, notes=w.notes)
    return sub, idx.astype(np.int64)


def spawn_local(n: int, argv: Sequence[str], env_extra=None, master_port: int = 0, timeout=None) -> List[Tuple[int, str]]:
    """Starts `n` local ranks of the command `argv` (one process per GPU: RANK = LOCAL_RANK = 0..n-1,
    WORLD_SIZE = n, rendezvous on 127.0.0.1) and waits for all of them.  Returns [(exit code, stdout text)]
    by rank; stderr passes through.  If one rank fails the others are left to their process-group timeout
    or are terminated once `timeout` seconds have passed."""
    import socket
    import subprocess
    if master_port <= 0:
        s = socket.socket()
        s.bind(("127.0.0.1", 0))
        master_port = s.getsockname()[1]
        s.close()
    procs = []
    for r in range(n):
        env = dict(os.environ)
        env.update(env_extra or {})
        env.update(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(master_port))
        procs.append(subprocess.Popen(list(argv), env=env, stdout=subprocess.PIPE, text=True))
    results: List[Tuple[int, str]] = []
    for p in procs:
        try:
            out, _ = p.communicate(timeout=timeout)
        except subprocess.TimeoutExpired:
            p.kill()
            out, _ = p.communicate()
        results.append((p.returncode, out or ""))
    return results
