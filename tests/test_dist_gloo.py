"""The N > 1 path on CPU: two gloo ranks shard a packed batch by trace (no data-path
collective), each computes its shard, and the union equals the unsharded result."""
import os
import socket
import sys

import numpy as np
import torch
import torch.multiprocessing as mp

from paper_2609_35750_b200 import dist as D
from paper_2609_35750_b200 import workloads as W


def test_partition_traces_balanced_and_deterministic():
    costs = [10, 1, 7, 3, 3, 8, 2]
    parts = D.partition_traces(costs, 3)
    assert sorted(sum(parts, [])) == list(range(7))
    loads = [sum(costs[i] for i in p) for p in parts]
    assert max(loads) - min(loads) <= max(costs) and parts == D.partition_traces(costs, 3)
    assert D.partition_traces([5.0], 2) == [[0], []]


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world_size, port, tmpdir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world_size), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    from oracle import kvs_oracle as O
    assert D.init_from_env(backend="gloo")
    w = W.make_workload(3, seed=0, shrink=128, batch=5, Hq=2, Hkv=1)
    q, k, v, do = (t.float().numpy() for t in W.make_tensors(w, 0))
    sub, idx = D.shard_workload(w, rank, world_size)
    D.barrier()
    o, lse = O.varlen_fwd(q[idx], k[idx], v[idx], sub.evict_at, sub.cu_seqlens, w.scale)
    dq, dk, dv = O.varlen_bwd(q[idx], k[idx], v[idx], do[idx], sub.evict_at, sub.cu_seqlens, w.scale)
    np.savez(os.path.join(tmpdir, f"r{rank}.npz"), idx=idx, o=o, lse=lse, dq=dq, dk=dk, dv=dv)
    ms, units = D.aggregate(10.0 + rank, float(sub.total_tokens))
    assert ms == 10.0 + (world_size - 1) and units == float(w.total_tokens)
    D.barrier()
    D.shutdown()


def test_two_ranks_shard_by_trace_and_agree_with_unsharded(tmp_path):
    from oracle import kvs_oracle as O
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    w = W.make_workload(3, seed=0, shrink=128, batch=5, Hq=2, Hkv=1)
    q, k, v, do = (t.float().numpy() for t in W.make_tensors(w, 0))
    o, lse = O.varlen_fwd(q, k, v, w.evict_at, w.cu_seqlens, w.scale)
    dq, dk, dv = O.varlen_bwd(q, k, v, do, w.evict_at, w.cu_seqlens, w.scale)
    seen = np.zeros(w.total_tokens, dtype=bool)
    for r in range(2):
        z = np.load(os.path.join(str(tmp_path), f"r{r}.npz"))
        idx = z["idx"]
        assert not seen[idx].any()
        seen[idx] = True
        assert np.array_equal(z["o"], o[idx]) and np.array_equal(z["lse"], lse[:, idx])
        assert np.array_equal(z["dq"], dq[idx]) and np.array_equal(z["dk"], dk[idx]) and np.array_equal(z["dv"], dv[idx])
    assert seen.all()


def test_single_process_aggregate_is_identity():
    assert D.aggregate(3.5, 7.0) == (3.5, 7.0)
    assert not D.active()


# ---- the launcher-less start that `bench.py --gpus N` uses -----------------------------------------
_STUB = r'''
import os, sys, json
sys.path.insert(0, sys.argv[1])
import numpy as np
from oracle import kvs_oracle as O
from paper_2609_35750_b200 import dist as D, workloads as W
rank, world = D.world()
assert int(os.environ["LOCAL_RANK"]) == rank and D.init_from_env(backend="gloo")
w = W.make_workload(0, seed=rank, Hq=2, Hkv=1)               # every rank its own batch of the configuration (weak scaling)
q, k, v, do = (t.float().numpy() for t in W.make_tensors(w, rank))
D.barrier()
o, lse = O.varlen_fwd(q, k, v, w.evict_at, w.cu_seqlens, w.scale)     # stands in for the GPU step
D.barrier()
ms, units = D.aggregate(5.0 + rank, float(W.fwd_bwd_flops(w)))
print("noise from rank", rank)
if rank == 0:
    print(json.dumps({"metric": "stub", "n_gpus": world, "ms": ms, "units": units, "lse0": float(lse[0, 0])}))
D.shutdown()
'''


def test_spawn_local_starts_n_ranks_and_rank0_reports(tmp_path):
    import json
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "stub_rank.py"
    script.write_text(_STUB)
    res = D.spawn_local(2, [sys.executable, str(script), root], timeout=300)
    assert [rc for rc, _ in res] == [0, 0]
    lines = [ln for ln in res[0][1].splitlines() if ln.startswith("{")]
    line = json.loads(lines[-1])
    w = W.make_workload(0, Hq=2, Hkv=1)
    assert line["n_gpus"] == 2 and line["ms"] == 6.0 and line["units"] == 2.0 * W.fwd_bwd_flops(w)
    assert not any(ln.startswith("{") for ln in res[1][1].splitlines())      # only rank 0 reports


def test_bench_gpus_2_without_a_launcher_spawns_ranks_and_fails_loudly_without_cuda():
    # on a machine without a GPU every rank must refuse (there is no CPU path), and the parent must say so
    import subprocess
    if torch.cuda.is_available():
        import pytest
        pytest.skip("a CUDA device is present: this checks the refusal on CPU-only machines")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    p = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "1", "--warmup", "0",
                        "--no-cpu-baseline", "--no-e2e"], env=env, capture_output=True, text=True, timeout=600)
    assert p.returncode != 0
    assert "ranks failed" in p.stderr and "needs a CUDA device" in p.stderr
    assert not any(ln.startswith("{") for ln in p.stdout.splitlines())
