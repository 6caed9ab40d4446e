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
