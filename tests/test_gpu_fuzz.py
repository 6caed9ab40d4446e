"""Seeded random shapes against the fp64 oracle: group sizes 1..8 (even, odd, no grouping), both head dims,
batches of ragged traces, four mask families.  Every case runs mask metadata, forward and backward through the
C ABI and compares all five outputs.

Bounds: relative L2 5e-3 as everywhere.  The absolute bound 2e-2 is stated for the named configs; here group size,
trace length and mask are arbitrary.  P and dS are rounded to bf16 (relative rms 1.66e-3) before they are summed into
dv, dk, dq over the G heads of a group and over every query that sees a key, so the first keys of a trace, which every
query sees with a large probability, collect the most noise.  The oracle propagates those roundings to a standard
deviation per element (oracle.rounding_sigma); an element's bound is max(2e-2, six of its standard deviations)."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _case(rng):
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 2, 3, 4, 5, 6, 7, 8]))
    d = int(rng.choice([64, 128, 128]))
    lens = [int(rng.choice([1, 5, 127, 128, 129, 300, 517, 900, 1400])) for _ in range(int(rng.integers(1, 5)))]
    evs = []
    for T in lens:
        ev = np.full(T, int(W.INF), dtype=np.int64)
        mode = int(rng.integers(0, 4))
        if mode == 1:                                   # random lifetimes on 60 % of the keys
            sel = rng.random(T) < 0.6
            ev[sel] = (np.arange(T) + rng.integers(1, 400, size=T))[sel]
        elif mode == 2 and T > 64:                      # keep the last k turns
            turns = rng.integers(16, 200, size=T // 16 + 2)
            ev = W.keep_last_k_evict_at(T, min(32, T // 2), turns, int(rng.integers(1, 4))).astype(np.int64)
        elif mode == 3:                                 # every key short-lived
            ev = np.arange(T) + rng.integers(1, 50, size=T)
        evs.append(np.minimum(ev, int(W.INF)).astype(np.int32))
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return W.Workload("fuzz", cu, np.concatenate(evs), Hkv * G, Hkv, d)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_shapes_match_the_oracle(seed):
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(seed)
    f = lambda t: t.float().cpu().numpy().astype(np.float64)
    for _ in range(16):
        w = _case(rng)
        q, k, v, do = W.make_tensors(w, int(rng.integers(0, 1 << 30)))
        qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
        meta = B.kvs_mask_meta(torch.from_numpy(w.evict_at).cuda(), torch.from_numpy(w.cu_seqlens).cuda(), w.max_seqlen)
        out, lse = B.kvs_attn_fwd(qd, kd, vd, meta, w.batch, w.max_seqlen, w.softmax_scale)
        dq, dk, dv = B.kvs_attn_bwd(dod, qd, kd, vd, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32)
        assert B.kvs_device_status(meta) == B.KVS_OK
        ro, rl = O.varlen_fwd(f(q), f(k), f(v), w.evict_at, w.cu_seqlens, w.scale)
        rdq, rdk, rdv = O.varlen_bwd(f(q), f(k), f(v), f(do), w.evict_at, w.cu_seqlens, w.scale)
        sg = O.varlen_rounding_sigma(f(q), f(k), f(v), f(do), w.evict_at, w.cu_seqlens, w.scale)
        what = dict(Hq=w.Hq, Hkv=w.Hkv, d=w.d, lens=np.diff(w.cu_seqlens).tolist())
        for name, got, ref in (("out", out, ro), ("lse", lse, rl), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
            g = f(got)
            assert np.isfinite(g).all(), (name, what)
            bound = np.maximum(2e-2, 6.0 * sg[name]) if name in sg and name != "out" else 2e-2
            assert (np.abs(g - ref) <= bound).all(), (name, what, float(np.abs(g - ref).max()))
            nref = np.linalg.norm(ref)
            if nref > 1e-3:
                assert np.linalg.norm(g - ref) / nref <= 5e-3, (name, what)


def test_many_short_traces():
    # a packed batch of 300 traces of 1..200 tokens: many block -> trace lookups, class matrices of one or two tiles,
    # offsets that are rarely multiples of anything
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(21)
    lens = rng.integers(1, 201, size=300)
    evs = []
    for T in lens:
        ev = np.full(T, int(W.INF), dtype=np.int64)
        sel = rng.random(T) < 0.5
        ev[sel] = (np.arange(T) + rng.integers(1, 60, size=T))[sel]
        evs.append(ev.astype(np.int32))
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    w = W.Workload("many", cu, np.concatenate(evs), 4, 2, 64)
    q, k, v, do = W.make_tensors(w, 21)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
    meta = B.kvs_mask_meta(torch.from_numpy(w.evict_at).cuda(), torch.from_numpy(w.cu_seqlens).cuda(), w.max_seqlen)
    out, lse = B.kvs_attn_fwd(qd, kd, vd, meta, w.batch, w.max_seqlen, w.softmax_scale)
    dq, dk, dv = B.kvs_attn_bwd(dod, qd, kd, vd, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32)
    assert B.kvs_device_status(meta) == B.KVS_OK
    cls, kmin, kmax = B.kvs_mask_meta_export(meta, w.cu_seqlens, w.total_tokens, w.max_seqlen)
    assert np.array_equal(cls, np.concatenate([O.tile_classes_rule(w.trace(b)).ravel() for b in range(w.batch)]))
    f = lambda t: t.float().cpu().numpy().astype(np.float64)
    ro, rl = O.varlen_fwd(f(q), f(k), f(v), w.evict_at, w.cu_seqlens, w.scale)
    rdq, rdk, rdv = O.varlen_bwd(f(q), f(k), f(v), f(do), w.evict_at, w.cu_seqlens, w.scale)
    for name, got, ref in (("out", out, ro), ("lse", lse, rl), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        g = f(got)
        assert np.isfinite(g).all() and np.abs(g - ref).max() <= 2e-2, (name, float(np.abs(g - ref).max()))
        assert np.linalg.norm(g - ref) / np.linalg.norm(ref) <= 5e-3, name
