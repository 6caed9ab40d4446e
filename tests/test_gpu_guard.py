"""Out-of-bounds writes, unwritten outputs and a mismatched meta buffer (needs a B200).

Every output and scratch buffer of a call is fenced and poisoned (tests/guard.py): after the call the
guard bands must be untouched and no output element may still hold the poison.  The cases are chosen for
the code paths that could overstep: the backward's reduce-add of whole 128-row boxes where a trace ends
inside a tile and the next trace (or the end of the tensor) follows, both gradient types, the
allocation-free backward, and decode attention over a cache that is exactly as large as its pages, so
that a page box reaching past it would read poison.  Results are still compared with the oracle, so a
stray READ of poison shows up as a non-finite value.
"""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import binding as B
from paper_2609_35750_b200 import workloads as W
from tests.guard import Fenced

pytestmark = pytest.mark.gpu
DEV = "cuda"
MAX_ABS, REL_L2 = 2e-2, 5e-3


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _close(name, got, ref, max_abs=MAX_ABS):
    got = _f64(got) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    assert np.isfinite(got).all(), f"{name}: non-finite values"
    err = np.abs(got - ref).max()
    assert err <= max_abs, f"{name}: max-abs {err:.4f}"
    n = np.linalg.norm(ref)
    if n > 1e-3:
        assert np.linalg.norm(got - ref) / n <= REL_L2, name


def _fenced_inputs(w, seed):
    q, k, v, do = W.make_tensors(w, seed)
    row = w.Hq * w.d * 2
    fq = Fenced(q.shape, torch.bfloat16, 130 * row, fill_from=q.to(DEV))
    fk = Fenced(k.shape, torch.bfloat16, 130 * row, fill_from=k.to(DEV))
    fv = Fenced(v.shape, torch.bfloat16, 130 * row, fill_from=v.to(DEV))
    fdo = Fenced(do.shape, torch.bfloat16, 130 * row, fill_from=do.to(DEV))
    return (q, k, v, do), (fq, fk, fv, fdo)


def _run_fenced(w, seed, grad_dtype, noalloc=False):
    """Metadata + forward + backward with every buffer fenced.  Returns host inputs and device outputs."""
    host, (fq, fk, fv, fdo) = _fenced_inputs(w, seed)
    Tt, Hq, Hkv, d = w.total_tokens, w.Hq, w.Hkv, w.d
    gdt = torch.float32 if grad_dtype == B.GRAD_FP32 else torch.bfloat16
    gsz = 4 if grad_dtype == B.GRAD_FP32 else 2
    guard = 130 * Hq * d * 4                                   # more than a 128-row box of the widest tensor
    ev = torch.from_numpy(w.evict_at).to(DEV)
    cu = torch.from_numpy(w.cu_seqlens).to(DEV)
    fmeta = Fenced((B.kvs_mask_meta_bytes(w.batch, Tt, w.max_seqlen),), torch.uint8, 1 << 16)
    fout = Fenced((Tt, Hq, d), torch.bfloat16, guard)
    flse = Fenced((Hq, Tt), torch.float32, guard)
    fdq = Fenced((Tt, Hq, d), gdt, guard)
    fdk = Fenced((Tt, Hkv, d), gdt, guard)
    fdv = Fenced((Tt, Hkv, d), gdt, guard)
    B.kvs_mask_meta(ev, cu, w.max_seqlen, meta_buf=fmeta.t)
    B.kvs_attn_fwd(fq.t, fk.t, fv.t, fmeta.t, w.batch, w.max_seqlen, w.softmax_scale, out=fout.t, lse=flse.t)
    if noalloc:
        B.kvs_attn_bwd_noalloc(fdo.t, fq.t, fk.t, fv.t, fout.t, flse.t, fmeta.t, w.batch, w.max_seqlen, w.softmax_scale,
                               dq=fdq.t, dk=fdk.t, dv=fdv.t)
        fws = None
    else:
        fws = Fenced((B.kvs_attn_bwd_workspace_bytes(Tt, Hq, Hkv, d, grad_dtype),), torch.uint8, guard)
        B.kvs_attn_bwd(fdo.t, fq.t, fk.t, fv.t, fout.t, flse.t, fmeta.t, w.batch, w.max_seqlen, w.softmax_scale, grad_dtype,
                       dq=fdq.t, dk=fdk.t, dv=fdv.t, workspace=fws.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(fmeta.t) == B.KVS_OK
    if fws is not None:
        assert B.kvs_device_status(fws.t) == B.KVS_OK
        fws.check("workspace", written=False)
    fmeta.check("meta_buf", written=False)
    for name, f in (("q", fq), ("k", fk), ("v", fv), ("dout", fdo)):
        f.check(name)                                         # inputs: bands intact, and nobody scribbled NaNs into them
    for name, f in (("out", fout), ("lse", flse), ("dq", fdq), ("dk", fdk), ("dv", fdv)):
        f.check(name)
    return host, (fout.t, flse.t, fdq.t, fdk.t, fdv.t)


def _custom(lens, evs, Hq, Hkv, d):
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    return W.Workload("custom", cu, np.concatenate(evs).astype(np.int32), Hq, Hkv, d)


def _rand_ev(T, rng, maxlife):
    ev = np.full(T, int(W.INF), dtype=np.int64)
    sel = rng.random(T) < 0.5
    ev[sel] = (np.arange(T) + rng.integers(1, maxlife + 1, size=T))[sel]
    return ev.astype(np.int32)


@pytest.mark.parametrize("grad", ["fp32", "bf16", "noalloc"])
@pytest.mark.parametrize("lens,Hq,Hkv,d", [
    ([300, 200, 77], 4, 2, 128),          # every trace ends inside a tile; the last one ends the tensor mid-tile
    ([129, 1, 255], 3, 1, 64),            # a one-token trace between two ragged ones, an odd group
    ([512], 8, 2, 128),                   # whole tiles only
])
def test_nothing_written_outside_and_nothing_left_unwritten(grad, lens, Hq, Hkv, d):
    rng = np.random.default_rng(len(lens) * 1000 + Hq)
    w = _custom(lens, [_rand_ev(T, rng, 260) for T in lens], Hq, Hkv, d)
    gd = B.GRAD_BF16 if grad == "bf16" else B.GRAD_FP32
    (q, k, v, do), (out, lse, dq, dk, dv) = _run_fenced(w, 21, gd, noalloc=(grad == "noalloc"))
    ro, rl = O.varlen_fwd(_f64(q), _f64(k), _f64(v), w.evict_at, w.cu_seqlens, w.scale)
    rdq, rdk, rdv = O.varlen_bwd(_f64(q), _f64(k), _f64(v), _f64(do), w.evict_at, w.cu_seqlens, w.scale)
    sg = O.varlen_rounding_sigma(_f64(q), _f64(k), _f64(v), _f64(do), w.evict_at, w.cu_seqlens, w.scale)
    _close("out", out, ro)
    _close("lse", lse, rl)
    for name, got, ref in (("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        g = _f64(got)
        assert np.isfinite(g).all(), name
        half_ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 8) if grad == "bf16" else 0.0
        bound = np.maximum(MAX_ABS, 6.0 * sg[name] + half_ulp)
        assert (np.abs(g - ref) <= bound).all(), (name, float(np.abs(g - ref).max()))
        assert np.linalg.norm(g - ref) / np.linalg.norm(ref) <= REL_L2, name


def test_shrunk_config3_ragged_batch_fenced():
    w = W.make_workload(3, seed=2, shrink=32, Hq=8, Hkv=2, batch=4)
    (q, k, v, do), (out, lse, dq, dk, dv) = _run_fenced(w, 22, B.GRAD_BF16)
    ro, rl = O.varlen_fwd(_f64(q), _f64(k), _f64(v), w.evict_at, w.cu_seqlens, w.scale)
    _close("out", out, ro)
    _close("lse", lse, rl)


# ---- a meta buffer that does not belong to the call ---------------------------------------------------
@pytest.mark.parametrize("kind", ["other_max_seqlen", "other_batch", "zero_filled"])
def test_mismatched_meta_is_refused_on_the_device_and_outputs_stay_untouched(kind):
    w = W.make_workload(2, seed=1, shrink=32, Hq=4, Hkv=2, batch=2)
    q, k, v, do = (t.to(DEV) for t in W.make_tensors(w, 1))
    Tt, Hq, Hkv, d = w.total_tokens, w.Hq, w.Hkv, w.d
    ev = torch.from_numpy(w.evict_at).to(DEV)
    cu = torch.from_numpy(w.cu_seqlens).to(DEV)
    good = B.kvs_mask_meta(ev, cu, w.max_seqlen)
    out, lse = B.kvs_attn_fwd(q, k, v, good, w.batch, w.max_seqlen, w.softmax_scale)
    if kind == "other_max_seqlen":
        # a valid buffer, but built with another (still sufficient) max_seqlen: its arrays sit at other offsets
        meta = B.kvs_mask_meta(ev, cu, w.max_seqlen + 512)
        call_batch, call_msl = w.batch, w.max_seqlen
    elif kind == "other_batch":
        cu1 = torch.tensor([0, Tt], dtype=torch.int32, device=DEV)
        ev1 = torch.full((Tt,), int(W.INF), dtype=torch.int32, device=DEV)
        meta = B.kvs_mask_meta(ev1, cu1, Tt)
        call_batch, call_msl = w.batch, Tt
    else:
        meta = torch.zeros(B.kvs_mask_meta_bytes(w.batch, Tt, w.max_seqlen), dtype=torch.uint8, device=DEV)
        call_batch, call_msl = w.batch, w.max_seqlen
    fout = Fenced((Tt, Hq, d), torch.bfloat16, 1 << 18)
    flse = Fenced((Hq, Tt), torch.float32, 1 << 18)
    B.kvs_attn_fwd(q, k, v, meta, call_batch, call_msl, w.softmax_scale, out=fout.t, lse=flse.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(meta) == B.KVS_ERR_BAD_META
    assert fout.untouched() and flse.untouched() and fout.guards_intact() and flse.guards_intact()
    # backward: the refusal lands in the workspace's status word, the gradients stay untouched
    fdq = Fenced((Tt, Hq, d), torch.float32, 1 << 18)
    fdk = Fenced((Tt, Hkv, d), torch.float32, 1 << 18)
    fdv = Fenced((Tt, Hkv, d), torch.float32, 1 << 18)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, Hq, Hkv, d, B.GRAD_FP32), dtype=torch.uint8, device=DEV)
    B.kvs_attn_bwd(do, q, k, v, out, lse, meta, call_batch, call_msl, w.softmax_scale, B.GRAD_FP32,
                   dq=fdq.t, dk=fdk.t, dv=fdv.t, workspace=ws)
    torch.cuda.synchronize()
    assert B.kvs_device_status(ws) == B.KVS_ERR_BAD_META
    assert fdk.untouched() and fdv.untouched() and fdk.guards_intact() and fdv.guards_intact() and fdq.guards_intact()
    # the device is still usable and the right buffer still works
    out2, lse2 = B.kvs_attn_fwd(q, k, v, good, w.batch, w.max_seqlen, w.softmax_scale)
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    assert B.kvs_device_status(good) == B.KVS_OK


# ---- decode attention over a cache that is exactly as large as its pages ----------------------------------
def _decode_ref(q, kc, vc, table, n, ps, scale):
    """Plain definition over the rows the table names (fp64)."""
    S, Hq, d = q.shape
    Hkv = kc.shape[2]
    G = Hq // Hkv
    out = np.zeros((S, Hq, d))
    lse = np.full((S, Hq), -np.inf)
    for s in range(S):
        rows = [(table[s][t // ps], t % ps) for t in range(n[s])]
        if not rows:
            continue
        for h in range(Hq):
            g = h // G
            K = np.stack([kc[p, o, g] for p, o in rows])
            V = np.stack([vc[p, o, g] for p, o in rows])
            x = scale * (K @ q[s, h])
            m = x.max()
            e = np.exp(x - m)
            out[s, h] = (e / e.sum()) @ V
            lse[s, h] = m + np.log(e.sum())
    return out, lse


@pytest.mark.parametrize("ps,G,d", [(16, 4, 128), (1, 4, 128), (16, 2, 64), (8, 8, 128)])
def test_decode_reads_only_its_pages_and_writes_only_its_outputs(ps, G, d):
    rng = np.random.default_rng(ps * 100 + G)
    S, Hkv = 3, 2
    Hq = Hkv * G
    lens = [5 * ps + max(1, ps // 2), 130 if ps == 1 else 9 * ps, ps]          # ends inside a page, long, exactly one page
    pages_per_seq = [(n + ps - 1) // ps for n in lens]
    num_pages = sum(pages_per_seq)                                             # not one page to spare
    max_pages = max(pages_per_seq)
    cache = B.PagedCache(num_pages, ps, S, max_pages, Hkv, d)
    g = torch.Generator().manual_seed(5)
    kc = torch.randn((num_pages, ps, Hkv, d), generator=g).to(torch.bfloat16)
    vc = torch.randn((num_pages, ps, Hkv, d), generator=g).to(torch.bfloat16)
    fk = Fenced(kc.shape, torch.bfloat16, 1 << 20, fill_from=kc.to(DEV))
    fv = Fenced(vc.shape, torch.bfloat16, 1 << 20, fill_from=vc.to(DEV))
    cache.k_cache, cache.v_cache = fk.t, fv.t
    perm = rng.permutation(num_pages)                                          # the last page of the cache is in use
    table, pos = [], 0
    bt = np.zeros((S, max_pages), dtype=np.int32)
    for s in range(S):
        table.append(perm[pos:pos + pages_per_seq[s]].tolist())
        bt[s, :pages_per_seq[s]] = table[s]
        pos += pages_per_seq[s]
    cache.block_table.copy_(torch.from_numpy(bt))
    cache.n_tokens.copy_(torch.tensor(lens, dtype=torch.int32))
    q = torch.randn((S, Hq, d), generator=g).to(torch.bfloat16)
    splits = 2
    fout = Fenced((S, Hq, d), torch.bfloat16, 1 << 16)
    flse = Fenced((S, Hq), torch.float32, 1 << 16)
    fws = Fenced((int(B.load().kvs_decode_workspace_bytes(S, Hq, d, splits)),), torch.uint8, 1 << 16)
    cache.decode(q.to(DEV), num_splits=splits, out=fout.t, lse=flse.t, workspace=fws.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(fws.t) == B.KVS_OK
    for name, f in (("out", fout), ("lse", flse)):
        f.check(name)
    fws.check("workspace", written=False)
    fk.check("k_cache")
    fv.check("v_cache")
    ro, rl = _decode_ref(_f64(q), _f64(kc), _f64(vc), table, lens, ps, 1.0 / np.sqrt(d))
    _close("out", fout.t, ro)
    _close("lse", flse.t, rl)
    # a table entry that names no page of the cache is reported, not followed
    bt_bad = bt.copy()
    bt_bad[1, 2] = num_pages + 5
    cache.block_table.copy_(torch.from_numpy(bt_bad))
    cache.decode(q.to(DEV), num_splits=splits, out=fout.t, lse=flse.t, workspace=fws.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(fws.t) == B.KVS_ERR_INVALID_ARG
    assert fout.guards_intact() and flse.guards_intact() and fws.guards_intact()
    bt_bad[1, 2] = -3
    cache.block_table.copy_(torch.from_numpy(bt_bad))
    cache.decode(q.to(DEV), num_splits=splits, out=fout.t, lse=flse.t, workspace=fws.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(fws.t) == B.KVS_ERR_INVALID_ARG
