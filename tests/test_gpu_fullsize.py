"""Full-size configurations, in the launch configuration bench.py times (needs a B200).

The oracle cannot produce whole tensors at these sizes, so each config is checked by
  * mask metadata: bit-exact against the oracle's min/max rule on every tile;
  * sampled query rows (first/last rows, rows around every kind of eviction boundary and
    tile edge, random rows): out, lse and dq rows computed one by one by the oracle;
  * a backward run whose dout is zero except on a few sampled rows of one KV-head group:
    by linearity dq, dk and dv are then the sum of those rows' contributions, which the oracle
    computes row by row, and the comparison covers EVERY element of dq, dk, dv (the kernels
    take no shortcut on zeros, and every other group must come out exactly zero);
  * dk, dv of the last keys of a trace with the dense dout (few rows see them);
  * zero-query live-key counts on every row, and the scalar gradient identities.
"""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import binding as B
from paper_2609_35750_b200 import workloads as W

pytestmark = pytest.mark.gpu

MAX_ABS = 2e-2
REL_L2 = 5e-3
DEV = "cuda"

CASES = [
    ("cfg1", dict(cfg=1)),
    ("cfg2", dict(cfg=2)),
    ("cfg3", dict(cfg=3)),
    ("cfg4", dict(cfg=4)),
    ("cfg4_control", dict(cfg=4, variant="control")),
    ("cfg6_markovian_pick", dict(cfg=6)),          # non-monotone evict_at at full size
]


def _np64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _sample_rows(ev, rng, n_random):
    """Stratified rows of one trace: ends, eviction boundaries +-1, tile edges, random."""
    T = ev.shape[0]
    rows = {0, T - 1, min(127, T - 1), min(128, T - 1), max(T - 129, 0), max(T - 128, 0)}
    fin = np.unique(ev[ev < T])
    for e in fin[:: max(1, len(fin) // 6)][:6]:
        rows.update({int(e) - 1, int(e), min(int(e) + 1, T - 1)})
    change = np.nonzero(np.diff(ev.astype(np.int64)) != 0)[0]
    for c in change[:: max(1, len(change) // 4)][:4]:
        rows.update({int(c), int(c) + 1})
    rows.update(int(x) for x in rng.integers(0, T, size=n_random))
    return sorted(r for r in rows if 0 <= r < T)


def _cmp(name, got, ref, max_abs=MAX_ABS):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    assert np.isfinite(got).all(), name
    assert np.abs(got - ref).max() <= max_abs, f"{name}: max-abs {np.abs(got - ref).max():.4f}"
    if np.linalg.norm(ref) > 1e-3:
        rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert rel <= REL_L2, f"{name}: rel-L2 {rel:.3e}"


@pytest.mark.parametrize("name,kw", CASES)
def test_full_size(name, kw):
    w = W.make_workload(seed=0, **kw)
    G = w.Hq // w.Hkv
    rng = np.random.default_rng(11)
    q, k, v, do = W.make_tensors(w, seed=0, device=DEV)
    ev_d = torch.from_numpy(w.evict_at).to(DEV)
    cu_d = torch.from_numpy(w.cu_seqlens).to(DEV)
    Tt = w.total_tokens

    # ---- the bench's launch configuration: meta + fwd + bwd with bf16 gradients ---------------
    meta = B.kvs_mask_meta(ev_d, cu_d, w.max_seqlen)
    out, lse = B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, w.Hq, w.Hkv, w.d, B.GRAD_BF16), dtype=torch.uint8, device=DEV)
    dq, dk, dv = B.kvs_attn_bwd(do, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_BF16, workspace=ws)
    assert B.kvs_device_status(meta) == B.KVS_OK and B.kvs_device_status(ws) == B.KVS_OK
    for t in (out, lse, dq, dk, dv):
        assert bool(torch.isfinite(t).all())

    # ---- metadata, every tile ---------------------------------------------------------------------
    cls, kmin, kmax = B.kvs_mask_meta_export(meta, w.cu_seqlens, Tt, w.max_seqlen)
    assert np.array_equal(cls, np.concatenate([O.tile_classes_rule(w.trace(b)).ravel() for b in range(w.batch)]))
    mm = [O.block_minmax(w.trace(b)) for b in range(w.batch)]
    assert np.array_equal(kmin, np.concatenate([a for a, _ in mm])) and np.array_equal(kmax, np.concatenate([b for _, b in mm]))

    # ---- scalar identities on the dense run (bf16 gradients, loose) -------------------------------
    qf, kf, vf = q.float(), k.float(), v.float()
    lhs = (qf * dq.float()).sum(dim=(0, 2)).view(w.Hkv, G).sum(1).double()
    rhs = (kf * dk.float()).sum(dim=(0, 2)).double()
    scale_ref = float((qf * dq.float()).abs().sum() / np.sqrt(qf.numel())) + 1e-6
    assert float((lhs - rhs).abs().max()) <= 0.2 * scale_ref, (lhs, rhs, scale_ref)
    dsum = (do.float() * out.float()).sum(dim=(0, 2)).view(w.Hkv, G).sum(1).double()
    vsum = (vf * dv.float()).sum(dim=(0, 2)).double()
    scale_ref = float((vf * dv.float()).abs().sum() / np.sqrt(vf.numel())) + 1e-6
    assert float((dsum - vsum).abs().max()) <= 0.2 * scale_ref, (dsum, vsum, scale_ref)
    del qf, kf, vf

    # ---- fp32 gradients for the element checks ----------------------------------------------------
    del dq, ws
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, w.Hq, w.Hkv, w.d, B.GRAD_FP32), dtype=torch.uint8, device=DEV)
    dq, dk32, dv32 = B.kvs_attn_bwd(do, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32, workspace=ws)

    traces = sorted(set([0, w.batch - 1, int(rng.integers(0, w.batch))]))
    budget_rows = 200 // len(traces)
    sparse_rows = []            # (b, i) rows that get a non-zero dout in the sparse run
    g_sel = int(rng.integers(0, w.Hkv))
    host_kv = {}
    for b in traces:
        a, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        ev = w.trace(b)
        kb, vb = _np64(k[a:e, g_sel]), _np64(v[a:e, g_sel])
        host_kv[b] = (kb, vb)
        rows = _sample_rows(ev, rng, max(8, budget_rows - 30))
        got_o, ref_o, got_l, ref_l, got_dq, ref_dq = [], [], [], [], [], []
        for i in rows:
            h = g_sel * G + int(rng.integers(0, G))
            o, l, dqi, *_ = O.row_fwd_bwd(_np64(q[a + i, h]), kb, vb, _np64(do[a + i, h]), ev, i, w.scale)
            ref_o.append(o); ref_l.append(l); ref_dq.append(dqi)
            got_o.append(_np64(out[a + i, h])); got_l.append(float(lse[h, a + i])); got_dq.append(_np64(dq[a + i, h]))
        _cmp(f"{name} trace {b} out rows", np.stack(got_o), np.stack(ref_o))
        _cmp(f"{name} trace {b} lse rows", np.array(got_l), np.array(ref_l))
        _cmp(f"{name} trace {b} dq rows", np.stack(got_dq), np.stack(ref_dq))
        sparse_rows += [(b, i) for i in rows[:: max(1, len(rows) // 12)][:12]]

        # dk, dv of the last keys of the trace under the dense dout
        T = e - a
        j0 = max(0, T - 72)
        # float32 host copies hold the bf16 values exactly; the oracle widens each row to fp64
        bk, bv = O.key_block_dkdv(q[a:e, g_sel * G:(g_sel + 1) * G].float().cpu().numpy(), kb[:, None, :], vb[:, None, :],
                                  do[a:e, g_sel * G:(g_sel + 1) * G].float().cpu().numpy(), ev, j0, T, 0, G, w.scale)
        _cmp(f"{name} trace {b} dk tail", _np64(dk32[a + j0:e, g_sel]), bk)
        _cmp(f"{name} trace {b} dv tail", _np64(dv32[a + j0:e, g_sel]), bv)

    # ---- sparse dout: every element of dq, dk, dv --------------------------------------------------
    do_s = torch.zeros_like(do)
    ref_dq = {}
    ref_dk = np.zeros((Tt, w.d))
    ref_dv = np.zeros((Tt, w.d))
    for (b, i) in sparse_rows:
        a = int(w.cu_seqlens[b])
        kb, vb = host_kv[b]
        for h in range(g_sel * G, (g_sel + 1) * G):
            do_s[a + i, h] = do[a + i, h]
            _, _, dqi, vis, dkc, dvc = O.row_fwd_bwd(_np64(q[a + i, h]), kb, vb, _np64(do[a + i, h]), w.trace(b), i, w.scale)
            ref_dq[(a + i, h)] = dqi
            ref_dk[a + vis] += dkc
            ref_dv[a + vis] += dvc
    dq_s, dk_s, dv_s = B.kvs_attn_bwd(do_s, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32, workspace=ws)
    assert B.kvs_device_status(ws) == B.KVS_OK
    _cmp(f"{name} sparse dk", _np64(dk_s[:, g_sel]), ref_dk)
    _cmp(f"{name} sparse dv", _np64(dv_s[:, g_sel]), ref_dv)
    others = [g for g in range(w.Hkv) if g != g_sel]
    if others:
        assert float(dk_s[:, others].abs().max()) == 0.0 and float(dv_s[:, others].abs().max()) == 0.0
    keys = sorted(ref_dq)
    got = np.stack([_np64(dq_s[t, h]) for (t, h) in keys])
    _cmp(f"{name} sparse dq rows", got, np.stack([ref_dq[kk] for kk in keys]))
    mask = torch.ones((Tt, w.Hq), dtype=torch.bool, device=DEV)
    for (t, h) in keys:
        mask[t, h] = False
    assert float(dq_s[mask].abs().max()) == 0.0            # rows with dout = 0 get exactly zero
    del dq_s, dk_s, dv_s, do_s, dq, dk32, dv32, mask

    # ---- zero queries: exp(lse) counts the live keys on every row ----------------------------------
    out0, lse0 = B.kvs_attn_fwd(torch.zeros_like(q), k, v, meta, w.batch, w.max_seqlen, w.softmax_scale)
    n_gpu = torch.exp(lse0[0].double()).cpu().numpy()
    live = []
    for b in range(w.batch):
        ev = w.trace(b).astype(np.int64)
        T = ev.shape[0]
        delta = np.zeros(T + 1, dtype=np.int64)
        np.add.at(delta, np.arange(T), 1)
        np.add.at(delta, np.minimum(ev, T), -1)
        live.append(np.cumsum(delta)[:T])
    live = np.concatenate(live)
    assert np.abs(n_gpu / live - 1.0).max() < 2e-4
    del out0, lse0
    torch.cuda.empty_cache()


def test_full_size_token_level_with_reordered_keys():
    # config 4 in the launch configuration bench.py times for its "keys re-ordered" line: window 4096, bf16 gradients.
    # Checked against the oracle on sampled rows and on the metadata of every tile, and against the plain-order run of the
    # same inputs (which test_full_size[cfg4] checks against the oracle) on every element.
    w = W.make_workload(4, seed=0)
    G = w.Hq // w.Hkv
    rng = np.random.default_rng(12)
    q, k, v, do = W.make_tensors(w, seed=0, device=DEV)
    ev_d = torch.from_numpy(w.evict_at).to(DEV)
    cu_d = torch.from_numpy(w.cu_seqlens).to(DEV)
    Tt = w.total_tokens
    perm, kf, ke = B.kvs_reorder_keys(ev_d, cu_d, w.max_seqlen, 4096)
    ref_perm = O.reorder_keys(w.trace(0), 4096)
    assert np.array_equal(perm.cpu().numpy(), ref_perm)
    kp, vp = B.kvs_permute_rows(k, perm), B.kvs_permute_rows(v, perm)
    meta = B.kvs_mask_meta_keys(kf, ke, cu_d, w.max_seqlen)
    cls, kmin, kmax = B.kvs_mask_meta_export(meta, w.cu_seqlens, Tt, w.max_seqlen)
    ref_cls = O.tile_classes_rule(w.evict_at[ref_perm], key_first=ref_perm)
    assert np.array_equal(cls, ref_cls.ravel())
    assert (ref_cls != O.EMPTY).sum() * 1.6 < 524800                      # 1.67x fewer tiles than the causal triangle
    out, lse = B.kvs_attn_fwd(q, kp, vp, meta, w.batch, w.max_seqlen, w.softmax_scale)
    ws = torch.empty(B.kvs_attn_bwd_workspace_bytes(Tt, w.Hq, w.Hkv, w.d, B.GRAD_BF16), dtype=torch.uint8, device=DEV)
    dq, dkp, dvp = B.kvs_attn_bwd(do, q, kp, vp, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_BF16, workspace=ws)
    assert B.kvs_device_status(meta) == B.KVS_OK and B.kvs_device_status(ws) == B.KVS_OK
    dk, dv = B.kvs_permute_rows(dkp, perm, inverse=True), B.kvs_permute_rows(dvp, perm, inverse=True)
    # sampled rows against the oracle
    g_sel = int(rng.integers(0, w.Hkv))
    ev = w.trace(0)
    kb, vb = _np64(k[:, g_sel]), _np64(v[:, g_sel])
    rows = _sample_rows(ev, rng, 40)
    got_o, ref_o, got_l, ref_l, got_dq, ref_dq = [], [], [], [], [], []
    for i in rows:
        h = g_sel * G + int(rng.integers(0, G))
        o, l, dqi, *_ = O.row_fwd_bwd(_np64(q[i, h]), kb, vb, _np64(do[i, h]), ev, i, w.scale)
        ref_o.append(o); ref_l.append(l); ref_dq.append(dqi)
        got_o.append(_np64(out[i, h])); got_l.append(float(lse[h, i])); got_dq.append(_np64(dq[i, h]))
    _cmp("reordered out rows", np.stack(got_o), np.stack(ref_o))
    _cmp("reordered lse rows", np.array(got_l), np.array(ref_l))
    ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(np.stack(ref_dq)), 1e-30))) - 7)
    assert (np.abs(np.stack(got_dq) - np.stack(ref_dq)) <= np.maximum(MAX_ABS, ulp)).all()
    # every element against the plain key order
    del kp, vp, dkp, dvp
    meta0 = B.kvs_mask_meta(ev_d, cu_d, w.max_seqlen)
    out0, lse0 = B.kvs_attn_fwd(q, k, v, meta0, w.batch, w.max_seqlen, w.softmax_scale)
    dq0, dk0, dv0 = B.kvs_attn_bwd(do, q, k, v, out0, lse0, meta0, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_BF16, workspace=ws)
    # two bf16 results of the same quantity, each within its own rounding of it
    for name, a, b in (("out", out, out0), ("dq", dq, dq0), ("dk", dk, dk0), ("dv", dv, dv0)):
        d = (a.float() - b.float()).abs()
        tol = torch.clamp(2.0 ** (torch.floor(torch.log2(b.float().abs().clamp_min(1e-30))) - 6), min=MAX_ABS)
        assert bool((d <= tol).all()), (name, float(d.max()))
        assert float((a.float() - b.float()).norm() / b.float().norm()) <= REL_L2, name
    assert float((lse - lse0).abs().max()) <= 1e-3


def test_full_size_student_and_teacher_forward():
    # kvs_attn_fwd_dual on config 2 at full size (the call bench.py --path dual times): sampled rows of both streams
    # against the oracle, the student stream against the plain forward bit for bit
    w = W.make_workload(2, seed=0)
    G = w.Hq // w.Hkv
    rng = np.random.default_rng(13)
    q, k, v, _ = W.make_tensors(w, seed=0, device=DEV, with_dout=False)
    ev_d = torch.from_numpy(w.evict_at).to(DEV)
    cu_d = torch.from_numpy(w.cu_seqlens).to(DEV)
    meta = B.kvs_mask_meta(ev_d, cu_d, w.max_seqlen)
    meta_e = B.kvs_mask_meta_evicted(ev_d, cu_d, w.max_seqlen)
    os_, ls_, ot_, lt_ = B.kvs_attn_fwd_dual(q, k, v, meta, meta_e, w.batch, w.max_seqlen, w.softmax_scale)
    assert B.kvs_device_status(meta) == B.KVS_OK and B.kvs_device_status(meta_e) == B.KVS_OK
    out, lse = B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale)
    assert torch.equal(out, os_) and torch.equal(lse, ls_)
    for b in range(w.batch):
        a, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        evb = w.trace(b)
        inf = np.full(e - a, O.INF, dtype=np.int64)
        g_sel = int(rng.integers(0, w.Hkv))
        kb, vb = _np64(k[a:e, g_sel]), _np64(v[a:e, g_sel])
        rows = _sample_rows(evb, rng, 24)
        got_s, ref_s, got_t, ref_t, gl, rl = [], [], [], [], [], []
        for i in rows:
            h = g_sel * G + int(rng.integers(0, G))
            o_s, l_s, _, _ = O.row_fwd(_np64(q[a + i, h]), kb, vb, evb, i, w.scale)
            o_t, l_t, _, _ = O.row_fwd(_np64(q[a + i, h]), kb, vb, inf, i, w.scale)
            ref_s.append(o_s); ref_t.append(o_t); rl += [l_s, l_t]
            got_s.append(_np64(os_[a + i, h])); got_t.append(_np64(ot_[a + i, h])); gl += [float(ls_[h, a + i]), float(lt_[h, a + i])]
        _cmp(f"trace {b} student rows", np.stack(got_s), np.stack(ref_s))
        # the teacher is merged from two bf16 partial results: up to half an ulp more than a once-rounded output
        ref_t = np.stack(ref_t)
        ulp_half = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref_t), 1e-30))) - 8)
        assert (np.abs(np.stack(got_t) - ref_t) <= MAX_ABS + ulp_half).all()
        assert np.linalg.norm(np.stack(got_t) - ref_t) / np.linalg.norm(ref_t) <= REL_L2
        _cmp(f"trace {b} lse rows", np.array(gl), np.array(rl))
    # the teacher's normaliser counts every causal key: with q = 0, exp(lse_teacher) = i + 1
    z = torch.zeros_like(q)
    _, _, _, lt0 = B.kvs_attn_fwd_dual(z, k, v, meta, meta_e, w.batch, w.max_seqlen, w.softmax_scale)
    n_gpu = torch.exp(lt0[0].double()).cpu().numpy()
    want = np.concatenate([np.arange(1, int(w.cu_seqlens[b + 1] - w.cu_seqlens[b]) + 1) for b in range(w.batch)])
    assert np.abs(n_gpu / want - 1.0).max() < 2e-4
