"""Key slots with their own visibility interval, and the key order for token-level eviction.

CPU: the oracle's general mask (slot j visible to query i iff key_first[j] <= i < key_evict[j]) is pinned by
permutation invariance against the plain form, by brute-force loops, by the rule-vs-brute-force tile classes on
random intervals, and by the union identity (student part + evicted part = full causal attention).  GPU: the
re-ordered path through the C ABI against the oracle in the ORIGINAL key order, metadata bit-exact, fenced."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

MAX_ABS, REL_L2 = 2e-2, 5e-3


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def _rand_trace(T, seed, frac=0.6, maxlife=200):
    r = np.random.default_rng(seed)
    ev = np.full(T, int(W.INF), dtype=np.int64)
    sel = r.random(T) < frac
    ev[sel] = (np.arange(T) + r.integers(1, maxlife + 1, size=T))[sel]
    return ev.astype(np.int32)


# ---- CPU ------------------------------------------------------------------------------------------------
def test_reorder_keys_by_hand_and_properties():
    #            j: 0   1  2  3   4  5   6  7
    ev = np.array([9, 100, 3, 9, 100, 7, 100, 8])
    assert O.reorder_keys(ev, 4).tolist() == [2, 0, 3, 1, 5, 7, 4, 6]       # two windows of four, ties by index
    assert O.reorder_keys(ev, 8).tolist() == [2, 5, 7, 0, 3, 1, 4, 6]
    assert O.reorder_keys(ev, 1).tolist() == list(range(8))
    ev = _rand_trace(1000, 1)
    for window in (7, 128, 4096):
        p = O.reorder_keys(ev, window)
        assert sorted(p.tolist()) == list(range(1000))
        for w0 in range(0, 1000, window):
            seg = p[w0:w0 + window]
            assert seg.min() == w0 and seg.max() == min(w0 + window, 1000) - 1              # stays inside its window
            keys = [(int(ev[j]), int(j)) for j in seg]
            assert keys == sorted(keys)
    # turn-aligned evictions are already in that order
    w = W.make_workload(2, shrink=32, batch=1)
    assert np.array_equal(O.reorder_keys(w.trace(0)[4096 // 32:], 4096), np.arange(w.total_tokens - 4096 // 32))


def test_general_mask_is_invariant_under_key_permutation():
    T, Hq, Hkv, d = 300, 4, 2, 16
    r = np.random.default_rng(2)
    q, k, v, do = (r.standard_normal(s) for s in ((T, Hq, d), (T, Hkv, d), (T, Hkv, d), (T, Hq, d)))
    ev = _rand_trace(T, 3, maxlife=80)
    o, l = O.dense_fwd(q, k, v, ev, 0.3)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, 0.3)
    for perm in (O.reorder_keys(ev, 64), r.permutation(T)):
        o2, l2 = O.dense_fwd(q, k[perm], v[perm], ev[perm], 0.3, key_first=perm)
        dq2, dk2, dv2 = O.dense_bwd(q, k[perm], v[perm], do, ev[perm], 0.3, key_first=perm)
        assert np.allclose(o, o2, rtol=1e-11, atol=1e-12) and np.allclose(l, l2, rtol=1e-11, atol=1e-12)
        assert np.allclose(dq, dq2, rtol=1e-10, atol=1e-11)
        assert np.allclose(dk[perm], dk2, rtol=1e-10, atol=1e-11) and np.allclose(dv[perm], dv2, rtol=1e-10, atol=1e-11)
    # key_first = arange is the plain form, bit for bit
    o3, l3 = O.dense_fwd(q, k, v, ev, 0.3, key_first=np.arange(T))
    assert np.array_equal(o, o3) and np.array_equal(l, l3)


def test_general_mask_by_brute_force_loops_and_rows_without_keys():
    T, d = 40, 4
    r = np.random.default_rng(4)
    q, k, v = (r.standard_normal((T, 1, d)) for _ in range(3))
    first = r.integers(0, T + 5, size=T)
    evict = first + r.integers(-3, 15, size=T)                   # some slots are visible to nobody
    o, l = O.dense_fwd(q, k, v, evict, 0.5, key_first=first)
    for i in range(T):
        js = [j for j in range(T) if first[j] <= i < evict[j]]
        if not js:
            assert np.all(o[i] == 0) and l[0, i] == -np.inf
            continue
        x = np.array([0.5 * float(q[i, 0] @ k[j, 0]) for j in js])
        p = np.exp(x - x.max())
        p /= p.sum()
        assert np.allclose(o[i, 0], sum(pj * v[j, 0] for pj, j in zip(p, js)), atol=1e-12)
        assert abs(l[0, i] - (x.max() + np.log(np.exp(x - x.max()).sum()))) < 1e-12


def test_tile_rule_equals_or_is_safer_than_brute_force_on_key_slots():
    # plain keys: rule == brute force (pinned elsewhere).  General slots: the rule may call a tile PARTIAL that brute force
    # finds EMPTY or FULL (lifetimes inside a block need not overlap), never the other way round.
    for seed in range(4):
        T = 700
        ev = _rand_trace(T, 10 + seed, maxlife=300)
        perm = O.reorder_keys(ev, 256)
        rule = O.tile_classes_rule(ev[perm], key_first=perm)
        brute = O.tile_classes_brute(ev[perm], key_first=perm)
        assert ((rule == brute) | (rule == O.PARTIAL)).all()
        assert (brute[rule == O.EMPTY] == O.EMPTY).all() and (brute[rule == O.FULL] == O.FULL).all()
    assert np.array_equal(O.tile_classes_rule(ev, key_first=np.arange(T)), O.tile_classes_rule(ev))
    # and the order does what it is for: on the token-level pattern (alternate keys short-lived) far fewer tiles are
    # visited and most of those are FULL, where in the original order nearly all were PARTIAL
    # (lengths and lifetimes shrunk 8x, tiles still 128 wide, so the effect is weaker than at full size, where the
    # visited tiles drop 1.67x and 91 % of them are FULL)
    w = W.make_workload(4, shrink=8)
    ev = w.trace(0)
    plain = O.tile_classes_rule(ev)
    perm = O.reorder_keys(ev, 4096 // 8)
    rule = O.tile_classes_rule(ev[perm], key_first=perm)
    assert (plain == O.PARTIAL).sum() > 0.9 * (plain != O.EMPTY).sum()
    assert (rule != O.EMPTY).sum() * 1.3 < (plain != O.EMPTY).sum()
    assert (rule == O.FULL).sum() > 0.6 * (rule != O.EMPTY).sum()


def test_student_part_plus_evicted_part_is_full_causal_attention():
    # keys visible under the eviction mask and keys already evicted partition the causal set; merging the two partial
    # results reproduces the teacher of the self-distillation objective (App. D.3)
    w = W.make_workload(2, seed=5, shrink=64, Hq=4, Hkv=2, batch=1)
    q, k, v, _ = (_f64(t) for t in W.make_tensors(w, 5))
    ev = w.trace(0).astype(np.int64)
    T = ev.shape[0]
    os_, ls_ = O.dense_fwd(q, k, v, ev, w.scale)
    oc, lc = O.dense_fwd(q, k, v, np.full(T, O.INF), w.scale, key_first=ev)      # visible from its eviction on
    ot, lt = O.merge_partial(os_, ls_, oc, lc)
    rt, rl = O.dense_fwd(q, k, v, np.full(T, O.INF), w.scale)
    assert np.allclose(ot, rt, rtol=1e-11, atol=1e-12) and np.allclose(lt, rl, rtol=1e-11, atol=1e-12)
    assert np.isinf(lc[:, :10]).all()                             # early rows: nothing has been evicted yet


# ---- GPU ------------------------------------------------------------------------------------------------
def _close(name, got, ref, sigma=None):
    got = _f64(got) if isinstance(got, torch.Tensor) else got
    assert np.isfinite(got).all(), name
    bound = MAX_ABS if sigma is None else np.maximum(MAX_ABS, 6.0 * sigma)
    err = np.abs(got - ref)
    assert (err <= bound).all(), f"{name}: max-abs {err.max():.4f}"
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= REL_L2, name


@pytest.mark.gpu
@pytest.mark.parametrize("kw,window", [
    (dict(cfg=4, shrink=32, Hq=8, Hkv=1), 1024),
    (dict(cfg=4, shrink=32, Hq=4, Hkv=2, variant="b"), 4096),
    (dict(cfg=3, shrink=32, Hq=4, Hkv=2, batch=4), 512),            # ragged traces, turn-aligned: order barely changes
    (dict(cfg=6, shrink=32, Hq=4, Hkv=1, batch=2), 2048),
    (dict(cfg=0), 100),                                             # a window that is no multiple of anything
])
def test_reordered_keys_match_the_oracle_in_original_order(kw, window):
    from paper_2609_35750_b200 import binding as B
    from tests.guard import Fenced
    w = W.make_workload(seed=2, **kw)
    q, k, v, do = W.make_tensors(w, 2)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
    ev = torch.from_numpy(w.evict_at).cuda()
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    Tt = w.total_tokens
    perm, kf, ke = B.kvs_reorder_keys(ev, cu, w.max_seqlen, window)
    # bit-exact against the oracle's order
    ref_perm = np.concatenate([w.cu_seqlens[b] + O.reorder_keys(w.trace(b), window) for b in range(w.batch)])
    assert np.array_equal(perm.cpu().numpy(), ref_perm)
    loc = ref_perm - np.repeat(w.cu_seqlens[:-1], np.diff(w.cu_seqlens))
    assert np.array_equal(kf.cpu().numpy(), loc) and np.array_equal(ke.cpu().numpy(), w.evict_at[ref_perm])
    kp, vp = B.kvs_permute_rows(kd, perm), B.kvs_permute_rows(vd, perm)
    assert torch.equal(kp, kd[perm.long()]) and torch.equal(vp, vd[perm.long()])
    meta = B.kvs_mask_meta_keys(kf, ke, cu, w.max_seqlen)
    cls, kmin, kmax = B.kvs_mask_meta_export(meta, w.cu_seqlens, Tt, w.max_seqlen)
    ref_cls = []
    for b in range(w.batch):
        a, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        ref_cls.append(O.tile_classes_rule(w.evict_at[ref_perm[a:e]], key_first=loc[a:e]).ravel())
    assert np.array_equal(cls, np.concatenate(ref_cls))
    guard = 130 * w.Hq * w.d * 4
    fo, fl = Fenced(q.shape, torch.bfloat16, guard), Fenced((w.Hq, Tt), torch.float32, guard)
    fdq, fdk, fdv = Fenced(q.shape, torch.float32, guard), Fenced(k.shape, torch.float32, guard), Fenced(k.shape, torch.float32, guard)
    B.kvs_attn_fwd(qd, kp, vp, meta, w.batch, w.max_seqlen, w.softmax_scale, out=fo.t, lse=fl.t)
    B.kvs_attn_bwd(dod, qd, kp, vp, fo.t, fl.t, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32, dq=fdq.t, dk=fdk.t, dv=fdv.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(meta) == B.KVS_OK
    for name, f in (("out", fo), ("lse", fl), ("dq", fdq), ("dk", fdk), ("dv", fdv)):
        f.check(name)
    dk = B.kvs_permute_rows(fdk.t, perm, inverse=True)
    dv = B.kvs_permute_rows(fdv.t, perm, inverse=True)
    qn, kn, vn, don = (_f64(t) for t in (q, k, v, do))
    ro, rl = O.varlen_fwd(qn, kn, vn, w.evict_at, w.cu_seqlens, w.scale)
    rdq, rdk, rdv = O.varlen_bwd(qn, kn, vn, don, w.evict_at, w.cu_seqlens, w.scale)
    sg = O.varlen_rounding_sigma(qn, kn, vn, don, w.evict_at, w.cu_seqlens, w.scale)
    _close("out", fo.t, ro)
    _close("lse", fl.t, rl)
    _close("dq", fdq.t, rdq, sg["dq"])
    _close("dk", dk, rdk, sg["dk"])
    _close("dv", dv, rdv, sg["dv"])
    # bf16 gradients through the same path
    dq2, dk2, dv2 = B.kvs_attn_bwd(dod, qd, kp, vp, fo.t, fl.t, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_BF16)
    assert np.linalg.norm(_f64(B.kvs_permute_rows(dk2, perm, inverse=True)) - rdk) / np.linalg.norm(rdk) <= REL_L2
    assert np.linalg.norm(_f64(dq2) - rdq) / np.linalg.norm(rdq) <= REL_L2


@pytest.mark.gpu
def test_complement_slots_and_slots_nobody_sees():
    # "visible from its eviction on": never-evicted keys are visible to nobody, early rows see no key at all, whole
    # key blocks have no query block (their gradients must come back as zeros, not as whatever the buffer held)
    from paper_2609_35750_b200 import binding as B
    from tests.guard import Fenced
    w = W.make_workload(2, seed=3, shrink=32, Hq=4, Hkv=2, batch=2)
    q, k, v, do = W.make_tensors(w, 3)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
    Tt = w.total_tokens
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    kf = torch.from_numpy(w.evict_at).cuda()
    ke = torch.full((Tt,), int(W.INF), dtype=torch.int32, device="cuda")
    meta = B.kvs_mask_meta_keys(kf, ke, cu, w.max_seqlen)
    guard = 130 * w.Hq * w.d * 4
    fo, fl = Fenced(q.shape, torch.bfloat16, guard), Fenced((w.Hq, Tt), torch.float32, guard)
    fdq, fdk, fdv = Fenced(q.shape, torch.float32, guard), Fenced(k.shape, torch.float32, guard), Fenced(k.shape, torch.float32, guard)
    B.kvs_attn_fwd(qd, kd, vd, meta, w.batch, w.max_seqlen, w.softmax_scale, out=fo.t, lse=fl.t)
    B.kvs_attn_bwd(dod, qd, kd, vd, fo.t, fl.t, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32, dq=fdq.t, dk=fdk.t, dv=fdv.t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(meta) == B.KVS_OK
    for name, f in (("out", fo), ("dq", fdq), ("dk", fdk), ("dv", fdv)):
        f.check(name)
    assert fl.guards_intact()
    qn, kn, vn, don = (_f64(t) for t in (q, k, v, do))
    for b in range(w.batch):
        a, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        T = e - a
        ro, rl = O.dense_fwd(qn[a:e], kn[a:e], vn[a:e], np.full(T, O.INF), w.scale, key_first=w.evict_at[a:e])
        rdq, rdk, rdv = O.dense_bwd(qn[a:e], kn[a:e], vn[a:e], don[a:e], np.full(T, O.INF), w.scale, key_first=w.evict_at[a:e])
        lse = _f64(fl.t)[:, a:e]
        dead = np.isinf(rl)
        assert dead.any() and np.array_equal(np.isinf(lse) & (lse < 0), dead)
        assert np.abs(lse[~dead] - rl[~dead]).max() <= MAX_ABS
        assert np.abs(_f64(fo.t)[a:e] - ro).max() <= MAX_ABS
        for name, got, ref in (("dq", fdq.t, rdq), ("dk", fdk.t, rdk), ("dv", fdv.t, rdv)):
            g = _f64(got)[a:e]
            assert np.abs(g - ref).max() <= 3e-2 and np.linalg.norm(g - ref) / np.linalg.norm(ref) <= REL_L2, name
        assert (rdk == 0).all(axis=(1, 2)).sum() > 128                 # whole key blocks that nobody sees exist in this case
