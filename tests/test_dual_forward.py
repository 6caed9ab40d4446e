"""Student + teacher forward (self-distillation, App. D.3 "Training Objectives").

CPU: the oracle's dual forward is pinned to things other than itself: the teacher is plain causal
attention (torch's fp64 scaled_dot_product_attention), the student is the masked attention already
pinned elsewhere, and where nothing is ever evicted the two coincide (the identity the CUDA path rests on,
student part + evicted part = full causal attention, is pinned in tests/test_key_slots.py).  GPU:
kvs_attn_fwd_dual against the oracle on shrunk configurations, ragged batches and the numerically awkward
cases, and against the two plain forwards it replaces."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

MAX_ABS, REL_L2 = 2e-2, 5e-3


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def test_oracle_teacher_is_plain_causal_sdpa_and_student_is_the_masked_forward():
    w = W.make_workload(2, seed=2, shrink=64, Hq=4, Hkv=2, batch=1)
    q, k, v, _ = (_f64(t) for t in W.make_tensors(w, 2))
    ev = w.trace(0)
    os_, ls_, ot_, lt_ = O.dual_fwd(q, k, v, ev, w.scale)
    G = w.Hq // w.Hkv
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(np.repeat(k, G, axis=1)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(np.repeat(v, G, axis=1)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=w.scale)[0].permute(1, 0, 2).numpy()
    assert np.abs(ot_ - ref).max() < 1e-12
    so, sl = O.dense_fwd(q, k, v, ev, w.scale)
    assert np.array_equal(os_, so) and np.array_equal(ls_, sl)
    # the teacher sees a superset of the student's keys: its normaliser is never smaller
    assert (lt_ >= ls_ - 1e-12).all() and (lt_ > ls_ + 1e-6).any()
    # nothing evicted: the two streams coincide
    a, b, c, d = O.dual_fwd(q, k, v, np.full(ev.shape[0], O.INF), w.scale)
    assert np.array_equal(a, c) and np.array_equal(b, d)


def _close(name, got, ref, sigma=None):
    """sigma: for the teacher's output, which is a weighted sum of two partial results that were each rounded to bf16
    before the merge and is rounded once more after it.  The oracle's rounding model gives the standard deviation of a
    once-rounded output (probability rounding + half an ulp of its own); an element's bound is 2e-2, or six of those
    deviations plus half a bf16 ulp for the additional rounding where that is larger."""
    got = _f64(got)
    assert np.isfinite(got).all(), name
    err = np.abs(got - ref)
    bound = np.full(ref.shape, MAX_ABS)
    if sigma is not None:
        bound = np.maximum(bound, 6.0 * sigma + 2.0 ** (np.floor(np.log2(np.maximum(np.abs(ref), 1e-30))) - 8))
    assert (err <= bound).all(), f"{name}: max-abs {err.max():.4f}"
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= REL_L2, f"{name}: rel-L2 {rel:.3e}"


def _run_dual(w, tensors):
    from paper_2609_35750_b200 import binding as B
    from tests.guard import Fenced
    q, k, v, _ = tensors
    qd, kd, vd = (t.cuda() for t in (q, k, v))
    ev, cu = torch.from_numpy(w.evict_at).cuda(), torch.from_numpy(w.cu_seqlens).cuda()
    meta = B.kvs_mask_meta(ev, cu, w.max_seqlen)
    meta_e = B.kvs_mask_meta_evicted(ev, cu, w.max_seqlen)
    guard = 130 * w.Hq * w.d * 2
    f = [Fenced(q.shape, torch.bfloat16, guard), Fenced((w.Hq, w.total_tokens), torch.float32, guard),
         Fenced(q.shape, torch.bfloat16, guard), Fenced((w.Hq, w.total_tokens), torch.float32, guard)]
    B.kvs_attn_fwd_dual(qd, kd, vd, meta, meta_e, w.batch, w.max_seqlen, w.softmax_scale,
                        out_student=f[0].t, lse_student=f[1].t, out_teacher=f[2].t, lse_teacher=f[3].t)
    torch.cuda.synchronize()
    assert B.kvs_device_status(meta) == B.KVS_OK and B.kvs_device_status(meta_e) == B.KVS_OK
    for name, x in zip(("out_student", "lse_student", "out_teacher", "lse_teacher"), f):
        x.check(name)
    return meta, qd, kd, vd, [x.t for x in f]


def _check_dual(w, tensors, exact_vs_single=True):
    from paper_2609_35750_b200 import binding as B
    meta, qd, kd, vd, got = _run_dual(w, tensors)
    q, k, v, _ = (_f64(t) for t in tensors)
    ref = O.varlen_dual_fwd(q, k, v, w.evict_at, w.cu_seqlens, w.scale)
    inf = np.full(w.total_tokens, O.INF, dtype=np.int64)
    sg_t = O.varlen_rounding_sigma(q, k, v, np.zeros_like(q), inf, w.cu_seqlens, w.scale)["out"]
    for name, g, r in zip(("out_student", "lse_student", "out_teacher", "lse_teacher"), got, ref):
        _close(name, g, r, sigma=(sg_t if name == "out_teacher" else None))
    # against the two kernels it replaces: same masks, same arithmetic up to the order of the row sums
    so, sl = B.kvs_attn_fwd(qd, kd, vd, meta, w.batch, w.max_seqlen, w.softmax_scale)
    inf = torch.full((w.total_tokens,), int(W.INF), dtype=torch.int32, device="cuda")
    meta_c = B.kvs_mask_meta(inf, torch.from_numpy(w.cu_seqlens).cuda(), w.max_seqlen)
    to, tl = B.kvs_attn_fwd(qd, kd, vd, meta_c, w.batch, w.max_seqlen, w.softmax_scale)
    assert (got[0].float() - so.float()).abs().max().item() <= 2e-2 and (got[1] - sl).abs().max().item() <= 1e-3
    assert (got[2].float() - to.float()).abs().max().item() <= 2 * 2.0 ** -7 * max(1.0, to.float().abs().max().item())
    assert (got[3] - tl).abs().max().item() <= 1e-3


@pytest.mark.gpu
@pytest.mark.parametrize("kw", [
    dict(cfg=0),
    dict(cfg=1, shrink=16, Hq=7, Hkv=1, batch=2),
    dict(cfg=2, shrink=16, Hq=8, Hkv=2, batch=2),
    dict(cfg=3, shrink=32, Hq=4, Hkv=2, batch=4),          # ragged
    dict(cfg=4, shrink=32, Hq=8, Hkv=1),                   # token-level: almost every tile PARTIAL
    dict(cfg=4, shrink=32, Hq=2, Hkv=2, variant="b"),      # many tiles EMPTY for the student
    dict(cfg=6, shrink=32, Hq=4, Hkv=1, batch=1),
])
def test_dual_forward_matches_oracle_on_shrunk_configs(kw):
    w = W.make_workload(seed=1, **kw)
    _check_dual(w, W.make_tensors(w, 1))


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_dual_forward_ragged_lengths(d):
    rng = np.random.default_rng(7)
    lens = [1, 2, 127, 128, 129, 255, 257, 1, 640, 3]
    evs = []
    for T in lens:
        ev = np.full(T, int(W.INF), dtype=np.int64)
        sel = rng.random(T) < 0.6
        ev[sel] = (np.arange(T) + rng.integers(1, 301, size=T))[sel]
        evs.append(ev.astype(np.int32))
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    w = W.Workload("custom", cu, np.concatenate(evs), 4, 2, d)
    _check_dual(w, W.make_tensors(w, 3))


@pytest.mark.gpu
def test_dual_forward_when_the_teacher_sees_a_huge_logit_the_student_does_not():
    # keys 0..199 leave at 200; one of them has an enormous logit.  For rows >= 200 the teacher's reference
    # maximum is far above anything the student sees: the student's probabilities must not be lost to the
    # teacher's scale (the two parts are computed with their own maxima and merged through their lse).
    T = 512
    ev = np.full(T, int(W.INF), dtype=np.int64)
    ev[:200] = 200
    w = W.Workload("custom", np.array([0, T], dtype=np.int32), ev.astype(np.int32), 2, 1, 128, softmax_scale=1.0)
    q, k, v, do = W.make_tensors(w, 7)
    k = k.clone()
    k[50] = 40.0
    _check_dual(w, (q, k, v, do))


@pytest.mark.gpu
def test_dual_forward_growing_logits():
    T = 1024
    w = W.Workload("custom", np.array([0, T], dtype=np.int32), (np.arange(T) + 300).astype(np.int32), 2, 2, 64, softmax_scale=1.0)
    q, k, v, do = W.make_tensors(w, 8)
    q = torch.zeros_like(q)
    k = torch.zeros_like(k)
    q[:, :, 0] = 1.0
    k[:, :, 0] = (torch.arange(T, dtype=torch.float32) * 0.08).to(torch.bfloat16)[:, None]     # the maximum moves in every block
    _check_dual(w, (q, k, v, do))
