"""Rotary embedding of q, k on one continuous trace, and the packed QKV entry points.

CPU pins of the oracle's rotation (against things other than itself): positions 0 leave the input unchanged; a
two-dimensional head is a plane rotation by pos radians; norms are preserved; the score of rotated q_i, k_j depends on
i - j only, so shifting every position by a constant leaves the attention output unchanged (a wrong sign or a wrong
pairing of components breaks this); inverse undoes forward and is its transpose; gradients through rotation + attention
against central differences.  GPU: kvs_rope_qk against the oracle (one rounding), the whole rotated path forward and
backward, and the packed entry points against the separate-tensor ones bit for bit."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

MAX_ABS, REL_L2 = 2e-2, 5e-3


def _f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


# ---- CPU ------------------------------------------------------------------------------------------------
def test_rotation_special_cases():
    r = np.random.default_rng(0)
    x = r.standard_normal((5, 3, 8))
    assert np.array_equal(O.rope_rotate(x, np.zeros(5, dtype=int)), x)
    # d = 2: one plane, inverse frequency 1: a rotation by pos radians
    e = np.array([[[1.0, 0.0]], [[1.0, 0.0]], [[0.0, 1.0]]])
    y = O.rope_rotate(e, np.array([0, 1, 2]))
    assert np.allclose(y[0, 0], [1, 0]) and np.allclose(y[1, 0], [np.cos(1), np.sin(1)]) and np.allclose(y[2, 0], [-np.sin(2), np.cos(2)])
    # d = 4: component c pairs with c + 2, the second pair turns base^(-1/2) times as fast
    z = O.rope_rotate(np.array([[[1.0, 1.0, 0.0, 0.0]]]), np.array([3]), theta_base=100.0)
    assert np.allclose(z[0, 0], [np.cos(3), np.cos(0.3), np.sin(3), np.sin(0.3)])
    pos = r.integers(0, 100000, size=5)
    y = O.rope_rotate(x, pos)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-12)
    assert np.allclose(O.rope_rotate(y, pos, inverse=True), x, atol=1e-10)
    # inverse is the transpose: <R x, g> = <x, R^T g>
    g = r.standard_normal(x.shape)
    assert abs((y * g).sum() - (x * O.rope_rotate(g, pos, inverse=True)).sum()) < 1e-9


def test_scores_depend_on_position_differences_only():
    T, Hq, Hkv, d = 60, 2, 1, 16
    r = np.random.default_rng(1)
    q, k, v = r.standard_normal((T, Hq, d)), r.standard_normal((T, Hkv, d)), r.standard_normal((T, Hkv, d))
    ev = np.where(r.random(T) < 0.5, np.arange(T) + r.integers(1, 20, size=T), O.INF)
    pos = np.arange(T)
    a, la = O.dense_fwd(O.rope_rotate(q, pos), O.rope_rotate(k, pos), v, ev, 0.25)
    b, lb = O.dense_fwd(O.rope_rotate(q, pos + 977), O.rope_rotate(k, pos + 977), v, ev, 0.25)
    assert np.allclose(a, b, atol=1e-9) and np.allclose(la, lb, atol=1e-9)
    c, _ = O.dense_fwd(q, k, v, ev, 0.25)
    assert np.abs(a - c).max() > 1e-2                     # and the rotation does change the result
    assert np.array_equal(O.trace_positions([0, 3, 3, 5]), [0, 1, 2, 0, 1])


def test_gradients_through_rotation_by_central_differences():
    T, d = 12, 4
    r = np.random.default_rng(2)
    q, k, v, do = (r.standard_normal((T, 1, d)) for _ in range(4))
    ev = np.where(r.random(T) < 0.5, np.arange(T) + r.integers(1, 6, size=T), O.INF)
    pos = np.arange(T) * 37

    def f(qq, kk):
        o, _ = O.dense_fwd(O.rope_rotate(qq, pos), O.rope_rotate(kk, pos), v, ev, 0.5)
        return (o * do).sum()

    dq_r, dk_r, _ = O.dense_bwd(O.rope_rotate(q, pos), O.rope_rotate(k, pos), v, do, ev, 0.5)
    dq, dk = O.rope_rotate(dq_r, pos, inverse=True), O.rope_rotate(dk_r, pos, inverse=True)
    h = 1e-6
    for (t, c) in [(0, 0), (5, 1), (11, 3), (7, 2)]:
        e = np.zeros_like(q)
        e[t, 0, c] = h
        assert abs((f(q + e, k) - f(q - e, k)) / (2 * h) - dq[t, 0, c]) < 1e-6
        assert abs((f(q, k + e) - f(q, k - e)) / (2 * h) - dk[t, 0, c]) < 1e-6


# ---- GPU ------------------------------------------------------------------------------------------------
@pytest.mark.gpu
@pytest.mark.parametrize("d,dtype", [(64, torch.bfloat16), (128, torch.bfloat16), (128, torch.float32)])
def test_rope_kernel_matches_oracle_to_one_rounding(d, dtype):
    from paper_2609_35750_b200 import binding as B
    lens = [300, 1, 4000, 77]
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    T = int(cu[-1])
    g = torch.Generator().manual_seed(3)
    q = torch.randn((T, 6, d), generator=g).to(dtype)
    k = torch.randn((T, 2, d), generator=g).to(dtype)
    cud = torch.from_numpy(cu).cuda()
    qr, kr = B.kvs_rope_qk(q.cuda(), k.cuda(), cu_seqlens=cud, theta_base=1e6)
    pos = O.trace_positions(cu)
    rq, rk = O.rope_rotate(_f64(q), pos, 1e6), O.rope_rotate(_f64(k), pos, 1e6)
    # bf16: one rounding of the result; fp32: cos, sin and the two products are each rounded, so the error scales with
    # the size of the inputs of the pair, not of the (possibly cancelling) result
    tol = lambda ref: 2.0 ** -8 * np.maximum(np.abs(ref), 1e-3) if dtype == torch.bfloat16 else 1e-6 * (1.0 + np.abs(ref))
    assert (np.abs(_f64(qr) - rq) <= tol(rq)).all() and (np.abs(_f64(kr) - rk) <= tol(rk)).all()
    # explicit positions far out (angles of 1e5 rad), the transposed rotation, in place, k alone
    far = torch.from_numpy((pos + 100000).astype(np.int32)).cuda()
    kf = k.cuda().clone()
    B.kvs_rope_qk(None, kf, positions=far, theta_base=1e4, k_out=kf)
    rkf = O.rope_rotate(_f64(k), pos + 100000, 1e4)
    assert (np.abs(_f64(kf) - rkf) <= tol(rkf)).all()
    _, back = B.kvs_rope_qk(None, kr, cu_seqlens=cud, theta_base=1e6, inverse=True)
    assert np.abs(_f64(back) - _f64(k)).max() <= (2.0 ** -6 if dtype == torch.bfloat16 else 1e-5)


@pytest.mark.gpu
@pytest.mark.parametrize("kw", [dict(cfg=2, shrink=32, Hq=8, Hkv=2, batch=2), dict(cfg=3, shrink=32, Hq=4, Hkv=1, batch=3), dict(cfg=0)])
def test_rotated_path_forward_and_backward(kw):
    # rotate q, k (positions kept across evictions), attend, and take the gradients back through the rotation
    from paper_2609_35750_b200 import binding as B
    w = W.make_workload(seed=6, **kw)
    q, k, v, do = W.make_tensors(w, 6)
    qd, kd, vd, dod = (t.cuda() for t in (q, k, v, do))
    ev, cu = torch.from_numpy(w.evict_at).cuda(), torch.from_numpy(w.cu_seqlens).cuda()
    qr, kr = B.kvs_rope_qk(qd, kd, cu_seqlens=cu, theta_base=1e6)
    meta = B.kvs_mask_meta(ev, cu, w.max_seqlen)
    out, lse = B.kvs_attn_fwd(qr, kr, vd, meta, w.batch, w.max_seqlen, w.softmax_scale)
    dq, dk, dv = B.kvs_attn_bwd(dod, qr, kr, vd, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, B.GRAD_FP32)
    B.kvs_rope_qk(dq, dk, cu_seqlens=cu, theta_base=1e6, inverse=True, q_out=dq, k_out=dk)
    assert B.kvs_device_status(meta) == B.KVS_OK
    pos = O.trace_positions(w.cu_seqlens)
    qn, kn, vn, don = (_f64(t) for t in (q, k, v, do))
    rq, rk = O.rope_rotate(qn, pos, 1e6), O.rope_rotate(kn, pos, 1e6)
    ro, rl = O.varlen_fwd(rq, rk, vn, w.evict_at, w.cu_seqlens, w.scale)
    rdq, rdk, rdv = O.varlen_bwd(rq, rk, vn, don, w.evict_at, w.cu_seqlens, w.scale)
    rdq, rdk = O.rope_rotate(rdq, pos, 1e6, inverse=True), O.rope_rotate(rdk, pos, 1e6, inverse=True)
    # the rotated q, k are rounded to bf16 once more before the products: the logits move by about 1.6e-3, which the
    # relative bound has room for; the absolute bound of the gradients follows the rounding model of the unrotated path
    sg = O.varlen_rounding_sigma(rq, rk, vn, don, w.evict_at, w.cu_seqlens, w.scale)
    for name, got, ref in (("out", out, ro), ("lse", lse, rl), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        g = _f64(got)
        assert np.isfinite(g).all(), name
        bound = np.maximum(MAX_ABS, 8.0 * sg[name]) if name in ("dk", "dv") else MAX_ABS
        assert (np.abs(g - ref) <= bound).all(), (name, float(np.abs(g - ref).max()))
        assert np.linalg.norm(g - ref) / np.linalg.norm(ref) <= REL_L2, (name, float(np.linalg.norm(g - ref) / np.linalg.norm(ref)))


@pytest.mark.gpu
@pytest.mark.parametrize("grad", ["bf16", "fp32"])
@pytest.mark.parametrize("kw", [dict(cfg=2, shrink=32, Hq=8, Hkv=2, batch=2), dict(cfg=3, shrink=32, Hq=6, Hkv=2, batch=3), dict(cfg=0)])
def test_packed_entry_points_equal_the_separate_ones(kw, grad):
    from paper_2609_35750_b200 import binding as B
    from tests.guard import Fenced
    w = W.make_workload(seed=7, **kw)
    q, k, v, do = (t.cuda() for t in W.make_tensors(w, 7))
    gd = B.GRAD_BF16 if grad == "bf16" else B.GRAD_FP32
    gdt = torch.bfloat16 if grad == "bf16" else torch.float32
    meta = B.kvs_mask_meta(torch.from_numpy(w.evict_at).cuda(), torch.from_numpy(w.cu_seqlens).cuda(), w.max_seqlen)
    out, lse = B.kvs_attn_fwd(q, k, v, meta, w.batch, w.max_seqlen, w.softmax_scale)
    dq, dk, dv = B.kvs_attn_bwd(do, q, k, v, out, lse, meta, w.batch, w.max_seqlen, w.softmax_scale, gd)
    H = w.Hq + 2 * w.Hkv
    guard = 130 * H * w.d * 4
    fqkv = Fenced((w.total_tokens, H, w.d), torch.bfloat16, guard, fill_from=torch.cat([q, k, v], dim=1))
    fd = Fenced((w.total_tokens, H, w.d), gdt, guard)
    out2, lse2 = B.kvs_attn_fwd_packed(fqkv.t, meta, w.batch, w.max_seqlen, w.Hq, w.Hkv, w.softmax_scale)
    B.kvs_attn_bwd_packed(do, fqkv.t, out2, lse2, meta, w.batch, w.max_seqlen, w.Hq, w.Hkv, w.softmax_scale, gd, dqkv=fd.t)
    torch.cuda.synchronize()
    fqkv.check("qkv")
    fd.check("dqkv")
    assert torch.equal(out, out2) and torch.equal(lse, lse2)
    assert torch.equal(fd.t[:, w.Hq:w.Hq + w.Hkv], dk) and torch.equal(fd.t[:, w.Hq + w.Hkv:], dv)       # written once, fixed order
    assert torch.allclose(fd.t[:, :w.Hq].float(), dq.float(), atol=2e-2 if grad == "bf16" else 1e-4, rtol=2e-2 if grad == "bf16" else 1e-4)
