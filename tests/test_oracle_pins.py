"""Pins for the CPU oracle against things other than itself (CPU only).

Each test is chosen so that a plausible slip in the oracle (a dropped term, a
wrong sign, a transposed operand, an off-by-one in the mask) fails it.
"""
import os

import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _rand(T, Hq, Hkv, d, seed):
    r = np.random.default_rng(seed)
    return (r.standard_normal((T, Hq, d)), r.standard_normal((T, Hkv, d)),
            r.standard_normal((T, Hkv, d)), r.standard_normal((T, Hq, d)))


def _random_evict_at(T, seed, frac=0.6, maxlife=None):
    r = np.random.default_rng(seed)
    ev = np.full(T, O.INF, dtype=np.int64)
    sel = r.random(T) < frac
    life = r.integers(1, (maxlife or T) + 1, size=T)
    ev[sel] = (np.arange(T) + life)[sel]
    return ev.astype(np.int32)


# ---- P1: dense mask == physical eviction replay -------------------------------------------
@pytest.mark.parametrize("removal", ["ordered", "swap"])
def test_dense_equals_replay_random_masks(removal):
    for seed, (T, Hq, Hkv, d) in enumerate([(37, 4, 2, 8), (64, 3, 3, 16), (50, 6, 2, 4)]):
        q, k, v, do = _rand(T, Hq, Hkv, d, seed)
        ev = _random_evict_at(T, 100 + seed, maxlife=20)
        s = 0.37
        o1, l1 = O.dense_fwd(q, k, v, ev, s)
        dq1, dk1, dv1 = O.dense_bwd(q, k, v, do, ev, s)
        o2, l2, dq2, dk2, dv2, sizes = O.replay_fwd_bwd(q, k, v, do, ev, s, removal=removal)
        for a, b in [(o1, o2), (l1, l2), (dq1, dq2), (dk1, dk2), (dv1, dv2)]:
            assert np.allclose(a, b, rtol=1e-11, atol=1e-12)
        assert np.array_equal(sizes, O.live_counts(ev))


def test_dense_equals_replay_cfg0_and_shrunk_configs():
    cases = [W.make_workload(0, Hq=2, Hkv=1), W.make_workload(1, shrink=64, Hq=2, Hkv=1, batch=1),
             W.make_workload(2, shrink=64, Hq=2, Hkv=2, batch=1), W.make_workload(4, shrink=256, Hq=2, Hkv=1)]
    for w in cases:
        ev = w.trace(0)
        T = ev.shape[0]
        q, k, v, do = _rand(T, w.Hq, w.Hkv, 8, 5)
        o1, l1 = O.dense_fwd(q, k, v, ev, 0.3)
        g1 = O.dense_bwd(q, k, v, do, ev, 0.3)
        o2, l2, dq2, dk2, dv2, sizes = O.replay_fwd_bwd(q, k, v, do, ev, 0.3)
        assert np.allclose(o1, o2, rtol=1e-11, atol=1e-12) and np.allclose(l1, l2, rtol=1e-11, atol=1e-12)
        for a, b in zip(g1, (dq2, dk2, dv2)):
            assert np.allclose(a, b, rtol=1e-10, atol=1e-12)
        assert np.array_equal(sizes, O.live_counts(ev))


# ---- P2: no eviction == plain causal attention (library routine) --------------------------
def test_no_eviction_is_plain_causal_sdpa():
    T, Hq, Hkv, d = 96, 4, 2, 16
    q, k, v, do = _rand(T, Hq, Hkv, d, 7)
    ev = np.full(T, O.INF, dtype=np.int32)
    s = 1.0 / np.sqrt(d)
    o, lse = O.dense_fwd(q, k, v, ev, s)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, s)
    tq = torch.tensor(q).permute(1, 0, 2).clone().requires_grad_(True)          # [H,T,d]
    tk = torch.tensor(k).permute(1, 0, 2).clone().requires_grad_(True)
    tv = torch.tensor(v).permute(1, 0, 2).clone().requires_grad_(True)
    ke = tk.repeat_interleave(Hq // Hkv, dim=0)
    ve = tv.repeat_interleave(Hq // Hkv, dim=0)
    to = torch.nn.functional.scaled_dot_product_attention(tq[None], ke[None], ve[None], is_causal=True, scale=s)[0]
    to.backward(torch.tensor(do).permute(1, 0, 2))
    assert np.allclose(o, to.detach().permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)
    assert np.allclose(dq, tq.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dk, tk.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dv, tv.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_general_mask_matches_sdpa_with_boolean_mask_and_autograd():
    T, Hq, Hkv, d = 80, 2, 1, 8
    q, k, v, do = _rand(T, Hq, Hkv, d, 8)
    ev = _random_evict_at(T, 9, maxlife=30)
    # the boolean mask is retyped here on purpose, element by element
    M = torch.zeros(T, T, dtype=torch.bool)
    for i in range(T):
        for j in range(T):
            M[i, j] = (j <= i) and (i < int(ev[j]))
    o, lse = O.dense_fwd(q, k, v, ev, 0.25)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, 0.25)
    tq = torch.tensor(q).permute(1, 0, 2).clone().requires_grad_(True)
    tk = torch.tensor(k).permute(1, 0, 2).clone().requires_grad_(True)
    tv = torch.tensor(v).permute(1, 0, 2).clone().requires_grad_(True)
    to = torch.nn.functional.scaled_dot_product_attention(
        tq[None], tk.repeat_interleave(2, 0)[None], tv.repeat_interleave(2, 0)[None], attn_mask=M, scale=0.25)[0]
    to.backward(torch.tensor(do).permute(1, 0, 2))
    assert np.allclose(o, to.detach().permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)
    assert np.allclose(dq, tq.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dk, tk.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    assert np.allclose(dv, tv.grad.permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)
    # LSE against torch.logsumexp of the masked logits
    S = 0.25 * torch.einsum("hid,hjd->hij", tq.detach(), tk.detach().repeat_interleave(2, 0))
    S = S.masked_fill(~M[None], float("-inf"))
    assert np.allclose(lse, torch.logsumexp(S, dim=-1).numpy(), rtol=1e-12, atol=1e-12)


# ---- P3: softmax rows sum to one ----------------------------------------------------------
def test_rows_sum_to_one_and_constant_v():
    T, Hq, Hkv, d = 70, 2, 2, 8
    q, k, v, do = _rand(T, Hq, Hkv, d, 10)
    ev = _random_evict_at(T, 11, maxlife=25)
    v1 = np.ones_like(v)
    o, lse = O.dense_fwd(q, k, v1, ev, 0.5)
    assert np.allclose(o, 1.0, rtol=0, atol=1e-13)
    A = O.allowed(ev)
    for h in range(Hq):
        S = 0.5 * q[:, h] @ k[:, h].T
        P = np.where(A, np.exp(S - lse[h][:, None]), 0.0)
        assert np.allclose(P.sum(1), 1.0, atol=1e-12)


# ---- P4: finite differences ---------------------------------------------------------------
@pytest.mark.parametrize("G", [1, 2, 3])
def test_gradients_by_central_differences(G):
    T, Hkv, d = 14, 2, 5
    Hq = Hkv * G
    q, k, v, do = _rand(T, Hq, Hkv, d, 20 + G)
    ev = _random_evict_at(T, 30 + G, maxlife=6)
    s = 0.41

    def f(q_, k_, v_):
        o, _ = O.dense_fwd(q_, k_, v_, ev, s)
        return float((o * do).sum())

    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, s)
    h = 1e-5
    r = np.random.default_rng(0)
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(25):
            idx = tuple(int(r.integers(0, n)) for n in x.shape)
            xp, xm = x.copy(), x.copy()
            xp[idx] += h
            xm[idx] -= h
            args_p = {"q": (xp, k, v), "k": (q, xp, v), "v": (q, k, xp)}[name]
            args_m = {"q": (xm, k, v), "k": (q, xm, v), "v": (q, k, xm)}[name]
            fd = (f(*args_p) - f(*args_m)) / (2 * h)
            assert abs(fd - g[idx]) <= 1e-7 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


# ---- P5: zero-query closed form, printed values -------------------------------------------
def test_zero_query_live_counts_cfg0_golden():
    w = W.make_workload(0, Hq=1, Hkv=1)
    ev = w.trace(0)
    T = 1024
    r = np.random.default_rng(3)
    k = r.standard_normal((T, 1, 4))
    v = r.standard_normal((T, 1, 4))
    q = np.zeros((T, 1, 4))
    o, lse = O.dense_fwd(q, k, v, ev, 0.125)
    n = np.exp(lse[0])
    for i, ni in _read("cfg0_live_counts.txt"):
        assert abs(n[int(i)] - int(ni)) < 1e-9, (i, ni, n[int(i)])
    assert round(n.max()) == 384
    # o_i is then the mean of the visible v rows
    A = O.allowed(ev)
    for i in (0, 352, 575, 1023):
        assert np.allclose(o[i, 0], v[A[i], 0].mean(0), atol=1e-13)
    _, _, _, _, _, sizes = O.replay_fwd_bwd(q, k, v, None, ev, 0.125)
    assert np.array_equal(sizes, np.rint(n).astype(np.int64))


def test_cfg1_constant_memory_peak():
    g = {r[0]: [int(x) for x in r[1:]] for r in _read("cfg1_counts.txt")}
    ev = W.make_workload(1, batch=1).trace(0).astype(np.int64)
    # live count without the dense mask: +1 at j, -1 at evict_at[j]
    T = ev.shape[0]
    delta = np.zeros(T + 1, dtype=np.int64)
    np.add.at(delta, np.arange(T), 1)
    np.add.at(delta, np.minimum(ev, T), -1)
    live = np.cumsum(delta)[:T]
    assert live.max() == g["max_live"][0]
    # and the dense oracle agrees on a shrunk copy
    evs = W.make_workload(1, shrink=32, batch=1).trace(0)
    assert O.live_counts(evs).max() == g["max_live"][0] // 32


# ---- closed form: every key visible only to itself ----------------------------------------
def test_evict_after_one_step_closed_form():
    T, Hq, Hkv, d = 33, 4, 2, 6
    q, k, v, do = _rand(T, Hq, Hkv, d, 40)
    ev = (np.arange(T) + 1).astype(np.int32)
    s = 0.7
    o, lse = O.dense_fwd(q, k, v, ev, s)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, s)
    for h in range(Hq):
        assert np.allclose(o[:, h], v[:, h // 2], atol=1e-14)
        assert np.allclose(lse[h], s * (q[:, h] * k[:, h // 2]).sum(-1), atol=1e-13)
    assert np.allclose(dq, 0, atol=1e-13) and np.allclose(dk, 0, atol=1e-13)
    assert np.allclose(dv[:, 0], do[:, 0] + do[:, 1], atol=1e-13)
    assert np.allclose(dv[:, 1], do[:, 2] + do[:, 3], atol=1e-13)


# ---- retrieval-task mask: one early span evicted ------------------------------------------
def test_single_evicted_span_by_brute_force_loops():
    T, d = 20, 3
    q, k, v, do = _rand(T, 1, 1, d, 41)
    ev = np.full(T, O.INF, dtype=np.int32)
    ev[4:9] = 12                      # the assignment turn leaves before the answer tokens
    s = 0.9
    o, lse = O.dense_fwd(q, k, v, ev, s)
    for i in range(T):
        num = np.zeros(d)
        den = 0.0
        for j in range(T):
            if j <= i and not (4 <= j < 9 and i >= 12):
                wgt = np.exp(s * float(q[i, 0] @ k[j, 0]))
                num += wgt * v[j, 0]
                den += wgt
        assert np.allclose(o[i, 0], num / den, atol=1e-12)
        assert abs(lse[0, i] - np.log(den)) < 1e-12


# ---- P6 / P7: tile classes ----------------------------------------------------------------
def test_tile_rule_equals_brute_force():
    for seed in range(6):
        T = [1, 127, 128, 129, 300, 517][seed]
        ev = _random_evict_at(T, 50 + seed, maxlife=200)
        assert np.array_equal(O.tile_classes_rule(ev), O.tile_classes_brute(ev)), T
    for w in (W.make_workload(0), W.make_workload(2, shrink=16, batch=1), W.make_workload(3, shrink=8, batch=3),
              W.make_workload(4, shrink=32), W.make_workload(1, shrink=8, batch=1)):
        for b in range(w.batch):
            ev = w.trace(b)
            assert np.array_equal(O.tile_classes_rule(ev), O.tile_classes_brute(ev)), (w.name, b)
    # smaller tile edge exercises the same rule on tiny inputs
    ev = _random_evict_at(23, 77, maxlife=9)
    assert np.array_equal(O.tile_classes_rule(ev, block=4), O.tile_classes_brute(ev, block=4))


def test_tile_counts_cfg0_cfg1_golden():
    want0 = [int(x) for x in [r for r in _read("cfg0_evict_at.txt") if r[0] == "tiles"][0][1:]]
    c = O.tile_classes_rule(W.make_workload(0).trace(0))
    low = c[np.tril_indices(c.shape[0])]
    assert [int((low == O.FULL).sum()), int((low == O.PARTIAL).sum()), int((low == O.EMPTY).sum())] == want0
    assert int((np.diag(c) == O.PARTIAL).sum()) == 8 and np.all(c[np.triu_indices(8, 1)] == O.EMPTY)
    want1 = [int(x) for x in [r for r in _read("cfg1_counts.txt") if r[0] == "tiles"][0][1:]]
    c = O.tile_classes_rule(W.make_workload(1, batch=1).trace(0))
    low = c[np.tril_indices(c.shape[0])]
    assert [int((low == O.FULL).sum()), int((low == O.PARTIAL).sum()), int((low == O.EMPTY).sum())] == want1
    assert np.all(np.diag(c) == O.PARTIAL)


def test_tail_tile_one_by_one_is_full():
    ev = np.full(129, O.INF, dtype=np.int32)
    c = O.tile_classes_rule(ev)
    assert c[1, 1] == O.FULL and c[0, 0] == O.PARTIAL and c[1, 0] == O.FULL and c[0, 1] == O.EMPTY


# ---- row / key-block samplers agree with the dense route ----------------------------------
def test_row_and_block_samplers_match_dense():
    w = W.make_workload(2, shrink=64, Hq=4, Hkv=2, batch=1)
    ev = w.trace(0)
    T = ev.shape[0]
    q, k, v, do = _rand(T, 4, 2, 8, 60)
    s = 0.3
    o, lse = O.dense_fwd(q, k, v, ev, s)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, s)
    for i in (0, 1, 63, 64, 500, T - 1):
        for h in (0, 3):
            oi, li, dqi, *_ = O.row_fwd_bwd(q[i, h], k[:, h // 2], v[:, h // 2], do[i, h], ev, i, s)
            assert np.allclose(oi, o[i, h], atol=1e-12) and abs(li - lse[h, i]) < 1e-12
            assert np.allclose(dqi, dq[i, h], atol=1e-12)
    for (j0, j1, g) in ((0, 16, 0), (200, 264, 1), (T - 10, T, 0)):
        bk, bv = O.key_block_dkdv(q, k, v, do, ev, j0, j1, g, 2, s)
        assert np.allclose(bk, dk[j0:j1, g], atol=1e-11) and np.allclose(bv, dv[j0:j1, g], atol=1e-11)


# ---- P8 / P10: identities -----------------------------------------------------------------
def test_gradient_identities_and_gqa_duplication():
    T, Hq, Hkv, d = 60, 4, 2, 8
    q, k, v, do = _rand(T, Hq, Hkv, d, 70)
    ev = _random_evict_at(T, 71, maxlife=25)
    s = 0.33
    o, lse = O.dense_fwd(q, k, v, ev, s)
    dq, dk, dv = O.dense_bwd(q, k, v, do, ev, s)
    for g in range(Hkv):
        hs = slice(2 * g, 2 * g + 2)
        assert abs((q[:, hs] * dq[:, hs]).sum() - (k[:, g] * dk[:, g]).sum()) < 1e-10
        assert abs((v[:, g] * dv[:, g]).sum() - (do[:, hs] * o[:, hs]).sum()) < 1e-10
    # duplicating each KV head G times with Hkv = Hq gives the same output; shared-head grads are the sums
    k2, v2 = np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1)
    o2, _ = O.dense_fwd(q, k2, v2, ev, s)
    _, dk2, dv2 = O.dense_bwd(q, k2, v2, do, ev, s)
    assert np.allclose(o, o2, atol=1e-13)
    assert np.allclose(dk, dk2[:, 0::2] + dk2[:, 1::2], atol=1e-12)
    assert np.allclose(dv, dv2[:, 0::2] + dv2[:, 1::2], atol=1e-12)


def test_varlen_wrapper_is_per_trace():
    w = W.make_workload(3, shrink=128, batch=3, Hq=2, Hkv=1)
    T = w.total_tokens
    q, k, v, do = _rand(T, 2, 1, 8, 80)
    o, lse = O.varlen_fwd(q, k, v, w.evict_at, w.cu_seqlens, 0.3)
    dq, dk, dv = O.varlen_bwd(q, k, v, do, w.evict_at, w.cu_seqlens, 0.3)
    a, e = int(w.cu_seqlens[1]), int(w.cu_seqlens[2])
    o1, l1 = O.dense_fwd(q[a:e], k[a:e], v[a:e], w.trace(1), 0.3)
    g1 = O.dense_bwd(q[a:e], k[a:e], v[a:e], do[a:e], w.trace(1), 0.3)
    assert np.array_equal(o[a:e], o1) and np.array_equal(lse[:, a:e], l1)
    assert np.array_equal(dq[a:e], g1[0]) and np.array_equal(dk[a:e], g1[1]) and np.array_equal(dv[a:e], g1[2])


def test_bad_evict_at_rejected():
    with pytest.raises(ValueError):
        O.dense_fwd(np.zeros((3, 1, 2)), np.zeros((3, 1, 2)), np.zeros((3, 1, 2)), np.array([5, 1, 5]), 1.0)
