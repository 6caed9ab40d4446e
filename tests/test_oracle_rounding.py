"""Pins for the oracle's statement of the method's operand rounding (CPU only).

dense_fwd_bwd_rounded is the dense definition with the three bf16 roundings of the method (P, dS and
the stored O) switched on; rounding_sigma is the first-order standard deviation of what they cause.
Pinned by: (1) with the roundings off the emulation IS the dense definition, bit for bit; (2) the
rounding helper against torch's own bf16 conversion, including ties; (3) the rms relative rounding
error constant against a direct measurement on log-uniform significands; (4) the predicted deviations
against the emulation's actual error, element by element (normalised errors: rms close to 1, none
beyond 6.5), on several mask families and group sizes; (5) special cases where a source of error
vanishes (evict-after-one-step: P is exactly 0 or 1, so only the rounding of the stored O remains).
"""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W


def _f64(t):
    return t.float().numpy().astype(np.float64)


def _inputs(w, seed):
    return tuple(_f64(t) for t in W.make_tensors(w, seed))


def test_round_bf16_matches_torch_including_ties():
    r = np.random.default_rng(0)
    x = np.concatenate([r.standard_normal(20000) * 10.0 ** r.integers(-6, 6, size=20000),
                        # exact ties between two bf16 neighbours (8th significant bit boundary) and their neighbours
                        np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8, -(2.0 + 2.0 ** -7), 0.0, 2.0 ** -130, 65280.0 + 128.0]),
                        ])
    want = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(O.round_bf16(x), want)
    assert O.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0                # tie -> even significand
    assert O.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_rms_relative_rounding_error_constant():
    r = np.random.default_rng(1)
    x = np.exp(r.uniform(np.log(1e-4), np.log(1e4), size=400000))           # log-uniform: significands log-uniform on [1, 2)
    xb = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    rel = (xb - x) / x
    assert np.abs(rel).max() <= O.U_BF16 * (1 + 1e-6)
    assert abs(np.sqrt((rel ** 2).mean()) / O.RHO_BF16 - 1.0) < 0.01
    assert abs(O.RHO_BF16 - 1.659e-3) < 2e-6


@pytest.mark.parametrize("case", ["cfg0", "cfg2_G4", "random_G3"])
def test_roundings_off_is_the_dense_definition_bit_for_bit(case):
    if case == "cfg0":
        w = W.make_workload(0, Hq=2, Hkv=2)
    elif case == "cfg2_G4":
        w = W.make_workload(2, shrink=64, Hq=4, Hkv=1, batch=1)
    else:
        T = 200
        r = np.random.default_rng(3)
        ev = np.where(r.random(T) < 0.5, np.arange(T) + r.integers(1, 60, size=T), int(W.INF)).astype(np.int32)
        w = W.Workload("r", np.array([0, T], dtype=np.int32), ev, 3, 1, 64)
    q, k, v, do = _inputs(w, 2)
    ev = w.trace(0)
    o, l, dq, dk, dv = O.dense_fwd_bwd_rounded(q, k, v, do, ev, w.scale, round_p=False, round_ds=False, round_out=False)
    ro, rl = O.dense_fwd(q, k, v, ev, w.scale)
    rdq, rdk, rdv = O.dense_bwd(q, k, v, do, ev, w.scale)
    for a, b in ((o, ro), (l, rl), (dq, rdq), (dk, rdk), (dv, rdv)):
        assert np.array_equal(a, b)
    # each switch alone changes what it should and nothing upstream of it
    o2, l2, dq2, dk2, dv2 = O.dense_fwd_bwd_rounded(q, k, v, do, ev, w.scale, round_p=False, round_ds=True, round_out=False)
    assert np.array_equal(o2, ro) and np.array_equal(dv2, rdv) and not np.array_equal(dq2, rdq) and not np.array_equal(dk2, rdk)
    o3, l3, dq3, dk3, dv3 = O.dense_fwd_bwd_rounded(q, k, v, do, ev, w.scale, round_p=True, round_ds=False, round_out=False)
    assert np.array_equal(l3, rl) and not np.array_equal(o3, ro) and not np.array_equal(dv3, rdv)
    o4 = O.dense_fwd_bwd_rounded(q, k, v, do, ev, w.scale, round_p=False, round_ds=False, round_out=True)[0]
    assert np.array_equal(o4, O.round_bf16(ro))


@pytest.mark.parametrize("kw", [dict(cfg=0), dict(cfg=2, shrink=64, Hq=8, Hkv=1, batch=1), dict(cfg=4, shrink=128, Hq=4, Hkv=2),
                                dict(cfg=1, shrink=32, Hq=7, Hkv=1, batch=1, variant="B")])
def test_predicted_deviation_matches_the_emulated_error(kw):
    w = W.make_workload(seed=3, **kw)
    q, k, v, do = _inputs(w, 3)
    ev = w.trace(0)
    T = ev.shape[0]
    q, k, v, do = q[:T], k[:T], v[:T], do[:T]
    o, l, dq, dk, dv = O.dense_fwd_bwd_rounded(q, k, v, do, ev, w.scale)
    ro, rl = O.dense_fwd(q, k, v, ev, w.scale)
    rdq, rdk, rdv = O.dense_bwd(q, k, v, do, ev, w.scale)
    sg = O.rounding_sigma(q, k, v, do, ev, w.scale)
    assert np.abs(l - rl).max() < 1e-12                                  # the row sums are taken before any rounding
    for name, got, ref in (("out", o, ro), ("dq", dq, rdq), ("dk", dk, rdk), ("dv", dv, rdv)):
        z = (got - ref) / np.maximum(sg[name], 1e-300)
        rms = float(np.sqrt((z ** 2).mean()))
        assert 0.85 <= rms <= 1.15, (name, rms)
        assert np.abs(z).max() <= 6.5, (name, float(np.abs(z).max()))
        # and the stated tolerances do hold for the method's own rounding on these inputs
        assert np.linalg.norm(got - ref) / np.linalg.norm(ref) <= 5e-3


def test_no_probability_rounding_when_every_key_is_seen_only_by_itself():
    T = 150
    w = W.Workload("one_step", np.array([0, T], dtype=np.int32), (np.arange(T) + 1).astype(np.int32), 4, 2, 64)
    q, k, v, do = _inputs(w, 5)
    sg = O.rounding_sigma(q, k, v, do, w.evict_at, w.scale)
    o, l, dq, dk, dv = O.dense_fwd_bwd_rounded(q, k, v, do, w.evict_at, w.scale)
    # P is the identity: bf16 represents it exactly, O = v is already bf16, dS = P (dP - D) = 0
    assert np.array_equal(o, np.repeat(v, 2, axis=1)) and np.abs(dq).max() == 0 and np.abs(dk).max() == 0
    # the model still charges the rounding of P = 1 (it does not know the value is representable) and of O;
    # what it must not do is predict noise for dq and dk, whose dS is identically zero apart from D's share
    assert sg["dv"].max() <= O.RHO_BF16 * np.abs(do).max() * np.sqrt(2) * 1.0001
    assert sg["out"].max() <= np.sqrt((O.RHO_BF16 * np.abs(v).max()) ** 2 + (2.0 ** -8 * np.abs(v).max()) ** 2)


def test_varlen_sigma_is_per_trace():
    w = W.make_workload(3, seed=1, shrink=128, Hq=2, Hkv=1, batch=3)
    q, k, v, do = _inputs(w, 1)
    sg = O.varlen_rounding_sigma(q, k, v, do, w.evict_at, w.cu_seqlens, w.scale)
    a, e = int(w.cu_seqlens[1]), int(w.cu_seqlens[2])
    one = O.rounding_sigma(q[a:e], k[a:e], v[a:e], do[a:e], w.evict_at[a:e], w.scale)
    for name in sg:
        assert np.array_equal(sg[name][a:e], one[name])
