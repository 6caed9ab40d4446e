"""Generators: exact integer pins for the synthetic traces (CPU only)."""
import os

import numpy as np
import pytest

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


def test_cfg0_evict_at_and_pairs_match_hand_derivation():
    w = W.make_workload(0)
    assert w.total_tokens == 1024 and w.batch == 1 and (w.Hq, w.Hkv, w.d) == (4, 4, 64)
    for r in _read("cfg0_evict_at.txt"):
        if r[0] == "pairs":
            assert W.count_pairs(w) == int(r[1])
        elif r[0] == "tiles":
            pass  # checked against the oracle classifiers in test_oracle_pins
        else:
            want = int(W.INF) if r[1] == "INF" else int(r[1])
            assert int(w.evict_at[int(r[0])]) == want, r
    assert W.fwd_bwd_flops(w) == 14 * 64 * 4 * 245248


def test_cfg1_counts():
    w = W.make_workload(1)
    assert w.batch == 4 and w.total_tokens == 131072 and (w.Hq, w.Hkv, w.d) == (28, 4, 128)
    g = {r[0]: [int(x) for x in r[1:]] for r in _read("cfg1_counts.txt")}
    assert W.count_pairs(w) == 4 * g["pairs"][0]
    T = 32768
    assert T * (T + 1) // 2 == g["causal_pairs"][0]
    ev = w.trace(0)
    # leftover (unfinished segment) never evicts; last complete segment's work leaves at its end
    assert int(ev[2048 + 6 * 4608]) == int(W.INF) and int(ev[-1]) == int(W.INF)
    assert int(ev[2048 + 5 * 4608]) == 2048 + 6 * 4608
    assert int(ev[2048 + 5 * 4608 + 4096]) == int(W.INF)      # newest summary
    assert int(ev[2048 + 4 * 4608 + 4096]) == 2048 + 6 * 4608  # previous summary leaves one segment later


def test_every_key_visible_to_itself_all_configs():
    for cfg, kw in [(0, {}), (1, {}), (2, {}), (3, {}), (4, {}), (4, {"variant": "b"}), (4, {"variant": "control"})]:
        w = W.make_workload(cfg, seed=0, **kw)
        for b in range(w.batch):
            ev = w.trace(b).astype(np.int64)
            assert np.all(ev > np.arange(ev.shape[0])), (cfg, b)
        assert w.cu_seqlens[0] == 0 and np.all(np.diff(w.cu_seqlens) > 0)


def test_cfg2_structure():
    w = W.make_workload(2, seed=0)
    assert w.batch == 2 and w.total_tokens == 131072
    for b in range(2):
        ev = w.trace(b).astype(np.int64)
        assert np.all(ev[:4096] == int(W.INF))           # prompt never evicted
        fin = ev[ev < int(W.INF)]
        j = np.nonzero(ev < int(W.INF))[0]
        life = fin - j
        # a token of turn t-4 lives until the end of turn t: between 4 and 5 turns plus itself
        assert life.min() >= 4 * 256 and life.max() <= 5 * 2048
    dens = W.count_pairs(w) / (2 * 65536 * 65537 // 2)
    assert 0.2 < dens < 0.35
    # seeds differ, same seed repeats
    w2 = W.make_workload(2, seed=0)
    w3 = W.make_workload(2, seed=1)
    assert np.array_equal(w.evict_at, w2.evict_at) and not np.array_equal(w.evict_at, w3.evict_at)


def test_cfg3_varlen_ragged():
    w = W.make_workload(3, seed=0)
    lens = np.diff(w.cu_seqlens)
    assert w.batch == 16 and lens.min() >= 8192 and lens.max() <= 32768
    assert any(L % 128 for L in lens)                      # ragged tails exist
    assert {"summary"} <= set(w.rules) and any(r.startswith("keep_last_") for r in w.rules)


def test_cfg4_geometric_mean_and_parity_of_keys():
    w = W.make_workload(4, seed=0)
    ev = w.trace(0).astype(np.int64)
    j = np.arange(ev.shape[0])
    fin = ev < int(W.INF)
    assert not fin[:1024].any()
    assert np.all(((j[fin] - 1024) % 2) == 1)
    assert fin[1024:].sum() == (131072 - 1024) // 2
    g = ev[fin] - j[fin] - 1
    assert g.min() >= 0 and abs(g.mean() - 8192) < 200
    c = W.make_workload(4, variant="control")
    assert np.all(c.evict_at == W.INF)
    assert W.count_pairs(c) == 131072 * 131073 // 2


def test_keep_last_k_small_by_hand():
    # prompt 2, turns of 3,2,4,... tokens, keep last 1 turn: turn t-1 leaves when turn t ends
    ev = W.keep_last_k_evict_at(12, 2, [3, 2, 4, 9], 1)
    I = int(W.INF)
    assert ev.tolist() == [I, I, 7, 7, 7, 11, 11, 12, 12, 12, 12, I]


def test_summary_small_by_hand():
    # prompt 1, work 2 + summary 1, T=9: segments [1,4) [4,7), leftover [7,9)
    ev = W.summary_evict_at(9, 1, 2, 1)
    I = int(W.INF)
    assert ev.tolist() == [I, 4, 4, 7, 7, 7, I, I, I]


def test_make_tensors_deterministic_and_bf16():
    import torch
    w = W.make_workload(0)
    a = W.make_tensors(w, seed=3)
    b = W.make_tensors(w, seed=3)
    c = W.make_tensors(w, seed=4)
    for x, y in zip(a, b):
        assert x.dtype == torch.bfloat16 and torch.equal(x, y)
    assert not torch.equal(a[0], c[0])
    assert a[0].shape == (1024, 4, 64) and a[1].shape == (1024, 4, 64)


def test_control_variant_of_any_config_is_plain_causal():
    for cfg in (0, 2, 3):
        a = W.make_workload(cfg, shrink=8 if cfg else 1)
        c = W.make_workload(cfg, shrink=8 if cfg else 1, variant="control")
        assert np.array_equal(a.cu_seqlens, c.cu_seqlens) and (a.Hq, a.Hkv, a.d) == (c.Hq, c.Hkv, c.d)
        assert np.all(c.evict_at == W.INF) and c.name.endswith("_control_causal")
        lens = np.diff(c.cu_seqlens).astype(np.int64)
        assert W.count_pairs(c) == int((lens * (lens + 1) // 2).sum())      # closed form of the causal triangle
        assert W.count_pairs(a) < W.count_pairs(c)
