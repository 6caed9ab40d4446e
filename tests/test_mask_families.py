"""More mask families through the same kernels: Markovian Thinker, Markovian Pick, sliding
window with stride one turn, the controlled-retrieval mask, the SFT study's truncation mask,
and the utility that turns a compaction event log into evict_at."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

I = int(W.INF)


# ---- CPU: generators and the event-log oracle, by hand --------------------------------------------
def test_events_oracle_by_hand():
    # trace 0 (T=10): span [2,5) leaves at 6, span [4,8) leaves at 9 -> key 4 leaves at 6
    # trace 1 (T=6):  span [0,100) clipped to the trace, leaves at 3; a row for trace 7 is ignored
    cu = [0, 10, 16]
    events = [(0, 6, 2, 5), (0, 9, 4, 8), (1, 3, 0, 100), (7, 1, 0, 4)]
    got = O.evict_at_from_events(cu, events)
    assert got.tolist() == [I, I, 6, 6, 6, 9, 9, 9, I, I] + [3] * 6
    # the generator-side range assignment agrees with the key-by-key oracle
    a = W.events_to_evict_at(10, [(6, 2, 5), (9, 4, 8)])
    assert a.tolist() == got[:10].tolist()


def test_markovian_thinker_by_hand():
    # prompt 2, turns of 4 tokens, budget 10: after turn 2 the live context is 12 >= 10, so the oldest
    # turns go until <= 5 remain: turns 0 and 1 leave at the end of turn 2 (token 14); turn 2 stays until the next compaction, at the end of turn 4 (token 22)
    T = 30
    evs = W.markovian_thinker_events(T, 2, [4] * 10, 10)
    assert evs[:2] == [(14, 2, 6), (14, 6, 10)]
    ev = W.events_to_evict_at(T, evs)
    assert ev[:2].tolist() == [I, I] and ev[2:10].tolist() == [14] * 8 and ev[10:14].tolist() == [22] * 4
    # live context after a compaction never exceeds half the budget; before it, the budget plus one turn
    live = O.live_counts(ev) - 2 - 1          # minus prompt, minus the query itself
    assert live.max() <= 10 + 4


def test_markovian_pick_is_non_monotone_and_keeps_k():
    rng = np.random.default_rng(0)
    T = 400
    evs = W.markovian_pick_events(T, 10, [10] * 60, 5, 2, rng)
    ev = W.events_to_evict_at(T, evs).astype(np.int64)
    assert np.all(ev > np.arange(T))
    fin = ev[10:]
    # some later turn leaves before an earlier one: retention is not a suffix of the context
    d = np.diff(np.minimum(fin, T))
    assert (d < 0).any()
    # right after each compaction exactly `keep` old turns (+ nothing else) remain besides the prompt
    for when in sorted({e[0] for e in evs}):
        live = int(((np.arange(T) < when) & (ev > when)).sum())
        assert live == 10 + 2 * 10, (when, live)


def test_retrieval_and_truncation_masks():
    ev = W.events_to_evict_at(50, W.single_evicted_turn_events(50, 5, 15, 30))
    assert ev[4] == I and ev[5] == 30 and ev[14] == 30 and ev[15] == I
    A = O.allowed(ev)
    assert A[29, 10] and not A[30, 10] and A[40, 20]       # answer tokens do not see the assignment turn
    ev = W.events_to_evict_at(40, W.half_context_truncation_events(40, 8))
    assert ev[7] == I and ev[8] == 24 and ev[23] == 24 and ev[24] == I


def test_new_configs_are_valid_and_carry_their_event_log():
    for cfg in (5, 6, 7):
        w = W.make_workload(cfg, shrink=16, batch=2)
        assert w.events is not None and w.events.shape[1] == 4
        assert np.array_equal(O.evict_at_from_events(w.cu_seqlens, w.events), w.evict_at)
        for b in range(w.batch):
            ev = w.trace(b).astype(np.int64)
            assert np.all(ev > np.arange(ev.shape[0]))
        cls = O.tile_classes_rule(w.trace(0))
        assert np.array_equal(cls, O.tile_classes_brute(w.trace(0)))


# ---- GPU ------------------------------------------------------------------------------------------
@pytest.mark.gpu
def test_evict_at_from_events_on_gpu_is_bit_exact():
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(3)
    lens = [1, 300, 129, 4096]
    cu = np.zeros(len(lens) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    rows = []
    for _ in range(200):
        b = int(rng.integers(-1, len(lens) + 1))              # some rows name no trace
        T = lens[b] if 0 <= b < len(lens) else 100
        a = int(rng.integers(-5, T))
        z = a + int(rng.integers(0, 400))
        rows.append((b, int(rng.integers(1, T + 50)), a, z))
    events = np.asarray(rows, dtype=np.int32)
    want = O.evict_at_from_events(cu, events)
    got = B.kvs_evict_at_from_events(torch.from_numpy(events).cuda(), torch.from_numpy(cu).cuda(), int(cu[-1]))
    assert np.array_equal(got.cpu().numpy(), want)
    # no events at all: everything stays
    got = B.kvs_evict_at_from_events(torch.zeros((0, 4), dtype=torch.int32, device="cuda"), torch.from_numpy(cu).cuda(), int(cu[-1]))
    assert bool((got == I).all())
    for cfg in (5, 6):
        w = W.make_workload(cfg, shrink=4, batch=2)
        got = B.kvs_evict_at_from_events(torch.from_numpy(w.events).cuda(), torch.from_numpy(w.cu_seqlens).cuda(), w.total_tokens)
        assert np.array_equal(got.cpu().numpy(), w.evict_at)


@pytest.mark.gpu
@pytest.mark.parametrize("cfg", [5, 6, 7])
def test_mask_families_parity(cfg):
    from tests.test_gpu_parity import _full_parity
    _full_parity(W.make_workload(cfg, seed=2, shrink=16, Hq=8, Hkv=2, batch=2), seed=2)


@pytest.mark.gpu
def test_retrieval_mask_parity_from_event_log_built_on_gpu():
    from paper_2609_35750_b200 import binding as B
    from tests.test_gpu_parity import _full_parity
    T = 1500
    events = np.asarray([(0, 900, 200, 520)], dtype=np.int32)      # the assignment turn leaves before token 900
    cu = np.asarray([0, T], dtype=np.int32)
    ev = B.kvs_evict_at_from_events(torch.from_numpy(events).cuda(), torch.from_numpy(cu).cuda(), T).cpu().numpy()
    w = W.Workload("retrieval", cu, ev, 4, 2, 128)
    _full_parity(w, seed=5)


# ---- the re-prefill comparison workload (Sec. 2 "Prefill-compaction", App. E) ---------------------
def test_reprefill_token_accounting_matches_the_closed_form():
    # Summary layout of config 1: N = 30720 generated entries, r = prompt + summary = 2560 retained,
    # b = 4608 new entries per compaction, budget B = r + b = 7168 (the peak live-key count)
    lens = W.reprefill_summary_lengths(32768, 2048, 4096, 512)
    assert lens == [6656, 7168, 7168, 7168, 7168, 7168, 5632] and max(lens) == 7168
    extra = sum(lens) - 32768
    assert extra == 6 * 2560                                  # six compactions, each re-emits r entries
    closed = W.reprefill_extra_entries(30720, 2560, 7168)     # N r / (B - r), a continuous count of compactions
    assert abs(closed - 30720 / 4608 * 2560) < 1e-9 and 0 <= closed - extra < 2560
    # r = B/4 gives N/3 (the example printed with the derivation)
    assert abs(W.reprefill_extra_entries(3000, 25, 100) - 1000) < 1e-9
    # KV-streams prefills nothing again: the single trace has exactly N + prompt tokens
    assert W.make_workload(1, batch=1).total_tokens == 32768
    w = W.make_workload(1, variant="reprefill", batch=1)
    assert w.total_tokens == sum(lens) and np.all(w.evict_at == W.INF)


def test_reprefill_keep_last_k_by_hand_and_high_retention():
    # prompt 2, turns 3,2,4,3 (T=14), keep 1: first trace = prompt + turns 0,1 = 7; then every turn u >= 2
    # starts a trace with prompt + turn u-1 + turn u: 2+2+4 = 8, 2+4+3 = 9
    assert W.reprefill_keep_last_k_lengths(14, 2, [3, 2, 4, 3], 1) == [7, 8, 9]
    a, b = W.make_workload(2), W.make_workload(2, variant="reprefill")
    ratio = b.total_tokens / a.total_tokens
    # sliding window keeps almost the whole budget, so nearly everything is prefilled again at every turn:
    # with r ~ prompt + 4 turns and b ~ one turn the closed form gives r / b ~ 7.6 extra copies
    assert 6.0 < ratio < 9.0
    mean_turn = (256 + 2048) / 2
    closed = W.reprefill_extra_entries(65536 - 4096, 4096 + 4 * mean_turn, 4096 + 5 * mean_turn) / 65536
    assert abs((ratio - 1.0) - closed) / closed < 0.15


@pytest.mark.gpu
def test_reprefill_workload_parity():
    from tests.test_gpu_parity import _full_parity
    _full_parity(W.make_workload(2, variant="reprefill", shrink=32, Hq=4, Hkv=2, batch=1), seed=3)
