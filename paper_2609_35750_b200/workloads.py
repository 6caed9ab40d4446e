"""Seeded synthetic workloads: eviction patterns and Q/K/V/dO tensors.

This module holds inputs only.  It builds, from a seed, the per-key eviction
step ``evict_at`` that a compacting rollout would leave behind (Sec. 2,
"KV-streams" paragraph: the trainer sees one continuous trace plus the spans
the inference engine deleted) for the retention strategies of Sec. 3
(Summary, Sliding Window / keep-last-k-turns) and for a token-level stress
pattern (App. B.4 discusses token-level eviction), and it draws Gaussian
Q/K/V/dO.  None of the attention arithmetic lives here, so both the CPU
oracle and the CUDA path may be fed from it.

Conventions
-----------
* ``evict_at`` is int32, one entry per packed token, in TRACE-LOCAL
  coordinates: key ``j`` of a trace is visible to query ``i`` of the same
  trace iff ``j <= i < evict_at[j]``.
* "never evicted" is ``INF = 2**31 - 1``.
* ``cu_seqlens`` is int32 ``[batch + 1]`` with ``cu_seqlens[0] = 0``.
"""
from __future__ import annotations

import dataclasses
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

INF = np.int32(2**31 - 1)
BLOCK = 128  # tile edge used for the class statistics only


# --------------------------------------------------------------------------
# eviction patterns
# --------------------------------------------------------------------------
def summary_evict_at(T: int, prompt: int, work_lens, summary: int) -> np.ndarray:
    """Summary compaction (Sec. 3 "Summary": keep nothing, o = 0, bridge s).

    Layout: ``prompt`` tokens, then segments of ``work_lens[s]`` work tokens
    followed by ``summary`` summary tokens.  A segment completes iff its work
    and its summary both end at or before ``T``.  When segment ``s``
    completes at boundary ``e_s`` its work tokens and the summary of segment
    ``s - 1`` get ``evict_at = e_s``.  The prompt, the newest summary and the
    tokens of an unfinished trailing segment never evict.

    ``work_lens`` may be an int (every segment the same) or an iterable that
    yields one work length per segment.
    """
    ev = np.full(T, INF, dtype=np.int32)
    if isinstance(work_lens, (int, np.integer)):
        def _gen():
            while True:
                yield int(work_lens)
        it = _gen()
    else:
        it = iter(work_lens)
    pos = min(prompt, T)
    prev_summary = None  # (start, end) of the previous segment's summary
    while pos < T:
        try:
            w = int(next(it))
        except StopIteration:
            break
        w0, w1 = pos, pos + w
        s0, s1 = w1, w1 + summary
        if s1 > T:
            break  # unfinished trailing segment: nothing more is evicted
        ev[w0:w1] = s1
        if prev_summary is not None:
            ev[prev_summary[0]:prev_summary[1]] = s1
        prev_summary = (s0, s1)
        pos = s1
    return ev


def keep_last_k_evict_at(T: int, prompt: int, turn_lens, k: int) -> np.ndarray:
    """Keep-last-k-turns (Sec. 3 "Sliding Window": o close to B, s = 0).

    Turns follow the never-evicted prompt.  When turn ``t`` ends, every token
    of turn ``t - k`` gets ``evict_at`` = that end.  The last turn is cut at
    ``T``.
    """
    ev = np.full(T, INF, dtype=np.int32)
    starts: List[int] = []
    ends: List[int] = []
    pos = min(prompt, T)
    for L in turn_lens:
        if pos >= T:
            break
        e = min(pos + int(L), T)
        starts.append(pos)
        ends.append(e)
        pos = e
    assert pos >= T, "turn_lens too short to fill the trace"
    for t in range(k, len(starts)):
        ev[starts[t - k]:ends[t - k]] = ends[t]
    return ev


def fine_grained_evict_at(T: int, prompt: int, rng: np.random.Generator,
                          mean: float, every_other: bool = True) -> np.ndarray:
    """Token-level stress: key ``j >= prompt`` with ``(j - prompt)`` odd gets
    ``evict_at = j + 1 + G_j``, ``G_j`` geometric on {0,1,...} with the given
    mean (inverse CDF ``floor(log U / log(1 - p))``, ``p = 1/(mean + 1)``).
    With ``every_other=False`` every non-prompt key is evicted this way."""
    ev = np.full(T, INF, dtype=np.int32)
    if T <= prompt:
        return ev
    j = np.arange(prompt, T, dtype=np.int64)
    sel = ((j - prompt) % 2 == 1) if every_other else np.ones_like(j, dtype=bool)
    p = 1.0 / (mean + 1.0)
    u = rng.random(j.shape[0])
    u = np.maximum(u, np.finfo(np.float64).tiny)
    g = np.floor(np.log(u) / np.log1p(-p)).astype(np.int64)
    val = np.minimum(j + 1 + g, int(INF) - 1)
    ev[prompt:][sel] = val[sel].astype(np.int32)
    return ev


def events_to_evict_at(T: int, events) -> np.ndarray:
    """Turns a compaction event log into ``evict_at``.  ``events`` is an iterable of
    ``(when, start, end)``: at step ``when`` (the index of the first token generated after
    the compaction) the keys ``[start, end)`` leave the cache.  A key named by several
    events leaves at the earliest one."""
    ev = np.full(T, INF, dtype=np.int32)
    for when, a, b in events:
        a, b = max(0, int(a)), min(T, int(b))
        if b > a:
            ev[a:b] = np.minimum(ev[a:b], np.int32(when))
    return ev


def _turn_bounds(T: int, prompt: int, turn_lens):
    starts, ends = [], []
    pos = min(prompt, T)
    for L in turn_lens:
        if pos >= T:
            break
        e = min(pos + int(L), T)
        starts.append(pos)
        ends.append(e)
        pos = e
    assert pos >= T, "turn_lens too short to fill the trace"
    return starts, ends


def markovian_thinker_events(T: int, prompt: int, turn_lens, budget: int):
    """Markovian Thinker (Sec. 3: o = B/2, s = 0): whenever the live context (prompt excluded)
    reaches ``budget`` tokens at the end of a turn, the oldest live turns are deleted until at
    most half the budget remains.  Whole turns only (App. B.4).  Returns the event list."""
    starts, ends = _turn_bounds(T, prompt, turn_lens)
    live = []                       # indices of live turns, oldest first
    events = []
    for t in range(len(starts)):
        live.append(t)
        size = sum(ends[u] - starts[u] for u in live)
        if size >= budget and ends[t] < T:
            while live and size > budget // 2:
                u = live.pop(0)
                size -= ends[u] - starts[u]
                events.append((ends[t], starts[u], ends[u]))
    return events


def markovian_pick_events(T: int, prompt: int, turn_lens, interval: int, keep: int, rng: np.random.Generator):
    """Markovian Pick (Sec. 3): every ``interval`` turns the model chooses ``keep`` of the live
    turns to retain and deletes all the others; here the choice is uniform at random, which
    gives the arbitrary, non-contiguous retention the strategy allows."""
    starts, ends = _turn_bounds(T, prompt, turn_lens)
    live = []
    events = []
    for t in range(len(starts)):
        live.append(t)
        if (t + 1) % interval == 0 and ends[t] < T and len(live) > keep:
            kept = set(rng.choice(len(live), size=keep, replace=False).tolist())
            for idx, u in enumerate(live):
                if idx not in kept:
                    events.append((ends[t], starts[u], ends[u]))
            live = [u for idx, u in enumerate(live) if idx in kept]
    return events


def single_evicted_turn_events(T: int, start: int, end: int, when: int):
    """The controlled-retrieval mask (App. C.1 "Eviction and retrieval"): one early turn (the
    assignment) leaves the cache before the answer tokens; everything else stays."""
    return [(when, start, end)]


def half_context_truncation_events(T: int, prompt: int):
    """The SFT study's truncation mask (Sec. 6.1: half of the context masked, B = N/2): the
    first half of the non-prompt context leaves once it has been generated."""
    half = prompt + (T - prompt) // 2
    return [(half, prompt, half)] if half > prompt else []


# --------------------------------------------------------------------------
# re-prefill compaction: the comparison workload (Sec. 2 "Prefill-compaction", App. E)
# --------------------------------------------------------------------------
def reprefill_summary_lengths(T: int, prompt: int, work: int, summary: int) -> List[int]:
    """Trace lengths when the Summary rollout of `summary_evict_at` is trained the re-prefill
    way: every compaction starts a fresh trace that re-emits the retained entries (prompt and
    the newest summary, r = prompt + summary) and then holds the next segment."""
    lens, pos, first = [], min(prompt, T), True
    while pos < T:
        seg = min(work + summary, T - pos)
        complete = seg == work + summary
        lens.append((prompt if first else prompt + summary) + seg)
        pos += seg
        first = False
        if not complete:
            break
    return lens


def reprefill_keep_last_k_lengths(T: int, prompt: int, turn_lens, k: int) -> List[int]:
    """Trace lengths when the keep-last-k-turns rollout is trained the re-prefill way: a
    compaction happens at the end of every turn t >= k (turn t - k is deleted), and the fresh
    trace re-emits the prompt and the k retained turns before generating the next turn."""
    starts, ends = _turn_bounds(T, prompt, turn_lens)
    n = len(starts)
    if n <= k + 1:
        return [T]
    lens = [ends[k]]                                     # prompt + turns 0..k, no compaction yet
    for u in range(k + 1, n):
        retained = ends[u - 1] - starts[u - k]
        lens.append(prompt + retained + (ends[u] - starts[u]))
    return lens


def reprefill_extra_entries(N: float, r: float, B: float) -> float:
    """Closed form of the extra prefilled entries (Sec. 2): N r / (B - r)."""
    return N * r / (B - r)


# --------------------------------------------------------------------------
# workloads
# --------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    cu_seqlens: np.ndarray          # int32 [batch + 1]
    evict_at: np.ndarray            # int32 [Ttot], trace-local
    Hq: int
    Hkv: int
    d: int
    q_prescale: float = 1.0         # multiplier applied to Q before bf16 rounding
    softmax_scale: float = 0.0      # 0 => 1/sqrt(d)
    notes: str = ""
    rules: List[str] = field(default_factory=list)
    events: Optional[np.ndarray] = None   # int32 [n, 4] rows (trace, when, start, end), when the mask came from an event log

    @property
    def batch(self) -> int:
        return int(self.cu_seqlens.shape[0] - 1)

    @property
    def total_tokens(self) -> int:
        return int(self.cu_seqlens[-1])

    @property
    def max_seqlen(self) -> int:
        return int(np.diff(self.cu_seqlens).max()) if self.batch else 0

    @property
    def scale(self) -> float:
        return self.softmax_scale if self.softmax_scale != 0.0 else 1.0 / float(np.sqrt(self.d))

    def trace(self, b: int) -> np.ndarray:
        return self.evict_at[self.cu_seqlens[b]:self.cu_seqlens[b + 1]]


def _rng(seed: int, cfg: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) + cfg, stream]))


def _pack(traces) -> (np.ndarray, np.ndarray):
    lens = np.array([len(t) for t in traces], dtype=np.int64)
    cu = np.zeros(len(traces) + 1, dtype=np.int32)
    cu[1:] = np.cumsum(lens)
    ev = np.concatenate(traces).astype(np.int32) if len(traces) else np.zeros(0, np.int32)
    return cu, ev


def make_workload(cfg: int, seed: int = 0, shrink: int = 1,
                  Hq: Optional[int] = None, Hkv: Optional[int] = None,
                  batch: Optional[int] = None, variant: str = "") -> Workload:
    """The five synthetic traces.  ``shrink`` divides every length of the
    layout (trace, prompt, segment, turn) by an integer so that the CPU oracle
    can run the whole tensor; head counts and batch may be overridden for the
    same reason.  ``variant``: cfg 1 "B" (scale folded into Q, softmax scale
    1); cfg 4 "b" (every non-prompt key evicted); any cfg "control" (same
    shapes and values, nothing ever evicted: plain causal attention);
    cfg 1, 2 "reprefill" (the rollouts cut into re-prefill's fresh traces).
    """
    s = int(shrink)
    assert s >= 1
    if variant == "control" and cfg != 4:
        w = make_workload(cfg, seed, shrink, Hq, Hkv, batch, "")
        return dataclasses.replace(w, name=w.name + "_control_causal", evict_at=np.full_like(w.evict_at, INF),
                                   rules=None, events=None, notes=w.notes + "; control: evict_at = INF everywhere")
    if variant == "reprefill":
        # the same rollouts cut into the fresh traces re-prefill compaction trains on: plain causal
        # attention (nothing is evicted inside a trace), retained entries present again in every trace
        if cfg == 1:
            lens = reprefill_summary_lengths(32768 // s, 2048 // s, 4096 // s, 512 // s) * (batch or 4)
            hq, hkv, pre, name = 28, 4, 1.0 / np.sqrt(128), "cfg1_reprefill"
        elif cfg == 2:
            T, prompt = 65536 // s, 4096 // s
            lo, hi = max(1, 256 // s), max(1, 2048 // s)
            lens = []
            for b in range(batch or 2):
                r = _rng(seed, 2, b)                       # the turn lengths of the KV-streams trace of config 2
                tl = r.integers(lo, hi + 1, size=(T - prompt) // lo + 2)
                lens += reprefill_keep_last_k_lengths(T, prompt, tl, 4)
            hq, hkv, pre, name = 32, 8, 1.0, "cfg2_reprefill"
        else:
            raise ValueError("the re-prefill variant exists for configs 1 and 2")
        cu = np.zeros(len(lens) + 1, dtype=np.int32)
        cu[1:] = np.cumsum(lens)
        return Workload(name, cu, np.full(int(cu[-1]), INF, dtype=np.int32), Hq or hq, Hkv or hkv, 128, q_prescale=pre,
                        notes=f"{len(lens)} fresh traces, plain causal; retained entries re-emitted at every compaction")
    if cfg == 0:
        T, prompt, work, summ = 1024 // s, 128 // s, 192 // s, 32 // s
        ev = summary_evict_at(T, prompt, work, summ)
        cu, eva = _pack([ev] * (batch or 1))
        return Workload("cfg0_tiny_summary", cu, eva, Hq or 4, Hkv or 4, 64,
                        notes="1 trace T=1024, prompt 128, 4x(192 work + 32 summary)")
    if cfg == 1:
        T, prompt, work, summ = 32768 // s, 2048 // s, 4096 // s, 512 // s
        ev = summary_evict_at(T, prompt, work, summ)
        cu, eva = _pack([ev] * (batch or 4))
        d = 128
        if variant == "B":
            return Workload("cfg1B_7b_summary", cu, eva, Hq or 28, Hkv or 4, d,
                            q_prescale=1.0 / np.sqrt(d), softmax_scale=1.0,
                            notes="scale folded into Q, softmax_scale=1")
        return Workload("cfg1_7b_summary", cu, eva, Hq or 28, Hkv or 4, d,
                        q_prescale=1.0 / np.sqrt(d),
                        notes="4 traces T=32768, prompt 2048, 6x(4096+512)+3072 leftover; "
                              "Q drawn N(0,1)*1/sqrt(d), kernel scale 1/sqrt(d)")
    if cfg == 2:
        T, prompt = 65536 // s, 4096 // s
        lo, hi = max(1, 256 // s), max(1, 2048 // s)
        traces = []
        for b in range(batch or 2):
            r = _rng(seed, 2, b)
            lens = r.integers(lo, hi + 1, size=(T - prompt) // lo + 2)
            traces.append(keep_last_k_evict_at(T, prompt, lens, 4))
        cu, eva = _pack(traces)
        return Workload("cfg2_keep_last_4_turns", cu, eva, Hq or 32, Hkv or 8, 128,
                        notes="2 traces T=65536, prompt 4096, turns U[256,2048], keep last 4")
    if cfg == 3:
        nb = batch or 16
        r = _rng(seed, 3, 0)
        lens = r.integers(8192 // s, 32768 // s + 1, size=nb)
        traces, rules = [], []
        for b in range(nb):
            rb = _rng(seed, 3, 1 + b)
            T = int(lens[b])
            if rb.integers(0, 2) == 0:
                wl = rb.integers(max(1, 1024 // s), max(1, 4096 // s) + 1, size=T // max(1, 1024 // s) + 2)
                traces.append(summary_evict_at(T, 2048 // s, wl, max(1, 256 // s)))
                rules.append("summary")
            else:
                k = int(rb.integers(2, 7))
                lo, hi = max(1, 256 // s), max(1, 2048 // s)
                tl = rb.integers(lo, hi + 1, size=T // lo + 2)
                traces.append(keep_last_k_evict_at(T, 4096 // s, tl, k))
                rules.append(f"keep_last_{k}")
        cu, eva = _pack(traces)
        return Workload("cfg3_varlen_packed", cu, eva, Hq or 32, Hkv or 8, 128, rules=rules,
                        notes="16 traces U[8192,32768], mixed summary / keep-last-k rules")
    if cfg == 4:
        T, prompt = 131072 // s, 1024 // s
        if variant == "control":
            ev = np.full(T, INF, dtype=np.int32)
            name = "cfg4_control_causal"
        else:
            ev = fine_grained_evict_at(T, prompt, _rng(seed, 4, 0), 8192.0 / s,
                                       every_other=(variant != "b"))
            name = "cfg4b_fine_grained_all" if variant == "b" else "cfg4_fine_grained"
        cu, eva = _pack([ev] * (batch or 1))
        return Workload(name, cu, eva, Hq or 64, Hkv or 8, 128,
                        notes="1 trace T=131072, prompt 1024, alternate keys evicted after 1+Geom(8192)")
    if cfg in (5, 6, 7):
        # further mask families through the same kernels (not in the five headline configs)
        T, prompt = 65536 // s, 4096 // s
        lo, hi = max(1, 256 // s), max(1, 2048 // s)
        traces, log = [], []
        for b in range(batch or 2):
            r = _rng(seed, cfg, b)
            lens = r.integers(lo, hi + 1, size=(T - prompt) // lo + 2)
            if cfg == 5:
                evs = markovian_thinker_events(T, prompt, lens, 16384 // s)
            elif cfg == 6:
                evs = markovian_pick_events(T, prompt, lens, 10, 4, r)
            else:
                evs = half_context_truncation_events(T, prompt) if b % 2 else \
                    [(e, a, z) for (e, a, z) in _sliding_window_events(T, prompt, lens, 10)]
            traces.append(events_to_evict_at(T, evs))
            log += [(b, int(e), int(a), int(z)) for (e, a, z) in evs]
        cu, eva = _pack(traces)
        name = {5: "cfg5_markovian_thinker", 6: "cfg6_markovian_pick", 7: "cfg7_sft_random_masks"}[cfg]
        note = {5: "turns U[256,2048], budget 16384: oldest turns deleted down to half the budget",
                6: "turns U[256,2048], every 10 turns keep 4 random live turns",
                7: "sliding window of 10 turns (stride 1) or half-context truncation, alternating"}[cfg]
        return Workload(name, cu, eva, Hq or 32, Hkv or 8, 128, notes=f"{batch or 2} traces T={T}, prompt {prompt}; " + note,
                        events=np.asarray(log, dtype=np.int32).reshape(-1, 4))
    raise ValueError(f"unknown config {cfg}")


def _sliding_window_events(T: int, prompt: int, turn_lens, window: int):
    """Sliding window over turns with stride 1 (Sec. 6.1: B = 10): when turn t ends, turn
    t - window leaves."""
    starts, ends = _turn_bounds(T, prompt, turn_lens)
    return [(ends[t], starts[t - window], ends[t - window]) for t in range(window, len(starts))]


# --------------------------------------------------------------------------
# integer statistics of a workload (used for FLOP accounting and as pins)
# --------------------------------------------------------------------------
def count_pairs(w: Workload) -> int:
    """Number of allowed (i, j) pairs, head independent:
    sum_j (min(evict_at[j], T) - j) per trace."""
    total = 0
    for b in range(w.batch):
        ev = w.trace(b).astype(np.int64)
        T = ev.shape[0]
        j = np.arange(T, dtype=np.int64)
        total += int((np.minimum(ev, T) - j).sum())
    return total


def fwd_bwd_flops(w: Workload) -> int:
    """Unmasked FLOPs: 2 GEMMs forward + 5 backward, 2 flops per MAC."""
    return 14 * w.d * w.Hq * count_pairs(w)


# --------------------------------------------------------------------------
# tensors
# --------------------------------------------------------------------------
def make_tensors(w: Workload, seed: int = 0, device: str = "cpu", with_dout: bool = True):
    """bf16 q [Ttot,Hq,d], k, v [Ttot,Hkv,d], dout [Ttot,Hq,d] ~ N(0,1) (q times
    ``q_prescale`` before rounding), drawn by torch's seeded generator on the
    requested device.  Returns torch tensors."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(1000003 * seed + 17)
    T = w.total_tokens

    def draw(h, mul=1.0):
        x = torch.randn((T, h, w.d), generator=g, device=device, dtype=torch.float32)
        if mul != 1.0:
            x = x * mul
        return x.to(torch.bfloat16)

    q = draw(w.Hq, w.q_prescale)
    k = draw(w.Hkv)
    v = draw(w.Hkv)
    dout = draw(w.Hq) if with_dout else None
    return q, k, v, dout
