"""CPU fp64 oracle for eviction-masked causal attention (TEST INFRASTRUCTURE).

This file is the slow, plain statement of what the CUDA path must compute.  It
is imported only by the tests, by the smoke check and by the benchmark's CPU
baseline leg; the library never calls it, and it shares no code with the CUDA
sources.

What it states, and where that comes from:

* Mask.  Sec. 2 ("KV-streams" paragraph) and the caption of Fig. 2 say that the
  trainer processes ONE continuous trace and that a custom attention mask
  blocks attention to the span the inference engine deleted, so that one
  forward pass reproduces the rollout's evictions.  Encoded per key as an
  eviction step: query ``i`` may read key ``j`` iff ``j <= i < evict_at[j]``.
  Positions are not reset (Sec. 2: retained entries keep their ``(k_i, v_i)``),
  so q and k are used as given.
* ``dense_*``: softmax attention under that boolean mask, written out from the
  definition, with its analytic gradients.
* ``replay_*``: the rollout itself (Sec. 1 and Sec. 2: KV entries are evicted
  directly in the engine's cache).  A cache of rows is kept; before token ``i``
  is processed every row whose eviction step is ``i`` is physically removed;
  token ``i`` is appended; ``q_i`` attends over exactly the rows present.  No
  mask is ever consulted.  Agreement of the two routes is the check that the
  mask above is the one that reproduces eviction.
* Tile classes: the min/max rule per 128x128 tile and, independently, a brute
  force classification from the dense boolean mask.

* Key slots: a trace's keys may be stored in any order if each slot carries the index and the
  eviction step of the key it holds (``key_first``), e.g. sorted by eviction step for token-level
  eviction (App. B.4), ``reorder_keys``; ``merge_partial`` is attention over a union of disjoint key sets.
* ``dual_fwd``: student under the eviction mask + full-context teacher (self-distillation, App. D.3).
* ``rope_rotate``: rotary embedding with positions that are never reset (Sec. 2).
* ``dense_fwd_bwd_rounded`` / ``rounding_sigma``: the three bf16 roundings of the method (P, dS, the
  stored O) switched on inside the fp64 definition, and their first-order propagation to a standard
  deviation per output element: what the stated tolerances have to absorb.

Everything is fp64 on inputs that were already rounded to bf16 by the caller.
Pins (tests/test_oracle_pins.py, test_mask_families.py, test_oracle_rounding.py, test_key_slots.py,
test_dual_forward.py, test_rope_and_packed.py): two-route agreement, no-eviction == plain causal
attention (torch's CPU scaled_dot_product_attention in fp64), softmax rows summing to one, central
finite differences for dQ/dK/dV (also through the rotation), zero-query closed forms (exp(LSE) =
live-key count, values printed in tests/golden), evict-after-one-step closed form, exact integer pair and
tile counts; key slots: invariance under key permutation, brute-force loops, rule vs brute-force
classes; merge: student part + evicted part == full causal attention; rotation: plane rotation by hand,
norm preservation, dependence on position differences only, inverse == transpose; rounding: roundings
off == the dense definition bit for bit, the rounding helper against torch's bf16 conversion, the
predicted deviation against the emulated error.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

INF = 2**31 - 1
BLOCK = 128
EMPTY, PARTIAL, FULL = 0, 1, 2


# --------------------------------------------------------------------------
# mask
# --------------------------------------------------------------------------
def allowed(evict_at: np.ndarray, key_first=None) -> np.ndarray:
    """Boolean [T, T]: allowed[i, j] = (j <= i) and (i < evict_at[j]).

    With ``key_first`` (int [T]) column j is a key SLOT that carries its own interval: allowed[i, j] =
    (key_first[j] <= i) and (i < evict_at[j]).  Attention does not depend on the order of its keys, so a
    trace's keys may be stored in any order as long as slot j carries the index and the eviction step of
    the key it holds; ``key_first[j] = j`` is the plain case."""
    ev = np.asarray(evict_at, dtype=np.int64)
    T = ev.shape[0]
    i = np.arange(T, dtype=np.int64)[:, None]
    first = np.arange(T, dtype=np.int64) if key_first is None else np.asarray(key_first, dtype=np.int64)
    return (first[None, :] <= i) & (i < ev[None, :])


def check_evict_at(evict_at: np.ndarray) -> None:
    """Precondition: every key is visible at least to its own query."""
    ev = np.asarray(evict_at, dtype=np.int64)
    j = np.arange(ev.shape[0], dtype=np.int64)
    if np.any(ev <= j):
        raise ValueError("evict_at[j] <= j for some key")


# --------------------------------------------------------------------------
# dense masked attention, one trace
# --------------------------------------------------------------------------
def dense_fwd(q, k, v, evict_at, scale, key_first=None):
    """q [T,Hq,d], k,v [T,Hkv,d] (any float dtype; widened to fp64).
    Returns out [T,Hq,d] fp64, lse [Hq,T] fp64 (natural log, scale included).
    With ``key_first`` the rows of k, v are key slots (see ``allowed``); a query that sees no slot gets
    out = 0 and lse = -inf."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    if key_first is None:
        check_evict_at(evict_at)
    A = allowed(evict_at, key_first)
    out = np.zeros((T, Hq, d))
    lse = np.zeros((Hq, T))
    for h in range(Hq):
        g = h // G
        S = scale * (q[:, h, :] @ k[:, g, :].T)
        S = np.where(A, S, -np.inf)
        m = S.max(axis=1, keepdims=True)
        m = np.where(np.isfinite(m), m, 0.0)           # a row that sees nothing: every term below is zero
        E = np.exp(S - m)
        l = E.sum(axis=1, keepdims=True)
        P = E / np.where(l > 0, l, 1.0)
        out[:, h, :] = P @ v[:, g, :]
        with np.errstate(divide="ignore"):
            lse[h, :] = (m + np.log(l))[:, 0]
    return out, lse


def dense_bwd(q, k, v, dout, evict_at, scale, key_first=None):
    """Analytic gradients of sum(out * dout) w.r.t. q, k, v.
    Returns dq [T,Hq,d], dk, dv [T,Hkv,d] (fp64).  ``key_first``: as in dense_fwd."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    A = allowed(evict_at, key_first)
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for h in range(Hq):
        g = h // G
        S = scale * (q[:, h, :] @ k[:, g, :].T)
        S = np.where(A, S, -np.inf)
        m = S.max(axis=1, keepdims=True)
        m = np.where(np.isfinite(m), m, 0.0)
        E = np.exp(S - m)
        l = E.sum(axis=1, keepdims=True)
        P = E / np.where(l > 0, l, 1.0)
        O = P @ v[:, g, :]
        dP = dout[:, h, :] @ v[:, g, :].T
        D = (dout[:, h, :] * O).sum(axis=1, keepdims=True)
        dS = P * (dP - D)
        dq[:, h, :] = scale * (dS @ k[:, g, :])
        dk[:, g, :] += scale * (dS.T @ q[:, h, :])
        dv[:, g, :] += P.T @ dout[:, h, :]
    return dq, dk, dv


# --------------------------------------------------------------------------
# incremental replay with physical eviction, one trace
# --------------------------------------------------------------------------
def replay_fwd_bwd(q, k, v, dout, evict_at, scale, removal="ordered"):
    """Replays the rollout token by token.  The cache is a Python list of
    original key indices; rows leave it for good at their eviction step.

    removal: "ordered" keeps the surviving rows in order, "swap" moves the
    last row into the hole (row order must not matter).
    Returns out, lse, dq, dk, dv, cache_sizes (int array, rows present when
    token i attends).  ``dout`` may be None (then the gradients are None)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    ev = np.asarray(evict_at, dtype=np.int64)
    check_evict_at(ev)
    # keys bucketed by the step at which the engine drops them
    leaving = {}
    for j in range(T):
        if ev[j] < T:
            leaving.setdefault(int(ev[j]), []).append(j)
    out = np.zeros((T, Hq, d))
    lse = np.zeros((Hq, T))
    sizes = np.zeros(T, dtype=np.int64)
    want_grad = dout is not None
    if want_grad:
        dout = np.asarray(dout, dtype=np.float64)
        dq = np.zeros_like(q)
        dk = np.zeros_like(k)
        dv = np.zeros_like(v)
    cache = []          # original indices of the rows present
    where = {}          # original index -> slot in `cache`
    for i in range(T):
        for j in leaving.get(i, ()):
            slot = where.pop(j)
            if removal == "swap":
                last = cache.pop()
                if last != j:
                    cache[slot] = last
                    where[last] = slot
            else:
                del cache[slot]
                for s in range(slot, len(cache)):
                    where[cache[s]] = s
        where[i] = len(cache)
        cache.append(i)
        rows = np.asarray(cache, dtype=np.int64)
        sizes[i] = rows.shape[0]
        for h in range(Hq):
            g = h // G
            Kc = k[rows, g, :]
            Vc = v[rows, g, :]
            s = scale * (Kc @ q[i, h, :])
            m = s.max()
            e = np.exp(s - m)
            l = e.sum()
            p = e / l
            o = p @ Vc
            out[i, h, :] = o
            lse[h, i] = m + np.log(l)
            if want_grad:
                do = dout[i, h, :]
                dp = Vc @ do
                ds = p * (dp - do @ o)
                dq[i, h, :] = scale * (ds @ Kc)
                np.add.at(dk[:, g, :], rows, scale * np.outer(ds, q[i, h, :]))
                np.add.at(dv[:, g, :], rows, np.outer(p, do))
    if want_grad:
        return out, lse, dq, dk, dv, sizes
    return out, lse, None, None, None, sizes


# --------------------------------------------------------------------------
# packed (varlen) wrappers
# --------------------------------------------------------------------------
def varlen_fwd(q, k, v, evict_at, cu_seqlens, scale):
    q = np.asarray(q, dtype=np.float64)
    Ttot, Hq, d = q.shape
    out = np.zeros((Ttot, Hq, d))
    lse = np.zeros((Hq, Ttot))
    for b in range(len(cu_seqlens) - 1):
        a, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == a:
            continue
        o, l = dense_fwd(q[a:e], k[a:e], v[a:e], evict_at[a:e], scale)
        out[a:e] = o
        lse[:, a:e] = l
    return out, lse


def varlen_bwd(q, k, v, dout, evict_at, cu_seqlens, scale):
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(k)
    for b in range(len(cu_seqlens) - 1):
        a, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == a:
            continue
        x, y, z = dense_bwd(q[a:e], k[a:e], v[a:e], dout[a:e], evict_at[a:e], scale)
        dq[a:e], dk[a:e], dv[a:e] = x, y, z
    return dq, dk, dv


# --------------------------------------------------------------------------
# single rows / single key blocks of a long trace (for full-size sampling)
# --------------------------------------------------------------------------
def row_fwd(q_i, k, v, evict_at, i, scale):
    """One query row ``i`` of one head.  q_i [d]; k, v [T, d] of its KV head.
    Returns o [d], lse (float), visible key indices, p over them."""
    ev = np.asarray(evict_at[: i + 1], dtype=np.int64)
    vis = np.nonzero(ev > i)[0]
    Kc = np.asarray(k[vis], dtype=np.float64)
    Vc = np.asarray(v[vis], dtype=np.float64)
    s = scale * (Kc @ np.asarray(q_i, dtype=np.float64))
    m = s.max()
    e = np.exp(s - m)
    l = e.sum()
    p = e / l
    return p @ Vc, m + np.log(l), vis, p


def row_fwd_bwd(q_i, k, v, do_i, evict_at, i, scale):
    """As row_fwd, plus dq_i [d] and this row's contributions (vis, dk_rows, dv_rows)."""
    o, lse, vis, p = row_fwd(q_i, k, v, evict_at, i, scale)
    Kc = np.asarray(k[vis], dtype=np.float64)
    Vc = np.asarray(v[vis], dtype=np.float64)
    do = np.asarray(do_i, dtype=np.float64)
    dp = Vc @ do
    ds = p * (dp - do @ o)
    dq = scale * (ds @ Kc)
    return o, lse, dq, vis, scale * np.outer(ds, np.asarray(q_i, dtype=np.float64)), np.outer(p, do)


def key_block_dkdv(q, k, v, dout, evict_at, j0, j1, g, G, scale):
    """dK, dV for keys [j0, j1) of KV head ``g`` of one trace: every query row
    that can see any of those keys is evaluated in full (its softmax needs all
    of its visible keys).  q, dout [T,Hq,d]; k, v [T,Hkv,d].
    Returns dk [j1-j0, d], dv [j1-j0, d]."""
    ev = np.asarray(evict_at, dtype=np.int64)
    T = ev.shape[0]
    last = int(min(T, ev[j0:j1].max()))          # first row that sees none of them
    dk = np.zeros((j1 - j0, q.shape[2]))
    dv = np.zeros((j1 - j0, q.shape[2]))
    kg = np.asarray(k[:, g, :], dtype=np.float64)
    vg = np.asarray(v[:, g, :], dtype=np.float64)
    for i in range(j0, last):
        vis = np.nonzero(ev[: i + 1] > i)[0]
        sel = (vis >= j0) & (vis < j1)
        if not sel.any():
            continue
        Kc, Vc = kg[vis], vg[vis]
        for h in range(g * G, (g + 1) * G):
            qi = np.asarray(q[i, h, :], dtype=np.float64)
            do = np.asarray(dout[i, h, :], dtype=np.float64)
            s = scale * (Kc @ qi)
            e = np.exp(s - s.max())
            p = e / e.sum()
            o = p @ Vc
            ds = p * (Vc @ do - do @ o)
            dk[vis[sel] - j0] += scale * np.outer(ds[sel], qi)
            dv[vis[sel] - j0] += np.outer(p[sel], do)
    return dk, dv


# --------------------------------------------------------------------------
# tile classes
# --------------------------------------------------------------------------
def block_minmax(evict_at, block=BLOCK):
    """kmin[n], kmax[n] over the valid keys (key slots) of key block n (one trace)."""
    ev = np.asarray(evict_at, dtype=np.int64)
    T = ev.shape[0]
    nb = (T + block - 1) // block
    kmin = np.zeros(nb, dtype=np.int32)
    kmax = np.zeros(nb, dtype=np.int32)
    for n in range(nb):
        blk = ev[n * block: min((n + 1) * block, T)]
        kmin[n] = blk.min()
        kmax[n] = blk.max()
    return kmin, kmax


def tile_classes_rule(evict_at, block=BLOCK, key_first=None):
    """Classes [nb, nb] uint8 from the min/max rule.  With q0, q1 the first and
    last valid query of block m and k0, k1 the first and last valid key of
    block n: EMPTY if k0 > q1 or q0 >= kmax[n]; FULL if k1 <= q0 and
    q1 < kmin[n]; otherwise PARTIAL.  With ``key_first`` (key slots, see ``allowed``) k0 and k1 are
    the smallest and the largest key_first of the block's slots."""
    T = len(evict_at)
    nb = (T + block - 1) // block
    kmin, kmax = block_minmax(evict_at, block)
    if key_first is None:
        fmin = np.arange(nb, dtype=np.int64) * block
        fmax = np.minimum(fmin + block - 1, T - 1)
    else:
        fmin, fmax = block_minmax(key_first, block)
    cls = np.zeros((nb, nb), dtype=np.uint8)
    for m in range(nb):
        q0, q1 = m * block, min(m * block + block - 1, T - 1)
        for n in range(nb):
            k0, k1 = int(fmin[n]), int(fmax[n])
            if k0 > q1 or q0 >= int(kmax[n]):
                c = EMPTY
            elif k1 <= q0 and q1 < int(kmin[n]):
                c = FULL
            else:
                c = PARTIAL
            cls[m, n] = c
    return cls


def tile_classes_brute(evict_at, block=BLOCK, key_first=None):
    """Classes [nb, nb] uint8 straight from the boolean mask: all allowed ->
    FULL, none -> EMPTY, else PARTIAL."""
    A = allowed(evict_at, key_first)
    T = A.shape[0]
    nb = (T + block - 1) // block
    cls = np.zeros((nb, nb), dtype=np.uint8)
    for m in range(nb):
        for n in range(nb):
            t = A[m * block: min((m + 1) * block, T), n * block: min((n + 1) * block, T)]
            cls[m, n] = FULL if t.all() else (EMPTY if not t.any() else PARTIAL)
    return cls


def live_counts(evict_at):
    """n_i = number of keys visible to query i (one trace)."""
    return allowed(evict_at).sum(axis=1)


# --------------------------------------------------------------------------
# compaction event log -> evict_at
# --------------------------------------------------------------------------
def evict_at_from_events(cu_seqlens, events):
    """events: rows (trace, when, start, end): at step ``when`` of trace ``trace`` the keys
    [start, end) (trace-local) leave the cache (Sec. 2: the delete operator removes a span).
    Key by key: evict_at[j] = the earliest ``when`` among the events whose span holds j,
    2^31-1 if none.  Spans are clipped to the trace; rows naming no trace are ignored."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    total = int(cu[-1])
    out = np.full(total, INF, dtype=np.int64)
    ev = np.asarray(events, dtype=np.int64).reshape(-1, 4)
    for b in range(len(cu) - 1):
        T = int(cu[b + 1] - cu[b])
        mine = ev[ev[:, 0] == b]
        for j in range(T):
            best = INF
            for (_, when, a, z) in mine:
                if a <= j < z and when < best:
                    best = int(when)
            out[cu[b] + j] = best
    return out.astype(np.int32)


# --------------------------------------------------------------------------
# paged KV cache with physical eviction (the engine's bookkeeping, Sec. 4 / App. B.3)
# --------------------------------------------------------------------------
class PagedCacheModel:
    """Plain-Python model of the block tables and the free stack: pages of `page_size`
    tokens; a sequence's table lists the pages of its live cache in order; eviction removes
    table entries (whole pages) and pushes the pages back; appending pops a page when the
    last one is full.  Page 0 is handed out first; freed pages are pushed in table order."""

    def __init__(self, num_pages, page_size, num_seqs):
        self.page_size = page_size
        self.free = list(range(num_pages - 1, -1, -1))     # stack, top at the end
        self.tables = [[] for _ in range(num_seqs)]
        self.n_tokens = [0] * num_seqs

    def append(self, s):
        if self.n_tokens[s] % self.page_size == 0:
            if not self.free:
                raise RuntimeError("cache full")
            self.tables[s].append(self.free.pop())
        slot = self.n_tokens[s]
        self.n_tokens[s] += 1
        return self.tables[s][slot // self.page_size], slot % self.page_size

    def evict(self, s, ranges):
        """ranges: (first_page_slot, n_pages) in positions of the current table."""
        npages = len(self.tables[s])
        gone = set()
        for a, cnt in ranges:
            if a < 0 or cnt < 0 or a + cnt > npages:
                raise ValueError("range outside the table")
            if a + cnt == npages and cnt > 0 and self.n_tokens[s] % self.page_size != 0:
                raise ValueError("the partially filled last page cannot leave")
            gone.update(range(a, a + cnt))
        kept = [p for i, p in enumerate(self.tables[s]) if i not in gone]
        freed = [p for i, p in enumerate(self.tables[s]) if i in gone]
        self.tables[s] = kept
        self.free.extend(freed)
        self.n_tokens[s] -= len(freed) * self.page_size


# --------------------------------------------------------------------------
# operand rounding: what the 2e-2 / 5e-3 tolerances have to absorb
# --------------------------------------------------------------------------
# The method computes with bf16 operands and fp32 accumulation.  Apart from the inputs (already
# bf16) three intermediate quantities are rounded to bf16 before they are used again: the
# probabilities P (operand of P V and of P^T dO), the score gradients dS (operand of dS K and
# dS^T Q) and the stored output O (which the row sums D = dO . O are formed from).  Two functions
# state the consequence in fp64:
#   dense_fwd_bwd_rounded   the definition with exactly those three roundings switched on or off;
#                           with all of them off it is dense_fwd / dense_bwd, bit for bit
#   rounding_sigma          first-order propagation of those roundings, as a standard deviation
#                           per output element, treating every rounding error as independent with
#                           the rms relative size RHO_BF16
# The tests use them to bound the CUDA path's max-abs error element by element: 2e-2 wherever six
# standard deviations of the inherent rounding stay below it, six standard deviations elsewhere.
U_BF16 = 2.0 ** -8            # largest relative error of round-to-nearest to 8 significant bits
# rms relative error of that rounding for significands spread log-uniformly over [1, 2):
# sqrt(E[1/m^2] / 3) * 2^-8 with E[1/m^2] = (1/2 - 1/8) / ln 2
RHO_BF16 = U_BF16 * float(np.sqrt((0.5 - 0.125) / np.log(2.0) / 3.0))


def round_bf16(x):
    """Nearest bf16 value (ties to even) of every element, returned as fp64."""
    x32 = np.ascontiguousarray(np.asarray(x, dtype=np.float64).astype(np.float32))
    bits = x32.view(np.uint32).astype(np.uint64)
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return bits.astype(np.uint32).view(np.float32).reshape(x32.shape).astype(np.float64)


def dense_fwd_bwd_rounded(q, k, v, dout, evict_at, scale, round_p=True, round_ds=True, round_out=True):
    """dense_fwd + dense_bwd with the method's three operand roundings (see above).
    Returns out, lse, dq, dk, dv (fp64; out holds bf16 values when round_out)."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    check_evict_at(evict_at)
    A = allowed(evict_at)
    out = np.zeros((T, Hq, d))
    lse = np.zeros((Hq, T))
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for h in range(Hq):
        g = h // G
        S = scale * (q[:, h, :] @ k[:, g, :].T)
        S = np.where(A, S, -np.inf)
        m = S.max(axis=1, keepdims=True)
        E = np.exp(S - m)
        l = E.sum(axis=1, keepdims=True)       # the row sum is taken before the rounding
        P = E / l
        Pv = round_bf16(E) / l if round_p else P
        O = Pv @ v[:, g, :]
        if round_out:
            O = round_bf16(O)
        out[:, h, :] = O
        lse[h, :] = (m + np.log(l))[:, 0]
        Pb = round_bf16(P) if round_p else P
        dP = dout[:, h, :] @ v[:, g, :].T
        D = (dout[:, h, :] * O).sum(axis=1, keepdims=True)
        dS = P * (dP - D)
        if round_ds:
            dSs = round_bf16(scale * dS)       # the scale is folded in before the rounding
            dq[:, h, :] = dSs @ k[:, g, :]
            dk[:, g, :] += dSs.T @ q[:, h, :]
        else:
            dq[:, h, :] = scale * (dS @ k[:, g, :])
            dk[:, g, :] += scale * (dS.T @ q[:, h, :])
        dv[:, g, :] += Pb.T @ dout[:, h, :]
    return out, lse, dq, dk, dv


def rounding_sigma(q, k, v, dout, evict_at, scale):
    """Standard deviation, per element of out, dq, dk, dv, of the error that the three operand
    roundings cause, to first order, every rounding error independent with relative rms RHO_BF16
    (the output rounding of O: uniform within half a bf16 ulp of O).

        out_ic:  P_ij e_ij v_jc summed over j, plus its own rounding
        D_i   :  sum_c dO_ic (error of the stored O_ic); common to the whole row i of dS
        dv_jc :  sum_{h,i} P_ij e_ij dO_ic
        dq_ic :  s sum_j dS_ij e'_ij k_jc  -  s dD_i sum_j P_ij k_jc
        dk_jc :  s sum_{h,i} (dS_ij e'_ij - P_ij dD_i) q_ic

    Returns a dict of fp64 arrays shaped like the tensors."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    dout = np.asarray(dout, dtype=np.float64)
    T, Hq, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    A = allowed(evict_at)
    r2 = RHO_BF16 ** 2
    var_out = np.zeros((T, Hq, d))
    var_dq = np.zeros_like(q)
    var_dk = np.zeros_like(k)
    var_dv = np.zeros_like(v)
    for h in range(Hq):
        g = h // G
        kk, vv, qq, do = k[:, g, :], v[:, g, :], q[:, h, :], dout[:, h, :]
        S = np.where(A, scale * (qq @ kk.T), -np.inf)
        E = np.exp(S - S.max(axis=1, keepdims=True))
        P = E / E.sum(axis=1, keepdims=True)
        O = P @ vv
        P2 = P * P
        var_o_p = r2 * (P2 @ (vv * vv))                              # from the rounding of P
        ulp_half = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(O), 1e-300))) - 8)
        var_o = var_o_p + ulp_half ** 2 / 3.0                         # plus the rounding of O itself
        var_out[:, h, :] = var_o
        var_D = ((do * do) * var_o).sum(axis=1, keepdims=True)       # [T, 1]
        dS = P * (do @ vv.T - (do * O).sum(axis=1, keepdims=True))
        dS2 = dS * dS
        var_dv[:, g, :] += r2 * (P2.T @ (do * do))
        var_dq[:, h, :] = scale ** 2 * (r2 * (dS2 @ (kk * kk)) + var_D * (P @ kk) ** 2)
        var_dk[:, g, :] += scale ** 2 * (r2 * (dS2.T @ (qq * qq)) + (P2 * var_D).T @ (qq * qq))
    return {"out": np.sqrt(var_out), "dq": np.sqrt(var_dq), "dk": np.sqrt(var_dk), "dv": np.sqrt(var_dv)}


def varlen_rounding_sigma(q, k, v, dout, evict_at, cu_seqlens, scale):
    """rounding_sigma trace by trace over a packed batch."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    res = {"out": np.zeros_like(q), "dq": np.zeros_like(q), "dk": np.zeros_like(k), "dv": np.zeros_like(k)}
    for b in range(len(cu_seqlens) - 1):
        a, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == a:
            continue
        s = rounding_sigma(q[a:e], k[a:e], v[a:e], dout[a:e], evict_at[a:e], scale)
        for name in res:
            res[name][a:e] = s[name]
    return res


# --------------------------------------------------------------------------
# student + teacher forward (self-distillation, App. D.3 "Training Objectives")
# --------------------------------------------------------------------------
def dual_fwd(q, k, v, evict_at, scale):
    """The two passes of the self-distillation objective on one trace, same q, k, v: the student under
    the eviction mask, the teacher with the full causal context (nothing evicted).  By definition two
    calls of dense_fwd.  Returns (out_student, lse_student, out_teacher, lse_teacher)."""
    T = np.asarray(evict_at).shape[0]
    os_, ls_ = dense_fwd(q, k, v, evict_at, scale)
    ot_, lt_ = dense_fwd(q, k, v, np.full(T, INF, dtype=np.int64), scale)
    return os_, ls_, ot_, lt_


def varlen_dual_fwd(q, k, v, evict_at, cu_seqlens, scale):
    q = np.asarray(q, dtype=np.float64)
    Ttot, Hq, d = q.shape
    res = [np.zeros((Ttot, Hq, d)), np.zeros((Hq, Ttot)), np.zeros((Ttot, Hq, d)), np.zeros((Hq, Ttot))]
    for b in range(len(cu_seqlens) - 1):
        a, e = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        if e == a:
            continue
        r = dual_fwd(q[a:e], k[a:e], v[a:e], evict_at[a:e], scale)
        res[0][a:e], res[1][:, a:e], res[2][a:e], res[3][:, a:e] = r
    return tuple(res)


# --------------------------------------------------------------------------
# key order for token-level eviction; partial results over disjoint key sets
# --------------------------------------------------------------------------
def reorder_keys(evict_at, window):
    """Permutation of one trace's keys: within every window of ``window`` consecutive keys, sorted by
    (evict_at, index).  Returns perm (perm[s] = index of the key stored in slot s).  The slots then carry
    key_first = perm and key_evict = evict_at[perm]; the attention result is unchanged (sums over keys do
    not depend on their order), but the slots of a 128-slot block now leave the cache at about the same
    time, which is what lets a tile be classified FULL or EMPTY (App. B.4 discusses token-level eviction)."""
    ev = np.asarray(evict_at, dtype=np.int64)
    T = ev.shape[0]
    perm = np.zeros(T, dtype=np.int64)
    for w0 in range(0, T, window):
        idx = list(range(w0, min(w0 + window, T)))
        idx.sort(key=lambda j: (int(ev[j]), j))
        perm[w0:w0 + len(idx)] = idx
    return perm


def merge_partial(out_a, lse_a, out_b, lse_b):
    """Attention over the union of two DISJOINT key sets from the results over each: with weights
    w_x = exp(lse_x - lse), lse = log(exp(lse_a) + exp(lse_b)):  out = w_a out_a + w_b out_b.
    out_* [T,Hq,d], lse_* [Hq,T]; a part that saw no key has lse = -inf and weight 0."""
    la = np.asarray(lse_a, dtype=np.float64)
    lb = np.asarray(lse_b, dtype=np.float64)
    m = np.maximum(la, lb)
    m0 = np.where(np.isfinite(m), m, 0.0)
    with np.errstate(divide="ignore"):
        lse = m0 + np.log(np.exp(la - m0) + np.exp(lb - m0))
    wa = np.exp(la - np.where(np.isfinite(lse), lse, 0.0)) * np.isfinite(la)
    wb = np.exp(lb - np.where(np.isfinite(lse), lse, 0.0)) * np.isfinite(lb)
    out = wa.T[:, :, None] * np.asarray(out_a, dtype=np.float64) + wb.T[:, :, None] * np.asarray(out_b, dtype=np.float64)
    return out, lse


# --------------------------------------------------------------------------
# rotary position embedding on one continuous trace
# --------------------------------------------------------------------------
def rope_rotate(x, positions, theta_base=10000.0, inverse=False):
    """x [T, H, d]; positions int [T].  Rotate-half convention: for c < d/2 and angle = pos * base^(-2c/d),
    y[c] = x[c] cos - x[c + d/2] sin,  y[c + d/2] = x[c + d/2] cos + x[c] sin.
    KV-streams never resets positions when entries are evicted (Sec. 2), so on the training trace
    ``positions`` is simply each token's index in its trace.  ``inverse`` rotates by the opposite angle,
    which is the transpose: the map from gradients w.r.t. y to gradients w.r.t. x."""
    x = np.asarray(x, dtype=np.float64)
    T, H, d = x.shape
    half = d // 2
    pos = np.asarray(positions, dtype=np.float64)
    inv_freq = theta_base ** (-2.0 * np.arange(half) / d)
    ang = pos[:, None] * inv_freq[None, :]
    if inverse:
        ang = -ang
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    y = np.empty_like(x)
    y[..., :half] = x[..., :half] * c - x[..., half:] * s
    y[..., half:] = x[..., half:] * c + x[..., :half] * s
    return y


def trace_positions(cu_seqlens):
    """Trace-local index of every packed token."""
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    return np.concatenate([np.arange(cu[b + 1] - cu[b]) for b in range(len(cu) - 1)] or [np.zeros(0, np.int64)])
