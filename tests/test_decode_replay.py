"""Rollout side on the GPU: a paged KV cache with physical eviction and decode attention, replayed
token by token and compared with the oracle's replay (which removes rows from a cache and never
looks at a mask) and with the masked forward kernel on the same trace."""
import numpy as np
import pytest
import torch

from oracle import kvs_oracle as O
from paper_2609_35750_b200 import workloads as W

MAX_ABS, REL_L2 = 2e-2, 5e-3


def _page_ranges(live, leaving, page_size):
    """The engine's translation of "these original tokens leave" into table slots: positions of the
    leaving tokens in the live order, grouped into runs, each run a whole number of pages."""
    pos = sorted(live.index(j) for j in leaving)
    runs, start, prev = [], None, None
    for p in pos:
        if start is None:
            start = prev = p
        elif p == prev + 1:
            prev = p
        else:
            runs.append((start, prev + 1))
            start = prev = p
    if start is not None:
        runs.append((start, prev + 1))
    out = []
    for a, z in runs:
        assert a % page_size == 0 and z % page_size == 0, "eviction must cover whole pages (turns are padded to page multiples)"
        out.append((a // page_size, (z - a) // page_size))
    return out


# ---- CPU: the bookkeeping model and the slot translation ---------------------------------------------
def test_paged_cache_model_by_hand():
    m = O.PagedCacheModel(num_pages=4, page_size=2, num_seqs=1)
    slots = [m.append(0) for _ in range(5)]
    assert slots == [(0, 0), (0, 1), (1, 0), (1, 1), (2, 0)] and m.tables[0] == [0, 1, 2] and m.free == [3]
    with pytest.raises(ValueError):
        m.evict(0, [(2, 1)])                      # the partially filled last page cannot leave
    m.evict(0, [(0, 1)])
    assert m.tables[0] == [1, 2] and m.n_tokens[0] == 3 and m.free == [3, 0]
    assert m.append(0) == (2, 1) and m.append(0) == (0, 0)        # page 0 is used again
    assert m.tables[0] == [1, 2, 0] and m.n_tokens[0] == 5


def test_page_range_translation():
    live = list(range(40, 72))                    # 32 live tokens, two of them groups leave
    assert _page_ranges(live, list(range(40, 48)) + list(range(56, 64)), 8) == [(0, 1), (2, 1)]
    assert _page_ranges(live, [41, 43, 44], 1) == [(1, 1), (3, 2)]
    with pytest.raises(AssertionError):
        _page_ranges(live, list(range(41, 49)), 8)


# ---- GPU --------------------------------------------------------------------------------------------
def _replay_gpu(w, q, k, v, page_size, num_pages, check_tables):
    """Replays trace 0 of w on the GPU cache.  Returns out [T,Hq,d], lse [T,Hq], n_tokens per step."""
    from paper_2609_35750_b200 import binding as B
    ev = w.trace(0).astype(np.int64)
    T = ev.shape[0]
    cache = B.PagedCache(num_pages, page_size, 1, (T + page_size - 1) // page_size + 1, w.Hkv, w.d)
    model = O.PagedCacheModel(num_pages, page_size, 1)
    leaving = {}
    for j in range(T):
        if ev[j] < T:
            leaving.setdefault(int(ev[j]), []).append(j)
    qd, kd, vd = q.cuda(), k.cuda(), v.cuda()
    outs = torch.empty((T, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    lses = torch.empty((T, w.Hq), dtype=torch.float32, device="cuda")
    ws = torch.empty(1 << 22, dtype=torch.uint8, device="cuda")
    sizes, live = [], []
    for i in range(T):
        if i in leaving:
            ranges = _page_ranges(live, leaving[i], page_size)
            cache.evict(torch.tensor([(0, a, c) for a, c in ranges], dtype=torch.int32, device="cuda"))
            model.evict(0, ranges)
            gone = set(leaving[i])
            live = [j for j in live if j not in gone]
        cache.append(kd[i:i + 1], vd[i:i + 1])
        model.append(0)
        live.append(i)
        cache.decode(qd[i:i + 1], softmax_scale=w.softmax_scale, num_splits=2, out=outs[i:i + 1], lse=lses[i:i + 1], workspace=ws)
        sizes.append(len(live))
        if check_tables and (i % 97 == 0 or i in leaving or i == T - 1):
            n = int(cache.n_tokens[0])
            assert n == model.n_tokens[0] == len(live)
            np_ = (n + page_size - 1) // page_size
            assert cache.block_table[0, :np_].cpu().tolist() == model.tables[0]
    rc, free = cache.status()
    assert rc == B.KVS_OK and free == len(model.free)
    return outs, lses, np.asarray(sizes)


def _cmp(name, got, ref):
    got, ref = np.asarray(got, np.float64), np.asarray(ref, np.float64)
    assert np.isfinite(got).all(), name
    assert np.abs(got - ref).max() <= MAX_ABS, f"{name}: max-abs {np.abs(got - ref).max():.4f}"
    rel = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert rel <= REL_L2, f"{name}: rel-L2 {rel:.3e}"


@pytest.mark.gpu
@pytest.mark.parametrize("case", ["cfg0_pages16", "cfg4_tokens", "cfg1_G7_pages16"])
def test_replay_with_physical_eviction_matches_oracle_and_masked_forward(case):
    from paper_2609_35750_b200 import binding as B
    if case == "cfg0_pages16":
        w, ps = W.make_workload(0), 16                      # every boundary of the tiny trace is a multiple of 32
        pool = 384 // 16 + 2                                # peak live cache 384 tokens: far fewer pages than T/16 = 64
    elif case == "cfg4_tokens":
        w, ps = W.make_workload(4, shrink=128, Hq=8, Hkv=1), 1     # token-level eviction, block size 1
        pool = int(O.live_counts(w.trace(0)).max()) + 2
    else:
        w, ps = W.make_workload(1, shrink=16, Hq=7, Hkv=1, batch=1), 16
        pool = int(O.live_counts(w.trace(0)).max()) // 16 + 2
    q, k, v, _ = W.make_tensors(w, 1)
    T = w.total_tokens
    assert pool * ps < T                                     # the pool is smaller than the trace: pages must be reused
    outs, lses, sizes = _replay_gpu(w, q, k, v, ps, pool, check_tables=True)
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    ro, rl, _, _, _, rsizes = O.replay_fwd_bwd(f64(q), f64(k), f64(v), None, w.trace(0), w.scale)
    assert np.array_equal(sizes, rsizes)                     # the live cache has the oracle's size at every step
    _cmp("decode out vs replay oracle", f64(outs), ro)
    _cmp("decode lse vs replay oracle", f64(lses).T, rl)
    # the masked forward kernel on the whole trace gives the same rows: eviction == mask, on the GPU
    ev = torch.from_numpy(w.evict_at).cuda()
    cu = torch.from_numpy(w.cu_seqlens).cuda()
    meta = B.kvs_mask_meta(ev, cu, w.max_seqlen)
    fo, fl = B.kvs_attn_fwd(q.cuda(), k.cuda(), v.cuda(), meta, 1, w.max_seqlen, w.softmax_scale)
    assert float((outs.float() - fo.float()).abs().max()) <= MAX_ABS
    assert float((lses.t() - fl).abs().max()) <= 1e-3


@pytest.mark.gpu
def test_batched_decode_three_sequences_and_error_reporting():
    from paper_2609_35750_b200 import binding as B
    w = W.make_workload(2, seed=5, shrink=64, Hq=4, Hkv=2, batch=3)          # three traces of 1024 tokens, arbitrary turn lengths
    q, k, v, _ = W.make_tensors(w, 5)
    T, S = 1024, 3
    cache = B.PagedCache(600, 1, S, T, w.Hkv, w.d)
    qd, kd, vd = (t.cuda().view(S, T, t.shape[1], t.shape[2]) for t in (q, k, v))
    evs = [w.trace(b).astype(np.int64) for b in range(S)]
    lives = [[] for _ in range(S)]
    outs = torch.empty((T, S, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
    lses = torch.empty((T, S, w.Hq), dtype=torch.float32, device="cuda")
    for i in range(T):
        ranges = []
        for b in range(S):
            gone = [j for j in lives[b] if evs[b][j] == i]
            if gone:
                ranges += [(b, a, c) for a, c in _page_ranges(lives[b], gone, 1)]
                lives[b] = [j for j in lives[b] if evs[b][j] != i]
            lives[b].append(i)
        if ranges:
            cache.evict(torch.tensor(ranges, dtype=torch.int32, device="cuda"))
        cache.append(kd[:, i].contiguous(), vd[:, i].contiguous())
        cache.decode(qd[:, i].contiguous(), out=outs[i], lse=lses[i], max_tokens=T)
    assert cache.n_tokens.cpu().tolist() == [len(l) for l in lives]
    # pages are disjoint across sequences and, with the free stack, make up the whole pool
    tables = [cache.block_table[b, :len(lives[b])].cpu().tolist() for b in range(S)]
    rc, free = cache.status()
    used = sum(tables, [])
    assert rc == B.KVS_OK and len(set(used)) == len(used) and len(used) + free == 600
    f64 = lambda t: t.float().cpu().numpy().astype(np.float64)
    for b in range(S):
        a, e = int(w.cu_seqlens[b]), int(w.cu_seqlens[b + 1])
        ro, rl, *_ = O.replay_fwd_bwd(f64(q[a:e]), f64(k[a:e]), f64(v[a:e]), None, evs[b], w.scale)
        _cmp(f"seq {b} out", f64(outs[:, b]), ro)
        _cmp(f"seq {b} lse", f64(lses[:, b]).T, rl)
    # errors are reported through the status word, and the device stays usable
    bad = B.PagedCache(2, 4, 1, 8, 1, 64)
    kk = torch.zeros((1, 1, 64), dtype=torch.bfloat16, device="cuda")
    for _ in range(9):                                        # the ninth token needs a third page
        bad.append(kk, kk)
    assert bad.status()[0] == B.KVS_ERR_WORKSPACE and int(bad.n_tokens[0]) == 8
    bad2 = B.PagedCache(4, 4, 1, 8, 1, 64)
    for _ in range(6):
        bad2.append(kk, kk)
    bad2.evict(torch.tensor([(0, 1, 1)], dtype=torch.int32, device="cuda"))        # the half-filled last page
    assert bad2.status()[0] == B.KVS_ERR_INVALID_ARG and int(bad2.n_tokens[0]) == 6


@pytest.mark.gpu
@pytest.mark.parametrize("G,Hkv,ps", [(4, 2, 16), (8, 1, 16), (7, 2, 8), (8, 2, 32), (4, 1, 128), (8, 1, 64),
                                      (8, 1, 1), (4, 2, 4), (7, 1, 3), (2, 2, 16), (1, 2, 1), (2, 2, 1), (2, 1, 2), (4, 2, 1),
                                      (1, 1, 5), (7, 2, 1)])
def test_decode_attention_from_a_hand_built_cache(G, Hkv, ps):
    """Decode attention against its plain definition (softmax over exactly the rows the block table names), on a
    cache built by hand: scattered pages, lengths that end inside a page / inside a 128-token tile / at zero, and NaN
    in every row no token was written to (such rows must not leak into the result)."""
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(100 * G + ps)
    d, Hq = 128, G * Hkv
    lens = [0, 1, ps - 1, ps, 127, 128, 129, 300, 1000, 1537]
    S = len(lens)
    max_pages = (max(lens) + ps - 1) // ps + 1
    num_pages = sum((n + ps - 1) // ps for n in lens) + 5
    k_cache = torch.full((num_pages, ps, Hkv, d), float("nan"), dtype=torch.bfloat16)
    v_cache = torch.full((num_pages, ps, Hkv, d), float("nan"), dtype=torch.bfloat16)
    table = torch.zeros((S, max_pages), dtype=torch.int32)
    perm = rng.permutation(num_pages)
    nxt, rows = 0, []
    for s, n in enumerate(lens):
        kk = torch.from_numpy(rng.standard_normal((n, Hkv, d)).astype(np.float32)).to(torch.bfloat16)
        vv = torch.from_numpy(rng.standard_normal((n, Hkv, d)).astype(np.float32)).to(torch.bfloat16)
        rows.append((kk, vv))
        for pi in range((n + ps - 1) // ps):
            page = int(perm[nxt]); nxt += 1
            table[s, pi] = page
            m = min(ps, n - pi * ps)
            k_cache[page, :m] = kk[pi * ps: pi * ps + m]
            v_cache[page, :m] = vv[pi * ps: pi * ps + m]
    q = torch.from_numpy(rng.standard_normal((S, Hq, d)).astype(np.float32)).to(torch.bfloat16)
    n_tokens = torch.tensor(lens, dtype=torch.int32)
    cache = B.PagedCache(num_pages, ps, S, max_pages, Hkv, d)
    cache.k_cache.copy_(k_cache)
    cache.v_cache.copy_(v_cache)
    cache.block_table.copy_(table)
    cache.n_tokens.copy_(n_tokens)
    for splits in (1, 3):
        ws = torch.empty(int(B.load().kvs_decode_workspace_bytes(S, Hq, d, splits)), dtype=torch.uint8, device="cuda")
        out, lse = cache.decode(q.cuda(), num_splits=splits, workspace=ws)
        assert B.kvs_device_status(ws) == B.KVS_OK
        out, lse = out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
        scale = 1.0 / np.sqrt(d)
        for s, n in enumerate(lens):
            kk, vv = (t.float().numpy().astype(np.float64) for t in rows[s])
            for h in range(Hq):
                if n == 0:
                    assert np.all(out[s, h] == 0) and lse[s, h] == -np.inf
                    continue
                sc = kk[:, h // G] @ q[s, h].float().numpy().astype(np.float64) * scale
                mx = sc.max()
                w = np.exp(sc - mx)
                ref_o, ref_l = (w[:, None] * vv[:, h // G]).sum(0) / w.sum(), mx + np.log(w.sum())
                assert np.isfinite(out[s, h]).all(), (s, h, n)
                assert np.abs(out[s, h] - ref_o).max() < 2e-2 and abs(lse[s, h] - ref_l) < 2e-3, (splits, s, h, n)


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(12))
def test_decode_attention_fuzz(seed):
    """Seeded random shapes of the decode step against its plain definition: page size, group width, KV heads, head
    dimension, number of sequences, lengths (zero, one, ragged, several tiles), scattered pages with NaN in every row
    that holds no token, split count chosen by the library or forced."""
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(9000 + seed)
    d = 64 if seed % 6 == 5 else 128
    ps = int(rng.choice([1, 1, 2, 3, 4, 8, 16, 16, 32, 64, 128]))
    G = int(rng.choice([1, 2, 4, 7, 8]))
    Hkv = int(rng.choice([1, 2, 3]))
    Hq = G * Hkv
    S = int(rng.integers(1, 7))
    lens = [int(x) for x in rng.choice([0, 1, ps, 127, 128, 129, 255, 640, 1500, 2900], size=S)]
    lens[int(rng.integers(0, S))] = int(rng.integers(1, 3000))
    max_pages = (max(lens) + ps - 1) // ps + 2
    num_pages = sum((n + ps - 1) // ps for n in lens) + 3
    k_cache = torch.full((num_pages, ps, Hkv, d), float("nan"), dtype=torch.bfloat16)
    v_cache = torch.full((num_pages, ps, Hkv, d), float("nan"), dtype=torch.bfloat16)
    table = torch.zeros((S, max_pages), dtype=torch.int32)
    perm, nxt, rows = rng.permutation(num_pages), 0, []
    for s, n in enumerate(lens):
        kk = torch.from_numpy(rng.standard_normal((n, Hkv, d)).astype(np.float32)).to(torch.bfloat16)
        vv = torch.from_numpy(rng.standard_normal((n, Hkv, d)).astype(np.float32)).to(torch.bfloat16)
        rows.append((kk, vv))
        for pi in range((n + ps - 1) // ps):
            page = int(perm[nxt]); nxt += 1
            table[s, pi] = page
            m = min(ps, n - pi * ps)
            k_cache[page, :m] = kk[pi * ps: pi * ps + m]
            v_cache[page, :m] = vv[pi * ps: pi * ps + m]
    q = torch.from_numpy((rng.standard_normal((S, Hq, d)) * rng.choice([0.5, 1.0, 3.0])).astype(np.float32)).to(torch.bfloat16)
    cache = B.PagedCache(num_pages, ps, S, max_pages, Hkv, d)
    cache.k_cache.copy_(k_cache)
    cache.v_cache.copy_(v_cache)
    cache.block_table.copy_(table)
    cache.n_tokens.copy_(torch.tensor(lens, dtype=torch.int32))
    splits = int(rng.choice([0, 0, 1, 2, 5]))
    out, lse = cache.decode(q.cuda(), num_splits=splits, max_tokens=max(max(lens), 1))
    out, lse = out.float().cpu().numpy().astype(np.float64), lse.cpu().numpy().astype(np.float64)
    scale = 1.0 / np.sqrt(d)
    for s, n in enumerate(lens):
        kk, vv = (t.float().numpy().astype(np.float64) for t in rows[s])
        for h in range(Hq):
            if n == 0:
                assert np.all(out[s, h] == 0) and lse[s, h] == -np.inf
                continue
            sc = kk[:, h // G] @ q[s, h].float().numpy().astype(np.float64) * scale
            w = np.exp(sc - sc.max())
            ref_o, ref_l = (w[:, None] * vv[:, h // G]).sum(0) / w.sum(), sc.max() + np.log(w.sum())
            assert np.isfinite(out[s, h]).all(), (ps, G, s, h, n)
            assert np.abs(out[s, h] - ref_o).max() < 2e-2 and abs(lse[s, h] - ref_l) < 2e-3, (ps, G, Hkv, d, splits, s, h, n)


@pytest.mark.gpu
@pytest.mark.parametrize("ps", [16, 1])
def test_decode_step_replays_from_a_cuda_graph(ps):
    """Appending a token and attending over the live cache keep their state (token counts, block tables, free stack)
    on the device and take no host decision, so the pair can be captured once and replayed for every generated token,
    as rollout engines do; the results equal the eager calls token by token."""
    from paper_2609_35750_b200 import binding as B
    rng = np.random.default_rng(5 + ps)
    S, Hkv, G, d, T = 3, 2, 4, 128, 200
    Hq = G * Hkv
    num_pages, max_pages = S * ((T + ps - 1) // ps) + 2, (T + ps - 1) // ps + 1
    ks = torch.from_numpy(rng.standard_normal((T, S, Hkv, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    vs = torch.from_numpy(rng.standard_normal((T, S, Hkv, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    qs = torch.from_numpy(rng.standard_normal((T, S, Hq, d)).astype(np.float32)).to(torch.bfloat16).cuda()
    splits = 2

    def run(graphed):
        cache = B.PagedCache(num_pages, ps, S, max_pages, Hkv, d)
        q, k, v = torch.empty_like(qs[0]), torch.empty_like(ks[0]), torch.empty_like(vs[0])
        out, lse = torch.empty_like(q), torch.empty((S, Hq), dtype=torch.float32, device="cuda")
        ws = torch.empty(int(B.load().kvs_decode_workspace_bytes(S, Hq, d, splits)), dtype=torch.uint8, device="cuda")
        outs, lses = [], []

        def step():
            cache.append(k, v)
            cache.decode(q, num_splits=splits, out=out, lse=lse, workspace=ws)

        graph, first = None, 0
        if graphed:
            q.copy_(qs[0]); k.copy_(ks[0]); v.copy_(vs[0])
            step()                                      # token 0 eagerly (sets up function attributes), then capture
            outs.append(out.clone()); lses.append(lse.clone())
            first = 1
            torch.cuda.synchronize()
            graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
            with torch.cuda.stream(side):
                with torch.cuda.graph(graph, stream=side):
                    step()
            # the capture itself ran nothing: the cache still holds one token per sequence
            assert cache.n_tokens.cpu().tolist() == [1] * S
        for i in range(first, T):
            q.copy_(qs[i]); k.copy_(ks[i]); v.copy_(vs[i])
            if graphed:
                graph.replay()
            else:
                step()
            outs.append(out.clone()); lses.append(lse.clone())
        torch.cuda.synchronize()
        assert cache.status()[0] == B.KVS_OK and cache.n_tokens.cpu().tolist() == [T] * S
        return torch.stack(outs), torch.stack(lses)

    eo, el = run(False)
    go, gl = run(True)
    assert torch.equal(eo, go) and torch.equal(el, gl)
    # and the eager path is the definition: the last token against a plain softmax over all T keys
    kk, vv, qq = (t.float().cpu().numpy().astype(np.float64) for t in (ks, vs, qs))
    for s in range(S):
        for h in range(Hq):
            sc = kk[:, s, h // G] @ qq[T - 1, s, h] / np.sqrt(d)
            w = np.exp(sc - sc.max())
            ref = (w[:, None] * vv[:, s, h // G]).sum(0) / w.sum()
            assert np.abs(eo[T - 1, s, h].float().cpu().numpy() - ref).max() < 2e-2
