// Mask metadata: per key block min/max of evict_at, per-tile class, per-row lists.
// Integer work only.  Three small kernels on the caller's stream, no host synchronisation.
#include "kvs_common.cuh"

namespace kvs {

// ---- kernel 0: header, per-trace offsets, block -> trace table -----------------------------
__global__ void meta_prefix_kernel(const int32_t* __restrict__ cu_seqlens, int batch, int total_tokens, int max_seqlen, int general,
                                   MetaHeader* hdr, int32_t* blk_off, uint32_t* cls_off, int32_t* seq_start,
                                   int32_t* blk_trace, int nb_cap, unsigned long long cls_cap) {
    __shared__ int s_bad;
    if (threadIdx.x == 0) {
        int bad = 0;
        long long nblk = 0;
        unsigned long long ncls = 0;
        if (cu_seqlens[0] != 0 || cu_seqlens[batch] != total_tokens) bad = 1;
        for (int b = 0; b < batch; ++b) {
            long long a = cu_seqlens[b], e = cu_seqlens[b + 1];
            long long T = e - a;
            if (T < 0 || T > max_seqlen || a < 0 || e > total_tokens) { bad = 1; T = 0; }
            long long nb = (T + TILE - 1) / TILE;
            blk_off[b] = (int32_t)nblk;
            cls_off[b] = (uint32_t)ncls;
            seq_start[b] = (int32_t)a;
            nblk += nb;
            ncls += (unsigned long long)(nb * nb);
            if (nblk > nb_cap || ncls > cls_cap) { bad = 1; nblk = 0; ncls = 0; break; }
        }
        if (bad) { nblk = 0; ncls = 0; }
        blk_off[batch] = (int32_t)nblk;
        cls_off[batch] = (uint32_t)ncls;
        seq_start[batch] = total_tokens;
        hdr->magic = META_MAGIC;
        hdr->status = bad ? KVS_ERR_BAD_EVICT : KVS_OK;
        hdr->batch = batch;
        hdr->total_tokens = total_tokens;
        hdr->max_seqlen = max_seqlen;
        hdr->nblk_total = (int32_t)nblk;
        hdr->ncls_total = (uint32_t)ncls;
        hdr->general = general;
        s_bad = bad;
    }
    __syncthreads();
    if (s_bad) return;
    for (int b = 0; b < batch; ++b) {
        int lo = blk_off[b], hi = blk_off[b + 1];
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) blk_trace[i] = b;
    }
}

// ---- kernel 1: one warp per key block: min / max over its key slots, validity ---------------
// Slot j of a trace holds a key that query i may read iff first[j] <= i < evict[j].  Plain metadata
// (key_first == nullptr): first[j] = j and evict[j] > j is required.  General metadata: both arrays come
// from the caller (keys re-ordered, or another visibility rule) and a slot may be visible to nobody.
// complement != 0: the slots of the EVICTED keys: slot j becomes visible at evict_at[j] and stays (first = evict_at,
// evict = never), i.e. the causal key set minus what the eviction mask still shows.
__global__ void meta_minmax_kernel(const int32_t* __restrict__ evict_at, const int32_t* __restrict__ key_first, int complement,
                                   MetaHeader* hdr,
                                   const int32_t* __restrict__ blk_off, const int32_t* __restrict__ seq_start,
                                   const int32_t* __restrict__ blk_trace, int32_t* kmin, int32_t* kmax, int32_t* fmin, int32_t* fmax,
                                   int32_t* col_first, int32_t* col_last, int32_t* evict_copy, int32_t* first_copy) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= hdr->nblk_total) return;
    const int b = blk_trace[warp];
    const int n = warp - blk_off[b];
    const int tok0 = seq_start[b];
    const int T = seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    int mn = INT32_MAX, mx = INT32_MIN, fmn = INT32_MAX, fmx = INT32_MIN;
    bool bad = false;
#pragma unroll
    for (int t = 0; t < TILE / 32; ++t) {
        const int j = n * TILE + t * 32 + lane;
        if (j < T) {
            const int e = complement ? INT32_MAX : evict_at[tok0 + j];
            const int f = complement ? evict_at[tok0 + j] : (key_first ? key_first[tok0 + j] : j);
            const bool general = complement || key_first;
            evict_copy[tok0 + j] = e;
            if (general) first_copy[tok0 + j] = f;
            bad |= general ? (f < 0) : (e <= j);
            mn = min(mn, e);
            mx = max(mx, e);
            fmn = min(fmn, f);
            fmx = max(fmx, f);
        }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    fmn = __reduce_min_sync(0xffffffffu, fmn);
    fmx = __reduce_max_sync(0xffffffffu, fmx);
    const unsigned any_bad = __ballot_sync(0xffffffffu, bad);
    if (lane == 0) {
        kmin[warp] = mn;
        kmax[warp] = mx;
        fmin[warp] = fmn;
        fmax[warp] = fmx;
        // last query block whose first row q0 = 128 m is still below kmax; first one whose last row reaches fmin
        long long last = ((long long)mx - 1) / TILE;
        if (last > nb - 1) last = nb - 1;
        long long first = fmn / TILE;
        if (first > nb) first = nb;
        if (first < 0) first = 0;                  // a negative key_first is reported below; never an index
        if (!key_first && !complement && last < n) last = n;
        col_first[warp] = (int32_t)first;
        col_last[warp] = (mx <= 0) ? -1 : (int32_t)last;
        if (any_bad) set_status(&hdr->status, KVS_ERR_BAD_EVICT);
    }
}

// ---- kernel 2: one warp per query block row: classes and the compact non-empty list --------
__global__ void meta_classify_kernel(MetaHeader* hdr, const int32_t* __restrict__ blk_off, const uint32_t* __restrict__ cls_off,
                                     const int32_t* __restrict__ seq_start, const int32_t* __restrict__ blk_trace,
                                     const int32_t* __restrict__ kmin, const int32_t* __restrict__ kmax,
                                     const int32_t* __restrict__ fmin, const int32_t* __restrict__ fmax,
                                     uint8_t* tile_class, uint16_t* row_list, int32_t* row_cnt) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= hdr->nblk_total) return;
    const int b = blk_trace[warp];
    const int base = blk_off[b];
    const int m = warp - base;
    const int T = seq_start[b + 1] - seq_start[b];
    const int nb = (T + TILE - 1) / TILE;
    const int q0 = m * TILE;
    const int q1 = min(q0 + TILE - 1, T - 1);
    uint8_t* cls_row = tile_class + cls_off[b] + (size_t)m * nb;
    uint16_t* list_row = row_list + cls_off[b] + (size_t)m * nb;
    int count = 0;
    for (int n0 = 0; n0 < nb; n0 += 32) {
        const int n = n0 + lane;
        int c = KVS_CLASS_EMPTY;
        if (n < nb) {
            // f0, f1: the earliest / latest "first query that may see the slot" of the block; for plain
            // metadata these are the block's first and last valid key, k0 and k1
            const int f0 = fmin[base + n], f1 = fmax[base + n];
            const int mn = kmin[base + n], mx = kmax[base + n];
            if (f0 > q1 || q0 >= mx) c = KVS_CLASS_EMPTY;
            else if (f1 <= q0 && q1 < mn) c = KVS_CLASS_FULL;
            else c = KVS_CLASS_PARTIAL;
            cls_row[n] = (uint8_t)c;
        }
        const unsigned live = __ballot_sync(0xffffffffu, c != KVS_CLASS_EMPTY);
        if (c != KVS_CLASS_EMPTY) list_row[count + __popc(live & ((1u << lane) - 1u))] = (uint16_t)n;
        count += __popc(live);
    }
    if (lane == 0) row_cnt[warp] = count;
}

// ---- kernel 3: work orders, heaviest first (bucket sort, one CTA per order) -------------------
// blockIdx.x = 0: query blocks by their number of non-empty key blocks (forward);
// blockIdx.x = 1: key blocks by the length of their query-block range (backward).
// Only the launch order of work depends on it; ties keep their order in the batch.
constexpr int ORDER_BINS = 4096;
__global__ void __launch_bounds__(1024)
meta_order_kernel(MetaHeader* hdr, const int32_t* __restrict__ row_cnt, const int32_t* __restrict__ col_first,
                  const int32_t* __restrict__ col_last, int32_t* fwd_order, int32_t* bwd_order) {
    __shared__ int bins[ORDER_BINS];
    __shared__ int warp_tot[32];
    const int n = hdr->nblk_total;
    const bool bwd = blockIdx.x == 1;
    int32_t* order = bwd ? bwd_order : fwd_order;
    auto key = [&](int i) {
        // coarse buckets (16 tiles): exact lengths would interleave blocks from all over the batch,
        // coarse ones keep runs of neighbouring blocks together while still starting the long ones first
        const int k = bwd ? (col_last[i] - col_first[i] + 1) : row_cnt[i];
        return min(max(k >> 4, 0), ORDER_BINS - 1);
    };
    for (int i = threadIdx.x; i < ORDER_BINS; i += blockDim.x) bins[i] = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) atomicAdd(&bins[key(i)], 1);
    __syncthreads();
    // exclusive scan over the bins in DESCENDING key order: thread t owns 4 consecutive reversed bins
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int c[4], sum = 0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        c[u] = bins[ORDER_BINS - 1 - (threadIdx.x * 4 + u)];
        sum += c[u];
    }
    int incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane], wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += t;
        }
        warp_tot[lane] = wi - w;     // exclusive prefix of the warp totals
    }
    __syncthreads();
    int run = warp_tot[warp] + incl - sum;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        bins[ORDER_BINS - 1 - (threadIdx.x * 4 + u)] = run;
        run += c[u];
    }
    __syncthreads();
    // Stable scatter by one warp, 32 blocks at a time in index order: blocks with equal keys keep their
    // order in the trace, so CTAs launched together work on neighbouring blocks and share tiles in L2.
    if (warp == 0) {
        for (int i0 = 0; i0 < n; i0 += 32) {
            const int i = i0 + lane;
            const int k = (i < n) ? key(i) : -1;
            const unsigned same = __match_any_sync(0xffffffffu, k);
            if (i < n) order[bins[k] + __popc(same & ((1u << lane) - 1u))] = i;
            __syncwarp();
            if (i < n && lane == (__ffs(same) - 1)) bins[k] += __popc(same);
            __syncwarp();
        }
    }
}

// ---- compaction event log -> evict_at ---------------------------------------------------------
__global__ void evict_fill_kernel(int32_t* evict_at, int total_tokens) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < total_tokens) evict_at[i] = INT32_MAX;
}

// one CTA per event: the earliest `when` wins for every key of the span
__global__ void evict_events_kernel(const int32_t* __restrict__ events, int n_events, const int32_t* __restrict__ cu_seqlens,
                                    int batch, int32_t* evict_at) {
    const int e = blockIdx.x;
    if (e >= n_events) return;
    const int b = events[4 * e + 0], when = events[4 * e + 1];
    if (b < 0 || b >= batch) return;
    const int tok0 = cu_seqlens[b];
    const int T = cu_seqlens[b + 1] - tok0;
    const int a = max(events[4 * e + 2], 0), z = min(events[4 * e + 3], T);
    for (int j = a + threadIdx.x; j < z; j += blockDim.x) atomicMin(&evict_at[tok0 + j], when);
}

}  // namespace kvs

using namespace kvs;

extern "C" int kvs_evict_at_from_events(const int32_t* events, int n_events, const int32_t* cu_seqlens, int batch, int total_tokens,
                                        int32_t* evict_at, kvs_stream_t stream) {
    if (n_events < 0 || batch < 0 || total_tokens < 0) return KVS_ERR_INVALID_ARG;
    if (total_tokens == 0) return KVS_OK;
    if (!evict_at || !cu_seqlens || (n_events > 0 && !events)) return KVS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    evict_fill_kernel<<<(total_tokens + 255) / 256, 256, 0, st>>>(evict_at, total_tokens);
    if (n_events > 0) evict_events_kernel<<<n_events, 256, 0, st>>>(events, n_events, cu_seqlens, batch, evict_at);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" size_t kvs_mask_meta_bytes(int batch, int total_tokens, int max_seqlen) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0) return 0;
    return meta_layout(batch, total_tokens, max_seqlen).total;
}

namespace {
int launch_mask_meta(const int32_t* key_evict, const int32_t* key_first, int complement, const int32_t* cu_seqlens, int batch,
                     int total_tokens, int max_seqlen, void* meta_buf, size_t meta_bytes, kvs_stream_t stream) {
    if (!cu_seqlens || !meta_buf || batch < 0 || total_tokens < 0 || max_seqlen < 0) return KVS_ERR_INVALID_ARG;
    if (total_tokens > 0 && !key_evict) return KVS_ERR_INVALID_ARG;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    if (((uintptr_t)meta_buf & 255) != 0) return KVS_ERR_ALIGNMENT;
    if (((uintptr_t)key_evict & 3) != 0 || ((uintptr_t)key_first & 3) != 0 || ((uintptr_t)cu_seqlens & 3) != 0) return KVS_ERR_ALIGNMENT;
    if ((long long)((max_seqlen + TILE - 1) / TILE) > 65535) return KVS_ERR_UNSUPPORTED;
    const MetaLayout L = meta_layout(batch, total_tokens, max_seqlen);
    if (L.cls_cap > 0xFFFFFFF0ull) return KVS_ERR_UNSUPPORTED;
    if (meta_bytes < L.total) return KVS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    MetaView v = meta_view(meta_buf, L);
    meta_prefix_kernel<<<1, 256, 0, st>>>(cu_seqlens, batch, total_tokens, max_seqlen, (key_first || complement) ? 1 : 0, v.hdr, (int32_t*)v.blk_off,
                                          (uint32_t*)v.cls_off, (int32_t*)v.seq_start, (int32_t*)v.blk_trace, L.nb_cap,
                                          (unsigned long long)L.cls_cap);
    const int warps_per_cta = 8;
    const int grid = (L.nb_cap + warps_per_cta - 1) / warps_per_cta;
    meta_minmax_kernel<<<grid, warps_per_cta * 32, 0, st>>>(key_evict, key_first, complement, v.hdr, v.blk_off, v.seq_start, v.blk_trace,
                                                            (int32_t*)v.kmin, (int32_t*)v.kmax, (int32_t*)v.fmin, (int32_t*)v.fmax,
                                                            (int32_t*)v.col_first, (int32_t*)v.col_last, (int32_t*)v.evict,
                                                            (int32_t*)v.kfirst);
    meta_classify_kernel<<<grid, warps_per_cta * 32, 0, st>>>(v.hdr, v.blk_off, v.cls_off, v.seq_start, v.blk_trace, v.kmin, v.kmax,
                                                              v.fmin, v.fmax, (uint8_t*)v.tile_class, (uint16_t*)v.row_list,
                                                              (int32_t*)v.row_cnt);
    meta_order_kernel<<<2, 1024, 0, st>>>(v.hdr, v.row_cnt, v.col_first, v.col_last, (int32_t*)v.fwd_order, (int32_t*)v.bwd_order);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}
}  // namespace

extern "C" int kvs_mask_meta(const int32_t* evict_at, const int32_t* cu_seqlens, int batch, int total_tokens, int max_seqlen,
                             void* meta_buf, size_t meta_bytes, kvs_stream_t stream) {
    return launch_mask_meta(evict_at, nullptr, 0, cu_seqlens, batch, total_tokens, max_seqlen, meta_buf, meta_bytes, stream);
}

extern "C" int kvs_mask_meta_keys(const int32_t* key_first, const int32_t* key_evict, const int32_t* cu_seqlens, int batch,
                                  int total_tokens, int max_seqlen, void* meta_buf, size_t meta_bytes, kvs_stream_t stream) {
    if (total_tokens > 0 && !key_first) return KVS_ERR_INVALID_ARG;
    return launch_mask_meta(key_evict, key_first, 0, cu_seqlens, batch, total_tokens, max_seqlen, meta_buf, meta_bytes, stream);
}

extern "C" int kvs_mask_meta_evicted(const int32_t* key_evict, const int32_t* cu_seqlens, int batch, int total_tokens, int max_seqlen,
                                     void* meta_buf, size_t meta_bytes, kvs_stream_t stream) {
    return launch_mask_meta(key_evict, nullptr, 1, cu_seqlens, batch, total_tokens, max_seqlen, meta_buf, meta_bytes, stream);
}

// ---- key re-ordering for token-level eviction ------------------------------------------------------
namespace kvs {
constexpr int REORDER_MAX_WINDOW = 4096;
// One CTA per (window, trace): the window's keys sorted by (eviction step, index) with a bitonic network in shared memory.
__global__ void __launch_bounds__(1024)
reorder_sort_kernel(const int32_t* __restrict__ evict_at, const int32_t* __restrict__ cu_seqlens, int window, int32_t* perm,
                    int32_t* key_first, int32_t* key_evict) {
    __shared__ unsigned long long keys[REORDER_MAX_WINDOW];
    const int b = blockIdx.y;
    const int tok0 = cu_seqlens[b];
    const int T = cu_seqlens[b + 1] - tok0;
    const int w0 = blockIdx.x * window;
    if (w0 >= T) return;
    const int n = min(window, T - w0);
    int cap = 1;
    while (cap < n) cap <<= 1;
    for (int i = threadIdx.x; i < cap; i += blockDim.x)
        keys[i] = (i < n) ? (((unsigned long long)(uint32_t)evict_at[tok0 + w0 + i] << 32) | (uint32_t)i) : ~0ull;
    __syncthreads();
    for (int k = 2; k <= cap; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = threadIdx.x; i < cap; i += blockDim.x) {
                const int l = i ^ j;
                if (l > i) {
                    const unsigned long long a = keys[i], c = keys[l];
                    const bool up = (i & k) == 0;
                    if ((a > c) == up) {
                        keys[i] = c;
                        keys[l] = a;
                    }
                }
            }
            __syncthreads();
        }
    }
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int src = w0 + (int)(uint32_t)keys[i];           // trace-local index of the key that lands in slot w0 + i
        perm[tok0 + w0 + i] = tok0 + src;
        key_first[tok0 + w0 + i] = src;
        key_evict[tok0 + w0 + i] = (int32_t)(keys[i] >> 32);
    }
}

// dst row r = src row perm[r] (inverse == 0) or dst row perm[r] = src row r (inverse != 0); 16 bytes per lane
__global__ void permute_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ perm, uint4* __restrict__ dst,
                                    long long n_rows, int row_vec, int inverse) {
    const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long r = idx / row_vec;
    const int c = (int)(idx % row_vec);
    if (r >= n_rows) return;
    const long long p = perm[r];
    if (inverse) dst[p * row_vec + c] = src[r * row_vec + c];
    else dst[r * row_vec + c] = src[p * row_vec + c];
}
}  // namespace kvs

extern "C" int kvs_reorder_keys(const int32_t* evict_at, const int32_t* cu_seqlens, int batch, int total_tokens, int max_seqlen,
                                int window, int32_t* perm, int32_t* key_first, int32_t* key_evict, kvs_stream_t stream) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0) return KVS_ERR_INVALID_ARG;
    if (window < 1 || window > REORDER_MAX_WINDOW) return KVS_ERR_UNSUPPORTED;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    if (!evict_at || !cu_seqlens || !perm || !key_first || !key_evict) return KVS_ERR_INVALID_ARG;
    if (batch > 65535) return KVS_ERR_UNSUPPORTED;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    const int nwin = (max_seqlen + window - 1) / window;
    dim3 grid(nwin > 0 ? nwin : 1, batch, 1);
    reorder_sort_kernel<<<grid, 1024, 0, (cudaStream_t)stream>>>(evict_at, cu_seqlens, window, perm, key_first, key_evict);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_permute_rows(const void* src, const int32_t* perm, void* dst, long long n_rows, long long row_bytes, int inverse,
                                kvs_stream_t stream) {
    if (n_rows < 0 || row_bytes <= 0 || row_bytes % 16 != 0 || row_bytes / 16 > 0x7fffffffLL) return KVS_ERR_INVALID_ARG;
    if (n_rows == 0) return KVS_OK;
    if (!src || !perm || !dst || src == dst) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)src | (uintptr_t)dst) & 15) != 0 || ((uintptr_t)perm & 3) != 0) return KVS_ERR_ALIGNMENT;
    const int row_vec = (int)(row_bytes / 16);
    const long long total = n_rows * row_vec;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
    permute_rows_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((const uint4*)src, perm, (uint4*)dst, n_rows, row_vec, inverse);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_mask_meta_export(const void* meta_buf, int batch, const int32_t* cu_seqlens_host, int total_tokens,
                                    int max_seqlen, uint8_t* tile_class_host, int32_t* kmin_host, int32_t* kmax_host,
                                    kvs_stream_t stream) {
    if (!meta_buf || !cu_seqlens_host || batch < 0) return KVS_ERR_INVALID_ARG;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    const MetaLayout L = meta_layout(batch, total_tokens, max_seqlen);
    cudaStream_t st = (cudaStream_t)stream;
    size_t nblk = 0, ncls = 0;
    for (int b = 0; b < batch; ++b) {
        long long T = (long long)cu_seqlens_host[b + 1] - cu_seqlens_host[b];
        if (T < 0 || T > max_seqlen) return KVS_ERR_INVALID_ARG;
        size_t nb = (size_t)((T + TILE - 1) / TILE);
        nblk += nb;
        ncls += nb * nb;
    }
    if (nblk > (size_t)L.nb_cap || ncls > L.cls_cap) return KVS_ERR_INVALID_ARG;
    MetaHeader h;
    const char* p = (const char*)meta_buf;
    if (cudaMemcpyAsync(&h, p, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (tile_class_host && ncls)
        if (cudaMemcpyAsync(tile_class_host, p + L.tile_class, ncls, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (kmin_host && nblk)
        if (cudaMemcpyAsync(kmin_host, p + L.kmin, nblk * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (kmax_host && nblk)
        if (cudaMemcpyAsync(kmax_host, p + L.kmax, nblk * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    if (h.magic != META_MAGIC || h.batch != batch || h.total_tokens != total_tokens || h.max_seqlen != max_seqlen) return KVS_ERR_BAD_META;
    if (h.status != KVS_OK) return h.status;
    if ((size_t)h.nblk_total != nblk || (size_t)h.ncls_total != ncls) return KVS_ERR_BAD_META;
    return KVS_OK;
}
