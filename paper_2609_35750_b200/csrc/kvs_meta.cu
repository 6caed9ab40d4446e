// Mask metadata: per key block min/max of evict_at, per-tile class, per-row lists.
// Integer work only.  Three small kernels on the caller's stream, no host synchronisation.
#include "kvs_common.cuh"

namespace kvs {

// ---- kernel 0: header, per-trace offsets, block -> trace table -----------------------------
__global__ void meta_prefix_kernel(const int32_t* __restrict__ cu_seqlens, int batch, int total_tokens, int max_seqlen,
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
        hdr->pad = 0;
        s_bad = bad;
    }
    __syncthreads();
    if (s_bad) return;
    for (int b = 0; b < batch; ++b) {
        int lo = blk_off[b], hi = blk_off[b + 1];
        for (int i = lo + threadIdx.x; i < hi; i += blockDim.x) blk_trace[i] = b;
    }
}

// ---- kernel 1: one warp per key block: min / max of evict_at, validity ---------------------
__global__ void meta_minmax_kernel(const int32_t* __restrict__ evict_at, MetaHeader* hdr, const int32_t* __restrict__ blk_off,
                                   const int32_t* __restrict__ seq_start, const int32_t* __restrict__ blk_trace,
                                   int32_t* kmin, int32_t* kmax, int32_t* col_last, int32_t* evict_copy) {
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= hdr->nblk_total) return;
    const int b = blk_trace[warp];
    const int n = warp - blk_off[b];
    const int tok0 = seq_start[b];
    const int T = seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    int mn = INT32_MAX, mx = INT32_MIN;
    bool bad = false;
#pragma unroll
    for (int t = 0; t < TILE / 32; ++t) {
        const int j = n * TILE + t * 32 + lane;
        if (j < T) {
            const int e = evict_at[tok0 + j];
            evict_copy[tok0 + j] = e;
            bad |= (e <= j);
            mn = min(mn, e);
            mx = max(mx, e);
        }
    }
    mn = __reduce_min_sync(0xffffffffu, mn);
    mx = __reduce_max_sync(0xffffffffu, mx);
    const unsigned any_bad = __ballot_sync(0xffffffffu, bad);
    if (lane == 0) {
        kmin[warp] = mn;
        kmax[warp] = mx;
        // last query block whose first row q0 = 128 m is still below kmax
        long long last = ((long long)mx - 1) / TILE;
        if (last > nb - 1) last = nb - 1;
        if (last < n) last = n;
        col_last[warp] = (int32_t)last;
        if (any_bad) set_status(&hdr->status, KVS_ERR_BAD_EVICT);
    }
}

// ---- kernel 2: one warp per query block row: classes and the compact non-empty list --------
__global__ void meta_classify_kernel(MetaHeader* hdr, const int32_t* __restrict__ blk_off, const uint32_t* __restrict__ cls_off,
                                     const int32_t* __restrict__ seq_start, const int32_t* __restrict__ blk_trace,
                                     const int32_t* __restrict__ kmin, const int32_t* __restrict__ kmax,
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
            const int k0 = n * TILE;
            const int k1 = min(k0 + TILE - 1, T - 1);
            const int mn = kmin[base + n], mx = kmax[base + n];
            if (k0 > q1 || q0 >= mx) c = KVS_CLASS_EMPTY;
            else if (k1 <= q0 && q1 < mn) c = KVS_CLASS_FULL;
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
meta_order_kernel(MetaHeader* hdr, const int32_t* __restrict__ blk_off, const int32_t* __restrict__ blk_trace,
                  const int32_t* __restrict__ row_cnt, const int32_t* __restrict__ col_last, int32_t* fwd_order,
                  int32_t* bwd_order) {
    __shared__ int bins[ORDER_BINS];
    __shared__ int warp_tot[32];
    const int n = hdr->nblk_total;
    const bool bwd = blockIdx.x == 1;
    int32_t* order = bwd ? bwd_order : fwd_order;
    auto key = [&](int i) {
        // coarse buckets (16 tiles): exact lengths would interleave blocks from all over the batch,
        // coarse ones keep runs of neighbouring blocks together while still starting the long ones first
        const int k = bwd ? (col_last[i] - (i - blk_off[blk_trace[i]]) + 1) : row_cnt[i];
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

extern "C" int kvs_mask_meta(const int32_t* evict_at, const int32_t* cu_seqlens, int batch, int total_tokens, int max_seqlen,
                             void* meta_buf, size_t meta_bytes, kvs_stream_t stream) {
    if (!cu_seqlens || !meta_buf || batch < 0 || total_tokens < 0 || max_seqlen < 0) return KVS_ERR_INVALID_ARG;
    if (total_tokens > 0 && !evict_at) return KVS_ERR_INVALID_ARG;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    if (((uintptr_t)meta_buf & 255) != 0) return KVS_ERR_ALIGNMENT;
    if (((uintptr_t)evict_at & 3) != 0 || ((uintptr_t)cu_seqlens & 3) != 0) return KVS_ERR_ALIGNMENT;
    if ((long long)((max_seqlen + TILE - 1) / TILE) > 65535) return KVS_ERR_UNSUPPORTED;
    const MetaLayout L = meta_layout(batch, total_tokens, max_seqlen);
    if (L.cls_cap > 0xFFFFFFF0ull) return KVS_ERR_UNSUPPORTED;
    if (meta_bytes < L.total) return KVS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    MetaView v = meta_view(meta_buf, L);
    meta_prefix_kernel<<<1, 256, 0, st>>>(cu_seqlens, batch, total_tokens, max_seqlen, v.hdr, (int32_t*)v.blk_off,
                                          (uint32_t*)v.cls_off, (int32_t*)v.seq_start, (int32_t*)v.blk_trace, L.nb_cap,
                                          (unsigned long long)L.cls_cap);
    const int warps_per_cta = 8;
    const int grid = (L.nb_cap + warps_per_cta - 1) / warps_per_cta;
    meta_minmax_kernel<<<grid, warps_per_cta * 32, 0, st>>>(evict_at, v.hdr, v.blk_off, v.seq_start, v.blk_trace, (int32_t*)v.kmin,
                                                            (int32_t*)v.kmax, (int32_t*)v.col_last, (int32_t*)v.evict);
    meta_classify_kernel<<<grid, warps_per_cta * 32, 0, st>>>(v.hdr, v.blk_off, v.cls_off, v.seq_start, v.blk_trace, v.kmin, v.kmax,
                                                              (uint8_t*)v.tile_class, (uint16_t*)v.row_list, (int32_t*)v.row_cnt);
    meta_order_kernel<<<2, 1024, 0, st>>>(v.hdr, v.blk_off, v.blk_trace, v.row_cnt, v.col_last, (int32_t*)v.fwd_order,
                                          (int32_t*)v.bwd_order);
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
    if (h.magic != META_MAGIC || h.batch != batch || h.total_tokens != total_tokens) return KVS_ERR_BAD_META;
    if (h.status != KVS_OK) return h.status;
    if ((size_t)h.nblk_total != nblk || (size_t)h.ncls_total != ncls) return KVS_ERR_BAD_META;
    return KVS_OK;
}
