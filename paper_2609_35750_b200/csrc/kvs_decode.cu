// Rollout side: paged KV cache with physical eviction, and decode attention over the live cache.
//
// The inference engine of the method evicts KV entries directly in its paged cache (Sec. 1, Sec. 4
// "Inference engine implementation": 16-token blocks in one engine, with completions padded to
// block multiples (App. A.3); block size 1 in the other) and keeps decoding on the same stream.
// Here: a block table per sequence lists the pages of its LIVE cache in order; eviction removes
// whole pages from the table (the rows themselves never move) and returns them to a free list;
// appending a token takes a page from the free list when the last page is full; decode attention
// reads exactly the pages the table names.  It never sees a mask.
//
// Decode attention is bound by HBM (every live K and V row is read once per step), so the kernel
// is organised around coalesced 256-byte row reads, not around the tensor cores: one CTA per
// (split, KV head, sequence); each half-warp reads one K (or V) row per load instruction and
// serves all G query heads of the group from it; 16-token blocks get one softmax update each;
// partial results of the warps and of the splits are merged at the end.
#include "kvs_common.cuh"

namespace kvs {

constexpr int DEC_THREADS = 128;

struct DecodeParams {
    const __nv_bfloat16* q;          // [S, Hq, D]
    const __nv_bfloat16* k_cache;    // [num_pages, page_size, Hkv, D]
    const __nv_bfloat16* v_cache;
    const int32_t* block_table;      // [S, max_pages]
    const int32_t* n_tokens;         // [S]
    int S, Hq, Hkv, page_size, max_pages, nsplit;
    float scale_log2;
    float* part_o;                   // [S, Hq, nsplit, D] unnormalised
    float* part_ml;                  // [S, Hq, nsplit, 2]  (max in base-2 units, sum)
};

// 16 bytes (CH = 8) or 8 bytes (CH = 4) of a bf16 row, widened to fp32
template <int CH>
struct RowChunk {
    uint32_t w[CH / 2];
    __device__ __forceinline__ void load(const __nv_bfloat16* ptr) {
        if constexpr (CH == 8) {
            const uint4 raw = *reinterpret_cast<const uint4*>(ptr);
            w[0] = raw.x; w[1] = raw.y; w[2] = raw.z; w[3] = raw.w;
        } else {
            const uint2 raw = *reinterpret_cast<const uint2*>(ptr);
            w[0] = raw.x; w[1] = raw.y;
        }
    }
    __device__ __forceinline__ void widen(float (&f)[CH]) const {
#pragma unroll
        for (int e = 0; e < CH / 2; ++e) {
            f[2 * e] = __uint_as_float(w[e] << 16);               // low half: element 2e
            f[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);   // high half: element 2e+1
        }
    }
};

template <int D, int G>
__global__ void __launch_bounds__(DEC_THREADS, (G > 4) ? 2 : 3)
decode_partial_kernel(DecodeParams p) {
    constexpr int CH = D / 16;                  // elements of a row per lane (16 lanes per row): 8 or 4
    constexpr int ROWS = (G > 4) ? 4 : 8;       // rows per half-warp per block (register budget)
    constexpr int BLK = 2 * ROWS;               // tokens per softmax update
    const int z = blockIdx.x, g = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int half = lane >> 4, l16 = lane & 15;
    const int n = p.n_tokens[s];
    const int ps = p.page_size;
    const int nblocks = (n + BLK - 1) / BLK;
    // blocks of this split, dealt round-robin to (split, warp)
    const int stride = p.nsplit * (DEC_THREADS / 32);
    const int first = z * (DEC_THREADS / 32) + warp;

    // q of the G heads: this lane's CH elements of each head, in fp32, pre-scaled
    float qv[G][CH];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        RowChunk<CH> c;
        c.load(p.q + ((size_t)s * p.Hq + g * G + h) * D + l16 * CH);
        c.widen(qv[h]);
#pragma unroll
        for (int e = 0; e < CH; ++e) qv[h][e] *= p.scale_log2;
    }
    float m_run[G], l_run[G], acc[G][CH];
#pragma unroll
    for (int h = 0; h < G; ++h) {
        m_run[h] = -INFINITY;
        l_run[h] = 0.f;
#pragma unroll
        for (int e = 0; e < CH; ++e) acc[h][e] = 0.f;
    }
    const int32_t* bt = p.block_table + (size_t)s * p.max_pages;
    const size_t row_stride = (size_t)p.Hkv * D;             // elements between tokens of a page
    const size_t lane_off = (size_t)g * D + l16 * CH;

    for (int b = first; b < nblocks; b += stride) {
        const int t0 = b * BLK;
        // row index (page * page_size + offset) of token t0 + l16, fetched once per block by every lane;
        // tokens past the end are clamped to the last one (their scores are discarded below)
        const int tl = min(t0 + (l16 & (BLK - 1)), n - 1);
        const int my_row = bt[tl / ps] * ps + tl % ps;
        // ---- all K rows of the block in flight, then the scores ----
        RowChunk<CH> raw[ROWS];
        int rowi[ROWS];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            rowi[r] = __shfl_sync(0xffffffffu, my_row, 2 * r + half);
            raw[r].load(p.k_cache + (size_t)rowi[r] * row_stride + lane_off);
        }
        float sc[ROWS][G];
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float kf[CH];
            raw[r].widen(kf);
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float v = 0.f;
#pragma unroll
                for (int e = 0; e < CH; ++e) v = fmaf(qv[h][e], kf[e], v);
                sc[r][h] = v;
            }
        }
        // ---- the V rows go in flight while the scores are reduced and exponentiated ----
#pragma unroll
        for (int r = 0; r < ROWS; ++r) raw[r].load(p.v_cache + (size_t)rowi[r] * row_stride + lane_off);
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            const bool ok = (t0 + 2 * r + half) < n;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float v = sc[r][h];
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);      // within the 16 lanes of the row
                sc[r][h] = ok ? v : -INFINITY;
            }
        }
        // one softmax update per head for the ROWS tokens of this half-warp
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float bm = sc[0][h];
#pragma unroll
            for (int r = 1; r < ROWS; ++r) bm = fmaxf(bm, sc[r][h]);
            const float m_new = fmaxf(m_run[h], bm);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = fast_exp2(m_run[h] - m_use);
            float sum = 0.f;
#pragma unroll
            for (int r = 0; r < ROWS; ++r) {
                sc[r][h] = fast_exp2(sc[r][h] - m_use);       // the score becomes the weight, in place
                sum += sc[r][h];
            }
            l_run[h] = l_run[h] * alpha + sum;
            m_run[h] = m_new;
#pragma unroll
            for (int e = 0; e < CH; ++e) acc[h][e] *= alpha;
        }
        // ---- acc += p * v (a token past the end has weight 0) ----
#pragma unroll
        for (int r = 0; r < ROWS; ++r) {
            float vf[CH];
            raw[r].widen(vf);
#pragma unroll
            for (int h = 0; h < G; ++h)
#pragma unroll
                for (int e = 0; e < CH; ++e) acc[h][e] = fmaf(sc[r][h], vf[e], acc[h][e]);
        }
    }

    // ---- merge the 8 half-warp states of the CTA through shared memory ----
    __shared__ float s_m[8][G], s_l[8][G];
    __shared__ float s_o[8][G][D];
    const int slot = warp * 2 + half;
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (l16 == 0) {
            s_m[slot][h] = m_run[h];
            s_l[slot][h] = l_run[h];
        }
#pragma unroll
        for (int e = 0; e < CH; ++e) s_o[slot][h][l16 * CH + e] = acc[h][e];
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += DEC_THREADS) {
        const int h = idx / D, c = idx % D;
        float M = -INFINITY;
#pragma unroll
        for (int k = 0; k < 8; ++k) M = fmaxf(M, s_m[k][h]);
        const float Mu = (M == -INFINITY) ? 0.f : M;
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const float w = fast_exp2(s_m[k][h] - Mu);
            L += s_l[k][h] * w;
            o += s_o[k][h][c] * w;
        }
        const size_t base = ((size_t)s * p.Hq + g * G + h) * p.nsplit + z;
        p.part_o[base * D + c] = o;
        if (c == 0) {
            p.part_ml[base * 2 + 0] = M;
            p.part_ml[base * 2 + 1] = L;
        }
    }
}

// one warp per (sequence, query head): merge the splits, normalise, write bf16 out and fp32 lse
template <int D>
__global__ void decode_combine_kernel(const float* __restrict__ part_o, const float* __restrict__ part_ml, int rows, int nsplit,
                                      __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int row = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (row >= rows) return;
    constexpr int PER = D / 32;
    float M = -INFINITY;
    for (int z = 0; z < nsplit; ++z) M = fmaxf(M, part_ml[((size_t)row * nsplit + z) * 2]);
    const float Mu = (M == -INFINITY) ? 0.f : M;
    float L = 0.f, o[PER];
#pragma unroll
    for (int e = 0; e < PER; ++e) o[e] = 0.f;
    for (int z = 0; z < nsplit; ++z) {
        const size_t base = (size_t)row * nsplit + z;
        const float w = fast_exp2(part_ml[base * 2] - Mu);
        L += part_ml[base * 2 + 1] * w;
#pragma unroll
        for (int e = 0; e < PER; ++e) o[e] += part_o[base * D + lane * PER + e] * w;
    }
    const float inv = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
    for (int e = 0; e < PER; ++e) out[(size_t)row * D + lane * PER + e] = __float2bfloat16(o[e] * inv);
    if (lane == 0) lse[row] = (L > 0.f) ? M * 0.6931471805599453f + logf(L) : -INFINITY;
}

// ---- cache maintenance ---------------------------------------------------------------------------
struct CacheHeader {            // the first 16 bytes of the free-list buffer
    int32_t top;                // number of free pages on the stack
    int32_t status;             // KVS_OK or an error recorded by a kernel
    int32_t pad[2];
};

__global__ void cache_init_kernel(int32_t* free_buf, int num_pages) {
    CacheHeader* hdr = reinterpret_cast<CacheHeader*>(free_buf);
    int32_t* stack = free_buf + 4;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        hdr->top = num_pages;
        hdr->status = KVS_OK;
    }
    if (i < num_pages) stack[i] = num_pages - 1 - i;       // page 0 is handed out first
}

// one thread per sequence: take a page when the last one is full, write the token's K and V rows
__global__ void cache_append_kernel(const __nv_bfloat16* __restrict__ k_new, const __nv_bfloat16* __restrict__ v_new,
                                    const uint8_t* __restrict__ active, int S, int Hkv, int D, int page_size, int max_pages,
                                    int32_t* block_table, int32_t* n_tokens, int32_t* free_buf, __nv_bfloat16* k_cache,
                                    __nv_bfloat16* v_cache) {
    CacheHeader* hdr = reinterpret_cast<CacheHeader*>(free_buf);
    int32_t* stack = free_buf + 4;
    const int s = blockIdx.x;
    if (s >= S || (active && !active[s])) return;
    __shared__ int s_page;
    const int slot = n_tokens[s];
    if (threadIdx.x == 0) {
        int page = -1;
        if (slot % page_size == 0) {
            if (slot / page_size >= max_pages) {
                atomicCAS(&hdr->status, 0, KVS_ERR_WORKSPACE);
            } else {
                const int top = atomicSub(&hdr->top, 1);
                if (top <= 0) {
                    atomicAdd(&hdr->top, 1);
                    atomicCAS(&hdr->status, 0, KVS_ERR_WORKSPACE);       // cache full
                } else {
                    page = stack[top - 1];
                    block_table[(size_t)s * max_pages + slot / page_size] = page;
                }
            }
        } else {
            page = block_table[(size_t)s * max_pages + slot / page_size];
        }
        s_page = page;
    }
    __syncthreads();
    const int page = s_page;
    if (page < 0) return;
    const size_t dst = ((size_t)page * page_size + slot % page_size) * Hkv * D;
    const size_t src = (size_t)s * Hkv * D;
    for (int i = threadIdx.x; i < Hkv * D; i += blockDim.x) {
        k_cache[dst + i] = k_new[src + i];
        v_cache[dst + i] = v_new[src + i];
    }
    __syncthreads();
    if (threadIdx.x == 0) n_tokens[s] = slot + 1;
}

// one CTA per sequence: remove the pages [first_page, first_page + n_pages) of every listed range from the
// block table (stable compaction of the table; the rows never move) and push them on the free list
__global__ void cache_evict_kernel(const int32_t* __restrict__ ranges, int n_ranges, int S, int page_size, int max_pages,
                                   int32_t* block_table, int32_t* n_tokens, int32_t* free_buf) {
    CacheHeader* hdr = reinterpret_cast<CacheHeader*>(free_buf);
    int32_t* stack = free_buf + 4;
    const int s = blockIdx.x;
    if (s >= S) return;
    extern __shared__ int32_t sh[];              // keep flags / new positions, max_pages entries
    __shared__ int s_base, s_bad;
    const int n = n_tokens[s];
    const int npages = (n + page_size - 1) / page_size;
    int32_t* bt = block_table + (size_t)s * max_pages;
    for (int i = threadIdx.x; i < npages; i += blockDim.x) sh[i] = 1;
    if (threadIdx.x == 0) s_bad = 0;
    __syncthreads();
    for (int r = 0; r < n_ranges; ++r) {
        if (ranges[3 * r] != s) continue;
        const int a = ranges[3 * r + 1], cnt = ranges[3 * r + 2];
        // only whole pages can leave: a range must lie inside the table and must not touch a partial last page
        if (a < 0 || cnt < 0 || a + cnt > npages || (a + cnt == npages && cnt > 0 && n % page_size != 0)) {
            if (threadIdx.x == 0) s_bad = 1;
            continue;
        }
        for (int i = a + threadIdx.x; i < a + cnt; i += blockDim.x) sh[i] = 0;
    }
    __syncthreads();
    if (s_bad) {
        if (threadIdx.x == 0) atomicCAS(&hdr->status, 0, KVS_ERR_INVALID_ARG);
        return;
    }
    // stable compaction by one warp (tables are short: a few thousand pages at most)
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        int kept = 0, freed = 0;
        // pass 1: count the freed pages to reserve room on the free stack
        for (int i0 = 0; i0 < npages; i0 += 32) {
            const int i = i0 + lane;
            const unsigned gone = __ballot_sync(0xffffffffu, i < npages && sh[i] == 0);
            freed += __popc(gone);
        }
        if (lane == 0) s_base = atomicAdd(&hdr->top, freed);
        __syncwarp();
        const int base = s_base;
        int fpos = 0;
        for (int i0 = 0; i0 < npages; i0 += 32) {
            const int i = i0 + lane;
            const bool valid = i < npages;
            const int page = valid ? bt[i] : -1;
            const bool keep = valid && sh[i] != 0;
            const unsigned km = __ballot_sync(0xffffffffu, keep);
            const unsigned gm = __ballot_sync(0xffffffffu, valid && !keep);
            const unsigned lt = (1u << lane) - 1u;
            __syncwarp();
            if (keep) bt[kept + __popc(km & lt)] = page;          // kept + rank <= i: never ahead of the reads of this round
            else if (valid) stack[base + fpos + __popc(gm & lt)] = page;
            kept += __popc(km);
            fpos += __popc(gm);
            __syncwarp();
        }
        if (lane == 0) n_tokens[s] = n - freed * page_size;
    }
}

}  // namespace kvs

using namespace kvs;

extern "C" size_t kvs_cache_free_list_bytes(int num_pages) {
    if (num_pages < 0) return 0;
    return sizeof(int32_t) * (4 + (size_t)num_pages);
}

extern "C" int kvs_cache_init(int32_t* free_list, int num_pages, kvs_stream_t stream) {
    if (!free_list || num_pages < 0) return KVS_ERR_INVALID_ARG;
    cache_init_kernel<<<(num_pages + 256) / 256, 256, 0, (cudaStream_t)stream>>>(free_list, num_pages);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_cache_status(const int32_t* free_list, int* free_pages_host, kvs_stream_t stream) {
    if (!free_list) return KVS_ERR_INVALID_ARG;
    int32_t h[2] = {0, 0};
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(h, free_list, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    if (free_pages_host) *free_pages_host = h[0];
    return h[1];
}

extern "C" int kvs_cache_append(const void* k_new, const void* v_new, const uint8_t* active, int num_seqs, int Hkv, int head_dim,
                                int page_size, int max_pages, int32_t* block_table, int32_t* n_tokens, int32_t* free_list,
                                void* k_cache, void* v_cache, kvs_stream_t stream) {
    if (!k_new || !v_new || !block_table || !n_tokens || !free_list || !k_cache || !v_cache) return KVS_ERR_INVALID_ARG;
    if (num_seqs < 0 || Hkv <= 0 || head_dim <= 0 || page_size <= 0 || max_pages <= 0) return KVS_ERR_INVALID_ARG;
    if (num_seqs == 0) return KVS_OK;
    cache_append_kernel<<<num_seqs, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, active,
                                                                   num_seqs, Hkv, head_dim, page_size, max_pages, block_table,
                                                                   n_tokens, free_list, (__nv_bfloat16*)k_cache,
                                                                   (__nv_bfloat16*)v_cache);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_cache_evict(const int32_t* ranges, int n_ranges, int num_seqs, int page_size, int max_pages, int32_t* block_table,
                               int32_t* n_tokens, int32_t* free_list, kvs_stream_t stream) {
    if (!block_table || !n_tokens || !free_list || n_ranges < 0 || num_seqs < 0 || page_size <= 0 || max_pages <= 0)
        return KVS_ERR_INVALID_ARG;
    if (n_ranges > 0 && !ranges) return KVS_ERR_INVALID_ARG;
    if ((size_t)max_pages * sizeof(int32_t) > 200 * 1024) return KVS_ERR_UNSUPPORTED;
    if (n_ranges == 0 || num_seqs == 0) return KVS_OK;
    const size_t smem = (size_t)max_pages * sizeof(int32_t);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(cache_evict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return KVS_ERR_CUDA;
    cache_evict_kernel<<<num_seqs, 256, smem, (cudaStream_t)stream>>>(ranges, n_ranges, num_seqs, page_size, max_pages, block_table,
                                                                     n_tokens, free_list);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_decode_num_splits(int num_seqs, int Hkv, int max_tokens) {
    if (num_seqs <= 0 || Hkv <= 0 || max_tokens <= 0) return 1;
    // enough CTAs for two waves at three resident CTAs per SM (148 SMs), but at least 4 blocks of 16
    // tokens per warp of a split
    long long want = (2 * 3 * 148 + (long long)num_seqs * Hkv - 1) / ((long long)num_seqs * Hkv);
    long long cap = ((long long)max_tokens + 16 * 4 * 4 - 1) / (16 * 4 * 4);
    long long n = want < cap ? want : cap;
    if (n < 1) n = 1;
    if (n > 64) n = 64;
    return (int)n;
}

extern "C" size_t kvs_decode_workspace_bytes(int num_seqs, int Hq, int head_dim, int num_splits) {
    if (num_seqs < 0 || Hq <= 0 || head_dim <= 0 || num_splits <= 0) return 0;
    return align_up(sizeof(float) * (size_t)num_seqs * Hq * num_splits * (head_dim + 2), 256);
}

template <int D>
static int launch_decode(const DecodeParams& p, int G, void* out, float* lse, cudaStream_t st) {
    dim3 grid(p.nsplit, p.Hkv, p.S);
    switch (G) {
        case 1: decode_partial_kernel<D, 1><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 2: decode_partial_kernel<D, 2><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 4: decode_partial_kernel<D, 4><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 7: decode_partial_kernel<D, 7><<<grid, DEC_THREADS, 0, st>>>(p); break;
        case 8: decode_partial_kernel<D, 8><<<grid, DEC_THREADS, 0, st>>>(p); break;
        default: return KVS_ERR_UNSUPPORTED;
    }
    const int rows = p.S * p.Hq;
    decode_combine_kernel<D><<<(rows * 32 + 255) / 256, 256, 0, st>>>(p.part_o, p.part_ml, rows, p.nsplit, (__nv_bfloat16*)out, lse);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_decode_attn(const void* q, const void* k_cache, const void* v_cache, const int32_t* block_table,
                               const int32_t* n_tokens, int num_seqs, int Hq, int Hkv, int head_dim, int page_size, int max_pages,
                               float softmax_scale, int num_splits, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               kvs_stream_t stream) {
    if (num_seqs < 0 || Hq <= 0 || Hkv <= 0 || page_size <= 0 || max_pages <= 0 || num_splits <= 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || num_seqs > 65535 || Hkv > 65535) return KVS_ERR_UNSUPPORTED;
    if (num_seqs == 0) return KVS_OK;
    if (!q || !k_cache || !v_cache || !block_table || !n_tokens || !out || !lse || !workspace) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)q | (uintptr_t)k_cache | (uintptr_t)v_cache | (uintptr_t)out) & 15) != 0 || ((uintptr_t)workspace & 255) != 0)
        return KVS_ERR_ALIGNMENT;
    if (workspace_bytes < kvs_decode_workspace_bytes(num_seqs, Hq, head_dim, num_splits)) return KVS_ERR_WORKSPACE;
    if (softmax_scale < 0.f || softmax_scale != softmax_scale) return KVS_ERR_INVALID_ARG;
    DecodeParams p;
    p.q = (const __nv_bfloat16*)q;
    p.k_cache = (const __nv_bfloat16*)k_cache;
    p.v_cache = (const __nv_bfloat16*)v_cache;
    p.block_table = block_table;
    p.n_tokens = n_tokens;
    p.S = num_seqs;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.page_size = page_size;
    p.max_pages = max_pages;
    p.nsplit = num_splits;
    const float s = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = s * 1.4426950408889634f;
    p.part_o = (float*)workspace;
    p.part_ml = p.part_o + (size_t)num_seqs * Hq * num_splits * head_dim;
    cudaStream_t st = (cudaStream_t)stream;
    return head_dim == 64 ? launch_decode<64>(p, Hq / Hkv, out, lse, st) : launch_decode<128>(p, Hq / Hkv, out, lse, st);
}
