// Rollout side: paged KV cache with physical eviction, and decode attention over the live cache.
//
// The inference engine of the method evicts KV entries directly in its paged cache (Sec. 1, Sec. 4
// "Inference engine implementation": 16-token blocks in one engine, with completions padded to
// block multiples (App. B.3); block size 1 in the other) and keeps decoding on the same stream.
// Here: a block table per sequence lists the pages of its LIVE cache in order; eviction removes
// whole pages from the table (the rows themselves never move) and returns them to a free list;
// appending a token takes a page from the free list when the last page is full; decode attention
// reads exactly the pages the table names.  It never sees a mask.
//
// Decode attention is bound by HBM (every live K and V row is read once per step).  Two kernels
// produce per-split partial results that a third merges:
//   decode_partial_kernel  CUDA cores, organised around coalesced 256-byte row reads: one CTA per
//                          (split, KV head, sequence); each half-warp reads one K (or V) row per load
//                          instruction and serves all G query heads of the group from it;
//   decode_tc_kernel       (head_dim 128) the same work with both products on the tensor core,
//                          because with a wide GQA group the CUDA-core kernel is bound by its
//                          arithmetic, not by the bytes, and because TMA keeps more bytes in flight
//                          than the load/store unit can.
#include "kvs_common.cuh"
#include <cstring>

namespace kvs {

constexpr int DEC_THREADS = 128;
constexpr size_t DEC_WS_HEADER = 256;

struct DecodeParams {
    const __nv_bfloat16* q;          // [S, Hq, D]
    const __nv_bfloat16* k_cache;    // [num_pages, page_size, Hkv, D]
    const __nv_bfloat16* v_cache;
    const int32_t* block_table;      // [S, max_pages]
    const int32_t* n_tokens;         // [S]
    int S, Hq, Hkv, page_size, max_pages, num_pages, nsplit;
    int page_shift;                  // log2(page_size) when it is a power of two, else -1
    int32_t* status;                 // workspace status word: a page id outside [0, num_pages) is recorded there
    float scale_log2;
    float* part_o;                   // [S, Hq, nsplit, D] unnormalised
    float* part_ml;                  // [S, Hq, nsplit, 2]  (max in base-2 units, sum)
};

// A block-table entry is only followed if it names a page of the cache: anything else (a stale or
// corrupt table) is recorded as KVS_ERR_INVALID_ARG and read as page 0, so no kernel reads outside the cache.
// token index -> (entry of the block table, row inside the page) without a division for power-of-two pages
__device__ __forceinline__ void split_token(const DecodeParams& p, int tok, int& entry, int& offset) {
    if (p.page_shift >= 0) {
        entry = tok >> p.page_shift;
        offset = tok & (p.page_size - 1);
    } else {
        entry = tok / p.page_size;
        offset = tok - entry * p.page_size;
    }
}
__device__ __forceinline__ int checked_page(const DecodeParams& p, int page) {
    if ((unsigned)page < (unsigned)p.num_pages) return page;
    set_status(p.status, KVS_ERR_INVALID_ARG);
    return 0;
}

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
    const int n = min(max(p.n_tokens[s], 0), p.max_pages * p.page_size);    // never past the sequence's table
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

    // the block-table entry of a block's token t0 + l16 is read one block ahead of its use
    auto page_of = [&](int b) {
        int e = 0, o;
        if (b < nblocks) split_token(p, min(b * BLK + (l16 & (BLK - 1)), n - 1), e, o);
        return (b < nblocks) ? bt[e] : 0;
    };
    int page_id = page_of(first);
    for (int b = first; b < nblocks; b += stride) {
        const int t0 = b * BLK;
        // row index (page * page_size + offset) of token t0 + l16, fetched once per block by every lane;
        // tokens past the end are clamped to the last one (their scores are discarded below)
        const int tl = min(t0 + (l16 & (BLK - 1)), n - 1);
        int tl_entry, tl_off;
        split_token(p, tl, tl_entry, tl_off);
        const int my_row = checked_page(p, page_id) * ps + tl_off;
        page_id = page_of(b + stride);
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

// ---- tensor-core variant (head_dim 128) ------------------------------------------------------------
// With G >= 4 query heads per KV head the CUDA-core kernel above is bound by its arithmetic (every K/V
// element is multiplied G times in fp32), not by HBM.  Here the two products run on the tensor core in
// the transposed form, so that the 128 keys of a tile (not the few query heads) fill the 128 rows:
//   S^T [128 keys x 16] = K [128 x d] (Q_pad [16 x d])^T        A = K tile, B = Q (rows >= G are zero)
//   O^T [d x 16]      += (V [128 keys x d])^T P^T [128 keys x 16]   A = V tile read MN-major, B = P^T
// One CTA per (split, KV head, sequence), 4 softmax warps (thread = key in the S^T phase, = output
// column d in the O^T phase) and one control warp (block-table reads, TMA loads, MMA issue).  Three CTAs
// per SM overlap one another's loads, MMAs and softmax.  Inside a CTA the K and the V buffer are
// refilled at different times: K of tile t+1 is requested as soon as S^T of tile t is complete (the
// softmax and the second product of tile t hide its latency), V of tile t as soon as the second product
// of tile t-1 is complete (S^T and the softmax of tile t hide it).  How rows reach shared memory:
//   pages of 8..128 tokens that tile 128 exactly: one TMA box per page and 64-column half;
//   anything else (one token per page): K by TMA gather4, four cache rows per instruction, V by cp.async
//   from the softmax warps, 16 lanes per 256-byte row.  A TMA instruction costs the SM's TMA unit about
//   16 - 20 clocks whatever it moves, so with both K and V gathered (128 instructions per tile) the
//   kernel is bound by that unit; splitting the rows between the TMA unit and the load/store unit is
//   what gets past it.
// Block-table entries are read with independent loads ahead of their use and checked afterwards: a load
// whose value decides a branch at once would put one memory latency per entry into the tile's chain.
// Tensor memory: 32 columns (S^T | O^T).  The per-head maximum over the 128 keys of a tile is a warp
// reduction plus one exchange through shared memory; the reference maximum moves lazily (threshold
// 8 in base-2 units), so O^T is rescaled in tensor memory only rarely.
constexpr int DTC_THREADS = 160;
constexpr int DTC_PAGES = 1;     // one TMA box per page
constexpr int DTC_ROWS = 2;      // K: TMA gather4; V: cp.async rows

struct DtcSmem {
    static constexpr int OFF_K = 0;                    // [128 keys x 128 d] bf16, two 64-column boxes, 128-byte swizzle
    static constexpr int OFF_V = 32768;
    static constexpr int OFF_Q = 65536;                // [16 x 128] bf16, two boxes of [16 x 64]
    static constexpr int OFF_P = 65536 + 4096;         // P^T as [16 heads x 128 keys] bf16, two boxes of [16 x 64]
    static constexpr int OFF_BAR = 65536 + 8192;       // 8 mbarriers
    static constexpr int OFF_MISC = OFF_BAR + 64;      // tmem base, abort flag
    static constexpr int OFF_WMAX = OFF_MISC + 64;     // [2 buffers][4 warps][16] fp32
    static constexpr int OFF_WSUM = OFF_WMAX + 512;    // [4 warps][16] fp32
    static constexpr int TOTAL = OFF_WSUM + 256;
    static constexpr int DYN_BYTES = TOTAL + 1024;     // slack for the 1024-byte alignment
};

// order-preserving map float -> int, so that a warp-wide integer max gives the float max
__device__ __forceinline__ int float_order(float x) {
    const int i = __float_as_int(x);
    return i ^ ((i >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float float_unorder(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// TMA gather: the 64-column slice starting at column c0 of the four rows r0..r3 of a 2-D tensor lands in four
// consecutive 128-byte rows at dst (swizzled by address like a tiled box); completes 512 bytes on the barrier.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap* map, int c0, int r0, int r1, int r2, int r3, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar)
        : "memory");
}

template <int G, int LOAD>
__global__ void __launch_bounds__(DTC_THREADS, 3)
decode_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v, DecodeParams p, int32_t* status) {
    constexpr int D = 128;
    constexpr int BOX = 16384;                  // one 64-column box of a 128-row tile
    constexpr uint32_t IDESC_S = make_idesc(16, 0, 0);
    constexpr uint32_t IDESC_O = make_idesc(16, 1, 0);
    constexpr bool PAGES = LOAD == DTC_PAGES;
    extern __shared__ uint8_t smem_raw[];
    const int z = blockIdx.x, g = blockIdx.y, s = blockIdx.z;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int n = min(max(p.n_tokens[s], 0), p.max_pages * p.page_size);    // never past the sequence's table
    const int ps = p.page_size;
    const int ppt = 128 / ps;                                   // pages per tile (PAGES)
    const int ntiles = (n + 127) >> 7;
    const int per = (ntiles + p.nsplit - 1) / p.nsplit;         // contiguous tiles per split
    const int t_begin = min(z * per, ntiles), t_end = min(t_begin + per, ntiles);
    const int my_tiles = t_end - t_begin;

    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sbase = (sraw + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - sraw);
    const uint32_t sK = sbase + DtcSmem::OFF_K, sV = sbase + DtcSmem::OFF_V, sQ = sbase + DtcSmem::OFF_Q, sP = sbase + DtcSmem::OFF_P;
    const uint32_t bars = sbase + DtcSmem::OFF_BAR;
    // kfull / vfull: the tile's K / V rows have landed (TMA);  s: S^T is complete, hence K consumed and, the tensor pipe
    // being in order, the previous tile's second product too (V, P^T consumed, O^T up to date);  p: P^T is written (and,
    // with DTC_ROWS, the thread's V rows have landed);  done: the second product of a tile is complete
    const uint32_t bar_kfull = bars, bar_vfull = bars + 8, bar_s = bars + 16, bar_p = bars + 24, bar_done = bars + 32;
    uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sgen + DtcSmem::OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + DtcSmem::OFF_MISC + 4);
    float* s_wmax = reinterpret_cast<float*>(sgen + DtcSmem::OFF_WMAX);
    float* s_wsum = reinterpret_cast<float*>(sgen + DtcSmem::OFF_WSUM);

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_kfull, 1);
        mbar_init(bar_vfull, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_p, 128);
        mbar_init(bar_done, 1);
        fence_mbar_init();
    }
    if (warp == 4) {
        tmem_alloc(smem_u32(s_tmem), 32);
        tmem_relinquish();
    } else {
        // V starts as zeros (rows no page is loaded into must stay finite: their weight is 0, and 0 x NaN is NaN);
        // Q: rows 0..G-1 of the 16-row B operand, the rest zero; P^T: rows >= G stay zero for good
        uint4 zero4 = make_uint4(0, 0, 0, 0);
        for (int i = tid; i < 32768 / 16; i += 128) reinterpret_cast<uint4*>(sgen + DtcSmem::OFF_V)[i] = zero4;
        for (int i = tid; i < 8192 / 16; i += 128) reinterpret_cast<uint4*>(sgen + DtcSmem::OFF_Q)[i] = zero4;
        named_bar_sync(1, 128);
        // Q row h, 16-byte chunk c (8 elements) of box b: physical chunk c ^ (h % 8) of the 128-byte row
        for (int i = tid; i < G * 16; i += 128) {
            const int h = i >> 4, c16 = i & 15, b = c16 >> 3, c = c16 & 7;
            const uint4 v = *reinterpret_cast<const uint4*>(p.q + ((size_t)s * p.Hq + g * G + h) * D + c16 * 8);
            *reinterpret_cast<uint4*>(sgen + DtcSmem::OFF_Q + b * 2048 + h * 128 + ((c ^ (h & 7)) << 4)) = v;
        }
        fence_proxy_async();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;
    const uint32_t tmem_S = tmem, tmem_O = tmem + 16;
    const int32_t* bt = p.block_table + (size_t)s * p.max_pages;

    if (warp == 4) {
        // ================= control warp: block table, TMA loads, MMA issue =================
        const bool leader = elect_one();
        const uint64_t dK = smem_desc(sK, 16, 1024), dQ = smem_desc(sQ, 16, 1024);
        const uint64_t dV = smem_desc(sV, BOX, 1024), dP = smem_desc(sP, 16, 1024);
        // Block-table entries of a tile, held by the lanes: PAGES: lane i has page i of the tile (at most 16);
        // ROWS: lane L has the pages of rows 4L .. 4L+3; a row past the end of the sequence repeats the last valid
        // token (finite values, weight 0).
        struct Ids { int v[PAGES ? 1 : 4]; };
        auto fetch_ids = [&](int tt, Ids& id) {
            if (tt >= t_end) return;
            if (PAGES) {
                const int npages = min(ppt, (n - tt * 128 + ps - 1) / ps);
                id.v[0] = (lane < npages) ? bt[tt * ppt + lane] : 0;
            } else {
                const int nvalid = min(128, n - tt * 128);
#pragma unroll
                for (int j = 0; j < (PAGES ? 1 : 4); ++j) {
                    int e, o;
                    split_token(p, tt * 128 + min(4 * lane + j, nvalid - 1), e, o);
                    id.v[j] = bt[e];
                }
            }
        };
        auto load_k = [&](int tt, const Ids& id) {          // K buffer must be free
            if (PAGES) {
                const int npages = min(ppt, (n - tt * 128 + ps - 1) / ps);
                const int row = checked_page(p, id.v[0]) * ps;
                if (leader) mbar_expect_tx(bar_kfull, (uint32_t)(npages * ps) * 256u);
                __syncwarp();
                if (lane < npages) {
                    const uint32_t off = (uint32_t)(lane * ps) * 128u;
                    tma_load_3d(sK + off, &tm_k, 0, g, row, bar_kfull);
                    tma_load_3d(sK + BOX + off, &tm_k, 64, g, row, bar_kfull);
                }
            } else {
                const int nvalid = min(128, n - tt * 128);
                const int ngroups = (nvalid + 3) >> 2;      // groups wholly past the end are not fetched
                int row[4];
#pragma unroll
                for (int j = 0; j < (PAGES ? 1 : 4); ++j) {
                    int e, o;
                    split_token(p, tt * 128 + min(4 * lane + j, nvalid - 1), e, o);
                    row[j] = checked_page(p, id.v[j]) * ps + o;
                }
                if (leader) mbar_expect_tx(bar_kfull, (uint32_t)ngroups * 1024u);
                __syncwarp();
                if (lane < ngroups) {
                    const uint32_t off = (uint32_t)lane * 512u;
                    tma_gather4(sK + off, &tm_k, g * D, row[0], row[1], row[2], row[3], bar_kfull);
                    tma_gather4(sK + BOX + off, &tm_k, g * D + 64, row[0], row[1], row[2], row[3], bar_kfull);
                }
            }
        };
        auto load_v = [&](int tt, const Ids& id) {          // PAGES only; V buffer must be free
            const int npages = min(ppt, (n - tt * 128 + ps - 1) / ps);
            const int row = checked_page(p, id.v[0]) * ps;
            if (leader) mbar_expect_tx(bar_vfull, (uint32_t)(npages * ps) * 256u);
            __syncwarp();
            if (lane < npages) {
                const uint32_t off = (uint32_t)(lane * ps) * 128u;
                tma_load_3d(sV + off, &tm_v, 0, g, row, bar_vfull);
                tma_load_3d(sV + BOX + off, &tm_v, 64, g, row, bar_vfull);
            }
        };
        Ids cur, nxt;
        for (int j = 0; j < (PAGES ? 1 : 4); ++j) cur.v[j] = nxt.v[j] = 0;
        fetch_ids(t_begin, cur);
        fetch_ids(t_begin + 1, nxt);
        if (my_tiles > 0) load_k(t_begin, cur);
        for (int it = 0; it < my_tiles; ++it) {
            const int tt = t_begin + it;
            mbar_wait(bar_kfull, it & 1, abort_flag, status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {      // S^T = K Q^T, 16 elements of d per step
                const uint64_t offk = (uint64_t)(((kk >> 2) * BOX + (kk & 3) * 32) >> 4);
                const uint64_t offq = (uint64_t)(((kk >> 2) * 2048 + (kk & 3) * 32) >> 4);
                if (leader) mma_ss(tmem_S, dK + offk, dQ + offq, IDESC_S, kk > 0);
            }
            if (leader) mma_commit(bar_s);
            mbar_wait(bar_s, it & 1, abort_flag, status);      // K is consumed; so are V and P^T of the previous tile
            if (PAGES) load_v(tt, cur);
            if (it + 1 < my_tiles) load_k(tt + 1, nxt);
            cur = nxt;
            fetch_ids(tt + 2, nxt);
            mbar_wait(bar_p, it & 1, abort_flag, status);
            if (PAGES) mbar_wait(bar_vfull, it & 1, abort_flag, status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 8; ++kk) {           // O^T += V^T P^T, 16 keys per step
                const uint64_t offp = (uint64_t)(((kk >> 2) * 2048 + (kk & 3) * 32) >> 4);
                if (leader) mma_ss(tmem_O, dV + (uint64_t)(kk * 128), dP + offp, IDESC_O, (it > 0) || (kk > 0));
            }
            if (leader) mma_commit(bar_done);
        }
    } else {
        // ================= softmax warps =================
        const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
        float m_run[G], l_part[G];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            m_run[h] = -INFINITY;
            l_part[h] = 0.f;
        }
        // DTC_ROWS: this thread's 16 rows of a tile's V (row r = warp * 32 + 2 j + lane / 16, 16 lanes per 256-byte row,
        // cp.async into the swizzled layout).  Rows past the end of the sequence are not fetched and keep their earlier,
        // finite contents (their weight is 0).  The block-table entries are loaded one tile ahead.
        int pid[PAGES ? 1 : 16];
        auto fetch_pids = [&](int tt) {
            if (PAGES || tt >= t_end) return;
            const int nvalid = min(128, n - tt * 128);
#pragma unroll
            for (int j = 0; j < (PAGES ? 1 : 16); ++j) {
                int e, o;
                split_token(p, tt * 128 + min(warp * 32 + 2 * j + (lane >> 4), nvalid - 1), e, o);
                pid[j] = bt[e];
            }
        };
        const __nv_bfloat16* v_lane = p.v_cache + (size_t)g * D + (lane & 15) * 8;       // this lane's 16 bytes of a row of head g
        const int v_row_elems = p.Hkv * D;
        auto load_v_rows = [&](int tt) {
            const int nvalid = min(128, n - tt * 128);
            const int c = lane & 15;
#pragma unroll
            for (int j = 0; j < (PAGES ? 1 : 16); ++j) {
                const int r = warp * 32 + 2 * j + (lane >> 4);
                int e, o;
                split_token(p, tt * 128 + r, e, o);
                const int crow = checked_page(p, pid[j]) * ps + o;
                if (r < nvalid) {
                    const uint32_t dst = (uint32_t)((c >> 3) * BOX + r * 128 + (((c & 7) ^ (r & 7)) << 4));
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(sV + dst), "l"(v_lane + (long long)crow * v_row_elems) : "memory");
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
        fetch_pids(t_begin);
        for (int it = 0; it < my_tiles; ++it) {
            const int tt = t_begin + it;
            const int nvalid = min(128, n - tt * 128);
            mbar_wait(bar_s, it & 1, abort_flag, status);       // S^T ready; V, P^T free; O^T up to date
            tc_fence_after();
            if (!PAGES) {
                load_v_rows(tt);
                fetch_pids(tt + 1);
            }
            uint32_t r[16];
            tmem_ld16(tmem_S + lane_sel, r);
            tmem_wait_ld();
            float sc[G];
            float* wmax = s_wmax + (it & 1) * 64;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                sc[h] = (tid < nvalid) ? __uint_as_float(r[h]) * p.scale_log2 : -INFINITY;
                const int wm = __reduce_max_sync(0xffffffffu, float_order(sc[h]));
                if (lane == 0) wmax[warp * 16 + h] = float_unorder(wm);
            }
            named_bar_sync(1, 128);
            bool grow_any = false;
            float tmax[G];
#pragma unroll
            for (int h = 0; h < G; ++h) {
                tmax[h] = fmaxf(fmaxf(wmax[h], wmax[16 + h]), fmaxf(wmax[32 + h], wmax[48 + h]));
                grow_any |= (tmax[h] > m_run[h] + 8.0f) || (m_run[h] == -INFINITY && tmax[h] > -INFINITY);
            }
            if (grow_any) {                      // the same decision in every thread: the maxima are CTA-wide
                float alpha[16];
#pragma unroll
                for (int h = 0; h < 16; ++h) alpha[h] = 1.f;
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const bool grow = (tmax[h] > m_run[h] + 8.0f) || (m_run[h] == -INFINITY && tmax[h] > -INFINITY);
                    const float m_new = grow ? tmax[h] : m_run[h];
                    alpha[h] = (m_new == -INFINITY) ? 1.f : fast_exp2(m_run[h] - m_new);
                    l_part[h] *= alpha[h];
                    m_run[h] = m_new;
                }
                if (it > 0) {                     // O^T row d = tid: every MMA issued before S^T(it) has completed
                    uint32_t o[16];
                    tmem_ld16(tmem_O + lane_sel, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int h = 0; h < 16; ++h) o[h] = __float_as_uint(__uint_as_float(o[h]) * alpha[h]);
                    tmem_st16(tmem_O + lane_sel, o);
                    tmem_wait_st();
                }
            }
            // weights of key tid for the G heads -> P^T[h][tid] (bf16), row h of box tid / 64
            uint8_t* prow = sgen + DtcSmem::OFF_P + (tid >> 6) * 2048 + ((tid & 7) << 1);
            const int chunk = (tid & 63) >> 3;
#pragma unroll
            for (int h = 0; h < G; ++h) {
                const float m_use = (m_run[h] == -INFINITY) ? 0.f : m_run[h];
                const float w = fast_exp2(sc[h] - m_use);
                l_part[h] += w;
                *reinterpret_cast<__nv_bfloat16*>(prow + h * 128 + ((chunk ^ (h & 7)) << 4)) = __float2bfloat16(w);
            }
            if (PAGES) {
                const int loaded = min(ppt, (n - tt * 128 + ps - 1) / ps) * ps;
                if (loaded > nvalid) {            // the same decision in every thread
                    // rows of the last page past the end of the sequence hold whatever the cache holds there
                    mbar_wait(bar_vfull, it & 1, abort_flag, status);
                    if (tid >= nvalid && tid < loaded) {
                        const uint4 zero4 = make_uint4(0, 0, 0, 0);
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            *reinterpret_cast<uint4*>(sgen + DtcSmem::OFF_V + tid * 128 + c * 16) = zero4;
                            *reinterpret_cast<uint4*>(sgen + DtcSmem::OFF_V + BOX + tid * 128 + c * 16) = zero4;
                        }
                    }
                }
            } else {
                asm volatile("cp.async.wait_group 0;" ::: "memory");
            }
            fence_proxy_async();      // P^T and the V rows written by this thread visible to the tensor core's reads of shared memory
            tc_fence_before();
            mbar_arrive(bar_p);
        }
        // ---- this split's partial result: O^T (unnormalised), the reference maxima and the sums ----
        if (my_tiles > 0) {
            mbar_wait(bar_done, (my_tiles - 1) & 1, abort_flag, status);
            tc_fence_after();
        }
        uint32_t o[16];
        if (my_tiles > 0) {
            tmem_ld16(tmem_O + lane_sel, o);
            tmem_wait_ld();
        } else {
#pragma unroll
            for (int h = 0; h < 16; ++h) o[h] = 0u;
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float v = l_part[h];
#pragma unroll
            for (int ofs = 16; ofs > 0; ofs >>= 1) v += __shfl_xor_sync(0xffffffffu, v, ofs);
            if (lane == 0) s_wsum[warp * 16 + h] = v;
            const size_t base = ((size_t)s * p.Hq + g * G + h) * p.nsplit + z;
            p.part_o[base * D + tid] = __uint_as_float(o[h]);
        }
        named_bar_sync(1, 128);
#pragma unroll
        for (int h = 0; h < G; ++h) {
            if (tid == h) {
                const size_t base = ((size_t)s * p.Hq + g * G + h) * p.nsplit + z;
                p.part_ml[base * 2 + 0] = m_run[h];
                p.part_ml[base * 2 + 1] = s_wsum[h] + s_wsum[16 + h] + s_wsum[32 + h] + s_wsum[48 + h];
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) {
        __syncwarp();
        tmem_dealloc(tmem, 32);
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
                                    int num_pages, int32_t* block_table, int32_t* n_tokens, int32_t* free_buf, __nv_bfloat16* k_cache,
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
                if (top <= 0 || top > num_pages) {
                    atomicAdd(&hdr->top, 1);
                    atomicCAS(&hdr->status, 0, top <= 0 ? KVS_ERR_WORKSPACE : KVS_ERR_INVALID_ARG);   // cache full / corrupt stack
                } else {
                    page = stack[top - 1];
                    block_table[(size_t)s * max_pages + slot / page_size] = page;
                }
            }
        } else {
            page = block_table[(size_t)s * max_pages + slot / page_size];
        }
        if (page >= num_pages || (page < 0 && page != -1)) {       // an entry that names no page of this cache
            atomicCAS(&hdr->status, 0, KVS_ERR_INVALID_ARG);
            page = -1;
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
                                   int num_pages, int32_t* block_table, int32_t* n_tokens, int32_t* free_buf) {
    CacheHeader* hdr = reinterpret_cast<CacheHeader*>(free_buf);
    int32_t* stack = free_buf + 4;
    const int s = blockIdx.x;
    if (s >= S) return;
    extern __shared__ int32_t sh[];              // keep flags / new positions, max_pages entries
    __shared__ int s_base, s_bad;
    const int n = n_tokens[s];
    const int npages = (n + page_size - 1) / page_size;
    int32_t* bt = block_table + (size_t)s * max_pages;
    if (threadIdx.x == 0) s_bad = (n < 0 || npages > max_pages) ? 1 : 0;
    __syncthreads();
    if (s_bad) {
        if (threadIdx.x == 0) atomicCAS(&hdr->status, 0, KVS_ERR_INVALID_ARG);
        return;
    }
    for (int i = threadIdx.x; i < npages; i += blockDim.x) sh[i] = 1;
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
        if (lane == 0) {
            s_base = atomicAdd(&hdr->top, freed);
            if (s_base < 0 || s_base + freed > num_pages) {        // more pages coming back than the cache has: corrupt state
                atomicSub(&hdr->top, freed);
                atomicCAS(&hdr->status, 0, KVS_ERR_INVALID_ARG);
                s_base = -1;
            }
        }
        __syncwarp();
        const int base = s_base;
        if (base < 0) return;
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
            if (keep) bt[kept + __popc(km & lt)] = page;          // kept + rank <= i: never ahead of the reads of this pass
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
                                int page_size, int max_pages, int num_pages, int32_t* block_table, int32_t* n_tokens, int32_t* free_list,
                                void* k_cache, void* v_cache, kvs_stream_t stream) {
    if (!k_new || !v_new || !block_table || !n_tokens || !free_list || !k_cache || !v_cache) return KVS_ERR_INVALID_ARG;
    if (num_seqs < 0 || Hkv <= 0 || head_dim <= 0 || page_size <= 0 || max_pages <= 0 || num_pages <= 0) return KVS_ERR_INVALID_ARG;
    if (num_seqs == 0) return KVS_OK;
    cache_append_kernel<<<num_seqs, 128, 0, (cudaStream_t)stream>>>((const __nv_bfloat16*)k_new, (const __nv_bfloat16*)v_new, active,
                                                                   num_seqs, Hkv, head_dim, page_size, max_pages, num_pages, block_table,
                                                                   n_tokens, free_list, (__nv_bfloat16*)k_cache,
                                                                   (__nv_bfloat16*)v_cache);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_cache_evict(const int32_t* ranges, int n_ranges, int num_seqs, int page_size, int max_pages, int num_pages,
                               int32_t* block_table,
                               int32_t* n_tokens, int32_t* free_list, kvs_stream_t stream) {
    if (!block_table || !n_tokens || !free_list || n_ranges < 0 || num_seqs < 0 || page_size <= 0 || max_pages <= 0 || num_pages <= 0)
        return KVS_ERR_INVALID_ARG;
    if (n_ranges > 0 && !ranges) return KVS_ERR_INVALID_ARG;
    if ((size_t)max_pages * sizeof(int32_t) > 200 * 1024) return KVS_ERR_UNSUPPORTED;
    if (n_ranges == 0 || num_seqs == 0) return KVS_OK;
    const size_t smem = (size_t)max_pages * sizeof(int32_t);
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(cache_evict_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return KVS_ERR_CUDA;
    cache_evict_kernel<<<num_seqs, 256, smem, (cudaStream_t)stream>>>(ranges, n_ranges, num_seqs, page_size, max_pages, num_pages, block_table,
                                                                     n_tokens, free_list);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

extern "C" int kvs_decode_num_splits(int num_seqs, int Hkv, int max_tokens) {
    if (num_seqs <= 0 || Hkv <= 0 || max_tokens <= 0) return 1;
    // Three CTAs are resident per SM (148 SMs).  At least two waves of CTAs, at least 4 tiles of 128 tokens per split,
    // and from there up to three times as many the first count whose last wave is at least 92 % full (else the
    // fullest): a CTA of a sparse last wave runs at the latency of its own loads instead of sharing the memory
    // system's bandwidth.
    const long long slots = 3 * 148, base = (long long)num_seqs * Hkv;
    long long want = (2 * slots + base - 1) / base;
    long long cap = ((long long)max_tokens + 128 * 4 - 1) / (128 * 4);
    if (cap > 64) cap = 64;
    if (want > cap) want = cap;
    if (want < 1) want = 1;
    long long best = want;
    double best_eff = 0.0;
    for (long long n = want; n <= cap && n <= 3 * want; ++n) {
        const long long ctas = base * n, waves = (ctas + slots - 1) / slots;
        const double eff = (double)ctas / (double)(waves * slots);
        if (eff > best_eff) {
            best_eff = eff;
            best = n;
        }
        if (eff >= 0.92) break;                 // the smallest count that fills its last wave well
    }
    return (int)best;
}

extern "C" size_t kvs_decode_workspace_bytes(int num_seqs, int Hq, int head_dim, int num_splits) {
    if (num_seqs < 0 || Hq <= 0 || head_dim <= 0 || num_splits <= 0) return 0;
    return DEC_WS_HEADER + align_up(sizeof(float) * (size_t)num_seqs * Hq * num_splits * (head_dim + 2), 256);
}

// the first 256 bytes of the workspace: {magic, status} as in the backward workspace, so that
// kvs_device_status() reads it; the partial results follow
__global__ void decode_header_kernel(int32_t* hdr) {
    hdr[0] = (int32_t)WS_MAGIC;
    hdr[1] = KVS_OK;
}

template <int G, int LOAD>
static int launch_decode_tc(const CUtensorMap& tk, const CUtensorMap& tv, const DecodeParams& p, int32_t* status, cudaStream_t st) {
    auto kern = decode_tc_kernel<G, LOAD>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, DtcSmem::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    dim3 grid(p.nsplit, p.Hkv, p.S);
    kern<<<grid, DTC_THREADS, DtcSmem::DYN_BYTES, st>>>(tk, tv, p, status);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

template <int D>
static int launch_decode(const DecodeParams& p, int G, const void* k_cache, const void* v_cache, int32_t* status, void* out, float* lse,
                         cudaStream_t st) {
    dim3 grid(p.nsplit, p.Hkv, p.S);
    const int ps = p.page_size;
    // tensor-core variant (head_dim 128).  Pages that are whole 8-row swizzle atoms and tile 128 tokens exactly come in
    // by TMA, one box per page: at the HBM roofline for every group size.  Smaller pages (one token per page) come in
    // row by row (K by TMA gather, V by cp.async), which beats the CUDA-core kernel from G = 2 on (measured at one
    // token per page, fraction of the HBM roofline: G = 1 0.93 against 0.99, G = 2 0.93 against 0.84, G = 4 0.92).
    const bool paged_tma = (ps % 8 == 0) && (ps <= 128) && (128 % ps == 0);
    const bool tc = (D == 128) && (G == 1 || G == 2 || G == 4 || G == 7 || G == 8) && (paged_tma || G >= 2);
    if (tc) {
        int rc = check_device_sm100();
        if (rc != KVS_OK) return rc;
        CUtensorMap tk, tv;
        memset(&tk, 0, sizeof(tk));
        memset(&tv, 0, sizeof(tv));
        if (paged_tma) {
            // the caches as (d, Hkv, rows) with rows = num_pages * page_size: a box is one page, and no box
            // can reach past the cache (the table entries are range-checked on top of that)
            if ((long long)p.num_pages * ps > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
            if ((rc = make_tmap_thd(&tk, k_cache, p.num_pages * ps, p.Hkv, 128, ps)) != KVS_OK) return rc;
            if ((rc = make_tmap_thd(&tv, v_cache, p.num_pages * ps, p.Hkv, 128, ps)) != KVS_OK) return rc;
            switch (G) {
                case 1: rc = launch_decode_tc<1, DTC_PAGES>(tk, tv, p, status, st); break;
                case 2: rc = launch_decode_tc<2, DTC_PAGES>(tk, tv, p, status, st); break;
                case 4: rc = launch_decode_tc<4, DTC_PAGES>(tk, tv, p, status, st); break;
                case 7: rc = launch_decode_tc<7, DTC_PAGES>(tk, tv, p, status, st); break;
                default: rc = launch_decode_tc<8, DTC_PAGES>(tk, tv, p, status, st); break;
            }
        } else {
            // the K cache as (Hkv * d, rows): a gather names four rows and a 64-column slice of one KV head (V is
            // fetched with plain row copies and needs no tensor map)
            if ((long long)p.num_pages * ps > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
            if ((rc = make_tmap_rows(&tk, k_cache, p.num_pages * ps, p.Hkv * 128)) != KVS_OK) return rc;
            switch (G) {
                case 1: rc = launch_decode_tc<1, DTC_ROWS>(tk, tv, p, status, st); break;
                case 2: rc = launch_decode_tc<2, DTC_ROWS>(tk, tv, p, status, st); break;
                case 4: rc = launch_decode_tc<4, DTC_ROWS>(tk, tv, p, status, st); break;
                case 7: rc = launch_decode_tc<7, DTC_ROWS>(tk, tv, p, status, st); break;
                default: rc = launch_decode_tc<8, DTC_ROWS>(tk, tv, p, status, st); break;
            }
        }
        if (rc != KVS_OK) return rc;
    } else
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
                               int num_pages, float softmax_scale, int num_splits, void* out, float* lse, void* workspace, size_t workspace_bytes,
                               kvs_stream_t stream) {
    if (num_seqs < 0 || Hq <= 0 || Hkv <= 0 || page_size <= 0 || max_pages <= 0 || num_pages <= 0 || num_splits <= 0)
        return KVS_ERR_INVALID_ARG;
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
    p.page_shift = (page_size & (page_size - 1)) == 0 ? __builtin_ctz((unsigned)page_size) : -1;
    p.max_pages = max_pages;
    p.num_pages = num_pages;
    p.status = (int32_t*)workspace + 1;
    p.nsplit = num_splits;
    const float s = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = s * 1.4426950408889634f;
    p.part_o = (float*)((char*)workspace + DEC_WS_HEADER);
    p.part_ml = p.part_o + (size_t)num_seqs * Hq * num_splits * head_dim;
    cudaStream_t st = (cudaStream_t)stream;
    decode_header_kernel<<<1, 1, 0, st>>>((int32_t*)workspace);
    int32_t* status = (int32_t*)workspace + 1;
    return head_dim == 64 ? launch_decode<64>(p, Hq / Hkv, k_cache, v_cache, status, out, lse, st)
                          : launch_decode<128>(p, Hq / Hkv, k_cache, v_cache, status, out, lse, st);
}
