// Backward: dQ, dK, dV of eviction-masked causal attention.
//
//   pre-pass   D_i = dout_i . out_i                         (one warp per (token, head))
//   main       one CTA per (key block n, KV head g), longest key blocks first; K and V tiles stay in
//              shared memory; the CTA loops over the G query heads of the group and over the
//              contiguous range of query blocks n .. col_last[n] that can see the key block
//              (see the comment above bwd_kernel for the pipeline)
//   post-pass  fp32 dQ accumulator -> bf16 (bf16 gradients only)
#include "kvs_common.cuh"

namespace kvs {

struct BwdWsLayout {
    size_t dvec, dq_acc, total;
};

__host__ __device__ inline BwdWsLayout bwd_ws_layout(int total_tokens, int Hq, int head_dim, int grad_dtype) {
    BwdWsLayout L;
    size_t o = align_up(sizeof(WsHeader), 256);
    L.dvec = o;
    o = align_up(o + sizeof(float) * (size_t)total_tokens * Hq, 256);
    L.dq_acc = o;
    if (grad_dtype == KVS_GRAD_BF16) o = align_up(o + sizeof(float) * (size_t)total_tokens * Hq * head_dim, 256);
    L.total = o;
    return L;
}

// ---- pre-pass ---------------------------------------------------------------------------------
// D[h][tok] = sum_c dout[tok][h][c] * out[tok][h][c], and the fp32 dQ accumulator cleared in the same pass (it is
// the destination of the main kernel's reduce-adds).  16 bytes per lane and tensor, D/8 lanes per row, DOT_ROWS rows in
// flight per lane: the pass streams 2 x 2 B in and 4 B out per element and is bound by HBM.
constexpr int DOT_ROWS = 4;
template <int D>
__global__ void __launch_bounds__(256)
bwd_dot_kernel(const __nv_bfloat16* __restrict__ dout, const __nv_bfloat16* __restrict__ out,
               float* __restrict__ dvec, float* __restrict__ dq_acc, long long dq_ts, int total_tokens, int Hq, WsHeader* hdr) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        hdr->magic = WS_MAGIC;
        hdr->status = KVS_OK;
    }
    constexpr int LPR = D / 8;                  // lanes per row: 16 or 8
    constexpr int RPW = 32 / LPR;               // rows per warp and step
    const long long rows = (long long)total_tokens * Hq;
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, c = lane % LPR;
    const long long row0 = gw * (RPW * DOT_ROWS) + sub;
    uint4 x[DOT_ROWS], y[DOT_ROWS];
#pragma unroll
    for (int r = 0; r < DOT_ROWS; ++r) {
        const long long row = row0 + (long long)r * RPW;
        if (row < rows) {
            x[r] = *reinterpret_cast<const uint4*>(dout + (size_t)row * D + c * 8);
            y[r] = *reinterpret_cast<const uint4*>(out + (size_t)row * D + c * 8);
        } else {
            x[r] = y[r] = make_uint4(0, 0, 0, 0);
        }
    }
    const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int r = 0; r < DOT_ROWS; ++r) {
        const long long row = row0 + (long long)r * RPW;
        const uint32_t xa[4] = {x[r].x, x[r].y, x[r].z, x[r].w}, ya[4] = {y[r].x, y[r].y, y[r].z, y[r].w};
        float acc = 0.f;
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            acc = fmaf(__uint_as_float(xa[e] << 16), __uint_as_float(ya[e] << 16), acc);
            acc = fmaf(__uint_as_float(xa[e] & 0xffff0000u), __uint_as_float(ya[e] & 0xffff0000u), acc);
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (row < rows) {
            if (dq_acc) {
                float4* z = reinterpret_cast<float4*>(dq_acc + (size_t)(row / Hq) * dq_ts + (size_t)(row % Hq) * D + c * 8);
                z[0] = zero;
                z[1] = zero;
            }
            if (c == 0) dvec[(size_t)(row % Hq) * total_tokens + (row / Hq)] = acc;
        }
    }
}

// ---- post-pass --------------------------------------------------------------------------------
// acc: contiguous [tokens, row_elems]; dq: rows of row_elems elements, dq_ts elements apart
__global__ void bwd_cast_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, size_t n4, int row_elems, long long dq_ts) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 x = reinterpret_cast<const float4*>(acc)[i];
    uint2 w;
    w.x = pack_bf16(x.x, x.y);
    w.y = pack_bf16(x.z, x.w);
    const size_t e = i * 4;
    *reinterpret_cast<uint2*>(dq + (e / row_elems) * (size_t)dq_ts + e % row_elems) = w;
}

// ---- main -------------------------------------------------------------------------------------
// Warp-specialised, 16 warps in four warp groups:
//   warps 0-7   compute: one key row per thread, 64 of the 128 query columns each (P^T, dS^T)
//   warps 8-11  drain:   dQ tile, tensor memory -> registers -> swizzled shared memory -> TMA
//               reduce-add into the fp32 accumulator (global `red` instructions are processed at
//               about one thread per clock per SM, which alone would exceed the MMA time of a tile)
//   warp 12     producer (TMA for K, V, Q, dO; plain loads for lse and D)
//   warp 13     MMA issuer;   warps 14-15 idle (they only complete the warp group)
// Registers are re-balanced per warp group with setmaxnreg (compute 144, drain 136, the rest 88).
//
// Tensor memory (512 columns):  [0,128) S^T fp32, then P^T bf16 in [0,32) and [64,96)
//                               [128,256) dP^T fp32, then dQ fp32
//                               [256,256+D) dV     [384,384+D) dK
// Per iteration j (one (head, query block) tile) the tensor pipe runs, in this order,
//     dP^T(j) = V dO^T,  dV(j) += P^T dO,  S^T(j+1) = K Q^T,  dQ(j) = dS K,  dK(j) += dS^T Q
// while the compute warps run  dS(j), P(j+1)  and the drain warps empty dQ(j).  The softmax scale
// is folded into dS (dS = P (scale dP - scale D)), so dK and dQ leave the tensor core scaled.
// Rows of a dQ tile past the end of a trace are exactly zero (their P is zero), so the reduce-add
// of a whole 128-row box is harmless where it overlaps the next trace.
constexpr int BWD_THREADS = 512;

template <int D>
struct BwdSmem {
    static constexpr int TB = TILE * D * 2;
    static constexpr int STG_BYTES = TILE * 128;     // 128 rows x 32 fp32
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = TB;
    static constexpr int OFF_Q = 2 * TB;             // 2 stages
    static constexpr int OFF_DO = 4 * TB;            // 1 stage
    static constexpr int OFF_DS = 5 * TB;            // 128 keys x 128 queries bf16
    static constexpr int OFF_STG = OFF_DS + TILE * TILE * 2;   // 2 staging buffers for dQ chunks
    static constexpr int OFF_LSE = OFF_STG + 2 * STG_BYTES;    // 2 stages x 128 fp32: -lse * log2 e
    static constexpr int OFF_DVEC = OFF_LSE + 2 * TILE * 4;    // 2 stages x 128 fp32: -D * scale
    static constexpr int OFF_BAR = OFF_DVEC + 2 * TILE * 4;
    static constexpr int OFF_MISC = OFF_BAR + 16 * 8;          // tmem base, abort flag
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int MAX_DYN = 232448;                     // 227 KB
    static constexpr int DYN_BYTES = (TOTAL + 1024 > MAX_DYN) ? MAX_DYN : TOTAL + 1024;
};

struct BwdParams {
    int batch, total_tokens, max_seqlen;   // what the caller says meta_buf was built for
    int Hq, Hkv;
    float scale, scale_log2;
    const float* lse;
    const float* dvec;
    void* dk;
    void* dv;
    long long dkv_ts;       // elements between consecutive tokens of dk and dv
    int grad_fp32;
    int32_t* status;
};

template <int D>
__global__ void __launch_bounds__(BWD_THREADS, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do,
           const __grid_constant__ CUtensorMap tm_dq, MetaView mv, BwdParams p) {
    using L = BwdSmem<D>;
    constexpr int NBOX = D / 64;
    constexpr int BOX_BYTES = TILE * 128;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_ST = make_idesc(TILE, 0, 0);    // K-major x K-major, N = 128 queries
    constexpr uint32_t IDESC_KV = make_idesc(D, 0, 1);       // A from tensor memory, B MN-major, N = D
    constexpr uint32_t IDESC_DQ = make_idesc(D, 1, 1);       // A, B MN-major, N = D
    constexpr int HALF_D = D / 2;

    extern __shared__ uint8_t smem_raw[];

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    // meta_buf must be the one kvs_mask_meta wrote for these sizes: every index below comes out of it
    if (!meta_matches(mv.hdr, p.batch, p.total_tokens, p.max_seqlen)) {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) set_status(p.status, KVS_ERR_BAD_META);
        return;
    }
    if ((int)blockIdx.x >= mv.hdr->nblk_total) return;
    const int gb = mv.bwd_order[blockIdx.x];
    const int g = blockIdx.y;
    const int G = p.Hq / p.Hkv;
    const int b = mv.blk_trace[gb];
    const int n = gb - mv.blk_off[b];
    const int tok0 = mv.seq_start[b];
    const int T = mv.seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    const int m_first = mv.col_first[gb];           // == n unless the key slots were re-ordered
    const int m_last = mv.col_last[gb];
    const int nm = m_last - m_first + 1;            // query blocks m_first .. m_last can see this key block
    const int n_iter = G * nm;
    int32_t* status = p.status;
    const bool general = mv.hdr->general != 0;
    if (nm <= 0) {
        // no query sees any key of the block (general metadata only): its gradients are zero
        const int rows = min(TILE, T - n * TILE);
        const size_t per_row = (size_t)D * (p.grad_fp32 ? 4 : 2) / 16;          // 16-byte words of one (token, head) row
        for (int i = tid; i < rows * (int)per_row; i += BWD_THREADS) {
            const size_t off = (size_t)(tok0 + n * TILE + i / (int)per_row) * (size_t)(p.dkv_ts / D) * per_row + (size_t)g * per_row + i % (int)per_row;
            reinterpret_cast<uint4*>(p.dk)[off] = make_uint4(0, 0, 0, 0);
            reinterpret_cast<uint4*>(p.dv)[off] = make_uint4(0, 0, 0, 0);
        }
        return;
    }

    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sbase = (sraw + 1023u) & ~1023u;
    if ((sbase - sraw) + L::TOTAL > (uint32_t)L::DYN_BYTES) {      // shared window not aligned as expected
        if (tid == 0) set_status(status, KVS_ERR_CUDA);
        return;
    }
    uint8_t* sgen = smem_raw + (sbase - sraw);
    const uint32_t sK = sbase + L::OFF_K, sV = sbase + L::OFF_V, sQ = sbase + L::OFF_Q, sDO = sbase + L::OFF_DO,
                   sDS = sbase + L::OFF_DS, sSTG = sbase + L::OFF_STG;
    uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(sgen + L::OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + L::OFF_MISC + 4);
    const uint32_t bars = sbase + L::OFF_BAR;
    const uint32_t bar_kv = bars;
    auto bar_qfull = [&](int s) { return bars + 8 * (1 + s); };
    auto bar_ldfull = [&](int s) { return bars + 8 * (3 + s); };
    auto bar_qfree = [&](int s) { return bars + 8 * (5 + s); };
    const uint32_t bar_dofull = bars + 8 * 7, bar_dofree = bars + 8 * 8, bar_s = bars + 8 * 9, bar_dp = bars + 8 * 10,
                   bar_p = bars + 8 * 11, bar_dq = bars + 8 * 13, bar_drained = bars + 8 * 14,
                   bar_dss = bars + 8 * 15;

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_kv, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_qfull(s), 1);
            mbar_init(bar_ldfull(s), 32);
            mbar_init(bar_qfree(s), 1);
        }
        mbar_init(bar_dofull, 1);
        mbar_init(bar_dofree, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_dp, 1);
        mbar_init(bar_p, 8);
        mbar_init(bar_dss, 8);
        mbar_init(bar_dq, 1);
        mbar_init(bar_drained, 4);
        fence_mbar_init();
    }
    if (warp == 13) {
        tmem_alloc(smem_u32(s_tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem_base;
    const uint32_t tmem_S = tmem;
    const uint32_t tmem_P = tmem + 128;
    const uint32_t tmem_dV = tmem + 256;
    const uint32_t tmem_dK = tmem + 384;

    if (warp >= 12) {
        reg_dec<88>();
        if (warp == 12) {
            // ================= producer =================
            float* sLse = reinterpret_cast<float*>(sgen + L::OFF_LSE);
            float* sDv = reinterpret_cast<float*>(sgen + L::OFF_DVEC);
            if (lane == 0) {
                mbar_expect_tx(bar_kv, 2 * L::TB);
                for (int c = 0; c < NBOX; ++c) tma_load_3d(sK + c * BOX_BYTES, &tm_k, c * 64, g, tok0 + n * TILE, bar_kv);
                for (int c = 0; c < NBOX; ++c) tma_load_3d(sV + c * BOX_BYTES, &tm_v, c * 64, g, tok0 + n * TILE, bar_kv);
            }
            for (int j = 0; j < n_iter; ++j) {
                const int s = j & 1;
                const int h = g * G + j / nm;
                const int m = m_first + j % nm;
                const int qtok = tok0 + m * TILE;
                // Q(j), lse(j), D(j): stage s, free once every MMA of iteration j-2 has completed
                if (j >= 2) mbar_wait(bar_qfree(s), ((j >> 1) + 1) & 1, abort_flag, status);
                if (lane == 0) {
                    mbar_expect_tx(bar_qfull(s), L::TB);
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(sQ + s * L::TB + c * BOX_BYTES, &tm_q, c * 64, h, qtok, bar_qfull(s));
                }
                const size_t rowbase = (size_t)h * p.total_tokens + qtok;
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = lane * 4 + u;
                    const bool qv = (m * TILE + i) < T;
                    // stored negated (they are subtracted with one fused multiply-add); -inf makes P vanish
                    // for the rows past the end of the trace
                    sLse[s * TILE + i] = qv ? p.lse[rowbase + i] * -1.4426950408889634f : -INFINITY;
                    sDv[s * TILE + i] = qv ? p.dvec[rowbase + i] * -p.scale : 0.f;
                }
                mbar_arrive(bar_ldfull(s));
                // dO(j): single buffer, free once dP(j-1) and dV(j-1) have completed
                if (lane == 0) {
                    if (j >= 1) mbar_wait(bar_dofree, (j - 1) & 1, abort_flag, status);
                    mbar_expect_tx(bar_dofull, L::TB);
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(sDO + c * BOX_BYTES, &tm_do, c * 64, h, qtok, bar_dofull);
                }
                __syncwarp();
            }
        } else if (warp == 13) {
            // ================= MMA issuer (all lanes walk the loop, one elected lane issues) =================
            const bool leader = elect_one();
            // descriptors of stage 0; a stage or a k-step adds a constant to the 14-bit address field
            const uint64_t dK_k = smem_desc(sK, 16, 1024), dV_k = smem_desc(sV, 16, 1024);
            const uint64_t dQ_k = smem_desc(sQ, 16, 1024), dDO_k = smem_desc(sDO, 16, 1024);
            const uint64_t dK_mn = smem_desc(sK, BOX_BYTES, 1024), dDS_mn = smem_desc(sDS, BOX_BYTES, 1024);
            const uint64_t dDS_k = smem_desc(sDS, 16, 1024);
            const uint64_t dQ_mn = smem_desc(sQ, BOX_BYTES, 1024), dDO_mn = smem_desc(sDO, BOX_BYTES, 1024);
            constexpr uint64_t STAGE = (uint64_t)(L::TB >> 4);
            mbar_wait(bar_kv, 0, abort_flag, status);
            mbar_wait(bar_qfull(0), 0, abort_flag, status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                if (leader) mma_ss(tmem_S, dK_k + off, dQ_k + off, IDESC_ST, kk > 0);
            }
            if (leader) mma_commit(bar_s);
            for (int j = 0; j < n_iter; ++j) {
                const int s = j & 1;
                const uint32_t ph = j & 1;
                const uint64_t so = s ? STAGE : 0;
                // dP^T(j) = V dO^T  (its columns hold dQ(j-1) until the drain warps have read it)
                mbar_wait(bar_dofull, ph, abort_flag, status);
                if (j > 0) mbar_wait(bar_drained, (j - 1) & 1, abort_flag, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                    if (leader) mma_ss(tmem_P, dV_k + off, dDO_k + off, IDESC_ST, kk > 0);
                }
                if (leader) mma_commit(bar_dp);
                // dV(j) += P^T dO
                mbar_wait(bar_p, ph, abort_flag, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk)
                    if (leader) mma_ts(tmem_dV, tmem_S + (kk >> 2) * 64 + (kk & 3) * 8, dDO_mn + (uint64_t)(kk * 128), IDESC_KV,
                           (j > 0) || (kk > 0));
                if (leader) mma_commit(bar_dofree);
                // S^T(j+1) = K Q^T
                if (j + 1 < n_iter) {
                    const uint64_t so1 = s ? 0 : STAGE;
                    mbar_wait(bar_qfull(s ^ 1), ((j + 1) >> 1) & 1, abort_flag, status);
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < D / 16; ++kk) {
                        const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                        if (leader) mma_ss(tmem_S, dK_k + off, dQ_k + so1 + off, IDESC_ST, kk > 0);
                    }
                    if (leader) mma_commit(bar_s);
                }
                // dQ(j) = dS K, then dK(j) += dS^T Q.  Both read dS from shared memory: the same swizzled buffer
                // is the MN-major A operand of dQ (queries contiguous) and, read as [keys x queries] rows, the
                // K-major A operand of dK; dQ goes first so that the drain can start while dK still runs.
                mbar_wait(bar_dss, ph, abort_flag, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk)
                    if (leader) mma_ss(tmem_P, dDS_mn + (uint64_t)(kk * 128), dK_mn + (uint64_t)(kk * 128), IDESC_DQ, kk > 0);
                if (leader) mma_commit(bar_dq);
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                    if (leader) mma_ss(tmem_dK, dDS_k + off, dQ_mn + so + (uint64_t)(kk * 128), IDESC_KV, (j > 0) || (kk > 0));
                }
                if (leader) mma_commit(bar_qfree(s));
            }
        }
    } else if (warp >= 8) {
        // ================= drain warps: dQ(j), query rows on lanes =================
        reg_inc<136>();
        const int quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
        uint8_t* stg_row = sgen + L::OFF_STG + row * 128;
        for (int j = 0; j < n_iter; ++j) {
            const int h = g * G + j / nm;
            const int m = m_first + j % nm;
            mbar_wait(bar_dq, j & 1, abort_flag, status);
            tc_fence_after();
            uint32_t r[D];
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                uint32_t t[32];
                tmem_ld32(tmem_P + lane_sel + ch * 32, t);
#pragma unroll
                for (int e = 0; e < 32; ++e) r[ch * 32 + e] = t[e];
            }
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_drained);      // the columns may be overwritten from here on
            // chunks of 32 head-dim columns through two staging buffers
#pragma unroll
            for (int ch = 0; ch < D / 32; ++ch) {
                const int buf = ch & 1;
                if (tid == 256) bulk_wait_read<1>();      // the reduce that last read this buffer has finished reading
                named_bar_sync(1, 128);
#pragma unroll
                for (int c = 0; c < 8; ++c)
                    *reinterpret_cast<uint4*>(stg_row + buf * L::STG_BYTES + ((c ^ (row & 7)) << 4)) =
                        make_uint4(r[ch * 32 + c * 4], r[ch * 32 + c * 4 + 1], r[ch * 32 + c * 4 + 2], r[ch * 32 + c * 4 + 3]);
                fence_proxy_async();
                named_bar_sync(1, 128);
                if (tid == 256) {
                    tma_reduce_add_3d(&tm_dq, ch * 32, h, tok0 + m * TILE, sSTG + buf * L::STG_BYTES);
                    bulk_commit();
                }
            }
        }
        if (tid == 256) bulk_wait<0>();
    } else {
        // ================= compute warps =================
        reg_inc<144>();
        const int quad = warp & 3;
        const int half = warp >> 2;
        const int row = quad * 32 + lane;                  // TMEM lane: key row of S^T, dP^T
        const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
        const int col0 = half * 64;                        // this thread's 64 query columns
        const int kj = n * TILE + row;
        const int my_ev = (kj < T) ? mv.evict[tok0 + kj] : 0;          // 0: visible to nobody
        const int my_first = (general && kj < T) ? mv.kfirst[tok0 + kj] : kj;   // first query that may see this key slot
        const bool key_tail = (n * TILE + TILE > T);
        const uint8_t* cls_col = mv.tile_class + mv.cls_off[b] + n;   // class of (m, n) at cls_col[m * nb]
        const float* sLse = reinterpret_cast<const float*>(sgen + L::OFF_LSE);
        const float* sDv = reinterpret_cast<const float*>(sgen + L::OFF_DVEC);
        uint8_t* sDS_row = sgen + L::OFF_DS + half * BOX_BYTES + row * 128;
        float pv[64];
        int cls_next = cls_col[(size_t)m_first * nb];      // class of the tile of the next phase_p, fetched early

        auto phase_p = [&](int j) {        // P^T(j) = exp2(S^T * c - lse), masked
            const int s = j & 1;
            const int m = m_first + j % nm;
            const bool need_mask = (cls_next != KVS_CLASS_FULL) || key_tail || (m * TILE + TILE > T);
            if (j + 1 < n_iter) cls_next = cls_col[(size_t)(m_first + (j + 1) % nm) * nb];
            mbar_wait(bar_ldfull(s), (j >> 1) & 1, abort_flag, status);
            mbar_wait(bar_s, j & 1, abort_flag, status);
            tc_fence_after();
            const float4* l4 = reinterpret_cast<const float4*>(sLse + s * TILE + col0);
            uint32_t r0[32], r1[32];
            tmem_ld32(tmem_S + lane_sel + col0, r0);
            tmem_ld32(tmem_S + lane_sel + col0 + 32, r1);
            tmem_wait_ld();
            const float2 c2 = make_float2(p.scale_log2, p.scale_log2);
#pragma unroll
            for (int e4 = 0; e4 < 16; ++e4) {          // packed fp32x2 multiply-adds, then one ex2 per element
                const float4 l = l4[e4];
                const uint32_t* r = (e4 < 8) ? &r0[e4 * 4] : &r1[(e4 - 8) * 4];
                const float2 x01 = __ffma2_rn(make_float2(__uint_as_float(r[0]), __uint_as_float(r[1])), c2, make_float2(l.x, l.y));
                const float2 x23 = __ffma2_rn(make_float2(__uint_as_float(r[2]), __uint_as_float(r[3])), c2, make_float2(l.z, l.w));
                pv[e4 * 4 + 0] = fast_exp2(x01.x);
                pv[e4 * 4 + 1] = fast_exp2(x01.y);
                pv[e4 * 4 + 2] = fast_exp2(x23.x);
                pv[e4 * 4 + 3] = fast_exp2(x23.y);
            }
            if (need_mask) {
#pragma unroll
                for (int e = 0; e < 64; ++e) {
                    const int qi = m * TILE + col0 + e;
                    pv[e] = ((my_first <= qi) && (qi < my_ev) && (qi < T)) ? pv[e] : 0.f;
                }
            }
            uint32_t pk[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) pk[e] = pack_bf16(pv[2 * e], pv[2 * e + 1]);
            tmem_st32(tmem_S + lane_sel + col0, pk);       // 64 queries -> 32 packed columns at [col0, col0+32)
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p);
        };

        auto phase_ds = [&](int j) {       // dS^T(j) = P^T (scale dP^T - scale D)
            const int s = j & 1;
            mbar_wait(bar_dp, j & 1, abort_flag, status);
            tc_fence_after();
            const float4* d4 = reinterpret_cast<const float4*>(sDv + s * TILE + col0);
            uint32_t r0[32], r1[32];
            tmem_ld32(tmem_P + lane_sel + col0, r0);
            tmem_ld32(tmem_P + lane_sel + col0 + 32, r1);
            tmem_wait_ld();
            uint32_t dk_[32];
            const float2 sc2 = make_float2(p.scale, p.scale);
#pragma unroll
            for (int e4 = 0; e4 < 16; ++e4) {          // dS = P * (scale dP - scale D), two elements per instruction
                const float4 dd = d4[e4];
                const uint32_t* r = (e4 < 8) ? &r0[e4 * 4] : &r1[(e4 - 8) * 4];
                const float2 t01 = __ffma2_rn(make_float2(__uint_as_float(r[0]), __uint_as_float(r[1])), sc2, make_float2(dd.x, dd.y));
                const float2 t23 = __ffma2_rn(make_float2(__uint_as_float(r[2]), __uint_as_float(r[3])), sc2, make_float2(dd.z, dd.w));
                const float2 d01 = __fmul2_rn(make_float2(pv[e4 * 4 + 0], pv[e4 * 4 + 1]), t01);
                const float2 d23 = __fmul2_rn(make_float2(pv[e4 * 4 + 2], pv[e4 * 4 + 3]), t23);
                dk_[e4 * 2 + 0] = pack_bf16(d01.x, d01.y);
                dk_[e4 * 2 + 1] = pack_bf16(d23.x, d23.y);
            }
            // dS^T row -> shared memory, MN-major (queries contiguous), 128-byte swizzle: the 64 queries of
            // this half are the 128-byte row `row` of block `half`; 16-byte chunk c sits at (c ^ (row % 8))
#pragma unroll
            for (int c = 0; c < 8; ++c)
                *reinterpret_cast<uint4*>(sDS_row + ((c ^ (row & 7)) << 4)) =
                    make_uint4(dk_[c * 4], dk_[c * 4 + 1], dk_[c * 4 + 2], dk_[c * 4 + 3]);
            fence_proxy_async();                     // dS visible to the tensor core's reads of shared memory
            tc_fence_before();                       // orders this thread's reads of dP^T before the dQ MMA that overwrites it
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_dss);
        };

        phase_p(0);
        for (int j = 0; j < n_iter; ++j) {
            phase_ds(j);
            if (j + 1 < n_iter) phase_p(j + 1);
        }

        // ---- epilogue: dK, dV of this key block, once every MMA has completed ----
        mbar_wait(bar_qfree((n_iter - 1) & 1), ((n_iter - 1) >> 1) & 1, abort_flag, status);
        tc_fence_after();
        const bool kvalid = kj < T;
        const size_t orow = (size_t)(tok0 + kj) * (size_t)p.dkv_ts + (size_t)g * D + half * HALF_D;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const uint32_t src = (which == 0 ? tmem_dK : tmem_dV) + lane_sel + half * HALF_D;
            void* base = which == 0 ? p.dk : p.dv;
#pragma unroll
            for (int ch = 0; ch < HALF_D / 32; ++ch) {
                uint32_t r[32];
                tmem_ld32(src + ch * 32, r);
                tmem_wait_ld();
                if (kvalid) {
                    if (p.grad_fp32) {
                        float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + orow + ch * 32);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            dst[e] = make_float4(__uint_as_float(r[e * 4]), __uint_as_float(r[e * 4 + 1]), __uint_as_float(r[e * 4 + 2]),
                                                 __uint_as_float(r[e * 4 + 3]));
                    } else {
                        uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(base) + orow + ch * 32);
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            uint4 w;
                            w.x = pack_bf16(__uint_as_float(r[e * 8 + 0]), __uint_as_float(r[e * 8 + 1]));
                            w.y = pack_bf16(__uint_as_float(r[e * 8 + 2]), __uint_as_float(r[e * 8 + 3]));
                            w.z = pack_bf16(__uint_as_float(r[e * 8 + 4]), __uint_as_float(r[e * 8 + 5]));
                            w.w = pack_bf16(__uint_as_float(r[e * 8 + 6]), __uint_as_float(r[e * 8 + 7]));
                            dst[e] = w;
                        }
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 13) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

template <int D>
static int launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo,
                      const CUtensorMap& tdq, const MetaView& mv,
                      const BwdParams& p, const __nv_bfloat16* dout, const __nv_bfloat16* out, float* dvec, float* dq_acc, long long dq_ts,
                      WsHeader* hdr, int nb_cap, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1) {
    {
        const long long rows = (long long)p.total_tokens * p.Hq;
        const int rows_per_warp = (32 / (D / 8)) * DOT_ROWS;
        const long long warps = (rows + rows_per_warp - 1) / rows_per_warp;
        const int threads = 256;
        const long long blocks = (warps * 32 + threads - 1) / threads;
        if (blocks > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
        bwd_dot_kernel<D><<<(unsigned)(blocks > 0 ? blocks : 1), threads, 0, st>>>(dout, out, dvec, dq_acc, dq_ts, p.total_tokens, p.Hq, hdr);
    }
    auto kern = bwd_kernel<D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<D>::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    dim3 grid(nb_cap, p.Hkv, 1);
    if (ev0 && cudaEventRecord(ev0, st) != cudaSuccess) return KVS_ERR_CUDA;
    kern<<<grid, BWD_THREADS, BwdSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, tdo, tdq, mv, p);
    if (ev1 && cudaEventRecord(ev1, st) != cudaSuccess) return KVS_ERR_CUDA;
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

}  // namespace kvs

using namespace kvs;

extern "C" size_t kvs_attn_bwd_workspace_bytes(int total_tokens, int Hq, int Hkv, int head_dim, int grad_dtype) {
    if (total_tokens < 0 || Hq <= 0 || Hkv <= 0 || head_dim <= 0) return 0;
    if (grad_dtype != KVS_GRAD_BF16 && grad_dtype != KVS_GRAD_FP32) return 0;
    return bwd_ws_layout(total_tokens, Hq, head_dim, grad_dtype).total;
}

namespace {
// in_ts: elements between consecutive tokens of q and of k, v; g_ts: of dq and of dk, dv (0: tensors of their own)
int bwd_impl(const void* dout, const void* q, const void* k, const void* v, long long in_ts, const void* out, const float* lse,
             const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim,
             float softmax_scale, int grad_dtype, void* dq, void* dk, void* dv, long long g_ts, void* workspace,
             size_t workspace_bytes, kvs_stream_t stream, void* event_main_begin, void* event_main_end) {
    cudaEvent_t ev0 = (cudaEvent_t)event_main_begin, ev1 = (cudaEvent_t)event_main_end;
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || Hq > 65535) return KVS_ERR_UNSUPPORTED;
    if (grad_dtype != KVS_GRAD_BF16 && grad_dtype != KVS_GRAD_FP32) return KVS_ERR_INVALID_ARG;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    if (!dout || !q || !k || !v || !out || !lse || !meta_buf || !dq || !dk || !dv || !workspace) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)dout | (uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out | (uintptr_t)dq | (uintptr_t)dk | (uintptr_t)dv) & 15) != 0)
        return KVS_ERR_ALIGNMENT;
    if (((uintptr_t)lse & 3) != 0 || ((uintptr_t)workspace & 255) != 0 || ((uintptr_t)meta_buf & 255) != 0) return KVS_ERR_ALIGNMENT;
    if (softmax_scale < 0.f || softmax_scale != softmax_scale) return KVS_ERR_INVALID_ARG;
    const BwdWsLayout W = bwd_ws_layout(total_tokens, Hq, head_dim, grad_dtype);
    if (workspace_bytes < W.total) return KVS_ERR_WORKSPACE;
    int rc = check_device_sm100();
    if (rc != KVS_OK) return rc;
    const MetaLayout L = meta_layout(batch, total_tokens, max_seqlen);
    const MetaView mv = meta_view(meta_buf, L);
    CUtensorMap tq, tk, tv, tdo, tdq;
    if ((rc = make_tmap_thd(&tq, q, total_tokens, Hq, head_dim, TILE, in_ts)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tk, k, total_tokens, Hkv, head_dim, TILE, in_ts)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tv, v, total_tokens, Hkv, head_dim, TILE, in_ts)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tdo, dout, total_tokens, Hq, head_dim, TILE)) != KVS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)workspace;
    const size_t nq = (size_t)total_tokens * Hq * head_dim;
    BwdParams p;
    p.batch = batch;
    p.total_tokens = total_tokens;
    p.max_seqlen = max_seqlen < total_tokens ? max_seqlen : total_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = p.scale * 1.4426950408889634f;
    p.lse = lse;
    p.dvec = (const float*)(ws + W.dvec);
    // bf16 gradients: dq is accumulated in the workspace (contiguous) and cast into place afterwards;
    // fp32 gradients: straight into dq, whatever its token stride
    const long long dq_ts_out = g_ts > 0 ? g_ts : (long long)Hq * head_dim;
    float* dq_acc = grad_dtype == KVS_GRAD_FP32 ? (float*)dq : (float*)(ws + W.dq_acc);
    const long long dq_ts = grad_dtype == KVS_GRAD_FP32 ? dq_ts_out : (long long)Hq * head_dim;
    if ((rc = make_tmap_f32_thd(&tdq, dq_acc, total_tokens, Hq, head_dim, TILE, dq_ts)) != KVS_OK) return rc;
    p.dk = dk;
    p.dv = dv;
    p.dkv_ts = g_ts > 0 ? g_ts : (long long)Hkv * head_dim;
    p.grad_fp32 = grad_dtype == KVS_GRAD_FP32;
    p.status = &((WsHeader*)ws)->status;
    rc = head_dim == 64 ? launch_bwd<64>(tq, tk, tv, tdo, tdq, mv, p, (const __nv_bfloat16*)dout, (const __nv_bfloat16*)out, (float*)(ws + W.dvec),
                                         dq_acc, dq_ts, (WsHeader*)ws, L.nb_cap, st, ev0, ev1)
                        : launch_bwd<128>(tq, tk, tv, tdo, tdq, mv, p, (const __nv_bfloat16*)dout, (const __nv_bfloat16*)out,
                                          (float*)(ws + W.dvec), dq_acc, dq_ts, (WsHeader*)ws, L.nb_cap, st, ev0, ev1);
    if (rc != KVS_OK) return rc;
    if (grad_dtype == KVS_GRAD_BF16) {
        const size_t n4 = nq / 4;
        const size_t blocks = (n4 + 255) / 256;
        if (blocks > 0x7fffffffull) return KVS_ERR_UNSUPPORTED;
        bwd_cast_kernel<<<(unsigned)blocks, 256, 0, st>>>(dq_acc, (__nv_bfloat16*)dq, n4, Hq * head_dim, dq_ts_out);
        if (cudaGetLastError() != cudaSuccess) return KVS_ERR_CUDA;
    }
    return KVS_OK;
}
}  // namespace

extern "C" int kvs_attn_bwd_ex(const void* dout, const void* q, const void* k, const void* v, const void* out, const float* lse,
                               const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim,
                               float softmax_scale, int grad_dtype, void* dq, void* dk, void* dv, void* workspace,
                               size_t workspace_bytes, kvs_stream_t stream, void* event_main_begin, void* event_main_end) {
    return bwd_impl(dout, q, k, v, 0, out, lse, meta_buf, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, grad_dtype,
                    dq, dk, dv, 0, workspace, workspace_bytes, stream, event_main_begin, event_main_end);
}

extern "C" int kvs_attn_bwd_packed(const void* dout, const void* qkv, const void* out, const float* lse, const void* meta_buf,
                                   int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale,
                                   int grad_dtype, void* dqkv, void* workspace, size_t workspace_bytes, kvs_stream_t stream) {
    if (Hq <= 0 || Hkv <= 0 || head_dim <= 0) return KVS_ERR_INVALID_ARG;
    if (grad_dtype != KVS_GRAD_BF16 && grad_dtype != KVS_GRAD_FP32) return KVS_ERR_INVALID_ARG;
    if (total_tokens > 0 && batch > 0 && (!qkv || !dqkv)) return KVS_ERR_INVALID_ARG;
    const long long ts = (long long)(Hq + 2 * Hkv) * head_dim;
    const size_t gsz = grad_dtype == KVS_GRAD_FP32 ? 4 : 2;
    const char* in = (const char*)qkv;
    char* g = (char*)dqkv;
    return bwd_impl(dout, in, in + (size_t)Hq * head_dim * 2, in + (size_t)(Hq + Hkv) * head_dim * 2, ts, out, lse, meta_buf, batch,
                    total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, grad_dtype, g, g + (size_t)Hq * head_dim * gsz,
                    g + (size_t)(Hq + Hkv) * head_dim * gsz, ts, workspace, workspace_bytes, stream, nullptr, nullptr);
}

extern "C" int kvs_attn_bwd(const void* dout, const void* q, const void* k, const void* v, const void* out, const float* lse,
                            const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim,
                            float softmax_scale, int grad_dtype, void* dq, void* dk, void* dv, void* workspace,
                            size_t workspace_bytes, kvs_stream_t stream) {
    return kvs_attn_bwd_ex(dout, q, k, v, out, lse, meta_buf, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale,
                           grad_dtype, dq, dk, dv, workspace, workspace_bytes, stream, nullptr, nullptr);
}

