// Backward: dQ, dK, dV of eviction-masked causal attention.
//
//   pre-pass   D_i = dout_i . out_i                         (one warp per (token, head))
//   main       one CTA per (key block n, KV head g); K and V tiles stay in shared memory;
//              loop over the G query heads of the group and over the contiguous range of
//              query blocks m = n .. col_last[n] that can see the key block:
//                TMA Q, dO tiles
//                tcgen05.mma  S^T  = K Q^T,  dP^T = V dO^T        (tensor memory, keys on lanes)
//                128 threads, one key row each: P^T = exp2(S^T*c - lse*log2e) (masked on
//                  PARTIAL tiles; the key's eviction step is a per-thread scalar),
//                  dS^T = P^T (dP^T - D); both -> bf16 in tensor memory (over S^T, dP^T),
//                  dS^T also -> shared memory (MN-major) for the dQ product
//                tcgen05.mma  dV += P^T dO,  dK += dS^T Q         (A from tensor memory)
//                tcgen05.mma  dQ  = dS K                          (into the S^T columns)
//                dQ tile -> fp32 atomics into the accumulator
//              epilogue: dK * scale, dV written once by their owner CTA
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
template <int D>
__global__ void bwd_dot_kernel(const __nv_bfloat16* __restrict__ dout, const __nv_bfloat16* __restrict__ out,
                               float* __restrict__ dvec, int total_tokens, int Hq, WsHeader* hdr) {
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        hdr->magic = WS_MAGIC;
        hdr->status = KVS_OK;
    }
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp >= (long long)total_tokens * Hq) return;
    const int tok = (int)(warp / Hq), h = (int)(warp % Hq);
    constexpr int PER = D / 32;     // 2 or 4 bf16 per lane
    const __nv_bfloat16* a = dout + (size_t)warp * D + lane * PER;
    const __nv_bfloat16* b = out + (size_t)warp * D + lane * PER;
    float acc = 0.f;
#pragma unroll
    for (int e = 0; e < PER; e += 2) {
        const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(a + e));
        const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(b + e));
        acc += x.x * y.x + x.y * y.y;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) dvec[(size_t)h * total_tokens + tok] = acc;
}

// ---- post-pass --------------------------------------------------------------------------------
__global__ void bwd_cast_kernel(const float* __restrict__ acc, __nv_bfloat16* __restrict__ dq, size_t n4) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n4) return;
    const float4 x = reinterpret_cast<const float4*>(acc)[i];
    uint2 w;
    w.x = pack_bf16(x.x, x.y);
    w.y = pack_bf16(x.z, x.w);
    reinterpret_cast<uint2*>(dq)[i] = w;
}

// ---- main -------------------------------------------------------------------------------------
template <int D>
struct BwdSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int OFF_K = 0;
    static constexpr int OFF_V = OFF_K + TILE_BYTES;
    static constexpr int OFF_Q = OFF_V + TILE_BYTES;
    static constexpr int OFF_DO = OFF_Q + TILE_BYTES;
    static constexpr int OFF_DS = OFF_DO + TILE_BYTES;          // 128 keys x 128 queries bf16
    static constexpr int OFF_LSE = OFF_DS + TILE * TILE * 2;
    static constexpr int OFF_DV = OFF_LSE + TILE * 4;
    static constexpr int OFF_BAR = OFF_DV + TILE * 4;
    static constexpr int TOTAL = OFF_BAR + 64;
    static constexpr int DYN_BYTES = TOTAL + 1024;
};

struct BwdParams {
    int total_tokens, Hq, Hkv;
    float scale, scale_log2;
    const float* lse;
    const float* dvec;
    float* dq_acc;          // fp32 [Ttot, Hq, D], zeroed before the launch
    void* dk;
    void* dv;
    int grad_fp32;
    int32_t* status;
};

__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

template <int D>
__global__ void __launch_bounds__(128, 1)
bwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_do, MetaView mv, BwdParams p) {
    using L = BwdSmem<D>;
    constexpr int NBOX = D / 64;
    constexpr int BOX_BYTES = TILE * 128;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_ST = make_idesc(TILE, 0, 0);    // K-major x K-major, N = 128 queries
    constexpr uint32_t IDESC_KV = make_idesc(D, 0, 1);       // A from tensor memory, B MN-major, N = D
    constexpr uint32_t IDESC_DQ = make_idesc(D, 1, 1);       // A, B MN-major, N = D

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    if ((int)blockIdx.x >= mv.hdr->nblk_total) return;
    const int gb = blockIdx.x;
    const int g = blockIdx.y;
    const int G = p.Hq / p.Hkv;
    const int b = mv.blk_trace[gb];
    const int n = gb - mv.blk_off[b];
    const int tok0 = mv.seq_start[b];
    const int T = mv.seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    const int m_last = mv.col_last[gb];
    const uint8_t* cls_col = mv.tile_class + mv.cls_off[b] + n;   // class of (m, n) at cls_col[m * nb]
    int32_t* status = p.status;

    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t sK = sbase + L::OFF_K, sV = sbase + L::OFF_V, sQ = sbase + L::OFF_Q, sDO = sbase + L::OFF_DO,
                   sDS = sbase + L::OFF_DS;
    uint8_t* sDS_gen = sgen + L::OFF_DS;
    float* sLse = reinterpret_cast<float*>(sgen + L::OFF_LSE);
    float* sDv = reinterpret_cast<float*>(sgen + L::OFF_DV);
    const uint32_t bar_kv = sbase + L::OFF_BAR, bar_ld = bar_kv + 8, bar_s = bar_kv + 16, bar_a = bar_kv + 24, bar_q = bar_kv + 32;

    if (tid == 0) {
        s_abort = 0;
        mbar_init(bar_kv, 1);
        mbar_init(bar_ld, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_a, 1);
        mbar_init(bar_q, 1);
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
        prefetch_tmap(&tm_do);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    const uint32_t tmem_S = tmem;             // S^T fp32 [0,128) -> P^T bf16 [0,64); later dQ fp32 [0,D)
    const uint32_t tmem_P = tmem + 128;       // dP^T fp32 [128,256) -> dS^T bf16 [128,192)
    const uint32_t tmem_dV = tmem + 256;      // [256, 256+D)
    const uint32_t tmem_dK = tmem + 384;      // [384, 384+D)
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;
    volatile int* abort_flag = &s_abort;

    if (tid == 0) {
        mbar_expect_tx(bar_kv, 2 * L::TILE_BYTES);
        for (int c = 0; c < NBOX; ++c) tma_load_3d(sK + c * BOX_BYTES, &tm_k, c * 64, g, tok0 + n * TILE, bar_kv);
        for (int c = 0; c < NBOX; ++c) tma_load_3d(sV + c * BOX_BYTES, &tm_v, c * 64, g, tok0 + n * TILE, bar_kv);
    }

    const int kj = n * TILE + tid;                                     // this thread's key (trace local)
    const int my_ev = (kj < T) ? mv.evict[tok0 + kj] : 0;              // 0: visible to nobody
    const bool key_tail = (n * TILE + TILE > T);

    int it = 0;
    for (int hh = 0; hh < G; ++hh) {
        const int h = g * G + hh;
        for (int m = n; m <= m_last; ++m) {
            const int c = cls_col[(size_t)m * nb];
            if (c == KVS_CLASS_EMPTY) continue;
            const bool need_mask = (c != KVS_CLASS_FULL) || key_tail;
            const uint32_t ph = it & 1;
            const int qtok = tok0 + m * TILE;
            if (tid == 0) {
                mbar_expect_tx(bar_ld, 2 * L::TILE_BYTES);
                for (int cc = 0; cc < NBOX; ++cc) tma_load_3d(sQ + cc * BOX_BYTES, &tm_q, cc * 64, h, qtok, bar_ld);
                for (int cc = 0; cc < NBOX; ++cc) tma_load_3d(sDO + cc * BOX_BYTES, &tm_do, cc * 64, h, qtok, bar_ld);
            }
            {
                const int qi = m * TILE + tid;
                const bool qv = qi < T;
                // +inf makes P vanish for the rows past the end of the trace
                sLse[tid] = qv ? p.lse[(size_t)h * p.total_tokens + qtok + tid] * 1.4426950408889634f : INFINITY;
                sDv[tid] = qv ? p.dvec[(size_t)h * p.total_tokens + qtok + tid] : 0.f;
            }
            if (tid == 0) {
                if (it == 0) mbar_wait(bar_kv, 0, abort_flag, status);
                mbar_wait(bar_ld, ph, abort_flag, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * BOX_BYTES + (kk & 3) * 32;
                    mma_ss(tmem_S, smem_desc(sK + off, 16, 1024), smem_desc(sQ + off, 16, 1024), IDESC_ST, kk > 0);
                }
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint32_t off = (kk >> 2) * BOX_BYTES + (kk & 3) * 32;
                    mma_ss(tmem_P, smem_desc(sV + off, 16, 1024), smem_desc(sDO + off, 16, 1024), IDESC_ST, kk > 0);
                }
                mma_commit(bar_s);
            }
            __syncthreads();                      // sLse / sDv visible
            mbar_wait(bar_s, ph, abort_flag, status);
            tc_fence_after();

            // ---- this thread's key row: 128 queries in 4 chunks of 32 ---------------------------
#pragma unroll
            for (int ch = 0; ch < TILE / 32; ++ch) {
                uint32_t rs[32], rp[32];
                tmem_ld32(tmem_S + lane_sel + ch * 32, rs);
                tmem_ld32(tmem_P + lane_sel + ch * 32, rp);
                tmem_wait_ld();
                uint32_t pk[16], dk_[16];
#pragma unroll
                for (int e = 0; e < 32; e += 2) {
                    float pv[2], dsv[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const int col = ch * 32 + e + u;
                        float pr = fast_exp2(__uint_as_float(rs[e + u]) * p.scale_log2 - sLse[col]);
                        if (need_mask) {
                            const int qi = m * TILE + col;
                            const bool ok = (kj <= qi) && (qi < my_ev);
                            pr = ok ? pr : 0.f;
                        }
                        pv[u] = pr;
                        dsv[u] = pr * (__uint_as_float(rp[e + u]) - sDv[col]);
                    }
                    pk[e >> 1] = pack_bf16(pv[0], pv[1]);
                    dk_[e >> 1] = pack_bf16(dsv[0], dsv[1]);
                }
                // bf16 P^T / dS^T over the fp32 columns already consumed
                tmem_st16(tmem_S + lane_sel + ch * 16, pk);
                tmem_st16(tmem_P + lane_sel + ch * 16, dk_);
                // dS^T row -> shared memory, MN-major (queries contiguous), 128-byte swizzle:
                // 16-byte chunk q of this key row lives in block q/8, row tid, position (q%8) ^ (tid%8)
#pragma unroll
                for (int v4 = 0; v4 < 4; ++v4) {
                    const int q16 = ch * 4 + v4;                    // 16-byte chunk index, 0..15
                    const uint32_t off = (q16 >> 3) * BOX_BYTES + tid * 128 + (((q16 & 7) ^ (tid & 7)) << 4);
                    *reinterpret_cast<uint4*>(sDS_gen + off) = make_uint4(dk_[v4 * 4], dk_[v4 * 4 + 1], dk_[v4 * 4 + 2], dk_[v4 * 4 + 3]);
                }
            }
            tmem_wait_st();
            fence_proxy_async();
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk) {     // contraction over 16 queries per step
                    mma_ts(tmem_dV, tmem_S + kk * 8, smem_desc(sDO + kk * 2048, BOX_BYTES, 1024), IDESC_KV, (it > 0) || (kk > 0));
                }
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk) {
                    mma_ts(tmem_dK, tmem_P + kk * 8, smem_desc(sQ + kk * 2048, BOX_BYTES, 1024), IDESC_KV, (it > 0) || (kk > 0));
                }
                mma_commit(bar_a);
                mbar_wait(bar_a, ph, abort_flag, status);     // P^T consumed before dQ overwrites its columns
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk) {     // contraction over 16 keys per step
                    mma_ss(tmem_S, smem_desc(sDS + kk * 2048, BOX_BYTES, 1024), smem_desc(sK + kk * 2048, BOX_BYTES, 1024),
                           IDESC_DQ, kk > 0);
                }
                mma_commit(bar_q);
            }
            mbar_wait(bar_q, ph, abort_flag, status);
            tc_fence_after();
            // ---- dQ tile (query rows on lanes) -> fp32 atomics --------------------------------------
            {
                const int qi = m * TILE + tid;
                const bool qv = qi < T;
                float* dst = p.dq_acc + ((size_t)(qtok + tid) * p.Hq + h) * D;
#pragma unroll
                for (int ch = 0; ch < D / 32; ++ch) {
                    uint32_t r[32];
                    tmem_ld32(tmem_S + lane_sel + ch * 32, r);
                    tmem_wait_ld();
                    if (qv) {
#pragma unroll
                        for (int e = 0; e < 32; e += 4)
                            red_add_v4(dst + ch * 32 + e, __uint_as_float(r[e]) * p.scale, __uint_as_float(r[e + 1]) * p.scale,
                                       __uint_as_float(r[e + 2]) * p.scale, __uint_as_float(r[e + 3]) * p.scale);
                    }
                }
            }
            tc_fence_before();
            __syncthreads();                      // dQ columns, Q/dO/dS tiles and sLse free again
            ++it;
        }
    }
    if (it == 0 && tid == 0) mbar_wait(bar_kv, 0, abort_flag, status);   // drain the K/V load

    // ---- epilogue: dK, dV of this key block -----------------------------------------------------
    tc_fence_after();
    const bool kvalid = kj < T;
    const size_t orow = ((size_t)(tok0 + kj) * p.Hkv + g) * D;
#pragma unroll
    for (int which = 0; which < 2; ++which) {
        const uint32_t src = which == 0 ? tmem_dK : tmem_dV;
        const float mul = which == 0 ? p.scale : 1.f;
        void* base = which == 0 ? p.dk : p.dv;
#pragma unroll
        for (int ch = 0; ch < D / 32; ++ch) {
            uint32_t r[32];
            tmem_ld32(src + lane_sel + ch * 32, r);
            tmem_wait_ld();
            if (it == 0) {
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = 0u;
            }
            if (kvalid) {
                if (p.grad_fp32) {
                    float4* dst = reinterpret_cast<float4*>(reinterpret_cast<float*>(base) + orow + ch * 32);
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        dst[e] = make_float4(__uint_as_float(r[e * 4]) * mul, __uint_as_float(r[e * 4 + 1]) * mul,
                                             __uint_as_float(r[e * 4 + 2]) * mul, __uint_as_float(r[e * 4 + 3]) * mul);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(base) + orow + ch * 32);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(r[e * 8 + 0]) * mul, __uint_as_float(r[e * 8 + 1]) * mul);
                        w.y = pack_bf16(__uint_as_float(r[e * 8 + 2]) * mul, __uint_as_float(r[e * 8 + 3]) * mul);
                        w.z = pack_bf16(__uint_as_float(r[e * 8 + 4]) * mul, __uint_as_float(r[e * 8 + 5]) * mul);
                        w.w = pack_bf16(__uint_as_float(r[e * 8 + 6]) * mul, __uint_as_float(r[e * 8 + 7]) * mul);
                        dst[e] = w;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D>
static int launch_bwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const CUtensorMap& tdo, const MetaView& mv,
                      const BwdParams& p, const __nv_bfloat16* dout, const __nv_bfloat16* out, float* dvec, WsHeader* hdr,
                      int nb_cap, cudaStream_t st, cudaEvent_t ev0, cudaEvent_t ev1) {
    {
        const long long warps = (long long)p.total_tokens * p.Hq;
        const int threads = 256;
        const long long blocks = (warps * 32 + threads - 1) / threads;
        if (blocks > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
        bwd_dot_kernel<D><<<(unsigned)blocks, threads, 0, st>>>(dout, out, dvec, p.total_tokens, p.Hq, hdr);
    }
    auto kern = bwd_kernel<D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdSmem<D>::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    dim3 grid(nb_cap, p.Hkv, 1);
    if (ev0 && cudaEventRecord(ev0, st) != cudaSuccess) return KVS_ERR_CUDA;
    kern<<<grid, 128, BwdSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, tdo, mv, p);
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

extern "C" int kvs_attn_bwd_ex(const void* dout, const void* q, const void* k, const void* v, const void* out, const float* lse,
                               const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim,
                               float softmax_scale, int grad_dtype, void* dq, void* dk, void* dv, void* workspace,
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
    CUtensorMap tq, tk, tv, tdo;
    if ((rc = make_tmap_thd(&tq, q, total_tokens, Hq, head_dim, TILE)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tk, k, total_tokens, Hkv, head_dim, TILE)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tv, v, total_tokens, Hkv, head_dim, TILE)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tdo, dout, total_tokens, Hq, head_dim, TILE)) != KVS_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    char* ws = (char*)workspace;
    const size_t nq = (size_t)total_tokens * Hq * head_dim;
    BwdParams p;
    p.total_tokens = total_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    p.scale = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = p.scale * 1.4426950408889634f;
    p.lse = lse;
    p.dvec = (const float*)(ws + W.dvec);
    p.dq_acc = grad_dtype == KVS_GRAD_FP32 ? (float*)dq : (float*)(ws + W.dq_acc);
    p.dk = dk;
    p.dv = dv;
    p.grad_fp32 = grad_dtype == KVS_GRAD_FP32;
    p.status = &((WsHeader*)ws)->status;
    if (cudaMemsetAsync(p.dq_acc, 0, nq * sizeof(float), st) != cudaSuccess) return KVS_ERR_CUDA;
    rc = head_dim == 64 ? launch_bwd<64>(tq, tk, tv, tdo, mv, p, (const __nv_bfloat16*)dout, (const __nv_bfloat16*)out, (float*)(ws + W.dvec),
                                         (WsHeader*)ws, L.nb_cap, st, ev0, ev1)
                        : launch_bwd<128>(tq, tk, tv, tdo, mv, p, (const __nv_bfloat16*)dout, (const __nv_bfloat16*)out,
                                          (float*)(ws + W.dvec), (WsHeader*)ws, L.nb_cap, st, ev0, ev1);
    if (rc != KVS_OK) return rc;
    if (grad_dtype == KVS_GRAD_BF16) {
        const size_t n4 = nq / 4;
        const size_t blocks = (n4 + 255) / 256;
        if (blocks > 0x7fffffffull) return KVS_ERR_UNSUPPORTED;
        bwd_cast_kernel<<<(unsigned)blocks, 256, 0, st>>>(p.dq_acc, (__nv_bfloat16*)dq, n4);
        if (cudaGetLastError() != cudaSuccess) return KVS_ERR_CUDA;
    }
    return KVS_OK;
}

extern "C" int kvs_attn_bwd(const void* dout, const void* q, const void* k, const void* v, const void* out, const float* lse,
                            const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim,
                            float softmax_scale, int grad_dtype, void* dq, void* dk, void* dv, void* workspace,
                            size_t workspace_bytes, kvs_stream_t stream) {
    return kvs_attn_bwd_ex(dout, q, k, v, out, lse, meta_buf, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale,
                           grad_dtype, dq, dk, dv, workspace, workspace_bytes, stream, nullptr, nullptr);
}
