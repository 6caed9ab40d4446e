// Forward: eviction-masked causal attention, one CTA per (query block, query head).
//
// Per CTA: the 128 x D query tile is staged once by TMA; the CTA walks the ascending list of
// non-empty key blocks of its row (EMPTY tiles are never touched).  Per key block:
//   TMA  K, V tiles -> shared memory (128-byte swizzle)
//   tcgen05.mma  S = Q K^T            (fp32, tensor memory columns [0,128))
//   128 threads, one query row each: scale, element mask on PARTIAL tiles only, online
//     softmax in registers (base-2), P -> bf16 written over S in tensor memory,
//     O rescaled in tensor memory when the running maximum moved
//   tcgen05.mma  O += P V             (P from tensor memory, V MN-major from shared memory)
// Epilogue: O / l -> bf16, LSE -> fp32.
#include "kvs_common.cuh"

namespace kvs {

template <int D>
struct FwdSmem {
    static constexpr int TILE_BYTES = TILE * D * 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = OFF_Q + TILE_BYTES;
    static constexpr int OFF_V = OFF_K + TILE_BYTES;
    static constexpr int OFF_EV = OFF_V + TILE_BYTES;
    static constexpr int OFF_BAR = OFF_EV + TILE * 4;
    static constexpr int TOTAL = OFF_BAR + 64;
    static constexpr int DYN_BYTES = TOTAL + 1024;   // slack for the 1024-byte alignment
};

struct FwdParams {
    int total_tokens, Hq, Hkv;
    float scale_log2;   // softmax_scale * log2(e)
    __nv_bfloat16* out;
    float* lse;
};

template <int D>
__global__ void __launch_bounds__(128, 2)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, MetaView mv, FwdParams p) {
    using L = FwdSmem<D>;
    constexpr int NBOX = D / 64;             // 64-column TMA boxes per tile row
    constexpr int BOX_BYTES = TILE * 128;    // 128 rows x 128 bytes
    constexpr uint32_t TMEM_COLS = 256;
    constexpr uint32_t IDESC_S = make_idesc(TILE, 0, 0);
    constexpr uint32_t IDESC_O = make_idesc(D, 0, 1);

    extern __shared__ uint8_t smem_raw[];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int nblk_total = mv.hdr->nblk_total;
    if ((int)blockIdx.x >= nblk_total) return;
    const int gb = mv.fwd_order[blockIdx.x];
    const int h = blockIdx.y;
    const int g = h / (p.Hq / p.Hkv);
    const int b = mv.blk_trace[gb];
    const int m = gb - mv.blk_off[b];
    const int tok0 = mv.seq_start[b];
    const int T = mv.seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    const int nlist = mv.row_cnt[gb];
    const uint16_t* list = mv.row_list + mv.cls_off[b] + (size_t)m * nb;
    const uint8_t* cls = mv.tile_class + mv.cls_off[b] + (size_t)m * nb;
    int32_t* status = &mv.hdr->status;

    const uint32_t sbase = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - smem_u32(smem_raw));
    const uint32_t sQ = sbase + L::OFF_Q, sK = sbase + L::OFF_K, sV = sbase + L::OFF_V;
    int32_t* sEv = reinterpret_cast<int32_t*>(sgen + L::OFF_EV);
    const uint32_t bar_q = sbase + L::OFF_BAR, bar_kv = bar_q + 8, bar_s = bar_q + 16, bar_o = bar_q + 24;

    if (tid == 0) {
        s_abort = 0;
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_s, 1);
        mbar_init(bar_o, 1);
        fence_mbar_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    if (warp == 0) {
        tmem_alloc(smem_u32(&s_tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem_base;
    const uint32_t tmem_S = tmem;            // columns [0,128): S fp32, then P bf16 in [0,64)
    const uint32_t tmem_O = tmem + 128;      // columns [128,128+D)
    const uint32_t lane_sel = (uint32_t)(warp * 32) << 16;   // this warp's 32 TMEM lanes

    if (tid == 0) {
        mbar_expect_tx(bar_q, L::TILE_BYTES);
        for (int c = 0; c < NBOX; ++c) tma_load_3d(sQ + c * BOX_BYTES, &tm_q, c * 64, h, tok0 + m * TILE, bar_q);
    }

    const int row = tid;                      // query row of the tile == TMEM lane
    const int qi = m * TILE + row;            // trace-local query index
    float run_max = -INFINITY;                // base-2 domain
    float run_sum = 0.f;
    volatile int* abort_flag = &s_abort;

    for (int t = 0; t < nlist; ++t) {
        const int n = list[t];
        const uint32_t ph = t & 1;
        const bool need_mask = (cls[n] != KVS_CLASS_FULL) || (n * TILE + TILE > T);
        if (tid == 0) {
            mbar_expect_tx(bar_kv, 2 * L::TILE_BYTES);
            for (int c = 0; c < NBOX; ++c) tma_load_3d(sK + c * BOX_BYTES, &tm_k, c * 64, g, tok0 + n * TILE, bar_kv);
            for (int c = 0; c < NBOX; ++c) tma_load_3d(sV + c * BOX_BYTES, &tm_v, c * 64, g, tok0 + n * TILE, bar_kv);
        }
        if (need_mask) {
            const int j = n * TILE + tid;
            sEv[tid] = (j < T) ? mv.evict[tok0 + j] : 0;   // 0: visible to nobody
        }
        if (tid == 0) {
            if (t == 0) mbar_wait(bar_q, 0, abort_flag, status);
            mbar_wait(bar_kv, ph, abort_flag, status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < D / 16; ++kk) {
                const uint32_t off = (kk >> 2) * BOX_BYTES + (kk & 3) * 32;
                mma_ss(tmem_S, smem_desc(sQ + off, 16, 1024), smem_desc(sK + off, 16, 1024), IDESC_S, kk > 0);
            }
            mma_commit(bar_s);
        }
        __syncthreads();                       // sEv visible; also keeps the warps together
        mbar_wait(bar_s, ph, abort_flag, status);
        tc_fence_after();

        // ---- softmax on this thread's row --------------------------------------------------
        float sv[TILE];
#pragma unroll
        for (int c = 0; c < TILE / 32; ++c) {
            uint32_t r[32];
            tmem_ld32(tmem_S + lane_sel + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int e = 0; e < 32; ++e) sv[c * 32 + e] = __uint_as_float(r[e]) * p.scale_log2;
        }
        if (need_mask) {
#pragma unroll
            for (int e = 0; e < TILE; ++e) {
                const int j = n * TILE + e;
                const bool ok = (j <= qi) && (qi < sEv[e]);
                sv[e] = ok ? sv[e] : -INFINITY;
            }
        }
        float tile_max = sv[0];
#pragma unroll
        for (int e = 1; e < TILE; ++e) tile_max = fmaxf(tile_max, sv[e]);
        const float new_max = fmaxf(run_max, tile_max);
        const float use_max = (new_max == -INFINITY) ? 0.f : new_max;
        const float alpha = fast_exp2(run_max - use_max);      // run_max = -inf -> 0
        float tile_sum = 0.f;
        uint32_t pk[TILE / 2];
#pragma unroll
        for (int e = 0; e < TILE; e += 2) {
            const float p0 = fast_exp2(sv[e] - use_max);
            const float p1 = fast_exp2(sv[e + 1] - use_max);
            tile_sum += p0 + p1;
            pk[e >> 1] = pack_bf16(p0, p1);
        }
        run_sum = run_sum * alpha + tile_sum;
        run_max = new_max;
        // P (bf16, 64 columns) over the S columns this thread has already read
#pragma unroll
        for (int c = 0; c < 2; ++c) {
            uint32_t r[32];
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = pk[c * 32 + e];
            tmem_st32(tmem_S + lane_sel + c * 32, r);
        }
        // rescale O when some row of the warp moved its maximum
        if (t > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_O + lane_sel + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st32(tmem_O + lane_sel + c * 32, r);
            }
        }
        tmem_wait_st();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < TILE / 16; ++kk) {
                // A: P rows, 16 keys = 8 packed columns per step.  B: V, MN-major, 16 key rows per step.
                mma_ts(tmem_O, tmem_S + kk * 8, smem_desc(sV + kk * 2048, BOX_BYTES, 1024), IDESC_O, (t > 0) || (kk > 0));
            }
            mma_commit(bar_o);
        }
        mbar_wait(bar_o, ph, abort_flag, status);   // K, V, P free again; O complete
        tc_fence_after();
    }

    // A row of blocks with no visible key block can only come from a bad evict_at (already
    // reported by the metadata pass): drain the Q load and write zeros.
    if (nlist == 0 && tid == 0) mbar_wait(bar_q, 0, abort_flag, status);

    // ---- epilogue ------------------------------------------------------------------------------
    const bool valid = qi < T;
    const float inv = (run_sum > 0.f && nlist > 0) ? 1.f / run_sum : 0.f;
    __nv_bfloat16* orow = p.out + ((size_t)(tok0 + qi) * p.Hq + h) * D;
#pragma unroll
    for (int c = 0; c < D / 32; ++c) {
        uint32_t r[32];
        tmem_ld32(tmem_O + lane_sel + c * 32, r);
        tmem_wait_ld();
        if (nlist == 0) {
#pragma unroll
            for (int e = 0; e < 32; ++e) r[e] = 0u;
        }
        if (valid) {
            uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                uint4 w;
                w.x = pack_bf16(__uint_as_float(r[e * 8 + 0]) * inv, __uint_as_float(r[e * 8 + 1]) * inv);
                w.y = pack_bf16(__uint_as_float(r[e * 8 + 2]) * inv, __uint_as_float(r[e * 8 + 3]) * inv);
                w.z = pack_bf16(__uint_as_float(r[e * 8 + 4]) * inv, __uint_as_float(r[e * 8 + 5]) * inv);
                w.w = pack_bf16(__uint_as_float(r[e * 8 + 6]) * inv, __uint_as_float(r[e * 8 + 7]) * inv);
                dst[e] = w;
            }
        }
    }
    if (valid) p.lse[(size_t)h * p.total_tokens + tok0 + qi] = run_max * 0.6931471805599453f + logf(run_sum);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, TMEM_COLS);
}

template <int D>
static int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const MetaView& mv, const FwdParams& p,
                      int nb_cap, cudaStream_t st) {
    auto kern = fwd_kernel<D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    dim3 grid(nb_cap, p.Hq, 1);
    kern<<<grid, 128, FwdSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, mv, p);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

}  // namespace kvs

using namespace kvs;

extern "C" int kvs_attn_fwd(const void* q, const void* k, const void* v, const void* meta_buf, int batch, int total_tokens,
                            int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale, void* out, float* lse,
                            kvs_stream_t stream) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || Hq > 65535) return KVS_ERR_UNSUPPORTED;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    if (!q || !k || !v || !meta_buf || !out || !lse) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15) != 0 || ((uintptr_t)lse & 3) != 0) return KVS_ERR_ALIGNMENT;
    if (((uintptr_t)meta_buf & 255) != 0) return KVS_ERR_ALIGNMENT;
    if (softmax_scale < 0.f || softmax_scale != softmax_scale) return KVS_ERR_INVALID_ARG;
    int rc = check_device_sm100();
    if (rc != KVS_OK) return rc;
    const MetaLayout L = meta_layout(batch, total_tokens, max_seqlen);
    const MetaView mv = meta_view(meta_buf, L);
    CUtensorMap tq, tk, tv;
    if ((rc = make_tmap_thd(&tq, q, total_tokens, Hq, head_dim, TILE)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tk, k, total_tokens, Hkv, head_dim, TILE)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tv, v, total_tokens, Hkv, head_dim, TILE)) != KVS_OK) return rc;
    FwdParams p;
    p.total_tokens = total_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    const float s = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = s * 1.4426950408889634f;
    p.out = (__nv_bfloat16*)out;
    p.lse = lse;
    cudaStream_t st = (cudaStream_t)stream;
    return head_dim == 64 ? launch_fwd<64>(tq, tk, tv, mv, p, L.nb_cap, st) : launch_fwd<128>(tq, tk, tv, mv, p, L.nb_cap, st);
}
