// Rotary position embedding for q and k, and its transpose for their gradients.
//
// KV-streams keeps every token's position when entries are evicted (Sec. 2: retained entries keep their
// (k_i, v_i); only re-prefill compaction resets positions), so on one continuous trace the rotation of a
// token is a function of its index in the trace alone and can be applied once, before the attention, for
// all layers' kernels that follow.  Rotate-half convention: with d the head dimension, c < d/2 and
// angle(t, c) = pos_t * base^(-2c/d):
//     y[c]       = x[c] cos - x[c + d/2] sin
//     y[c + d/2] = x[c + d/2] cos + x[c] sin
// The gradient of a loss with respect to x is the same rotation by the opposite angle applied to the
// gradient with respect to y (`inverse`).
//
// Why this is a streaming pass and not part of the tile load: a K tile is loaded by every query block
// that sees it and a Q tile by every key block of the backward (about 70 times each on the keep-last-4
// configuration), so rotating inside the load would repeat the sine/cosine work that many times inside
// kernels that are already bound by their softmax and shared-memory traffic; the pass below touches each
// element once, at HBM speed, and is under one percent of a step.
#include "kvs_common.cuh"

namespace kvs {

constexpr int ROPE_THREADS = 256;
constexpr int ROPE_TOKENS = 8;      // tokens per CTA

// One CTA handles ROPE_TOKENS consecutive packed tokens: their cos/sin rows go to shared memory once (angles in
// double: pos * inv_freq reaches 1e5 rad, where fp32 would already be off by 1e-2), then every thread rotates 8-element
// chunks of all heads.  T: bf16 or float elements; rows = heads of one tensor.
template <typename T, int D>
__device__ __forceinline__ void rope_rows(const T* __restrict__ src, T* __restrict__ dst, int heads, int tok0, int ntok,
                                          const float (*cs)[D / 2][2]) {
    constexpr int HALF = D / 2;
    constexpr int CH = 16 / sizeof(T);                 // elements per 16-byte access: 8 bf16 or 4 fp32
    constexpr int CPR = HALF / CH;                     // chunks per half row
    const int total = ntok * heads * CPR;
    for (int i = threadIdx.x; i < total; i += ROPE_THREADS) {
        const int t = i / (heads * CPR);
        const int r = i % (heads * CPR);
        const int h = r / CPR, c0 = (r % CPR) * CH;
        const size_t base = ((size_t)(tok0 + t) * heads + h) * D;
        const uint4 lo4 = *reinterpret_cast<const uint4*>(src + base + c0);
        const uint4 hi4 = *reinterpret_cast<const uint4*>(src + base + HALF + c0);
        float lo[CH], hi[CH];
        if constexpr (sizeof(T) == 2) {
            const uint32_t a[4] = {lo4.x, lo4.y, lo4.z, lo4.w}, b[4] = {hi4.x, hi4.y, hi4.z, hi4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                lo[2 * e] = __uint_as_float(a[e] << 16);
                lo[2 * e + 1] = __uint_as_float(a[e] & 0xffff0000u);
                hi[2 * e] = __uint_as_float(b[e] << 16);
                hi[2 * e + 1] = __uint_as_float(b[e] & 0xffff0000u);
            }
        } else {
            lo[0] = __uint_as_float(lo4.x); lo[1] = __uint_as_float(lo4.y); lo[2] = __uint_as_float(lo4.z); lo[3] = __uint_as_float(lo4.w);
            hi[0] = __uint_as_float(hi4.x); hi[1] = __uint_as_float(hi4.y); hi[2] = __uint_as_float(hi4.z); hi[3] = __uint_as_float(hi4.w);
        }
        float ylo[CH], yhi[CH];
#pragma unroll
        for (int e = 0; e < CH; ++e) {
            const float c = cs[t][c0 + e][0], s = cs[t][c0 + e][1];
            ylo[e] = lo[e] * c - hi[e] * s;
            yhi[e] = hi[e] * c + lo[e] * s;
        }
        uint4 olo, ohi;
        if constexpr (sizeof(T) == 2) {
            olo = make_uint4(pack_bf16(ylo[0], ylo[1]), pack_bf16(ylo[2], ylo[3]), pack_bf16(ylo[4], ylo[5]), pack_bf16(ylo[6], ylo[7]));
            ohi = make_uint4(pack_bf16(yhi[0], yhi[1]), pack_bf16(yhi[2], yhi[3]), pack_bf16(yhi[4], yhi[5]), pack_bf16(yhi[6], yhi[7]));
        } else {
            olo = make_uint4(__float_as_uint(ylo[0]), __float_as_uint(ylo[1]), __float_as_uint(ylo[2]), __float_as_uint(ylo[3]));
            ohi = make_uint4(__float_as_uint(yhi[0]), __float_as_uint(yhi[1]), __float_as_uint(yhi[2]), __float_as_uint(yhi[3]));
        }
        *reinterpret_cast<uint4*>(dst + base + c0) = olo;
        *reinterpret_cast<uint4*>(dst + base + HALF + c0) = ohi;
    }
}

template <typename T, int D>
__global__ void __launch_bounds__(ROPE_THREADS)
rope_kernel(const T* __restrict__ q, const T* __restrict__ k, const int32_t* __restrict__ positions,
            const int32_t* __restrict__ cu_seqlens, int batch, int total_tokens, int Hq, int Hkv, double log_base, int inverse,
            T* __restrict__ q_out, T* __restrict__ k_out) {
    __shared__ float cs[ROPE_TOKENS][D / 2][2];
    const int tok0 = blockIdx.x * ROPE_TOKENS;
    const int ntok = min(ROPE_TOKENS, total_tokens - tok0);
    for (int i = threadIdx.x; i < ntok * (D / 2); i += ROPE_THREADS) {
        const int t = i / (D / 2), c = i % (D / 2);
        int pos;
        if (positions) {
            pos = positions[tok0 + t];
        } else {
            // trace-local index: the last trace whose first token is not after this one
            int lo = 0, hi = batch;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (cu_seqlens[mid] <= tok0 + t) lo = mid; else hi = mid;
            }
            pos = tok0 + t - cu_seqlens[lo];
        }
        const double inv_freq = exp(-log_base * (2.0 * c / D));
        double sn, cn;
        sincos((double)pos * inv_freq, &sn, &cn);
        cs[t][c][0] = (float)cn;
        cs[t][c][1] = (float)(inverse ? -sn : sn);
    }
    __syncthreads();
    if (q) rope_rows<T, D>(q, q_out, Hq, tok0, ntok, cs);
    if (k) rope_rows<T, D>(k, k_out, Hkv, tok0, ntok, cs);
}

template <typename T>
static int launch_rope(const void* q, const void* k, const int32_t* positions, const int32_t* cu, int batch, int total_tokens, int Hq,
                       int Hkv, int head_dim, double log_base, int inverse, void* q_out, void* k_out, cudaStream_t st) {
    const int grid = (total_tokens + ROPE_TOKENS - 1) / ROPE_TOKENS;
    if (head_dim == 64)
        rope_kernel<T, 64><<<grid, ROPE_THREADS, 0, st>>>((const T*)q, (const T*)k, positions, cu, batch, total_tokens, Hq, Hkv, log_base,
                                                         inverse, (T*)q_out, (T*)k_out);
    else
        rope_kernel<T, 128><<<grid, ROPE_THREADS, 0, st>>>((const T*)q, (const T*)k, positions, cu, batch, total_tokens, Hq, Hkv, log_base,
                                                          inverse, (T*)q_out, (T*)k_out);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

}  // namespace kvs

using namespace kvs;

extern "C" int kvs_rope_qk(const void* q, const void* k, const int32_t* positions, const int32_t* cu_seqlens, int batch,
                           int total_tokens, int Hq, int Hkv, int head_dim, float theta_base, int elem_dtype, int inverse,
                           void* q_out, void* k_out, kvs_stream_t stream) {
    if (batch < 0 || total_tokens < 0 || Hq < 0 || Hkv < 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (elem_dtype != KVS_GRAD_BF16 && elem_dtype != KVS_GRAD_FP32) return KVS_ERR_INVALID_ARG;
    if (!(theta_base > 1.f)) return KVS_ERR_INVALID_ARG;
    if (total_tokens == 0) return KVS_OK;
    if ((q && !q_out) || (k && !k_out) || (!q && !k)) return KVS_ERR_INVALID_ARG;
    if (!positions && (!cu_seqlens || batch < 1)) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)q_out | (uintptr_t)k_out) & 15) != 0) return KVS_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    const double log_base = log((double)theta_base);
    return elem_dtype == KVS_GRAD_BF16
               ? launch_rope<__nv_bfloat16>(q, k, positions, cu_seqlens, batch, total_tokens, Hq, Hkv, head_dim, log_base, inverse, q_out, k_out, st)
               : launch_rope<float>(q, k, positions, cu_seqlens, batch, total_tokens, Hq, Hkv, head_dim, log_base, inverse, q_out, k_out, st);
}
