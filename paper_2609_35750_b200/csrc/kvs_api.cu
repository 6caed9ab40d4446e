// Host glue shared by the entry points: error text, tensor maps, device check, status read.
#include <cudaTypedefs.h>

#include "kvs_common.cuh"

namespace kvs {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;   // looked up once; the driver entry point never changes
    if (!fn) {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        fn = (EncodeTiledFn)ptr;
    }
    return fn;
}

// bf16 [total_tokens, heads, head_dim] viewed as (head_dim, heads, tokens); box = 64 columns x
// 1 head x box_rows tokens, 128-byte swizzle, out-of-range rows read as zero.
int make_tmap_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KVS_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)heads, (cuuint64_t)total_tokens};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)heads * head_dim * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVS_OK : KVS_ERR_CUDA;
}

// fp32 [total_tokens, heads, head_dim] viewed as (head_dim, heads, tokens); box = 32 columns (128 bytes) x
// 1 head x box_rows tokens, 128-byte swizzle.  Used as the destination of TMA reduce-adds.
int make_tmap_f32_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KVS_ERR_CUDA;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)heads, (cuuint64_t)total_tokens};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 4, (cuuint64_t)heads * head_dim * 4};
    cuuint32_t box[3] = {32, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVS_OK : KVS_ERR_CUDA;
}

int check_device_sm100() {
    int dev = 0, major = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return KVS_ERR_CUDA;
    return major == 10 ? KVS_OK : KVS_ERR_UNSUPPORTED;
}

}  // namespace kvs

using namespace kvs;

extern "C" const char* kvs_strerror(int code) {
    switch (code) {
        case KVS_OK: return "ok";
        case KVS_ERR_INVALID_ARG: return "invalid argument";
        case KVS_ERR_UNSUPPORTED: return "unsupported configuration (head_dim must be 64 or 128, Hq % Hkv == 0, device sm_100)";
        case KVS_ERR_ALIGNMENT: return "pointer not sufficiently aligned";
        case KVS_ERR_WORKSPACE: return "meta buffer, workspace or arena too small";
        case KVS_ERR_CUDA: return "CUDA call failed";
        case KVS_ERR_BAD_EVICT: return "evict_at[j] <= j for some key, or malformed cu_seqlens";
        case KVS_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case KVS_ERR_BAD_META: return "meta buffer does not match these dimensions";
        default: return "unknown error code";
    }
}

extern "C" int kvs_device_status(const void* meta_or_workspace, kvs_stream_t stream) {
    if (!meta_or_workspace) return KVS_ERR_INVALID_ARG;
    // both headers start with {magic, status}
    int32_t h[2] = {0, 0};
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemcpyAsync(h, meta_or_workspace, sizeof(h), cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    if ((uint32_t)h[0] != META_MAGIC && (uint32_t)h[0] != WS_MAGIC) return KVS_ERR_BAD_META;
    return h[1];
}

// ---- self-test of the bounded wait ---------------------------------------------------------------
namespace kvs {
// One CTA waits on an mbarrier that expects `expected` arrivals while only thread 0 arrives once:
// with expected == 1 the wait completes; with expected == 2 nothing ever completes it, the wait gives
// up after `limit_clocks`, records KVS_ERR_TIMEOUT, and every other waiter of the CTA falls through.
__global__ void selftest_wait_kernel(int32_t* status, int expected, long long limit_clocks) {
    __shared__ __align__(8) unsigned long long s_bar;
    __shared__ int s_abort;
    const uint32_t bar = smem_u32(&s_bar);
    if (threadIdx.x == 0) {
        s_abort = 0;
        mbar_init(bar, (uint32_t)expected);
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) mbar_arrive(bar);
    mbar_wait_limit(bar, 0, &s_abort, status, limit_clocks);
    __syncthreads();
}
}  // namespace kvs

extern "C" int kvs_selftest_bounded_wait(int32_t* status_word, int expected_arrivals, long long limit_clocks, kvs_stream_t stream) {
    if (!status_word || expected_arrivals < 1 || expected_arrivals > 2 || limit_clocks <= 0 || limit_clocks > 4000000000LL)
        return KVS_ERR_INVALID_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    if (cudaMemsetAsync(status_word, 0, sizeof(int32_t), st) != cudaSuccess) return KVS_ERR_CUDA;
    selftest_wait_kernel<<<1, 128, 0, st>>>(status_word, expected_arrivals, limit_clocks);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

// ---- whole path from host buffers ------------------------------------------------------------
namespace {
struct ArenaLayout {
    size_t evict, cu, q, k, v, dout, out, lse, dq, dk, dv, meta, ws, total;
    size_t meta_bytes, ws_bytes, nq_bytes, nkv_bytes, gq_bytes, gkv_bytes, lse_bytes;
};
ArenaLayout arena_layout(int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, int grad_dtype) {
    ArenaLayout A;
    const size_t gsz = grad_dtype == KVS_GRAD_FP32 ? 4 : 2;
    A.nq_bytes = (size_t)total_tokens * Hq * head_dim * 2;
    A.nkv_bytes = (size_t)total_tokens * Hkv * head_dim * 2;
    A.gq_bytes = (size_t)total_tokens * Hq * head_dim * gsz;
    A.gkv_bytes = (size_t)total_tokens * Hkv * head_dim * gsz;
    A.lse_bytes = (size_t)total_tokens * Hq * 4;
    A.meta_bytes = kvs_mask_meta_bytes(batch, total_tokens, max_seqlen);
    A.ws_bytes = kvs_attn_bwd_workspace_bytes(total_tokens, Hq, Hkv, head_dim, grad_dtype);
    size_t o = 0;
    A.evict = o; o = align_up(o + (size_t)total_tokens * 4, 256);
    A.cu = o;    o = align_up(o + (size_t)(batch + 1) * 4, 256);
    A.q = o;     o = align_up(o + A.nq_bytes, 256);
    A.k = o;     o = align_up(o + A.nkv_bytes, 256);
    A.v = o;     o = align_up(o + A.nkv_bytes, 256);
    A.dout = o;  o = align_up(o + A.nq_bytes, 256);
    A.out = o;   o = align_up(o + A.nq_bytes, 256);
    A.lse = o;   o = align_up(o + A.lse_bytes, 256);
    A.dq = o;    o = align_up(o + A.gq_bytes, 256);
    A.dk = o;    o = align_up(o + A.gkv_bytes, 256);
    A.dv = o;    o = align_up(o + A.gkv_bytes, 256);
    A.meta = o;  o = align_up(o + A.meta_bytes, 256);
    A.ws = o;    o = align_up(o + A.ws_bytes, 256);
    A.total = o;
    return A;
}
}  // namespace

extern "C" size_t kvs_host_arena_bytes(int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, int grad_dtype) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0 || head_dim <= 0) return 0;
    if (grad_dtype != KVS_GRAD_BF16 && grad_dtype != KVS_GRAD_FP32) return 0;
    return arena_layout(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype).total;
}

extern "C" int kvs_attn_fwd_bwd_host(const int32_t* evict_at_host, const int32_t* cu_seqlens_host, const void* q_host,
                                     const void* k_host, const void* v_host, const void* dout_host, int batch, int total_tokens,
                                     int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale, int grad_dtype,
                                     void* out_host, float* lse_host, void* dq_host, void* dk_host, void* dv_host, void* arena,
                                     size_t arena_bytes, kvs_stream_t stream) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0) return KVS_ERR_UNSUPPORTED;
    if (grad_dtype != KVS_GRAD_BF16 && grad_dtype != KVS_GRAD_FP32) return KVS_ERR_INVALID_ARG;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    if (!evict_at_host || !cu_seqlens_host || !q_host || !k_host || !v_host || !dout_host || !out_host || !lse_host || !dq_host ||
        !dk_host || !dv_host || !arena)
        return KVS_ERR_INVALID_ARG;
    if (((uintptr_t)arena & 255) != 0) return KVS_ERR_ALIGNMENT;
    const ArenaLayout A = arena_layout(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype);
    if (arena_bytes < A.total) return KVS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* a = (char*)arena;
    // A second stream carries the copies that can overlap compute (PCIe is full duplex): dout goes in
    // while the forward runs, out and lse come back while the backward runs.  Stream and events live
    // for this call only.
    cudaStream_t cp = nullptr;
    cudaEvent_t ev_in = nullptr, ev_fwd = nullptr, ev_dout = nullptr, ev_out = nullptr;
    struct Cleanup {
        cudaStream_t& cp;
        cudaEvent_t &e0, &e1, &e2, &e3;
        ~Cleanup() {
            if (e0) cudaEventDestroy(e0);
            if (e1) cudaEventDestroy(e1);
            if (e2) cudaEventDestroy(e2);
            if (e3) cudaEventDestroy(e3);
            if (cp) cudaStreamDestroy(cp);
        }
    } cleanup{cp, ev_in, ev_fwd, ev_dout, ev_out};
    if (cudaStreamCreateWithFlags(&cp, cudaStreamNonBlocking) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaEventCreateWithFlags(&ev_in, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ev_fwd, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ev_dout, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&ev_out, cudaEventDisableTiming) != cudaSuccess)
        return KVS_ERR_CUDA;
#define KVS_CP(strm, dst, src, bytes, kind) \
    if (cudaMemcpyAsync(dst, src, bytes, kind, strm) != cudaSuccess) return KVS_ERR_CUDA
#define KVS_CK(call) \
    if ((call) != cudaSuccess) return KVS_ERR_CUDA
    KVS_CP(st, a + A.evict, evict_at_host, (size_t)total_tokens * 4, cudaMemcpyHostToDevice);
    KVS_CP(st, a + A.cu, cu_seqlens_host, (size_t)(batch + 1) * 4, cudaMemcpyHostToDevice);
    KVS_CP(st, a + A.q, q_host, A.nq_bytes, cudaMemcpyHostToDevice);
    KVS_CP(st, a + A.k, k_host, A.nkv_bytes, cudaMemcpyHostToDevice);
    KVS_CP(st, a + A.v, v_host, A.nkv_bytes, cudaMemcpyHostToDevice);
    KVS_CK(cudaEventRecord(ev_in, st));                       // dout follows q, k, v on the wire (they are needed first)
    KVS_CK(cudaStreamWaitEvent(cp, ev_in, 0));
    KVS_CP(cp, a + A.dout, dout_host, A.nq_bytes, cudaMemcpyHostToDevice);      // overlaps the forward
    KVS_CK(cudaEventRecord(ev_dout, cp));
    int rc = kvs_mask_meta((const int32_t*)(a + A.evict), (const int32_t*)(a + A.cu), batch, total_tokens, max_seqlen, a + A.meta,
                           A.meta_bytes, stream);
    if (rc != KVS_OK) return rc;
    rc = kvs_attn_fwd(a + A.q, a + A.k, a + A.v, a + A.meta, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale,
                      a + A.out, (float*)(a + A.lse), stream);
    if (rc != KVS_OK) return rc;
    KVS_CK(cudaEventRecord(ev_fwd, st));
    KVS_CK(cudaStreamWaitEvent(cp, ev_fwd, 0));
    KVS_CP(cp, out_host, a + A.out, A.nq_bytes, cudaMemcpyDeviceToHost);         // overlaps the backward
    KVS_CP(cp, lse_host, a + A.lse, A.lse_bytes, cudaMemcpyDeviceToHost);
    KVS_CK(cudaEventRecord(ev_out, cp));
    KVS_CK(cudaStreamWaitEvent(st, ev_dout, 0));
    rc = kvs_attn_bwd(a + A.dout, a + A.q, a + A.k, a + A.v, a + A.out, (const float*)(a + A.lse), a + A.meta, batch, total_tokens,
                      max_seqlen, Hq, Hkv, head_dim, softmax_scale, grad_dtype, a + A.dq, a + A.dk, a + A.dv, a + A.ws, A.ws_bytes,
                      stream);
    if (rc != KVS_OK) return rc;
    KVS_CP(st, dq_host, a + A.dq, A.gq_bytes, cudaMemcpyDeviceToHost);
    KVS_CP(st, dk_host, a + A.dk, A.gkv_bytes, cudaMemcpyDeviceToHost);
    KVS_CP(st, dv_host, a + A.dv, A.gkv_bytes, cudaMemcpyDeviceToHost);
    KVS_CK(cudaStreamWaitEvent(st, ev_out, 0));               // the caller's stream ends after every copy
#undef KVS_CP
#undef KVS_CK
    int32_t hm[2] = {0, 0}, hw[2] = {0, 0};
    if (cudaMemcpyAsync(hm, a + A.meta, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaMemcpyAsync(hw, a + A.ws, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    if (hm[1] != KVS_OK) return hm[1];
    return hw[1];
}
