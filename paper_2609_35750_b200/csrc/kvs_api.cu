// Host glue shared by the entry points: error text, tensor maps, device check, status read.
#include <cudaTypedefs.h>

#include "kvs_common.cuh"
#include <mutex>
#include <vector>

namespace kvs {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    // looked up once (thread-safe static initialisation); the driver entry point never changes
    static const EncodeTiledFn fn = []() -> EncodeTiledFn {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess)
            return nullptr;
        return (EncodeTiledFn)ptr;
    }();
    return fn;
}

// bf16 [total_tokens, heads, head_dim] viewed as (head_dim, heads, tokens); box = 64 columns x
// 1 head x box_rows tokens, 128-byte swizzle, out-of-range rows read as zero.
int make_tmap_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows, long long token_stride) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KVS_ERR_CUDA;
    if (token_stride <= 0) token_stride = (long long)heads * head_dim;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)heads, (cuuint64_t)total_tokens};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 2, (cuuint64_t)token_stride * 2};
    cuuint32_t box[3] = {64, 1, (cuuint32_t)box_rows};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? KVS_OK : KVS_ERR_CUDA;
}

// fp32 [total_tokens, heads, head_dim] viewed as (head_dim, heads, tokens); box = 32 columns (128 bytes) x
// 1 head x box_rows tokens, 128-byte swizzle.  Used as the destination of TMA reduce-adds.
int make_tmap_f32_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows,
                      long long token_stride) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KVS_ERR_CUDA;
    if (token_stride <= 0) token_stride = (long long)heads * head_dim;
    cuuint64_t dims[3] = {(cuuint64_t)head_dim, (cuuint64_t)heads, (cuuint64_t)total_tokens};
    cuuint64_t strides[2] = {(cuuint64_t)head_dim * 4, (cuuint64_t)token_stride * 4};
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
// The work is cut into one chunk per KV head (its G query heads, all tokens): chunks are independent
// in the forward and the backward, so while chunk c computes, the inputs of chunk c+1 arrive and
// the results of chunk c-1 leave (PCIe is full duplex; two copy streams besides the caller's).
// Each chunk lives in one of HOST_SLOTS sets of contiguous [tokens, G, d] / [tokens, 1, d] buffers,
// packed and unpacked by strided 2-D copies; the kernels run on a chunk as on any (Hq = G, Hkv = 1) problem.
namespace {
constexpr int HOST_SLOTS = 3;
constexpr int kMaxHostDevices = 64;
struct HostPipe {
    cudaStream_t in = nullptr, outs = nullptr;
    std::vector<cudaEvent_t> ev;
};
std::mutex g_host_mu[kMaxHostDevices];
HostPipe g_host_pipe[kMaxHostDevices];
// A slot's workspace status is reset by the next chunk that uses the slot; the first failure is kept here.
__global__ void fold_status_kernel(const int32_t* ws_words, int32_t* sticky) {
    if (ws_words[1] != KVS_OK && *sticky == KVS_OK) *sticky = ws_words[1];
}
struct ArenaLayout {
    size_t evict, cu, sticky, meta, slot0, slot_stride, total;      // global part, then HOST_SLOTS equal slots
    size_t q, k, v, dout, out, lse, dq, dk, dv, ws;          // offsets inside a slot
    size_t meta_bytes, ws_bytes, nq_bytes, nkv_bytes, gq_bytes, gkv_bytes, lse_bytes;   // per chunk
    int slots;
};
ArenaLayout arena_layout(int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, int grad_dtype) {
    ArenaLayout A;
    const int G = Hq / Hkv;
    const size_t gsz = grad_dtype == KVS_GRAD_FP32 ? 4 : 2;
    A.slots = Hkv < HOST_SLOTS ? Hkv : HOST_SLOTS;
    A.nq_bytes = (size_t)total_tokens * G * head_dim * 2;
    A.nkv_bytes = (size_t)total_tokens * head_dim * 2;
    A.gq_bytes = (size_t)total_tokens * G * head_dim * gsz;
    A.gkv_bytes = (size_t)total_tokens * head_dim * gsz;
    A.lse_bytes = (size_t)total_tokens * G * 4;
    A.meta_bytes = kvs_mask_meta_bytes(batch, total_tokens, max_seqlen);
    A.ws_bytes = kvs_attn_bwd_workspace_bytes(total_tokens, G, 1, head_dim, grad_dtype);
    size_t o = 0;
    A.evict = o; o = align_up(o + (size_t)total_tokens * 4, 256);
    A.cu = o;    o = align_up(o + (size_t)(batch + 1) * 4, 256);
    A.sticky = o; o += 256;
    A.meta = o;  o = align_up(o + A.meta_bytes, 256);
    A.slot0 = o;
    size_t t = 0;
    A.q = t;     t = align_up(t + A.nq_bytes, 256);
    A.k = t;     t = align_up(t + A.nkv_bytes, 256);
    A.v = t;     t = align_up(t + A.nkv_bytes, 256);
    A.dout = t;  t = align_up(t + A.nq_bytes, 256);
    A.out = t;   t = align_up(t + A.nq_bytes, 256);
    A.lse = t;   t = align_up(t + A.lse_bytes, 256);
    A.dq = t;    t = align_up(t + A.gq_bytes, 256);
    A.dk = t;    t = align_up(t + A.gkv_bytes, 256);
    A.dv = t;    t = align_up(t + A.gkv_bytes, 256);
    A.ws = t;    t = align_up(t + A.ws_bytes, 256);
    A.slot_stride = t;
    A.total = A.slot0 + (size_t)A.slots * A.slot_stride;
    return A;
}
}  // namespace

extern "C" size_t kvs_host_arena_bytes(int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, int grad_dtype) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0 || head_dim <= 0) return 0;
    if (Hq % Hkv != 0) return 0;
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
    if (Hq % Hkv != 0 || Hkv > 1024) return KVS_ERR_UNSUPPORTED;
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
    const int G = Hq / Hkv;
    const int NC = Hkv;                                    // chunks
    const size_t gsz = grad_dtype == KVS_GRAD_FP32 ? 4 : 2;
    // Two copy streams and five events per chunk.  They belong to the device, not to the call: created the first time
    // the entry point runs on a device, reused by every later call (a trainer calls this once per layer and step) and
    // kept until the process ends.  Calls on one device take turns (each ends with a synchronisation anyway).
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxHostDevices) return KVS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_host_mu[dev]);
    HostPipe& R = g_host_pipe[dev];
    if (!R.in && cudaStreamCreateWithFlags(&R.in, cudaStreamNonBlocking) != cudaSuccess) return KVS_ERR_CUDA;
    if (!R.outs && cudaStreamCreateWithFlags(&R.outs, cudaStreamNonBlocking) != cudaSuccess) return KVS_ERR_CUDA;
    while (R.ev.size() < (size_t)NC * 5 + 1) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return KVS_ERR_CUDA;
        R.ev.push_back(e);
    }
    auto ev_qkv = [&](int c) { return R.ev[(size_t)c * 5 + 0]; };    // q, k, v of chunk c are on the device
    auto ev_dout = [&](int c) { return R.ev[(size_t)c * 5 + 1]; };   // dout of chunk c is on the device
    auto ev_fwd = [&](int c) { return R.ev[(size_t)c * 5 + 2]; };    // forward of chunk c done
    auto ev_bwd = [&](int c) { return R.ev[(size_t)c * 5 + 3]; };    // backward of chunk c done
    auto ev_down = [&](int c) { return R.ev[(size_t)c * 5 + 4]; };   // every result of chunk c is on the host
    cudaEvent_t ev_start = R.ev[(size_t)NC * 5];
#define KVS_CK(call) \
    if ((call) != cudaSuccess) return KVS_ERR_CUDA
    // rows of `width` bytes, `tokens` of them: host row pitch hp, device row pitch = width
    auto h2d = [&](cudaStream_t s_, void* dst, const void* src, size_t hoff, size_t hp, size_t width) {
        return cudaMemcpy2DAsync(dst, width, (const char*)src + hoff, hp, width, (size_t)total_tokens, cudaMemcpyHostToDevice, s_);
    };
    auto d2h = [&](cudaStream_t s_, void* dst, size_t hoff, size_t hp, const void* src, size_t width) {
        return cudaMemcpy2DAsync((char*)dst + hoff, hp, src, width, width, (size_t)total_tokens, cudaMemcpyDeviceToHost, s_);
    };
    KVS_CK(cudaMemcpyAsync(a + A.evict, evict_at_host, (size_t)total_tokens * 4, cudaMemcpyHostToDevice, st));
    KVS_CK(cudaMemcpyAsync(a + A.cu, cu_seqlens_host, (size_t)(batch + 1) * 4, cudaMemcpyHostToDevice, st));
    KVS_CK(cudaMemsetAsync(a + A.sticky, 0, 4, st));
    KVS_CK(cudaEventRecord(ev_start, st));                 // the copy streams start after what the caller queued before
    KVS_CK(cudaStreamWaitEvent(R.in, ev_start, 0));
    KVS_CK(cudaStreamWaitEvent(R.outs, ev_start, 0));
    int rc = kvs_mask_meta((const int32_t*)(a + A.evict), (const int32_t*)(a + A.cu), batch, total_tokens, max_seqlen, a + A.meta,
                           A.meta_bytes, stream);
    if (rc != KVS_OK) return rc;
    const size_t hq_pitch = (size_t)Hq * head_dim * 2, hkv_pitch = (size_t)Hkv * head_dim * 2;
    const size_t wq = (size_t)G * head_dim * 2, wkv = (size_t)head_dim * 2;
    const size_t gq_pitch = (size_t)Hq * head_dim * gsz, gkv_pitch = (size_t)Hkv * head_dim * gsz;
    const size_t wgq = (size_t)G * head_dim * gsz, wgkv = (size_t)head_dim * gsz;
    auto upload = [&](int c) -> int {
        char* sl = a + A.slot0 + (size_t)(c % A.slots) * A.slot_stride;
        if (c >= A.slots) KVS_CK(cudaStreamWaitEvent(R.in, ev_down(c - A.slots), 0));     // the slot's previous chunk is finished
        KVS_CK(h2d(R.in, sl + A.q, q_host, (size_t)c * wq, hq_pitch, wq));
        KVS_CK(h2d(R.in, sl + A.k, k_host, (size_t)c * wkv, hkv_pitch, wkv));
        KVS_CK(h2d(R.in, sl + A.v, v_host, (size_t)c * wkv, hkv_pitch, wkv));
        KVS_CK(cudaEventRecord(ev_qkv(c), R.in));
        KVS_CK(h2d(R.in, sl + A.dout, dout_host, (size_t)c * wq, hq_pitch, wq));
        KVS_CK(cudaEventRecord(ev_dout(c), R.in));
        return KVS_OK;
    };
    for (int c = 0; c < A.slots && c < NC; ++c)
        if ((rc = upload(c)) != KVS_OK) return rc;
    for (int c = 0; c < NC; ++c) {
        char* sl = a + A.slot0 + (size_t)(c % A.slots) * A.slot_stride;
        KVS_CK(cudaStreamWaitEvent(st, ev_qkv(c), 0));
        rc = kvs_attn_fwd(sl + A.q, sl + A.k, sl + A.v, a + A.meta, batch, total_tokens, max_seqlen, G, 1, head_dim, softmax_scale,
                          sl + A.out, (float*)(sl + A.lse), stream);
        if (rc != KVS_OK) return rc;
        KVS_CK(cudaEventRecord(ev_fwd(c), st));
        KVS_CK(cudaStreamWaitEvent(R.outs, ev_fwd(c), 0));
        KVS_CK(d2h(R.outs, out_host, (size_t)c * wq, hq_pitch, sl + A.out, wq));
        KVS_CK(cudaMemcpyAsync((char*)lse_host + (size_t)c * A.lse_bytes, sl + A.lse, A.lse_bytes, cudaMemcpyDeviceToHost, R.outs));
        KVS_CK(cudaStreamWaitEvent(st, ev_dout(c), 0));
        rc = kvs_attn_bwd(sl + A.dout, sl + A.q, sl + A.k, sl + A.v, sl + A.out, (const float*)(sl + A.lse), a + A.meta, batch,
                          total_tokens, max_seqlen, G, 1, head_dim, softmax_scale, grad_dtype, sl + A.dq, sl + A.dk, sl + A.dv,
                          sl + A.ws, A.ws_bytes, stream);
        if (rc != KVS_OK) return rc;
        fold_status_kernel<<<1, 1, 0, st>>>((const int32_t*)(sl + A.ws), (int32_t*)(a + A.sticky));
        KVS_CK(cudaEventRecord(ev_bwd(c), st));
        KVS_CK(cudaStreamWaitEvent(R.outs, ev_bwd(c), 0));
        KVS_CK(d2h(R.outs, dq_host, (size_t)c * wgq, gq_pitch, sl + A.dq, wgq));
        KVS_CK(d2h(R.outs, dk_host, (size_t)c * wgkv, gkv_pitch, sl + A.dk, wgkv));
        KVS_CK(d2h(R.outs, dv_host, (size_t)c * wgkv, gkv_pitch, sl + A.dv, wgkv));
        KVS_CK(cudaEventRecord(ev_down(c), R.outs));
        if (c + A.slots < NC && (rc = upload(c + A.slots)) != KVS_OK) return rc;
    }
    KVS_CK(cudaStreamWaitEvent(st, ev_down(NC - 1), 0));   // the caller's stream ends after every copy (the out stream is in order)
#undef KVS_CK
    // status words: the metadata buffer's (mask validation, forward) and the folded workspace status (backward)
    int32_t hm[2] = {0, 0}, hs = 0;
    if (cudaMemcpyAsync(hm, a + A.meta, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaMemcpyAsync(&hs, a + A.sticky, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    if (hm[1] != KVS_OK) return hm[1];
    if (hs != KVS_OK) return hs;
    return KVS_OK;
}
