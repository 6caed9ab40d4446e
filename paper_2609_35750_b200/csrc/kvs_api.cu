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

int make_tmap_rows(CUtensorMap* map, const void* base, int rows, int cols) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return KVS_ERR_CUDA;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
    cuuint32_t box[2] = {64, 1};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
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
// The work is cut into chunks of (a contiguous range of traces, one KV head with its G query heads): chunks are
// independent in the forward and the backward, so while chunk c computes, the inputs of chunk c+1 arrive and
// the results of chunk c-1 leave (PCIe is full duplex; two copy streams besides the caller's).  What cannot
// overlap is the first chunk's upload and the last chunk's download, so the batch is cut into as many trace
// ranges as it takes to have about HOST_TARGET_CHUNKS chunks.  Every range gets mask metadata of its own
// (its traces re-based to token 0).  Each chunk lives in one of HOST_SLOTS sets of contiguous
// [tokens, G, d] / [tokens, 1, d] buffers, packed and unpacked by strided 2-D copies; the kernels run on a
// chunk as on any (Hq = G, Hkv = 1) problem.
namespace {
#ifndef KVS_HOST_SLOTS
#define KVS_HOST_SLOTS 3
#endif
#ifndef KVS_HOST_CHUNKS
#define KVS_HOST_CHUNKS 8
#endif
constexpr int HOST_SLOTS = KVS_HOST_SLOTS;
constexpr int HOST_TARGET_CHUNKS = KVS_HOST_CHUNKS;
constexpr int kMaxHostDevices = 64;
struct HostPipe {
    cudaStream_t in = nullptr, outs = nullptr;
    std::vector<cudaEvent_t> ev;
    std::vector<int32_t> cu_ranges;          // re-based cu_seqlens of the trace ranges (staging for one upload)
};
std::mutex g_host_mu[kMaxHostDevices];
HostPipe g_host_pipe[kMaxHostDevices];

// A slot's workspace status and a range's metadata status are folded into one sticky word: one failure is kept.
__global__ void fold_status_kernel(const int32_t* words, int32_t* sticky) {
    if (words[1] != KVS_OK) atomicCAS(sticky, KVS_OK, words[1]);
}

inline int host_ranges(int batch, int Hkv) {
    int r = (HOST_TARGET_CHUNKS + Hkv - 1) / Hkv;
    if (r > batch) r = batch;
    return r < 1 ? 1 : r;
}

// A contiguous range of traces [b0, b1): its first token, token count, longest trace, and where its re-based
// cu_seqlens (b1 - b0 + 1 entries starting with 0) sit in the staging array.
struct Range { int b0, b1, tok0, tokens, maxlen, cu_off; };

// Cuts the batch into at most `want` contiguous ranges of traces: a range is closed once it holds its share
// ceil(total / want) of the tokens (so it exceeds the share by less than one trace) or when the traces left are
// only enough to give every remaining range one; the last range takes what is left.  Ranges without a token are dropped.
void plan_trace_ranges(const int32_t* cu, int batch, int total_tokens, int want, std::vector<Range>& ranges, std::vector<int32_t>& cu_ranges) {
    ranges.clear();
    cu_ranges.clear();
    if (want < 1) want = 1;
    const long long share = ((long long)total_tokens + want - 1) / want;
    int b = 0;
    while (b < batch) {
        Range r;
        r.b0 = b;
        r.tok0 = cu[b];
        r.maxlen = 0;
        r.cu_off = (int)cu_ranges.size();
        cu_ranges.push_back(0);
        const int left_ranges = want - (int)ranges.size();          // >= 1: the last one takes all that is left
        while (b < batch) {
            const int T = cu[b + 1] - cu[b];
            cu_ranges.push_back(cu[b + 1] - r.tok0);
            if (T > r.maxlen) r.maxlen = T;
            ++b;
            if (left_ranges > 1 && ((long long)cu[b] - r.tok0 >= share || batch - b <= left_ranges - 1)) break;
        }
        r.b1 = b;
        r.tokens = cu[b] - r.tok0;
        if (r.tokens > 0) ranges.push_back(r);
        else cu_ranges.resize(r.cu_off);
    }
}

struct ArenaLayout {
    size_t evict, cu, sticky, meta, slot0, slot_stride, total;      // global part, then HOST_SLOTS equal slots
    size_t q, k, v, dout, out, lse, dq, dk, dv, ws;                  // offsets inside a slot
    size_t meta_stride, ws_bytes;
    int slots, ranges, slot_tokens;
};
ArenaLayout arena_layout(int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, int grad_dtype) {
    ArenaLayout A;
    const int G = Hq / Hkv;
    const size_t gsz = grad_dtype == KVS_GRAD_FP32 ? 4 : 2;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    A.ranges = host_ranges(batch, Hkv);
    const long long nchunks = (long long)A.ranges * Hkv;
    A.slots = nchunks < HOST_SLOTS ? (int)nchunks : HOST_SLOTS;
    // a range is closed as soon as it holds its share of the tokens, so it exceeds the share by less than one trace
    long long st = (long long)total_tokens / A.ranges + max_seqlen;
    if (st > total_tokens) st = total_tokens;
    A.slot_tokens = (int)st;
    const size_t nq = (size_t)st * G * head_dim * 2, nkv = (size_t)st * head_dim * 2;
    const size_t gq = (size_t)st * G * head_dim * gsz, gkv = (size_t)st * head_dim * gsz;
    A.meta_stride = align_up(kvs_mask_meta_bytes(batch, A.slot_tokens, max_seqlen), 256);
    A.ws_bytes = kvs_attn_bwd_workspace_bytes(A.slot_tokens, G, 1, head_dim, grad_dtype);
    size_t o = 0;
    A.evict = o; o = align_up(o + (size_t)total_tokens * 4, 256);
    A.cu = o;    o = align_up(o + (size_t)(batch + A.ranges) * 4, 256);
    A.sticky = o; o += 256;
    A.meta = o;  o += (size_t)A.ranges * A.meta_stride;
    A.slot0 = o;
    size_t t = 0;
    A.q = t;     t = align_up(t + nq, 256);
    A.k = t;     t = align_up(t + nkv, 256);
    A.v = t;     t = align_up(t + nkv, 256);
    A.dout = t;  t = align_up(t + nq, 256);
    A.out = t;   t = align_up(t + nq, 256);
    A.lse = t;   t = align_up(t + (size_t)st * G * 4, 256);
    A.dq = t;    t = align_up(t + gq, 256);
    A.dk = t;    t = align_up(t + gkv, 256);
    A.dv = t;    t = align_up(t + gkv, 256);
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
    if (batch == 0 || total_tokens == 0) return 256;
    return arena_layout(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype).total;
}

extern "C" int kvs_host_chunk_plan(const int32_t* cu_seqlens_host, int batch, int total_tokens, int max_seqlen, int Hkv,
                                   int32_t* range_trace_begin, int* num_ranges) {
    if (!cu_seqlens_host || !range_trace_begin || !num_ranges || batch < 0 || total_tokens < 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    *num_ranges = 0;
    if (batch == 0 || total_tokens == 0) return KVS_OK;
    if (cu_seqlens_host[0] != 0 || cu_seqlens_host[batch] != total_tokens) return KVS_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        const long long T = (long long)cu_seqlens_host[b + 1] - cu_seqlens_host[b];
        if (T < 0 || T > max_seqlen) return KVS_ERR_INVALID_ARG;
    }
    std::vector<Range> ranges;
    std::vector<int32_t> cu_ranges;
    plan_trace_ranges(cu_seqlens_host, batch, total_tokens, host_ranges(batch, Hkv), ranges, cu_ranges);
    for (size_t i = 0; i < ranges.size(); ++i) {
        range_trace_begin[2 * i] = ranges[i].b0;
        range_trace_begin[2 * i + 1] = ranges[i].b1;
    }
    *num_ranges = (int)ranges.size();
    return KVS_OK;
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
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;
    // cu_seqlens is a host array here, so it can be checked before anything is queued
    if (cu_seqlens_host[0] != 0 || cu_seqlens_host[batch] != total_tokens) return KVS_ERR_INVALID_ARG;
    for (int b = 0; b < batch; ++b) {
        const long long T = (long long)cu_seqlens_host[b + 1] - cu_seqlens_host[b];
        if (T < 0 || T > max_seqlen) return KVS_ERR_INVALID_ARG;
    }
    const ArenaLayout A = arena_layout(batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, grad_dtype);
    if (arena_bytes < A.total) return KVS_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    char* a = (char*)arena;
    const int G = Hq / Hkv;
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

    std::vector<Range> ranges;
    plan_trace_ranges(cu_seqlens_host, batch, total_tokens, A.ranges, ranges, R.cu_ranges);
    const int NR = (int)ranges.size();
    for (const Range& r : ranges)
        if (r.tokens > A.slot_tokens) return KVS_ERR_WORKSPACE;      // cannot happen: see arena_layout
    const int NC = NR * Hkv;                                          // chunk c = (range c / Hkv, KV head c % Hkv)
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
    KVS_CK(cudaMemcpyAsync(a + A.evict, evict_at_host, (size_t)total_tokens * 4, cudaMemcpyHostToDevice, st));
    KVS_CK(cudaMemcpyAsync(a + A.cu, R.cu_ranges.data(), R.cu_ranges.size() * 4, cudaMemcpyHostToDevice, st));
    KVS_CK(cudaMemsetAsync(a + A.sticky, 0, 4, st));
    int rc = KVS_OK;
    for (int r = 0; r < NR; ++r) {
        const Range& g = ranges[r];
        char* meta = a + A.meta + (size_t)r * A.meta_stride;
        rc = kvs_mask_meta((const int32_t*)(a + A.evict) + g.tok0, (const int32_t*)(a + A.cu) + g.cu_off, g.b1 - g.b0, g.tokens, g.maxlen,
                           meta, A.meta_stride, stream);
        if (rc != KVS_OK) return rc;
    }
    KVS_CK(cudaEventRecord(ev_start, st));                 // the internal streams start after what the caller queued before
    KVS_CK(cudaStreamWaitEvent(R.in, ev_start, 0));
    KVS_CK(cudaStreamWaitEvent(R.outs, ev_start, 0));
    const size_t hq_pitch = (size_t)Hq * head_dim * 2, hkv_pitch = (size_t)Hkv * head_dim * 2;
    const size_t wq = (size_t)G * head_dim * 2, wkv = (size_t)head_dim * 2;
    const size_t gq_pitch = (size_t)Hq * head_dim * gsz, gkv_pitch = (size_t)Hkv * head_dim * gsz;
    const size_t wgq = (size_t)G * head_dim * gsz, wgkv = (size_t)head_dim * gsz;
    // rows of `width` bytes, one per token of the chunk's range: host row pitch hp, device row pitch = width
    auto h2d = [&](cudaStream_t s_, void* dst, const void* src, size_t hoff, size_t hp, size_t width, const Range& g) {
        return cudaMemcpy2DAsync(dst, width, (const char*)src + (size_t)g.tok0 * hp + hoff, hp, width, (size_t)g.tokens,
                                 cudaMemcpyHostToDevice, s_);
    };
    auto d2h = [&](cudaStream_t s_, void* dst, size_t hoff, size_t hp, const void* src, size_t width, const Range& g) {
        return cudaMemcpy2DAsync((char*)dst + (size_t)g.tok0 * hp + hoff, hp, src, width, width, (size_t)g.tokens,
                                 cudaMemcpyDeviceToHost, s_);
    };
    auto upload = [&](int c) -> int {
        const Range& g = ranges[c / Hkv];
        const int kh = c % Hkv;
        char* sl = a + A.slot0 + (size_t)(c % A.slots) * A.slot_stride;
        if (c >= A.slots) KVS_CK(cudaStreamWaitEvent(R.in, ev_down(c - A.slots), 0));     // the slot's previous chunk is finished
        KVS_CK(h2d(R.in, sl + A.q, q_host, (size_t)kh * wq, hq_pitch, wq, g));
        KVS_CK(h2d(R.in, sl + A.k, k_host, (size_t)kh * wkv, hkv_pitch, wkv, g));
        KVS_CK(h2d(R.in, sl + A.v, v_host, (size_t)kh * wkv, hkv_pitch, wkv, g));
        KVS_CK(cudaEventRecord(ev_qkv(c), R.in));
        KVS_CK(h2d(R.in, sl + A.dout, dout_host, (size_t)kh * wq, hq_pitch, wq, g));
        KVS_CK(cudaEventRecord(ev_dout(c), R.in));
        return KVS_OK;
    };
    for (int c = 0; c < A.slots && c < NC; ++c)
        if ((rc = upload(c)) != KVS_OK) return rc;
    for (int c = 0; c < NC; ++c) {
        const Range& g = ranges[c / Hkv];
        const int kh = c % Hkv, nb = g.b1 - g.b0;
        char* sl = a + A.slot0 + (size_t)(c % A.slots) * A.slot_stride;
        char* meta = a + A.meta + (size_t)(c / Hkv) * A.meta_stride;
        KVS_CK(cudaStreamWaitEvent(st, ev_qkv(c), 0));
        rc = kvs_attn_fwd(sl + A.q, sl + A.k, sl + A.v, meta, nb, g.tokens, g.maxlen, G, 1, head_dim, softmax_scale, sl + A.out,
                          (float*)(sl + A.lse), stream);
        if (rc != KVS_OK) return rc;
        KVS_CK(cudaEventRecord(ev_fwd(c), st));
        KVS_CK(cudaStreamWaitEvent(R.outs, ev_fwd(c), 0));
        KVS_CK(d2h(R.outs, out_host, (size_t)kh * wq, hq_pitch, sl + A.out, wq, g));
        // lse: G rows of the range's tokens, host rows total_tokens apart
        KVS_CK(cudaMemcpy2DAsync((char*)lse_host + ((size_t)kh * G * total_tokens + g.tok0) * 4, (size_t)total_tokens * 4, sl + A.lse,
                                 (size_t)g.tokens * 4, (size_t)g.tokens * 4, (size_t)G, cudaMemcpyDeviceToHost, R.outs));
        KVS_CK(cudaStreamWaitEvent(st, ev_dout(c), 0));
        rc = kvs_attn_bwd(sl + A.dout, sl + A.q, sl + A.k, sl + A.v, sl + A.out, (const float*)(sl + A.lse), meta, nb, g.tokens, g.maxlen,
                          G, 1, head_dim, softmax_scale, grad_dtype, sl + A.dq, sl + A.dk, sl + A.dv, sl + A.ws, A.ws_bytes, stream);
        if (rc != KVS_OK) return rc;
        fold_status_kernel<<<1, 1, 0, st>>>((const int32_t*)(sl + A.ws), (int32_t*)(a + A.sticky));
        if (kh == Hkv - 1) fold_status_kernel<<<1, 1, 0, st>>>((const int32_t*)meta, (int32_t*)(a + A.sticky));
        KVS_CK(cudaEventRecord(ev_bwd(c), st));
        KVS_CK(cudaStreamWaitEvent(R.outs, ev_bwd(c), 0));
        KVS_CK(d2h(R.outs, dq_host, (size_t)kh * wgq, gq_pitch, sl + A.dq, wgq, g));
        KVS_CK(d2h(R.outs, dk_host, (size_t)kh * wgkv, gkv_pitch, sl + A.dk, wgkv, g));
        KVS_CK(d2h(R.outs, dv_host, (size_t)kh * wgkv, gkv_pitch, sl + A.dv, wgkv, g));
        KVS_CK(cudaEventRecord(ev_down(c), R.outs));
        if (c + A.slots < NC && (rc = upload(c + A.slots)) != KVS_OK) return rc;
    }
    KVS_CK(cudaStreamWaitEvent(st, ev_down(NC - 1), 0));   // the caller's stream ends after every copy (the out stream is in order)
#undef KVS_CK
    // the sticky word holds the first failure of any range's metadata (mask validation, forward) or workspace (backward)
    int32_t hs = 0;
    if (cudaMemcpyAsync(&hs, a + A.sticky, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) return KVS_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return KVS_ERR_CUDA;
    return hs;
}
