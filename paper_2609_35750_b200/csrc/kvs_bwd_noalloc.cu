// Backward for callers that cannot allocate device memory: the scratch that kvs_attn_bwd takes as a
// caller-provided workspace lives here in a fixed device array that is part of the library image.
#include <mutex>

#include "kvs_common.cuh"

namespace {

// Room for the workspace header plus one fp32 row sum per (token, query head):
// total_tokens * Hq <= KVS_NOALLOC_MAX_ROWS.  Every GPU that loads the library holds these
// 4 MiB + 256 B until the process exits.
constexpr size_t kScratchBytes = 256 + sizeof(float) * (size_t)KVS_NOALLOC_MAX_ROWS;
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};   // device address of g_scratch, per device ordinal

// `g_scratch` named in host code is only a handle for the runtime, not a device address: the
// address the kernels need comes from cudaGetSymbolAddress, asked once per device while that
// device is current.
int scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return KVS_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || !p) return KVS_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return KVS_OK;
}

}  // namespace

extern "C" int kvs_attn_bwd_noalloc(const void* dout, const void* q, const void* k, const void* v, const void* out,
                                    const float* lse, const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq,
                                    int Hkv, int head_dim, float softmax_scale, float* dq, float* dk, float* dv,
                                    void** scratch_out, kvs_stream_t stream) {
    if (total_tokens < 0 || Hq <= 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    if ((long long)total_tokens * Hq > (long long)KVS_NOALLOC_MAX_ROWS) return KVS_ERR_WORKSPACE;
    const size_t need = kvs_attn_bwd_workspace_bytes(total_tokens, Hq, Hkv, head_dim, KVS_GRAD_FP32);
    if (need == 0) return KVS_ERR_INVALID_ARG;
    if (need > kScratchBytes) return KVS_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int rc = scratch_for_current_device(&scratch);
    if (rc != KVS_OK) return rc;
    if (scratch_out) *scratch_out = scratch;
    // Nothing in the scratch has to start at zero: the row-sum pass rewrites the header and every
    // row sum this call reads before the main kernel runs.
    return kvs_attn_bwd(dout, q, k, v, out, lse, meta_buf, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale,
                        KVS_GRAD_FP32, dq, dk, dv, scratch, kScratchBytes, stream);
}
