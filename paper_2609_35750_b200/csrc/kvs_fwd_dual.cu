// Student + teacher forward of the self-distillation objective (App. D.3 "Training Objectives"): the
// student attends under the eviction mask, the teacher sees the full causal context; same model, same
// tokens, same q, k, v.
//
// The causal key set of a query splits into the keys the student still sees and the keys that were
// evicted before the query.  Attention over a union of disjoint key sets is the merge of the attention
// over each: with lse = log(e^lse_a + e^lse_b),  out = e^(lse_a - lse) out_a + e^(lse_b - lse) out_b.
// So the teacher costs one more forward over the EVICTED keys only (metadata for key slots that become
// visible at their eviction step and stay, kvs_mask_meta_evicted) and one streaming merge: every
// (query, key) pair of a FULL or EMPTY tile is scored once for both streams, only tiles that are PARTIAL
// for the student are visited by both passes.  Both passes run the forward kernel as it is (two query
// heads of a group share every K/V tile).  A fused kernel with both accumulators of one head in tensor
// memory was measured first: 512 columns hold S twice and the two outputs of ONE head, so a CTA cannot
// keep two query tiles in flight, its eight softmax warps move through load / maximum / exponentials /
// store in lockstep and the special-function unit idles half the time; it was slower than two plain
// forwards and is not kept.
#include "kvs_common.cuh"

namespace kvs {

// One row = one (token, head): out_t = w_s out_s + w_c out_t(in) where out_t(in), lse_t(in) hold the result over the
// evicted keys.  16 bytes per lane and tensor, D / 8 lanes per row, MERGE_ROWS rows in flight per lane: HBM-bound.
constexpr int MERGE_ROWS = 4;
template <int D>
__global__ void __launch_bounds__(256)
dual_merge_kernel(const __nv_bfloat16* __restrict__ out_s, const float* __restrict__ lse_s, __nv_bfloat16* __restrict__ out_t,
                  float* __restrict__ lse_t, int total_tokens, int Hq) {
    constexpr int LPR = D / 8;
    constexpr int RPW = 32 / LPR;
    const long long rows = (long long)total_tokens * Hq;
    const long long gw = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, c = lane % LPR;
    const long long row0 = gw * (RPW * MERGE_ROWS) + sub;
    uint4 a[MERGE_ROWS], b[MERGE_ROWS];
    float la[MERGE_ROWS], lb[MERGE_ROWS];
#pragma unroll
    for (int r = 0; r < MERGE_ROWS; ++r) {
        const long long row = row0 + (long long)r * RPW;
        if (row < rows) {
            a[r] = *reinterpret_cast<const uint4*>(out_s + (size_t)row * D + c * 8);
            b[r] = *reinterpret_cast<const uint4*>(out_t + (size_t)row * D + c * 8);
            const size_t li = (size_t)(row % Hq) * total_tokens + (row / Hq);
            la[r] = lse_s[li];
            lb[r] = lse_t[li];
        } else {
            a[r] = b[r] = make_uint4(0, 0, 0, 0);
            la[r] = lb[r] = -INFINITY;
        }
    }
#pragma unroll
    for (int r = 0; r < MERGE_ROWS; ++r) {
        const long long row = row0 + (long long)r * RPW;
        if (row >= rows) continue;
        const float m = fmaxf(la[r], lb[r]);
        float wa = 0.f, wb = 0.f, lse = -INFINITY;
        if (m > -INFINITY) {
            const float ea = __expf(la[r] - m), eb = __expf(lb[r] - m);      // exp(-inf) = 0 for a part that saw no key
            const float sum = ea + eb;
            wa = ea / sum;
            wb = eb / sum;
            lse = m + logf(sum);
        }
        const uint32_t xa[4] = {a[r].x, a[r].y, a[r].z, a[r].w}, xb[4] = {b[r].x, b[r].y, b[r].z, b[r].w};
        uint32_t o[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float lo = wa * __uint_as_float(xa[e] << 16) + wb * __uint_as_float(xb[e] << 16);
            const float hi = wa * __uint_as_float(xa[e] & 0xffff0000u) + wb * __uint_as_float(xb[e] & 0xffff0000u);
            o[e] = pack_bf16(lo, hi);
        }
        *reinterpret_cast<uint4*>(out_t + (size_t)row * D + c * 8) = make_uint4(o[0], o[1], o[2], o[3]);
        if (c == 0) lse_t[(size_t)(row % Hq) * total_tokens + (row / Hq)] = lse;
    }
}

}  // namespace kvs

using namespace kvs;

extern "C" int kvs_attn_fwd_dual(const void* q, const void* k, const void* v, const void* meta_student, const void* meta_evicted,
                                 int batch, int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale,
                                 void* out_student, float* lse_student, void* out_teacher, float* lse_teacher, kvs_stream_t stream) {
    if (!meta_student || !meta_evicted) return KVS_ERR_INVALID_ARG;
    if (out_student == out_teacher || lse_student == lse_teacher) return KVS_ERR_INVALID_ARG;
    int rc = kvs_attn_fwd(q, k, v, meta_student, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, out_student,
                          lse_student, stream);
    if (rc != KVS_OK) return rc;
    // the part of the teacher's context that the student no longer sees, into the teacher's buffers
    rc = kvs_attn_fwd(q, k, v, meta_evicted, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, out_teacher,
                      lse_teacher, stream);
    if (rc != KVS_OK) return rc;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    const long long rows = (long long)total_tokens * Hq;
    const int rows_per_warp = (32 / (head_dim / 8)) * MERGE_ROWS;
    const long long warps = (rows + rows_per_warp - 1) / rows_per_warp;
    const long long blocks = (warps * 32 + 255) / 256;
    if (blocks > 0x7fffffffLL) return KVS_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    if (head_dim == 64)
        dual_merge_kernel<64><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)out_student, lse_student, (__nv_bfloat16*)out_teacher,
                                                               lse_teacher, total_tokens, Hq);
    else
        dual_merge_kernel<128><<<(unsigned)blocks, 256, 0, st>>>((const __nv_bfloat16*)out_student, lse_student, (__nv_bfloat16*)out_teacher,
                                                                lse_teacher, total_tokens, Hq);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}
