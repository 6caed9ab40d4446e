// Shared declarations of the CUDA sources: meta buffer layout, sm_100a PTX wrappers.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kvs.h"

namespace kvs {

constexpr int TILE = KVS_TILE;
constexpr uint32_t META_MAGIC = 0x4B565331u;  // "KVS1"
constexpr uint32_t WS_MAGIC = 0x4B565357u;    // "KVSW"

// ------------------------------------------------------------------------------------------
// meta buffer
// ------------------------------------------------------------------------------------------
struct MetaHeader {
    uint32_t magic;
    int32_t status;        // KVS_OK or a KVS_ERR_* recorded by a kernel
    int32_t batch;
    int32_t total_tokens;
    int32_t max_seqlen;
    int32_t nblk_total;    // sum over traces of ceil(T_b / 128), written on the device
    uint32_t ncls_total;   // sum over traces of nb^2
    int32_t general;       // 1: every key slot carries its own first visible query (kvs_mask_meta_keys); 0: slot j is key j
};

// Byte offsets of the arrays inside meta_buf; a pure function of the three sizes so that
// every entry point can recompute it.
struct MetaLayout {
    size_t blk_off, cls_off, seq_start, blk_trace, kmin, kmax, fmin, fmax, col_first, col_last, row_cnt, fwd_order, bwd_order, evict, kfirst,
        tile_class, row_list, total;
    int nb_cap;            // capacity in blocks
    size_t cls_cap;        // capacity in tiles
};

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

__host__ __device__ inline MetaLayout meta_layout(int batch, int total_tokens, int max_seqlen) {
    MetaLayout L;
    if (max_seqlen > total_tokens) max_seqlen = total_tokens;   // a trace cannot be longer than the batch
    long long nbmax = (max_seqlen + TILE - 1) / TILE;
    long long cap1 = (long long)batch * nbmax;
    long long cap2 = (long long)total_tokens / TILE + batch;
    long long nb_cap = cap1 < cap2 ? cap1 : cap2;
    if (nb_cap < 1) nb_cap = 1;
    // sum nb_b^2 <= nbmax * sum nb_b
    long long cls_cap = nb_cap * nbmax;
    if (cls_cap < 1) cls_cap = 1;
    L.nb_cap = (int)nb_cap;
    L.cls_cap = (size_t)cls_cap;
    size_t o = align_up(sizeof(MetaHeader), 256);
    L.blk_off = o;   o = align_up(o + sizeof(int32_t) * (batch + 1), 256);
    L.cls_off = o;   o = align_up(o + sizeof(uint32_t) * (batch + 1), 256);
    L.seq_start = o; o = align_up(o + sizeof(int32_t) * (batch + 1), 256);
    L.blk_trace = o; o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.kmin = o;      o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.kmax = o;      o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.fmin = o;      o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.fmax = o;      o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.col_first = o; o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.col_last = o;  o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.row_cnt = o;   o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.fwd_order = o; o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.bwd_order = o; o = align_up(o + sizeof(int32_t) * nb_cap, 256);
    L.evict = o;     o = align_up(o + sizeof(int32_t) * (size_t)(total_tokens > 0 ? total_tokens : 1), 256);
    L.kfirst = o;    o = align_up(o + sizeof(int32_t) * (size_t)(total_tokens > 0 ? total_tokens : 1), 256);
    L.tile_class = o; o = align_up(o + L.cls_cap, 256);
    L.row_list = o;  o = align_up(o + sizeof(uint16_t) * L.cls_cap, 256);
    L.total = o;
    return L;
}

// Typed view used by the kernels.
struct MetaView {
    MetaHeader* hdr;
    const int32_t* blk_off;     // [batch+1] first global block of each trace
    const uint32_t* cls_off;    // [batch+1] first tile of each trace's class matrix
    const int32_t* seq_start;   // [batch+1] copy of cu_seqlens
    const int32_t* blk_trace;   // [nblk] trace of a global block
    const int32_t* kmin;        // [nblk] min / max over the block's key slots of the eviction step
    const int32_t* kmax;        // [nblk]
    const int32_t* fmin;        // [nblk] min / max over the block's key slots of the first query that may see the slot
    const int32_t* fmax;        // [nblk]
    const int32_t* col_first;   // [nblk] first query block (trace local) that can see the key block
    const int32_t* col_last;    // [nblk] last query block (trace local) that sees the key block (< col_first: none does)
    const int32_t* row_cnt;     // [nblk] non-empty key blocks of a query block row
    const int32_t* fwd_order;   // [nblk] query blocks, heaviest first
    const int32_t* bwd_order;   // [nblk] key blocks, longest query range first
    const int32_t* evict;       // [total_tokens] eviction step of every key slot (copy of evict_at / key_evict)
    const int32_t* kfirst;      // [total_tokens] first query that may see the slot (general metadata only)
    const uint8_t* tile_class;  // [ncls]
    const uint16_t* row_list;   // [ncls] row m of trace b at cls_off[b] + m * nb
};

inline MetaView meta_view(const void* buf, const MetaLayout& L) {
    char* p = (char*)buf;
    MetaView v;
    v.hdr = (MetaHeader*)p;
    v.blk_off = (const int32_t*)(p + L.blk_off);
    v.cls_off = (const uint32_t*)(p + L.cls_off);
    v.seq_start = (const int32_t*)(p + L.seq_start);
    v.blk_trace = (const int32_t*)(p + L.blk_trace);
    v.kmin = (const int32_t*)(p + L.kmin);
    v.kmax = (const int32_t*)(p + L.kmax);
    v.fmin = (const int32_t*)(p + L.fmin);
    v.fmax = (const int32_t*)(p + L.fmax);
    v.col_first = (const int32_t*)(p + L.col_first);
    v.col_last = (const int32_t*)(p + L.col_last);
    v.row_cnt = (const int32_t*)(p + L.row_cnt);
    v.fwd_order = (const int32_t*)(p + L.fwd_order);
    v.bwd_order = (const int32_t*)(p + L.bwd_order);
    v.evict = (const int32_t*)(p + L.evict);
    v.kfirst = (const int32_t*)(p + L.kfirst);
    v.tile_class = (const uint8_t*)(p + L.tile_class);
    v.row_list = (const uint16_t*)(p + L.row_list);
    return v;
}

// backward workspace header
struct WsHeader {
    uint32_t magic;
    int32_t status;
    int32_t pad[2];
};

// Host helpers implemented in kvs_api.cu
// token_stride: elements between consecutive tokens (0: heads * head_dim, i.e. a tensor of its own; larger when the
// tensor is a slice of heads of a packed [tokens, all heads, head_dim] buffer)
int make_tmap_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows, long long token_stride = 0);
int make_tmap_f32_thd(CUtensorMap* map, const void* base, int total_tokens, int heads, int head_dim, int box_rows,
                      long long token_stride = 0);
// bf16 [rows, cols] as a 2-D tensor whose box is 64 columns of ONE row: the form TMA gather4 takes (four row
// coordinates per instruction), 128-byte swizzle
int make_tmap_rows(CUtensorMap* map, const void* base, int rows, int cols);
int check_device_sm100();

#ifdef __CUDACC__
// ------------------------------------------------------------------------------------------
// device: status
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void set_status(int32_t* status, int code) { atomicCAS(status, 0, code); }

// True when `hdr` is the header kvs_mask_meta wrote for exactly these sizes (max_seqlen already
// clamped to total_tokens, as kvs_mask_meta stores it).  The attention kernels test this before
// they read any index out of the buffer: a buffer built for other sizes has its arrays at other
// offsets, and one that was never built holds arbitrary indices.
__device__ __forceinline__ bool meta_matches(const MetaHeader* hdr, int batch, int total_tokens, int max_seqlen) {
    return hdr->magic == META_MAGIC && hdr->batch == batch && hdr->total_tokens == total_tokens &&
           hdr->max_seqlen == max_seqlen;
}

// ------------------------------------------------------------------------------------------
// device: PTX wrappers (sm_100a)
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}

// Bounded wait.  `abort_flag` is a CTA-shared word: once any wait of the CTA gives up, every
// later wait falls through at once, so the CTA still walks its normal barrier structure,
// finishes, frees its tensor memory and returns; the result is garbage and the status word
// says so.  The limit is about two seconds of SM clocks.
constexpr long long WAIT_LIMIT_CLOCKS = 4000000000LL;
// try_wait with a suspend-time hint: the warp sleeps in hardware until the phase completes or the
// hint (nanoseconds) runs out, instead of polling shared memory (polling by many warps takes issue
// slots and shared-memory cycles away from the MMA issuer and the tensor core's operand reads).
__device__ __forceinline__ uint32_t mbar_try_wait_hint(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok;
}
#ifndef KVS_WAIT_HINT_NS
#define KVS_WAIT_HINT_NS 20000u
#endif
__device__ __forceinline__ void mbar_wait_limit(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                                long long limit_clocks) {
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (true) {
        if (mbar_try_wait_hint(bar, parity, KVS_WAIT_HINT_NS)) return;
        if (*abort_flag) return;
        if (clock64() - t0 > limit_clocks) {
            *abort_flag = 1;
            set_status(status, KVS_ERR_TIMEOUT);
            return;
        }
    }
}
__device__ __forceinline__ void mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status) {
    mbar_wait_limit(bar, parity, abort_flag, status, WAIT_LIMIT_CLOCKS);
}

// Register re-balancing between warp groups (all four warps of a warp group execute it).
template <int N>
__device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(N)); }
template <int N>
__device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(N)); }

// TMA: 3-D tiled load, global -> shared of this CTA only, completion on an mbarrier.
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
        : "memory");
}
// TMA: 3-D tiled reduce-add, shared -> global (element type from the tensor map), bulk-group completion.
__device__ __forceinline__ void tma_reduce_add_3d(const CUtensorMap* map, int c0, int c1, int c2, uint32_t src) {
    asm volatile(
        "cp.reduce.async.bulk.tensor.3d.global.shared::cta.add.tile.bulk_group [%0, {%1, %2, %3}], [%4];"
        ::"l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(src)
        : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait() { asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
__device__ __forceinline__ void prefetch_tmap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

// Tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t smem_result, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_result), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// One lane of a converged warp.  The MMA warp keeps all 32 lanes in its loops and predicates the
// tcgen05 instructions on this: with warp-uniform control flow the descriptors and addresses stay
// in uniform registers, which is what those instructions read, so issuing one MMA takes a few
// instructions instead of a chain of vector-to-uniform moves.
__device__ __forceinline__ bool elect_one() {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok));
    return ok != 0;
}

// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// mbarrier arrives once every MMA issued so far by this thread has completed
__device__ __forceinline__ void mma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor, 128-byte swizzle, tile base 1024-byte aligned.
//   K-major  operand (rows = M or N index, 64 bf16 = 128 B per row): sbo = 1024 (8 rows), lbo unused.
//   MN-major operand (rows = K index, 64 bf16 of M/N per row): sbo = 1024 (8 K rows),
//                     lbo = byte distance to the next 64 M/N elements.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFF) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version for sm_100
    d |= (uint64_t)2 << 61;   // 128-byte swizzle
    return d;
}

// Instruction descriptor: bf16 x bf16 -> fp32, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n, int a_mn_major, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)a_mn_major << 15) | ((uint32_t)b_mn_major << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// TMEM <-> registers: 32 lanes x 32 consecutive columns, one row per thread of the warp.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr),
          "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);   // .x = lo (low 16 bits), .y = hi
    return *reinterpret_cast<uint32_t*>(&t);
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fmax3(float a, float b, float c) {
    float y;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
    return y;
}
#endif  // __CUDACC__

}  // namespace kvs
