/*
 * kvs.h -- C ABI of the eviction-masked causal attention library (B200, sm_100a).
 *
 * The operation (Sec. 2, "KV-streams" paragraph; Fig. 2 caption): a rollout that was
 * compacted by evicting KV entries in the inference engine is trained on as ONE continuous
 * trace; the attention mask hides every evicted key from the queries that came after its
 * eviction, so one forward pass reproduces what the engine's cache held at every step.
 * Per key j the caller supplies the step evict_at[j] at which it left the cache; query i
 * reads key j of the same trace iff   j <= i < evict_at[j].
 * Positions are not reset by eviction (Sec. 2), so q and k are taken as given.
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.
 *   - The caller owns every buffer.  No entry point allocates or frees device memory unless
 *     its comment says so.
 *   - q, out, dout, dq : bf16 [total_tokens, Hq,  head_dim], contiguous ("thd")
 *     k, v, dk, dv     : bf16 [total_tokens, Hkv, head_dim], contiguous
 *     lse              : fp32 [Hq, total_tokens], natural log of sum_j exp(scale * q_i.k_j)
 *     evict_at         : int32 [total_tokens], TRACE-LOCAL coordinates; 2^31-1 = never
 *     cu_seqlens       : int32 [batch+1], cu_seqlens[0] = 0, cu_seqlens[batch] = total_tokens
 *   - Traces are packed back to back; the 128x128 tile grid of a trace starts at its first
 *     token.  Precondition: evict_at[j] > j (a key is visible at least to its own query).
 *   - All work is enqueued on `stream` and the call returns without synchronising, except
 *     where stated.  Return value: KVS_OK or a negative KVS_ERR_* code.  Argument errors are
 *     detected on the host before anything is launched.  Conditions only the device can see
 *     (a bad evict_at, a bounded wait that expired) are recorded in a status word inside
 *     meta_buf / workspace and read back with kvs_device_status().
 *   - Requires head_dim in {64, 128}, Hq % Hkv == 0, 16-byte aligned tensors.
 */
#ifndef KVS_H_
#define KVS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* kvs_stream_t;   /* a cudaStream_t */

#define KVS_OK                 0
#define KVS_ERR_INVALID_ARG   (-1)   /* null pointer, negative size, inconsistent dims        */
#define KVS_ERR_UNSUPPORTED   (-2)   /* head_dim not 64/128, Hq % Hkv != 0, device not sm_100 */
#define KVS_ERR_ALIGNMENT     (-3)   /* a tensor pointer is not 16-byte aligned               */
#define KVS_ERR_WORKSPACE     (-4)   /* meta_buf / workspace / arena too small                */
#define KVS_ERR_CUDA          (-5)   /* a CUDA runtime or driver call failed                  */
#define KVS_ERR_BAD_EVICT     (-6)   /* device saw evict_at[j] <= j or a malformed cu_seqlens */
#define KVS_ERR_TIMEOUT       (-7)   /* a bounded device-side wait expired                    */
#define KVS_ERR_BAD_META      (-8)   /* meta_buf was not produced for these dims              */

#define KVS_TILE        128          /* tile edge, queries and keys */
#define KVS_CLASS_EMPTY   0
#define KVS_CLASS_PARTIAL 1
#define KVS_CLASS_FULL    2

#define KVS_GRAD_BF16 0
#define KVS_GRAD_FP32 1

/* Text for an error code.  Never NULL. */
const char* kvs_strerror(int code);

/* Bytes needed for meta_buf.  Pure host arithmetic; 0 on invalid arguments. */
size_t kvs_mask_meta_bytes(int batch, int total_tokens, int max_seqlen);

/*
 * Compaction event log -> evict_at (Sec. 2: a compaction deletes a span of the context; the trainer
 * masks that span from then on).  events: int32 [n_events, 4] rows (trace, when, start, end), trace-local
 * token indices: at step `when` the keys [start, end) of that trace leave the cache.  evict_at
 * [total_tokens] is overwritten: 2^31-1 where no event applies, else the earliest `when`.  Spans are
 * clipped to their trace; rows naming a trace outside [0, batch) are ignored.  Whether the result
 * satisfies evict_at[j] > j is checked by kvs_mask_meta.
 */
int kvs_evict_at_from_events(const int32_t* events, int n_events, const int32_t* cu_seqlens,
                             int batch, int total_tokens, int32_t* evict_at, kvs_stream_t stream);

/*
 * Mask metadata (the tile classification that lets the attention kernels skip evicted spans;
 * the paper states only that the deleted span is masked, Sec. 2 -- the tiling is this
 * library's).  For every key block n of every trace: kmin/kmax of evict_at over its valid
 * keys.  For every (query block m, key block n):
 *     EMPTY   if k0 > q1 or q0 >= kmax[n]
 *     FULL    if k1 <= q0 and q1 < kmin[n]
 *     PARTIAL otherwise
 * (q0,q1 / k0,k1 = first,last valid token of the block).  Also builds, per query block, the
 * ascending list of its non-empty key blocks and, per key block, the last query block that
 * sees it, and keeps a copy of evict_at and cu_seqlens, so meta_buf is self-contained and
 * may be reused by every layer and head that shares (evict_at, cu_seqlens).
 * max_seqlen must be >= the longest trace.  meta_bytes >= kvs_mask_meta_bytes(...).
 */
int kvs_mask_meta(const int32_t* evict_at, const int32_t* cu_seqlens,
                  int batch, int total_tokens, int max_seqlen,
                  void* meta_buf, size_t meta_bytes, kvs_stream_t stream);

/*
 * Mask metadata for key slots that carry their own visibility interval: slot j of a trace holds a key
 * that query i of the trace may read iff  key_first[j] <= i < key_evict[j]  (both int32 [total_tokens],
 * trace-local).  kvs_mask_meta is the case key_first[j] = j.  Two uses:
 *   - token-level eviction (App. B.4): with the keys of a trace re-ordered by kvs_reorder_keys, the
 *     slots of a 128-slot block die at about the same time, so most tiles are FULL or EMPTY instead of
 *     PARTIAL; the attention calls then take k, v in the re-ordered slot order (kvs_permute_rows) and
 *     return dk, dv in that order;
 *   - any other visibility rule of this form, e.g. "visible from its eviction on" (key_first = evict_at,
 *     key_evict = never), the complement of the eviction mask within the causal one.
 * A slot may be visible to no query at all (key_first >= key_evict); a query row that sees no key gets
 * out = 0 and lse = -inf.  Per block the classes use min/max of both arrays:
 *     EMPTY if min key_first > q1 or q0 >= max key_evict;  FULL if max key_first <= q0 and q1 < min key_evict.
 */
int kvs_mask_meta_keys(const int32_t* key_first, const int32_t* key_evict, const int32_t* cu_seqlens,
                       int batch, int total_tokens, int max_seqlen,
                       void* meta_buf, size_t meta_bytes, kvs_stream_t stream);

/*
 * Key order for token-level eviction (App. B.4 "Turn-Wise Compaction" discusses token-level eviction):
 * attention does not depend on the order of its keys, so the keys of a trace may be stored in any order
 * as long as each carries its index and its eviction step.  Within every window of `window` consecutive
 * keys of a trace (1 <= window <= 4096) the keys are sorted by (evict_at, index).  Outputs, all int32
 * [total_tokens]: perm[s] = packed token index of the key that goes to slot s; key_first[s] = its
 * trace-local index; key_evict[s] = its evict_at.  With turn-aligned evictions the order does not change.
 */
int kvs_reorder_keys(const int32_t* evict_at, const int32_t* cu_seqlens, int batch, int total_tokens, int max_seqlen,
                     int window, int32_t* perm, int32_t* key_first, int32_t* key_evict, kvs_stream_t stream);

/*
 * Row permutation for tensors whose leading dimension is the packed token: rows of row_bytes bytes
 * (a multiple of 16).  inverse == 0: dst row s = src row perm[s] (k, v into slot order);
 * inverse != 0: dst row perm[s] = src row s (dk, dv back to token order).  src and dst must not overlap.
 */
int kvs_permute_rows(const void* src, const int32_t* perm, void* dst, long long n_rows, long long row_bytes,
                     int inverse, kvs_stream_t stream);

/*
 * Test/inspection hook: copies the classes and per-block min/max to HOST arrays and
 * SYNCHRONISES the stream.  tile_class_host: uint8, trace after trace, each trace a dense
 * row-major [nb x nb] matrix (nb = ceil(T_b/128); n > m is EMPTY).  kmin_host/kmax_host:
 * int32 [sum nb].  Any of the three may be NULL.  Returns the device status if it is set.
 */
int kvs_mask_meta_export(const void* meta_buf, int batch, const int32_t* cu_seqlens_host,
                         int total_tokens, int max_seqlen,
                         uint8_t* tile_class_host, int32_t* kmin_host, int32_t* kmax_host,
                         kvs_stream_t stream);

/*
 * Forward of the trainer-side attention (Sec. 2, "KV-streams" paragraph; Fig. 2 caption: one continuous
 * trace, the mask hides the deleted span, one forward pass reproduces the rollout's evictions):
 *           S_ij = scale * q_i.k_j over allowed j;  lse_i = log sum_j exp S_ij;
 *           out_i = sum_j exp(S_ij - lse_i) v_j.   Query head h reads KV head h / (Hq/Hkv).
 * EMPTY tiles are never loaded; element masks are evaluated on PARTIAL tiles only.
 * softmax_scale == 0 selects 1/sqrt(head_dim).  bf16 operands, fp32 accumulation.
 */
int kvs_attn_fwd(const void* q, const void* k, const void* v, const void* meta_buf,
                 int batch, int total_tokens, int max_seqlen,
                 int Hq, int Hkv, int head_dim, float softmax_scale,
                 void* out, float* lse, kvs_stream_t stream);

/*
 * Metadata for the keys the eviction mask no longer shows: slot j is visible to query i iff
 * key_evict[j] <= i, i.e. from its eviction step on, for good (kvs_mask_meta_keys with key_first =
 * key_evict and key_evict = never, without the caller having to build those arrays).  key_evict is the
 * evict_at of kvs_mask_meta, or the key_evict of re-ordered slots.  Together with the student's visible
 * keys these are exactly the causal keys of a query: what kvs_attn_fwd_dual needs for the teacher.
 */
int kvs_mask_meta_evicted(const int32_t* key_evict, const int32_t* cu_seqlens,
                          int batch, int total_tokens, int max_seqlen,
                          void* meta_buf, size_t meta_bytes, kvs_stream_t stream);

/*
 * Student and teacher forward of the self-distillation objective (App. D.3 "Training Objectives": the
 * student is conditioned under the eviction mask, the teacher is a full-context pass of the same model
 * on the same tokens).  Both use the same q, k, v:
 *     student:  kvs_attn_fwd's result under meta_student
 *     teacher:  attention over every key the student sees or has lost to eviction: with keys in token
 *               order that is plain causal attention over the trace
 * The teacher is not a second full pass: the forward runs once more over the evicted keys only
 * (meta_evicted, from kvs_mask_meta_evicted on the same evict_at / key_evict) and the two partial results
 * are merged row by row (lse = log(e^lse_a + e^lse_b), out = e^(lse_a - lse) out_a + e^(lse_b - lse) out_b),
 * so a (query, key) pair is scored twice only inside tiles that are PARTIAL for the student.
 * Arguments as kvs_attn_fwd, with one (out, lse) pair per stream, all four overwritten; the two pairs
 * must be distinct buffers.
 */
int kvs_attn_fwd_dual(const void* q, const void* k, const void* v, const void* meta_student, const void* meta_evicted,
                      int batch, int total_tokens, int max_seqlen,
                      int Hq, int Hkv, int head_dim, float softmax_scale,
                      void* out_student, float* lse_student, void* out_teacher, float* lse_teacher,
                      kvs_stream_t stream);

/*
 * Forward and backward on a packed projection output (the layout the QKV and its gradient GEMM work
 * on, so that no split / concatenation copy is needed around the attention):
 *     qkv, dqkv : [total_tokens, Hq + 2 Hkv, head_dim]; heads 0..Hq-1 are q, then Hkv heads of k, then v
 * qkv is bf16; dqkv is bf16 or fp32 (grad_dtype) and receives dq, dk, dv in the same head order.
 * Everything else (out, lse, dout, meta_buf, workspace, errors) as in kvs_attn_fwd / kvs_attn_bwd; the
 * workspace size is that of kvs_attn_bwd_workspace_bytes for the same dims.
 */
int kvs_attn_fwd_packed(const void* qkv, const void* meta_buf,
                        int batch, int total_tokens, int max_seqlen,
                        int Hq, int Hkv, int head_dim, float softmax_scale,
                        void* out, float* lse, kvs_stream_t stream);
int kvs_attn_bwd_packed(const void* dout, const void* qkv, const void* out, const float* lse, const void* meta_buf,
                        int batch, int total_tokens, int max_seqlen,
                        int Hq, int Hkv, int head_dim, float softmax_scale, int grad_dtype,
                        void* dqkv, void* workspace, size_t workspace_bytes, kvs_stream_t stream);

/*
 * Rotary position embedding of q and k (and, with inverse != 0, the transposed rotation that takes
 * gradients with respect to the rotated tensors back to the unrotated ones).  KV-streams keeps every
 * token's position under eviction (Sec. 2: only re-prefill compaction resets positions), so on one
 * continuous trace a token's rotation depends on its trace index alone.  Rotate-half convention:
 *     angle(t, c) = pos_t * theta_base^(-2c / head_dim),  c < head_dim / 2
 *     y[c] = x[c] cos - x[c + d/2] sin;   y[c + d/2] = x[c + d/2] cos + x[c] sin
 * q [total_tokens, Hq, head_dim], k [total_tokens, Hkv, head_dim], contiguous, bf16 (elem_dtype =
 * KVS_GRAD_BF16) or fp32 (KVS_GRAD_FP32); either may be NULL; q_out / k_out may alias q / k.
 * positions: int32 [total_tokens], or NULL for the trace-local index (cu_seqlens, batch then required).
 * Angles are formed in double precision, the rotation in fp32, one rounding to the output type.
 */
int kvs_rope_qk(const void* q, const void* k, const int32_t* positions, const int32_t* cu_seqlens,
                int batch, int total_tokens, int Hq, int Hkv, int head_dim, float theta_base,
                int elem_dtype, int inverse, void* q_out, void* k_out, kvs_stream_t stream);

/* Bytes needed for the backward workspace (row sums, fp32 dQ accumulator, status). */
size_t kvs_attn_bwd_workspace_bytes(int total_tokens, int Hq, int Hkv, int head_dim, int grad_dtype);

/*
 * Backward of the same operation (Sec. 2, "KV-streams" paragraph: the trainer trains on that one trace,
 * so the same mask governs the gradients; gradients of sum(out * dout)):
 *   D_i = dout_i.out_i;  P_ij = exp(S_ij - lse_i);  dP_ij = dout_i.v_j;  dS_ij = P_ij (dP_ij - D_i)
 *   dq_i = scale sum_j dS_ij k_j;  dk_j = scale sum_{h in group} sum_i dS_ij q_i;
 *   dv_j = sum_{h in group} sum_i P_ij dout_i
 * grad_dtype: KVS_GRAD_BF16 (dq/dk/dv are bf16) or KVS_GRAD_FP32 (they are fp32, same shapes).
 * dq is accumulated with fp32 atomics (last bits may differ run to run); dk, dv are
 * written once, in a fixed order.  The workspace is scratch: its contents after the call
 * are unspecified, and two calls sharing one workspace must not overlap on the device.
 */
int kvs_attn_bwd(const void* dout, const void* q, const void* k, const void* v,
                 const void* out, const float* lse, const void* meta_buf,
                 int batch, int total_tokens, int max_seqlen,
                 int Hq, int Hkv, int head_dim, float softmax_scale, int grad_dtype,
                 void* dq, void* dk, void* dv,
                 void* workspace, size_t workspace_bytes, kvs_stream_t stream);

/*
 * kvs_attn_bwd with two optional cudaEvent_t handles (may be NULL) that are recorded on
 * `stream` immediately before and after the main dQ/dK/dV kernel, so that a caller can time
 * that kernel apart from the row-sum pre-pass and the cast post-pass.
 */
int kvs_attn_bwd_ex(const void* dout, const void* q, const void* k, const void* v,
                    const void* out, const float* lse, const void* meta_buf,
                    int batch, int total_tokens, int max_seqlen,
                    int Hq, int Hkv, int head_dim, float softmax_scale, int grad_dtype,
                    void* dq, void* dk, void* dv,
                    void* workspace, size_t workspace_bytes, kvs_stream_t stream,
                    void* event_main_begin, void* event_main_end);

/*
 * Backward without any device allocation by anyone (no counterpart in the paper: it exists for
 * deployment).  Some callers cannot obtain device memory at call time: a runtime that handed the
 * whole HBM to its own pool at start-up (a later cudaMalloc fails), or a step loop that must not
 * pay the device-wide synchronisation cudaMalloc/cudaFree imply.  For them the scratch that
 * kvs_attn_bwd takes as `workspace` is a fixed array inside the library, of
 * 256 B + 4 B * KVS_NOALLOC_MAX_ROWS per GPU, resident on every GPU that loads the library.
 *   - Gradients are fp32 only (dq is accumulated in place, so it needs no scratch); otherwise the
 *     arguments and results are those of kvs_attn_bwd with KVS_GRAD_FP32.
 *   - total_tokens * Hq must not exceed KVS_NOALLOC_MAX_ROWS, else KVS_ERR_WORKSPACE is returned
 *     and nothing is launched.
 *   - The first call on a device looks up the array's device address (with that device current);
 *     make that first call outside any stream capture.  Later calls only launch.
 *   - All calls on a GPU share the one array, which keeps whatever the previous call left; this
 *     call overwrites everything it reads, so nothing needs clearing, but two calls whose kernels
 *     overlap on the GPU (different streams, or another process thread) race on it.
 *   - scratch_out (may be NULL) receives the array's device address, for kvs_device_status().
 * The call itself uses no cudaMalloc, cudaFree or other allocating routine.
 */
#define KVS_NOALLOC_MAX_ROWS (1 << 20)
int kvs_attn_bwd_noalloc(const void* dout, const void* q, const void* k, const void* v,
                         const void* out, const float* lse, const void* meta_buf,
                         int batch, int total_tokens, int max_seqlen,
                         int Hq, int Hkv, int head_dim, float softmax_scale,
                         float* dq, float* dk, float* dv,
                         void** scratch_out, kvs_stream_t stream);

/*
 * Reads the status word of a meta_buf or of a backward workspace.  SYNCHRONISES the stream.
 * Returns KVS_OK, the recorded KVS_ERR_* code, or KVS_ERR_CUDA.
 */
int kvs_device_status(const void* meta_or_workspace, kvs_stream_t stream);

/*
 * Self-test of the bounded device-side wait every kernel of the library uses (failure detection
 * without a fault: no trap, no endless loop).  Launches one CTA whose threads wait on a barrier that
 * needs `expected_arrivals` (1 or 2) arrivals while exactly one is made.  With 1 the wait completes and
 * *status_word (device int32) stays KVS_OK; with 2 it can never complete: after limit_clocks SM clocks
 * (at most 4e9) the first waiter records KVS_ERR_TIMEOUT there, all other waiters of the CTA fall
 * through, and the kernel returns normally, leaving the context usable.
 */
int kvs_selftest_bounded_wait(int32_t* status_word, int expected_arrivals, long long limit_clocks,
                              kvs_stream_t stream);

/* Bytes of device arena needed by kvs_attn_fwd_bwd_host for these dims. */
size_t kvs_host_arena_bytes(int batch, int total_tokens, int max_seqlen,
                            int Hq, int Hkv, int head_dim, int grad_dtype);

/*
 * How kvs_attn_fwd_bwd_host cuts a batch into ranges of traces (host arrays only, no CUDA call): range i covers
 * traces [range_traces[2 i], range_traces[2 i + 1]).  range_traces: host int32, room for 2 * batch entries.
 * The ranges are contiguous, in order, leave out only traces without tokens, are at most ceil(8 / Hkv) (and at most
 * batch), and none holds more than total_tokens / ranges + max_seqlen tokens.  Returns KVS_ERR_INVALID_ARG for a
 * malformed cu_seqlens.
 */
int kvs_host_chunk_plan(const int32_t* cu_seqlens_host, int batch, int total_tokens, int max_seqlen, int Hkv,
                        int32_t* range_traces, int* num_ranges);

/*
 * Whole path from HOST buffers (the call a trainer without device tensors makes): copies
 * evict_at, cu_seqlens, q, k, v, dout to the device arena, runs mask metadata, forward and
 * backward, copies out, lse, dq, dk, dv back, and SYNCHRONISES the stream.  Host buffers
 * should be page-locked for the copies to be asynchronous.  arena: device memory the caller
 * provides, >= kvs_host_arena_bytes(...), 256-byte aligned.  Returns the device status.
 * The work is pipelined over chunks of (a contiguous range of traces, one KV-head group), which are
 * independent: while one chunk's forward and backward run, the next chunk's inputs are uploaded and
 * the previous chunk's results downloaded, on two internal streams that (with their events) are
 * created on the first call on a device and reused by later calls until the process ends; no device
 * memory is allocated.  With Hkv >= 8 a chunk is one KV-head group over all tokens; with fewer KV
 * heads the batch is cut into ceil(8 / Hkv) trace ranges of about equal token counts (at most one per
 * trace), each with mask metadata of its own.  Calls on the same device take turns.  The arena holds
 * three chunks at a time, so it is smaller than the tensors when there are more than three.
 * cu_seqlens_host is checked on the host before anything is queued (KVS_ERR_INVALID_ARG).
 */
int kvs_attn_fwd_bwd_host(const int32_t* evict_at_host, const int32_t* cu_seqlens_host,
                          const void* q_host, const void* k_host, const void* v_host,
                          const void* dout_host,
                          int batch, int total_tokens, int max_seqlen,
                          int Hq, int Hkv, int head_dim, float softmax_scale, int grad_dtype,
                          void* out_host, float* lse_host,
                          void* dq_host, void* dk_host, void* dv_host,
                          void* arena, size_t arena_bytes, kvs_stream_t stream);

/* ------------------------------------------------------------------------------------------------
 * Rollout side (Sec. 1; Sec. 4 "Inference engine implementation"; App. B.3): the engine evicts KV
 * entries directly in its paged cache and keeps decoding on the same stream.  Pages hold page_size
 * tokens (16 in one engine, with turns padded to page multiples; 1 in the other):
 *   k_cache, v_cache : bf16 [num_pages, page_size, Hkv, head_dim]
 *   block_table      : int32 [num_seqs, max_pages], the pages of each sequence's LIVE cache, in order
 *   n_tokens         : int32 [num_seqs], live tokens (every page full except possibly the last)
 *   free_list        : int32 [4 + num_pages]: {top, status, -, -} then a stack of free page ids
 * Eviction removes whole pages from a table and returns them to the stack; the rows never move.
 * Decode attention reads exactly the pages a table names; it never sees a mask.  Device-side
 * failures (cache full, a range that is not whole pages) set the status word, read with
 * kvs_cache_status().  num_pages is the size of the cache: a table or stack entry outside
 * [0, num_pages) is never followed; it is recorded as KVS_ERR_INVALID_ARG (in the cache status word by
 * append/evict, in the workspace status word by decode attention, which then reads page 0 instead).
 * ---------------------------------------------------------------------------------------------- */
size_t kvs_cache_free_list_bytes(int num_pages);
/* All pages free, status OK. */
int kvs_cache_init(int32_t* free_list, int num_pages, kvs_stream_t stream);
/* Appends one token (k_new, v_new: bf16 [num_seqs, Hkv, head_dim]) to every sequence whose `active`
 * byte is non-zero (active == NULL: all), taking a page from the stack when the last one is full. */
int kvs_cache_append(const void* k_new, const void* v_new, const uint8_t* active,
                     int num_seqs, int Hkv, int head_dim, int page_size, int max_pages, int num_pages,
                     int32_t* block_table, int32_t* n_tokens, int32_t* free_list,
                     void* k_cache, void* v_cache, kvs_stream_t stream);
/* Physical eviction.  ranges: int32 [n_ranges, 3] rows (sequence, first_page_slot, n_pages) in
 * positions of the CURRENT table; the named table entries are removed (the rest keep their order),
 * n_tokens drops by n_pages * page_size, the pages go back on the stack. */
int kvs_cache_evict(const int32_t* ranges, int n_ranges, int num_seqs, int page_size, int max_pages, int num_pages,
                    int32_t* block_table, int32_t* n_tokens, int32_t* free_list, kvs_stream_t stream);
/* Reads the cache status word.  SYNCHRONISES the stream. */
int kvs_cache_status(const int32_t* free_list, int* free_pages_host, kvs_stream_t stream);
/* A split count that fills the GPU for this batch, and the workspace decode attention needs. */
int kvs_decode_num_splits(int num_seqs, int Hkv, int max_tokens);
size_t kvs_decode_workspace_bytes(int num_seqs, int Hq, int head_dim, int num_splits);
/*
 * One decode step: out[s,h] = softmax_j(scale * q[s,h].k_j) v_j over the live cache of sequence s
 * (query head h reads KV head h / (Hq/Hkv)), lse[s,h] = log sum_j exp(scale * q.k_j).
 * q, out: bf16 [num_seqs, Hq, head_dim]; lse: fp32 [num_seqs, Hq].  Hq/Hkv in {1,2,4,7,8}.
 * A sequence with no live token gets out = 0, lse = -inf.  Rows of the cache that no token was
 * written to (the tail of a sequence's last page) may hold anything, NaN included.
 * workspace: >= kvs_decode_workspace_bytes(...), 256-byte aligned; its first words are a
 * {magic, status} header that kvs_device_status() reads (a bounded device wait that expired).
 */
int kvs_decode_attn(const void* q, const void* k_cache, const void* v_cache,
                    const int32_t* block_table, const int32_t* n_tokens,
                    int num_seqs, int Hq, int Hkv, int head_dim, int page_size, int max_pages, int num_pages,
                    float softmax_scale, int num_splits, void* out, float* lse,
                    void* workspace, size_t workspace_bytes, kvs_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* KVS_H_ */
