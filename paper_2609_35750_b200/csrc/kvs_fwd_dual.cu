// Student + teacher forward in one pass (self-distillation: App. D.3 "Training Objectives").
//
// The student attends under the eviction mask, the teacher sees the full causal context; same model,
// same tokens, so both use the same Q K^T.  One CTA per (query block, query head) walks every causal key
// block n = 0..m once: the tensor core forms S = Q K^T once per block, the softmax warps turn a row of S
// into the teacher's probabilities (one exponential per element) and derive the student's from them
// (the same exponential times 2^(ref_teacher - ref_student), zero where the eviction mask hides the
// key), and two P V products accumulate the two outputs.  Key blocks that are EMPTY for the student
// cost it nothing.  384 threads:
//   warps 0-3   softmax, keys  0..63 of a block (one query row per thread)   } the two groups of a row
//   warps 4-7   softmax, keys 64..127                                        } exchange their partial maxima
//   warp 8      producer (TMA: Q once, a K ring of three stages running two key blocks ahead of a V ring of two;
//               evict_at of a block by plain loads)
//   warp 9      MMA issuer (all lanes walk the loop, an elected lane issues);  warps 10-11 idle
// Tensor memory: S_a [0,128)  S_b [128,256)  O_teacher [256,256+D)  O_student [384,384+D).  The two S
// buffers alternate, so S of block i+1 is ready when the softmax of block i ends.  The probabilities
// (bf16, two per column) overwrite the S buffer they came from: teacher in its columns [0,64), student
// in [64,128).  Both outputs are rescaled lazily (reference maximum moves only when the running maximum
// exceeds it by more than 8 in base-2 units).
#include "kvs_common.cuh"

namespace kvs {

constexpr int DUAL_THREADS = 384;
constexpr float DUAL_RESCALE_THRESHOLD = 8.0f;
// Above this gap between the two references the student's probabilities are exponentiated directly:
// the teacher's could have lost them to underflow.
constexpr float DUAL_DIRECT_GAP = 64.0f;

template <int D>
struct DualSmem {
    static constexpr int TB = TILE * D * 2;
    static constexpr int OFF_Q = 0;
    static constexpr int OFF_K = TB;                       // 3 stages
    static constexpr int OFF_V = 4 * TB;                   // 2 stages
    static constexpr int OFF_EV = 6 * TB;                  // 2 stages x 128 int32
    static constexpr int OFF_MAX = OFF_EV + 2 * TILE * 4;  // [2 buffers][teacher, student][2 groups][128 rows] fp32
    static constexpr int OFF_FLAG = OFF_MAX + 2 * 2 * 2 * TILE * 4;
    static constexpr int OFF_BAR = OFF_FLAG + 16;
    static constexpr int OFF_MISC = OFF_BAR + 24 * 8;      // 21 barriers in use
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;         // slack for the 1024-byte alignment
};

struct DualParams {
    int batch, total_tokens, max_seqlen;
    int Hq, Hkv;
    float scale_log2;
    __nv_bfloat16* out_s;
    float* lse_s;
    __nv_bfloat16* out_t;
    float* lse_t;
};

// flag bits the producer publishes per ring stage
constexpr int DF_STUDENT = 1;        // the block is not EMPTY for the student
constexpr int DF_MASK_S = 2;         // the student's element mask has to be evaluated
constexpr int DF_MASK_T = 4;         // the teacher's (causal / ragged) mask has to be evaluated

template <int D>
__global__ void __launch_bounds__(DUAL_THREADS, 1)
fwd_dual_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                const __grid_constant__ CUtensorMap tm_v, MetaView mv, DualParams p) {
    using L = DualSmem<D>;
    constexpr int NBOX = D / 64;
    constexpr int BOX_BYTES = TILE * 128;
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_S = make_idesc(TILE, 0, 0);
    constexpr uint32_t IDESC_O = make_idesc(D, 0, 1);
    constexpr int DH = D / 2;                 // output columns each of a row's two threads owns

    extern __shared__ uint8_t smem_raw[];
    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    if (!meta_matches(mv.hdr, p.batch, p.total_tokens, p.max_seqlen)) {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) set_status(&mv.hdr->status, KVS_ERR_BAD_META);
        return;
    }
    if (mv.hdr->general) {          // the teacher's mask is defined for keys in their original order only
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) set_status(&mv.hdr->status, KVS_ERR_UNSUPPORTED);
        return;
    }
    const int nblk = mv.hdr->nblk_total;
    if ((int)blockIdx.x >= nblk) return;
    const int gb = nblk - 1 - (int)blockIdx.x;       // late query blocks (the long walks) first
    const int h = blockIdx.y;
    const int g = h / (p.Hq / p.Hkv);
    const int b = mv.blk_trace[gb];
    const int m = gb - mv.blk_off[b];
    const int tok0 = mv.seq_start[b];
    const int T = mv.seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    const int nt = m + 1;                             // the teacher walks key blocks 0..m
    const uint8_t* cls = mv.tile_class + mv.cls_off[b] + (size_t)m * nb;
    int32_t* status = &mv.hdr->status;

    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sbase = (sraw + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - sraw);
    const uint32_t sQ = sbase + L::OFF_Q, sK = sbase + L::OFF_K, sV = sbase + L::OFF_V;
    int32_t* sEv = reinterpret_cast<int32_t*>(sgen + L::OFF_EV);
    float* sMax = reinterpret_cast<float*>(sgen + L::OFF_MAX);
    volatile int32_t* sFlag = reinterpret_cast<volatile int32_t*>(sgen + L::OFF_FLAG);
    uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(sgen + L::OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + L::OFF_MISC + 4);
    const uint32_t bars = sbase + L::OFF_BAR;
    const uint32_t bar_q = bars;
    auto bar_vfull = [&](int s) { return bars + 8 * (1 + s); };
    auto bar_vfree = [&](int s) { return bars + 8 * (3 + s); };     // the P V products reading the stage's V have completed
    auto bar_evfull = [&](int s) { return bars + 8 * (5 + s); };    // flags + evict_at of the stage (32 arrivals)
    auto bar_evfree = [&](int s) { return bars + 8 * (7 + s); };    // the softmax warps are done with them (8 arrivals)
    auto bar_s = [&](int t) { return bars + 8 * (9 + t); };         // S buffer t holds a fresh Q K^T
    auto bar_p = [&](int t) { return bars + 8 * (11 + t); };        // probabilities written over S buffer t (8 arrivals)
    const uint32_t bar_o = bars + 8 * 13;                            // every P V product issued so far has completed
    const uint32_t bar_done = bars + 8 * 14;
    auto bar_kfull = [&](int s) { return bars + 8 * (15 + s); };    // K ring of three stages: key block i sits in stage i % 3
    auto bar_kfree = [&](int s) { return bars + 8 * (18 + s); };    // the Q K^T product reading the stage's K has completed

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_q, 1);
        for (int s = 0; s < 3; ++s) {
            mbar_init(bar_kfull(s), 1);
            mbar_init(bar_kfree(s), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_vfull(s), 1);
            mbar_init(bar_vfree(s), 1);
            mbar_init(bar_evfull(s), 32);
            mbar_init(bar_evfree(s), 8);
            mbar_init(bar_s(s), 1);
            mbar_init(bar_p(s), 8);
        }
        mbar_init(bar_o, 1);
        mbar_init(bar_done, 1);
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(s_tmem_base), TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem_base;
    const uint32_t tmem_Ot = tmem + 256, tmem_Os = tmem + 384;

    if (warp >= 8) {
        reg_dec<88>();
        if (warp == 8) {
            // ================= producer =================
            if (lane == 0) {
                mbar_expect_tx(bar_q, L::TB);
                for (int c = 0; c < NBOX; ++c) tma_load_3d(sQ + c * BOX_BYTES, &tm_q, c * 64, h, tok0 + m * TILE, bar_q);
            }
            // K runs two key blocks ahead of V (three stages): S of block i + 2 is issued as soon as the softmax of
            // block i has ended, and a tile takes about a microsecond to arrive
            auto load_k = [&](int i) {
                const int s = i % 3;
                if (i >= 3) mbar_wait(bar_kfree(s), (uint32_t)(i / 3 + 1) & 1, abort_flag, status);
                if (lane == 0) {
                    mbar_expect_tx(bar_kfull(s), L::TB);
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(sK + s * L::TB + c * BOX_BYTES, &tm_k, c * 64, g, tok0 + i * TILE, bar_kfull(s));
                }
            };
            for (int i = 0; i < 3 && i < nt; ++i) load_k(i);
            int c_next = cls[0];
            for (int i = 0; i < nt; ++i) {
                const int s = i & 1;
                const int c = c_next;
                if (i + 1 < nt) c_next = cls[i + 1];                 // fetched a block ahead of its use
                if (i >= 2) {
                    mbar_wait(bar_vfree(s), ((i >> 1) + 1) & 1, abort_flag, status);
                    mbar_wait(bar_evfree(s), ((i >> 1) + 1) & 1, abort_flag, status);
                }
                if (lane == 0) {
                    mbar_expect_tx(bar_vfull(s), L::TB);
                    for (int c2 = 0; c2 < NBOX; ++c2) tma_load_3d(sV + s * L::TB + c2 * BOX_BYTES, &tm_v, c2 * 64, g, tok0 + i * TILE, bar_vfull(s));
                }
                const bool ragged = (i * TILE + TILE > T);
                const bool mask_s = (c != KVS_CLASS_EMPTY) && ((c != KVS_CLASS_FULL) || ragged);
                if (mask_s) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int j = i * TILE + lane * 4 + u;
                        sEv[s * TILE + lane * 4 + u] = (j < T) ? mv.evict[tok0 + j] : 0;   // 0: visible to nobody
                    }
                }
                if (lane == 0)
                    sFlag[s] = (c != KVS_CLASS_EMPTY ? DF_STUDENT : 0) | (mask_s ? DF_MASK_S : 0) | ((i == m || ragged) ? DF_MASK_T : 0);
                mbar_arrive(bar_evfull(s));
                if (i >= 1 && i + 2 < nt) load_k(i + 2);
            }
        } else if (warp == 9) {
            // ================= MMA issuer =================
            const bool leader = elect_one();
            const uint64_t dQ0 = smem_desc(sQ, 16, 1024);
            const uint64_t dK0 = smem_desc(sK, 16, 1024);
            const uint64_t dV0 = smem_desc(sV, BOX_BYTES, 1024);
            constexpr uint64_t TBU = (uint64_t)(L::TB >> 4);
            auto issue_s = [&](int i) {               // S buffer i % 2 = Q K(block i, ring stage i % 3)^T
                const int t = i & 1, ks = i % 3;
                mbar_wait(bar_kfull(ks), (uint32_t)(i / 3) & 1, abort_flag, status);
                tc_fence_after();
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                    if (leader) mma_ss(tmem + t * 128, dQ0 + off, dK0 + ks * TBU + off, IDESC_S, kk > 0);
                }
                if (leader) {
                    mma_commit(bar_s(t));
                    mma_commit(bar_kfree(ks));
                }
            };
            mbar_wait(bar_q, 0, abort_flag, status);
            for (int i = 0; i < 2 && i < nt; ++i) issue_s(i);
            bool student_started = false;
            int c_next = cls[0];
            for (int i = 0; i < nt; ++i) {
                const int t = i & 1;
                const uint32_t ph = (uint32_t)(i >> 1) & 1;
                const bool student = c_next != KVS_CLASS_EMPTY;
                if (i + 1 < nt) c_next = cls[i + 1];
                mbar_wait(bar_p(t), ph, abort_flag, status);
                mbar_wait(bar_vfull(t), ph, abort_flag, status);
                tc_fence_after();
                // O_teacher += P_teacher V: A = probabilities from tensor memory (16 keys = 8 packed columns a step)
#pragma unroll
                for (int kk = 0; kk < TILE / 16; ++kk)
                    if (leader) mma_ts(tmem_Ot, tmem + t * 128 + kk * 8, dV0 + t * TBU + (uint64_t)(kk * 128), IDESC_O, (i > 0) || (kk > 0));
                if (student) {
#pragma unroll
                    for (int kk = 0; kk < TILE / 16; ++kk)
                        if (leader) mma_ts(tmem_Os, tmem + t * 128 + 64 + kk * 8, dV0 + t * TBU + (uint64_t)(kk * 128), IDESC_O,
                                           student_started || (kk > 0));
                    student_started = true;
                }
                if (leader) {
                    mma_commit(bar_vfree(t));
                    mma_commit(bar_o);
                }
                if (i + 2 < nt) issue_s(i + 2);
            }
            if (leader) mma_commit(bar_done);
        }
    } else {
        // ================= softmax warps =================
        reg_inc<208>();
        const int grp = warp >> 2;                               // which 64 keys of a block
        const int quad = warp & 3;
        const int row = quad * 32 + lane;                        // query row of the block == TMEM lane
        const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
        const int qi = m * TILE + row;                           // trace-local query index
        float ref_t = -INFINITY, ref_s = -INFINITY;              // base-2 reference maxima
        float sum_t = 0.f, sum_s = 0.f;                          // this thread's share of the row sums
        int tiles_s = 0;                                         // student blocks accumulated so far

        // multiplies this thread's half of an output accumulator row by alpha
        auto rescale = [&](uint32_t tmem_O, float alpha) {
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_O + lane_sel + grp * DH + c * 32, r);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                tmem_st32(tmem_O + lane_sel + grp * DH + c * 32, r);
            }
            tmem_wait_st();
        };

        for (int i = 0; i < nt; ++i) {
            const int s = i & 1;
            const uint32_t ph = (uint32_t)(i >> 1) & 1;
            mbar_wait(bar_evfull(s), ph, abort_flag, status);
            const int flags = sFlag[s];
            const bool student = (flags & DF_STUDENT) != 0;
            mbar_wait(bar_s(s), ph, abort_flag, status);
            tc_fence_after();
            const uint32_t tmem_S = tmem + s * 128 + lane_sel;
            float sv[64];
            {
                uint32_t r0[32], r1[32];
                tmem_ld32(tmem_S + grp * 64, r0);
                tmem_ld32(tmem_S + grp * 64 + 32, r1);
                tmem_wait_ld();
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                    sv[e] = __uint_as_float(r0[e]);
                    sv[32 + e] = __uint_as_float(r1[e]);
                }
            }
            const int j0 = i * TILE + grp * 64;                  // first key of this thread's 64
            // visibility: bit e of vis_t / vis_s set when key j0 + e is visible to the teacher / the student
            uint64_t vis_t = ~0ull, vis_s = student ? ~0ull : 0ull;
            if (flags & DF_MASK_T) {
                vis_t = 0ull;
#pragma unroll
                for (int e = 0; e < 64; ++e) vis_t |= (uint64_t)((j0 + e <= qi) && (j0 + e < T)) << e;
                vis_s &= vis_t;
            }
            if (flags & DF_MASK_S) {
                const int4* ev4 = reinterpret_cast<const int4*>(sEv + s * TILE + grp * 64);
                uint64_t live = 0ull;
#pragma unroll
                for (int e4 = 0; e4 < 16; ++e4) {
                    const int4 ev = ev4[e4];
                    const int j = j0 + e4 * 4;
                    live |= (uint64_t)((j + 0 <= qi) && (qi < ev.x)) << (e4 * 4 + 0);
                    live |= (uint64_t)((j + 1 <= qi) && (qi < ev.y)) << (e4 * 4 + 1);
                    live |= (uint64_t)((j + 2 <= qi) && (qi < ev.z)) << (e4 * 4 + 2);
                    live |= (uint64_t)((j + 3 <= qi) && (qi < ev.w)) << (e4 * 4 + 3);
                }
                vis_s &= live;
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_evfree(s));
            // partial maxima over this thread's 64 keys (raw logits: the scale is positive)
            float mt = -INFINITY, ms = -INFINITY;
            if (vis_t == ~0ull && (vis_s == ~0ull || vis_s == 0ull)) {
                float mx[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) mx[u] = fmaxf(sv[u], sv[8 + u]);
#pragma unroll
                for (int e = 16; e < 64; e += 16) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) mx[u] = fmax3(mx[u], sv[e + u], sv[e + 8 + u]);
                }
                mt = fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7])));
                ms = vis_s ? mt : -INFINITY;
            } else {
#pragma unroll
                for (int e = 0; e < 64; ++e) {
                    mt = fmaxf(mt, ((vis_t >> e) & 1) ? sv[e] : -INFINITY);
                    ms = fmaxf(ms, ((vis_s >> e) & 1) ? sv[e] : -INFINITY);
                }
            }
            // the two threads of a row exchange their partial maxima (double-buffered by block parity)
            float* mex = sMax + s * (4 * TILE);
            mex[(0 * 2 + grp) * TILE + row] = mt;
            mex[(1 * 2 + grp) * TILE + row] = ms;
            named_bar_sync(2, 256);
            const float tile_t = fmaxf(mt, mex[(0 * 2 + (grp ^ 1)) * TILE + row]) * p.scale_log2;
            const float tile_s = fmaxf(ms, mex[(1 * 2 + (grp ^ 1)) * TILE + row]) * p.scale_log2;
            // lazy rescale of either output: both threads of a row take the same decision from the same numbers
            const bool grow_t = (tile_t > ref_t + DUAL_RESCALE_THRESHOLD) || (ref_t == -INFINITY && tile_t > -INFINITY);
            const bool grow_s = (tile_s > ref_s + DUAL_RESCALE_THRESHOLD) || (ref_s == -INFINITY && tile_s > -INFINITY);
            if (__any_sync(0xffffffffu, grow_t || grow_s)) {
                // the products of the previous block may still be adding to the accumulators
                if (i > 0) {
                    mbar_wait(bar_o, (uint32_t)(i - 1) & 1, abort_flag, status);
                    tc_fence_after();
                }
                if (__any_sync(0xffffffffu, grow_t)) {
                    const float new_ref = grow_t ? tile_t : ref_t;
                    const float alpha = (new_ref == -INFINITY) ? 1.f : fast_exp2(ref_t - new_ref);   // ref = -inf -> 0
                    sum_t *= alpha;
                    ref_t = new_ref;
                    if (i > 0) rescale(tmem_Ot, alpha);
                }
                if (__any_sync(0xffffffffu, grow_s)) {
                    const float new_ref = grow_s ? tile_s : ref_s;
                    const float alpha = (new_ref == -INFINITY) ? 1.f : fast_exp2(ref_s - new_ref);
                    sum_s *= alpha;
                    ref_s = new_ref;
                    if (tiles_s > 0) rescale(tmem_Os, alpha);
                }
                tc_fence_before();
            }
            // teacher: one exponential per element; student: the same value times 2^(ref_t - ref_s)
            const float neg_ref_t = (ref_t == -INFINITY) ? 0.f : -ref_t;
            const float neg_ref_s = (ref_s == -INFINITY) ? 0.f : -ref_s;
            const float gap = (ref_t == -INFINITY || ref_s == -INFINITY) ? 0.f : ref_t - ref_s;
            // a whole warp takes the direct formula as soon as one of its rows needs it (it is the exact one), so
            // the branch is uniform and the warp-wide tensor-memory stores may sit inside it
            const bool direct = student && __any_sync(0xffffffffu, gap > DUAL_DIRECT_GAP);
            const float2 c2 = make_float2(p.scale_log2, p.scale_log2);
            const float2 nr2 = make_float2(neg_ref_t, neg_ref_t);
            uint32_t pk[32];
            float2 acc[2];
            if (direct) {
                // rare: the references are so far apart that the teacher's values may have underflowed
                acc[0] = acc[1] = make_float2(0.f, 0.f);
#pragma unroll
                for (int e = 0; e < 64; e += 2) {
                    float2 pq = make_float2(fast_exp2(fmaf(sv[e], p.scale_log2, neg_ref_s)), fast_exp2(fmaf(sv[e + 1], p.scale_log2, neg_ref_s)));
                    pq.x = ((vis_s >> e) & 1) ? pq.x : 0.f;
                    pq.y = ((vis_s >> (e + 1)) & 1) ? pq.y : 0.f;
                    acc[(e >> 1) & 1] = __fadd2_rn(acc[(e >> 1) & 1], pq);
                    pk[e >> 1] = pack_bf16(pq.x, pq.y);
                }
                const float2 s01 = __fadd2_rn(acc[0], acc[1]);
                sum_s += s01.x + s01.y;
                tmem_st32(tmem_S + 64 + grp * 32, pk);
            }
            // the teacher's probabilities take the place of the logits; summed and packed as they are formed
            acc[0] = acc[1] = make_float2(0.f, 0.f);
            if (vis_t == ~0ull) {
#pragma unroll
                for (int e = 0; e < 64; e += 2) {
                    const float2 x = __ffma2_rn(make_float2(sv[e], sv[e + 1]), c2, nr2);
                    sv[e] = fast_exp2(x.x);
                    sv[e + 1] = fast_exp2(x.y);
                    acc[(e >> 1) & 1] = __fadd2_rn(acc[(e >> 1) & 1], make_float2(sv[e], sv[e + 1]));
                    pk[e >> 1] = pack_bf16(sv[e], sv[e + 1]);
                }
            } else {
#pragma unroll
                for (int e = 0; e < 64; e += 2) {
                    const float2 x = __ffma2_rn(make_float2(sv[e], sv[e + 1]), c2, nr2);
                    sv[e] = ((vis_t >> e) & 1) ? fast_exp2(x.x) : 0.f;
                    sv[e + 1] = ((vis_t >> (e + 1)) & 1) ? fast_exp2(x.y) : 0.f;
                    acc[(e >> 1) & 1] = __fadd2_rn(acc[(e >> 1) & 1], make_float2(sv[e], sv[e + 1]));
                    pk[e >> 1] = pack_bf16(sv[e], sv[e + 1]);
                }
            }
            {
                const float2 t01 = __fadd2_rn(acc[0], acc[1]);
                sum_t += t01.x + t01.y;
            }
            // probabilities go over the S columns that both groups have finished reading (the exchange barrier above)
            tmem_st32(tmem_S + grp * 32, pk);
            if (student && !direct) {
                if (vis_s != ~0ull) {
#pragma unroll
                    for (int e = 0; e < 64; ++e) sv[e] = ((vis_s >> e) & 1) ? sv[e] : 0.f;
                }
                const float cmul = fast_exp2(gap);
                const float2 cm2 = make_float2(cmul, cmul);
                acc[0] = acc[1] = make_float2(0.f, 0.f);
#pragma unroll
                for (int e = 0; e < 64; e += 2) {
                    const float2 pq = __fmul2_rn(make_float2(sv[e], sv[e + 1]), cm2);
                    acc[(e >> 1) & 1] = __fadd2_rn(acc[(e >> 1) & 1], pq);
                    pk[e >> 1] = pack_bf16(pq.x, pq.y);
                }
                const float2 s01 = __fadd2_rn(acc[0], acc[1]);
                sum_s += s01.x + s01.y;
                tmem_st32(tmem_S + 64 + grp * 32, pk);
            }
            if (student) ++tiles_s;
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p(s));
        }

        // ---- epilogue: both outputs, each thread its half of the columns ----
        mbar_wait(bar_done, 0, abort_flag, status);
        tc_fence_after();
        float* mex = sMax;                                        // reused: the row sums of the two groups
        named_bar_sync(2, 256);                                   // nobody still reads the last block's maxima
        mex[(0 * 2 + grp) * TILE + row] = sum_t;
        mex[(1 * 2 + grp) * TILE + row] = sum_s;
        named_bar_sync(2, 256);
        const float tot_t = sum_t + mex[(0 * 2 + (grp ^ 1)) * TILE + row];
        const float tot_s = sum_s + mex[(1 * 2 + (grp ^ 1)) * TILE + row];
        const bool valid = qi < T;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const float tot = which == 0 ? tot_t : tot_s;
            const float ref = which == 0 ? ref_t : ref_s;
            const bool any = which == 0 ? true : tiles_s > 0;     // a student row always sees itself unless evict_at was bad
            const float inv = (tot > 0.f && any) ? 1.f / tot : 0.f;
            __nv_bfloat16* obase = which == 0 ? p.out_t : p.out_s;
            float* lbase = which == 0 ? p.lse_t : p.lse_s;
            __nv_bfloat16* orow = obase + ((size_t)(tok0 + qi) * p.Hq + h) * D + grp * DH;
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t r[32];
                tmem_ld32((which == 0 ? tmem_Ot : tmem_Os) + lane_sel + grp * DH + c * 32, r);
                tmem_wait_ld();
                if (valid) {
                    uint4* dst = reinterpret_cast<uint4*>(orow + c * 32);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        uint4 w;
                        w.x = pack_bf16(__uint_as_float(r[e * 8 + 0]) * inv, __uint_as_float(r[e * 8 + 1]) * inv);
                        w.y = pack_bf16(__uint_as_float(r[e * 8 + 2]) * inv, __uint_as_float(r[e * 8 + 3]) * inv);
                        w.z = pack_bf16(__uint_as_float(r[e * 8 + 4]) * inv, __uint_as_float(r[e * 8 + 5]) * inv);
                        w.w = pack_bf16(__uint_as_float(r[e * 8 + 6]) * inv, __uint_as_float(r[e * 8 + 7]) * inv);
                        if (!any) w = make_uint4(0, 0, 0, 0);
                        dst[e] = w;
                    }
                }
            }
            if (valid && grp == 0)
                lbase[(size_t)h * p.total_tokens + tok0 + qi] = (tot > 0.f && any) ? ref * 0.6931471805599453f + logf(tot) : -INFINITY;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

template <int D>
static int launch_dual(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const MetaView& mv, const DualParams& p,
                       int nb_cap, cudaStream_t st) {
    auto kern = fwd_dual_kernel<D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, DualSmem<D>::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    dim3 grid(nb_cap, p.Hq, 1);
    kern<<<grid, DUAL_THREADS, DualSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, mv, p);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

}  // namespace kvs

using namespace kvs;

extern "C" int kvs_attn_fwd_dual(const void* q, const void* k, const void* v, const void* meta_buf, int batch, int total_tokens,
                                 int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale, void* out_student,
                                 float* lse_student, void* out_teacher, float* lse_teacher, kvs_stream_t stream) {
    if (batch < 0 || total_tokens < 0 || max_seqlen < 0 || Hq <= 0 || Hkv <= 0) return KVS_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128) return KVS_ERR_UNSUPPORTED;
    if (Hq % Hkv != 0 || Hq > 65535) return KVS_ERR_UNSUPPORTED;
    if (total_tokens == 0 || batch == 0) return KVS_OK;
    if (!q || !k || !v || !meta_buf || !out_student || !lse_student || !out_teacher || !lse_teacher) return KVS_ERR_INVALID_ARG;
    if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out_student | (uintptr_t)out_teacher) & 15) != 0 ||
        (((uintptr_t)lse_student | (uintptr_t)lse_teacher) & 3) != 0)
        return KVS_ERR_ALIGNMENT;
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
    DualParams p;
    p.batch = batch;
    p.total_tokens = total_tokens;
    p.max_seqlen = max_seqlen < total_tokens ? max_seqlen : total_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    const float s = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = s * 1.4426950408889634f;
    p.out_s = (__nv_bfloat16*)out_student;
    p.lse_s = lse_student;
    p.out_t = (__nv_bfloat16*)out_teacher;
    p.lse_t = lse_teacher;
    cudaStream_t st = (cudaStream_t)stream;
    return head_dim == 64 ? launch_dual<64>(tq, tk, tv, mv, p, L.nb_cap, st) : launch_dual<128>(tq, tk, tv, mv, p, L.nb_cap, st);
}
