// Forward: eviction-masked causal attention.
//
// One CTA per (query block, pair of query heads of one GQA group).  The two heads share every K/V
// tile (identical key-block list and element mask), so each tile is fetched once for two 128-row
// query tiles.  The last head of an odd group (and every head when there is no grouping) gets a CTA
// of its own, in which the two softmax groups take alternate key blocks of that one head as two
// independent streams, merged at the end.  384 threads in three warp groups:
//   warps 0-3   softmax of tile 0 (one query row per thread)        } registers re-balanced with
//   warps 4-7   softmax of tile 1                                    } setmaxnreg (208 / 208 / 88)
//   warp 8      producer: TMA for Q0, Q1 and the K and V rings (2 stages each; K runs one key
//               block ahead of V, its slot being released a whole iteration earlier); plain loads
//               for evict_at
//   warp 9      MMA issuer: all 32 lanes walk the loop and one elected lane issues, so descriptor
//               arithmetic stays in uniform registers and an MMA costs a few issue slots even while
//               the softmax warps of the same scheduler are busy;  warps 10-11 idle
// Tensor memory: S0 [0,128)  S1 [128,256)  O0 [256,256+D)  O1 [384,384+D); P (bf16) overwrites S.
// Per key block i the tensor pipe runs  O0 += P0 V, S0(i+1) = Q0 K^T, O1 += P1 V, S1(i+1) = Q1 K^T
// while the two softmax groups alternate, so the exponentials of one tile overlap the MMAs of the
// other.  A row's probabilities are handed over in two parts (the first P_SPLIT keys, then the
// rest), so most of P V overlaps the last exponentials of the row.  EMPTY tiles are never visited (the CTA walks the row's non-empty list); the element mask
// is evaluated on PARTIAL or ragged tiles only.  O is rescaled lazily: a row keeps its reference
// maximum until the running maximum exceeds it by more than 8 (base-2), so exp2 arguments stay
// below 2^8 and the rescale of O in tensor memory is rare.
#include "kvs_common.cuh"

namespace kvs {

constexpr int FWD_THREADS = 384;
constexpr float RESCALE_THRESHOLD = 8.0f;
constexpr int P_SPLIT = 96;     // keys of a tile whose probabilities are handed to the MMA warp early

template <int D>
struct FwdSmem {
    static constexpr int TB = TILE * D * 2;
    static constexpr int OFF_Q = 0;                      // 2 query tiles
    static constexpr int OFF_KV = 2 * TB;                // 2 stages x (K, V)
    static constexpr int OFF_EV = OFF_KV + 4 * TB;       // 2 stages x 128 int32: eviction step of the stage's key slots
    static constexpr int OFF_KF = OFF_EV + 2 * TILE * 4; // 2 stages x 128 int32: first query that may see the slot
    static constexpr int OFF_FLAG = OFF_KF + 2 * TILE * 4;   // 2 stages x need_mask
    static constexpr int OFF_BAR = OFF_FLAG + 16;
    static constexpr int OFF_MISC = OFF_BAR + 24 * 8;
    static constexpr int TOTAL = OFF_MISC + 16;
    static constexpr int DYN_BYTES = TOTAL + 1024;          // slack for the 1024-byte alignment
};

struct FwdParams {
    int batch, total_tokens, max_seqlen;   // what the caller says meta_buf was built for
    int Hq, Hkv;
    float scale_log2;   // softmax_scale * log2(e)
    __nv_bfloat16* out;
    float* lse;
};


template <int D>
__global__ void __launch_bounds__(FWD_THREADS, 1)
fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
           const __grid_constant__ CUtensorMap tm_v, MetaView mv, FwdParams p) {
    using L = FwdSmem<D>;
    constexpr int NBOX = D / 64;             // 64-column TMA boxes per tile row
    constexpr int BOX_BYTES = TILE * 128;    // 128 rows x 128 bytes
    constexpr uint32_t TMEM_COLS = 512;
    constexpr uint32_t IDESC_S = make_idesc(TILE, 0, 0);
    constexpr uint32_t IDESC_O = make_idesc(D, 0, 1);

    extern __shared__ uint8_t smem_raw[];

    const int tid = threadIdx.x;
    const int warp = tid >> 5;
    const int lane = tid & 31;
    // meta_buf must be the one kvs_mask_meta wrote for these sizes: every index below comes out of it
    if (!meta_matches(mv.hdr, p.batch, p.total_tokens, p.max_seqlen)) {
        if (tid == 0 && blockIdx.x == 0 && blockIdx.y == 0) set_status(&mv.hdr->status, KVS_ERR_BAD_META);
        return;
    }
    if ((int)blockIdx.x >= mv.hdr->nblk_total) return;
    const int gb = mv.fwd_order[blockIdx.x];
    const int G = p.Hq / p.Hkv;
    const int pairs_per_group = (G + 1) >> 1;
    const int g = blockIdx.y / pairs_per_group;
    const int h0 = g * G + 2 * (blockIdx.y % pairs_per_group);
    const int ntile = (h0 + 1 < (g + 1) * G) ? 2 : 1;       // an odd group ends with a single head
    // A CTA with a single head still runs both softmax groups: they take alternate key blocks of that head as two
    // independent streams (own S, O, running maximum and sum), merged at the end like the splits of a split-KV decode.
    const bool dual = (ntile == 1);
    const int b = mv.blk_trace[gb];
    const int m = gb - mv.blk_off[b];
    const int tok0 = mv.seq_start[b];
    const int T = mv.seq_start[b + 1] - tok0;
    const int nb = (T + TILE - 1) / TILE;
    const int nlist = mv.row_cnt[gb];
    const uint16_t* list = mv.row_list + mv.cls_off[b] + (size_t)m * nb;
    const uint8_t* cls = mv.tile_class + mv.cls_off[b] + (size_t)m * nb;
    int32_t* status = &mv.hdr->status;

    const uint32_t sraw = smem_u32(smem_raw);
    const uint32_t sbase = (sraw + 1023u) & ~1023u;
    uint8_t* sgen = smem_raw + (sbase - sraw);
    const uint32_t sQ = sbase + L::OFF_Q, sKV = sbase + L::OFF_KV;
    int32_t* sEv = reinterpret_cast<int32_t*>(sgen + L::OFF_EV);
    int32_t* sKf = reinterpret_cast<int32_t*>(sgen + L::OFF_KF);
    const bool general = mv.hdr->general != 0;       // key slots carry their own first visible query (re-ordered keys)
    volatile int32_t* sFlag = reinterpret_cast<volatile int32_t*>(sgen + L::OFF_FLAG);
    uint32_t* s_tmem_base = reinterpret_cast<uint32_t*>(sgen + L::OFF_MISC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(sgen + L::OFF_MISC + 4);
    const uint32_t bars = sbase + L::OFF_BAR;
    const uint32_t bar_q = bars;
    auto bar_vfull = [&](int s) { return bars + 8 * (1 + s); };     // TMA bytes of V
    auto bar_kfull = [&](int s) { return bars + 8 * (16 + s); };    // TMA bytes of K
    auto bar_evfull = [&](int s) { return bars + 8 * (3 + s); };    // evict_at tile + need_mask flag (32 arrivals)
    auto bar_vfree = [&](int s) { return bars + 8 * (5 + s); };     // every P V product reading the stage's V has completed
    auto bar_kfree = [&](int s) { return bars + 8 * (18 + s); };    // every Q K^T product reading the stage's K has completed
    auto bar_s = [&](int t) { return bars + 8 * (7 + t); };         // S_t ready
    auto bar_p = [&](int t) { return bars + 8 * (9 + t); };         // all of P_t written (4 arrivals)
    auto bar_p0 = [&](int t) { return bars + 8 * (14 + t); };       // first P_SPLIT keys of P_t written (4 arrivals)
    auto bar_evfree = [&](int s) { return bars + 8 * (11 + s); };   // softmax groups done with the evict_at tile
    const uint32_t bar_done = bars + 8 * 13;                         // all MMAs complete

    if (tid == 0) {
        *abort_flag = 0;
        mbar_init(bar_q, 1);
        for (int s = 0; s < 2; ++s) {
            mbar_init(bar_vfull(s), 1);
            mbar_init(bar_kfull(s), 1);
            mbar_init(bar_evfull(s), 32);
            mbar_init(bar_vfree(s), 1);
            mbar_init(bar_kfree(s), 1);
            mbar_init(bar_evfree(s), 4 * ntile);
            mbar_init(bar_s(s), 1);
            mbar_init(bar_p(s), 4);
            mbar_init(bar_p0(s), 4);
        }
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

    if (warp >= 8) {
        reg_dec<88>();
        if (warp == 8) {
            // ================= producer =================
            if (lane == 0) {
                mbar_expect_tx(bar_q, ntile * L::TB);
                for (int t = 0; t < ntile; ++t)
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(sQ + t * L::TB + c * BOX_BYTES, &tm_q, c * 64, h0 + t, tok0 + m * TILE, bar_q);
            }
            // K runs one key block ahead of V: the slot of K(i+1) is released by the Q K^T products of
            // block i-1, which are issued a whole iteration before the P V products that release V's slot.
            auto load_k = [&](int i) {
                const int s = i & 1;
                if (i >= 2) mbar_wait(bar_kfree(s), ((i >> 1) + 1) & 1, abort_flag, status);
                if (lane == 0) {
                    mbar_expect_tx(bar_kfull(s), L::TB);
                    const uint32_t dst = sKV + s * 2 * L::TB;
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(dst + c * BOX_BYTES, &tm_k, c * 64, g, tok0 + list[i] * TILE, bar_kfull(s));
                }
            };
            if (nlist > 0) load_k(0);
            for (int i = 0; i < nlist; ++i) {
                const int s = i & 1;
                const int n = list[i];
                if (i >= 2) {
                    mbar_wait(bar_vfree(s), ((i >> 1) + 1) & 1, abort_flag, status);
                    mbar_wait(bar_evfree(s), ((i >> 1) + 1) & 1, abort_flag, status);
                }
                if (lane == 0) {
                    mbar_expect_tx(bar_vfull(s), L::TB);
                    const uint32_t dst = sKV + s * 2 * L::TB;
                    for (int c = 0; c < NBOX; ++c) tma_load_3d(dst + L::TB + c * BOX_BYTES, &tm_v, c * 64, g, tok0 + n * TILE, bar_vfull(s));
                }
                if (i + 1 < nlist) load_k(i + 1);
                const bool need_mask = (cls[n] != KVS_CLASS_FULL) || (n * TILE + TILE > T);
                if (need_mask) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int j = n * TILE + lane * 4 + u;
                        sEv[s * TILE + lane * 4 + u] = (j < T) ? mv.evict[tok0 + j] : 0;   // 0: visible to nobody
                        sKf[s * TILE + lane * 4 + u] = (general && j < T) ? mv.kfirst[tok0 + j] : j;
                    }
                }
                if (lane == 0) sFlag[s] = need_mask ? 1 : 0;
                mbar_arrive(bar_evfull(s));
            }
        } else if (warp == 9) {
            // ================= MMA issuer (all lanes walk the loop, one elected lane issues) =================
            const bool leader = elect_one();
            const uint64_t dQ0 = smem_desc(sQ, 16, 1024);
            const uint64_t dK0 = smem_desc(sKV, 16, 1024);
            const uint64_t dV0 = smem_desc(sKV + L::TB, BOX_BYTES, 1024);
            constexpr uint64_t TBU = (uint64_t)(L::TB >> 4);
            auto issue_s_q = [&](int t, int s, int qt) {      // S_t = Q_qt K(stage s)^T
#pragma unroll
                for (int kk = 0; kk < D / 16; ++kk) {
                    const uint64_t off = (uint64_t)(((kk >> 2) * BOX_BYTES + (kk & 3) * 32) >> 4);
                    if (leader) mma_ss(tmem + t * 128, dQ0 + qt * TBU + off, dK0 + s * 2 * TBU + off, IDESC_S, kk > 0);
                }
                if (leader) mma_commit(bar_s(t));
            };
            auto issue_s = [&](int t, int s) { issue_s_q(t, s, t); };
            if (dual) {
                // One head, two streams: stream t = key blocks i with i % 2 == t, on S_t / O_t and ring stage t.
                if (nlist > 0) {
                    mbar_wait(bar_q, 0, abort_flag, status);
                    for (int t = 0; t < 2 && t < nlist; ++t) {
                        mbar_wait(bar_kfull(t), 0, abort_flag, status);
                        tc_fence_after();
                        issue_s_q(t, t, 0);
                        if (leader) mma_commit(bar_kfree(t));
                    }
                }
                for (int i = 0; i < nlist; ++i) {
                    const int t = i & 1;
                    const uint32_t ph = (uint32_t)(i >> 1) & 1;
                    mbar_wait(bar_p0(t), ph, abort_flag, status);
                    mbar_wait(bar_vfull(t), ph, abort_flag, status);
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < P_SPLIT / 16; ++kk)
                        if (leader) mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, dV0 + t * 2 * TBU + (uint64_t)(kk * 128), IDESC_O,
                               (i > 1) || (kk > 0));
                    mbar_wait(bar_p(t), ph, abort_flag, status);
                    tc_fence_after();
#pragma unroll
                    for (int kk = P_SPLIT / 16; kk < TILE / 16; ++kk)
                        if (leader) mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, dV0 + t * 2 * TBU + (uint64_t)(kk * 128), IDESC_O, true);
                    if (leader) mma_commit(bar_vfree(t));
                    if (i + 2 < nlist) {
                        mbar_wait(bar_kfull(t), (uint32_t)((i + 2) >> 1) & 1, abort_flag, status);
                        tc_fence_after();
                        issue_s_q(t, t, 0);
                        if (leader) mma_commit(bar_kfree(t));
                    }
                }
                if (leader) mma_commit(bar_done);
            } else {
            if (nlist > 0) {
                mbar_wait(bar_q, 0, abort_flag, status);
                mbar_wait(bar_kfull(0), 0, abort_flag, status);
                tc_fence_after();
                for (int t = 0; t < ntile; ++t) issue_s(t, 0);
                if (leader) mma_commit(bar_kfree(0));
            }
            for (int i = 0; i < nlist; ++i) {
                const int s = i & 1;
                for (int t = 0; t < ntile; ++t) {
                    // O_t += P_t V(i):  A = P rows from tensor memory (16 keys = 8 packed columns per step),
                    //                   B = V, MN-major, 16 key rows per step
                    // The first P_SPLIT keys of P arrive while the row's last exponentials are still being
                    // taken, so most of this product overlaps the tail of the softmax.
                    mbar_wait(bar_p0(t), i & 1, abort_flag, status);
                    if (t == 0) mbar_wait(bar_vfull(s), (i >> 1) & 1, abort_flag, status);
                    tc_fence_after();
#pragma unroll
                    for (int kk = 0; kk < P_SPLIT / 16; ++kk)
                        if (leader) mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, dV0 + s * 2 * TBU + (uint64_t)(kk * 128), IDESC_O,
                               (i > 0) || (kk > 0));
                    mbar_wait(bar_p(t), i & 1, abort_flag, status);
                    tc_fence_after();
#pragma unroll
                    for (int kk = P_SPLIT / 16; kk < TILE / 16; ++kk)
                        if (leader) mma_ts(tmem + 256 + t * 128, tmem + t * 128 + kk * 8, dV0 + s * 2 * TBU + (uint64_t)(kk * 128), IDESC_O, true);
                    if (leader && t == ntile - 1) mma_commit(bar_vfree(s));       // V(i) is not read by anything issued later
                    if (i + 1 < nlist) {
                        if (t == 0) {
                            mbar_wait(bar_kfull(s ^ 1), ((i + 1) >> 1) & 1, abort_flag, status);
                            tc_fence_after();
                        }
                        issue_s(t, s ^ 1);
                        if (leader && t == ntile - 1) mma_commit(bar_kfree(s ^ 1));
                    }
                }
            }
            if (leader) mma_commit(bar_done);
            }
        }
    } else {
        // ================= softmax groups =================
        reg_inc<208>();
        const int t = warp >> 2;                                  // which query tile / head (or stream of the single head)
        if (t < ntile || dual) {
            const int quad = warp & 3;
            const int row = quad * 32 + lane;                     // query row of the tile == TMEM lane
            const uint32_t lane_sel = (uint32_t)(quad * 32) << 16;
            const uint32_t tmem_S = tmem + t * 128 + lane_sel;
            const uint32_t tmem_O = tmem + 256 + t * 128 + lane_sel;
            const int h = dual ? h0 : h0 + t;
            const int qi = m * TILE + row;                        // trace-local query index
            float ref_max = -INFINITY;                            // base-2 domain; the exponent's reference
            float run_sum = 0.f;

            for (int i = dual ? t : 0; i < nlist; i += dual ? 2 : 1) {
                const int s = i & 1;
                const int n = list[i];
                const int it = dual ? (i >> 1) : i;               // how many key blocks this group has done before
                mbar_wait(bar_evfull(s), (i >> 1) & 1, abort_flag, status);
                const bool need_mask = sFlag[s] != 0;
                mbar_wait(bar_s(t), it & 1, abort_flag, status);
                tc_fence_after();
                // raw logits of this row (the softmax scale is positive, so the maximum can be taken before it)
                float sv[TILE];
                {
                    uint32_t r0[32], r1[32], r2[32], r3[32];
                    tmem_ld32(tmem_S, r0);
                    tmem_ld32(tmem_S + 32, r1);
                    tmem_ld32(tmem_S + 64, r2);
                    tmem_ld32(tmem_S + 96, r3);
                    tmem_wait_ld();
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        sv[e] = __uint_as_float(r0[e]);
                        sv[32 + e] = __uint_as_float(r1[e]);
                        sv[64 + e] = __uint_as_float(r2[e]);
                        sv[96 + e] = __uint_as_float(r3[e]);
                    }
                }
                
                if (need_mask) {
                    const int4* ev4 = reinterpret_cast<const int4*>(sEv + s * TILE);
                    if (!general) {
#pragma unroll
                        for (int e4 = 0; e4 < TILE / 4; ++e4) {
                            const int4 ev = ev4[e4];
                            const int j = n * TILE + e4 * 4;
                            sv[e4 * 4 + 0] = ((j + 0 <= qi) && (qi < ev.x)) ? sv[e4 * 4 + 0] : -INFINITY;
                            sv[e4 * 4 + 1] = ((j + 1 <= qi) && (qi < ev.y)) ? sv[e4 * 4 + 1] : -INFINITY;
                            sv[e4 * 4 + 2] = ((j + 2 <= qi) && (qi < ev.z)) ? sv[e4 * 4 + 2] : -INFINITY;
                            sv[e4 * 4 + 3] = ((j + 3 <= qi) && (qi < ev.w)) ? sv[e4 * 4 + 3] : -INFINITY;
                        }
                    } else {
                        const int4* kf4 = reinterpret_cast<const int4*>(sKf + s * TILE);
#pragma unroll
                        for (int e4 = 0; e4 < TILE / 4; ++e4) {
                            const int4 ev = ev4[e4];
                            const int4 kf = kf4[e4];
                            sv[e4 * 4 + 0] = ((kf.x <= qi) && (qi < ev.x)) ? sv[e4 * 4 + 0] : -INFINITY;
                            sv[e4 * 4 + 1] = ((kf.y <= qi) && (qi < ev.y)) ? sv[e4 * 4 + 1] : -INFINITY;
                            sv[e4 * 4 + 2] = ((kf.z <= qi) && (qi < ev.z)) ? sv[e4 * 4 + 2] : -INFINITY;
                            sv[e4 * 4 + 3] = ((kf.w <= qi) && (qi < ev.w)) ? sv[e4 * 4 + 3] : -INFINITY;
                        }
                    }
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_evfree(s));
                // eight independent partial maxima (three-input max), then a short tree
                float mx[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) mx[u] = fmaxf(sv[u], sv[8 + u]);
#pragma unroll
                for (int e = 16; e < TILE; e += 16) {
#pragma unroll
                    for (int u = 0; u < 8; ++u) mx[u] = fmax3(mx[u], sv[e + u], sv[e + 8 + u]);
                }
                const float tile_max =
                    fmaxf(fmax3(mx[0], mx[1], mx[2]), fmaxf(fmax3(mx[3], mx[4], mx[5]), fmaxf(mx[6], mx[7]))) * p.scale_log2;
                // lazy rescale: move the reference only when the maximum ran away from it
                const bool grow = (tile_max > ref_max + RESCALE_THRESHOLD) || (ref_max == -INFINITY && tile_max > -INFINITY);
                if (__any_sync(0xffffffffu, grow)) {
                    const float new_ref = grow ? tile_max : ref_max;
                    const float alpha = (new_ref == -INFINITY) ? 1.f : fast_exp2(ref_max - new_ref);   // ref_max = -inf -> 0
                    run_sum *= alpha;
                    ref_max = new_ref;
                    if (it > 0) {
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld32(tmem_O + c * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) r[e] = __float_as_uint(__uint_as_float(r[e]) * alpha);
                            tmem_st32(tmem_O + c * 32, r);
                        }
                    }
                }
                const float neg_ref = (ref_max == -INFINITY) ? 0.f : -ref_max;
                // packed fp32x2: one multiply-add forms two exponents, one add accumulates two terms
                const float2 c2 = make_float2(p.scale_log2, p.scale_log2);
                const float2 nr2 = make_float2(neg_ref, neg_ref);
                float2 ts[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                uint32_t pk[TILE / 2];
#pragma unroll
                for (int e = 0; e < TILE; e += 8) {
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float2 x = __ffma2_rn(make_float2(sv[e + 2 * u], sv[e + 2 * u + 1]), c2, nr2);
                        const float2 pp = make_float2(fast_exp2(x.x), fast_exp2(x.y));
                        ts[u] = __fadd2_rn(ts[u], pp);
                        pk[(e >> 1) + u] = pack_bf16(pp.x, pp.y);
                    }
                    if (e + 8 == P_SPLIT) {
                        // P (bf16, packed two per column) goes over the S columns already read; the first
                        // P_SPLIT keys are handed to the MMA warp before the rest of the row is done
                        uint32_t r[32], r2[16];
#pragma unroll
                        for (int c = 0; c < 32; ++c) r[c] = pk[c];
#pragma unroll
                        for (int c = 0; c < 16; ++c) r2[c] = pk[32 + c];
                        tmem_st32(tmem_S, r);
                        tmem_st16(tmem_S + 32, r2);
                        tmem_wait_st();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(bar_p0(t));
                    }
                }
                const float2 t01 = __fadd2_rn(ts[0], ts[1]), t23 = __fadd2_rn(ts[2], ts[3]);
                const float tile_sum = (t01.x + t01.y) + (t23.x + t23.y);
                
                run_sum += tile_sum;
                {
                    uint32_t r2[16];
#pragma unroll
                    for (int c = 0; c < 16; ++c) r2[c] = pk[48 + c];
                    tmem_st16(tmem_S + 48, r2);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_p(t));
            }

            // ---- epilogue: O / l -> bf16, LSE -> fp32 ----
            mbar_wait(bar_done, 0, abort_flag, status);
            tc_fence_after();
            const bool valid = qi < T;
            // single head: stream 1 hands its partial result (O1 column by column, reference, sum) to stream 0
            // through the K/V ring's shared memory, which nothing uses any more
            float* x_o = reinterpret_cast<float*>(sgen + L::OFF_KV);           // [D][128 rows]
            float* x_ms = x_o + D * TILE;                                     // [2][128 rows]
            const bool has1 = dual && nlist > 1;
            float a0 = 1.f, a1 = 0.f;
            if (dual) {
                if (t == 1) {
                    if (has1) {
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t r[32];
                            tmem_ld32(tmem_O + c * 32, r);
                            tmem_wait_ld();
#pragma unroll
                            for (int e = 0; e < 32; ++e) x_o[(c * 32 + e) * TILE + row] = __uint_as_float(r[e]);
                        }
                    }
                    x_ms[row] = ref_max;
                    x_ms[TILE + row] = run_sum;
                }
                named_bar_sync(2, 256);
                if (t == 0) {
                    const float ref1 = has1 ? x_ms[row] : -INFINITY, sum1 = has1 ? x_ms[TILE + row] : 0.f;
                    const float mm = fmaxf(ref_max, ref1);
                    a0 = (ref_max == -INFINITY) ? 0.f : fast_exp2(ref_max - mm);
                    a1 = (ref1 == -INFINITY) ? 0.f : fast_exp2(ref1 - mm);
                    run_sum = run_sum * a0 + sum1 * a1;
                    ref_max = mm;
                }
            }
            if (!dual || t == 0) {
            const float inv = (run_sum > 0.f && nlist > 0) ? 1.f / run_sum : 0.f;
            __nv_bfloat16* orow = p.out + ((size_t)(tok0 + qi) * p.Hq + h) * D;
#pragma unroll
            for (int c = 0; c < D / 32; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem_O + c * 32, r);
                tmem_wait_ld();
                if (nlist == 0) {      // only a bad evict_at (already reported by the metadata pass) gets here
#pragma unroll
                    for (int e = 0; e < 32; ++e) r[e] = 0u;
                }
                if (dual) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) {
                        float o = __uint_as_float(r[e]) * a0;
                        if (a1 > 0.f) o = fmaf(x_o[(c * 32 + e) * TILE + row], a1, o);
                        r[e] = __float_as_uint(o);
                    }
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
            if (valid) p.lse[(size_t)h * p.total_tokens + tok0 + qi] = ref_max * 0.6931471805599453f + logf(run_sum);
            }
        }
    }
    // a Q load whose CTA had no key block to walk is drained before the CTA leaves
    if (nlist == 0 && tid == 0) mbar_wait(bar_q, 0, abort_flag, status);
    tc_fence_before();
    __syncthreads();
    if (warp == 9) {
        __syncwarp();
        tmem_dealloc(tmem, TMEM_COLS);
    }
}

template <int D>
static int launch_fwd(const CUtensorMap& tq, const CUtensorMap& tk, const CUtensorMap& tv, const MetaView& mv, const FwdParams& p,
                      int nb_cap, cudaStream_t st) {
    auto kern = fwd_kernel<D>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, FwdSmem<D>::DYN_BYTES) != cudaSuccess) return KVS_ERR_CUDA;
    const int G = p.Hq / p.Hkv;
    dim3 grid(nb_cap, p.Hkv * ((G + 1) / 2), 1);
    kern<<<grid, FWD_THREADS, FwdSmem<D>::DYN_BYTES, st>>>(tq, tk, tv, mv, p);
    return cudaGetLastError() == cudaSuccess ? KVS_OK : KVS_ERR_CUDA;
}

}  // namespace kvs

using namespace kvs;

namespace {
// q_ts / kv_ts: elements between consecutive tokens of q and of k, v (0: tensors of their own)
int fwd_impl(const void* q, const void* k, const void* v, long long q_ts, long long kv_ts, const void* meta_buf, int batch,
             int total_tokens, int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale, void* out, float* lse,
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
    if ((rc = make_tmap_thd(&tq, q, total_tokens, Hq, head_dim, TILE, q_ts)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tk, k, total_tokens, Hkv, head_dim, TILE, kv_ts)) != KVS_OK) return rc;
    if ((rc = make_tmap_thd(&tv, v, total_tokens, Hkv, head_dim, TILE, kv_ts)) != KVS_OK) return rc;
    FwdParams p;
    p.batch = batch;
    p.total_tokens = total_tokens;
    p.max_seqlen = max_seqlen < total_tokens ? max_seqlen : total_tokens;
    p.Hq = Hq;
    p.Hkv = Hkv;
    const float s = softmax_scale == 0.f ? 1.0f / sqrtf((float)head_dim) : softmax_scale;
    p.scale_log2 = s * 1.4426950408889634f;
    p.out = (__nv_bfloat16*)out;
    p.lse = lse;
    cudaStream_t st = (cudaStream_t)stream;
    return head_dim == 64 ? launch_fwd<64>(tq, tk, tv, mv, p, L.nb_cap, st) : launch_fwd<128>(tq, tk, tv, mv, p, L.nb_cap, st);
}
}  // namespace

extern "C" int kvs_attn_fwd(const void* q, const void* k, const void* v, const void* meta_buf, int batch, int total_tokens,
                            int max_seqlen, int Hq, int Hkv, int head_dim, float softmax_scale, void* out, float* lse,
                            kvs_stream_t stream) {
    return fwd_impl(q, k, v, 0, 0, meta_buf, batch, total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, out, lse, stream);
}

extern "C" int kvs_attn_fwd_packed(const void* qkv, const void* meta_buf, int batch, int total_tokens, int max_seqlen, int Hq,
                                   int Hkv, int head_dim, float softmax_scale, void* out, float* lse, kvs_stream_t stream) {
    if (Hq <= 0 || Hkv <= 0 || head_dim <= 0) return KVS_ERR_INVALID_ARG;
    if (total_tokens > 0 && batch > 0 && !qkv) return KVS_ERR_INVALID_ARG;
    const long long ts = (long long)(Hq + 2 * Hkv) * head_dim;
    const char* base = (const char*)qkv;
    return fwd_impl(base, base + (size_t)Hq * head_dim * 2, base + (size_t)(Hq + Hkv) * head_dim * 2, ts, ts, meta_buf, batch,
                    total_tokens, max_seqlen, Hq, Hkv, head_dim, softmax_scale, out, lse, stream);
}
