// Tensor-core attention of the active queries against all N keys of their request (paper Sec. 5 and
// Appendix A.6), head dim 128, on CTA pairs.
//
// One work item = 256 compact query rows of one request x one head.  A cluster of two CTAs takes it: each CTA
// owns 128 of the rows (its Q tile, its score / P buffers and accumulators in its own TMEM, its softmax and
// epilogue warps), and the two share every key tile (64 keys) through tcgen05.mma.cta_group::2:
//   S = Q K^T   M = 256 (both CTAs' query rows), N = 64 keys;  each CTA stages 32 of the tile's keys
//   O += P V    M = 256, N = 128 head dims;            each CTA stages all 64 keys of 64 of the head dims
// so a CTA brings in half of every K / V tile: the pair pulls each key and value from L2 once, where two
// independent CTAs pull it twice (the single-CTA kernel draws 8.6-10 TB/s from L2 across the chip at this head dim,
// which turned out to be a third of what that path sustains: not what paces it).  No load is multicast: every CTA
// fetches what it stages itself.
// Key tiles are 64 keys so that each softmax warpgroup has a score buffer of its own (2 x 64 score columns, 2 x 32
// P columns and 2 x 128 accumulator columns of TMEM): the product for tile g + 2 then only needs the scores of
// tile g to have left its buffer, which happened a whole tile earlier.
// MEASURED, AND WHY THIS KERNEL IS NOT THE DEFAULT (switch FD_ATT_PAIR=1): on the 480p video shape it halves the
// bytes drawn from L2 (11.7 GB per launch against 23.4 GB), yet takes 4.4 ms per launch against 3.05 ms for the
// single-CTA kernel (3.95 ms with 128-key tiles and one shared score buffer).  Timestamps taken inside the kernel show
// why: the issuing thread needs about 70 ns per cta_group::2 product instruction whatever its size (0.55 us for the
// eight N = 64 products of a score tile, 0.35 us for the four of P V), where the products themselves are 16-33 ns of
// tensor-core work each; a pair instruction only pays off when it carries N = 256 columns, as in the GEMMs.  An
// attention key tile cannot be that wide: its scores, P and two accumulators must fit the 512 TMEM columns.
// Passing the second CTA's barrier arrivals through relay threads instead of the softmax warps made it slower still
// (6.0 ms): every extra hop across the cluster adds most of a microsecond to the chain product -> softmax -> product.
//   warp 0        TMA producer (each CTA): Q tile double buffered across items, K / V halves in a ring
//   warps 1, 2    of the pair's first CTA issue S = Q K^T and O += P V for both CTAs; completion is
//                 broadcast to both CTAs' barriers with multicast commits
//   warps 4..11   softmax, as in the single-CTA kernel: warpgroup p takes the key tiles of parity p, one thread
//                 per query row, scores copied to registers at once, its own P buffer and accumulator O_p
//   warps 12..15  item epilogue: O = (a0 O_0 + a1 O_1) / (a0 l_0 + a1 l_1), stored through shared memory
// Barriers the issuing threads wait on (scores taken, P written, accumulators free) live in the first CTA and
// count the warps of both CTAs; the second CTA's warps arrive on them remotely.
// The items of a last, partly filled round of clusters are cut along the keys; attn_combine_pair_kernel puts
// the pieces together.  Every wait is bounded.
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace fd {

using namespace ptx;
using namespace attn;

namespace {

constexpr int PA_THREADS = 512;
constexpr int QROWS = 128, KEYS = 64, HD = 128;
constexpr int Q_SUB = 128 * 64 * 2;              // one [128 rows x 64 dims] sub-tile of Q, 128-byte rows
constexpr int Q_BYTES = 2 * Q_SUB;
constexpr int K_SUB = (KEYS / 2) * 64 * 2;       // this CTA's 32 keys x 64 dims
constexpr int KH_BYTES = 2 * K_SUB;
constexpr int VH_BYTES = KEYS * 64 * 2;          // 64 keys x this CTA's 64 head dims
constexpr int PA_STAGES = 8;
constexpr int PA_BAR_BYTES = 4608;
constexpr int PA_STAGE_OUT = 128 * 144;          // epilogue staging rows, 144 bytes apart
constexpr int PA_SMEM = 2 * Q_BYTES + PA_STAGES * (KH_BYTES + VH_BYTES) + PA_BAR_BYTES + PA_STAGE_OUT + 1024;

// TMEM columns: score buffers (one per tile parity, 64 columns), P buffers (32 columns each), accumulators (128 each)
constexpr uint32_t PCOL_S = 0, PCOL_P = 128, PCOL_O = 256, PA_TMEM_COLS = 512;

template <bool CUT>
__device__ __forceinline__ bool next_pair_task(const CutPlan& c, int n_items, int n_kv, int k, int cluster_id, int n_clusters,
                                               Task& t) {
    if constexpr (!CUT) {
        const int w = cluster_id + k * n_clusters;
        t = Task{w, 0, n_kv, 0};
        return w < n_items;
    }
    if (k < c.n_rounds) { t = Task{cluster_id + k * n_clusters, 0, n_kv, 0}; return true; }
    if (k > c.n_rounds || cluster_id >= c.n_tail * c.parts) return false;
    const int ti = cluster_id / c.parts, pt = cluster_id - ti * c.parts;
    const int j0 = pt * c.steps, j1 = j0 + c.steps < n_kv ? j0 + c.steps : n_kv;
    t = Task{c.n_rounds * n_clusters + ti, j0, j1, c.parts > 1 ? 1 : 0};
    return true;
}

template <bool CUT>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(PA_THREADS, 1)
tc_attention_pair_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ o, int o_ld,
                         const QTile* __restrict__ tiles2, int heads, int N, float scale_log2,
                         float* __restrict__ split_ws, Control* ctl) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem;                                   // [2]
    uint8_t* sK = smem + 2 * Q_BYTES;
    uint8_t* sV = sK + PA_STAGES * KH_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + PA_STAGES * VH_BYTES);
    uint64_t* k_full = bars;                  // [STAGES]  first CTA: both CTAs' K halves have landed
    uint64_t* k_empty = k_full + PA_STAGES;   // [STAGES]  each CTA: its K stage may be overwritten
    uint64_t* v_full = k_empty + PA_STAGES;
    uint64_t* v_empty = v_full + PA_STAGES;
    uint64_t* s_full = v_empty + PA_STAGES;   // [2]  each CTA: score tile (by tile parity) ready
    uint64_t* s_taken = s_full + 2;           // [2]  first CTA: both CTAs' softmax warps hold the tile's scores in registers
    uint64_t* p_ready = s_taken + 2;          // [2]  first CTA: both CTAs have written P of this parity
    uint64_t* pv_done = p_ready + 2;          // [2]  each CTA: the product that read this P buffer has completed
    uint64_t* q_full = pv_done + 2;           // [2]  first CTA
    uint64_t* q_empty = q_full + 2;           // [2]  each CTA
    uint64_t* o_free = q_empty + 2;           // [1]  first CTA: both CTAs' epilogue warps have read the accumulators
    uint64_t* stat_full = o_free + 1;         // [2]  each CTA: an item's row statistics are in shared memory
    uint64_t* stat_free = stat_full + 2;      // [2]
    uint64_t* item_done = stat_free + 2;      // [2]  each CTA: every product of an item (by item parity) has completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(item_done + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* s_xmax = reinterpret_cast<float*>(tmem_slot + 2);      // [2 items][2 parities][128 rows]
    float* s_xsum = s_xmax + 512;
    uint8_t* s_stage = reinterpret_cast<uint8_t*>(bars) + PA_BAR_BYTES;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;
    const bool aligned = (smem_u32(smem) & 1023u) == 0;  // never expected otherwise; refuse rather than compute garbage
    const int n_kv = (N + KEYS - 1) / KEYS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < PA_STAGES; ++s) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&s_taken[i], 8);        // 4 softmax warps of a parity in each of the two CTAs
            mbar_init(&p_ready[i], 8);
            mbar_init(&pv_done[i], 1);
            mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1);
            mbar_init(&stat_full[i], 8); mbar_init(&stat_free[i], 4); mbar_init(&item_done[i], 1);
        }
        mbar_init(&o_free[0], 8);             // 4 epilogue warps in each of the two CTAs
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_k);
        prefetch_tmap(&tm_v);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, PA_TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // both CTAs' barriers exist before anything remote arrives
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int wg = warp >> 2;                // 0: TMA + MMA issuers, 1 and 2: softmax, 3: item epilogue
    // everything above is local set-up; from here on the kernel reads what earlier kernels wrote
    pdl_trigger();
    pdl_wait();
    if (!aligned && threadIdx.x == 0) report(ctl, FD_ERR_STATE, -1025);
    const int n_tiles = aligned ? ctl->n_qtiles2 : 0;    // 256-row tiles; items are ordered head-major
    const int n_items = n_tiles * heads;
    const CutPlan cut = CUT ? cut_plan(n_items, n_kv, n_clusters, split_ws != nullptr) : CutPlan{0, 0, 1, 0};
    // barriers of the first CTA as both CTAs address them
    const uint32_t r_s_taken = map_to_cta(smem_u32(s_taken), 0), r_p_ready = map_to_cta(smem_u32(p_ready), 0);
    const uint32_t r_o_free = map_to_cta(smem_u32(o_free), 0);

    if (wg == 0) {
        reg_dec<48>();
        if (warp == 0) {
            // ---------------------------------------------------------------- TMA producer (each CTA)
            if (lane == 0) {
                uint32_t gk = 0;
                bool ok = true;
                int item_i = 0;
                Task tk;
                const uint32_t r_q_full = map_to_cta(smem_u32(q_full), 0), r_k_full = map_to_cta(smem_u32(k_full), 0);
                const uint32_t r_v_full = map_to_cta(smem_u32(v_full), 0);
                for (int k = 0; ok && next_pair_task<CUT>(cut, n_items, n_kv, k, cluster_id, n_clusters, tk); ++k, ++item_i) {
                    const int w = tk.w;
                    const QTile t = tiles2[w % n_tiles];
                    const int head = w / n_tiles;
                    const int qs = item_i & 1;
                    if (item_i >= 2 && !mbar_wait(&q_empty[qs], ((item_i >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    if (rank == 0) mbar_expect_tx(&q_full[qs], 2 * Q_BYTES);
                    // rows past the item's last one (a second CTA without rows) are computed and never stored
#pragma unroll
                    for (int sb = 0; sb < 2; ++sb)
                        tma_load_2d_pair(sQ + qs * Q_BYTES + sb * Q_SUB, &tm_q, head * HD + sb * 64, t.row0 + (int)rank * QROWS,
                                         r_q_full + qs * 8);
                    for (int j = tk.j0; j < tk.j1; ++j, ++gk) {
                        const int s = gk % PA_STAGES;
                        const uint32_t ph = ((gk / PA_STAGES) & 1) ^ 1;
                        if (!mbar_wait(&k_empty[s], ph, abort_flag)) { ok = false; break; }
                        if (rank == 0) mbar_expect_tx(&k_full[s], 2 * KH_BYTES);
#pragma unroll
                        for (int sb = 0; sb < 2; ++sb)
                            tma_load_3d_pair(sK + s * KH_BYTES + sb * K_SUB, &tm_k, head * HD + sb * 64,
                                             j * KEYS + (int)rank * (KEYS / 2), t.b * 2 + 0, r_k_full + s * 8);
                        if (!mbar_wait(&v_empty[s], ph, abort_flag)) { ok = false; break; }
                        if (rank == 0) mbar_expect_tx(&v_full[s], 2 * VH_BYTES);
                        tma_load_3d_pair(sV + s * VH_BYTES, &tm_v, head * HD + (int)rank * 64, j * KEYS, t.b * 2 + 1,
                                         r_v_full + s * 8);
                    }
                }
                if (!ok) report(ctl, FD_ERR_TIMEOUT, 1400 + (int)blockIdx.x);
            }
        } else if (warp == 1) {
            // ---------------------------------------------------------------- S = Q K^T issuer (first CTA)
            if (lane == 0 && rank == 0) {
                constexpr uint32_t idesc_qk = idesc_bf16(2 * QROWS, KEYS, 0, 0);
                uint32_t g = 0;
                bool ok = true;
                int item_i = 0;
                Task tk;
                for (int k = 0; ok && next_pair_task<CUT>(cut, n_items, n_kv, k, cluster_id, n_clusters, tk); ++k, ++item_i) {
                    const int qs = item_i & 1;
                    if (!mbar_wait(&q_full[qs], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
                    const uint32_t q_addr = smem_u32(sQ + qs * Q_BYTES);
                    for (int j = tk.j0; j < tk.j1; ++j, ++g) {
                        const int s = g % PA_STAGES;
                        if (!mbar_wait(&k_full[s], (g / PA_STAGES) & 1, abort_flag)) { ok = false; break; }
                        // this parity's score buffer is free once the scores of its previous tile (two tiles back) are in
                        // registers in both CTAs
                        if (g >= 2 && !mbar_wait_cluster(&s_taken[g & 1], ((g - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d = tmem_base + PCOL_S + (g & 1) * KEYS;
                        const uint32_t k_addr = smem_u32(sK + s * KH_BYTES);
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks)
                            mma_bf16_ss_pair(d, smem_desc(q_addr + (ks / 4) * Q_SUB + (ks % 4) * 32, 16, 1024, SWZ_128B),
                                             smem_desc(k_addr + (ks / 4) * K_SUB + (ks % 4) * 32, 16, 1024, SWZ_128B), idesc_qk,
                                             ks != 0);
                        mma_commit_pair(&k_empty[s], 0x3);
                        mma_commit_pair(&s_full[g & 1], 0x3);
                        if (j == tk.j1 - 1) mma_commit_pair(&q_empty[qs], 0x3);
                    }
                }
                if (!ok) report(ctl, FD_ERR_TIMEOUT, 1500 + (int)blockIdx.x);
            }
        } else if (warp == 2) {
            // ---------------------------------------------------------------- O += P V issuer (first CTA)
            if (lane == 0 && rank == 0) {
                constexpr uint32_t idesc_pv = idesc_bf16(2 * QROWS, HD, 0, 1);   // V: head dim contiguous (N-major)
                uint32_t g = 0;
                bool ok = true;
                int item_i = 0;
                Task tk;
                for (int k = 0; ok && next_pair_task<CUT>(cut, n_items, n_kv, k, cluster_id, n_clusters, tk); ++k, ++item_i) {
                    for (int j = tk.j0; j < tk.j1; ++j, ++g) {
                        const int s = g % PA_STAGES;
                        if (!mbar_wait(&v_full[s], (g / PA_STAGES) & 1, abort_flag)) { ok = false; break; }
                        // the two accumulators are free once both CTAs' epilogue warps have read the previous item's
                        if (j == tk.j0 && item_i > 0 && !mbar_wait_cluster(&o_free[0], (item_i - 1) & 1, abort_flag)) { ok = false; break; }
                        if (!mbar_wait_cluster(&p_ready[g & 1], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d = tmem_base + PCOL_O + (g & 1) * HD;        // even tiles O_0, odd tiles O_1
                        const uint32_t a = tmem_base + PCOL_P + (g & 1) * (KEYS / 2);
                        const uint32_t v_addr = smem_u32(sV + s * VH_BYTES);
#pragma unroll
                        for (int ks = 0; ks < KEYS / 16; ++ks)     // 16 keys further: 16 rows of 128 bytes
                            mma_bf16_ts_pair(d, a + ks * 8, smem_desc(v_addr + ks * 2048, VH_BYTES, 1024, SWZ_128B), idesc_pv,
                                             j - tk.j0 >= 2 || ks != 0);
                        mma_commit_pair(&v_empty[s], 0x3);
                        mma_commit_pair(&pv_done[g & 1], 0x3);
                        // the item's products complete in issue order: this one covers them all
                        if (j == tk.j1 - 1) mma_commit_pair(&item_done[item_i & 1], 0x3);
                    }
                }
                if (!ok) report(ctl, FD_ERR_TIMEOUT, 1550 + (int)blockIdx.x);
            }
        }
    } else if (wg == 1 || wg == 2) {
        // ---------------------------------------------------------------- softmax (each CTA, its own 128 rows)
        reg_inc<184>();
        const int quad = warp & 3;
        const int par = wg - 1;
        const int r = quad * 32 + lane;                       // query row inside this CTA's tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t s_addr = lane_addr + PCOL_S + par * KEYS;
        const uint32_t p_addr = lane_addr + PCOL_P + par * (KEYS / 2);
        const uint32_t o_addr = lane_addr + PCOL_O + par * HD;
        uint32_t g0 = 0;
        bool ok = true;
        int item_i = 0;
        const int rem = N - (n_kv - 1) * KEYS;                // valid keys of the last tile
        const uint64_t sc2 = pair(scale_log2, scale_log2);
        Task tk;
        for (int k = 0; ok && next_pair_task<CUT>(cut, n_items, n_kv, k, cluster_id, n_clusters, tk); ++k, ++item_i) {
            float m = -INFINITY, l = 0.f;
            for (int j = tk.j0 + ((g0 & 1) == (uint32_t)par ? 0 : 1); j < tk.j1 && ok; j += 2) {
                const uint32_t g = g0 + (j - tk.j0);
                if (!mbar_wait(&s_full[par], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const bool tail = j == n_kv - 1 && rem < KEYS;
                const bool first = j - tk.j0 < 2;            // this warpgroup's first tile of the item (or piece)
                uint32_t sr[KEYS];
#pragma unroll
                for (int c = 0; c < KEYS / 32; ++c) tmem_ld32(s_addr + c * 32, sr + c * 32);
                tmem_wait_ld();
                // the scores are in registers: the buffer can take this parity's next tile once the peer CTA says the same
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(r_s_taken + par * 8);
                if (tail) {
#pragma unroll
                    for (int i = 0; i < KEYS; ++i) if (i >= rem) sr[i] = 0xff800000u;         // -inf
                }
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < KEYS; i += 8) {          // three-input maxima: half the instructions
                    mx0 = max3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
                    mx1 = max3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
                    mx2 = max3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
                    mx3 = max3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
                }
                const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                // the P buffer is free, and O_par complete, once the product of this warpgroup's previous tile is done
                if (g >= 2 && !mbar_wait(&pv_done[par], ((g >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                if (first) {
                    m = mx;
                } else {
                    const bool need = (mx - m) * scale_log2 > RESCALE_LOG2;
                    if (__any_sync(0xffffffffu, need)) {
                        tc_fence_after();
                        const float f = need ? ex2((m - mx) * scale_log2) : 1.0f;
                        if (need) { l *= f; m = mx; }
#pragma unroll 1
                        for (int c = 0; c < HD / 8; ++c) {   // rare, and the scores are live: small pieces
                            uint32_t orr[8];
                            tmem_ld8(o_addr + c * 8, orr);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 8; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
                            tmem_st8(o_addr + c * 8, orr);
                        }
                        tmem_wait_st();
                    }
                }
                const float mb = m * scale_log2;
                const uint64_t nmb2 = pair(-mb, -mb);
                uint64_t sua = pair(0.f, 0.f), sub_ = pair(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < KEYS / 32; ++c) {
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {
                        float p[8];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint64_t x = fma2(pair(__uint_as_float(sr[c * 32 + 2 * i + 2 * e]),
                                                         __uint_as_float(sr[c * 32 + 2 * i + 2 * e + 1])), sc2, nmb2);
                            float xa, xb;
                            unpair(x, xa, xb);
                            p[2 * e] = ex2(xa);
                            p[2 * e + 1] = ex2(xb);
                        }
                        sua = add2(sua, add2(pair(p[0], p[1]), pair(p[2], p[3])));
                        sub_ = add2(sub_, add2(pair(p[4], p[5]), pair(p[6], p[7])));
#pragma unroll
                        for (int e = 0; e < 4; ++e) pk[i + e] = pack_bf16(p[2 * e], p[2 * e + 1]);
                    }
                    tmem_st16(p_addr + c * 16, pk);
                }
                {
                    float s0, s1;
                    unpair(add2(sua, sub_), s0, s1);
                    l += s0 + s1;
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(r_p_ready + par * 8);
            }
            if (!ok) break;
            // hand the row's statistics of this warpgroup's tiles to the epilogue warps and go on with the next
            // item; the slot was last used two items ago.  No tile at all (one-tile items): m = -inf, l = 0.
            const int slot = item_i & 1;
            if (item_i >= 2 && !mbar_wait(&stat_free[slot], ((item_i >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
            s_xmax[(slot * 2 + par) * 128 + r] = m;
            s_xsum[(slot * 2 + par) * 128 + r] = l;
            __syncwarp();
            if (lane == 0) mbar_arrive(&stat_full[slot]);
            g0 += tk.j1 - tk.j0;
        }
        if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 1650 + (int)blockIdx.x);
    } else {
        // ---------------------------------------------------------------- item epilogue (each CTA, its own 128 rows)
        reg_dec<96>();
        const int quad = warp & 3;
        const int r = quad * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        // staging rows are 144 bytes apart so that the 16-byte stores of a quarter warp fall into different banks
        uint8_t* wstage = s_stage + quad * 32 * 144;
        bool ok = true;
        int item_i = 0;
        Task tk;
        for (int k = 0; ok && next_pair_task<CUT>(cut, n_items, n_kv, k, cluster_id, n_clusters, tk); ++k, ++item_i) {
            const int w = tk.w;
            const QTile t = tiles2[w % n_tiles];
            const int head = w / n_tiles;
            const int row0 = t.row0 + (int)rank * QROWS;                       // this CTA's first compact row
            const int rows = min(QROWS, max(0, t.rows - (int)rank * QROWS));   // ... and how many of its 128 exist
            const int slot = item_i & 1;
            if (!mbar_wait(&stat_full[slot], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
            const float m0 = s_xmax[(slot * 2 + 0) * 128 + r], l0 = s_xsum[(slot * 2 + 0) * 128 + r];
            const float m1 = s_xmax[(slot * 2 + 1) * 128 + r], l1 = s_xsum[(slot * 2 + 1) * 128 + r];
            __syncwarp();
            if (lane == 0) mbar_arrive(&stat_free[slot]);
            // every product of the item must have landed
            if (!mbar_wait(&item_done[slot], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const float m_all = fmaxf(m0, m1);                // finite: at least one of the two had a tile
            const float a0 = m0 == -INFINITY ? 0.f : ex2((m0 - m_all) * scale_log2);
            const float a1 = m1 == -INFINITY ? 0.f : ex2((m1 - m_all) * scale_log2);
            // a cut item's piece stays un-normalised: its rows, maximum and sum go to the CTA's scratch slot
            const bool piece = CUT && tk.piece != 0;
            const float inv = piece ? 1.0f : 1.0f / (a0 * l0 + a1 * l1);
            const float w_0 = a0 * inv, w_1 = a1 * inv;       // weights of O_0, O_1
            float* prow = split_ws + (size_t)blockIdx.x * split_slot_floats(HD) + (size_t)r * (HD + 4);
            if (piece) {
                prow[HD] = m_all;
                prow[HD + 1] = a0 * l0 + a1 * l1;
            }
            // rolled loops on purpose: this code runs once per item, and the fewer instructions it fetches the
            // less it disturbs the softmax warps that share the instruction caches.  64 output columns per pass.
            const uint32_t acc0 = lane_addr + PCOL_O, acc1 = lane_addr + PCOL_O + HD;
#pragma unroll 1
            for (int hp = 0; hp < HD / 64; ++hp) {
#pragma unroll 1
                for (int q = 0; q < 8; ++q) {
                    uint32_t o0[8], o1[8];
                    tmem_ld8(acc0 + hp * 64 + q * 8, o0);
                    tmem_ld8(acc1 + hp * 64 + q * 8, o1);
                    tmem_wait_ld();
                    if (hp == HD / 64 - 1 && q == 7) {
                        // the accumulators are free for the next item as soon as they are in registers (in both CTAs)
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(r_o_free);
                    }
                    float v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        // a zero weight must also silence whatever an untouched accumulator holds
                        const float x0 = w_0 != 0.f ? __uint_as_float(o0[i]) * w_0 : 0.f;
                        const float x1 = w_1 != 0.f ? __uint_as_float(o1[i]) * w_1 : 0.f;
                        v[i] = x0 + x1;
                    }
                    if (piece) {
                        *reinterpret_cast<float4*>(prow + hp * 64 + q * 8) = make_float4(v[0], v[1], v[2], v[3]);
                        *reinterpret_cast<float4*>(prow + hp * 64 + q * 8 + 4) = make_float4(v[4], v[5], v[6], v[7]);
                        continue;
                    }
                    uint4 u;
                    u.x = pack_bf16(v[0], v[1]);
                    u.y = pack_bf16(v[2], v[3]);
                    u.z = pack_bf16(v[4], v[5]);
                    u.w = pack_bf16(v[6], v[7]);
                    *reinterpret_cast<uint4*>(wstage + lane * 144 + q * 16) = u;
                }
                if (piece) continue;
                __syncwarp();
                // eight neighbouring lanes write one row's 128 bytes: 4 lines per store instruction instead of 32
                __nv_bfloat16* obase = o + (size_t)(row0 + quad * 32) * o_ld + head * HD + hp * 64 + (lane & 7) * 8;
#pragma unroll 1
                for (int kk = 0; kk < 8; ++kk) {
                    const int rr = kk * 4 + (lane >> 3);      // row inside the warp's 32
                    const uint4 u = *reinterpret_cast<const uint4*>(wstage + rr * 144 + (lane & 7) * 16);
                    if (quad * 32 + rr < rows) *reinterpret_cast<uint4*>(obase + (size_t)rr * o_ld) = u;
                }
                __syncwarp();                                 // the staging rows are rewritten by the next pass / item
            }
        }
        if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 1700 + (int)blockIdx.x);
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // neither CTA leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, PA_TMEM_COLS);
    }
}

// Puts the pieces of the cut items together: O = sum_p c_p O_p / sum_p c_p l_p with c_p = 2^((m_p - m) scale).
// An item has up to 256 rows; the piece of part p left rows 0..127 in slot (ti * parts + p) * 2 and rows
// 128..255 in the slot after it (the two CTAs of the cluster that ran it).
constexpr int PCOMBINE_THREADS = 256;
__global__ void __launch_bounds__(PCOMBINE_THREADS)
attn_combine_pair_kernel(const float* __restrict__ ws, __nv_bfloat16* __restrict__ o, int o_ld, const QTile* __restrict__ tiles2,
                         int heads, int N, int n_clusters, float scale_log2, const Control* __restrict__ ctl) {
    constexpr int CG = HD / 4;                         // column groups of a row
    pdl_trigger();
    pdl_wait();
    const int n_tiles = ctl->n_qtiles2;
    const int n_items = n_tiles * heads;
    const int n_kv = (N + KEYS - 1) / KEYS;
    const CutPlan cut = cut_plan(n_items, n_kv, n_clusters, true);
    if (cut.parts < 2) return;
    const size_t slot = split_slot_floats(HD);
    for (int ti = blockIdx.x; ti < cut.n_tail; ti += gridDim.x) {
        const int w = cut.n_rounds * n_clusters + ti;
        const QTile t = tiles2[w % n_tiles];
        const int head = w / n_tiles;
        for (int idx = blockIdx.y * PCOMBINE_THREADS + threadIdx.x; idx < t.rows * CG; idx += gridDim.y * PCOMBINE_THREADS) {
            const int r = idx / CG, cg = idx - r * CG;
            const float* base = ws + ((size_t)ti * cut.parts * 2 + (r >> 7)) * slot + (size_t)(r & 127) * (HD + 4);
            float m = -INFINITY;
            for (int p = 0; p < cut.parts; ++p) m = fmaxf(m, base[(size_t)p * 2 * slot + HD]);
            float l = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int p = 0; p < cut.parts; ++p) {
                const float* row = base + (size_t)p * 2 * slot;
                const float c = ex2((row[HD] - m) * scale_log2);
                const float4 x = *reinterpret_cast<const float4*>(row + cg * 4);
                l = fmaf(c, row[HD + 1], l);
                acc.x = fmaf(c, x.x, acc.x); acc.y = fmaf(c, x.y, acc.y);
                acc.z = fmaf(c, x.z, acc.z); acc.w = fmaf(c, x.w, acc.w);
            }
            const float inv = 1.0f / l;
            uint2 u;
            u.x = pack_bf16(acc.x * inv, acc.y * inv);
            u.y = pack_bf16(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(o + (size_t)(t.row0 + r) * o_ld + head * HD + cg * 4) = u;
        }
    }
}

}  // namespace

bool tc_attention_pair_supported(const fd_config& c) { return c.dtype == FD_BF16 && c.head_dim == HD; }

cudaError_t tc_attention_pair_setup(int* max_clusters, int sm_count) {
    cudaError_t e = cudaFuncSetAttribute(tc_attention_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PA_SMEM);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PA_SMEM);
    if (e != cudaSuccess) return e;
    // as many CTA pairs as the device can keep resident at once
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3(sm_count & ~1);
    lc.blockDim = dim3(PA_THREADS);
    lc.dynamicSmemBytes = PA_SMEM;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    lc.attrs = at;
    lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, tc_attention_pair_kernel<false>, &lc) != cudaSuccess || n < 1) {
        cudaGetLastError();
        n = (sm_count & ~1) / 2;
    }
    *max_clusters = max(1, min(n, (sm_count & ~1) / 2));
    return cudaSuccess;
}

// tm_q: [q_ld, Mcap] boxes of 64 x 128.  The K / V maps are encoded here, per call (the cache pointer is an argument):
// [H, N, 2B] with boxes of 64 dims x 32 keys (a CTA's half of a key tile) and 64 dims x 64 keys (its half of V's head dims).
cudaError_t tc_attention_pair_launch(const CUtensorMap& tm_q, void* kv_block, int B, int H, void* o, int o_ld,
                                     const QTile* tiles2, int max_tiles2, int heads, int N, float scale_log2, float* split_ws,
                                     int split_slots, int max_clusters, bool may_cut, Control* ctl, cudaStream_t st, bool pdl,
                                     int* n_launch) {
    CUtensorMap tm_k, tm_v;
    const uint64_t dims[3] = {(uint64_t)H, (uint64_t)N, (uint64_t)B * 2};
    const uint64_t strides[2] = {(uint64_t)H * 2, (uint64_t)N * H * 2};
    const uint32_t box_k[3] = {64, KEYS / 2, 1}, box_v[3] = {64, KEYS, 1};
    std::string err;
    if (!encode_tmap_bf16(&tm_k, kv_block, 3, dims, strides, box_k, 128, &err)) return cudaErrorInvalidValue;
    if (!encode_tmap_bf16(&tm_v, kv_block, 3, dims, strides, box_v, 128, &err)) return cudaErrorInvalidValue;
    const int n_clusters = max(1, min(max_clusters, max_tiles2 * heads));
    const int grid = 2 * n_clusters;
    float* ws = (may_cut && split_ws && grid <= split_slots) ? split_ws : nullptr;
    __nv_bfloat16* ob = static_cast<__nv_bfloat16*>(o);
    cudaError_t e;
    if (ws) {
        e = launch_kernel(tc_attention_pair_kernel<true>, grid, PA_THREADS, PA_SMEM, st, pdl, tm_q, tm_k, tm_v, ob, o_ld, tiles2,
                          heads, N, scale_log2, ws, ctl);
        ++*n_launch;
        if (e == cudaSuccess) {
            const int cgrid = max(1, n_clusters / 2);        // at most half the clusters' worth of items can be cut
            e = launch_kernel(attn_combine_pair_kernel, dim3(cgrid, (2 * QROWS * (HD / 4) + PCOMBINE_THREADS - 1) / PCOMBINE_THREADS),
                              PCOMBINE_THREADS, 0, st, pdl, (const float*)ws, ob, o_ld, tiles2, heads, N, n_clusters, scale_log2,
                              (const Control*)ctl);
            ++*n_launch;
        }
    } else {
        e = launch_kernel(tc_attention_pair_kernel<false>, grid, PA_THREADS, PA_SMEM, st, pdl, tm_q, tm_k, tm_v, ob, o_ld, tiles2,
                          heads, N, scale_log2, (float*)nullptr, ctl);
        ++*n_launch;
    }
    return e;
}

}  // namespace fd
