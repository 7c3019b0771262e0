// Tensor-core attention of the active queries against all N keys of their request (fresh K/V rows
// of active tokens, previous-step rows of skipped tokens; paper Sec. 5 and Appendix A.6).
//
// One work item = one query tile (up to 128 compact rows of one request) x one head.  Persistent,
// warp-specialised CTAs of four warpgroups walk the device-built work list:
//   warp 0       TMA producer: Q tile (double buffered across items), K and V tiles (128 keys) in rings
//   warp 1       issues S = Q K^T (tcgen05.mma, both operands in shared memory) into the TMEM score buffer
//                as soon as the softmax has handed it back (one buffer; the older mass layouts below use two)
//   warp 2       issues O += P V with P read from TMEM and V as an N-major shared-memory operand
//   warps 4..11  softmax: tcgen05.ld of the scores, a reference maximum per row with lazy rescaling of O (a
//                tile's own maximum is computed only for a warpgroup's first tile of an item and when a
//                tile's row sum shows a score more than 2^24 above the reference), exp2, P written to TMEM
//                as packed bf16
//   warps 12..15 item epilogue (merge, normalise, store) while the softmax warps go on
// Warpgroup p takes the key tiles of parity p with its own P buffer,
// accumulator O_p and running maximum / row sum: one thread per row copies the tile's 128 scores to
// registers and hands the (single) score buffer back at once, so that the next S = Q K^T runs under
// this tile's exponentials; the two warpgroups never wait for each other.  The epilogue warpgroup
// merges the partial results, O = (a0 O_0 + a1 O_1) / (a0 l_0 + a1 l_1), a_p = 2^(m_p - m), while the
// softmax warps go on; at head dim 64 TMEM has room for four accumulators (item parity x tile
// parity), so the next item's products start under that merge.  Head dim 72 runs as 80.
// The mass variants of head dims 72 and 128 keep an older layout: one accumulator; two threads per query
// row, each with 64 of a tile's 128 keys, swap their partial maxima through shared memory and end the item
// themselves.
// Keys past N in the last tile are zero-filled by TMA and masked.
// For long key sequences the items of the last, partly filled round are cut along the keys (CutPlan below) and
// attn_combine_kernel puts their pieces together.
#include <cuda_bf16.h>

#include "attn_common.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace fd {

using namespace ptx;
using namespace attn;

void* tc_plan_attn(TcPlan* p);
int tc_plan_sm_count(TcPlan* p);
bool tc_plan_pdl(TcPlan* p);

namespace {

constexpr int ATT_THREADS = 512;          // 4 warpgroups: TMA/issuers, softmax x 2, item epilogue (head dim 64)
constexpr int QROWS = 128, KEYS = 128;
constexpr int SUB_BYTES = 128 * 64 * 2;          // one [128 x 64] bf16 sub-tile, 128-byte rows

constexpr int TAIL_BYTES = 128 * 16 * 2;         // one [128 x 16] bf16 sub-tile, 32-byte rows (head dim 72 only)

// Head dim 72 runs as 80: a 64-wide sub-tile (128-byte swizzle) plus a 16-wide one (32-byte swizzle).
// Q is stored with every head padded to 80 columns of which the last 8 are zero, so the 8 columns
// the 16-wide K sub-tile reads past its head contribute nothing; the matching 8 columns of O are
// never stored.
template <int D> struct AttCfg {
    static constexpr int DP = D == 72 ? 80 : D;                       // head dim as the MMAs see it
    static constexpr int SUBS = D / 64;                               // 64-wide sub-tiles
    static constexpr int TILE_BYTES = SUBS * SUB_BYTES + (D == 72 ? TAIL_BYTES : 0);
    // K/V rings deep enough that a tile is requested several tile periods before it is needed
    static constexpr int STAGES = D == 128 ? 2 : (D == 72 ? 4 : 5);
    static constexpr int SMEM = TILE_BYTES * (2 + 2 * STAGES) + 4608 + 128 * 144 + 2048;
};

// TMEM columns: two score buffers, the output accumulator, two P buffers (bf16 pairs)
constexpr uint32_t COL_S = 0, COL_O = 256, COL_P = 384, TMEM_COLS = 512;
// head dims 64 and 128: one score buffer, two P buffers (tile parity), accumulators from column 256: at head dim 64
// four (item parity x tile parity), at 128 two (tile parity)
constexpr uint32_t COL64_S = 0, COL64_P = 128, COL64_O = 256;
template <int D> __device__ __forceinline__ uint32_t acc_col(int item_i, int par) {
    return COL64_O + (uint32_t)((D == 64 ? (item_i & 1) * 2 : 0) + par) * (D == 72 ? 80 : D);
}

// What the MASS variant (head dim 64, launched for a step's first block when asked) needs on top: per region, the
// softmax mass its active queries put on keys of their own region (paper Sec. 4.2).
struct MassArgs {
    const int32_t* labels;       // [B, N]
    const int32_t* active_idx;   // compact row -> global token id
    double* region_mass;         // [B, R], accumulated with atomics
    int R;
    float inv_heads;
};

// CUT = false: whole items only, round after round (the plan is not looked at: the compiler sees constant bounds)
template <bool CUT>
__device__ __forceinline__ bool next_task(const CutPlan& c, int n_items, int n_kv, int k, Task& t) {
    if constexpr (!CUT) {
        const int w = (int)blockIdx.x + k * (int)gridDim.x;
        t = Task{w, 0, n_kv, 0};
        return w < n_items;
    }
    if (k < c.n_rounds) { t = Task{(int)blockIdx.x + k * (int)gridDim.x, 0, n_kv, 0}; return true; }
    if (k > c.n_rounds || (int)blockIdx.x >= c.n_tail * c.parts) return false;
    const int ti = (int)blockIdx.x / c.parts, pt = (int)blockIdx.x - ti * c.parts;
    const int j0 = pt * c.steps, j1 = j0 + c.steps < n_kv ? j0 + c.steps : n_kv;
    t = Task{c.n_rounds * (int)gridDim.x + ti, j0, j1, c.parts > 1 ? 1 : 0};
    return true;
}
template <int D, bool MASS = false, bool CUT = false>
__global__ void __launch_bounds__(ATT_THREADS, 1)
tc_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kv,
                    const __grid_constant__ CUtensorMap tm_q_tail, const __grid_constant__ CUtensorMap tm_kv_tail,
                    __nv_bfloat16* __restrict__ o, int o_ld, const QTile* __restrict__ tiles, int heads, int N,
                    float scale_log2, float* __restrict__ split_ws, Control* ctl, MassArgs ma) {
    using Cfg = AttCfg<D>;
    constexpr int DP = Cfg::DP;
    // tile-parity layout (an accumulator per softmax warpgroup, no exchange in the key loop); the mass variants of head
    // dims 72 and 128 stay on the two-threads-per-row layout (their label bookkeeping per score is cheaper there: 64
    // scores per thread)
    constexpr bool SPLIT = D == 64 || !MASS;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int TILE_BYTES = Cfg::TILE_BYTES;
    extern __shared__ __align__(1024) uint8_t smem[];    // 128-byte swizzled tiles need 1024-byte alignment
    uint8_t* sQ = smem;                                   // [2]
    uint8_t* sK = smem + 2 * TILE_BYTES;
    uint8_t* sV = sK + STAGES * TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + STAGES * TILE_BYTES);
    uint64_t* k_full = bars;                  // [STAGES]
    uint64_t* k_empty = k_full + STAGES;
    uint64_t* v_full = k_empty + STAGES;
    uint64_t* v_empty = v_full + STAGES;
    uint64_t* s_full = v_empty + STAGES;      // [2]  score tile ready
    uint64_t* p_full = s_full + 2;            // [2][2]  [buffer][0]: P written; [buffer][1] (head dim 64): the buffer's scores are in registers
    uint64_t* pv_done = p_full + 4;           // [2][2]  [buffer][0]: the product that read this P buffer has completed
    uint64_t* q_full = pv_done + 4;           // [2]
    uint64_t* q_empty = q_full + 2;           // [2]
    uint64_t* o_free = q_empty + 2;
    uint64_t* x_bar = o_free + 2;             // [4 quadrants][2]: the two threads of a row swap their partial maxima
    uint64_t* l_bar = x_bar + 8;              // [4 quadrants]: ... and, once per item, their partial sums
    uint64_t* stat_full = l_bar + 4;          // [2]  head dim 64: an item's row statistics are in shared memory
    uint64_t* stat_free = stat_full + 2;      // [2]  ... and have been read
    uint64_t* item_done = stat_free + 2;      // [2]  head dim 64: every product of an item (by item parity) has completed
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(item_done + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* s_xmax = reinterpret_cast<float*>(tmem_slot + 2);      // head dim 64: row maxima, [2 items][2 halves][128 rows]
    float* s_xsum = s_xmax + 512;                                 // [2 halves][128 rows]; head dim 64: [2 items][2 halves][128 rows]
    uint8_t* s_stage = reinterpret_cast<uint8_t*>(bars) + 4608;   // [128 rows][144 bytes], head dim 64 only
    // MASS: own-region mass, head dim 64 [2 items][2 halves][128 rows], otherwise [2 halves][128 rows]
    float* s_xown = reinterpret_cast<float*>(s_stage + (SPLIT ? 128 * 144 : 0));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (smem_u32(smem) & 1023u) {                        // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) report(ctl, FD_ERR_STATE, -1024);
        return;
    }
    const int n_kv = (N + KEYS - 1) / KEYS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&s_full[i], 1);
            mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1);
        }
        for (int i = 0; i < 4; ++i) { mbar_init(&p_full[i], SPLIT ? 4 : 8); mbar_init(&pv_done[i], 1); }
        for (int i = 0; i < 8; ++i) mbar_init(&x_bar[i], 64);
        for (int i = 0; i < 4; ++i) mbar_init(&l_bar[i], 64);
        mbar_init(&o_free[0], SPLIT ? 4 : 8);
        mbar_init(&o_free[1], SPLIT ? 4 : 8);
        for (int i = 0; i < 2; ++i) { mbar_init(&stat_full[i], 8); mbar_init(&stat_free[i], 4); mbar_init(&item_done[i], 1); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tm_q);
        prefetch_tmap(&tm_kv);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int wg = warp >> 2;                            // 0: TMA + MMA issuers, 1 and 2: softmax, 3: item epilogue
    // everything above is local set-up; from here on the kernel reads what earlier kernels wrote
    pdl_trigger();
    pdl_wait();
    // items are ordered head-major: the CTAs running at the same time work on the same one or two heads,
    // so that head's K/V stays in L2 however long the key sequence is
    const int n_tiles = ctl->n_qtiles;
    const int n_items = n_tiles * heads;
    static_assert(!(MASS && CUT), "the first block's mass variant never cuts items");
    const CutPlan cut = CUT ? cut_plan(n_items, n_kv, (int)gridDim.x, split_ws != nullptr) : CutPlan{0, 0, 1, 0};

    if (wg == 0) {
    reg_dec<48>();
    if (warp == 0) {
        // ---------------------------------------------------------------- TMA producer
        if (lane == 0) {
            uint32_t gk = 0;
            bool ok = true;
            int item_i = 0;
            Task tk;
            // The V tile of a key tile is requested one tile behind its K tile: K(g+1), then V(g).  A V stage is released
            // by the product P V two tiles back, long after the K stage of the same tile (released by S = Q K^T); issuing
            // K(g), V(g), K(g+1) in turn held every K load back behind that wait (timestamps at head dim 128, where the
            // rings are two stages deep: the S = Q K^T issuer waited 0.5 us of every 1.2 us tile for its K tile; -12 % on
            // the 480p video shape, -3 % at head dim 72).  With the five stages of head dim 64 nothing is held back and the
            // lag only costs a tile of V prefetch (+3 to +5 % there), so it is off.
            constexpr bool V_LAG = D != 64;
            int pv_head = 0, pv_j = 0, pv_b = -1;        // the V tile still to be requested (pv_b < 0: none)
            uint32_t pv_g = 0;
            auto load_v = [&](int head, int j, int b, uint32_t g) -> bool {
                const int s = g % STAGES;
                if (!mbar_wait(&v_empty[s], ((g / STAGES) & 1) ^ 1, abort_flag)) return false;
                mbar_expect_tx(&v_full[s], TILE_BYTES);
                if constexpr (D == 72) {
                    // V of a 72-wide head as five 16-column blocks (32-byte swizzle): one product of width 80 then
                    // reads all of them, where a 64-wide plus a 16-wide block would need two products per 16 keys
#pragma unroll
                    for (int a = 0; a < 5; ++a)
                        tma_load_3d(sV + s * TILE_BYTES + a * TAIL_BYTES, &tm_kv_tail, head * D + a * 16, j * KEYS, b * 2 + 1,
                                    &v_full[s]);
                } else {
#pragma unroll
                    for (int sb = 0; sb < Cfg::SUBS; ++sb)
                        tma_load_3d(sV + s * TILE_BYTES + sb * SUB_BYTES, &tm_kv, head * D + sb * 64, j * KEYS, b * 2 + 1,
                                    &v_full[s]);
                }
                return true;
            };
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                const QTile t = tiles[w % n_tiles];
                const int head = w / n_tiles;
                const int qs = item_i & 1;
                if (item_i >= 2 && !mbar_wait(&q_empty[qs], ((item_i >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&q_full[qs], TILE_BYTES);
#pragma unroll
                for (int sb = 0; sb < Cfg::SUBS; ++sb)
                    tma_load_2d(sQ + qs * TILE_BYTES + sb * SUB_BYTES, &tm_q, head * DP + sb * 64, t.row0, &q_full[qs]);
                if constexpr (D == 72)
                    tma_load_2d(sQ + qs * TILE_BYTES + SUB_BYTES, &tm_q_tail, head * DP + 64, t.row0, &q_full[qs]);
                for (int j = tk.j0; j < tk.j1; ++j, ++gk) {
                    const int s = gk % STAGES;
                    const uint32_t ph = ((gk / STAGES) & 1) ^ 1;
                    if (!mbar_wait(&k_empty[s], ph, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&k_full[s], TILE_BYTES);
#pragma unroll
                    for (int sb = 0; sb < Cfg::SUBS; ++sb)
                        tma_load_3d(sK + s * TILE_BYTES + sb * SUB_BYTES, &tm_kv, head * D + sb * 64, j * KEYS,
                                    t.b * 2 + 0, &k_full[s]);
                    if constexpr (D == 72)
                        tma_load_3d(sK + s * TILE_BYTES + SUB_BYTES, &tm_kv_tail, head * D + 64, j * KEYS, t.b * 2 + 0,
                                    &k_full[s]);
                    if constexpr (V_LAG) {
                        if (pv_b >= 0 && !load_v(pv_head, pv_j, pv_b, pv_g)) { ok = false; break; }
                        pv_head = head; pv_j = j; pv_b = t.b; pv_g = gk;
                    } else {
                        if (!load_v(head, j, t.b, gk)) { ok = false; break; }
                    }
                }
            }
            if (ok && pv_b >= 0 && !load_v(pv_head, pv_j, pv_b, pv_g)) ok = false;
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 400 + (int)blockIdx.x);
        }
    } else if (warp == 1) {
        // ---------------------------------------------------------------- S = Q K^T issuer
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(QROWS, KEYS, 0, 0);
            uint32_t g = 0;
            bool ok = true;
            int item_i = 0;
            Task tk;
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                const int qs = item_i & 1;
                if (!mbar_wait(&q_full[qs], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
                const uint32_t q_addr = smem_u32(sQ + qs * TILE_BYTES);
                for (int j = tk.j0; j < tk.j1; ++j, ++g) {
                    const int s = g % STAGES;
                    if (!mbar_wait(&k_full[s], (g / STAGES) & 1, abort_flag)) { ok = false; break; }
                    // the score buffer is free once the softmax has finished the tile that used it last
                    if constexpr (SPLIT) {
                        // one score buffer: free once the previous tile's scores are in its warpgroup's registers
                        if (g >= 1 && !mbar_wait(&p_full[((g - 1) & 1) * 2 + 1], ((g - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                    } else {
                        if (g >= 2 && !mbar_wait(&p_full[(g & 1) * 2], ((g - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
                    }
                    tc_fence_after();
                    const uint32_t d = tmem_base + (SPLIT ? COL64_S : COL_S + (g & 1) * 128);
                    const uint32_t k_addr = smem_u32(sK + s * TILE_BYTES);
#pragma unroll
                    for (int ks = 0; ks < Cfg::SUBS * 4; ++ks) {
                        const uint32_t off = (ks / 4) * SUB_BYTES + (ks % 4) * 32;
                        mma_bf16_ss(d, smem_desc(q_addr + off, 16, 1024, SWZ_128B),
                                    smem_desc(k_addr + off, 16, 1024, SWZ_128B), idesc_qk, ks != 0);
                    }
                    if constexpr (D == 72)      // columns 64..79: 32-byte rows, 8-row groups 256 bytes apart
                        mma_bf16_ss(d, smem_desc(q_addr + SUB_BYTES, 16, 256, SWZ_32B),
                                    smem_desc(k_addr + SUB_BYTES, 16, 256, SWZ_32B), idesc_qk, 1);
                    mma_commit(&k_empty[s]);
                    mma_commit(&s_full[g & 1]);
                    if (j == tk.j1 - 1) mma_commit(&q_empty[qs]);
                }
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 500 + (int)blockIdx.x);
        }
    } else if (warp == 2) {
        // ---------------------------------------------------------------- O += P V issuer
        if (lane == 0) {
            constexpr uint32_t idesc_pv = idesc_bf16(QROWS, DP, 0, 1);   // V: head dim contiguous (N-major)
            uint32_t g = 0;
            bool ok = true;
            int item_i = 0;
            Task tk;
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                for (int j = tk.j0; j < tk.j1; ++j, ++g) {
                    const int s = g % STAGES;
                    if (!mbar_wait(&v_full[s], (g / STAGES) & 1, abort_flag)) { ok = false; break; }
                    if constexpr (SPLIT) {
                        if constexpr (D == 64) {
                            // the accumulators alternate from item to item: these were last used two items ago
                            if (j == tk.j0 && item_i >= 2 && !mbar_wait(&o_free[item_i & 1], ((item_i >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                        } else {
                            if (j == tk.j0 && item_i > 0 && !mbar_wait(&o_free[0], (item_i - 1) & 1, abort_flag)) { ok = false; break; }
                        }
                    } else {
                        if (j == tk.j0 && item_i > 0 && !mbar_wait(&o_free[0], (item_i - 1) & 1, abort_flag)) { ok = false; break; }
                    }
                    const uint32_t v_addr = smem_u32(sV + s * TILE_BYTES);
                    if constexpr (SPLIT) {
                        // the tiles of one parity accumulate into their own O: even tiles O_0, odd tiles O_1
                        if (!mbar_wait(&p_full[(g & 1) * 2], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const uint32_t d = tmem_base + acc_col<D>(item_i, g & 1);
                        const uint32_t a = tmem_base + COL64_P + (g & 1) * 64;
#pragma unroll
                        for (int ks = 0; ks < KEYS / 16; ++ks) {
                            if constexpr (D == 72)
                                // 16 keys further: two 8-key groups of 256 bytes; the 16-column blocks sit TAIL_BYTES apart
                                mma_bf16_ts(d, a + ks * 8, smem_desc(v_addr + ks * 512, TAIL_BYTES, 256, SWZ_32B), idesc_pv,
                                            j - tk.j0 >= 2 || ks != 0);
                            else
                                mma_bf16_ts(d, a + ks * 8, smem_desc(v_addr + ks * 2048, SUB_BYTES, 1024, SWZ_128B), idesc_pv,
                                            j - tk.j0 >= 2 || ks != 0);
                        }
                        mma_commit(&v_empty[s]);
                        mma_commit(&pv_done[(g & 1) * 2]);
                        // the item's products complete in issue order: this one covers them all.  (Its own barrier: the
                        // per-tile ones run on into the next item and their parity would alias for a late epilogue.)
                        if (j == tk.j1 - 1) mma_commit(&item_done[item_i & 1]);
                        continue;
                    }
                    if (!mbar_wait(&p_full[(g & 1) * 2], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t d = tmem_base + COL_O;
                    const uint32_t a = tmem_base + COL_P + (g & 1) * 64;
#pragma unroll
                    for (int ks = 0; ks < KEYS / 16; ++ks) {
                        if constexpr (D == 72)
                            // 16 keys further: two 8-key groups of 256 bytes; the 16-column blocks sit TAIL_BYTES apart
                            mma_bf16_ts(d, a + ks * 8, smem_desc(v_addr + ks * 512, TAIL_BYTES, 256, SWZ_32B), idesc_pv,
                                        (j != tk.j0 || ks != 0));
                        else
                            // 16 keys further: 16 rows of 128 bytes; the second 64-wide half of V sits SUB_BYTES away
                            mma_bf16_ts(d, a + ks * 8, smem_desc(v_addr + ks * 2048, SUB_BYTES, 1024, SWZ_128B), idesc_pv,
                                        (j != tk.j0 || ks != 0));
                    }
                    mma_commit(&v_empty[s]);
                    mma_commit(&pv_done[(g & 1) * 2]);
                }
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 550 + (int)blockIdx.x);
        }
    }
    } else if (wg == 1 || wg == 2) {
        // ---------------------------------------------------------------- softmax
        if constexpr (SPLIT) reg_inc<184>(); else reg_inc<200>();
        if constexpr (SPLIT) {
            // Warpgroup `par` owns the key tiles of its parity (by the CTA-wide tile counter) with their score buffer,
            // P buffer and accumulator O_par: one thread per query row, all 128 keys of the tile.  The two warpgroups
            // never wait for each other, so on every scheduler one warp's exponentials overlap the other's loads,
            // maxima, conversions and barrier hand-offs.
            const int quad = warp & 3;
            const int par = wg - 1;
            const int r = quad * 32 + lane;                       // query row inside the tile
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
            const uint32_t s_addr = lane_addr + COL64_S;
            const uint32_t p_addr = lane_addr + COL64_P + par * 64;
            uint32_t g0 = 0;
            bool ok = true;
            int item_i = 0;
            const int rem = N - (n_kv - 1) * KEYS;                // valid keys of the last tile
            const uint64_t sc2 = pair(scale_log2, scale_log2);
            Task tk;
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                float m = -INFINITY, l = 0.f;
                const uint32_t o_addr = lane_addr + acc_col<D>(item_i, par);
                // MASS: the part of l that comes from keys carrying the query's own region label
                float own = 0.f;
                int my_lab = -1;
                const int32_t* key_lab = nullptr;
                if constexpr (MASS) {
                    const QTile t = tiles[w % n_tiles];
                    if (r < t.rows) my_lab = ma.labels[ma.active_idx[t.row0 + r]];
                    key_lab = ma.labels + (size_t)t.b * N;
                }
                for (int j = tk.j0 + ((g0 & 1) == (uint32_t)par ? 0 : 1); j < tk.j1 && ok; j += 2) {
                    const uint32_t g = g0 + (j - tk.j0);
                    if (!mbar_wait(&s_full[par], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const bool tail = j == n_kv - 1 && rem < KEYS;
                    const bool first = j - tk.j0 < 2;            // this warpgroup's first tile of the item (or piece)
                    uint32_t sr[128];
#pragma unroll
                    for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + c * 32, sr + c * 32);
                    tmem_wait_ld();
                    // the scores are in registers: the buffer can take this warpgroup's next tile already
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&p_full[par * 2 + 1]);
                    if (tail) {
#pragma unroll
                        for (int i = 0; i < 128; ++i) if (i >= rem) sr[i] = 0xff800000u;          // -inf
                    }
                    // the P buffer is free, and O_par complete, once the product of this warpgroup's previous tile is done
                    if (g >= 2 && !mbar_wait(&pv_done[par * 2], ((g >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    // The tile's own maximum is only computed when it is needed: for the warpgroup's first tile of an
                    // item, and when a tile's row sum shows that some score outgrew the reference maximum m by more
                    // than the rescaling threshold (p <= 2^24 for all 128 keys keeps the sum at or below 2^31; an
                    // overflow gives inf or NaN, which fails the same comparison).  Then the tile is done again with
                    // its true maximum: P is simply overwritten, nothing has consumed it yet.  (The mass variant keeps
                    // the maximum per tile: its label bookkeeping could not be redone.)
                    bool with_max = first || MASS;
#pragma unroll 1
                    for (;;) {
                        if (with_max) {
                            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                            for (int i = 0; i < 128; i += 8) {   // three-input maxima: half the instructions
                                mx0 = max3(mx0, __uint_as_float(sr[i]), __uint_as_float(sr[i + 1]));
                                mx1 = max3(mx1, __uint_as_float(sr[i + 2]), __uint_as_float(sr[i + 3]));
                                mx2 = max3(mx2, __uint_as_float(sr[i + 4]), __uint_as_float(sr[i + 5]));
                                mx3 = max3(mx3, __uint_as_float(sr[i + 6]), __uint_as_float(sr[i + 7]));
                            }
                            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                            if (first) {
                                m = mx;
                            } else {
                                const bool need = (mx - m) * scale_log2 > RESCALE_LOG2;
                                if (__any_sync(0xffffffffu, need)) {
                                    tc_fence_after();
                                    const float f = need ? ex2((m - mx) * scale_log2) : 1.0f;
                                    if (need) { l *= f; own *= f; m = mx; }
#pragma unroll 1
                                    for (int c = 0; c < D / 8; ++c) {    // rare, and 128 scores are live: small pieces
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
                        }
                        const float mb = m * scale_log2;
                        const uint64_t nmb2 = pair(-mb, -mb);
                        uint64_t sua = pair(0.f, 0.f), sub_ = pair(0.f, 0.f);
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            int kl = -2;                             // MASS: label of key `lane` of this chunk
                            if constexpr (MASS) {
                                const int k0 = j * KEYS + c * 32 + lane;
                                if (k0 < N) kl = __ldg(key_lab + k0);
                            }
                            uint32_t pk[16];
#pragma unroll
                            for (int i = 0; i < 16; i += 4) {
                                float p[8];
#pragma unroll
                                for (int e = 0; e < 4; ++e) {
                                    const uint64_t x = fma2(pair(__uint_as_float(sr[c * 32 + 2 * i + 2 * e]),
                                                                 __uint_as_float(sr[c * 32 + 2 * i + 2 * e + 1])), sc2, nmb2);
                                    // all on the special-function unit: a cubic on the FMA pipe costs six times the
                                    // instructions (measured: no share 4 % faster at 1024 keys than a quarter, within
                                    // 1 % at 8192)
                                    float xa, xb;
                                    unpair(x, xa, xb);
                                    p[2 * e] = ex2(xa);
                                    p[2 * e + 1] = ex2(xb);
                                }
                                sua = add2(sua, add2(pair(p[0], p[1]), pair(p[2], p[3])));
                                sub_ = add2(sub_, add2(pair(p[4], p[5]), pair(p[6], p[7])));
                                if constexpr (MASS) {
#pragma unroll
                                    for (int e = 0; e < 8; ++e) {
                                        const int klk = __shfl_sync(0xffffffffu, kl, 2 * i + e);
                                        own += klk == my_lab ? p[e] : 0.f;
                                    }
                                }
#pragma unroll
                                for (int e = 0; e < 4; ++e) pk[i + e] = pack_bf16(p[2 * e], p[2 * e + 1]);
                            }
                            tmem_st16(p_addr + c * 16, pk);
                        }
                        float s0, s1;
                        unpair(add2(sua, sub_), s0, s1);
                        const float tile_sum = s0 + s1;
                        if (with_max || !__any_sync(0xffffffffu, !(tile_sum <= 2147483648.0f))) {
                            l += tile_sum;
                            break;
                        }
                        with_max = true;
                    }
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&p_full[par * 2]);
                }
                if (!ok) break;
                // hand the row's statistics of this warpgroup's tiles to the epilogue warps and go on with the next
                // item; the slot was last used two items ago.  No tile at all (one-tile items): m = -inf, l = 0.
                const int slot = item_i & 1;
                if (item_i >= 2 && !mbar_wait(&stat_free[slot], ((item_i >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                s_xmax[(slot * 2 + par) * 128 + r] = m;
                s_xsum[(slot * 2 + par) * 128 + r] = l;
                if constexpr (MASS) s_xown[(slot * 2 + par) * 128 + r] = own;
                __syncwarp();
                if (lane == 0) mbar_arrive(&stat_full[slot]);
                g0 += tk.j1 - tk.j0;
            }
            if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 650 + (int)blockIdx.x);
        } else {
            const int quad = warp & 3;
            const int half = wg - 1;                              // which 64 keys of a tile / which half of O
            const int r = quad * 32 + lane;                       // query row inside the tile
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
            // output columns this thread owns: [half * DH, half * DH + DH), and for head dim 72 thread 0 also 64..79
            constexpr int DH = D == 72 ? 32 : D / 2;
            uint32_t g0 = 0;
            bool ok = true;
            int item_i = 0;
            const int rem = N - (n_kv - 1) * KEYS;                // valid keys of the last tile
            Task tk;
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                const QTile t = tiles[w % n_tiles];
                const int head = w / n_tiles;
                float m = -INFINITY, l = 0.f;
                // MASS: the part of l that comes from keys carrying the query's own region label
                float own = 0.f;
                int my_lab = -1;
                const int32_t* key_lab = nullptr;
                if constexpr (MASS) {
                    if (r < t.rows) my_lab = ma.labels[ma.active_idx[t.row0 + r]];
                    if (my_lab >= ma.R) my_lab = -1;
                    key_lab = ma.labels + (size_t)t.b * N;
                }
                for (int j = tk.j0; j < tk.j1 && ok; ++j) {
                    const uint32_t g = g0 + (j - tk.j0), bs = g & 1;
                    if (!mbar_wait(&s_full[bs], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    int kl0 = -2, kl1 = -2;                      // MASS: labels of this half's keys lane, lane + 32
                    if constexpr (MASS) {
                        const int k0 = j * KEYS + half * 64 + lane;
                        if (k0 < N) kl0 = __ldg(key_lab + k0);
                        if (k0 + 32 < N) kl1 = __ldg(key_lab + k0 + 32);
                    }
                    uint32_t sr[64];
                    tmem_ld32(lane_addr + COL_S + bs * 128 + half * 64, sr);
                    tmem_ld32(lane_addr + COL_S + bs * 128 + half * 64 + 32, sr + 32);
                    tmem_wait_ld();
                    if (j == n_kv - 1 && rem < KEYS) {
    #pragma unroll
                        for (int i = 0; i < 64; ++i) if (half * 64 + i >= rem) sr[i] = 0xff800000u;          // -inf
                    }
                    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
    #pragma unroll
                    for (int i = 0; i < 64; i += 4) {
                        mx0 = fmaxf(mx0, __uint_as_float(sr[i]));
                        mx1 = fmaxf(mx1, __uint_as_float(sr[i + 1]));
                        mx2 = fmaxf(mx2, __uint_as_float(sr[i + 2]));
                        mx3 = fmaxf(mx3, __uint_as_float(sr[i + 3]));
                    }
                    float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                    // row maximum over all 128 keys: swap partial maxima with the row's other thread
                    s_xmax[bs * 256 + half * 128 + r] = mx;
                    mbar_arrive(&x_bar[quad * 2 + bs]);
                    if (!mbar_wait(&x_bar[quad * 2 + bs], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                    mx = fmaxf(mx, s_xmax[bs * 256 + (half ^ 1) * 128 + r]);
                    if (j == tk.j0) {
                        m = mx;
                    } else {
                        const bool need = (mx - m) * scale_log2 > RESCALE_LOG2;
                        if (__any_sync(0xffffffffu, need)) {
                            // all earlier P V products must have landed before O is rescaled
                            if (!mbar_wait(&pv_done[((g - 1) & 1) * 2], ((g - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
                            tc_fence_after();
                            const float f = need ? ex2((m - mx) * scale_log2) : 1.0f;
                            if (need) { l *= f; m = mx; own *= f; }
    #pragma unroll
                            for (int c = 0; c < DH / 32; ++c) {
                                uint32_t orr[32];
                                tmem_ld32(lane_addr + COL_O + half * DH + c * 32, orr);
                                tmem_wait_ld();
    #pragma unroll
                                for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
                                tmem_st32(lane_addr + COL_O + half * DH + c * 32, orr);
                            }
                            if constexpr (D == 72) {
                                if (half == 0) {
                                    uint32_t ot[16];
                                    tmem_ld16(lane_addr + COL_O + 64, ot);
                                    tmem_wait_ld();
    #pragma unroll
                                    for (int i = 0; i < 16; ++i) ot[i] = __float_as_uint(__uint_as_float(ot[i]) * f);
                                    tmem_st16(lane_addr + COL_O + 64, ot);
                                }
                            }
                            tmem_wait_st();
                        }
                    }
                    const float mb = m * scale_log2;
                    uint32_t pk[32];
                    // of every 8 exponentials 6 go to the special-function unit and 2 to the FMA pipe
                    const uint64_t sc2 = pair(scale_log2, scale_log2), nmb2 = pair(-mb, -mb);
                    uint64_t sua = pair(0.f, 0.f), sub_ = pair(0.f, 0.f);
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        float p[8];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const uint64_t x = fma2(pair(__uint_as_float(sr[2 * i + 2 * e]), __uint_as_float(sr[2 * i + 2 * e + 1])), sc2, nmb2);
                            if (MASS || e < 3) {                 // MASS: no polynomial share, the body must stay small
                                float xa, xb;
                                unpair(x, xa, xb);
                                p[2 * e] = ex2(xa);
                                p[2 * e + 1] = ex2(xb);
                            } else {
                                unpair(ex2_poly2(x), p[2 * e], p[2 * e + 1]);
                            }
                        }
                        sua = add2(sua, add2(pair(p[0], p[1]), pair(p[2], p[3])));
                        sub_ = add2(sub_, add2(pair(p[4], p[5]), pair(p[6], p[7])));
                        if constexpr (MASS) {
#pragma unroll
                            for (int e = 0; e < 8; ++e) {
                                const int kk = 2 * i + e;
                                const int kl = __shfl_sync(0xffffffffu, kk < 32 ? kl0 : kl1, kk & 31);
                                own += kl == my_lab ? p[e] : 0.f;
                            }
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e) pk[i + e] = pack_bf16(p[2 * e], p[2 * e + 1]);
                    }
                    {
                        float s0, s1;
                        unpair(add2(sua, sub_), s0, s1);
                        l += s0 + s1;
                    }
                    // the P buffer is free once the product that read it two tiles ago has completed
                    if (g >= 2 && !mbar_wait(&pv_done[bs * 2], ((g >> 1) - 1) & 1, abort_flag)) { ok = false; break; }
                    tmem_st32(lane_addr + COL_P + bs * 64 + half * 32, pk);
                    tmem_wait_st();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&p_full[bs * 2]);
                }
                if (!ok) break;
                // epilogue: O / l for the rows of this tile (l = the two halves' partial sums)
                const uint32_t gl = g0 + (tk.j1 - tk.j0) - 1;
                s_xsum[half * 128 + r] = l;
                if constexpr (MASS) s_xown[half * 128 + r] = own;
                mbar_arrive(&l_bar[quad]);
                if (!mbar_wait(&l_bar[quad], item_i & 1, abort_flag)) { ok = false; break; }
                // a cut item's piece stays un-normalised: its rows, maximum, sum (and mass) go to the CTA's scratch slot
                const bool piece = CUT && tk.piece != 0;
                const float inv = piece ? 1.0f : 1.0f / (l + s_xsum[(half ^ 1) * 128 + r]);
                float* prow = split_ws + (size_t)blockIdx.x * split_slot_floats(DP) + (size_t)r * (DP + 4);
                if (piece && half == 0) {
                    prow[DP] = m;
                    prow[DP + 1] = l + s_xsum[128 + r];
                    if constexpr (MASS) prow[DP + 2] = own + s_xown[128 + r];
                }
                if (MASS && !piece) {
                    if (half == 0) {      // one of the row's two threads reports; the lanes of one label add up first
                        const float mine = my_lab >= 0 ? (own + s_xown[128 + r]) * inv * ma.inv_heads : 0.f;
                        const uint32_t peers = __match_any_sync(0xffffffffu, my_lab);
                        float sum = 0.f;
                        for (uint32_t rest = peers; rest; rest &= rest - 1) sum += __shfl_sync(peers, mine, __ffs(rest) - 1);
                        if (my_lab >= 0 && lane == __ffs(peers) - 1)
                            atomicAdd(&ma.region_mass[(size_t)t.b * ma.R + my_lab], (double)sum);
                    }
                }
                if (!mbar_wait(&pv_done[(gl & 1) * 2], (gl >> 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                __nv_bfloat16* dst = o + (size_t)(t.row0 + r) * o_ld + head * D + half * DH;
    #pragma unroll
                for (int c = 0; c < DH / 32; ++c) {
                    uint32_t orr[32];
                    tmem_ld32(lane_addr + COL_O + half * DH + c * 32, orr);
                    tmem_wait_ld();
                    if (piece) {
    #pragma unroll
                        for (int v = 0; v < 8; ++v)
                            *reinterpret_cast<float4*>(prow + half * DH + c * 32 + v * 4) =
                                make_float4(__uint_as_float(orr[4 * v]), __uint_as_float(orr[4 * v + 1]),
                                            __uint_as_float(orr[4 * v + 2]), __uint_as_float(orr[4 * v + 3]));
                    } else if (r < t.rows) {
    #pragma unroll
                        for (int v = 0; v < 4; ++v) {
                            uint4 u;
                            u.x = pack_bf16(__uint_as_float(orr[8 * v + 0]) * inv, __uint_as_float(orr[8 * v + 1]) * inv);
                            u.y = pack_bf16(__uint_as_float(orr[8 * v + 2]) * inv, __uint_as_float(orr[8 * v + 3]) * inv);
                            u.z = pack_bf16(__uint_as_float(orr[8 * v + 4]) * inv, __uint_as_float(orr[8 * v + 5]) * inv);
                            u.w = pack_bf16(__uint_as_float(orr[8 * v + 6]) * inv, __uint_as_float(orr[8 * v + 7]) * inv);
                            *reinterpret_cast<uint4*>(dst + c * 32 + v * 8) = u;
                        }
                    }
                }
                if constexpr (D == 72) {
                    if (half == 0) {                          // columns 64..71 of the head
                        uint32_t ot[8];
                        tmem_ld8(lane_addr + COL_O + 64, ot);
                        tmem_wait_ld();
                        if (piece) {
                            *reinterpret_cast<float4*>(prow + 64) = make_float4(__uint_as_float(ot[0]), __uint_as_float(ot[1]),
                                                                                __uint_as_float(ot[2]), __uint_as_float(ot[3]));
                            *reinterpret_cast<float4*>(prow + 68) = make_float4(__uint_as_float(ot[4]), __uint_as_float(ot[5]),
                                                                                __uint_as_float(ot[6]), __uint_as_float(ot[7]));
                        } else if (r < t.rows) {
                            uint4 u;
                            u.x = pack_bf16(__uint_as_float(ot[0]) * inv, __uint_as_float(ot[1]) * inv);
                            u.y = pack_bf16(__uint_as_float(ot[2]) * inv, __uint_as_float(ot[3]) * inv);
                            u.z = pack_bf16(__uint_as_float(ot[4]) * inv, __uint_as_float(ot[5]) * inv);
                            u.w = pack_bf16(__uint_as_float(ot[6]) * inv, __uint_as_float(ot[7]) * inv);
                            *reinterpret_cast<uint4*>(o + (size_t)(t.row0 + r) * o_ld + head * D + 64) = u;
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&o_free[0]);
                g0 += tk.j1 - tk.j0;
            }
            if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 600 + (int)blockIdx.x);
        }
    } else {
        // ---------------------------------------------------------------- item epilogue (head dim 64)
        if constexpr (SPLIT) reg_dec<96>(); else reg_dec<48>();
        // One thread per query row: merge the two halves' accumulators with the statistics the softmax warps
        // left, normalise and store, while those warps are already in the next item's key loop.
        if constexpr (SPLIT) {
            const int quad = warp & 3;
            const int r = quad * 32 + lane;
            const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
            // staging rows are 144 bytes apart so that the 16-byte stores of a quarter warp fall into different banks
            uint8_t* wstage = s_stage + quad * 32 * 144;
            bool ok = true;
            int item_i = 0;
            Task tk, tk_next;
            // the work item's descriptor is fetched one item ahead
            QTile t_next = next_task<CUT>(cut, n_items, n_kv, 0, tk_next) ? tiles[tk_next.w % n_tiles] : QTile{0, 0, 0, 0};
            for (int k = 0; ok && next_task<CUT>(cut, n_items, n_kv, k, tk); ++k, ++item_i) {
                const int w = tk.w;
                const QTile t = t_next;
                if (next_task<CUT>(cut, n_items, n_kv, k + 1, tk_next)) t_next = tiles[tk_next.w % n_tiles];
                const int head = w / n_tiles;
                const int slot = item_i & 1;
                if (!mbar_wait(&stat_full[slot], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
                const float m0 = s_xmax[(slot * 2 + 0) * 128 + r], l0 = s_xsum[(slot * 2 + 0) * 128 + r];
                const float m1 = s_xmax[(slot * 2 + 1) * 128 + r], l1 = s_xsum[(slot * 2 + 1) * 128 + r];
                float own0 = 0.f, own1 = 0.f;
                if constexpr (MASS) { own0 = s_xown[(slot * 2 + 0) * 128 + r]; own1 = s_xown[(slot * 2 + 1) * 128 + r]; }
                __syncwarp();
                if (lane == 0) mbar_arrive(&stat_free[slot]);
                // every product of the item must have landed
                if (!mbar_wait(&item_done[slot], (item_i >> 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const float m_all = fmaxf(m0, m1);                // finite: at least one of the two had a tile
                const float a0 = m0 == -INFINITY ? 0.f : ex2((m0 - m_all) * scale_log2);
                const float a1 = m1 == -INFINITY ? 0.f : ex2((m1 - m_all) * scale_log2);
                // a cut item's piece stays un-normalised: its rows, maximum, sum (and mass) go to the CTA's scratch slot
                const bool piece = CUT && tk.piece != 0;
                const float inv = piece ? 1.0f : 1.0f / (a0 * l0 + a1 * l1);
                const float w_0 = a0 * inv, w_1 = a1 * inv;       // weights of O_0, O_1
                float* prow = split_ws + (size_t)blockIdx.x * split_slot_floats(DP) + (size_t)r * (DP + 4);
                if (piece) {
                    prow[DP] = m_all;
                    prow[DP + 1] = a0 * l0 + a1 * l1;
                    if constexpr (MASS) prow[DP + 2] = a0 * own0 + a1 * own1;
                }
                if (MASS && !piece) {
                    // consecutive compact rows mostly share their region: the lanes of one label add up first, so that a
                    // region receives one atomic per warp instead of one per row
                    int lab = -1;
                    if (r < t.rows) lab = ma.labels[ma.active_idx[t.row0 + r]];
                    if (lab >= ma.R) lab = -1;
                    const float mine = lab >= 0 ? (w_0 * own0 + w_1 * own1) * ma.inv_heads : 0.f;
                    const uint32_t peers = __match_any_sync(0xffffffffu, lab);
                    float sum = 0.f;
                    for (uint32_t rest = peers; rest; rest &= rest - 1)
                        sum += __shfl_sync(peers, mine, __ffs(rest) - 1);
                    if (lab >= 0 && lane == __ffs(peers) - 1) atomicAdd(&ma.region_mass[(size_t)t.b * ma.R + lab], (double)sum);
                }
                // rolled loops on purpose: this code runs once per item, and the fewer instructions it fetches the
                // less it disturbs the softmax warps that share the instruction caches.  64 output columns per pass.
                const uint32_t acc0 = lane_addr + acc_col<D>(item_i, 0), acc1 = lane_addr + acc_col<D>(item_i, 1);
#pragma unroll 1
                for (int hp = 0; hp < D / 64; ++hp) {
#pragma unroll 1
                    for (int q = 0; q < 8; ++q) {
                        uint32_t o0[8], o1[8];
                        tmem_ld8(acc0 + hp * 64 + q * 8, o0);
                        tmem_ld8(acc1 + hp * 64 + q * 8, o1);
                        tmem_wait_ld();
                        if (D != 72 && hp == D / 64 - 1 && q == 7) {
                            // the accumulators are free for the next item as soon as they are in registers
                            tc_fence_before();
                            __syncwarp();
                            if (lane == 0) mbar_arrive(&o_free[D == 64 ? slot : 0]);
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
                    __nv_bfloat16* obase = o + (size_t)(t.row0 + quad * 32) * o_ld + head * D + hp * 64 + (lane & 7) * 8;
#pragma unroll 1
                    for (int k = 0; k < 8; ++k) {
                        const int rr = k * 4 + (lane >> 3);       // row inside the warp's 32
                        const uint4 u = *reinterpret_cast<const uint4*>(wstage + rr * 144 + (lane & 7) * 16);
                        if (quad * 32 + rr < t.rows) *reinterpret_cast<uint4*>(obase + (size_t)rr * o_ld) = u;
                    }
                    __syncwarp();                                 // the staging rows are rewritten by the next pass / item
                }
                if constexpr (D == 72) {
                    // columns 64..71 of the head: 16 bytes per row, stored by the row's thread
                    uint32_t o0[8], o1[8];
                    tmem_ld8(acc0 + 64, o0);
                    tmem_ld8(acc1 + 64, o1);
                    tmem_wait_ld();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&o_free[0]);
                    float v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float x0 = w_0 != 0.f ? __uint_as_float(o0[i]) * w_0 : 0.f;
                        const float x1 = w_1 != 0.f ? __uint_as_float(o1[i]) * w_1 : 0.f;
                        v[i] = x0 + x1;
                    }
                    if (piece) {
                        *reinterpret_cast<float4*>(prow + 64) = make_float4(v[0], v[1], v[2], v[3]);
                        *reinterpret_cast<float4*>(prow + 68) = make_float4(v[4], v[5], v[6], v[7]);
                    } else if (r < t.rows) {
                        uint4 u;
                        u.x = pack_bf16(v[0], v[1]);
                        u.y = pack_bf16(v[2], v[3]);
                        u.z = pack_bf16(v[4], v[5]);
                        u.w = pack_bf16(v[6], v[7]);
                        *reinterpret_cast<uint4*>(o + (size_t)(t.row0 + r) * o_ld + head * D + 64) = u;
                    }
                }
            }
            if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 700 + (int)blockIdx.x);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

// Puts the pieces of the cut items together: O = sum_p c_p O_p / sum_p c_p l_p with c_p = 2^((m_p - m) scale).
// One CTA per cut item (att_grid = the grid the attention kernel ran with); a thread takes four neighbouring
// columns of a row at a time, so that a row's threads read and write whole lines and every thread has several
// independent loads in flight (the statistics of a row are re-read by its threads: L1 hits).
constexpr int COMBINE_THREADS = 256;
template <int D>
__global__ void __launch_bounds__(COMBINE_THREADS)
attn_combine_kernel(const float* __restrict__ ws, __nv_bfloat16* __restrict__ o, int o_ld, const QTile* __restrict__ tiles,
                    int heads, int N, int att_grid, float scale_log2, const Control* __restrict__ ctl) {
    constexpr int DP = AttCfg<D>::DP;
    constexpr int CG = D / 4;                          // column groups of a row
    pdl_trigger();
    pdl_wait();
    const int n_tiles = ctl->n_qtiles;
    const int n_items = n_tiles * heads;
    const int n_kv = (N + KEYS - 1) / KEYS;
    const CutPlan cut = cut_plan(n_items, n_kv, att_grid, true);
    if (cut.parts < 2) return;
    const size_t slot = split_slot_floats(DP);
    for (int ti = blockIdx.x; ti < cut.n_tail; ti += gridDim.x) {
        const int w = cut.n_rounds * att_grid + ti;
        const QTile t = tiles[w % n_tiles];
        const int head = w / n_tiles;
        // blockIdx.y picks the work items: one per thread, so that a thread's two rounds of loads are all there is
        for (int idx = blockIdx.y * COMBINE_THREADS + threadIdx.x; idx < t.rows * CG; idx += gridDim.y * COMBINE_THREADS) {
            const int r = idx / CG, cg = idx - r * CG;
            const float* base = ws + (size_t)ti * cut.parts * slot + (size_t)r * (DP + 4);
            float m = -INFINITY;
            for (int p = 0; p < cut.parts; ++p) m = fmaxf(m, base[p * slot + DP]);
            float l = 0.f;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int p = 0; p < cut.parts; ++p) {
                const float* row = base + p * slot;
                const float c = ex2((row[DP] - m) * scale_log2);
                const float4 x = *reinterpret_cast<const float4*>(row + cg * 4);
                l = fmaf(c, row[DP + 1], l);
                acc.x = fmaf(c, x.x, acc.x); acc.y = fmaf(c, x.y, acc.y);
                acc.z = fmaf(c, x.z, acc.z); acc.w = fmaf(c, x.w, acc.w);
            }
            const float inv = 1.0f / l;
            uint2 u;
            u.x = pack_bf16(acc.x * inv, acc.y * inv);
            u.y = pack_bf16(acc.z * inv, acc.w * inv);
            *reinterpret_cast<uint2*>(o + (size_t)(t.row0 + r) * o_ld + head * D + cg * 4) = u;
        }
    }
}

struct AttnPlan {
    CUtensorMap q_map, q_tail_map;
    int heads, dh, dp, H, q_ld;
    void* o;
    float* split_ws;        // one slot per CTA for the pieces of cut items (nullptr: items are never cut)
    int split_slots;
    int split_mode;
    int pair_clusters;      // CTA pairs the pair kernel may run with (0: the pair kernel is not used)
};

}  // namespace

bool tc_attention_supported(const fd_config& c) {
    return c.dtype == FD_BF16 && (c.head_dim == 64 || c.head_dim == 128 || c.head_dim == 72);
}
int tc_attention_tile_rows() { return QROWS; }
int tc_attention_head_pad(int head_dim) { return head_dim == 72 ? 80 : head_dim; }
size_t tc_attention_scratch_bytes(int head_dim) {
    return (size_t)TC_ATTENTION_SLOTS * split_slot_floats(tc_attention_head_pad(head_dim)) * sizeof(float);
}

void* tc_attention_plan_create(const fd_config& cfg, const TcBuffers& buf, std::string* err) {
    AttnPlan* a = new AttnPlan();
    a->heads = cfg.n_heads;
    a->dh = cfg.head_dim;
    a->dp = tc_attention_head_pad(cfg.head_dim);
    a->H = cfg.hidden;
    a->q_ld = buf.q_ld;
    a->o = buf.o;
    a->split_ws = static_cast<float*>(buf.attn_ws);
    a->split_slots = buf.attn_slots;
    a->split_mode = 1;
    if (const char* v = getenv("FD_ATT_SPLIT")) a->split_mode = atoi(v);
    a->pair_clusters = 0;
    const uint64_t dims[2] = {(uint64_t)buf.q_ld, (uint64_t)buf.Mcap};
    const uint64_t strides[1] = {(uint64_t)buf.q_ld * 2};
    const uint32_t box[2] = {64, QROWS};
    bool ok = encode_tmap_bf16(&a->q_map, buf.q, 2, dims, strides, box, 128, err);
    const uint32_t box_tail[2] = {16, QROWS};
    if (ok) ok = encode_tmap_bf16(&a->q_tail_map, buf.q, 2, dims, strides, box_tail, 32, err);
    cudaError_t e = cudaSuccess;
    if (ok) e = cudaFuncSetAttribute(tc_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<64>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<64, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<64>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<72, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<72>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<128, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<128>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<64>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<128>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<72, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<72>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<128>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<72>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<72>::SMEM);
    if (e != cudaSuccess) {
        ok = false;
        if (err) *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
    }
    // head dim 128 can run on CTA pairs (switch FD_ATT_PAIR=1, read here).  Off by default: measured on the 480p video
    // shape the pair kernel takes 4.4 ms per launch against 3.05 ms for the single-CTA kernel (the reasons, with the
    // timestamps that show them, are in the pair kernel's file header).
    bool use_pair = false;
    if (const char* v = getenv("FD_ATT_PAIR")) use_pair = tc_attention_pair_supported(cfg) && atoi(v) != 0;
    if (ok && use_pair) {
        int sms = 0, dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (const char* lim = getenv("FD_TC_MAX_CTAS")) {
            const int v = atoi(lim);
            if (v > 0 && v < sms) sms = v;
        }
        e = sms >= 2 ? tc_attention_pair_setup(&a->pair_clusters, sms) : cudaSuccess;
        if (e != cudaSuccess) {
            ok = false;
            if (err) *err = std::string("pair attention set-up: ") + cudaGetErrorString(e);
        }
    }
    if (!ok) { delete a; return nullptr; }
    return a;
}

void tc_attention_plan_destroy(void* p) { delete static_cast<AttnPlan*>(p); }


cudaError_t tc_attention(TcPlan* p, int /*blk*/, void* kv_block, int B, int N, const QTile* tiles, int max_tiles,
                         const Control* ctl, cudaStream_t st, int* n_launch, const int32_t* labels,
                         const int32_t* active_idx, double* region_mass, int R, const QTile* tiles2) {
    AttnPlan* a = static_cast<AttnPlan*>(tc_plan_attn(p));
    if (!a) return cudaErrorNotSupported;
    CUtensorMap kv_map, kv_tail_map;
    const uint64_t dims[3] = {(uint64_t)a->H, (uint64_t)N, (uint64_t)B * 2};
    const uint64_t strides[2] = {(uint64_t)a->H * 2, (uint64_t)N * a->H * 2};
    const uint32_t box[3] = {64, KEYS, 1};
    const uint32_t box_tail[3] = {16, KEYS, 1};
    std::string err;
    if (!encode_tmap_bf16(&kv_map, kv_block, 3, dims, strides, box, 128, &err)) return cudaErrorInvalidValue;
    if (!encode_tmap_bf16(&kv_tail_map, kv_block, 3, dims, strides, box_tail, 32, &err)) return cudaErrorInvalidValue;
    const int grid = max(1, min(tc_plan_sm_count(p), max_tiles * a->heads));
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)a->dh);
    Control* c = const_cast<Control*>(ctl);
    __nv_bfloat16* o = static_cast<__nv_bfloat16*>(a->o);
    MassArgs ma{labels, active_idx, region_mass, R, 1.0f / (float)a->heads};
    cudaError_t e = cudaSuccess;
    // the items of the last, partly filled round are cut into pieces
    // (switch FD_ATT_SPLIT, read when the context is created: 0 = never, 2 = at every length, for tests)
    const int split_mode = a->split_mode;
    const bool split_on = split_mode != 0;
    // ... for long key sequences only: a piece pays an item's fixed costs (Q load, pipeline fill, hand-over) and the pieces
    // need a second, small kernel; measured, that is a loss at 1024 and 2048 keys and a gain of 3-8 % from 4096 on
    const bool long_keys = N >= 24 * KEYS || split_mode == 2;
    // (not in the launch that also collects the first block's attention mass)
    float* split_ws = (split_on && long_keys && !region_mass && a->split_ws && grid <= a->split_slots) ? a->split_ws : nullptr;
    const bool pdl = tc_plan_pdl(p);
    if (a->pair_clusters > 0 && tiles2 && !region_mass) {
        // head dim 128: 256-row items on CTA pairs; each CTA stages half of every key tile and half of V's head dims
        const int max_tiles2 = B * ((N + 2 * QROWS - 1) / (2 * QROWS));
        return tc_attention_pair_launch(a->q_map, kv_block, B, a->H, a->o, a->H, tiles2, max_tiles2, a->heads, N, scale_log2,
                                        a->split_ws, a->split_slots, a->pair_clusters, split_on && long_keys, c, st, pdl, n_launch);
    }
    const int cgrid = max(1, grid / 2);             // at most grid / 2 items can be cut
#define FD_ATT(DD, MM, CC)                                                                                          \
    do {                                                                                                            \
        e = launch_kernel(tc_attention_kernel<DD, MM, CC>, grid, ATT_THREADS, AttCfg<DD>::SMEM, st, pdl, a->q_map, kv_map, \
                          a->q_tail_map, kv_tail_map, o, a->H, tiles, a->heads, N, scale_log2, split_ws, c, ma);    \
        ++*n_launch;                                                                                                \
        if (e == cudaSuccess && (CC)) {                                                                             \
            e = launch_kernel(attn_combine_kernel<DD>, dim3(cgrid, (QROWS * (DD / 4) + COMBINE_THREADS - 1) / COMBINE_THREADS), \
                              COMBINE_THREADS, 0, st, pdl, (const float*)split_ws, o, a->H, tiles, a->heads, N, grid, \
                              scale_log2, ctl);                                                                     \
            ++*n_launch;                                                                                            \
        }                                                                                                           \
    } while (0)
    if (region_mass) {
        if (a->dh == 64) FD_ATT(64, true, false);
        else if (a->dh == 128) FD_ATT(128, true, false);
        else FD_ATT(72, true, false);
    } else if (split_ws) {
        if (a->dh == 64) FD_ATT(64, false, true);
        else if (a->dh == 128) FD_ATT(128, false, true);
        else FD_ATT(72, false, true);
    } else if (a->dh == 64) FD_ATT(64, false, false);
    else if (a->dh == 128) FD_ATT(128, false, false);
    else FD_ATT(72, false, false);
#undef FD_ATT
    return e;
}

}  // namespace fd
