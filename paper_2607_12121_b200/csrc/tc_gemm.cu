// Tensor-core GEMM for the dense contractions of the block on compacted tokens:
//   C[row, n] = sum_k A[row, k] W[n, k]      A: compact activations [rows, K], W: weights [n_out, K]
// both bf16 with K contiguous.  Persistent, warp-specialised kernel:
//   warp 0      TMA producer: 128 x 64 activation tile and BN x 64 weight tile per stage, 128-byte swizzle
//   warp 1      issues tcgen05.mma (M = 128, N = BN, K = 16) into a TMEM accumulator, two accumulator
//               stages so the next tile's MMAs overlap this tile's epilogue
//   warps 2..5  epilogue: tcgen05.ld of the fp32 accumulator (one row per thread), bias / GELU /
//               gated residual / K-V scatter, 128-bit global stores
// The number of active rows lives on the device; CTAs derive the tile count from it, so the host
// never synchronises.  Rows of the last tile beyond the active count are computed and dropped.
#include <cstdlib>

#include "epilogue.cuh"
#include "ptx.cuh"
#include "tc.cuh"

namespace fd {

using namespace ptx;

namespace {

constexpr int BM = 128, BK = 64;
constexpr int GEMM_THREADS = 320;        // TMA warp, MMA warp, 8 epilogue warps (two per TMEM lane quadrant)
constexpr int A_TILE_BYTES = BM * BK * 2;

constexpr int EPI_WARPS = 8;
constexpr int EPI_STAGE_BYTES = EPI_WARPS * EPI_STAGE_BYTES_PER_WARP;     // transposition tiles of the epilogue warps

template <int BN> struct GemmCfg {
    static constexpr int STAGES = BN == 256 ? 3 : 5;
    static constexpr int B_TILE_BYTES = BN * BK * 2;
    static constexpr int SMEM = STAGES * (A_TILE_BYTES + B_TILE_BYTES) + 1024 /*alignment slack*/ + 256 /*barriers*/ +
                                EPI_STAGE_BYTES;
};

template <int KIND, int BN>
__global__ void __launch_bounds__(GEMM_THREADS, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b, int n_out,
               int k_dim, EpiParams ep, Control* ctl, const int32_t* __restrict__ m_list) {
    using Cfg = GemmCfg<BN>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int B_TILE_BYTES = Cfg::B_TILE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + STAGES * A_TILE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + STAGES * (A_TILE_BYTES + B_TILE_BYTES));
    uint64_t* empty = full + STAGES;
    uint64_t* tfull = empty + STAGES;
    uint64_t* tempty = tfull + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* epi_stage = smem + STAGES * (A_TILE_BYTES + B_TILE_BYTES) + 256;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 8); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tm_a);
        prefetch_tmap(&tm_b);
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 2 * BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above is local set-up; from here on the kernel reads what earlier kernels wrote
    pdl_trigger();
    pdl_wait();
    const int a_total = ctl->a_total;
    // row tiles: all of them, or (dual stream, second pass) the listed ones that hold rows of the second stream
    const int m_tiles = m_list ? ctl->n_text_tiles[0] : (a_total + BM - 1) / BM;
    const int n_tiles = n_out / BN;
    const int total_tiles = m_tiles * n_tiles;
    const int k_tiles = k_dim / BK;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
                const int m = m_list ? m_list[tile / n_tiles] : tile / n_tiles, n = tile % n_tiles;
                for (int kt = 0; kt < k_tiles; ++kt, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&full[s], A_TILE_BYTES + B_TILE_BYTES);
                    tma_load_2d(sA + s * A_TILE_BYTES, &tm_a, kt * BK, m * BM, &full[s]);
                    tma_load_2d(sB + s * B_TILE_BYTES, &tm_b, kt * BK, n * BN, &full[s]);
                }
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 100 + (int)blockIdx.x);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, 0, 0);
            uint32_t it = 0, t_it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++t_it) {
                const uint32_t acc = t_it & 1, aph = (t_it >> 1) & 1;
                if (!mbar_wait(&tempty[acc], aph ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + acc * BN;
                for (int kt = 0; kt < k_tiles; ++kt, ++it) {
                    const int s = it % STAGES;
                    const uint32_t ph = (it / STAGES) & 1;
                    if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = smem_desc(smem_u32(sA + s * A_TILE_BYTES), 16, 1024, SWZ_128B);
                    const uint64_t db = smem_desc(smem_u32(sB + s * B_TILE_BYTES), 16, 1024, SWZ_128B);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)      // 32 bytes further along K inside the swizzle atom
                        mma_bf16_ss(d, da + 2 * k, db + 2 * k, idesc, (kt | k) != 0);
                    mma_commit(&empty[s]);                  // frees the stage when these MMAs are done
                }
                if (ok) mma_commit(&tfull[acc]);            // accumulator ready for the epilogue
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 200 + (int)blockIdx.x);
        }
    } else {
        const int quad = warp & 3;                          // TMEM lane quadrant this warp may read
        const int chalf = (warp - 2) >> 2;                  // which half of the tile's columns
        uint32_t t_it = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++t_it) {
            const int m = m_list ? m_list[tile / n_tiles] : tile / n_tiles, n = tile % n_tiles;
            const uint32_t acc = t_it & 1, aph = (t_it >> 1) & 1;
            if (KIND == EPI_RESID && ep.y)
                epilogue_prefetch_resid(ep, lane, m * BM + quad * 32, a_total, n * BN + chalf * (BN / 2), BN / 2);
            // the rows' request / cache-row data while the tile's products are still running
            const RowInfo ri = epilogue_row_info<KIND>(ep, lane, m * BM + quad * 32, a_total);
            if (!mbar_wait(&tfull[acc], aph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * BN;
            epilogue_warp<KIND>(ep, epi_stage + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane, m * BM + quad * 32, a_total,
                                t_row, n * BN, chalf * (BN / 2), (chalf + 1) * (BN / 2), ri);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty[acc]);
        }
        if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 300 + (int)blockIdx.x);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 2 * BN);
    }
}

// ------------------------------------------------------------------------------------------------
// CTA-pair variant: a cluster of two CTAs computes a 256 x 256 tile with tcgen05.mma.cta_group::2.
// Each CTA stages its own 128 activation rows and one half (128 rows) of the weight tile, so the
// shared-memory traffic per MMA drops by a third and the weight half is fetched once per pair.
// The MMA is issued by one thread of the pair's first CTA; completion is broadcast to both CTAs'
// barriers with a multicast commit.  No TMA load is multicast: every CTA fetches its own tiles.
// ------------------------------------------------------------------------------------------------
// The tile is 256 rows x PAIR_BN columns with PAIR_BN = 256, or 192 for output widths that are a multiple of
// 192 but not of 256 (1152, 3456): those would otherwise fall back to 128 x 128 single-CTA tiles, which the
// operand fetch limits to a quarter of the tensor pipe.
constexpr int PAIR_STAGES = 5;
template <int PAIR_BN> struct PairCfg {
    static constexpr int B_BYTES = (PAIR_BN / 2) * BK * 2;          // this CTA's half of the weight tile
    static constexpr int STAGE_BYTES = A_TILE_BYTES + B_BYTES;
    static constexpr int SMEM = PAIR_STAGES * STAGE_BYTES + 1024 + 256 + EPI_STAGE_BYTES;
    static constexpr int TMEM_COLS = 512;                            // two accumulators of PAIR_BN columns
};

// F8: both operands are E4M3 bytes; a stage holds the same bytes and thus twice the depth of K (128 values), the
// products are kind::f8f6f4 and the epilogue scales the accumulator (see EpiParams).
// GROUPED (dual stream in one launch): the tile sequence is every row tile with the first stream's weights (tm_b),
// followed by the listed row tiles -- those that hold rows of the second stream -- with the second stream's weights
// (tm_b2); a tile's epilogue finishes only the rows of its own stream.
template <int KIND, int PAIR_BN, bool F8 = false, bool GROUPED = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(GEMM_THREADS, 1)
tc_gemm_pair_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_b,
                    const __grid_constant__ CUtensorMap tm_r, int n_out, int k_dim, int stream_a, int tma_resid, EpiParams ep,
                    Control* ctl, const int32_t* __restrict__ m_list, const __grid_constant__ CUtensorMap tm_b2) {
    constexpr int PAIR_B_BYTES = PairCfg<PAIR_BN>::B_BYTES, PAIR_STAGE_BYTES = PairCfg<PAIR_BN>::STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* sA = smem;
    uint8_t* sB = smem + PAIR_STAGES * A_TILE_BYTES;
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + PAIR_STAGES * PAIR_STAGE_BYTES);   // used in the first CTA
    uint64_t* empty = full + PAIR_STAGES;                                                 // one set per CTA
    uint64_t* tfull = empty + PAIR_STAGES;                                                // one set per CTA
    uint64_t* tempty = tfull + 2;                                                         // used in the first CTA
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tempty + 2);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    uint8_t* epi_stage = smem + PAIR_STAGES * PAIR_STAGE_BYTES + 256;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();
    const int cluster_id = blockIdx.x >> 1, n_clusters = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < PAIR_STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 16); }
        *abort_flag = 0;
        fence_barrier_init();
        prefetch_tmap(&tm_a);
        prefetch_tmap(&tm_b);
        if (GROUPED) prefetch_tmap(&tm_b2);
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, PairCfg<PAIR_BN>::TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // both CTAs' barriers exist before anything remote arrives
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // everything above is local set-up; from here on the kernel reads what earlier kernels wrote
    pdl_trigger();
    pdl_wait();
    const int a_total = ctl->a_total;
    // 256-row tiles: all of them, or (dual stream, second pass) the listed ones that hold rows of the second stream
    const int m_all = (a_total + 2 * BM - 1) / (2 * BM);
    const int m_pairs = GROUPED ? m_all : (m_list ? ctl->n_text_tiles[1] : m_all);
    const int n_tiles = n_out / PAIR_BN;
    const int tiles0 = m_pairs * n_tiles;                                  // GROUPED: the first stream's tiles come first
    const int total_tiles = tiles0 + (GROUPED ? ctl->n_text_tiles[1] * n_tiles : 0);
    // row tile, column tile and stream of the tile at position `tile` of the sequence
    auto locate = [&](int tile, int& m, int& n, int& grp) {
        if (GROUPED && tile >= tiles0) {
            const int t2 = tile - tiles0;
            m = m_list[t2 / n_tiles]; n = t2 % n_tiles; grp = 1;
        } else {
            m = (!GROUPED && m_list) ? m_list[tile / n_tiles] : tile / n_tiles; n = tile % n_tiles; grp = 0;
        }
    };
    constexpr int BKE = F8 ? 2 * BK : BK;               // values of K per stage (128 bytes per row either way)
    const int k_tiles = k_dim / BKE;

    if (warp == 0) {
        if (lane == 0) {
            uint32_t it = 0;
            bool ok = true;
            const uint64_t evict_first = l2_evict_first();
            for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters) {
                int m, n, grp;
                locate(tile, m, n, grp);
                const CUtensorMap* wmap = (GROUPED && grp) ? &tm_b2 : &tm_b;
                for (int kt = 0; kt < k_tiles; ++kt, ++it) {
                    const int s = it % PAIR_STAGES;
                    const uint32_t ph = (it / PAIR_STAGES) & 1;
                    if (!mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
                    const uint32_t bar = map_to_cta(smem_u32(&full[s]), 0);     // the first CTA's barrier counts both halves
                    if (rank == 0) mbar_expect_tx(&full[s], 2 * PAIR_STAGE_BYTES);
                    if (stream_a)
                        tma_load_2d_pair_hint(sA + s * A_TILE_BYTES, &tm_a, kt * BKE, m * 2 * BM + (int)rank * BM, bar, evict_first);
                    else
                        tma_load_2d_pair(sA + s * A_TILE_BYTES, &tm_a, kt * BKE, m * 2 * BM + (int)rank * BM, bar);
                    tma_load_2d_pair(sB + s * PAIR_B_BYTES, wmap, kt * BKE, n * PAIR_BN + (int)rank * (PAIR_BN / 2), bar);
                }
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 700 + (int)blockIdx.x);
        }
    } else if (warp == 1) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = F8 ? idesc_e4m3(2 * BM, PAIR_BN) : idesc_bf16(2 * BM, PAIR_BN, 0, 0);
            uint32_t it = 0, t_it = 0;
            bool ok = true;
            for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters, ++t_it) {
                const uint32_t acc = t_it & 1, aph = (t_it >> 1) & 1;
                if (!mbar_wait(&tempty[acc], aph ^ 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d = tmem_base + acc * PAIR_BN;
                for (int kt = 0; kt < k_tiles; ++kt, ++it) {
                    const int s = it % PAIR_STAGES;
                    const uint32_t ph = (it / PAIR_STAGES) & 1;
                    if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint64_t da = smem_desc(smem_u32(sA + s * A_TILE_BYTES), 16, 1024, SWZ_128B);
                    const uint64_t db = smem_desc(smem_u32(sB + s * PAIR_B_BYTES), 16, 1024, SWZ_128B);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k) {       // 32 bytes of K per product, either operand type
                        if constexpr (F8) mma_f8_ss_pair(d, da + 2 * k, db + 2 * k, idesc, (kt | k) != 0);
                        else mma_bf16_ss_pair(d, da + 2 * k, db + 2 * k, idesc, (kt | k) != 0);
                    }
                    mma_commit_pair(&empty[s], 0x3);          // frees the stage in both CTAs
                }
                if (ok) mma_commit_pair(&tfull[acc], 0x3);    // both CTAs' epilogues may read their rows
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 800 + (int)blockIdx.x);
        }
    } else {
        const int quad = warp & 3;
        const int chalf = (warp - 2) >> 2;                  // which part of the tile's columns
        // column ranges of the two warps of a lane quadrant: halves, in whole chunks of the epilogue (32 columns
        // for the fp32 residual update, 64 for the bf16 outputs)
        constexpr int CH = KIND == EPI_RESID ? 32 : 64;
        constexpr int C_SPLIT = ((PAIR_BN / 2 + CH - 1) / CH) * CH;
        const int c_lo = chalf == 0 ? 0 : C_SPLIT, c_hi = chalf == 0 ? C_SPLIT : PAIR_BN;
        uint32_t t_it = 0;
        bool ok = true;
        const void* bias0 = ep.bias;
        const void* qn0 = ep.qn_w;
        const void* kn0 = ep.kn_w;
        const float* col_scale0 = ep.col_scale;
        const float act_scale0 = ep.act_scale, out_inv_scale0 = ep.out_inv_scale;
        for (int tile = cluster_id; tile < total_tiles && ok; tile += n_clusters, ++t_it) {
            int m, n, grp;
            locate(tile, m, n, grp);
            if constexpr (GROUPED) {                        // this tile's stream: its rows, bias and scales
                ep.group = grp;
                ep.bias = grp ? ep.bias2 : bias0;
                ep.qn_w = grp ? ep.qn_w2 : qn0;
                ep.kn_w = grp ? ep.kn_w2 : kn0;
                ep.col_scale = grp ? ep.col_scale2 : col_scale0;
                ep.act_scale = grp ? ep.act_scale2 : act_scale0;
                ep.out_inv_scale = grp ? ep.out_inv_scale2 : out_inv_scale0;
            }
            const uint32_t acc = t_it & 1, aph = (t_it >> 1) & 1;
            if (KIND == EPI_RESID && ep.y)
                epilogue_prefetch_resid(ep, lane, m * 2 * BM + (int)rank * BM + quad * 32, a_total,
                                        n * PAIR_BN + c_lo, c_hi - c_lo);
            // the rows' request / cache-row data while the tile's products are still running
            const RowInfo ri = epilogue_row_info<KIND>(ep, lane, m * 2 * BM + (int)rank * BM + quad * 32, a_total);
            if (!mbar_wait(&tfull[acc], aph, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + acc * PAIR_BN;
            epilogue_warp<KIND, F8>(ep, epi_stage + (warp - 2) * EPI_STAGE_BYTES_PER_WARP, lane,
                                m * 2 * BM + (int)rank * BM + quad * 32, a_total, t_row, n * PAIR_BN, c_lo, c_hi, ri,
                                (KIND == EPI_RESID && tma_resid) ? &tm_r : nullptr);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&tempty[acc]), 0));
        }
        if (KIND == EPI_RESID && lane == 0) bulk_wait_all();      // this thread's bulk reductions have landed
        if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 900 + (int)blockIdx.x);
    }

    tc_fence_before();
    __syncthreads();
    cluster_sync_all();                      // neither CTA leaves while its peer may still signal it
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, PairCfg<PAIR_BN>::TMEM_COLS);
    }
}

// Self-test of the bounded wait: one thread waits on an mbarrier that nothing ever arrives on.  The wait
// gives up after its poll limit (about a second), records FD_ERR_TIMEOUT in the control block and the
// kernel returns normally, so the context stays usable.
__global__ void bounded_wait_selftest_kernel(Control* ctl) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        fence_barrier_init();
        if (!mbar_wait(&bar, 0, &abort_flag)) report(ctl, FD_ERR_TIMEOUT, 999);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn(std::string* err) {
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !p) {
        if (err) *err = "cuTensorMapEncodeTiled is not available from the driver";
        return nullptr;
    }
    fn = reinterpret_cast<EncodeTiledFn>(p);
    return fn;
}

int pick_bn(int n_out) { return (n_out % 256 == 0) ? 256 : 128; }
int pick_pair_bn(int n_out) { return n_out % 256 == 0 ? 256 : (n_out % 192 == 0 ? 192 : 0); }

}  // namespace

static bool encode_tmap(CUtensorMap* out, CUtensorMapDataType dtype, void* base, int rank, const uint64_t* dims,
                        const uint64_t* strides_bytes, const uint32_t* box, int swizzle_bytes, std::string* err) {
    EncodeTiledFn fn = encode_fn(err);
    if (!fn) return false;
    cuuint64_t gd[5], gs[5];
    cuuint32_t bx[5], es[5];
    for (int i = 0; i < rank; ++i) { gd[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) gs[i] = strides_bytes[i];
    CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B
                          : swizzle_bytes == 64  ? CU_TENSOR_MAP_SWIZZLE_64B
                          : swizzle_bytes == 32  ? CU_TENSOR_MAP_SWIZZLE_32B
                                                 : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUresult r = fn(out, dtype, (cuuint32_t)rank, base, gd, gs, bx, es,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        if (err) *err = "cuTensorMapEncodeTiled failed with code " + std::to_string((int)r);
        return false;
    }
    return true;
}

bool encode_tmap_bf16(CUtensorMap* out, void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                      const uint32_t* box, int swizzle_bytes, std::string* err) {
    return encode_tmap(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, base, rank, dims, strides_bytes, box, swizzle_bytes, err);
}

struct GemmSpec {
    CUtensorMap a;              // activation operand
    int n_out, k, bn;
    int pair_bn;                // CTA-pair kernel with 256 x pair_bn tiles (0: single-CTA kernel); weight boxes are then pair_bn / 2 rows
};

struct TcPlan {
    fd_config cfg;
    TcBuffers buf;
    int sm_count;
    bool pdl;                   // launch the tensor-core kernels with programmatic stream serialization
    int pair_ctas;              // grid of the CTA-pair kernel: 2 x co-resident clusters
    GemmSpec spec[6];           // indexed by TcGemmKind
    CUtensorMap resid_map;      // fp32 residual stream [Mcap, H], 32 x 32 boxes for the bulk reductions of EPI_RESID
    bool tma_resid;
    CUtensorMap* w_maps;        // [L][4]
    CUtensorMap* w_maps_text;   // [L][4] second stream's weights (dual stream), or nullptr
    CUtensorMap* w_maps_cross;  // [L][2] cross-attention's query and out projections, or nullptr
    CUtensorMap* w_maps_f8;     // [L][3] E4M3 weights of QKV, fc1, fc2 (FP8 operands), or nullptr
    CUtensorMap* w_maps_f8_text;    // [L][3] the second stream's, or nullptr
    CUtensorMap a_maps_f8[2];   // the activation buffer and the MLP hidden buffer read as E4M3 bytes
    const int32_t* text_list128;    // device lists of the row tiles that hold rows of the second stream
    const int32_t* text_list256;
    // attention (filled by the attention part)
    void* attn;
};

bool tc_supported(const fd_config& c, std::string* why) {
    auto bad = [&](const char* m) { if (why) *why = m; return false; };
    if (c.dtype != FD_BF16) return bad("tensor-core engine needs bf16 storage");
    if (c.hidden % 128 || c.mlp_dim % 128) return bad("hidden and mlp_dim must be multiples of 128");
    if (c.cond_dim % 8) return bad("cond_dim must be a multiple of 8");
    return true;
}

void* tc_attention_plan_create(const fd_config& cfg, const TcBuffers& buf, std::string* err);
void tc_attention_plan_destroy(void* p);

TcPlan* tc_plan_create(const fd_config& cfg, const fd_weights& w, const TcBuffers& buf, std::string* err) {
    TcPlan* p = new TcPlan();
    p->cfg = cfg;
    p->buf = buf;
    p->w_maps = new CUtensorMap[(size_t)cfg.n_blocks * 4];
    p->w_maps_text = nullptr;
    p->w_maps_cross = nullptr;
    p->w_maps_f8 = nullptr;
    p->w_maps_f8_text = nullptr;
    p->text_list128 = p->text_list256 = nullptr;
    p->attn = nullptr;
    int dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, dev);
    // test knob: fewer persistent CTAs make every CTA walk many tiles (ring and accumulator wrap-around)
    if (const char* lim = getenv("FD_TC_MAX_CTAS")) {
        const int v = atoi(lim);
        if (v > 0 && v < p->sm_count) p->sm_count = v;
    }
    p->pdl = true;              // switch: FD_PDL=0 launches every kernel fully serialized
    if (const char* v = getenv("FD_PDL")) p->pdl = atoi(v) != 0;
    bool use_pair = true;       // switch: FD_TC_PAIR=0 keeps every GEMM on the single-CTA kernel
    if (const char* v = getenv("FD_TC_PAIR")) use_pair = atoi(v) != 0;
    const int H = cfg.hidden, M = cfg.mlp_dim;
    const int n_out[6] = {3 * H, H, M, H, H, H};
    const int kdim[6] = {H, H, H, M, H, H};
    void* a_base[6] = {buf.act, buf.o, buf.act, buf.g, buf.act, buf.o};
    const char* w_base[4] = {static_cast<const char*>(w.w_qkv), static_cast<const char*>(w.w_o),
                             static_cast<const char*>(w.w_fc1), static_cast<const char*>(w.w_fc2)};
    bool ok = true;
    for (int g = 0; g < 6 && ok; ++g) {
        GemmSpec& s = p->spec[g];
        s.n_out = n_out[g];
        s.k = kdim[g];
        s.bn = pick_bn(n_out[g]);
        s.pair_bn = use_pair ? pick_pair_bn(n_out[g]) : 0;
        const uint64_t dims[2] = {(uint64_t)kdim[g], (uint64_t)buf.Mcap};
        const uint64_t strides[1] = {(uint64_t)kdim[g] * 2};
        const uint32_t box[2] = {BK, BM};
        ok = encode_tmap_bf16(&s.a, a_base[g], 2, dims, strides, box, 128, err);
        for (int l = 0; l < cfg.n_blocks && ok && g < 4; ++l) {
            const uint64_t wd[2] = {(uint64_t)kdim[g], (uint64_t)n_out[g]};
            const uint32_t wb[2] = {BK, s.pair_bn ? (uint32_t)s.pair_bn / 2 : (uint32_t)s.bn};
            void* base = const_cast<char*>(w_base[g]) + (size_t)l * n_out[g] * kdim[g] * 2;
            ok = encode_tmap_bf16(&p->w_maps[(size_t)l * 4 + g], base, 2, wd, strides, wb, 128, err);
        }
    }
    p->tma_resid = true;        // switch: FD_TMA_RESID=0 keeps the per-thread vector reductions
    if (const char* v = getenv("FD_TMA_RESID")) p->tma_resid = atoi(v) != 0;
    if (ok) {
        const uint64_t rd[2] = {(uint64_t)H, (uint64_t)buf.Mcap};
        const uint64_t rs[1] = {(uint64_t)H * 4};
        const uint32_t rb[2] = {32, 32};
        ok = encode_tmap(&p->resid_map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, buf.resid, 2, rd, rs, rb, 0, err);
    }
    if (ok) {
        cudaError_t e = cudaSuccess;
#define FD_SET_SMEM(K, N)                                                                                  \
    if (e == cudaSuccess)                                                                                  \
        e = cudaFuncSetAttribute(tc_gemm_kernel<K, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, GemmCfg<N>::SMEM);
        FD_SET_SMEM(EPI_QKV, 128) FD_SET_SMEM(EPI_QKV, 256) FD_SET_SMEM(EPI_RESID, 128) FD_SET_SMEM(EPI_RESID, 256)
        FD_SET_SMEM(EPI_GELU, 128) FD_SET_SMEM(EPI_GELU, 256)
#undef FD_SET_SMEM
#define FD_SET_PAIR(K, N)                                                                                  \
    if (e == cudaSuccess)                                                                                  \
        e = cudaFuncSetAttribute(tc_gemm_pair_kernel<K, N>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<N>::SMEM);
        FD_SET_PAIR(EPI_QKV, 256) FD_SET_PAIR(EPI_RESID, 256) FD_SET_PAIR(EPI_GELU, 256)
        FD_SET_PAIR(EPI_QKV, 192) FD_SET_PAIR(EPI_RESID, 192) FD_SET_PAIR(EPI_GELU, 192)
#undef FD_SET_PAIR
#define FD_SET_PAIR8(K, N)                                                                                 \
    if (e == cudaSuccess)                                                                                  \
        e = cudaFuncSetAttribute(tc_gemm_pair_kernel<K, N, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<N>::SMEM);
        FD_SET_PAIR8(EPI_QKV, 256) FD_SET_PAIR8(EPI_RESID, 256) FD_SET_PAIR8(EPI_GELU, 256)
        FD_SET_PAIR8(EPI_QKV, 192) FD_SET_PAIR8(EPI_RESID, 192) FD_SET_PAIR8(EPI_GELU, 192)
#undef FD_SET_PAIR8
#define FD_SET_PAIRG(K, N, F)                                                                              \
    if (e == cudaSuccess)                                                                                  \
        e = cudaFuncSetAttribute(tc_gemm_pair_kernel<K, N, F, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PairCfg<N>::SMEM);
        FD_SET_PAIRG(EPI_QKV, 256, false) FD_SET_PAIRG(EPI_RESID, 256, false) FD_SET_PAIRG(EPI_GELU, 256, false)
        FD_SET_PAIRG(EPI_QKV, 192, false) FD_SET_PAIRG(EPI_RESID, 192, false) FD_SET_PAIRG(EPI_GELU, 192, false)
        FD_SET_PAIRG(EPI_QKV, 256, true) FD_SET_PAIRG(EPI_RESID, 256, true) FD_SET_PAIRG(EPI_GELU, 256, true)
        FD_SET_PAIRG(EPI_QKV, 192, true) FD_SET_PAIRG(EPI_RESID, 192, true) FD_SET_PAIRG(EPI_GELU, 192, true)
#undef FD_SET_PAIRG
        if (e != cudaSuccess) {
            ok = false;
            if (err) *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
        }
    }
    p->pair_ctas = p->sm_count & ~1;
    if (ok) {
        // as many CTA pairs as the device can keep resident at once (a pair needs both SMs of a TPC)
        cudaLaunchConfig_t lc = {};
        lc.gridDim = dim3(p->sm_count & ~1);
        lc.blockDim = dim3(GEMM_THREADS);
        lc.dynamicSmemBytes = PairCfg<256>::SMEM;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeClusterDimension;
        at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
        lc.attrs = at;
        lc.numAttrs = 1;
        int n_clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&n_clusters, tc_gemm_pair_kernel<EPI_GELU, 256>, &lc) == cudaSuccess && n_clusters > 0)
            p->pair_ctas = min(p->sm_count & ~1, 2 * n_clusters);
        else
            cudaGetLastError();
        if (p->pair_ctas < 2) p->pair_ctas = 2;
    }
    if (ok && tc_attention_supported(cfg)) {
        p->attn = tc_attention_plan_create(cfg, buf, err);
        ok = p->attn != nullptr;
    }
    if (!ok) {
        tc_plan_destroy(p);
        return nullptr;
    }
    return p;
}

void tc_plan_destroy(TcPlan* p) {
    if (!p) return;
    tc_attention_plan_destroy(p->attn);
    delete[] p->w_maps;
    delete[] p->w_maps_text;
    delete[] p->w_maps_cross;
    delete[] p->w_maps_f8;
    delete[] p->w_maps_f8_text;
    delete p;
}

cudaError_t launch_bounded_wait_selftest(Control* ctl, cudaStream_t st, int* n_launch) {
    bounded_wait_selftest_kernel<<<1, 32, 0, st>>>(ctl);
    ++*n_launch;
    return cudaGetLastError();
}

void* tc_plan_attn(TcPlan* p) { return p->attn; }
bool tc_plan_pdl(TcPlan* p) { return p->pdl; }
int tc_plan_sm_count(TcPlan* p) { return p->sm_count; }

// Dual stream: tensor maps of the second stream's weights (w == nullptr: back to a single stream) and the device lists
// of row tiles its launches walk.
bool tc_plan_set_text(TcPlan* p, const fd_weights* w, const int32_t* list128, const int32_t* list256, std::string* err) {
    delete[] p->w_maps_text;
    p->w_maps_text = nullptr;
    p->text_list128 = list128;
    p->text_list256 = list256;
    if (!w) return true;
    const fd_config& cfg = p->cfg;
    const int H = cfg.hidden, M = cfg.mlp_dim;
    const int n_out[4] = {3 * H, H, M, H};
    const int kdim[4] = {H, H, H, M};
    const char* w_base[4] = {static_cast<const char*>(w->w_qkv), static_cast<const char*>(w->w_o),
                             static_cast<const char*>(w->w_fc1), static_cast<const char*>(w->w_fc2)};
    p->w_maps_text = new CUtensorMap[(size_t)cfg.n_blocks * 4];
    for (int g = 0; g < 4; ++g) {
        const GemmSpec& s = p->spec[g];
        for (int l = 0; l < cfg.n_blocks; ++l) {
            const uint64_t wd[2] = {(uint64_t)kdim[g], (uint64_t)n_out[g]};
            const uint64_t strides[1] = {(uint64_t)kdim[g] * 2};
            const uint32_t wb[2] = {BK, s.pair_bn ? (uint32_t)s.pair_bn / 2 : (uint32_t)s.bn};
            void* base = const_cast<char*>(w_base[g]) + (size_t)l * n_out[g] * kdim[g] * 2;
            if (!encode_tmap_bf16(&p->w_maps_text[(size_t)l * 4 + g], base, 2, wd, strides, wb, 128, err)) {
                delete[] p->w_maps_text;
                p->w_maps_text = nullptr;
                return false;
            }
        }
    }
    return true;
}

bool tc_plan_set_cross(TcPlan* p, const void* w_q, const void* w_o, std::string* err) {
    delete[] p->w_maps_cross;
    p->w_maps_cross = nullptr;
    if (!w_q || !w_o) return true;
    const fd_config& cfg = p->cfg;
    const int H = cfg.hidden;
    const char* w_base[2] = {static_cast<const char*>(w_q), static_cast<const char*>(w_o)};
    p->w_maps_cross = new CUtensorMap[(size_t)cfg.n_blocks * 2];
    for (int g = 0; g < 2; ++g) {
        const GemmSpec& s = p->spec[TC_GEMM_XQ + g];
        for (int l = 0; l < cfg.n_blocks; ++l) {
            const uint64_t wd[2] = {(uint64_t)H, (uint64_t)H};
            const uint64_t strides[1] = {(uint64_t)H * 2};
            const uint32_t wb[2] = {BK, s.pair_bn ? (uint32_t)s.pair_bn / 2 : (uint32_t)s.bn};
            void* base = const_cast<char*>(w_base[g]) + (size_t)l * H * H * 2;
            if (!encode_tmap_bf16(&p->w_maps_cross[(size_t)l * 2 + g], base, 2, wd, strides, wb, 128, err)) {
                delete[] p->w_maps_cross;
                p->w_maps_cross = nullptr;
                return false;
            }
        }
    }
    return true;
}

// FP8 operands: tensor maps of the E4M3 weights (all nullptr: off) and of the two activation buffers read as bytes.
// Needs the CTA-pair kernel for the three projections.
bool tc_plan_set_fp8(TcPlan* p, const void* w8_qkv, const void* w8_fc1, const void* w8_fc2, std::string* err, bool text) {
    CUtensorMap*& maps = text ? p->w_maps_f8_text : p->w_maps_f8;
    delete[] maps;
    maps = nullptr;
    if (!w8_qkv || !w8_fc1 || !w8_fc2) return true;
    const fd_config& cfg = p->cfg;
    const TcGemmKind kinds[3] = {TC_GEMM_QKV, TC_GEMM_FC1, TC_GEMM_FC2};
    const char* w_base[3] = {static_cast<const char*>(w8_qkv), static_cast<const char*>(w8_fc1), static_cast<const char*>(w8_fc2)};
    for (int g = 0; g < 3; ++g)
        if (!p->spec[kinds[g]].pair_bn || p->spec[kinds[g]].k % 128) {
            if (err) *err = "FP8 operands need the CTA-pair kernel (output widths multiples of 192 or 256) and K a multiple of 128";
            return false;
        }
    maps = new CUtensorMap[(size_t)cfg.n_blocks * 3];
    bool ok = true;
    void* a_base[2] = {p->buf.act, p->buf.g};
    const int a_k[2] = {cfg.hidden, cfg.mlp_dim};
    for (int i = 0; i < 2 && ok; ++i) {
        const uint64_t dims[2] = {(uint64_t)a_k[i], (uint64_t)p->buf.Mcap};
        const uint64_t strides[1] = {(uint64_t)a_k[i]};
        const uint32_t box[2] = {128, BM};
        ok = encode_tmap(&p->a_maps_f8[i], CU_TENSOR_MAP_DATA_TYPE_UINT8, a_base[i], 2, dims, strides, box, 128, err);
    }
    for (int g = 0; g < 3 && ok; ++g) {
        const GemmSpec& s = p->spec[kinds[g]];
        for (int l = 0; l < cfg.n_blocks && ok; ++l) {
            const uint64_t wd[2] = {(uint64_t)s.k, (uint64_t)s.n_out};
            const uint64_t strides[1] = {(uint64_t)s.k};
            const uint32_t wb[2] = {128, (uint32_t)s.pair_bn / 2};
            void* base = const_cast<char*>(w_base[g]) + (size_t)l * s.n_out * s.k;
            ok = encode_tmap(&maps[(size_t)l * 3 + g], CU_TENSOR_MAP_DATA_TYPE_UINT8, base, 2, wd, strides, wb, 128, err);
        }
    }
    if (!ok) {
        delete[] maps;
        maps = nullptr;
    }
    return ok;
}

// Dual stream in one launch: every row tile with the first stream's weights, then the row tiles that hold rows of the
// second stream with the second stream's weights (ep.bias2 and, with FP8 operands, ep.col_scale2 / act_scale2 /
// out_inv_scale2 are that stream's).  Available where the CTA-pair kernel runs the projection (switch FD_TC_GROUPED=0
// keeps the two launches).
// The QKV epilogue can apply QK-RMSNorm and the rotary embedding itself when every head is a whole number of its
// 64-column chunks inside one warp's column range: head dim 64 at either tile width, head dim 128 at 256-wide tiles
// (switch FD_QK_FUSED=0 keeps the separate kernel).
bool tc_plan_qk_fusable(TcPlan* p) {
    const char* v = getenv("FD_QK_FUSED");
    if (v && atoi(v) == 0) return false;
    const int bn = p->spec[TC_GEMM_QKV].pair_bn, dh = p->cfg.head_dim;
    return bn != 0 && (dh == 64 || (dh == 128 && bn == 256));
}

bool tc_plan_grouped(TcPlan* p, TcGemmKind kind) {
    const char* v = getenv("FD_TC_GROUPED");
    const bool on = !v || atoi(v) != 0;
    return on && kind <= TC_GEMM_FC2 && p->spec[kind].pair_bn != 0 && p->w_maps_text != nullptr;
}

cudaError_t tc_gemm_both(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                         int* n_launch, bool fp8) {
    if (!tc_plan_grouped(p, kind)) return cudaErrorInvalidValue;
    const GemmSpec& s = p->spec[kind];
    const int g = kind == TC_GEMM_QKV ? 0 : kind == TC_GEMM_FC1 ? 1 : 2;
    if (fp8 && (!p->w_maps_f8 || !p->w_maps_f8_text || kind == TC_GEMM_OUT)) return cudaErrorInvalidValue;
    const CUtensorMap& wm = fp8 ? p->w_maps_f8[(size_t)blk * 3 + g] : p->w_maps[(size_t)blk * 4 + kind];
    const CUtensorMap& wm2 = fp8 ? p->w_maps_f8_text[(size_t)blk * 3 + g] : p->w_maps_text[(size_t)blk * 4 + kind];
    const CUtensorMap& am = fp8 ? p->a_maps_f8[kind == TC_GEMM_FC2 ? 1 : 0] : s.a;
    Control* c = const_cast<Control*>(ctl);
    const int pgrid = max(2, min(p->sm_count & ~1, p->pair_ctas));
    const int stream_a = kind == TC_GEMM_FC2 ? 1 : 0;
    cudaError_t e = cudaSuccess;
#define FD_LAUNCH_BOTH(K, N, F)                                                                                          \
    e = launch_kernel(tc_gemm_pair_kernel<K, N, F, true>, pgrid, GEMM_THREADS, PairCfg<N>::SMEM, st, p->pdl, am, wm, p->resid_map, \
                      s.n_out, s.k, stream_a, p->tma_resid ? 1 : 0, ep, c, p->text_list256, wm2)
#define FD_LAUNCH_BOTH_N(K, F) do { if (s.pair_bn == 256) FD_LAUNCH_BOTH(K, 256, F); else FD_LAUNCH_BOTH(K, 192, F); } while (0)
    if (fp8) {
        if (kind == TC_GEMM_QKV) FD_LAUNCH_BOTH_N(EPI_QKV, true);
        else if (kind == TC_GEMM_FC1) FD_LAUNCH_BOTH_N(EPI_GELU, true);
        else FD_LAUNCH_BOTH_N(EPI_RESID, true);
    } else {
        if (kind == TC_GEMM_QKV) FD_LAUNCH_BOTH_N(EPI_QKV, false);
        else if (kind == TC_GEMM_FC1) FD_LAUNCH_BOTH_N(EPI_GELU, false);
        else FD_LAUNCH_BOTH_N(EPI_RESID, false);
    }
#undef FD_LAUNCH_BOTH_N
#undef FD_LAUNCH_BOTH
    ++*n_launch;
    return e;
}

cudaError_t tc_gemm_fp8(TcPlan* p, TcGemmKind kind, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                        int* n_launch, bool text_pass) {
    const CUtensorMap* maps = text_pass ? p->w_maps_f8_text : p->w_maps_f8;
    if (!maps || (kind != TC_GEMM_QKV && kind != TC_GEMM_FC1 && kind != TC_GEMM_FC2)) return cudaErrorInvalidValue;
    const GemmSpec& s = p->spec[kind];
    const int g = kind == TC_GEMM_QKV ? 0 : kind == TC_GEMM_FC1 ? 1 : 2;
    const CUtensorMap& wm = maps[(size_t)blk * 3 + g];
    const CUtensorMap& am = p->a_maps_f8[kind == TC_GEMM_FC2 ? 1 : 0];
    Control* c = const_cast<Control*>(ctl);
    const int pgrid = max(2, min(p->sm_count & ~1, p->pair_ctas));
    const int stream_a = kind == TC_GEMM_FC2 ? 1 : 0;
    const int32_t* no_list = text_pass ? p->text_list256 : nullptr;   // second stream: the row tiles that hold its rows
    cudaError_t e = cudaSuccess;
#define FD_LAUNCH_PAIR8(K, N) \
    e = launch_kernel(tc_gemm_pair_kernel<K, N, true>, pgrid, GEMM_THREADS, PairCfg<N>::SMEM, st, p->pdl, am, wm, p->resid_map, s.n_out, \
                      s.k, stream_a, p->tma_resid ? 1 : 0, ep, c, no_list, wm)
    if (kind == TC_GEMM_QKV) {
        if (s.pair_bn == 256) FD_LAUNCH_PAIR8(EPI_QKV, 256); else FD_LAUNCH_PAIR8(EPI_QKV, 192);
    } else if (kind == TC_GEMM_FC1) {
        if (s.pair_bn == 256) FD_LAUNCH_PAIR8(EPI_GELU, 256); else FD_LAUNCH_PAIR8(EPI_GELU, 192);
    } else {
        if (s.pair_bn == 256) FD_LAUNCH_PAIR8(EPI_RESID, 256); else FD_LAUNCH_PAIR8(EPI_RESID, 192);
    }
#undef FD_LAUNCH_PAIR8
    ++*n_launch;
    return e;
}

cudaError_t tc_gemm(TcPlan* p, TcGemmKind kind_in, int blk, const EpiParams& ep, const Control* ctl, cudaStream_t st,
                    int* n_launch, bool text_pass) {
    const GemmSpec& s = p->spec[kind_in];
    const bool cross = kind_in >= TC_GEMM_XQ;
    if (text_pass && (!p->w_maps_text || cross)) return cudaErrorInvalidValue;
    if (cross && !p->w_maps_cross) return cudaErrorInvalidValue;
    const CUtensorMap& wm = cross       ? p->w_maps_cross[(size_t)blk * 2 + (kind_in - TC_GEMM_XQ)]
                            : text_pass ? p->w_maps_text[(size_t)blk * 4 + kind_in]
                                        : p->w_maps[(size_t)blk * 4 + kind_in];
    // the cross-attention's projections run the kernels of the projections they resemble
    const TcGemmKind kind = kind_in == TC_GEMM_XQ ? TC_GEMM_QKV : kind_in == TC_GEMM_XO ? TC_GEMM_OUT : kind_in;
    const int32_t* m_list = text_pass ? (s.pair_bn ? p->text_list256 : p->text_list128) : nullptr;
    Control* c = const_cast<Control*>(ctl);
    const int grid = p->sm_count;
    if (s.pair_bn) {
        const int pgrid = max(2, min(grid & ~1, p->pair_ctas));
        // fc2's input (rows x mlp_dim) is the one operand of the step larger than what L2 keeps beside the residual
        // stream; each of its row blocks is read by the block's column tiles together and then not again
        const int stream_a = kind == TC_GEMM_FC2 ? 1 : 0;
        cudaError_t e = cudaSuccess;
#define FD_LAUNCH_PAIR(K, N) \
    e = launch_kernel(tc_gemm_pair_kernel<K, N>, pgrid, GEMM_THREADS, PairCfg<N>::SMEM, st, p->pdl, s.a, wm, p->resid_map, s.n_out, s.k, \
                      stream_a, p->tma_resid ? 1 : 0, ep, c, m_list, wm)
        if (kind == TC_GEMM_QKV) {
            if (s.pair_bn == 256) FD_LAUNCH_PAIR(EPI_QKV, 256); else FD_LAUNCH_PAIR(EPI_QKV, 192);
        } else if (kind == TC_GEMM_FC1) {
            if (s.pair_bn == 256) FD_LAUNCH_PAIR(EPI_GELU, 256); else FD_LAUNCH_PAIR(EPI_GELU, 192);
        } else {
            if (s.pair_bn == 256) FD_LAUNCH_PAIR(EPI_RESID, 256); else FD_LAUNCH_PAIR(EPI_RESID, 192);
        }
#undef FD_LAUNCH_PAIR
        ++*n_launch;
        return e;
    }
    cudaError_t e = cudaSuccess;
#define FD_LAUNCH(K, N) \
    e = launch_kernel(tc_gemm_kernel<K, N>, grid, GEMM_THREADS, GemmCfg<N>::SMEM, st, p->pdl, s.a, wm, s.n_out, s.k, ep, c, m_list)
    if (kind == TC_GEMM_QKV) {
        if (s.bn == 256) FD_LAUNCH(EPI_QKV, 256); else FD_LAUNCH(EPI_QKV, 128);
    } else if (kind == TC_GEMM_FC1) {
        if (s.bn == 256) FD_LAUNCH(EPI_GELU, 256); else FD_LAUNCH(EPI_GELU, 128);
    } else {
        if (s.bn == 256) FD_LAUNCH(EPI_RESID, 256); else FD_LAUNCH(EPI_RESID, 128);
    }
#undef FD_LAUNCH
    ++*n_launch;
    return e;
}

}  // namespace fd
