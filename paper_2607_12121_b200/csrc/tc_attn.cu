// Tensor-core attention of the active queries against all N keys of their request (fresh K/V rows
// of active tokens, previous-step rows of skipped tokens; paper Sec. 5 and Appendix A.6).
//
// One work item = one query tile (up to 128 compact rows of one request) x one head.  Persistent,
// warp-specialised CTAs walk the device-built work list:
//   warp 0      TMA producer: Q tile once per item, K and V tiles (128 keys) through two rings
//   warp 1      issues tcgen05.mma: S = Q K^T into one of two TMEM score buffers, O_h += P V with P
//               read from TMEM and V as an N-major shared-memory operand
//   warps 2..5 and 6..9   two softmax groups, one thread per query row each.  Group h owns score
//               buffer h, i.e. every second key tile, with its own running maximum, row sum and
//               output accumulator O_h, so the two groups run out of phase and never wait for each
//               other inside the key loop: tcgen05.ld of the scores, lazy rescaling of O_h (only
//               when the maximum grew by more than 2^8), exp2, P written over the consumed scores
//               as packed bf16.  At the end the two partial results are merged,
//               O = (a0 O_0 + a1 O_1) / (a0 l_0 + a1 l_1) with a_h = 2^(m_h - m), and stored as bf16
// Keys past N in the last tile are zero-filled by TMA and masked to -inf before the softmax.
#include <cuda_bf16.h>

#include "ptx.cuh"
#include "tc.cuh"

namespace fd {

using namespace ptx;

void* tc_plan_attn(TcPlan* p);
int tc_plan_sm_count(TcPlan* p);

namespace {

constexpr int ATT_THREADS = 320;
constexpr int QROWS = 128, KEYS = 128;
constexpr int SUB_BYTES = 128 * 64 * 2;          // one [128 x 64] bf16 sub-tile, 128-byte rows

template <int D> struct AttCfg {
    static constexpr int SUBS = D / 64;
    static constexpr int TILE_BYTES = SUBS * SUB_BYTES;
    // deep K/V rings: a tile is requested several tile periods before the MMA needs it, which is what
    // hides the L2 / HBM latency of the TMA loads
    static constexpr int STAGES = D == 64 ? 6 : 3;
    static constexpr int SMEM = TILE_BYTES * (1 + 2 * STAGES) + 2560;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}

// TMEM columns: two score buffers (P_h overwrites the first 64 columns of S_h), two output accumulators
constexpr uint32_t COL_S = 0, COL_O = 256, TMEM_COLS = 512;

template <int D>
__global__ void __launch_bounds__(ATT_THREADS, 1)
tc_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kv,
                    __nv_bfloat16* __restrict__ o, int o_ld, const QTile* __restrict__ tiles, int heads, int N,
                    float scale_log2, Control* ctl) {
    using Cfg = AttCfg<D>;
    constexpr int STAGES = Cfg::STAGES;
    constexpr int TILE_BYTES = Cfg::TILE_BYTES;
    extern __shared__ __align__(1024) uint8_t smem[];    // 128-byte swizzled tiles need 1024-byte alignment
    uint8_t* sQ = smem;
    uint8_t* sK = smem + TILE_BYTES;
    uint8_t* sV = sK + STAGES * TILE_BYTES;
    uint64_t* bars = reinterpret_cast<uint64_t*>(sV + STAGES * TILE_BYTES);
    uint64_t* k_full = bars;                  // [STAGES]
    uint64_t* k_empty = k_full + STAGES;
    uint64_t* v_full = k_empty + STAGES;
    uint64_t* v_empty = v_full + STAGES;
    uint64_t* s_full = v_empty + STAGES;      // [2]
    uint64_t* p_full = s_full + 2;            // [2]
    uint64_t* pv_done = p_full + 2;           // [2]
    uint64_t* q_full = pv_done + 2;
    uint64_t* q_empty = q_full + 1;
    uint64_t* o_free = q_empty + 1;
    uint64_t* l_bar = o_free + 1;             // [4 quadrants]: the two threads of a row swap (m, l) once per item
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(l_bar + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* s_xm = reinterpret_cast<float*>(tmem_slot + 2);        // [2 groups][128 rows] running maximum
    float* s_xl = s_xm + 256;                                     // [2 groups][128 rows] row sum

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (smem_u32(smem) & 1023u) {                        // never expected; refuse rather than compute garbage
        if (threadIdx.x == 0) report(ctl, FD_ERR_STATE, -1024);
        return;
    }
    const int n_items = ctl->n_qtiles * heads;
    const int n_kv = (N + KEYS - 1) / KEYS;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(&k_full[s], 1); mbar_init(&k_empty[s], 1);
            mbar_init(&v_full[s], 1); mbar_init(&v_empty[s], 1);
        }
        for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); mbar_init(&pv_done[i], 1); }
        for (int i = 0; i < 4; ++i) mbar_init(&l_bar[i], 64);
        mbar_init(q_full, 1);
        mbar_init(q_empty, 1);
        mbar_init(o_free, 8);
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

    if (warp == 0) {
        if (lane == 0) {
            uint32_t gk = 0;
            bool ok = true;
            int item_i = 0;
            for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x, ++item_i) {
                const QTile t = tiles[w / heads];
                const int head = w % heads;
                if (item_i > 0 && !mbar_wait(q_empty, (item_i - 1) & 1, abort_flag)) { ok = false; break; }
                mbar_expect_tx(q_full, TILE_BYTES);
#pragma unroll
                for (int sb = 0; sb < Cfg::SUBS; ++sb)
                    tma_load_2d(sQ + sb * SUB_BYTES, &tm_q, head * D + sb * 64, t.row0, q_full);
                for (int j = 0; j < n_kv; ++j, ++gk) {
                    const int s = gk % STAGES;
                    const uint32_t ph = ((gk / STAGES) & 1) ^ 1;
                    if (!mbar_wait(&k_empty[s], ph, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&k_full[s], TILE_BYTES);
#pragma unroll
                    for (int sb = 0; sb < Cfg::SUBS; ++sb)
                        tma_load_3d(sK + s * TILE_BYTES + sb * SUB_BYTES, &tm_kv, head * D + sb * 64, j * KEYS,
                                    t.b * 2 + 0, &k_full[s]);
                    if (!mbar_wait(&v_empty[s], ph, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&v_full[s], TILE_BYTES);
#pragma unroll
                    for (int sb = 0; sb < Cfg::SUBS; ++sb)
                        tma_load_3d(sV + s * TILE_BYTES + sb * SUB_BYTES, &tm_kv, head * D + sb * 64, j * KEYS,
                                    t.b * 2 + 1, &v_full[s]);
                }
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 400 + (int)blockIdx.x);
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_qk = idesc_bf16(QROWS, KEYS, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(QROWS, D, 0, 1);      // V: head dim contiguous (N-major)
            uint32_t g0 = 0;          // score/P buffer counter at the start of the item
            bool ok = true;
            int item_i = 0;

            auto issue_qk = [&](uint32_t g, bool last) -> bool {
                const int s = g % STAGES;
                if (!mbar_wait(&k_full[s], (g / STAGES) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + COL_S + (g & 1) * 128;
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks) {
                    const uint32_t off = (ks / 4) * SUB_BYTES + (ks % 4) * 32;
                    const uint64_t da = smem_desc(smem_u32(sQ) + off, 16, 1024, SWZ_128B);
                    const uint64_t db = smem_desc(smem_u32(sK + s * TILE_BYTES) + off, 16, 1024, SWZ_128B);
                    mma_bf16_ss(d, da, db, idesc_qk, ks != 0);
                }
                mma_commit(&k_empty[s]);
                mma_commit(&s_full[g & 1]);
                if (last) mma_commit(q_empty);
                return true;
            };
            auto issue_pv = [&](uint32_t g, int j) -> bool {
                const int s = g % STAGES;
                if (!mbar_wait(&p_full[g & 1], (g >> 1) & 1, abort_flag)) return false;
                if (!mbar_wait(&v_full[s], (g / STAGES) & 1, abort_flag)) return false;
                if (j == 0 && item_i > 0 && !mbar_wait(o_free, (item_i - 1) & 1, abort_flag)) return false;
                tc_fence_after();
                const uint32_t d = tmem_base + COL_O + (g & 1) * D;           // this group's accumulator
                const uint32_t a = tmem_base + COL_S + (g & 1) * 128;         // P sits where the scores were
                const uint32_t first = j < 2 ? 0u : 1u;                       // first tile of the group in this item
#pragma unroll
                for (int ks = 0; ks < KEYS / 16; ++ks) {
                    // 16 keys further: 16 rows of 128 bytes; the second 64-wide half of V sits SUB_BYTES away
                    const uint64_t db = smem_desc(smem_u32(sV + s * TILE_BYTES) + ks * 2048, SUB_BYTES, 1024, SWZ_128B);
                    mma_bf16_ts(d, a + ks * 8, db, idesc_pv, first | (uint32_t)(ks != 0));
                }
                mma_commit(&v_empty[s]);
                mma_commit(&pv_done[g & 1]);
                return true;
            };

            for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x, ++item_i) {
                if (!mbar_wait(q_full, item_i & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                ok = issue_qk(g0, n_kv == 1);
                if (ok && n_kv > 1) ok = issue_qk(g0 + 1, n_kv == 2);
                for (int j = 0; j < n_kv && ok; ++j) {
                    ok = issue_pv(g0 + j, j);
                    if (ok && j + 2 < n_kv) ok = issue_qk(g0 + j + 2, j + 3 == n_kv);
                }
                g0 += n_kv;
            }
            if (!ok) report(ctl, FD_ERR_TIMEOUT, 500 + (int)blockIdx.x);
        }
    } else {
        const int quad = warp & 3;
        const int h = (warp - 2) >> 2;                        // softmax group = score buffer = accumulator
        const int r = quad * 32 + lane;                       // query row inside the tile
        const uint32_t lane_addr = tmem_base + ((uint32_t)(quad * 32) << 16);
        const uint32_t s_addr = lane_addr + COL_S + h * 128;
        const uint32_t o_addr = lane_addr + COL_O + h * D;
        uint32_t g0 = 0;
        bool ok = true;
        int item_i = 0;
        const int rem = N - (n_kv - 1) * KEYS;                // valid keys of the last tile
        for (int w = blockIdx.x; w < n_items && ok; w += gridDim.x, ++item_i) {
            const QTile t = tiles[w / heads];
            const int head = w % heads;
            float m = -INFINITY, l = 0.f;
            bool have = false;                                // this group has processed a tile of this item
            uint32_t g_last = 0;
            for (int j = 0; j < n_kv && ok; ++j) {
                const uint32_t g = g0 + j;
                if ((int)(g & 1) != h) continue;
                if (!mbar_wait(&s_full[h], (g >> 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const int n_valid = (j == n_kv - 1) ? rem : KEYS;
                // pass 1: row maximum (four independent chains)
                float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t sr[32];
                    tmem_ld32(s_addr + c * 32, sr);
                    tmem_wait_ld();
                    if (n_valid < KEYS) {
#pragma unroll
                        for (int i = 0; i < 32; ++i) if (c * 32 + i >= n_valid) sr[i] = 0xff800000u;     // -inf
                    }
#pragma unroll
                    for (int i = 0; i < 32; i += 4) {
                        mx0 = fmaxf(mx0, __uint_as_float(sr[i]));
                        mx1 = fmaxf(mx1, __uint_as_float(sr[i + 1]));
                        mx2 = fmaxf(mx2, __uint_as_float(sr[i + 2]));
                        mx3 = fmaxf(mx3, __uint_as_float(sr[i + 3]));
                    }
                }
                const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
                if (!have) {
                    m = mx;
                } else {
                    const bool need = (mx - m) * scale_log2 > 8.0f;
                    if (__any_sync(0xffffffffu, need)) {
                        // this group's earlier P V products must have landed before O_h is rescaled
                        if (!mbar_wait(&pv_done[h], ((g - 2) >> 1) & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        const float f = need ? ex2((m - mx) * scale_log2) : 1.0f;
                        if (need) { l *= f; m = mx; }
#pragma unroll
                        for (int c = 0; c < D / 32; ++c) {
                            uint32_t orr[32];
                            tmem_ld32(o_addr + c * 32, orr);
                            tmem_wait_ld();
#pragma unroll
                            for (int i = 0; i < 32; ++i) orr[i] = __float_as_uint(__uint_as_float(orr[i]) * f);
                            tmem_st32(o_addr + c * 32, orr);
                        }
                        tmem_wait_st();
                    }
                }
                // pass 2: p = 2^(s c - m c), row sum, P (bf16 pairs) over the consumed score columns
                const float mb = m * scale_log2;
                float su0 = 0.f, su1 = 0.f, su2 = 0.f, su3 = 0.f;
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t sr[32];
                    tmem_ld32(s_addr + c * 32, sr);
                    tmem_wait_ld();
                    uint32_t pk[16];
#pragma unroll
                    for (int i = 0; i < 16; i += 2) {
                        float p0 = ex2(fmaf(__uint_as_float(sr[2 * i]), scale_log2, -mb));
                        float p1 = ex2(fmaf(__uint_as_float(sr[2 * i + 1]), scale_log2, -mb));
                        float p2 = ex2(fmaf(__uint_as_float(sr[2 * i + 2]), scale_log2, -mb));
                        float p3 = ex2(fmaf(__uint_as_float(sr[2 * i + 3]), scale_log2, -mb));
                        if (n_valid < KEYS) {
                            const int k0 = c * 32 + 2 * i;
                            p0 = k0 < n_valid ? p0 : 0.f; p1 = k0 + 1 < n_valid ? p1 : 0.f;
                            p2 = k0 + 2 < n_valid ? p2 : 0.f; p3 = k0 + 3 < n_valid ? p3 : 0.f;
                        }
                        su0 += p0; su1 += p1; su2 += p2; su3 += p3;
                        pk[i] = pack_bf16(p0, p1);
                        pk[i + 1] = pack_bf16(p2, p3);
                    }
                    tmem_st16(s_addr + c * 16, pk);          // columns already read in this pass
                }
                l += (su0 + su1) + (su2 + su3);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_full[h]);
                have = true;
                g_last = g;
            }
            if (!ok) break;
            // merge the two groups' partial results and store the row
            s_xm[h * 128 + r] = m;
            s_xl[h * 128 + r] = have ? l : 0.f;
            mbar_arrive(&l_bar[quad]);
            if (!mbar_wait(&l_bar[quad], item_i & 1, abort_flag)) { ok = false; break; }
            const float m_o = s_xm[(h ^ 1) * 128 + r], l_o = s_xl[(h ^ 1) * 128 + r];
            const bool have_o = n_kv > 1 || (int)(g0 & 1) != h;   // the other group saw at least one tile
            const float m_all = have_o ? fmaxf(m, m_o) : m;
            const float a_me = have ? ex2((m - m_all) * scale_log2) : 0.f;
            const float a_ot = have_o ? ex2((m_o - m_all) * scale_log2) : 0.f;
            const float inv = 1.0f / (a_me * (have ? l : 0.f) + a_ot * l_o);
            const float w_0 = (h == 0 ? a_me : a_ot) * inv, w_1 = (h == 0 ? a_ot : a_me) * inv;   // weights of O_0, O_1
            const bool use0 = h == 0 ? have : have_o, use1 = h == 0 ? have_o : have;
            // every product of this item must have landed: the last tile of each group
            const uint32_t ge = g0 + n_kv - 1;
            if (!mbar_wait(&pv_done[ge & 1], (ge >> 1) & 1, abort_flag)) { ok = false; break; }
            if (n_kv > 1 && !mbar_wait(&pv_done[(ge - 1) & 1], ((ge - 1) >> 1) & 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
            constexpr int DH = D / 2;                         // this thread stores columns [h DH, (h+1) DH)
            __nv_bfloat16* dst = o + (size_t)(t.row0 + r) * o_ld + head * D + h * DH;
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
                uint32_t o0[32], o1[32];
                tmem_ld32(lane_addr + COL_O + h * DH + c * 32, o0);
                tmem_ld32(lane_addr + COL_O + D + h * DH + c * 32, o1);
                tmem_wait_ld();
                if (r < t.rows) {
                    float v[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        v[i] = (use0 ? __uint_as_float(o0[i]) * w_0 : 0.f) + (use1 ? __uint_as_float(o1[i]) * w_1 : 0.f);
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint4 u;
                        u.x = pack_bf16(v[8 * q + 0], v[8 * q + 1]);
                        u.y = pack_bf16(v[8 * q + 2], v[8 * q + 3]);
                        u.z = pack_bf16(v[8 * q + 4], v[8 * q + 5]);
                        u.w = pack_bf16(v[8 * q + 6], v[8 * q + 7]);
                        *reinterpret_cast<uint4*>(dst + c * 32 + q * 8) = u;
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_free);
            g0 += n_kv;
        }
        if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 600 + (int)blockIdx.x);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, TMEM_COLS);
    }
}

struct AttnPlan {
    CUtensorMap q_map;
    int heads, dh, H, q_ld;
    void* o;
};

}  // namespace

bool tc_attention_supported(const fd_config& c) {
    return c.dtype == FD_BF16 && (c.head_dim == 64 || c.head_dim == 128);
}
int tc_attention_tile_rows() { return QROWS; }

void* tc_attention_plan_create(const fd_config& cfg, const TcBuffers& buf, std::string* err) {
    AttnPlan* a = new AttnPlan();
    a->heads = cfg.n_heads;
    a->dh = cfg.head_dim;
    a->H = cfg.hidden;
    a->q_ld = buf.q_ld;
    a->o = buf.o;
    const uint64_t dims[2] = {(uint64_t)buf.q_ld, (uint64_t)buf.Mcap};
    const uint64_t strides[1] = {(uint64_t)buf.q_ld * 2};
    const uint32_t box[2] = {64, QROWS};
    bool ok = encode_tmap_bf16(&a->q_map, buf.q, 2, dims, strides, box, 128, err);
    cudaError_t e = cudaSuccess;
    if (ok) e = cudaFuncSetAttribute(tc_attention_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<64>::SMEM);
    if (ok && e == cudaSuccess)
        e = cudaFuncSetAttribute(tc_attention_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, AttCfg<128>::SMEM);
    if (e != cudaSuccess) {
        ok = false;
        if (err) *err = std::string("cudaFuncSetAttribute: ") + cudaGetErrorString(e);
    }
    if (!ok) { delete a; return nullptr; }
    return a;
}

void tc_attention_plan_destroy(void* p) { delete static_cast<AttnPlan*>(p); }

cudaError_t tc_attention(TcPlan* p, int /*blk*/, void* kv_block, int B, int N, const QTile* tiles, int max_tiles,
                         const Control* ctl, cudaStream_t st, int* n_launch) {
    AttnPlan* a = static_cast<AttnPlan*>(tc_plan_attn(p));
    if (!a) return cudaErrorNotSupported;
    CUtensorMap kv_map;
    const uint64_t dims[3] = {(uint64_t)a->H, (uint64_t)N, (uint64_t)B * 2};
    const uint64_t strides[2] = {(uint64_t)a->H * 2, (uint64_t)N * a->H * 2};
    const uint32_t box[3] = {64, KEYS, 1};
    std::string err;
    if (!encode_tmap_bf16(&kv_map, kv_block, 3, dims, strides, box, 128, &err)) return cudaErrorInvalidValue;
    const int grid = max(1, min(tc_plan_sm_count(p), max_tiles * a->heads));
    const float scale_log2 = 1.4426950408889634f / sqrtf((float)a->dh);
    Control* c = const_cast<Control*>(ctl);
    __nv_bfloat16* o = static_cast<__nv_bfloat16*>(a->o);
    if (a->dh == 64)
        tc_attention_kernel<64><<<grid, ATT_THREADS, AttCfg<64>::SMEM, st>>>(a->q_map, kv_map, o, a->H, tiles, a->heads, N,
                                                                           scale_log2, c);
    else
        tc_attention_kernel<128><<<grid, ATT_THREADS, AttCfg<128>::SMEM, st>>>(a->q_map, kv_map, o, a->H, tiles, a->heads,
                                                                             N, scale_log2, c);
    ++*n_launch;
    return cudaGetLastError();
}

}  // namespace fd
