// Sampler closure around the regional step (Appendix A.1, Eq. sf-update): patch embedding of the latent
// before the block stack, final layer and latent update after it.  An active patch moves along the drift
// read off its fresh block-stack output, a skipped patch along the drift cached at its last active step.
//
// Three small kernels outside the step's hot loop:
//   embed_kernel        x[b,j,:] = z[b,j,:] W_in^T + b_in + pos[j,:]                  (writes B N H elements)
//   final_drift_kernel  drift[tok,:] = LayerNorm(y[tok,:]) W_out^T + b_out, active tokens only
//   euler_kernel        z_next = z + h[b] drift                                      (all tokens)
// The contractions are skinny (D <= 256 on one side), so they run on CUDA cores with shared-memory tiles.
#include "common.cuh"

namespace fd {

namespace {

constexpr int EMB_TOK = 32;        // tokens per CTA
constexpr int EMB_THREADS = 256;   // one output column per thread

template <typename T>
__global__ void __launch_bounds__(EMB_THREADS)
embed_kernel(const float* __restrict__ z, const T* __restrict__ w_in, const T* __restrict__ b_in,
             const T* __restrict__ pos, T* __restrict__ x, long long n_tok, int N, int D, int H) {
    extern __shared__ float s_z[];                       // [EMB_TOK][D]
    const long long t0 = (long long)blockIdx.x * EMB_TOK;
    const int nt = (int)min((long long)EMB_TOK, n_tok - t0);
    for (int i = threadIdx.x; i < nt * D; i += EMB_THREADS) s_z[i] = z[t0 * D + i];
    __syncthreads();
    const int h = blockIdx.y * EMB_THREADS + threadIdx.x;
    if (h >= H) return;
    float acc[EMB_TOK];
#pragma unroll
    for (int t = 0; t < EMB_TOK; ++t) acc[t] = 0.f;
    const T* wr = w_in + (size_t)h * D;
    for (int d = 0; d < D; d += 4) {                     // D is a multiple of 4
        const float w0 = to_f<T>(wr[d]), w1 = to_f<T>(wr[d + 1]), w2 = to_f<T>(wr[d + 2]), w3 = to_f<T>(wr[d + 3]);
#pragma unroll
        for (int t = 0; t < EMB_TOK; ++t) {
            const float4 zv = *reinterpret_cast<const float4*>(s_z + t * D + d);     // same address for the whole warp
            acc[t] = fmaf(w3, zv.w, fmaf(w2, zv.z, fmaf(w1, zv.y, fmaf(w0, zv.x, acc[t]))));
        }
    }
    const float bias = to_f<T>(b_in[h]);
    int j = (int)(t0 % N);                               // position of the CTA's first token inside its request
#pragma unroll
    for (int t = 0; t < EMB_TOK; ++t) {
        if (t < nt) x[(size_t)(t0 + t) * H + h] = from_f<T>(acc[t] + bias + to_f<T>(pos[(size_t)j * H + h]));
        if (++j == N) j = 0;
    }
}

constexpr int FIN_ROWS = 8;        // active rows per CTA: one per warp
constexpr int FIN_THREADS = 256;
constexpr int FIN_KC = 64;         // columns of y per shared-memory chunk

// Warp w owns row w of the CTA's 8; its lane tx computes outputs tx, tx + 32, ... (D / 32 of them, at most 8).
template <typename T>
__global__ void __launch_bounds__(FIN_THREADS)
final_drift_kernel(const T* __restrict__ y, const int32_t* __restrict__ active_idx, const int32_t* __restrict__ cu_active,
                   int B, const T* __restrict__ w_out, const T* __restrict__ b_out, float* __restrict__ drift, int D,
                   int H, float ln_eps) {
    extern __shared__ float s_fin[];
    float* s_a = s_fin;                                  // [FIN_ROWS][FIN_KC + 1]  normalised rows, one chunk
    float* s_w = s_a + FIN_ROWS * (FIN_KC + 1);          // [D][FIN_KC + 1]
    float* s_mean = s_w + D * (FIN_KC + 1);              // [FIN_ROWS]
    float* s_rstd = s_mean + FIN_ROWS;
    __shared__ long long s_tok[FIN_ROWS];
    const int a_total = cu_active[B];
    const int row0 = blockIdx.x * FIN_ROWS;
    if (row0 >= a_total) return;
    const int nr = min(FIN_ROWS, a_total - row0);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // row statistics: warp w takes rows w, w + 8, ...
    for (int r = warp; r < FIN_ROWS; r += FIN_THREADS / 32) {
        if (r < nr) {
            const long long tok = active_idx[row0 + r];
            const T* yr = y + (size_t)tok * H;
            float sum = 0.f;
            for (int c = lane; c < H; c += 32) sum += to_f<T>(yr[c]);
            const float mean = warp_sum(sum) / (float)H;
            float sq = 0.f;
            for (int c = lane; c < H; c += 32) { const float d = to_f<T>(yr[c]) - mean; sq = fmaf(d, d, sq); }
            const float rstd = rsqrtf(warp_sum(sq) / (float)H + ln_eps);
            if (lane == 0) { s_mean[r] = mean; s_rstd[r] = rstd; s_tok[r] = tok; }
        } else if (lane == 0) {
            s_mean[r] = 0.f; s_rstd[r] = 0.f; s_tok[r] = -1;
        }
    }
    __syncthreads();
    const int ty = warp, tx = lane;
    const int nd = D / 32 + (D % 32 ? 1 : 0);            // outputs per thread (<= 8)
    float acc[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) acc[k] = 0.f;
    for (int c0 = 0; c0 < H; c0 += FIN_KC) {
        const int kc = min(FIN_KC, H - c0);
        for (int i = threadIdx.x; i < FIN_ROWS * FIN_KC; i += FIN_THREADS) {
            const int r = i / FIN_KC, c = i % FIN_KC;
            float v = 0.f;
            if (r < nr && c < kc) v = (to_f<T>(y[(size_t)s_tok[r] * H + c0 + c]) - s_mean[r]) * s_rstd[r];
            s_a[r * (FIN_KC + 1) + c] = v;
        }
        for (int i = threadIdx.x; i < D * FIN_KC; i += FIN_THREADS) {
            const int d = i / FIN_KC, c = i % FIN_KC;
            s_w[d * (FIN_KC + 1) + c] = c < kc ? to_f<T>(w_out[(size_t)d * H + c0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll 4
        for (int c = 0; c < FIN_KC; ++c) {
            const float a = s_a[ty * (FIN_KC + 1) + c];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                if (k < nd) {
                    const int d = tx + 32 * k;
                    acc[k] = fmaf(a, d < D ? s_w[d * (FIN_KC + 1) + c] : 0.f, acc[k]);
                }
            }
        }
        __syncthreads();
    }
    if (ty < nr) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const int d = tx + 32 * k;
            if (k < nd && d < D) drift[(size_t)s_tok[ty] * D + d] = acc[k] + to_f<T>(b_out[d]);
        }
    }
}

__global__ void __launch_bounds__(256)
euler_kernel(const float4* __restrict__ z, const float4* __restrict__ drift, const float* __restrict__ h,
             float4* __restrict__ z_next, long long n_vec, long long vec_per_request) {
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < n_vec; i += (long long)gridDim.x * blockDim.x) {
        const float hb = __ldg(h + i / vec_per_request);
        const float4 a = z[i], d = drift[i];
        z_next[i] = make_float4(fmaf(hb, d.x, a.x), fmaf(hb, d.y, a.y), fmaf(hb, d.z, a.z), fmaf(hb, d.w, a.w));
    }
}

// ---- bf16 storage: the two skinny contractions on mma.sync m16n8k16 ----------------------------------------
// Both read their operands straight from global memory in the lane layout of the instruction's fragments.
// Lane (g, t) = (lane / 4, lane % 4) always supplies consecutive k positions [kb + 4 t, kb + 4 t + 4) (or 8 of
// them for two products) on BOTH operands; the instruction's own k numbering differs, but a sum over k does
// not care in which order its terms are paired as long as both operands use the same order.
__device__ __forceinline__ void mma_bf16_16x8x16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                                 uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t bf16x2(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Final layer: drift[tok, d] = rstd_tok (sum_h y[tok, h] W[d, h] - mean_tok sum_h W[d, h]) + b[d].
// One warp = 8 active tokens x all D outputs (NS strips of 16); the row statistics of the tokens and the row sums
// of W come out of the same pass over y and W.
constexpr int FM_WARPS = 4;
template <int NS>
__global__ void __launch_bounds__(FM_WARPS * 32)
final_drift_mma_kernel(const __nv_bfloat16* __restrict__ y, const int32_t* __restrict__ active_idx,
                       const int32_t* __restrict__ cu_active, int B, const __nv_bfloat16* __restrict__ w_out,
                       const __nv_bfloat16* __restrict__ b_out, float* __restrict__ drift, int H, float ln_eps) {
    constexpr int D = NS * 16;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int a_total = cu_active[B];
    const int row0 = (blockIdx.x * FM_WARPS + warp) * 8;
    if (row0 >= a_total) return;
    const long long tok = active_idx[min(row0 + g, a_total - 1)];        // column g of the B operand
    const uint4* yr = reinterpret_cast<const uint4*>(y + (size_t)tok * H) + t;      // 8 elements at k = 32 blk + 8 t
    const float y0 = __bfloat162float(y[(size_t)tok * H]);
    float s1 = 0.f, s2 = 0.f;
    float wsa[NS], wsb[NS], c[NS][4];
#pragma unroll
    for (int s = 0; s < NS; ++s) { wsa[s] = 0.f; wsb[s] = 0.f; c[s][0] = c[s][1] = c[s][2] = c[s][3] = 0.f; }
    const int n_blk = H / 32;
#pragma unroll 2
    for (int kb = 0; kb < n_blk; ++kb) {
        const uint4 x = __ldg(yr + kb * 4);
        const uint32_t xw[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float e0 = bf_lo(xw[i]) - y0, e1 = bf_hi(xw[i]) - y0;
            s1 += e0 + e1;
            s2 = fmaf(e0, e0, fmaf(e1, e1, s2));
        }
#pragma unroll
        for (int s = 0; s < NS; ++s) {
            const uint4 va = __ldg(reinterpret_cast<const uint4*>(w_out + (size_t)(s * 16 + g) * H) + t + kb * 4);
            const uint4 vb = __ldg(reinterpret_cast<const uint4*>(w_out + (size_t)(s * 16 + g + 8) * H) + t + kb * 4);
            wsa[s] += (bf_lo(va.x) + bf_hi(va.x)) + (bf_lo(va.y) + bf_hi(va.y)) + (bf_lo(va.z) + bf_hi(va.z)) + (bf_lo(va.w) + bf_hi(va.w));
            wsb[s] += (bf_lo(vb.x) + bf_hi(vb.x)) + (bf_lo(vb.y) + bf_hi(vb.y)) + (bf_lo(vb.z) + bf_hi(vb.z)) + (bf_lo(vb.w) + bf_hi(vb.w));
            mma_bf16_16x8x16(c[s], va.x, vb.x, va.y, vb.y, x.x, x.y);
            mma_bf16_16x8x16(c[s], va.z, vb.z, va.w, vb.w, x.z, x.w);
        }
    }
    // the four lanes of a token (and of a W row) hold partial sums
    s1 += __shfl_xor_sync(0xffffffffu, s1, 1); s1 += __shfl_xor_sync(0xffffffffu, s1, 2);
    s2 += __shfl_xor_sync(0xffffffffu, s2, 1); s2 += __shfl_xor_sync(0xffffffffu, s2, 2);
    const float dm = s1 / (float)H;                                       // mean - y0
    const float mean = y0 + dm;
    const float rstd = rsqrtf(fmaxf(s2 / (float)H - dm * dm, 0.f) + ln_eps);
    // c[s][0..1]: output d = 16 s + g of tokens 2 t, 2 t + 1;  c[s][2..3]: d + 8.  Their statistics sit in lanes 8 t, 8 t + 4.
    const float mean0 = __shfl_sync(0xffffffffu, mean, 8 * t), mean1 = __shfl_sync(0xffffffffu, mean, 8 * t + 4);
    const float rstd0 = __shfl_sync(0xffffffffu, rstd, 8 * t), rstd1 = __shfl_sync(0xffffffffu, rstd, 8 * t + 4);
    const long long tok0 = __shfl_sync(0xffffffffu, tok, 8 * t), tok1 = __shfl_sync(0xffffffffu, tok, 8 * t + 4);
    const bool ok0 = row0 + 2 * t < a_total, ok1 = row0 + 2 * t + 1 < a_total;
#pragma unroll
    for (int s = 0; s < NS; ++s) {
        float wa = wsa[s], wb = wsb[s];
        wa += __shfl_xor_sync(0xffffffffu, wa, 1); wa += __shfl_xor_sync(0xffffffffu, wa, 2);
        wb += __shfl_xor_sync(0xffffffffu, wb, 1); wb += __shfl_xor_sync(0xffffffffu, wb, 2);
        const int da = s * 16 + g, db = da + 8;
        const float ba = __bfloat162float(b_out[da]), bb = __bfloat162float(b_out[db]);
        if (ok0) {
            drift[(size_t)tok0 * D + da] = rstd0 * (c[s][0] - mean0 * wa) + ba;
            drift[(size_t)tok0 * D + db] = rstd0 * (c[s][2] - mean0 * wb) + bb;
        }
        if (ok1) {
            drift[(size_t)tok1 * D + da] = rstd1 * (c[s][1] - mean1 * wa) + ba;
            drift[(size_t)tok1 * D + db] = rstd1 * (c[s][3] - mean1 * wb) + bb;
        }
    }
}

// Patch embedding: x[tok, h] = sum_d z[tok, d] W[h, d] + b[h] + pos[j, h].  z is fp32: it enters as a bf16 head plus a
// bf16 remainder (two products), which keeps fp32-level accuracy.  One warp = 16 tokens x EM_COLS output columns;
// each 64-column group goes through a shared-memory tile so that the rows leave as whole 128-byte lines.
constexpr int EM_WARPS = 8, EM_COLS = 128;       // columns per CTA: smaller chunks = more CTAs in flight (audio 41 -> 34 us)
template <int KB>                                  // D / 16
__global__ void __launch_bounds__(EM_WARPS * 32)
embed_mma_kernel(const float* __restrict__ z, const __nv_bfloat16* __restrict__ w_in, const __nv_bfloat16* __restrict__ b_in,
                 const __nv_bfloat16* __restrict__ pos, __nv_bfloat16* __restrict__ x, long long n_tok, int N, int H) {
    constexpr int D = KB * 16;
    __shared__ __align__(16) float s_tile[EM_WARPS][16][64 + 4];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const long long t0 = ((long long)blockIdx.x * EM_WARPS + warp) * 16;
    if (t0 >= n_tok) return;
    const long long ta = min(t0 + g, n_tok - 1), tb = min(t0 + g + 8, n_tok - 1);
    uint32_t ah[KB][4], al[KB][4];
#pragma unroll
    for (int kb = 0; kb < KB; ++kb) {
        const float4 za = *reinterpret_cast<const float4*>(z + (size_t)ta * D + kb * 16 + 4 * t);
        const float4 zb = *reinterpret_cast<const float4*>(z + (size_t)tb * D + kb * 16 + 4 * t);
        ah[kb][0] = bf16x2(za.x, za.y); ah[kb][1] = bf16x2(zb.x, zb.y); ah[kb][2] = bf16x2(za.z, za.w); ah[kb][3] = bf16x2(zb.z, zb.w);
        al[kb][0] = bf16x2(za.x - bf_lo(ah[kb][0]), za.y - bf_hi(ah[kb][0]));
        al[kb][1] = bf16x2(zb.x - bf_lo(ah[kb][1]), zb.y - bf_hi(ah[kb][1]));
        al[kb][2] = bf16x2(za.z - bf_lo(ah[kb][2]), za.w - bf_hi(ah[kb][2]));
        al[kb][3] = bf16x2(zb.z - bf_lo(ah[kb][3]), zb.w - bf_hi(ah[kb][3]));
    }
    const int h_begin = blockIdx.y * EM_COLS, h_end = min(H, h_begin + EM_COLS);
    for (int h0 = h_begin; h0 < h_end; h0 += 64) {
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            const int hcol = min(h0 + nt * 8 + g, H - 1);
            const uint2* wr = reinterpret_cast<const uint2*>(w_in + (size_t)hcol * D) + t;      // 4 elements at k = 16 kb + 4 t
#pragma unroll
            for (int kb = 0; kb < KB; ++kb) {
                const uint2 wv = __ldg(wr + kb * 4);
                mma_bf16_16x8x16(c, ah[kb][0], ah[kb][1], ah[kb][2], ah[kb][3], wv.x, wv.y);
                mma_bf16_16x8x16(c, al[kb][0], al[kb][1], al[kb][2], al[kb][3], wv.x, wv.y);
            }
            *reinterpret_cast<float2*>(&s_tile[warp][g][nt * 8 + 2 * t]) = make_float2(c[0], c[1]);
            *reinterpret_cast<float2*>(&s_tile[warp][g + 8][nt * 8 + 2 * t]) = make_float2(c[2], c[3]);
        }
        __syncwarp();
        // eight lanes write one token's 64 columns (128 bytes); four tokens per pass
        const int cu = (lane & 7) * 8, hh = h0 + cu;
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            const int r = p * 4 + (lane >> 3);
            const long long tk = t0 + r;
            if (tk < n_tok && hh < H) {
                const int j = (int)(tk % N);
                const float4 v0 = *reinterpret_cast<const float4*>(&s_tile[warp][r][cu]);
                const float4 v1 = *reinterpret_cast<const float4*>(&s_tile[warp][r][cu + 4]);
                const uint4 bv = __ldg(reinterpret_cast<const uint4*>(b_in + hh));
                const uint4 pv = __ldg(reinterpret_cast<const uint4*>(pos + (size_t)j * H + hh));
                uint4 o;
                o.x = bf16x2(v0.x + bf_lo(bv.x) + bf_lo(pv.x), v0.y + bf_hi(bv.x) + bf_hi(pv.x));
                o.y = bf16x2(v0.z + bf_lo(bv.y) + bf_lo(pv.y), v0.w + bf_hi(bv.y) + bf_hi(pv.y));
                o.z = bf16x2(v1.x + bf_lo(bv.z) + bf_lo(pv.z), v1.y + bf_hi(bv.z) + bf_hi(pv.z));
                o.w = bf16x2(v1.z + bf_lo(bv.w) + bf_lo(pv.w), v1.w + bf_hi(bv.w) + bf_hi(pv.w));
                *reinterpret_cast<uint4*>(x + (size_t)tk * H + hh) = o;
            }
        }
        __syncwarp();
    }
}

}  // namespace

template <typename T>
cudaError_t launch_embed(const float* z, const T* w_in, const T* b_in, const T* pos, T* x, int B, int N, int D, int H,
                         cudaStream_t st, int* n_launch) {
    const long long n_tok = (long long)B * N;
    if constexpr (sizeof(T) == 2) {
        if (H % 64 == 0 && (D == 16 || D == 32 || D == 64 || D == 128)) {
            dim3 mg((unsigned)((n_tok + EM_WARPS * 16 - 1) / (EM_WARPS * 16)), (unsigned)((H + EM_COLS - 1) / EM_COLS));
            if (D == 16) embed_mma_kernel<1><<<mg, EM_WARPS * 32, 0, st>>>(z, w_in, b_in, pos, x, n_tok, N, H);
            else if (D == 32) embed_mma_kernel<2><<<mg, EM_WARPS * 32, 0, st>>>(z, w_in, b_in, pos, x, n_tok, N, H);
            else if (D == 64) embed_mma_kernel<4><<<mg, EM_WARPS * 32, 0, st>>>(z, w_in, b_in, pos, x, n_tok, N, H);
            else embed_mma_kernel<8><<<mg, EM_WARPS * 32, 0, st>>>(z, w_in, b_in, pos, x, n_tok, N, H);
            ++*n_launch;
            return cudaGetLastError();
        }
    }
    dim3 grid((unsigned)((n_tok + EMB_TOK - 1) / EMB_TOK), (unsigned)((H + EMB_THREADS - 1) / EMB_THREADS));
    embed_kernel<T><<<grid, EMB_THREADS, (size_t)EMB_TOK * D * sizeof(float), st>>>(z, w_in, b_in, pos, x, n_tok, N, D, H);
    ++*n_launch;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_update(const float* z, const T* y, const int32_t* active_idx, const int32_t* cu_active, const float* h,
                          const T* w_out, const T* b_out, float* drift, float* z_next, int B, int N, int D, int H,
                          float ln_eps, cudaStream_t st, int* n_launch) {
    const size_t smem = ((size_t)FIN_ROWS * (FIN_KC + 1) + (size_t)D * (FIN_KC + 1) + 2 * FIN_ROWS) * sizeof(float);
    cudaError_t e = cudaFuncSetAttribute(final_drift_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long rows_cap = (long long)B * N;
    bool done = false;
    if constexpr (sizeof(T) == 2) {
        if (H % 32 == 0 && (D == 16 || D == 32 || D == 64)) {
            const unsigned mg = (unsigned)((rows_cap + FM_WARPS * 8 - 1) / (FM_WARPS * 8));
            if (D == 16) final_drift_mma_kernel<1><<<mg, FM_WARPS * 32, 0, st>>>(y, active_idx, cu_active, B, w_out, b_out, drift, H, ln_eps);
            else if (D == 32) final_drift_mma_kernel<2><<<mg, FM_WARPS * 32, 0, st>>>(y, active_idx, cu_active, B, w_out, b_out, drift, H, ln_eps);
            else final_drift_mma_kernel<4><<<mg, FM_WARPS * 32, 0, st>>>(y, active_idx, cu_active, B, w_out, b_out, drift, H, ln_eps);
            done = true;
        }
    }
    if (!done)
    final_drift_kernel<T><<<(unsigned)((rows_cap + FIN_ROWS - 1) / FIN_ROWS), FIN_THREADS, smem, st>>>(
        y, active_idx, cu_active, B, w_out, b_out, drift, D, H, ln_eps);
    ++*n_launch;
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    const long long n_vec = rows_cap * D / 4;
    const long long want = (n_vec + 255) / 256;
    const int grid = (int)(want < 148 * 8 ? want : 148 * 8);
    euler_kernel<<<max(grid, 1), 256, 0, st>>>(reinterpret_cast<const float4*>(z), reinterpret_cast<const float4*>(drift), h,
                                               reinterpret_cast<float4*>(z_next), n_vec, (long long)N * D / 4);
    ++*n_launch;
    return cudaGetLastError();
}

template cudaError_t launch_embed<float>(const float*, const float*, const float*, const float*, float*, int, int, int, int,
                                         cudaStream_t, int*);
template cudaError_t launch_embed<__nv_bfloat16>(const float*, const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                 __nv_bfloat16*, int, int, int, int, cudaStream_t, int*);
template cudaError_t launch_update<float>(const float*, const float*, const int32_t*, const int32_t*, const float*, const float*,
                                          const float*, float*, float*, int, int, int, int, float, cudaStream_t, int*);
template cudaError_t launch_update<__nv_bfloat16>(const float*, const __nv_bfloat16*, const int32_t*, const int32_t*, const float*,
                                                  const __nv_bfloat16*, const __nv_bfloat16*, float*, float*, int, int, int, int,
                                                  float, cudaStream_t, int*);

}  // namespace fd
