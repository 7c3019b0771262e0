// Row-wise, memory-bound pieces of the block: the adaLN conditioning vectors and the
// gather + LayerNorm + modulation that feeds the QKV and MLP projections.  The block is the
// adaLN-Zero DiT block the paper builds on (Sec. 2.1); only active rows are touched (Sec. 3).
#include "common.cuh"
#include "ptx.cuh"

namespace fd {

namespace {

// ---- 16-byte vector access to a row of storage type T, as floats -----------------------------
template <typename T> struct Vec;
template <> struct Vec<float> {
    static constexpr int N = 4;
    __device__ static void load(const float* p, float* f) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    }
    __device__ static void store(float* p, const float* f) {
        *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    }
};
template <> struct Vec<__nv_bfloat16> {
    static constexpr int N = 8;
    __device__ static void load(const __nv_bfloat16* p, float* f) {
        const uint4 v = *reinterpret_cast<const uint4*>(p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ static void store(__nv_bfloat16* p, const float* f) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// ---- adaLN: mod[l,b,o] = sum_c SiLU(cond[b,c]) W_ada[l,o,c] + b_ada[l,o] ----------------------
// HBM-bound on W_ada (read once).  SiLU(cond) of up to 8 requests sits in shared memory; every warp
// streams 4 weight rows at a time with 128-bit loads so each shared-memory read feeds 4 rows.
constexpr int ADA_THREADS = 256;
constexpr int ADA_BCH = 8;         // requests handled per pass over the weights
constexpr int ADA_RPW = 4;         // weight rows a warp processes together
constexpr int ADA_ROWS = 128;      // weight rows per CTA

template <typename T>
__global__ void __launch_bounds__(ADA_THREADS)
adaln_kernel(const T* __restrict__ cond, const T* __restrict__ w_ada, const T* __restrict__ b_ada,
             float* __restrict__ mod, int L, int B, int H6, int Hc) {
    extern __shared__ float s_act[];            // [min(B,ADA_BCH)][Hc]
    constexpr int VN = Vec<T>::N;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long rows_total = (long long)L * H6;
    for (int b0 = 0; b0 < B; b0 += ADA_BCH) {
        const int nb = min(ADA_BCH, B - b0);
        __syncthreads();
        for (int i = threadIdx.x; i < nb * Hc; i += ADA_THREADS) {
            const float v = to_f<T>(cond[(size_t)(b0 + i / Hc) * Hc + (i % Hc)]);
            s_act[i] = v / (1.0f + __expf(-v));
        }
        __syncthreads();
        for (int r = warp * ADA_RPW; r < ADA_ROWS; r += (ADA_THREADS / 32) * ADA_RPW) {
            const long long row0 = (long long)blockIdx.x * ADA_ROWS + r;
            if (row0 >= rows_total) break;
            float acc[ADA_RPW][ADA_BCH];
#pragma unroll
            for (int q = 0; q < ADA_RPW; ++q)
#pragma unroll
                for (int b = 0; b < ADA_BCH; ++b) acc[q][b] = 0.f;
            for (int c = lane * VN; c < Hc; c += 32 * VN) {
                float w[ADA_RPW][VN];
#pragma unroll
                for (int q = 0; q < ADA_RPW; ++q) {
                    const long long row = min(row0 + q, rows_total - 1);
                    Vec<T>::load(w_ada + (size_t)row * Hc + c, w[q]);
                }
#pragma unroll
                for (int b = 0; b < ADA_BCH; ++b) {
                    if (b < nb) {
                        float a[VN];
#pragma unroll
                        for (int k = 0; k < VN; k += 4) {
                            const float4 t = *reinterpret_cast<const float4*>(s_act + b * Hc + c + k);
                            a[k] = t.x; a[k + 1] = t.y; a[k + 2] = t.z; a[k + 3] = t.w;
                        }
#pragma unroll
                        for (int q = 0; q < ADA_RPW; ++q)
#pragma unroll
                            for (int k = 0; k < VN; ++k) acc[q][b] = fmaf(w[q][k], a[k], acc[q][b]);
                    }
                }
            }
#pragma unroll
            for (int q = 0; q < ADA_RPW; ++q) {
                const long long row = row0 + q;
#pragma unroll
                for (int b = 0; b < ADA_BCH; ++b) {
                    if (b < nb) {
                        const float v = warp_sum(acc[q][b]);
                        if (lane == 0 && row < rows_total) {
                            const int l = (int)(row / H6), o = (int)(row % H6);
                            mod[((size_t)l * B + (b0 + b)) * H6 + o] = v + to_f<T>(b_ada[row]);
                        }
                    }
                }
            }
        }
    }
}

// ---- adaLN on bf16 weights: a skinny contraction [L*6H, Hc] x [Hc, B] that must stream W_ada at HBM
// speed.  CUDA cores would be arithmetic-bound here (8 FMAs per weight element), so the products go
// through mma.sync m16n8k16 (16 weight rows x 8 requests per instruction).  SiLU(cond) is split into
// a bf16 head and a bf16 remainder, so the activations keep fp32-level accuracy.
__global__ void __launch_bounds__(256)
adaln_act_kernel(const __nv_bfloat16* __restrict__ cond, __nv_bfloat16* __restrict__ act, int B, int B8, int Hc) {
    // act[part][b][c], part 0 = head, part 1 = remainder; requests b >= B are zero
    const int i = blockIdx.x * 256 + threadIdx.x;
    if (i >= B8 * Hc) return;
    const int b = i / Hc;
    float v = 0.f;
    if (b < B) { const float x = __bfloat162float(cond[i]); v = x / (1.0f + __expf(-x)); }
    const __nv_bfloat16 hi = __float2bfloat16_rn(v);
    act[i] = hi;
    act[(size_t)B8 * Hc + i] = __float2bfloat16_rn(v - __bfloat162float(hi));
}

__device__ __forceinline__ void mma_16x8x16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                            uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

constexpr int ADM_WARPS = 8;
constexpr int ADM_UNROLL = 4;       // 32-wide k blocks in flight per lane

__global__ void __launch_bounds__(ADM_WARPS * 32)
adaln_mma_kernel(const __nv_bfloat16* __restrict__ act, const __nv_bfloat16* __restrict__ w_ada,
                 const __nv_bfloat16* __restrict__ b_ada, float* __restrict__ mod, long long rows_total, int B,
                 int B8, int H6, int Hc) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const long long strip = (long long)blockIdx.x * ADM_WARPS + warp;       // 16 weight rows
    const long long row0 = strip * 16;
    if (row0 >= rows_total) return;
    const long long ra = min(row0 + g, rows_total - 1), rb = min(row0 + g + 8, rows_total - 1);
    const uint4* wa = reinterpret_cast<const uint4*>(w_ada + (size_t)ra * Hc) + t;   // 8 elements at k = 32 blk + 8 t
    const uint4* wb = reinterpret_cast<const uint4*>(w_ada + (size_t)rb * Hc) + t;
    for (int b0 = 0; b0 < B8; b0 += 8) {
        // lane (g, t) supplies the activations of request b0 + g for the same 8 k positions
        const uint4* ah = reinterpret_cast<const uint4*>(act + (size_t)(b0 + g) * Hc) + t;
        const uint4* al = reinterpret_cast<const uint4*>(act + (size_t)B8 * Hc + (size_t)(b0 + g) * Hc) + t;
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        const int n_blk = Hc / 32;
        for (int kb = 0; kb < n_blk; kb += ADM_UNROLL) {
            uint4 va[ADM_UNROLL], vb[ADM_UNROLL], xh[ADM_UNROLL], xl[ADM_UNROLL];
#pragma unroll
            for (int u = 0; u < ADM_UNROLL; ++u) {
                const int k4 = min(kb + u, n_blk - 1) * 4;
                va[u] = __ldg(wa + k4);
                vb[u] = __ldg(wb + k4);
                xh[u] = __ldg(ah + k4);
                xl[u] = __ldg(al + k4);
            }
#pragma unroll
            for (int u = 0; u < ADM_UNROLL; ++u) {
                if (kb + u < n_blk) {
                    // the 8 k positions of this lane feed two k16 products: (x,y) then (z,w)
                    mma_16x8x16(c, va[u].x, vb[u].x, va[u].y, vb[u].y, xh[u].x, xh[u].y);
                    mma_16x8x16(c, va[u].z, vb[u].z, va[u].w, vb[u].w, xh[u].z, xh[u].w);
                    mma_16x8x16(c, va[u].x, vb[u].x, va[u].y, vb[u].y, xl[u].x, xl[u].y);
                    mma_16x8x16(c, va[u].z, vb[u].z, va[u].w, vb[u].w, xl[u].z, xl[u].w);
                }
            }
        }
        // c0,c1: row g, requests 2t, 2t+1;  c2,c3: row g + 8
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const long long row = row0 + g + (q >= 2 ? 8 : 0);
            const int b = b0 + 2 * t + (q & 1);
            if (row < rows_total && b < B) {
                const int l = (int)(row / H6), o = (int)(row % H6);
                mod[((size_t)l * B + b) * H6 + o] = c[q] + __bfloat162float(b_ada[row]);
            }
        }
    }
}

// ---- gather + LayerNorm + modulation, one warp per active row --------------------------------
// Pass 1 streams the row once (128-bit loads) and accumulates sum and sum of squares of (x - x0),
// x0 = the row's first element, which keeps the one-pass variance well conditioned.  Pass 2 reads
// the row again (it is still in L1/L2), normalises, modulates and writes 128-bit vectors.  Nothing
// of the row is kept in registers, so many warps per SM hide the memory latency.
constexpr int LN_THREADS = 128;

template <typename T>
__device__ __forceinline__ void ln_load4(const T* x_gather, const float* resid_in, size_t g_off, size_t r_off,
                                         float* f) {
    if (x_gather) {
        if constexpr (sizeof(T) == 2) {
            const uint2 u = *reinterpret_cast<const uint2*>(x_gather + g_off);
            f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
            f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
        } else {
            const float4 u = *reinterpret_cast<const float4*>(x_gather + g_off);
            f[0] = u.x; f[1] = u.y; f[2] = u.z; f[3] = u.w;
        }
    } else {
        const float4 u = *reinterpret_cast<const float4*>(resid_in + r_off);
        f[0] = u.x; f[1] = u.y; f[2] = u.z; f[3] = u.w;
    }
}

template <typename T>
__global__ void __launch_bounds__(LN_THREADS, 8)
ln_modulate_kernel(const T* __restrict__ x_gather, const float* __restrict__ resid_in,
                   float* __restrict__ resid_out, T* __restrict__ out, const int32_t* __restrict__ active_idx,
                   const float* __restrict__ shift, const float* __restrict__ scale, int mod_stride, int N,
                   int H, float ln_eps, const Control* __restrict__ ctl, TextSel ts, float fp8_inv) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    ptx::pdl_wait();                              // the rows come from the kernel launched just before
    const int a_total = ctl->a_total;
    const int nv = H / 128;                       // float4 slots per lane (H % 128 == 0 on this path)
    for (int row = blockIdx.x * (LN_THREADS / 32) + warp; row < a_total; row += gridDim.x * (LN_THREADS / 32)) {
        const int tok = active_idx[row];
        const int b = tok / N;
        const size_t g0 = (size_t)tok * H, r0 = (size_t)row * H;
        const float x0 = x_gather ? to_f<T>(x_gather[g0]) : resid_in[r0];
        float sum = 0.f, sq = 0.f;
#pragma unroll 4
        for (int i = 0; i < nv; ++i) {
            const int c = (i * 32 + lane) * 4;
            float v[4];
            ln_load4<T>(x_gather, resid_in, g0 + c, r0 + c, v);
            if (x_gather && resid_out)
                *reinterpret_cast<float4*>(resid_out + r0 + c) = make_float4(v[0], v[1], v[2], v[3]);
#pragma unroll
            for (int k = 0; k < 4; ++k) { const float d = v[k] - x0; sum += d; sq = fmaf(d, d, sq); }
        }
        sum = warp_sum(sum);
        sq = warp_sum(sq);
        const float dm = sum / (float)H;                       // mean - x0
        const float var = fmaxf(sq / (float)H - dm * dm, 0.f);
        const float rstd = rsqrtf(var + ln_eps);
        const float mean = x0 + dm;
        // dual stream: a token with label R takes the second stream's vectors
        const bool text_row = ts.labels && ts.labels[tok] == ts.R;
        const long long soff = text_row ? ts.mod_off : 0;
        const float q_inv = text_row ? ts.fp8_inv_text : fp8_inv;      // FP8 operands: the row's stream's scale
        const float* sh = shift + (size_t)b * mod_stride + soff;
        const float* sc = scale + (size_t)b * mod_stride + soff;
#pragma unroll 4
        for (int i = 0; i < nv; ++i) {
            const int c = (i * 32 + lane) * 4;
            float v[4];
            ln_load4<T>(x_gather, resid_in, g0 + c, r0 + c, v);
            const float4 s4 = __ldg(reinterpret_cast<const float4*>(sc + c));
            const float4 h4 = __ldg(reinterpret_cast<const float4*>(sh + c));
            const float o0 = (v[0] - mean) * rstd * (1.f + s4.x) + h4.x;
            const float o1 = (v[1] - mean) * rstd * (1.f + s4.y) + h4.y;
            const float o2 = (v[2] - mean) * rstd * (1.f + s4.z) + h4.z;
            const float o3 = (v[3] - mean) * rstd * (1.f + s4.w) + h4.w;
            T* dst = out + r0 + c;
            if constexpr (sizeof(T) == 2) {
                if (fp8_inv > 0.f) {          // FP8 operands: the projection reads this row as E4M3
                    *reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(out) + r0 + c) =
                        pack4_e4m3(o0 * q_inv, o1 * q_inv, o2 * q_inv, o3 * q_inv);
                    continue;
                }
                const __nv_bfloat162 p0 = __floats2bfloat162_rn(o0, o1), p1 = __floats2bfloat162_rn(o2, o3);
                uint2 u;
                u.x = *reinterpret_cast<const uint32_t*>(&p0);
                u.y = *reinterpret_cast<const uint32_t*>(&p1);
                *reinterpret_cast<uint2*>(dst) = u;
            } else {
                *reinterpret_cast<float4*>(dst) = make_float4(o0, o1, o2, o3);
            }
        }
    }
    // a multi-wave kernel: let the successor start only when this CTA is done, so that its waiting CTAs
    // do not take registers away from the waves still to run
    ptx::pdl_trigger();
}

// The same with the row held in registers (NV float4 slots per lane, H = 128 NV): every load of a row is in
// flight at once and the row is read a single time.
template <typename T, int NV, bool GATHER>
__global__ void __launch_bounds__(LN_THREADS, 6)
ln_modulate_reg_kernel(const T* __restrict__ x_gather, const float* __restrict__ resid_in,
                       float* __restrict__ resid_out, T* __restrict__ out, const int32_t* __restrict__ active_idx,
                       const float* __restrict__ shift, const float* __restrict__ scale, int mod_stride, int N,
                       float ln_eps, const Control* __restrict__ ctl, TextSel ts, float fp8_inv) {
    constexpr int H = NV * 128;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    ptx::pdl_wait();                              // the rows come from the kernel launched just before
    const int a_total = ctl->a_total;
    for (int row = blockIdx.x * (LN_THREADS / 32) + warp; row < a_total; row += gridDim.x * (LN_THREADS / 32)) {
        const int tok = active_idx[row];
        // one base pointer per stream and constant offsets: every lane's i-th vector is 32 vectors further
        float v[NV][4];
        if constexpr (GATHER) {
            const T* src = x_gather + (size_t)tok * H + lane * 4;
#pragma unroll
            for (int i = 0; i < NV; ++i) ln_load4<T>(src, nullptr, i * 128, 0, v[i]);
            if (resid_out) {
                float4* keep = reinterpret_cast<float4*>(resid_out + (size_t)row * H) + lane;
#pragma unroll
                for (int i = 0; i < NV; ++i) keep[i * 32] = make_float4(v[i][0], v[i][1], v[i][2], v[i][3]);
            }
        } else {
            const float4* src = reinterpret_cast<const float4*>(resid_in + (size_t)row * H) + lane;
#pragma unroll
            for (int i = 0; i < NV; ++i) {
                const float4 u = src[i * 32];
                v[i][0] = u.x; v[i][1] = u.y; v[i][2] = u.z; v[i][3] = u.w;
            }
        }
        // one pass, shifted by the row's first element (keeps the cancellation in sq - sum^2 harmless); four
        // independent accumulator pairs and the two reductions side by side keep the dependent chains short
        const float x0 = __shfl_sync(0xffffffffu, v[0][0], 0);
        float su[4] = {0.f, 0.f, 0.f, 0.f}, sq4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int i = 0; i < NV; ++i)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float d = v[i][k] - x0;
                su[k] += d;
                sq4[k] = fmaf(d, d, sq4[k]);
            }
        float sum = (su[0] + su[1]) + (su[2] + su[3]);
        float sq = (sq4[0] + sq4[1]) + (sq4[2] + sq4[3]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sum += __shfl_xor_sync(0xffffffffu, sum, o);
            sq += __shfl_xor_sync(0xffffffffu, sq, o);
        }
        const float dm = sum / (float)H;                       // mean - x0
        const float rstd = rsqrtf(fmaxf(sq / (float)H - dm * dm, 0.f) + ln_eps);
        const float mean = x0 + dm;
        const int b = tok / N;
        const bool text_row = ts.labels && ts.labels[tok] == ts.R;                          // dual stream
        const long long soff = text_row ? ts.mod_off : 0;
        const float q_inv = text_row ? ts.fp8_inv_text : fp8_inv;      // FP8 operands: the row's stream's scale
        const float4* sc4 = reinterpret_cast<const float4*>(scale + (size_t)b * mod_stride + soff) + lane;
        const float4* sh4 = reinterpret_cast<const float4*>(shift + (size_t)b * mod_stride + soff) + lane;
        T* dst = out + (size_t)row * H + lane * 4;
#pragma unroll
        for (int i = 0; i < NV; ++i) {
            const float4 s4 = __ldg(sc4 + i * 32);
            const float4 h4 = __ldg(sh4 + i * 32);
            const float o0 = (v[i][0] - mean) * rstd * (1.f + s4.x) + h4.x;
            const float o1 = (v[i][1] - mean) * rstd * (1.f + s4.y) + h4.y;
            const float o2 = (v[i][2] - mean) * rstd * (1.f + s4.z) + h4.z;
            const float o3 = (v[i][3] - mean) * rstd * (1.f + s4.w) + h4.w;
            if constexpr (sizeof(T) == 2) {
                if (fp8_inv > 0.f) {          // FP8 operands: the projection reads this row as E4M3
                    *reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(out) + (size_t)row * H + lane * 4 + i * 128) =
                        pack4_e4m3(o0 * q_inv, o1 * q_inv, o2 * q_inv, o3 * q_inv);
                    continue;
                }
                const __nv_bfloat162 p0 = __floats2bfloat162_rn(o0, o1), p1 = __floats2bfloat162_rn(o2, o3);
                uint2 u;
                u.x = *reinterpret_cast<const uint32_t*>(&p0);
                u.y = *reinterpret_cast<const uint32_t*>(&p1);
                *reinterpret_cast<uint2*>(dst + i * 128) = u;
            } else {
                *reinterpret_cast<float4*>(dst + i * 128) = make_float4(o0, o1, o2, o3);
            }
        }
    }
    ptx::pdl_trigger();
}

// Any width: three passes over the row (the re-reads hit L1/L2).
template <typename T>
__global__ void __launch_bounds__(LN_THREADS)
ln_modulate_generic_kernel(const T* __restrict__ x_gather, const float* __restrict__ resid_in,
                           float* __restrict__ resid_out, T* __restrict__ out,
                           const int32_t* __restrict__ active_idx, const float* __restrict__ shift,
                           const float* __restrict__ scale, int mod_stride, int N, int H, float ln_eps,
                           const Control* __restrict__ ctl, TextSel ts) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int a_total = ctl->a_total;
    for (int row = blockIdx.x * (LN_THREADS / 32) + warp; row < a_total; row += gridDim.x * (LN_THREADS / 32)) {
        const int tok = active_idx[row];
        const int b = tok / N;
        auto at = [&](int c) -> float {
            return x_gather ? to_f<T>(x_gather[(size_t)tok * H + c]) : resid_in[(size_t)row * H + c];
        };
        float sum = 0.f;
        for (int c = lane; c < H; c += 32) sum += at(c);
        const float mean = warp_sum(sum) / (float)H;
        float sq = 0.f;
        for (int c = lane; c < H; c += 32) { const float d = at(c) - mean; sq = fmaf(d, d, sq); }
        const float rstd = rsqrtf(warp_sum(sq) / (float)H + ln_eps);
        const long long soff = (ts.labels && ts.labels[tok] == ts.R) ? ts.mod_off : 0;      // dual stream
        const float* sh = shift + (size_t)b * mod_stride + soff;
        const float* sc = scale + (size_t)b * mod_stride + soff;
        for (int c = lane; c < H; c += 32) {
            const float u = at(c);
            if (x_gather && resid_out) resid_out[(size_t)row * H + c] = u;
            out[(size_t)row * H + c] = from_f<T>((u - mean) * rstd * (1.f + sc[c]) + sh[c]);
        }
    }
}

}  // namespace

template <typename T>
cudaError_t launch_adaln(const T* cond, const T* w_ada, const T* b_ada, float* mod, int L, int B, int H,
                         int Hc, void* act_scratch, cudaStream_t st, int* n_launch) {
    const long long rows = (long long)L * 6 * H;
    if constexpr (sizeof(T) == 2) {
        if (Hc % 32 == 0 && act_scratch) {
            const int B8 = (B + 7) / 8 * 8;
            __nv_bfloat16* act = static_cast<__nv_bfloat16*>(act_scratch);
            adaln_act_kernel<<<(B8 * Hc + 255) / 256, 256, 0, st>>>(cond, act, B, B8, Hc);
            ++*n_launch;
            const long long strips = (rows + 15) / 16;
            adaln_mma_kernel<<<(unsigned)((strips + ADM_WARPS - 1) / ADM_WARPS), ADM_WARPS * 32, 0, st>>>(
                act, w_ada, b_ada, mod, rows, B, B8, 6 * H, Hc);
            ++*n_launch;
            return cudaGetLastError();
        }
    }
    const int grid = (int)((rows + ADA_ROWS - 1) / ADA_ROWS);
    const size_t smem = (size_t)min(B, ADA_BCH) * Hc * sizeof(float);
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(adaln_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    adaln_kernel<T><<<grid, ADA_THREADS, smem, st>>>(cond, w_ada, b_ada, mod, L, B, 6 * H, Hc);
    ++*n_launch;
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_ln_modulate(const T* x_gather, const float* resid_in, float* resid_out, T* out,
                               const int32_t* active_idx, const float* shift, const float* scale,
                               int mod_stride, int N, int H, int rows_cap, float ln_eps, const Control* ctl,
                               cudaStream_t st, int* n_launch, bool pdl, TextSel ts, float fp8_inv) {
    if (fp8_inv > 0.f && (sizeof(T) != 2 || H % 128 != 0)) return cudaErrorInvalidValue;
    const int rows_per_cta = LN_THREADS / 32;
    const int grid = max(1, min((rows_cap + rows_per_cta - 1) / rows_per_cta, 148 * 16));
#define FD_LN_REG(NV)                                                                                              \
    if (H == NV * 128) {                                                                                           \
        cudaError_t e = x_gather                                                                                    \
            ? ptx::launch_kernel(ln_modulate_reg_kernel<T, NV, true>, grid, LN_THREADS, 0, st, pdl, x_gather,      \
                                 resid_in, resid_out, out, active_idx, shift, scale, mod_stride, N, ln_eps, ctl, ts, fp8_inv) \
            : ptx::launch_kernel(ln_modulate_reg_kernel<T, NV, false>, grid, LN_THREADS, 0, st, pdl, x_gather,     \
                                 resid_in, resid_out, out, active_idx, shift, scale, mod_stride, N, ln_eps, ctl, ts, fp8_inv); \
        ++*n_launch;                                                                                               \
        return e;                                                                                                  \
    }
    FD_LN_REG(8)
    FD_LN_REG(9)
    FD_LN_REG(12)
#undef FD_LN_REG
    if (H % 128 == 0) {
        cudaError_t e = ptx::launch_kernel(ln_modulate_kernel<T>, grid, LN_THREADS, 0, st, pdl, x_gather, resid_in, resid_out,
                                           out, active_idx, shift, scale, mod_stride, N, H, ln_eps, ctl, ts, fp8_inv);
        ++*n_launch;
        return e;
    } else
        ln_modulate_generic_kernel<T><<<grid, LN_THREADS, 0, st>>>(x_gather, resid_in, resid_out, out, active_idx,
                                                                  shift, scale, mod_stride, N, H, ln_eps, ctl, ts);
    ++*n_launch;
    return cudaGetLastError();
}

template cudaError_t launch_adaln<float>(const float*, const float*, const float*, float*, int, int, int, int, void*,
                                         cudaStream_t, int*);
template cudaError_t launch_adaln<__nv_bfloat16>(const __nv_bfloat16*, const __nv_bfloat16*, const __nv_bfloat16*,
                                                 float*, int, int, int, int, void*, cudaStream_t, int*);
template cudaError_t launch_ln_modulate<float>(const float*, const float*, float*, float*, const int32_t*,
                                               const float*, const float*, int, int, int, int, float, const Control*,
                                               cudaStream_t, int*, bool, TextSel, float);
template cudaError_t launch_ln_modulate<__nv_bfloat16>(const __nv_bfloat16*, const float*, float*, __nv_bfloat16*,
                                                       const int32_t*, const float*, const float*, int, int, int, int,
                                                       float, const Control*, cudaStream_t, int*, bool, TextSel, float);

}  // namespace fd
