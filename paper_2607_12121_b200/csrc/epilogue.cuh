// GEMM epilogues shared by the CUDA-core and tensor-core kernels.  Each call finishes four
// consecutive output columns of one compact row:
//   EPI_QKV   bias, then Q stays compact while K and V rows are scattered into the request's cache
//             (skipped tokens' rows are never written: they keep the previous step's K/V),
//   EPI_RESID bias, adaLN gate, residual add into the fp32 stream; the last block also scatters
//             the row into y,
//   EPI_GELU  bias and tanh-GELU.
#pragma once
#include "common.cuh"

namespace fd {

template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
template <typename T> __device__ __forceinline__ void load4(const T* p, float* f);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float* f) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
}

// row: compact row (< a_total), col: first of four columns, tok: active_idx[row]
template <typename T, int KIND>
__device__ __forceinline__ void epilogue4(const EpiParams& ep, int row, int col, int tok, const float* acc) {
    float bias[4];
    load4<T>(reinterpret_cast<const T*>(ep.bias) + col, bias);
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = acc[i] + bias[i];
    if constexpr (KIND == EPI_QKV) {
        const int sec = col / ep.H, c = col - sec * ep.H;
        if (sec == 0) {
            store4<T>(reinterpret_cast<T*>(ep.q) + (size_t)row * ep.q_ld + c, v[0], v[1], v[2], v[3]);
        } else {
            const int b = tok / ep.N, j = tok - b * ep.N;
            T* dst = reinterpret_cast<T*>(ep.kv) + (((size_t)b * 2 + (sec - 1)) * ep.N + j) * ep.H + c;
            store4<T>(dst, v[0], v[1], v[2], v[3]);
        }
    } else if constexpr (KIND == EPI_RESID) {
        const int b = tok / ep.N;
        const float4 g = *reinterpret_cast<const float4*>(ep.gate + (size_t)b * 6 * ep.H + col);
        float* rp = ep.resid + (size_t)row * ep.H + col;
        float4 r = *reinterpret_cast<const float4*>(rp);
        r.x = fmaf(g.x, v[0], r.x); r.y = fmaf(g.y, v[1], r.y);
        r.z = fmaf(g.z, v[2], r.z); r.w = fmaf(g.w, v[3], r.w);
        *reinterpret_cast<float4*>(rp) = r;
        if (ep.y) store4<T>(reinterpret_cast<T*>(ep.y) + (size_t)tok * ep.H + col, r.x, r.y, r.z, r.w);
    } else {
        store4<T>(reinterpret_cast<T*>(ep.out) + (size_t)row * ep.out_ld + col, gelu_tanh(v[0]), gelu_tanh(v[1]),
                  gelu_tanh(v[2]), gelu_tanh(v[3]));
    }
}

}  // namespace fd

// ---- 32-column variant for the tensor-core kernels (bf16 storage, H % 32 == 0) -----------------
namespace fd {

__device__ __forceinline__ float tanh_fast(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float gelu_tanh_fast(float a) {
    const float u = 0.7978845608028654f * fmaf(0.044715f * a * a, a, a);
    return 0.5f * a * (1.0f + tanh_fast(u));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ void store8_bf16(__nv_bfloat16* p, const float* v) {
    uint4 u;
    u.x = pack2_bf16(v[0], v[1]); u.y = pack2_bf16(v[2], v[3]);
    u.z = pack2_bf16(v[4], v[5]); u.w = pack2_bf16(v[6], v[7]);
    *reinterpret_cast<uint4*>(p) = u;
}

// acc: 32 consecutive fp32 accumulator columns of one row, starting at column col (col % 32 == 0)
template <int KIND>
__device__ __forceinline__ void epilogue32(const EpiParams& ep, int row, int col, int tok, const uint32_t* acc) {
    using T = __nv_bfloat16;
    float v[32];
    const uint4* bp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(ep.bias) + col);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const uint4 b = __ldg(bp + q);
        const uint32_t w[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[8 * q + 2 * i] = __uint_as_float(acc[8 * q + 2 * i]) + __uint_as_float(w[i] << 16);
            v[8 * q + 2 * i + 1] = __uint_as_float(acc[8 * q + 2 * i + 1]) + __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    if constexpr (KIND == EPI_QKV) {
        const int sec = col / ep.H, c = col - sec * ep.H;
        T* dst;
        if (sec == 0) {
            if (ep.q_head_dim) {             // heads padded (72 -> 80): place every 8-column group inside its head
                T* qrow = reinterpret_cast<T*>(ep.q) + (size_t)row * ep.q_ld;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int c8 = c + 8 * q, hd = c8 / ep.q_head_dim;
                    store8_bf16(qrow + hd * ep.q_head_pad + (c8 - hd * ep.q_head_dim), v + 8 * q);
                }
                return;
            }
            dst = reinterpret_cast<T*>(ep.q) + (size_t)row * ep.q_ld + c;
        } else {
            const int b = tok / ep.N, j = tok - b * ep.N;
            dst = reinterpret_cast<T*>(ep.kv) + (((size_t)b * 2 + (sec - 1)) * ep.N + j) * ep.H + c;
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) store8_bf16(dst + 8 * q, v + 8 * q);
    } else if constexpr (KIND == EPI_RESID) {
        const int b = tok / ep.N;
        const float4* gp = reinterpret_cast<const float4*>(ep.gate + (size_t)b * 6 * ep.H + col);
        float4* rp = reinterpret_cast<float4*>(ep.resid + (size_t)row * ep.H + col);
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const float4 g = __ldg(gp + q);
            float4 r = rp[q];
            r.x = fmaf(g.x, v[4 * q], r.x); r.y = fmaf(g.y, v[4 * q + 1], r.y);
            r.z = fmaf(g.z, v[4 * q + 2], r.z); r.w = fmaf(g.w, v[4 * q + 3], r.w);
            rp[q] = r;
            v[4 * q] = r.x; v[4 * q + 1] = r.y; v[4 * q + 2] = r.z; v[4 * q + 3] = r.w;
        }
        if (ep.y) {
            T* dst = reinterpret_cast<T*>(ep.y) + (size_t)tok * ep.H + col;
#pragma unroll
            for (int q = 0; q < 4; ++q) store8_bf16(dst + 8 * q, v + 8 * q);
        }
    } else {
        T* dst = reinterpret_cast<T*>(ep.out) + (size_t)row * ep.out_ld + col;
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] = gelu_tanh_fast(v[i]);
#pragma unroll
        for (int q = 0; q < 4; ++q) store8_bf16(dst + 8 * q, v + 8 * q);
    }
}

}  // namespace fd
